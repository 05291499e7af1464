"""Plain state model of a cached prefix whose tree nodes carry dual indices (paper Sec. 3.1.3, item 3 and the
window-4 figure): each node covers a run of tokens of one cached sequence and records, per token,

  - the Full Attention segment index: which (page, slot) of the Full pool holds the token's KV, or nothing once
    the whole segment has been evicted;
  - the SWA segment mapping: which (page, slot) of the SWA pool holds it, or nothing once its SWA part has been
    released (out-of-window release, item 2) or evicted on its own.

TEST INFRASTRUCTURE ONLY (like the rest of oracle/): the product never imports this module.  It holds
bookkeeping, no attention arithmetic: the usable hit length comes from hswa_oracle.prefix_hit_len over the two
per-token status vectors a path of nodes yields.

Nodes change by splitting and merging while requests come and go; neither operation may change any token's status.
Eviction is managed separately per index: the SWA part of a node can go while its Full part stays (the prefix is
then still reusable by Full layers, and by SWA layers as long as the tail the window needs lives in later nodes),
or the whole segment goes, which ends the usable prefix at the node's first token.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Optional, Tuple

import numpy as np

Loc = Optional[Tuple[int, int]]  # (page, slot) or None


@dataclass
class Node:
    start: int                       # position of the node's first token in the cached sequence
    full_loc: List[Loc]              # per token: location in the Full pool, None = evicted
    swa_loc: List[Loc]               # per token: location in the SWA pool, None = released / evicted

    @property
    def length(self) -> int:
        return len(self.full_loc)

    def full_status(self) -> np.ndarray:
        return np.array([loc is not None for loc in self.full_loc], dtype=np.uint8)

    def swa_status(self) -> np.ndarray:
        return np.array([loc is not None for loc in self.swa_loc], dtype=np.uint8)


@dataclass
class Path:
    """Root-to-leaf chain of nodes: one cached token sequence."""
    nodes: List[Node] = field(default_factory=list)

    @property
    def length(self) -> int:
        return sum(n.length for n in self.nodes)

    def check(self) -> None:
        pos = 0
        for n in self.nodes:
            assert n.start == pos and len(n.swa_loc) == len(n.full_loc)
            pos += n.length

    def status(self) -> Tuple[np.ndarray, np.ndarray]:
        """(full_valid, swa_valid) per token of the whole path, in logical order."""
        if not self.nodes:
            return np.zeros(0, np.uint8), np.zeros(0, np.uint8)
        return (np.concatenate([n.full_status() for n in self.nodes]),
                np.concatenate([n.swa_status() for n in self.nodes]))

    # ---- structure changes: no token's status may change ----
    def split(self, index: int, at: int) -> None:
        """Split node `index` after its first `at` tokens (a request diverges in the middle of a node)."""
        n = self.nodes[index]
        assert 0 < at < n.length
        a = Node(n.start, n.full_loc[:at], n.swa_loc[:at])
        b = Node(n.start + at, n.full_loc[at:], n.swa_loc[at:])
        self.nodes[index:index + 1] = [a, b]

    def merge(self, index: int) -> None:
        """Merge node `index` with its successor (the only child of a node is folded back into it)."""
        a, b = self.nodes[index], self.nodes[index + 1]
        self.nodes[index:index + 2] = [Node(a.start, a.full_loc + b.full_loc, a.swa_loc + b.swa_loc)]

    # ---- eviction, managed separately for the two indices ----
    def evict_swa(self, index: int) -> List[Tuple[int, int]]:
        """Drop the SWA part of a node, keep its Full part.  Returns the freed SWA locations."""
        n = self.nodes[index]
        freed = [loc for loc in n.swa_loc if loc is not None]
        n.swa_loc = [None] * n.length
        return freed

    def evict_segment(self, index: int) -> Tuple[List[Tuple[int, int]], List[Tuple[int, int]]]:
        """Drop a node entirely (Full and SWA parts).  Returns (freed Full locations, freed SWA locations)."""
        n = self.nodes[index]
        freed_full = [loc for loc in n.full_loc if loc is not None]
        freed_swa = self.evict_swa(index)
        n.full_loc = [None] * n.length
        return freed_full, freed_swa

    def release_out_of_window(self, length: int, window: int) -> List[Tuple[int, int]]:
        """Item 2 on a path: release the SWA part of every token the next token (at position `length`) cannot see,
        i.e. positions below length - (window - 1).  Returns the freed SWA locations."""
        cut = max(0, length - (window - 1))
        freed = []
        for n in self.nodes:
            for i in range(n.length):
                if n.start + i < cut and n.swa_loc[i] is not None:
                    freed.append(n.swa_loc[i])
                    n.swa_loc[i] = None
        return freed


def path_from_request(length: int, cuts: List[int], full_loc_of, swa_loc_of) -> Path:
    """A path for a cached sequence of `length` tokens, cut into nodes at the given positions; full_loc_of(p) and
    swa_loc_of(p) give each position's location (or None)."""
    edges = [0] + sorted(c for c in cuts if 0 < c < length) + [length]
    nodes = []
    for a, b in zip(edges[:-1], edges[1:]):
        nodes.append(Node(a, [full_loc_of(p) for p in range(a, b)], [swa_loc_of(p) for p in range(a, b)]))
    p = Path(nodes)
    p.check()
    return p
