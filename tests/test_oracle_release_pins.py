"""CPU pins of the oracle's out-of-window release bookkeeping and dual-index matching (paper Sec. 3.1.3 items 2
and 3, and the window-4 figure).  The closed-form state (one boundary per request) is checked against a brute-force
replay that tags every physical ring slot with the position it holds; the hit length against a replay of the reads
the continuing request would issue."""
import numpy as np
import pytest

from oracle import hswa_oracle as orc
from oracle import prefix_nodes as pn
from paper_2607_13095_b200 import workloads as wl
from helpers import oracle_config

D4 = wl.Dims(num_q_heads=2, num_kv_heads=1, head_dim=8, page_size=2, window=4)      # the figure's window; C = 6
D8 = wl.Dims(num_q_heads=4, num_kv_heads=2, head_dim=8, page_size=4, window=8)      # C = 12
DB = wl.BIG                                                                          # W = 128, C = 192


class TaggedRing:
    """Brute force: every slot remembers which position it holds (-1: nothing valid)."""

    def __init__(self, C, W):
        self.C, self.W, self.tags, self.len = C, W, [-1] * C, 0

    def append(self, n):
        for _ in range(n):
            self.tags[self.len % self.C] = self.len   # later writes win
            self.len += 1

    def release(self):
        cut = self.len - (self.W - 1)                  # the next token reads [len - (W - 1), len)
        self.tags = [t if t >= cut else -1 for t in self.tags]

    def mask(self):
        m = np.zeros(self.len, np.uint8)
        for t in self.tags:
            if t >= 0:
                m[t] = 1
        return m


@pytest.mark.parametrize("dims", [D4, D8, DB])
def test_release_state_matches_tagged_ring_replay(dims):
    cfg = oracle_config(dims)
    W, C = dims.window, dims.ring_slots
    rng = np.random.default_rng(5)
    for trial in range(12):
        every_n = int(rng.choice([1, 2, 3, 7, C - W + 1, C, 2 * C]))
        ring = TaggedRing(C, W)
        ctx = np.zeros(1, np.int32)
        valid_from = np.zeros(1, np.int32)
        chunks = [int(x) for x in rng.choice([1, 2, W - 1, W, W + 1, C - 1, C, C + 1, 3 * C + 1], size=int(rng.integers(1, 4)))]
        events = [("chunk", n) for n in chunks] + [("decode", 1)] * int(rng.integers(0, 3 * C)) + [("end", 0)]
        decoded = 0
        for kind, n in events:
            if kind != "end":
                ring.append(n)
                ctx[0] += n
            if kind == "decode":
                decoded += 1
            due = orc.release_due({"chunk": orc.RELEASE_CHUNK_END, "decode": orc.RELEASE_DECODE_TOKEN,
                                   "end": orc.RELEASE_REQUEST_END}[kind], decoded, every_n)
            assert due == (kind != "decode" or decoded % every_n == 0)
            if due:
                ring.release()
            orc.swa_release(cfg, ctx, np.array([due], np.uint8), valid_from)
            got = orc.swa_valid_mask(int(ctx[0]), int(valid_from[0]))
            assert np.array_equal(got, ring.mask()), (trial, kind, int(ctx[0]))
            # pool use stays at window magnitude (item 2): W - 1 right after a release, at most N - 1 more between
            # two decode releases, never above the ring
            n_valid = int(got.sum())
            assert n_valid <= C
            if due:
                assert n_valid == min(int(ctx[0]), W - 1)
            elif kind == "decode":
                assert n_valid <= min(C, W - 1 + every_n - 1 + 0)
        assert int(valid_from[0]) == max(0, int(ctx[0]) - (W - 1))   # request end always releases


def test_release_literals_window_4():
    cfg = oracle_config(D4)   # W = 4, C = 6
    ctx = np.array([5, 12, 12, 2], np.int32)
    vf = np.array([0, 0, 7, 0], np.int32)
    orc.swa_release(cfg, ctx, np.array([0, 0, 1, 1], np.uint8), vf)
    # request 0: nothing released, the ring of 6 slots still holds all 5 positions; request 1: no release but the
    # ring overwrote everything below 12 - 6; request 2: release keeps the 3 positions the next token reads;
    # request 3: shorter than the window, everything stays
    assert vf.tolist() == [0, 6, 9, 0]
    orc.swa_release(cfg, ctx, None, vf)                    # NULL flags: every request releases
    assert vf.tolist() == [2, 9, 9, 0]
    orc.swa_release(cfg, np.array([5, 12, 12, 2], np.int32), np.zeros(4, np.uint8), vf)
    assert vf.tolist() == [2, 9, 9, 0]                     # the boundary never moves back
    assert orc.swa_valid_mask(12, 9).tolist() == [0] * 9 + [1] * 3
    assert not orc.release_due(orc.RELEASE_DECODE_TOKEN, 5, 3) and orc.release_due(orc.RELEASE_DECODE_TOKEN, 6, 3)
    assert not orc.release_due(orc.RELEASE_DECODE_TOKEN, 6, 0)
    assert orc.release_due(orc.RELEASE_CHUNK_END) and orc.release_due(orc.RELEASE_REQUEST_END)


def replay_hit_len(m, W, full_valid, swa_valid):
    """Brute force: the continuing request's next token sits at position L; a Full layer reads 0 .. L - 1, an SWA
    layer reads the W - 1 positions before L.  L is usable iff no read touches an invalid entry."""
    best = 0
    for L in range(m + 1):
        reads_full = set(range(L))
        reads_swa = set(range(max(0, L - (W - 1)), L))
        if all(full_valid[i] for i in reads_full) and all(swa_valid[i] for i in reads_swa):
            best = L
    return best


def test_prefix_hit_len_matches_read_replay_and_window_safe_len():
    rng = np.random.default_rng(6)
    for W in (1, 2, 4, 8, 128):
        for _ in range(60):
            n = int(rng.integers(1, 260))
            swa = (rng.random(n) < rng.choice([0.5, 0.95])).astype(np.uint8)
            if rng.random() < 0.6:
                swa[: int(rng.integers(0, n))] = 0          # typical: only a tail survives
            full = np.ones(n, np.uint8)
            if rng.random() < 0.5:
                full[int(rng.integers(0, n)):] = rng.integers(0, 2, 1)[0]   # a segment evicted entirely
            m = int(rng.integers(0, n + 1))
            assert orc.prefix_hit_len(m, W, full, swa) == replay_hit_len(m, W, full, swa)
            assert orc.prefix_hit_len(m, W, np.ones(n, np.uint8), swa) == orc.window_safe_len(m, W, swa)


def test_window_4_figure_scenario_on_dual_index_nodes():
    """The figure's setting: window 4, nodes with per-token Full and SWA status.  A 12-token sequence cached as
    nodes A = [0, 5), B = [5, 9), C = [9, 12); locations are (page, slot) with 2 slots per page."""
    W = 4
    full_loc = lambda p: (100 + p // 2, p % 2)
    swa_loc = lambda p: (7 + (p % 6) // 2, p % 2)           # a ring of 6 slots: position p sits in slot p mod 6
    path = pn.path_from_request(12, [5, 9], full_loc, swa_loc)
    assert [n.length for n in path.nodes] == [5, 4, 3]
    # while the request was live the ring kept the last 6 positions only
    for n in path.nodes:
        n.swa_loc = [loc if n.start + i >= 6 else None for i, loc in enumerate(n.swa_loc)]
    full, swa = path.status()
    assert full.tolist() == [1] * 12 and swa.tolist() == [0] * 6 + [1] * 6
    hit = lambda m: orc.prefix_hit_len(m, W, *path.status())
    assert [hit(m) for m in (12, 11, 10, 9, 8, 5)] == [12, 11, 10, 9, 0, 0]   # 8 would need position 5's SWA slot
    # request end: out-of-window release keeps the W - 1 = 3 positions the next token reads; the freed slots are B's
    freed = path.release_out_of_window(12, W)
    assert freed == [swa_loc(6), swa_loc(7), swa_loc(8)]
    assert path.status()[1].tolist() == [0] * 9 + [1] * 3
    assert [hit(m) for m in (12, 11, 10)] == [12, 0, 0]      # only the complete sequence is still window-safe
    assert orc.swa_valid_mask(12, 9).tolist() == path.status()[1].tolist()   # same state as the per-request boundary
    # structure changes leave every token's status alone
    before = [x.copy() for x in path.status()]
    path.split(0, 2)
    path.split(3, 1)
    path.check()
    assert [n.length for n in path.nodes] == [2, 3, 4, 1, 2]
    path.merge(1)
    path.check()
    assert all(np.array_equal(a, b) for a, b in zip(before, path.status())) and hit(12) == 12
    # separate eviction: dropping the SWA part of an old node changes nothing for a hit whose tail is intact ...
    assert path.evict_swa(0) == [] and hit(12) == 12
    # ... dropping the SWA part of the tail node makes every hit a miss on SWA layers, though Full KV is all there
    tail = len(path.nodes) - 1
    assert len(path.evict_swa(tail)) == 2 and hit(12) == 0
    assert orc.prefix_hit_len(12, 1, *path.status()) == 12    # (a window of 1 needs no cached SWA key)
    # evicting a whole middle segment ends the usable prefix at its first token, whatever the SWA status
    path2 = pn.path_from_request(12, [5, 9], full_loc, swa_loc)
    freed_full, freed_swa = path2.evict_segment(1)
    assert freed_full == [full_loc(p) for p in range(5, 9)] and freed_swa == [swa_loc(p) for p in range(5, 9)]
    assert orc.prefix_hit_len(12, W, *path2.status()) == 5 and orc.prefix_hit_len(4, W, *path2.status()) == 4
