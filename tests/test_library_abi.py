"""CPU checks of the C-ABI library: it builds, loads and exports every symbol the header declares, and the
host-side config validation answers without touching a GPU."""
import ctypes as C
import os
import re

from paper_2607_13095_b200 import binding as hb

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "hswa.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(hswa_[a-z_]+)\s*\(", text)))


def test_exports_match_header():
    lib = hb.load()
    names = declared_symbols()
    assert set(names) == set(hb.EXPORTS), (names, hb.EXPORTS)
    for n in names:
        assert getattr(lib, n) is not None


def test_status_strings():
    for s in range(7):
        assert hb.status_string(s) not in ("", "unknown status")
    assert hb.status_string(99) == "unknown status"


def _create(**kw):
    base = dict(num_q_heads=64, num_kv_heads=8, head_dim=128, page_size=64, window=128, ring_pages=0,
                sm_scale=0.0, out_dtype=0)
    base.update(kw)
    cfg = hb.hswa_config(**base)
    h = C.c_void_p()
    st = hb.load().hswa_create(C.byref(cfg), C.byref(h))
    if st == hb.HSWA_OK:
        hb.load().hswa_destroy(h)
    return st


def test_create_rejects_bad_configs_on_host():
    assert _create(num_kv_heads=0) == hb.HSWA_ERR_INVALID_ARG
    assert _create(num_q_heads=63) == hb.HSWA_ERR_INVALID_ARG
    assert _create(window=0) == hb.HSWA_ERR_INVALID_ARG
    assert _create(out_dtype=7) == hb.HSWA_ERR_INVALID_ARG
    assert _create(sm_scale=-1.0) == hb.HSWA_ERR_INVALID_ARG
    assert _create(ring_pages=2) == hb.HSWA_ERR_INVALID_ARG          # 2 * 64 < W + 1
    assert _create(head_dim=96) == hb.HSWA_ERR_UNSUPPORTED
    assert _create(page_size=48) == hb.HSWA_ERR_UNSUPPORTED
    assert _create(num_q_heads=64, num_kv_heads=4) == hb.HSWA_ERR_UNSUPPORTED  # G = 16
    assert hb.load().hswa_create(None, None) == hb.HSWA_ERR_INVALID_ARG


def test_null_handle_paths():
    lib = hb.load()
    assert lib.hswa_workspace_bytes(None, 4, 4, 100) == 0
    assert lib.hswa_step_advance(None, 1, None, None, None, None) == hb.HSWA_ERR_INVALID_ARG
    lib.hswa_destroy(None)


def test_window_safe_len_host():
    import numpy as np
    from oracle import hswa_oracle as orc
    rng = np.random.default_rng(1)
    for W in (1, 2, 4, 128):
        for _ in range(200):
            n = int(rng.integers(1, 400))
            valid = (rng.random(n) < 0.9).astype(np.uint8)
            valid[: int(rng.integers(0, n))] = rng.integers(0, 2)
            m = int(rng.integers(0, n + 1))
            assert hb.hswa_window_safe_len(m, W, valid) == orc.window_safe_len(m, W, valid)


def test_prefix_hit_len_is_host_arithmetic_and_matches_oracle():
    import numpy as np
    from oracle import hswa_oracle as orc
    rng = np.random.default_rng(4)
    for W in (1, 2, 4, 128):
        for _ in range(80):
            n = int(rng.integers(1, 400))
            swa = (rng.random(n) < 0.9).astype(np.uint8)
            swa[: int(rng.integers(0, n))] = 0
            full = np.ones(n, np.uint8)
            if rng.random() < 0.5:
                full[int(rng.integers(0, n))] = 0
            m = int(rng.integers(0, n + 1))
            assert hb.hswa_prefix_hit_len(m, W, full, swa) == orc.prefix_hit_len(m, W, full, swa)
    assert hb.load().hswa_prefix_hit_len(10, 4, None, None) == 0
