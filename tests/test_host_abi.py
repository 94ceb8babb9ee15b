"""CPU-side checks of the C-ABI library: it loads without a GPU, exports every
symbol the header declares, and its host planner agrees bit-for-bit with the
oracle's planner on seeded random trajectories."""
import os
import re

import numpy as np
import pytest

from oracle.wd_oracle import SeqState, oracle_plan, oracle_commit
from paper_2601_20332_b200 import binding as wd
from paper_2601_20332_b200 import build as wd_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
INT32_MIN = -(1 << 31)


@pytest.fixture(scope="module", autouse=True)
def built():
    wd_build.build()


def test_library_exports_every_declared_symbol():
    header = open(os.path.join(ROOT, "include", "wd.h")).read()
    declared = set(re.findall(r"^WD_API[^;(]*?\b(wd_\w+)\s*\(", header, flags=re.M))
    assert len(declared) >= 20
    assert declared == set(wd.SIGNATURES), declared ^ set(wd.SIGNATURES)
    L = wd.lib()
    for name in declared:
        assert hasattr(L, name), name
    assert L.wd_version() >= 100
    assert b"null" in L.wd_status_string(wd.WD_ERR_NULL)


def test_sizes_and_dims_validation():
    import ctypes as C
    from paper_2601_20332_b200 import synth
    cfg = synth.get_config("llada8b")
    dims = wd.make_dims(cfg, 1, 512, 512, 256)
    ws = wd.lib().wd_workspace_bytes(C.byref(dims))
    assert ws > 512 * 12288 * 2
    kv = wd.lib().wd_state_bytes(C.byref(dims), 1, 512)
    assert kv >= 2 * 32 * 512 * 4096 * 2            # K and V, all layers, bf16
    bad = wd.make_dims(dict(cfg, Hq=30), 1, 512, 512, 256)          # 30 query heads over 32 kv heads
    assert wd.lib().wd_workspace_bytes(C.byref(bad)) == 0
    assert wd.lib().wd_state_bytes(C.byref(dims), 2, 512) == 0      # batch above max_batch
    out = C.c_void_p()
    assert wd.lib().wd_create(None, None, None, 0, C.byref(out)) == wd.WD_ERR_NULL
    # the K/V cache inside the state memory: K rows + transposed V rows (positions padded to 8), all layers, bf16
    assert wd.lib().wd_kv_bytes(C.byref(dims), 1, 512) == 2 * 32 * 32 * 128 * 512 * 2
    assert wd.lib().wd_kv_bytes(C.byref(dims), 1, 509) == 32 * 32 * 128 * (509 + 512) * 2
    assert wd.lib().wd_kv_bytes(C.byref(dims), 1, 512) < kv and wd.lib().wd_kv_bytes(C.byref(bad), 1, 512) == 0
    assert isinstance(wd.lib().wd_last_error(), bytes)              # no CUDA call has failed in this thread
    assert b"reset" in wd.lib().wd_status_string(wd.WD_ERR_POISONED)


def _walk(seed, S, frac, A, B, R, T, k, prefix, eos_id=None, eos_prob=0.0, refresh_mode=0, stagger=None):
    rng = np.random.default_rng(seed)
    dec = (np.arange(S) < int(S * frac)) if prefix else (rng.random(S) < frac)
    ids0 = np.where(dec, 3, 0)
    if eos_id is not None:
        ids0[: max(1, S // 8)] = np.where(dec[: max(1, S // 8)], eos_id, 0)     # eos ids among the GIVEN tokens
    st = SeqState(ids=ids0.astype(np.int64), decoded=dec, eos_id=eos_id, refresh_mode=refresh_mode, stagger=stagger)
    # mirror of the state kept by the test for the raw planner
    m_dec = dec.astype(np.uint8).copy()
    m_ids = ids0.astype(np.int32).copy()
    m_step = np.full(S, INT32_MIN, np.int32)
    m_t, m_since, m_wex = 0, 0, []
    steps = 0
    while True:
        want = oracle_plan(st, A, B, R, T)
        got = wd.plan_raw(m_dec, m_step, m_t, m_since, m_wex, A, B, R, T, token_ids=m_ids,
                          eos_id=-1 if eos_id is None else eos_id, refresh_mode=refresh_mode, stagger=stagger)
        assert got["done"] == want["done"]
        if want["done"]:
            break
        assert got["refresh"] == want["refresh"]
        for name, oname in (("active", "active"), ("buffer", "buffer"), ("decoded", "decoded"),
                            ("transient", "transient"), ("far_field", "far_field"), ("rows", "rows"),
                            ("vis", "vis"), ("ext_window", "wex")):
            assert got[name] == want[oname], (steps, name)
        assert got["vis_contiguous"] == (want["vis"] == list(range(len(want["vis"]))))
        n = min(k, len(want["active"]))
        pick = sorted(rng.choice(want["active"], size=n, replace=False).tolist())
        toks = [eos_id if (eos_id is not None and rng.random() < eos_prob) else 1 for _ in pick]
        oracle_commit(st, want, pick, toks)
        if got["refresh"]:
            m_wex, m_since = got["ext_window"], 0
        for p, tk in zip(pick, toks):
            m_dec[p] = 1
            m_ids[p] = tk
            m_step[p] = m_t
        m_t += 1
        m_since += 1
        steps += 1
    return steps


@pytest.mark.parametrize("case", [
    (0, 40, 0.3, 4, 6, 3, 1, 1, True), (1, 96, 0.33, 8, 16, 4, 2, 1, True), (2, 64, 0.5, 8, 0, 1, 0, 2, True),
    (3, 70, 0.4, 3, 5, 5, 9, 2, False), (4, 50, 0.1, 6, 2, 16, 3, 3, False), (5, 30, 0.0, 30, 0, 1, 0, 4, True),
    (6, 45, 0.3, 2, 1, 8, 2, 1, False), (7, 300, 0.3, 32, 64, 8, 2, 1, True), (8, 200, 0.5, 64, 128, 8, 2, 2, True),
])
def test_host_planner_matches_oracle_bit_exact(case):
    assert _walk(*case) > 0


@pytest.mark.parametrize("case", [
    (10, 60, 0.3, 4, 6, 3, 1, 1, True), (11, 96, 0.3, 8, 16, 4, 2, 2, True), (12, 70, 0.4, 3, 5, 5, 9, 2, False),
    (13, 200, 0.2, 16, 48, 8, 2, 1, True),
])
def test_host_planner_matches_oracle_with_adaptive_termination(case):
    full = _walk(*case)
    short = _walk(*case, eos_id=7, eos_prob=0.15)
    assert 0 < short < full                       # an eos token ended generation early


@pytest.mark.parametrize("case", [
    (20, 96, 0.33, 8, 16, 4, 2, 1, True), (21, 70, 0.4, 3, 5, 5, 9, 2, False), (22, 300, 0.3, 32, 64, 8, 2, 1, True),
    (23, 64, 0.5, 8, 0, 1, 0, 2, True), (24, 50, 0.1, 6, 2, 16, 3, 3, False),
])
def test_host_planner_matches_oracle_with_window_only_refresh(case):
    """The variant outside the paper (WD_REFRESH_WINDOW), with and without adaptive termination."""
    assert _walk(*case, refresh_mode=1) > 0
    assert _walk(*case, eos_id=7, eos_prob=0.1, refresh_mode=1) > 0


@pytest.mark.parametrize("case", [
    (30, 96, 0.33, 8, 16, 4, 2, 1, True), (31, 70, 0.4, 3, 5, 5, 9, 2, False), (32, 300, 0.3, 32, 64, 8, 2, 1, True),
    (33, 64, 0.5, 8, 0, 1, 0, 2, True), (34, 120, 0.2, 6, 10, 16, 3, 1, True),
])
def test_host_planner_matches_oracle_with_staggered_refresh(case):
    """The batch variant outside the paper (wd_state_set_stagger): sequence i of n, for several i and n,
    with the paper's refresh and with the window-only one."""
    for stagger in ((0, 4), (1, 4), (3, 4), (5, 8), (7, 8), (2, 3)):
        assert _walk(*case, stagger=stagger) > 0
    assert _walk(*case, stagger=(3, 8), refresh_mode=1) > 0
    assert _walk(*case, stagger=(1, 2), eos_id=7, eos_prob=0.1) > 0


def test_plan_raw_errors():
    dec = np.zeros(8, np.uint8)
    ds = np.full(8, INT32_MIN, np.int32)
    for bad in ((0, 1, 1, 0), (1, -1, 1, 0), (1, 1, 0, 0), (1, 1, 1, -1)):
        with pytest.raises(wd.WdError) as e:
            wd.plan_raw(dec, ds, 0, 0, [], *bad)
        assert e.value.status == wd.WD_ERR_BAD_PARAM
    with pytest.raises(wd.WdError) as e:
        wd.plan_raw(dec, ds, 1, 1, [9], 2, 2, 2, 1)               # window index outside the sequence
    assert e.value.status == wd.WD_ERR_BAD_PARAM
    with pytest.raises(wd.WdError) as e:
        wd.plan_raw(dec, ds, 0, 0, [], 2, 2, 2, 1, refresh_mode=2)
    assert e.value.status == wd.WD_ERR_BAD_PARAM
    with pytest.raises(wd.WdError) as e:
        wd.plan_raw(dec, ds, 0, 0, [], 2, 2, 2, 1, stagger=(4, 4))      # sequence index outside the batch
    assert e.value.status == wd.WD_ERR_BAD_PARAM
    # capacity too small for the lists
    import ctypes as C
    s, bufs = wd._index_sets(8)
    s.capacity = 2
    r = wd.lib().wd_plan_raw(dec.ctypes.data_as(wd.u8p), ds.ctypes.data_as(wd.i32p), None, -1, 8, 0, 0, None, 0, 4, 2,
                             2, 1, 0, 0, 0, C.byref(s))
    assert r == wd.WD_ERR_CAPACITY
    # huge window parameters must not overflow
    p = wd.plan_raw(dec, ds, 0, 0, [], 2**31 - 1, 2**31 - 1, 1, 0)
    assert p["active"] == list(range(8)) and p["far_field"] == []
