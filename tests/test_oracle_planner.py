"""Pins for the oracle's planner: the set identities of Section 4.2, the phase
structure of Section 4.3 and a hand-traced trajectory."""
import os

import numpy as np
import pytest

from oracle.wd_oracle import SeqState, oracle_plan, oracle_commit

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "planner_trace.txt")


def _state(P, G, mask_id=99):
    ids = np.array([1] * P + [mask_id] * G)
    dec = np.array([True] * P + [False] * G)
    return SeqState(ids=ids, decoded=dec)


def _parse(field):
    field = field.strip()
    return [] if field == "-" else [int(v) for v in field.split()]


def test_hand_traced_trajectory():
    st = _state(4, 10)
    A, B, R, T = 3, 3, 3, 1
    rows = [l for l in open(GOLDEN).read().splitlines() if l and not l.startswith("#")]
    assert len(rows) == 4
    for line in rows:
        f = [c.strip() for c in line.split("|")]
        pl = oracle_plan(st, A, B, R, T)
        assert st.t == int(f[0])
        assert pl["refresh"] == (f[1] == "refresh")
        for name, col in (("wex", 2), ("active", 3), ("buffer", 4), ("in_phase_decoded", 5),
                          ("transient", 6), ("far_field", 7), ("vis", 8), ("rows", 9)):
            assert pl[name] == _parse(f[col]), (f[0], name)
        oracle_commit(st, pl, [int(f[10])], [7])


def _random_walk(seed, S, frac, A, B, R, T, k, prefix):
    rng = np.random.default_rng(seed)
    if prefix:
        P = int(S * frac)
        dec = np.arange(S) < P
    else:
        dec = rng.random(S) < frac
    st = SeqState(ids=np.zeros(S, dtype=np.int64), decoded=dec)
    trace = []
    while True:
        pl = oracle_plan(st, A, B, R, T)
        if pl["done"]:
            break
        trace.append((st.t, st.since, pl, st.decoded.copy()))
        n = min(k, len(pl["active"]))
        pick = list(rng.choice(pl["active"], size=n, replace=False))
        oracle_commit(st, pl, pick, [5] * n)
    return st, trace


CASES = [  # seed, S, frac, A, B, R, T, k, prefix
    (0, 40, 0.3, 4, 6, 3, 1, 1, True),
    (1, 64, 0.25, 8, 16, 4, 2, 1, True),
    (2, 64, 0.5, 8, 0, 1, 0, 2, True),
    (3, 50, 0.4, 3, 5, 5, 9, 2, False),
    (4, 50, 0.1, 6, 2, 16, 3, 3, False),
    (5, 30, 0.0, 30, 0, 1, 0, 4, True),
    (6, 45, 0.3, 2, 1, 8, 2, 1, False),     # k*R > A+B: window exhausted mid-phase
]


@pytest.mark.parametrize("case", CASES)
def test_set_invariants(case):
    seed, S, frac, A, B, R, T, k, prefix = case
    st, trace = _random_walk(*case)
    assert st.decoded.all()
    prev_min_act, prev_max_wex, prev_vis, prev_refresh_t = -1, -1, None, None
    for t, since, pl, decoded in trace:
        U = set(np.flatnonzero(~decoded).tolist())
        D = set(np.flatnonzero(decoded).tolist())
        act, buf, far = set(pl["active"]), set(pl["buffer"]), set(pl["far_field"])
        # partition of the undecoded region (Section 4.2)
        assert act | buf | far == U
        assert not (act & buf) and not (act & far) and not (buf & far)
        assert len(act) + len(buf) + len(far) == len(U)
        assert set(pl["decoded"]) == D and D | U == set(range(S))
        wex = set(pl["wex"])
        # B = W_ex \ (A u D_p)
        assert buf == wex - (act | set(pl["in_phase_decoded"]))
        assert act <= wex and far == U - wex
        assert set(pl["transient"]) <= set(pl["in_phase_decoded"]) <= D
        # the internal window is the front of the undecoded prefix and keeps its size
        assert min(U) in act
        assert len(act) == min(A, len(wex & U))
        assert max(act) < min(buf | far | {S})
        # lists are ascending
        for name in ("active", "buffer", "far_field", "decoded", "vis", "rows", "transient"):
            assert pl[name] == sorted(pl[name])
        # window slides monotonically to the right
        # (the right edge is that of the visible set: near the end the external
        #  window is "whatever is left", whose maximum may lie left of an earlier one)
        assert min(act) >= prev_min_act and max(pl["vis"]) >= prev_max_wex
        prev_min_act, prev_max_wex = min(act), max(pl["vis"])
        assert len(pl["transient"]) <= k * min(T, since)
        if pl["refresh"]:
            assert pl["rows"] == pl["vis"] and not pl["in_phase_decoded"]
            assert len(wex) == min(A + B, len(U))
            prev_refresh_t = t
        else:
            assert set(pl["rows"]) == act | set(pl["transient"])
            assert pl["vis"] == prev_vis            # |vis| constant within a phase
            assert t - prev_refresh_t < R           # one refresh then at most R-1 normal steps
        prev_vis = pl["vis"]
        assert set(pl["vis"]) == D | (wex & U)
        # contiguity: with a decoded prefix the visible set is a range [0, hi]
        if prefix:
            assert pl["vis"] == list(range(len(pl["vis"])))


def test_phase_is_one_refresh_then_normal_steps():
    st, trace = _random_walk(7, 200, 0.2, 8, 24, 4, 2, 1, True)
    kinds = [pl["refresh"] for _, _, pl, _ in trace]
    # k*R <= A+B so no forced refresh: the pattern is strictly periodic
    assert kinds[:12] == [True, False, False, False] * 3


def test_paper_transient_mode():
    """Section 5.3: in the authors' implementation tokens decoded inside the
    window are recomputed until the next refresh, i.e. T >= R-1 makes the
    transient set equal the in-phase decoded set."""
    _, trace = _random_walk(8, 120, 0.25, 8, 24, 6, 5, 2, True)
    seen = 0
    for _, _, pl, _ in trace:
        assert pl["transient"] == pl["in_phase_decoded"]
        seen += len(pl["transient"])
    assert seen > 0


def test_transient_ages_out_and_resets_at_refresh():
    st = _state(2, 20)
    A, B, R, T = 4, 4, 5, 2
    ages = []
    for step in range(5):
        pl = oracle_plan(st, A, B, R, T)
        ages.append(sorted(st.t - int(st.dec_step[i]) for i in pl["transient"]))
        oracle_commit(st, pl, [pl["active"][0]], [3])
    assert ages == [[], [1], [1, 2], [1, 2], [1, 2]]
    pl = oracle_plan(st, A, B, R, T)
    assert pl["refresh"] and pl["transient"] == []


def test_forced_refresh_when_window_exhausted():
    st = _state(1, 12)
    A, B, R, T = 2, 0, 8, 1
    kinds = []
    for _ in range(4):
        pl = oracle_plan(st, A, B, R, T)
        kinds.append(pl["refresh"])
        oracle_commit(st, pl, pl["active"], [3] * len(pl["active"]))
    assert kinds == [True, True, True, True]


def test_plan_is_pure_and_done():
    st = _state(3, 2)
    before = (st.ids.copy(), st.decoded.copy(), st.t, st.since, list(st.wex))
    oracle_plan(st, 2, 2, 2, 1)
    assert (st.ids == before[0]).all() and (st.decoded == before[1]).all()
    assert (st.t, st.since, st.wex) == (before[2], before[3], before[4])
    done = SeqState(ids=np.zeros(3), decoded=np.ones(3, dtype=bool))
    assert oracle_plan(done, 2, 2, 2, 1)["done"]
    with pytest.raises(ValueError):
        oracle_plan(st, 0, 2, 2, 1)


def _run_with_eos(eos_picks, eos_id=42, P=3, G=30, A=4, B=4, R=3, T=1, prompt_has_eos=False):
    """Decode the first active position every step; positions in eos_picks get the eos id."""
    ids = np.array(([eos_id] if prompt_has_eos else [1]) + [1] * (P - 1) + [99] * G)
    st = SeqState(ids=ids, decoded=np.arange(P + G) < P, eos_id=eos_id)
    plans = []
    while True:
        pl = oracle_plan(st, A, B, R, T)
        if pl["done"]:
            break
        plans.append(pl)
        pos = pl["active"][0]
        oracle_commit(st, pl, [pos], [eos_id if pos in eos_picks else 5])
    return st, plans


def test_adaptive_termination_stops_the_window():
    """Section 4.2, adaptive termination: after an eos token is generated the internal window
    stops advancing, later positions stay far-field, and generation ends early."""
    st, plans = _run_with_eos({12})
    # positions 3..12 are decoded one by one, then everything after 12 is ignored for good
    assert len(plans) == 10
    assert st.decoded[:13].all() and not st.decoded[13:].any()
    for pl in plans:
        assert max(pl["active"] + pl["buffer"]) <= 12 + 8          # window never ran ahead of A + B
    # once the eos is in, a sequence with undecoded tokens only after it is done
    assert oracle_plan(st, 4, 4, 3, 1)["done"]
    # without an eos the same schedule runs through all 30 masks
    st2, plans2 = _run_with_eos(set())
    assert len(plans2) == 30 and st2.decoded.all()
    # and the plans before the eos appears are identical
    for a, b in zip(plans[:9], plans2[:9]):
        assert a == b


def test_adaptive_termination_ignores_given_eos_and_takes_the_first_in_position_order():
    st, plans = _run_with_eos(set(), prompt_has_eos=True)
    assert len(plans) == 30                                   # an eos id inside the prompt does not count
    # out-of-order decoding: eos generated at 20 first, then another at 10 moves the limit left
    ids = np.array([1] * 2 + [99] * 30)
    st = SeqState(ids=ids, decoded=np.arange(32) < 2, eos_id=42)
    pl = oracle_plan(st, 24, 0, 1, 0)
    oracle_commit(st, pl, [20], [42])
    pl = oracle_plan(st, 24, 0, 1, 0)
    assert max(pl["active"]) == 19 and set(range(21, 32)) <= set(pl["far_field"])
    oracle_commit(st, pl, [10], [42])
    pl = oracle_plan(st, 24, 0, 1, 0)
    assert pl["active"] == list(range(2, 10))
    assert set(pl["far_field"]) == set(range(11, 20)) | set(range(21, 32))
    assert 20 in pl["vis"] and 10 in pl["vis"]                 # decoded tokens stay visible context


# ---------------------------------------------------------------------------
# window-only refresh (a variant outside the paper, flagged by SeqState.refresh_mode)
# ---------------------------------------------------------------------------

def _walk(mode, S=96, P=20, A=6, B=10, R=4, T=2, k=2, steps=30, seed=3):
    rng = np.random.default_rng(seed)
    ids = np.where(np.arange(S) < P, 5, 99)
    st = SeqState(ids=ids, decoded=np.arange(S) < P, refresh_mode=mode)
    trace = []
    for _ in range(steps):
        pl = oracle_plan(st, A, B, R, T)
        if pl["done"]:
            break
        trace.append(pl)
        chosen = sorted(rng.choice(pl["active"], size=min(k, len(pl["active"])), replace=False).tolist())
        oracle_commit(st, pl, chosen, [7] * len(chosen))
    return trace


def test_window_refresh_rows_are_the_new_window_plus_the_previous_phase():
    full, win = _walk(0), _walk(1)
    assert len(full) == len(win) and sum(p["refresh"] for p in win) >= 4
    for i, (f, w) in enumerate(zip(full, win)):
        # the variant changes which rows a refresh computes and nothing else
        for key in ("refresh", "wex", "active", "buffer", "transient", "far_field", "decoded", "vis"):
            assert f[key] == w[key]
        assert f["rows"] == (f["vis"] if f["refresh"] else sorted(set(f["active"]) | set(f["transient"])))
        if not w["refresh"]:
            assert w["rows"] == f["rows"]
        elif i == 0:
            assert w["rows"] == w["vis"]                                    # nothing cached yet: everything
        else:
            # decoded during the phase that just ended = difference of the decoded sets at the two refreshes
            j = max(q for q in range(i) if win[q]["refresh"])
            decoded_in_prev_phase = set(w["decoded"]) - set(win[j]["decoded"])
            assert decoded_in_prev_phase
            assert w["rows"] == sorted(set(w["wex"]) | decoded_in_prev_phase)
            assert set(w["rows"]) < set(f["rows"])                          # strictly fewer rows than the paper's refresh


def test_window_refresh_first_step_is_a_full_refresh():
    w = _walk(1, steps=1)[0]
    assert w["refresh"] and w["rows"] == w["vis"]


# ---------------------------------------------------------------------------
# staggered refresh steps across a batch (a variant outside the paper, flagged by SeqState.stagger)
# ---------------------------------------------------------------------------

def _walk_batch(n, R, stagger, S=200, P=20, A=4, B=12, T=2, k=1, steps=40, seed=5):
    rng = np.random.default_rng(seed)
    ids = np.where(np.arange(S) < P, 5, 99)
    sts = [SeqState(ids=ids, decoded=np.arange(S) < P, stagger=(i, n) if stagger else None) for i in range(n)]
    traces = [[] for _ in range(n)]
    for _ in range(steps):
        for i, st in enumerate(sts):
            pl = oracle_plan(st, A, B, R, T)
            assert not pl["done"]
            traces[i].append(pl)
            chosen = sorted(rng.choice(pl["active"], size=min(k, len(pl["active"])), replace=False).tolist())
            oracle_commit(st, pl, chosen, [7] * len(chosen))
    return traces


@pytest.mark.parametrize("n,R", [(8, 4), (4, 8), (3, 5), (16, 4), (2, 2), (5, 1)])
def test_staggered_refresh_spreads_the_refresh_steps_of_a_batch(n, R):
    tr = _walk_batch(n, R, True)
    base = _walk_batch(n, R, False)
    for i in range(n):
        o = (i * R) // n
        got = [t for t, pl in enumerate(tr[i]) if pl["refresh"]]
        # step 0 (nothing cached), then step o if 0 < o < R, then every R steps: each phase is a phase of Section 4.3
        want = sorted({0} | {t for t in range(40) if t >= o and (t - o) % R == 0})
        assert got == want, (i, got)
        gaps = np.diff(got)
        assert (gaps[1:] == R).all() and gaps[0] in (R, o)
        # without the variant every sequence refreshes on the same steps
        assert [t for t, pl in enumerate(base[i]) if pl["refresh"]] == list(range(0, 40, R))
    # at most ceil(n / R) sequences refresh in any step after the first
    per_step = [sum(tr[i][t]["refresh"] for i in range(n)) for t in range(40)]
    assert per_step[0] == n and max(per_step[R:]) <= -(-n // R) and min(per_step[R:]) >= n // R
    # sequence 0 is never shifted: identical to the unstaggered run
    assert [pl for pl in tr[0]] == [pl for pl in base[0]]


def test_staggered_refresh_keeps_the_set_identities():
    """Only where the phases begin changes: the partition of Section 4.2 holds at every step."""
    for pls in _walk_batch(4, 8, True, steps=60):
        for pl in pls:
            act, buf, far, dec = set(pl["active"]), set(pl["buffer"]), set(pl["far_field"]), set(pl["decoded"])
            assert not (act & buf) and not (act & far) and not (buf & far) and not ((act | buf | far) & dec)
            assert len(act | buf | far | dec) == 200
            assert set(pl["transient"]) <= set(pl["in_phase_decoded"]) <= dec
            assert set(pl["vis"]) == dec | act | buf
            assert pl["rows"] == (pl["vis"] if pl["refresh"] else sorted(act | set(pl["transient"])))
            if pl["refresh"]:
                assert pl["transient"] == [] and pl["in_phase_decoded"] == []
