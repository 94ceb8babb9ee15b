"""Pins for the oracle's forward pass, attention, RoPE, RMSNorm and the
unmask rule: closed forms, brute force, invariants the paper fixes, and the
reduction to an independently written dense full-sequence forward."""
import math

import numpy as np
import pytest

from oracle import wd_oracle as wo
from oracle.dense_ref import dense_full_forward
from paper_2601_20332_b200 import synth


def small_cfg(**kw):
    base = dict(L=2, d=64, Hq=4, Hkv=4, dh=16, F=96, V=50, P=6, G=10, batch=1,
                A=3, B=4, R=3, T=1, k=1, wseed=11, iseed=12)
    base.update(kw)
    return synth.get_config("tiny", **base)


def make(cfg, jitter=0.2):
    w = synth.make_weights(cfg, "cpu", gain_jitter=jitter)
    # larger weights than N(0, 0.02) so that attention is far from uniform
    for lst in (w.wq, w.wk, w.wv, w.wo, w.w_gate, w.w_up, w.w_down):
        for t in lst:
            t.mul_(8.0)
    w.tok_embed.mul_(20.0)
    return synth.OracleModelView(w)


def fresh_states(cfg, ids=None):
    ids = synth.make_prompts(cfg) if ids is None else ids
    P = cfg["P"]
    return [wo.SeqState(ids=row, decoded=np.arange(len(row)) < P) for row in ids]


def caches_for(cfg, model, n, fill=np.nan):
    return [wo.KVCache.empty(model.dims, cfg["P"] + cfg["G"], fill) for _ in range(n)]


# ---------------------------------------------------------------- small pieces

def test_rmsnorm_closed_forms():
    rng = np.random.default_rng(0)
    x = rng.normal(size=(5, 32))
    g = np.ones(32)
    eps = 1e-5
    y = wo.rmsnorm(x, g, eps)
    ms = (x * x).mean(-1)
    np.testing.assert_allclose(np.sqrt((y * y).mean(-1)), 1 / np.sqrt(1 + eps / ms), rtol=1e-12)
    np.testing.assert_allclose(wo.rmsnorm(1e3 * x, g, 0.0), wo.rmsnorm(x, g, 0.0), rtol=1e-12)
    g2 = rng.normal(size=32)
    np.testing.assert_allclose(wo.rmsnorm(x, g2, eps), g2 * y, rtol=1e-12)
    # one explicit value: x = (3, 4) -> ms = 12.5
    np.testing.assert_allclose(wo.rmsnorm(np.array([[3.0, 4.0]]), np.array([1.0, 2.0]), 0.0),
                               [[3 / math.sqrt(12.5), 8 / math.sqrt(12.5)]], rtol=1e-15)


def test_silu_identities():
    z = np.linspace(-6, 6, 25)
    assert wo.silu(np.array([0.0]))[0] == 0.0
    np.testing.assert_allclose(wo.silu(z) - wo.silu(-z), z, atol=1e-14)   # z*s(z) + z*(1-s(z))
    np.testing.assert_allclose(wo.silu(np.array([1.0])), [1 / (1 + math.exp(-1))], rtol=1e-15)


def test_rope_against_explicit_rotation():
    rng = np.random.default_rng(1)
    dh, theta = 8, 100.0
    x = rng.normal(size=(3, 2, dh))
    pos = np.array([0, 5, 17])
    y = wo.rope(x, pos, theta)
    np.testing.assert_array_equal(y[0], x[0])                     # position 0 = identity
    for n in range(3):
        for h in range(2):
            for j in range(dh // 2):
                ang = pos[n] * theta ** (-2 * j / dh)
                rot = np.array([[math.cos(ang), -math.sin(ang)], [math.sin(ang), math.cos(ang)]])
                np.testing.assert_allclose(y[n, h, [j, j + dh // 2]], rot @ x[n, h, [j, j + dh // 2]],
                                           rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(np.linalg.norm(y, axis=-1), np.linalg.norm(x, axis=-1), rtol=1e-12)
    # j = 0 rotates by exactly pos radians
    e = np.zeros((1, 1, dh)); e[0, 0, 0] = 1.0
    r = wo.rope(e, np.array([2]), theta)
    np.testing.assert_allclose(r[0, 0, [0, dh // 2]], [math.cos(2.0), math.sin(2.0)], rtol=1e-15)


def test_rope_relative_position_property():
    rng = np.random.default_rng(2)
    q = rng.normal(size=(4, 2, 16)); k = rng.normal(size=(6, 2, 16)); v = rng.normal(size=(6, 2, 16))
    pq, pk = np.array([3, 4, 9, 10]), np.array([0, 1, 3, 4, 9, 10])
    _, p0 = wo.attention_rows(wo.rope(q, pq, 1e4), wo.rope(k, pk, 1e4), v, 1)
    _, p1 = wo.attention_rows(wo.rope(q, pq + 37, 1e4), wo.rope(k, pk + 37, 1e4), v, 1)
    np.testing.assert_allclose(p0, p1, atol=1e-9)


def brute_attention(q, K, V, group):
    n, Hq, dh = q.shape
    out = np.zeros_like(q)
    for i in range(n):
        for h in range(Hq):
            kv = h // group
            s = [sum(q[i, h, c] * K[j, kv, c] for c in range(dh)) / math.sqrt(dh) for j in range(K.shape[0])]
            m = max(s)
            e = [math.exp(v - m) for v in s]
            z = sum(e)
            for c in range(dh):
                out[i, h, c] = sum(e[j] / z * V[j, kv, c] for j in range(K.shape[0]))
    return out


@pytest.mark.parametrize("Hq,Hkv", [(4, 4), (6, 2), (7, 1)])
def test_attention_brute_force_and_invariants(Hq, Hkv):
    rng = np.random.default_rng(3)
    q = rng.normal(size=(3, Hq, 8)) * 2; K = rng.normal(size=(5, Hkv, 8)) * 2; V = rng.normal(size=(5, Hkv, 8))
    out, p = wo.attention_rows(q, K, V, Hq // Hkv)
    np.testing.assert_allclose(out, brute_attention(q, K, V, Hq // Hkv), rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(p.sum(-1), 1.0, atol=1e-12)                 # rows sum to 1
    for h in range(Hq):                                                    # convex hull of visible V
        kv = h // (Hq // Hkv)
        assert (out[:, h] <= V[:, kv].max(0) + 1e-12).all() and (out[:, h] >= V[:, kv].min(0) - 1e-12).all()
    # permuting the enumeration of visible positions changes nothing
    perm = rng.permutation(5)
    out2, _ = wo.attention_rows(q, K[perm], V[perm], Hq // Hkv)
    np.testing.assert_allclose(out, out2, atol=1e-12)
    # a single visible position returns its V row; identical keys give the mean of V
    o1, _ = wo.attention_rows(q, K[:1], V[:1], Hq // Hkv)
    for h in range(Hq):
        np.testing.assert_allclose(o1[:, h], np.broadcast_to(V[0, h // (Hq // Hkv)], (3, 8)), rtol=1e-14)
    om, _ = wo.attention_rows(q, np.repeat(K[:1], 5, 0), V, Hq // Hkv)
    for h in range(Hq):
        np.testing.assert_allclose(om[:, h], np.broadcast_to(V[:, h // (Hq // Hkv)].mean(0), (3, 8)), rtol=1e-12)


# ---------------------------------------------------------------- unmask rule

def test_unmask_closed_forms():
    V = 37
    um = wo.oracle_unmask(np.full((3, V), 0.25), [10, 4, 7], 2)
    np.testing.assert_allclose(um["conf"], 1.0 / V, rtol=1e-14)
    assert list(um["ids"]) == [0, 0, 0]
    assert um["positions"] == [4, 7]                       # equal confidence -> lowest position
    lg = np.zeros((1, V)); lg[0, 9] = 50.0
    um = wo.oracle_unmask(lg, [3], 1)
    assert um["token_ids"] == [9] and abs(um["confidence"][0] - 1.0) < 1e-15
    lg = np.zeros((1, V)); lg[0, [5, 20]] = 3.0            # tie -> lowest vocabulary index
    assert wo.oracle_unmask(lg, [0], 1)["token_ids"] == [5]
    # two-way softmax closed form: conf = 1 / (1 + e^-a)
    um = wo.oracle_unmask(np.array([[0.0, 1.5]]), [0], 1)
    np.testing.assert_allclose(um["confidence"], [1 / (1 + math.exp(-1.5))], rtol=1e-15)


def test_unmask_brute_force():
    rng = np.random.default_rng(4)
    for trial in range(20):
        n, V, k = int(rng.integers(1, 9)), int(rng.integers(2, 40)), int(rng.integers(0, 5))
        lg = rng.normal(size=(n, V)) * 3
        pos = sorted(rng.choice(100, size=n, replace=False).tolist())
        um = wo.oracle_unmask(lg, pos, k)
        probs = np.exp(lg) / np.exp(lg).sum(-1, keepdims=True)
        conf = probs.max(-1)
        np.testing.assert_allclose(um["conf"], conf, rtol=1e-12)
        assert (um["conf"] <= 1.0 + 1e-15).all() and (um["conf"] >= 1.0 / V - 1e-15).all()
        assert list(um["ids"]) == list(probs.argmax(-1))
        want = [pos[r] for r in np.argsort(-conf, kind="stable")[: min(k, n)]]
        assert um["positions"] == want
        assert len(um["positions"]) == min(k, n)


# ---------------------------------------------------------------- whole step

@pytest.mark.parametrize("heads", [(4, 4), (4, 2), (4, 1)])
def test_step_reduces_to_dense_full_forward(heads):
    """Window covers every undecoded token and R = 1: the windowed step must be
    the ordinary full-sequence bidirectional forward (Sections 3.1 and 4.3)."""
    cfg = small_cfg(Hq=heads[0], Hkv=heads[1])
    model = make(cfg)
    states = fresh_states(cfg)
    caches = caches_for(cfg, model, 1)
    S = cfg["P"] + cfg["G"]
    ids0 = states[0].ids.copy()
    out = wo.oracle_step(model, states, caches, A=cfg["G"], B=0, R=1, T=0, k=2)[0]
    ref = dense_full_forward(model, ids0)
    assert out["plan"]["rows"] == list(range(S)) and out["plan"]["far_field"] == []
    for l in range(cfg["L"]):
        np.testing.assert_allclose(out["layer_out"][l], ref["layer_out"][l], rtol=1e-10, atol=1e-10)
        np.testing.assert_allclose(out["attn_out"][l], ref["attn_out"][l], rtol=1e-10, atol=1e-10)
    act = out["plan"]["active"]
    assert act == list(range(cfg["P"], S))
    np.testing.assert_allclose(out["logits"], ref["logits"][act], rtol=1e-10, atol=1e-10)
    # and the unmask choice is the brute-force top-2 of the dense softmax
    lg = ref["logits"][act]
    pr = np.exp(lg - lg.max(-1, keepdims=True)); pr /= pr.sum(-1, keepdims=True)
    top = np.argsort(-pr.max(-1), kind="stable")[:2]
    assert out["unmask"]["positions"] == [act[i] for i in top]
    assert out["unmask"]["token_ids"] == [int(pr[i].argmax()) for i in top]


def test_pruned_refresh_equals_dense_forward_on_visible_tokens():
    """A refresh step with far-field tokens pruned is the dense forward over
    the visible subsequence with its original positions kept: here the far
    field is a suffix, so it equals the dense forward of the truncated
    sequence."""
    cfg = small_cfg()
    model = make(cfg)
    states = fresh_states(cfg)
    caches = caches_for(cfg, model, 1)
    ids0 = states[0].ids.copy()
    out = wo.oracle_step(model, states, caches, cfg["A"], cfg["B"], cfg["R"], cfg["T"], 1)[0]
    nvis = cfg["P"] + cfg["A"] + cfg["B"]
    assert out["plan"]["vis"] == list(range(nvis)) and out["plan"]["far_field"]
    ref = dense_full_forward(model, ids0[:nvis])
    np.testing.assert_allclose(out["layer_out"][-1], ref["layer_out"][-1], rtol=1e-10, atol=1e-10)
    np.testing.assert_allclose(out["logits"], ref["logits"][out["plan"]["active"]], rtol=1e-10, atol=1e-10)


def run_traj(cfg, model, n_steps, poison=np.nan, states=None, caches=None, k=None, forced_seq=None):
    states = fresh_states(cfg) if states is None else states
    caches = caches_for(cfg, model, len(states), poison) if caches is None else caches
    outs = []
    for s in range(n_steps):
        forced = None if forced_seq is None else forced_seq[s]
        outs.append(wo.oracle_step(model, states, caches, cfg["A"], cfg["B"], cfg["R"], cfg["T"],
                                   cfg["k"] if k is None else k, forced=forced, want_probs=True))
    return outs, states, caches


def test_trajectory_invariants():
    cfg = small_cfg(G=30)
    model = make(cfg)
    outs, states, caches = run_traj(cfg, model, 7)
    kinds = [o[0]["plan"]["refresh"] for o in outs]
    assert kinds == [True, False, False, True, False, False, True]
    for o in outs:
        o = o[0]
        assert not np.isnan(o["layer_out"][-1]).any()          # never reads an unwritten cache row
        for p in o["probs"]:
            np.testing.assert_allclose(p.sum(-1), 1.0, atol=1e-12)
        assert o["logits"].shape == (len(o["plan"]["active"]), cfg["V"])   # logits only for active rows
        assert o["layer_out"][0].shape[0] == len(o["plan"]["rows"])
    # far-field rows of the cache were never written
    far = outs[0][0]["plan"]["far_field"]
    last_vis_hi = max(outs[-1][0]["plan"]["vis"])
    never = [p for p in far if p > last_vis_hi]
    assert never and np.isnan(caches[0].K[:, never]).all()


def test_refresh_independent_of_cache_content():
    cfg = small_cfg()
    model = make(cfg)
    a, _, _ = run_traj(cfg, model, 4, poison=np.nan)
    b, _, _ = run_traj(cfg, model, 4, poison=123.0)
    for oa, ob in zip(a, b):
        np.testing.assert_array_equal(oa[0]["logits"], ob[0]["logits"])


def test_normal_step_leaves_buffer_and_prefix_cache_untouched():
    cfg = small_cfg()
    model = make(cfg)
    states = fresh_states(cfg)
    caches = caches_for(cfg, model, 1)
    wo.oracle_step(model, states, caches, cfg["A"], cfg["B"], cfg["R"], cfg["T"], 1)
    K0 = caches[0].K.copy()
    out = wo.oracle_step(model, states, caches, cfg["A"], cfg["B"], cfg["R"], cfg["T"], 1)[0]
    pl = out["plan"]
    assert not pl["refresh"] and pl["transient"]
    rows = set(pl["rows"])
    keep = [p for p in pl["vis"] if p not in rows]
    assert set(pl["buffer"]) <= set(keep)
    np.testing.assert_array_equal(caches[0].K[:, keep], K0[:, keep])
    assert not np.array_equal(caches[0].K[:, pl["rows"]], K0[:, pl["rows"]])


def test_dry_step_idempotence():
    """If nothing is unmasked at the refresh step, every cached K/V equals what
    recomputation would give, so the following normal step reproduces the
    refresh step's active rows and logits."""
    cfg = small_cfg()
    model = make(cfg)
    outs, _, _ = run_traj(cfg, model, 2, k=0)
    r, n = outs[0][0], outs[1][0]
    assert r["plan"]["refresh"] and not n["plan"]["refresh"]
    assert n["plan"]["rows"] == n["plan"]["active"] == r["plan"]["active"]
    sel = [r["plan"]["rows"].index(p) for p in n["plan"]["rows"]]
    for l in range(cfg["L"]):
        np.testing.assert_allclose(n["layer_out"][l], r["layer_out"][l][sel], rtol=1e-10, atol=1e-12)
    np.testing.assert_allclose(n["logits"], r["logits"], rtol=1e-10, atol=1e-12)


def test_far_field_independence():
    cfg = small_cfg()
    model = make(cfg)
    a, _, _ = run_traj(cfg, model, 3)
    ids = synth.make_prompts(cfg)
    far = a[0][0]["plan"]["far_field"]
    ids[0, far] = 7                                            # different ids at far-field positions
    states = fresh_states(cfg, ids)
    caches = caches_for(cfg, model, 1, 55.0)
    b, _, _ = run_traj(cfg, model, 3, states=states, caches=caches)
    for oa, ob in zip(a, b):
        np.testing.assert_array_equal(oa[0]["logits"], ob[0]["logits"])


def test_stale_cache_is_really_used():
    """A normal step is an approximation: after a token is unmasked the buffer
    K/V are stale, so its logits differ from those of a full refresh at the
    same state (guards against an oracle that silently recomputes everything)."""
    cfg = small_cfg(T=0)
    model = make(cfg)
    outs, states, caches = run_traj(cfg, model, 1)
    st2 = [wo.SeqState(ids=s.ids.copy(), decoded=s.decoded.copy(), dec_step=s.dec_step.copy(), t=s.t,
                       since=s.since, phase_start=s.phase_start, wex=list(s.wex)) for s in states]
    n = wo.oracle_step(model, states, caches, cfg["A"], cfg["B"], cfg["R"], 0, 1)[0]
    f = wo.oracle_step(model, st2, caches_for(cfg, model, 1), cfg["A"], cfg["B"], 1, 0, 1)[0]
    assert not n["plan"]["refresh"] and f["plan"]["refresh"]
    assert n["plan"]["active"] == f["plan"]["active"]
    diff = np.abs(n["logits"] - f["logits"]).max()
    assert 1e-6 < diff


def test_r1_is_history_independent():
    cfg = small_cfg(R=1)
    model = make(cfg)
    outs, states, _ = run_traj(cfg, model, 3)
    # rebuild the state reached after two steps from scratch and run one step
    ids = synth.make_prompts(cfg)
    dec = np.arange(ids.shape[1]) < cfg["P"]
    for o in outs[:2]:
        for p, v in zip(*o[0]["committed"]):
            ids[0, p] = v; dec[p] = True
    st = [wo.SeqState(ids=ids[0], decoded=dec)]
    o = wo.oracle_step(model, st, caches_for(cfg, model, 1), cfg["A"], cfg["B"], 1, cfg["T"], 1)[0]
    np.testing.assert_allclose(o["logits"], outs[2][0]["logits"], rtol=1e-12, atol=1e-13)


def test_batch_independence():
    cfg = small_cfg(batch=3)
    model = make(cfg)
    ids = synth.make_prompts(cfg)
    both, _, _ = run_traj(cfg, model, 4, states=fresh_states(cfg, ids))
    for i in range(3):
        solo, _, _ = run_traj(cfg, model, 4, states=fresh_states(cfg, ids[i:i + 1]))
        for ob, os_ in zip(both, solo):
            np.testing.assert_array_equal(ob[i]["logits"], os_[0]["logits"])
            assert ob[i]["committed"] == os_[0]["committed"]
    assert not np.array_equal(both[0][0]["logits"], both[0][1]["logits"])


def test_teacher_forcing_and_tiny_config_runs():
    cfg = synth.get_config("tiny")
    model = synth.OracleModelView(synth.make_weights(cfg, "cpu"))
    states = fresh_states(cfg)
    caches = caches_for(cfg, model, 1)
    pl = wo.oracle_plan(states[0], cfg["A"], cfg["B"], cfg["R"], cfg["T"])
    forced = [([pl["active"][3]], [17])]
    o = wo.oracle_step(model, states, caches, cfg["A"], cfg["B"], cfg["R"], cfg["T"], 1, forced=forced)[0]
    assert o["committed"] == ([pl["active"][3]], [17])
    assert states[0].decoded[pl["active"][3]] and states[0].ids[pl["active"][3]] == 17
    assert o["logits"].shape == (8, 1024)
    c = o["unmask"]["conf"]
    assert (c > 1.0 / 1024).all() and (c < 0.1).all()      # random init: near-uniform but not degenerate


# ---------------------------------------------------------------- window-only refresh (variant, not in the paper)

def _variant_traj(cfg, model, mode, n_steps):
    states = fresh_states(cfg)
    for st in states:
        st.refresh_mode = mode
    return run_traj(cfg, model, n_steps, states=states)


def test_window_refresh_is_exact_for_a_one_layer_model():
    """With ONE block the K/V of a position depend only on its token and its position, so keeping
    the cached K/V of positions whose token did not change is the same as recomputing them: the
    variant must reproduce the paper's refresh to rounding, step after step."""
    cfg = small_cfg(L=1, G=24, T=2, R=3, k=2)
    model = make(cfg)
    full, _, cf = _variant_traj(cfg, model, 0, 9)
    win, _, cw = _variant_traj(cfg, model, 1, 9)
    n_fewer = 0
    for f, w in zip(full, win):
        f, w = f[0], w[0]
        assert f["plan"]["refresh"] == w["plan"]["refresh"]
        n_fewer += len(w["plan"]["rows"]) < len(f["plan"]["rows"])
        np.testing.assert_allclose(w["logits"], f["logits"], rtol=1e-10, atol=1e-10)
        assert w["committed"] == f["committed"]
    assert n_fewer >= 2                                     # the later refreshes really computed fewer rows
    vis = full[-1][0]["plan"]["vis"]
    np.testing.assert_allclose(cw[0].K[:, vis], cf[0].K[:, vis], rtol=1e-10, atol=1e-10)
    np.testing.assert_allclose(cw[0].V[:, vis], cf[0].V[:, vis], rtol=1e-10, atol=1e-10)


def test_window_refresh_is_an_approximation_for_deeper_models():
    """From the second block on, K/V depend on the context, so stale prefix entries change the
    result: the variant must differ from the paper's refresh (it is not a no-op) while the first
    layer's cache and the first phase stay identical."""
    cfg = small_cfg(L=2, G=24, T=2, R=3, k=2)
    model = make(cfg)
    forced = []
    full, _, cf = _variant_traj(cfg, model, 0, 4)
    for o in full:
        forced.append([o[0]["committed"]])
    states = fresh_states(cfg)
    states[0].refresh_mode = 1
    win, _, cw = run_traj(cfg, model, 4, states=states, forced_seq=forced)
    for s in range(3):                                      # first phase: the same steps
        np.testing.assert_allclose(win[s][0]["logits"], full[s][0]["logits"], rtol=1e-10, atol=1e-10)
    assert win[3][0]["plan"]["refresh"] and len(win[3][0]["plan"]["rows"]) < len(full[3][0]["plan"]["rows"])
    assert np.abs(win[3][0]["logits"] - full[3][0]["logits"]).max() > 1e-6
    assert np.isfinite(win[3][0]["logits"]).all()
    vis = full[3][0]["plan"]["vis"]
    np.testing.assert_allclose(cw[0].K[0][vis], cf[0].K[0][vis], rtol=1e-10, atol=1e-10)   # layer 0: context-free


# ---------------------------------------------------------------- FP8 mode (option outside the paper)

def _all_e4m3_values():
    """Every finite e4m3 value from the format's definition: sign, 4 exponent bits (bias 7),
    3 mantissa bits; exponent 0 is subnormal; exponent 15 with mantissa 7 is NaN."""
    vals = set()
    for e in range(16):
        for m in range(8):
            if e == 15 and m == 7:
                continue
            v = (m / 8.0) * 2.0 ** (-6) if e == 0 else (1.0 + m / 8.0) * 2.0 ** (e - 7)
            vals.add(v)
            vals.add(-v)
    return np.array(sorted(vals))


def test_e4m3_rounding_against_the_format_definition():
    grid = _all_e4m3_values()
    assert grid.max() == 448.0 and len(grid) == 2 * (16 * 8 - 1) - 1           # +0 and -0 coincide
    np.testing.assert_array_equal(wo.e4m3_round(grid.astype(np.float32)), grid)   # representable values stay
    rng = np.random.default_rng(5)
    x = np.concatenate([rng.uniform(-448, 448, 4000), rng.normal(0, 3, 4000), rng.normal(0, 0.01, 2000)]).astype(np.float32)
    got = wo.e4m3_round(x)
    # brute force: the nearest grid value; on a tie the one whose mantissa is even
    for v, g in zip(x.astype(np.float64), got):
        d = np.abs(grid - v)
        best = np.flatnonzero(d == d.min())
        if len(best) == 1:
            assert g == grid[best[0]]
        else:
            lo, hi = grid[best[0]], grid[best[1]]
            even = [c for c in (lo, hi) if (abs(c) / 2.0 ** np.floor(np.log2(max(abs(c), 2.0 ** -6))) * 8) % 2 == 0]
            assert g in (lo, hi) and (not even or g in even)
    # exact midpoints between neighbours round to the even mantissa: 1.0625 is halfway between 1.0 and 1.125
    np.testing.assert_array_equal(wo.e4m3_round(np.array([1.0625, 1.1875, -1.0625], np.float32)), [1.0, 1.25, -1.0])


def test_fp8_row_quantisation_and_product():
    rng = np.random.default_rng(6)
    x = rng.normal(0, 2, (5, 64))
    q, s = wo.fp8_quant_rows(x)
    assert s.dtype == np.float32 and np.abs(q).max(axis=1).tolist() == [448.0] * 5      # the row maximum maps to 448
    assert np.abs(q * s[:, None] - x).max() <= np.abs(x).max() * 2.0 ** -4           # half a spacing of the top binade
    zq, zs = wo.fp8_quant_rows(np.zeros((2, 8)))
    assert (zq == 0).all() and (zs == 1).all()
    # operands that are already on the grid (times a power of two) multiply exactly
    grid = _all_e4m3_values()
    # (row maximum 7 = 448 / 2^6 and 1.75 = 448 / 2^8: the scales are then powers of two)
    a = rng.choice(grid[(np.abs(grid) <= 7) & (np.abs(grid) >= 2.0 ** -3)], size=(4, 32)); a[:, 0] = 7.0
    b = rng.choice(grid[(np.abs(grid) <= 1.75) & (np.abs(grid) >= 2.0 ** -5)], size=(6, 32)); b[:, 0] = 1.75
    np.testing.assert_allclose(wo.fp8_matmul(a, b), a @ b.T, rtol=1e-6)
    # and the quantised product stays within the format's relative precision of the exact one
    w = rng.normal(0, 0.02, (16, 256)); xx = rng.normal(0, 1, (7, 256))
    err = np.linalg.norm(wo.fp8_matmul(xx, w) - xx @ w.T) / np.linalg.norm(xx @ w.T)
    assert 1e-3 < err < 8e-2


def test_fp8_mode_changes_only_the_quantised_projections():
    cfg = small_cfg(G=12)
    model = make(cfg)
    base, _, _ = run_traj(cfg, model, 2)
    model.dims = dict(model.dims, fp8=True)
    f8, _, _ = run_traj(cfg, model, 2)
    a, b = base[0][0], f8[0][0]
    assert a["plan"] == b["plan"]
    rel = np.linalg.norm(a["logits"] - b["logits"]) / np.linalg.norm(a["logits"])
    assert 1e-4 < rel < 0.3 and np.isfinite(b["logits"]).all()


# ---------------------------------------------------------------- bfloat16 storage points (precision mode)

def test_bf16_rounding_against_the_format_definition():
    """bfloat16 = sign, 8 exponent bits, 7 mantissa bits.  Brute force: the nearest value of the form
    m * 2^(e-7) with an 8-bit integer significand m in [128, 256), ties to the even m; then torch's cast."""
    import torch
    rng = np.random.default_rng(9)
    x = np.concatenate([rng.normal(0, 1, 3000), rng.normal(0, 1e-3, 1000), rng.uniform(-300, 300, 1000)]).astype(np.float32)
    got = wo.bf16_round(x)
    for v, g in zip(x.astype(np.float64), got):
        e = math.floor(math.log2(abs(v)))
        ulp = 2.0 ** (e - 7)
        lo = math.floor(abs(v) / ulp)
        cands = [lo * ulp, (lo + 1) * ulp]
        d = [abs(abs(v) - c) for c in cands]
        want = cands[0] if d[0] < d[1] else cands[1] if d[1] < d[0] else (cands[0] if lo % 2 == 0 else cands[1])
        assert g == math.copysign(want, v)
    np.testing.assert_array_equal(got, torch.from_numpy(x).to(torch.bfloat16).to(torch.float64).numpy())
    # representable values stay; exact midpoints go to the even mantissa: 1 + 2^-8 is halfway between 1 and 1 + 2^-7
    np.testing.assert_array_equal(wo.bf16_round(np.array([1.0, 1.5, -0.0078125, 0.0])), [1.0, 1.5, -0.0078125, 0.0])
    np.testing.assert_array_equal(wo.bf16_round(np.array([1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -8, -(1.0 + 2.0 ** -8)])),
                                  [1.0, 1.0 + 2.0 ** -6, -1.0])
    assert wo.bf16_round(np.zeros((2, 3))).shape == (2, 3)


def test_bf16_points_mode_rounds_the_stored_activations_and_nothing_else():
    cfg = small_cfg(G=12)
    model = make(cfg)
    states = fresh_states(cfg)
    rounded = [wo.SeqState(ids=states[0].ids.copy(), decoded=states[0].decoded.copy(), bf16_points=True)]
    c0, c1 = caches_for(cfg, model, 1), caches_for(cfg, model, 1)
    a = wo.oracle_step(model, states, c0, cfg["A"], cfg["B"], cfg["R"], cfg["T"], cfg["k"])[0]
    b = wo.oracle_step(model, rounded, c1, cfg["A"], cfg["B"], cfg["R"], cfg["T"], cfg["k"])[0]
    assert a["plan"] == b["plan"]                                       # the planner is untouched
    vis = a["plan"]["vis"]
    # what the mode stores is on the bfloat16 grid: the cache and the attention output
    for t in (c1[0].K[:, vis], c1[0].V[:, vis], b["attn_out"][0]):
        np.testing.assert_array_equal(wo.bf16_round(t), t)
    assert not np.array_equal(wo.bf16_round(c0[0].K[:, vis]), c0[0].K[:, vis])
    # layer 0's cache is the rounding of the unrounded one up to the rounding of the normalised input
    rel = np.linalg.norm(c1[0].K[0][vis] - c0[0].K[0][vis]) / np.linalg.norm(c0[0].K[0][vis])
    assert 5e-4 < rel < 6e-3
    # the residual stream and the logits are not rounded, and stay close to the float64 run
    assert not np.array_equal(wo.bf16_round(b["layer_out"][-1]), b["layer_out"][-1])
    rel = np.linalg.norm(b["logits"] - a["logits"]) / np.linalg.norm(a["logits"])
    assert 1e-4 < rel < 5e-2
    # a batch may mix the two modes: each sequence keeps its own
    mixed = wo.oracle_step(model, fresh_states(cfg) + [wo.SeqState(ids=states[0].ids.copy() * 0 + fresh_states(cfg)[0].ids,
                                                                   decoded=fresh_states(cfg)[0].decoded, bf16_points=True)],
                           caches_for(cfg, model, 2), cfg["A"], cfg["B"], cfg["R"], cfg["T"], cfg["k"])
    np.testing.assert_array_equal(mixed[0]["logits"], a["logits"])
    np.testing.assert_array_equal(mixed[1]["logits"], b["logits"])


# ---------------------------------------------------------------- NVFP4 mode (option outside the paper)

def test_e2m1_rounding_against_the_format_definition():
    """e2m1 = sign, 2 exponent bits (bias 1), 1 mantissa bit; exponent 0 is subnormal (0 or 0.5)."""
    vals = []
    for e in range(4):
        for m in range(2):
            vals.append((m / 2.0) if e == 0 else (1.0 + m / 2.0) * 2.0 ** (e - 1))
    assert vals == wo.E2M1_GRID.tolist() == [0.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0]
    np.testing.assert_array_equal(wo.e2m1_round(np.array(vals + [-v for v in vals], np.float32)), vals + [-v for v in vals])
    rng = np.random.default_rng(7)
    x = np.concatenate([rng.uniform(-8, 8, 4000), rng.normal(0, 1, 2000)]).astype(np.float32)
    got = wo.e2m1_round(x)
    for v, g in zip(x.astype(np.float64), got):
        d = np.abs(wo.E2M1_GRID - abs(v))
        best = np.flatnonzero(d == d.min())
        assert abs(g) == wo.E2M1_GRID[best[0]] if len(best) == 1 else abs(g) in wo.E2M1_GRID[best]
        assert g == 0 or np.sign(g) == np.sign(v)
    # exact midpoints go to the even code: codes 0..7 = 0, .5, 1, 1.5, 2, 3, 4, 6
    np.testing.assert_array_equal(wo.e2m1_round(np.array([0.25, 0.75, 1.25, 1.75, 2.5, 3.5, 5.0, -2.5, 100.0], np.float32)),
                                  [0.0, 1.0, 1.0, 2.0, 2.0, 4.0, 4.0, -2.0, 6.0])


def test_nvfp4_row_quantisation_and_product():
    rng = np.random.default_rng(8)
    x = rng.normal(0, 2, (5, 64))
    q, s, g = wo.nvfp4_quant_rows(x)
    assert q.shape == (5, 64) and s.shape == (5, 4) and g.dtype == np.float32
    assert set(np.abs(q).ravel().tolist()) <= set(wo.E2M1_GRID.tolist())
    np.testing.assert_array_equal(wo.e4m3_round(s.astype(np.float32)), s)               # block scales sit on the e4m3 grid
    assert s.max() <= 448.0 and (s.max(axis=1) >= 416.0).all()                          # the largest block of a row uses the top of it
    xb = wo.bf16_round(x)
    rec = q * np.repeat(s, 16, axis=1) * g.astype(np.float64)[:, None]
    # a block's elements are within half an e2m1 spacing (at most 1 of 6) of the block maximum's scale
    bmax = np.abs(xb).reshape(5, 4, 16).max(axis=2)
    assert (np.abs(rec - xb).reshape(5, 4, 16).max(axis=2) <= bmax * (1.0 / 6.0) * 1.07 + 1e-12).all()
    zq, zs, zg = wo.nvfp4_quant_rows(np.zeros((2, 32)))
    assert (zq == 0).all() and (zs == 0).all() and (zg == 1).all()
    # operands that already are NVFP4 numbers multiply exactly: grid values, one block scale, row maximum 6 * 448 * 2^-9
    a = rng.choice(wo.E2M1_GRID, size=(3, 32)) * rng.choice([-1.0, 1.0], size=(3, 32)); a[:, 0] = 6.0; a[:, 16] = 6.0
    b = rng.choice(wo.E2M1_GRID, size=(4, 32)) * rng.choice([-1.0, 1.0], size=(4, 32)); b[:, 0] = 6.0; b[:, 16] = 6.0
    np.testing.assert_allclose(wo.nvfp4_matmul(a * 448 * 2.0 ** -9, b * 448 * 2.0 ** -6), (a @ b.T) * 448 * 448 * 2.0 ** -15, rtol=1e-6)
    # and a random product stays within the format's precision of the exact one
    w = rng.normal(0, 0.02, (16, 256)); xx = rng.normal(0, 1, (7, 256))
    err = np.linalg.norm(wo.nvfp4_matmul(xx, w) - xx @ w.T) / np.linalg.norm(xx @ w.T)
    assert 2e-2 < err < 0.25


def test_nvfp4_mode_changes_only_the_quantised_projections():
    cfg = small_cfg(G=12)
    model = make(cfg)
    base, _, _ = run_traj(cfg, model, 2)
    model.dims = dict(model.dims, nvfp4=True)
    f4, _, _ = run_traj(cfg, model, 2)
    a, b = base[0][0], f4[0][0]
    assert a["plan"] == b["plan"]
    rel = np.linalg.norm(a["logits"] - b["logits"]) / np.linalg.norm(a["logits"])
    assert 1e-3 < rel < 0.6 and np.isfinite(b["logits"]).all()
