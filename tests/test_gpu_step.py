"""Parity of the whole windowed step against the CPU oracle (GPU required)."""
import os

import numpy as np
import pytest
import torch

from paper_2601_20332_b200 import binding as wd
from paper_2601_20332_b200 import build as wd_build
from paper_2601_20332_b200 import synth
from wd_harness import Parity

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.fixture(scope="module", autouse=True)
def built():
    wd_build.build()


def run(cfg, n_steps, ids=None, decoded=None, impl=wd.WD_GEMM_AUTO, jitter=0.1, tol_layer=1e-2, tol_attn=2e-2,
        oracle_seqs=None, weights=None, fusion=wd.WD_FUSION_AUTO, refresh_mode=0, fp8=False, stagger=False, fp4=False):
    w = synth.make_weights(cfg, DEV, gain_jitter=jitter) if weights is None else weights
    ids = synth.make_prompts(cfg) if ids is None else ids
    p = Parity(cfg, w, ids, decoded, gemm_impl=impl, oracle_seqs=oracle_seqs, fusion=fusion, refresh_mode=refresh_mode,
               fp8=fp8, stagger=stagger, fp4=fp4)
    logs = []
    for _ in range(n_steps):
        r = p.step(cfg["A"], cfg["B"], cfg["R"], cfg["T"], cfg["k"], tol_layer, tol_attn)
        if r is None:
            break
        logs.append(r)
    p.check_state_mirror()
    p.close()
    return logs


def test_tiny_fp32_full_generation():
    """cfg 1: the whole 64-step generation, every step compared."""
    cfg = synth.get_config("tiny")
    logs = run(cfg, 70, tol_layer=2e-5, tol_attn=2e-5)
    assert len(logs) == 64
    kinds = [l["info"]["is_refresh"] for l in logs]
    assert kinds[:8] == [1, 0, 0, 0, 1, 0, 0, 0]
    assert sum(l["worst"]["ambiguous"] for l in logs) == 0
    assert max(l["info"]["n_rows"] for l in logs if not l["info"]["is_refresh"]) <= 8 + 2


SMALL_BF16 = dict(L=3, d=512, Hq=8, Hkv=8, dh=64, F=1408, V=5000, P=40, G=80, A=8, B=24, R=4, T=2, k=1)


@pytest.mark.parametrize("impl", [wd.WD_GEMM_PLAIN, wd.WD_GEMM_TCGEN05])
def test_small_bf16_trajectory(impl):
    cfg = synth.get_config("llada8b", **SMALL_BF16)
    logs = run(cfg, 10, impl=impl)
    assert [l["info"]["is_refresh"] for l in logs[:9]] == [1, 0, 0, 0, 1, 0, 0, 0, 1]
    assert all(l["info"]["gemm_impl"] == impl for l in logs)
    assert any(len(p["transient"]) == 2 for l in logs for p in l["plans"])


def test_small_bf16_gqa_batch_two_tokens():
    """GQA (7 query heads per KV head), batch of independent windows, k = 2, head_dim 128."""
    cfg = synth.get_config("dream7b", L=2, d=896, Hq=7, Hkv=1, dh=128, F=1024, V=3000, P=20, G=50, batch=3,
                           A=6, B=10, R=3, T=3, k=2)
    logs = run(cfg, 8)
    assert len(logs) == 8
    # sequences got different prompts, so their choices differ
    pos = np.array([l["res"]["positions"][:, 0] for l in logs])
    assert pos.shape == (8, 3)


DH128 = dict(L=2, d=512, Hq=4, Hkv=4, dh=128, F=1024, V=4000, P=200, G=150, A=16, B=40, R=3, T=2, k=2)


FUSIONS = [wd.WD_FUSION_NONE, wd.WD_FUSION_TILE, wd.WD_FUSION_CLUSTER, wd.WD_FUSION_CHAIN]


@pytest.mark.parametrize("Hkv,batch,fusion", [(4, 1, wd.WD_FUSION_NONE), (2, 2, wd.WD_FUSION_NONE), (1, 1, wd.WD_FUSION_NONE)] +
                         [(4, 1, f) for f in FUSIONS[1:]] + [(2, 2, f) for f in FUSIONS[1:]] + [(1, 3, f) for f in FUSIONS[2:]])
def test_bf16_head_dim_128_tensor_core_attention(Hkv, batch, fusion):
    """head_dim 128 takes the tcgen05 attention: two query tiles at the refresh (256 visible
    rows), key tiles with a ragged tail split across CTAs, MHA and GQA, batch of independent
    windows; with the consumers of the GEMMs as separate kernels and in every fused form (the
    cluster and chain forms serve the normal steps: 18 to 54 rows here)."""
    cfg = synth.get_config("llada8b", **dict(DH128, Hkv=Hkv, batch=batch))
    logs = run(cfg, 7, fusion=fusion)
    assert [l["info"]["is_refresh"] for l in logs] == [1, 0, 0, 1, 0, 0, 1]
    assert logs[0]["info"]["n_rows"] == batch * 256


def test_gate_up_swiglu_epilogue_with_ragged_ffn_width_and_token_tile():
    """d_ffn 19008 = 74 whole 256-row tiles + 64 rows, 262 rows at the second refresh (token tiles of
    144 and 118): every CTA pair gets two (gate tile, up tile) units, so the two-CTA GEMM writes
    h = silu(gate) * up itself; the last weight tile and the second token tile are partial.  The
    layer outputs (which h feeds through the down projection) follow the oracle."""
    cfg = synth.get_config("llada8b", L=1, d=256, Hq=2, Hkv=2, dh=128, F=19008, V=2000, P=200, G=100, A=16, B=40,
                           R=3, T=2, k=2)
    logs = run(cfg, 4)
    assert [l["info"]["is_refresh"] for l in logs] == [1, 0, 0, 1]
    assert logs[0]["info"]["n_rows"] == 256 and logs[3]["info"]["n_rows"] > 256
    if not any(os.environ.get(k) == "0" for k in ("WD_GEMM_DUAL", "WD_GEMM_SWIGLU", "WD_GEMM_PAIR_FROM")):
        # no SwiGLU kernel in the second refresh: one launch fewer than in the first (256 rows, one-CTA GEMMs)
        assert logs[3]["info"]["n_launches"] == logs[0]["info"]["n_launches"] - 1


@pytest.mark.parametrize("batch,A", [(2, 160), (4, 150), (4, 250)])
def test_lm_head_statistics_with_several_token_tiles(batch, A):
    """More than 256 active rows: the LM-head epilogue runs one CTA group per token tile (two
    tiles at 320 rows, three rounded up to four at 600, four at 1000); logits, per-row
    statistics and the unmask choice stay exact for every row."""
    cfg = synth.get_config("llada8b", **dict(DH128, L=1, P=30, G=260, A=A, B=8, R=2, T=1, k=3, batch=batch))
    logs = run(cfg, 3, oracle_seqs=[0, batch - 1])
    assert logs[0]["info"]["n_active"] == batch * A


@pytest.mark.parametrize("shape,batch", [(SMALL_BF16, 1), (DH128, 2)])
def test_window_only_refresh_variant_matches_its_oracle(shape, batch):
    """WD_REFRESH_WINDOW (not in the paper): refresh steps after the first compute only the new
    window and the previous phase's tokens; index sets, layer outputs, logits and unmask choices
    follow the oracle run in the same mode, through three phases (device-planned steps)."""
    cfg = synth.get_config("llada8b", **dict(shape, batch=batch))
    logs = run(cfg, 3 * cfg["R"] + 1, refresh_mode=wd.WD_REFRESH_WINDOW)
    refreshes = [l for l in logs if l["info"]["is_refresh"]]
    assert len(refreshes) == 4
    per_seq_window = cfg["A"] + cfg["B"] + cfg["k"] * cfg["R"]
    assert refreshes[0]["info"]["n_rows"] == refreshes[0]["info"]["n_vis"]        # first step: everything
    for r in refreshes[1:]:
        assert r["info"]["n_rows"] == batch * per_seq_window < r["info"]["n_vis"]


@pytest.mark.parametrize("shape,batch", [(SMALL_BF16, 1), (DH128, 2)])
def test_fp8_mode_matches_the_oracle_in_fp8_mode(shape, batch):
    """FP8 projections (outside the paper): e4m3 weights and activations with per-row scales for
    q/k/v, gate/up, down and the LM head; the oracle quantises the same operands the same way, so
    the usual tolerances hold (a few elements land on the other side of a rounding boundary)."""
    cfg = synth.get_config("llada8b", **dict(shape, batch=batch))
    # Tolerances: an upstream difference of bf16 size (4e-3, as in the bf16 tests) moves about 7 % of
    # the activations across an e4m3 rounding boundary (spacing 6-12 %), each by one spacing, which is
    # 0.06 * sqrt(0.07) = 1.6e-2 of relative RMS per quantised projection; the exact agreement of the
    # quantised product itself is checked on identical inputs in test_gemm_fp8_vs_oracle.
    logs = run(cfg, 2 * cfg["R"] + 1, fp8=True, tol_layer=5e-2, tol_attn=1e-1)
    assert sum(l["info"]["is_refresh"] for l in logs) == 3
    assert max(l["worst"]["layer"] for l in logs) > 1e-3      # and it is not the bf16 pipeline


def test_fp8_mode_differs_from_bf16_and_can_be_switched_off():
    cfg = synth.get_config("llada8b", **DH128)
    w = synth.make_weights(cfg, DEV)
    ids = synth.make_prompts(cfg)
    S = ids.shape[1]
    ctx = wd.Context(cfg, w, 1, S, S, S)
    lg = torch.zeros(S * cfg["V"], device=DEV)
    outs = []
    for mode in ("bf16", "fp8", "off again"):
        if mode == "fp8":
            ctx.fp8_enable()
        if mode == "off again":
            ctx.fp8_set(False)
        st = wd.State(ctx, ids)
        st.set_taps(logits=lg)
        _, info = st.step(cfg["A"], cfg["B"], cfg["R"], cfg["T"], 1)
        st.sync()
        outs.append(lg[: info["n_active"] * cfg["V"]].clone())
        st.close()
    assert torch.equal(outs[0], outs[2])
    rel = float((outs[1] - outs[0]).norm() / outs[0].norm())
    assert 1e-3 < rel < 0.3
    with pytest.raises(wd.WdError):
        wd.Context(synth.get_config("tiny"), synth.make_weights(synth.get_config("tiny"), DEV), 1, 96, 96, 8).fp8_enable()
    ctx.close()


NVFP4_SMALL = dict(SMALL_BF16, F=1536)       # the mode wants widths that are multiples of 256


@pytest.mark.parametrize("shape,batch", [(NVFP4_SMALL, 1), (DH128, 2)])
def test_nvfp4_mode_matches_the_oracle_in_nvfp4_mode(shape, batch):
    """NVFP4 projections (outside the paper): the oracle quantises the same operands the same way.  On
    identical inputs the quantised product agrees to 2e-5 (test_gemm_nvfp4_vs_oracle); in a step the two
    sides' activations differ upstream by bf16-size amounts, and a 4-bit code turns such a difference into
    a whole code step for the elements near a rounding boundary."""
    cfg = synth.get_config("llada8b", **dict(shape, batch=batch))
    # Tolerances: an upstream difference of 4e-3 (bf16) moves an element of magnitude |x| across an e2m1
    # boundary with probability 4e-3 |x| / spacing, about 1 % (spacing 1/6 to 1/2 of |x|), and then by a
    # whole spacing, a third of its value: 0.33 * sqrt(0.012) = 3.6e-2 relative RMS per quantised product;
    # a flipped e4m3 block scale (4 % of the blocks) redraws the block's rounding noise, another 3e-2.
    # Three quantised products in series per block and the LM head on top give, as the worst element over
    # the largest, 9e-2 for the block outputs and 1.5e-1 for the logits measured; bounds at 1.7x that.
    logs = run(cfg, 2 * cfg["R"] + 1, fp4=True, tol_layer=1.5e-1, tol_attn=1e-1)
    assert sum(l["info"]["is_refresh"] for l in logs) == 3
    assert max(l["worst"]["layer"] for l in logs) > 1e-2      # and it is not the bf16 pipeline
    assert max(l["worst"]["logits"] for l in logs) < 2.5e-1


def test_nvfp4_mode_differs_from_bf16_and_excludes_fp8():
    cfg = synth.get_config("llada8b", **DH128)
    w = synth.make_weights(cfg, DEV)
    ids = synth.make_prompts(cfg)
    S = ids.shape[1]
    ctx = wd.Context(cfg, w, 1, S, S, S)
    lg = torch.zeros(S * cfg["V"], device=DEV)
    outs = {}
    for mode in ("bf16", "fp4", "fp8", "fp4 again", "off"):
        if mode == "fp4":
            ctx.fp4_enable()
        if mode == "fp8":
            ctx.fp8_enable()            # switches NVFP4 off
        if mode == "fp4 again":
            ctx.fp4_set(True)           # ... and back, which switches FP8 off
        if mode == "off":
            ctx.fp4_set(False)
        st = wd.State(ctx, ids)
        st.set_taps(logits=lg)
        _, info = st.step(cfg["A"], cfg["B"], cfg["R"], cfg["T"], 1)
        st.sync()
        outs[mode] = lg[: info["n_active"] * cfg["V"]].clone()
        st.close()
    assert torch.equal(outs["bf16"], outs["off"])
    assert torch.equal(outs["fp4"], outs["fp4 again"])
    rel4 = float((outs["fp4"] - outs["bf16"]).norm() / outs["bf16"].norm())
    rel8 = float((outs["fp8"] - outs["bf16"]).norm() / outs["bf16"].norm())
    assert 1e-3 < rel8 < rel4 < 0.6
    with pytest.raises(wd.WdError):     # fp32 model
        wd.Context(synth.get_config("tiny"), synth.make_weights(synth.get_config("tiny"), DEV), 1, 96, 96, 8).fp4_enable()
    with pytest.raises(wd.WdError):     # d_ffn not a multiple of 256
        c2 = synth.get_config("llada8b", **SMALL_BF16)
        wd.Context(c2, synth.make_weights(c2, DEV), 1, 120, 120, 8).fp4_enable()
    ctx.close()


@pytest.mark.parametrize("mode", ["bf16", "fp8", "fp4"])
def test_step_graphs_replay_gives_the_same_generation(mode):
    """Steps replayed from a CUDA graph (wd_set_graphs, the default) run the same kernels with the same
    arguments as steps launched directly: token ids, confidences, per-step launch counts and step shapes of a
    whole generation are identical, graphs really are recorded and replayed, and a context with graphs off
    records none."""
    cfg = synth.get_config("llada8b", **dict(DH128, batch=2, G=96))
    w = synth.make_weights(cfg, DEV)
    ids = synth.make_prompts(cfg)
    S = ids.shape[1]
    runs = []
    stream = torch.cuda.Stream(device=DEV)         # (the legacy default stream cannot record graphs)
    for on in (False, True):
        ctx = wd.Context(cfg, w, 2, S, 2 * S, 2 * cfg["A"])
        ctx.set_graphs(on)
        if mode == "fp8":
            ctx.fp8_enable()
        if mode == "fp4":
            ctx.fp4_enable()
        st = wd.State(ctx, ids)
        infos, outs = [], []
        for i in range(200):
            status, info = st.step(cfg["A"], cfg["B"], cfg["R"], cfg["T"], cfg["k"], stream)
            if status == wd.WD_DONE:
                break
            infos.append((info["is_refresh"], info["n_rows"], info["n_active"], info["n_vis"], info["n_launches"]))
            if i % 5 == 4:                 # a few steps queue up between syncs
                outs += st.sync_all()
        outs += st.sync_all()
        final = [st.read(b)["ids"].copy() for b in range(2)]
        runs.append((infos, outs, final, ctx.graph_stats()))
        st.close()
        ctx.close()
    (i0, o0, f0, g0), (i1, o1, f1, g1) = runs
    assert i0 == i1 and len(i0) == 96 // cfg["k"]
    assert all(np.array_equal(a, b) for a, b in zip(f0, f1)) and all((f != cfg["mask_id"]).all() for f in f0)
    assert len(o0) == len(o1)
    for x, y in zip(o0, o1):
        assert np.array_equal(x["positions"], y["positions"]) and np.array_equal(x["token_ids"], y["token_ids"])
        assert np.array_equal(x["confidence"], y["confidence"])
    assert g0 == (0, 0)
    assert g1[0] >= 1 and g1[1] >= len(i1) // 3          # most normal steps are replays


def test_step_graphs_stay_off_without_the_tensor_core_attention():
    """head_dim 64 runs the index-list attention kernel, whose launch depends on the exact visible count: such
    steps are never recorded (and the generation still completes, queued steps and all)."""
    cfg = synth.get_config("llada8b", **dict(SMALL_BF16, G=40))
    w = synth.make_weights(cfg, DEV)
    ids = synth.make_prompts(cfg)
    S = ids.shape[1]
    ctx = wd.Context(cfg, w, 1, S, S, cfg["A"])
    st = wd.State(ctx, ids)
    stream = torch.cuda.Stream(device=DEV)
    status, steps, tokens = st.generate(cfg["A"], cfg["B"], cfg["R"], cfg["T"], cfg["k"], 0, stream)
    assert tokens == 40 and (st.read(0)["ids"] != cfg["mask_id"]).all()
    assert ctx.graph_stats() == (0, 0)
    st.close()
    ctx.close()


def test_plain_and_tensor_core_paths_agree():
    """The CUDA-core kernels and the tensor-core kernels compute the same step."""
    cfg = synth.get_config("llada8b", **DH128)
    w = synth.make_weights(cfg, DEV)
    ids = synth.make_prompts(cfg)
    S = ids.shape[1]
    outs = []
    for impl in (wd.WD_GEMM_PLAIN, wd.WD_GEMM_TCGEN05):
        ctx = wd.Context(cfg, w, 1, S, S, S)
        ctx.set_gemm_impl(impl)
        st = wd.State(ctx, ids)
        lay = torch.zeros(cfg["L"] * S * cfg["d"], device=DEV)
        st.set_taps(layer_out=lay)
        res = []
        for _ in range(3):
            _, info = st.step(cfg["A"], cfg["B"], cfg["R"], cfg["T"], 0)      # k = 0: same state on both paths
            st.sync()
            res.append(lay[: cfg["L"] * info["n_rows"] * cfg["d"]].clone())
        outs.append(res)
        st.close(); ctx.close()
    for a, b in zip(*outs):
        rel = (a - b).norm() / b.norm()
        assert rel < 5e-3, rel


def test_window_covering_everything_is_full_sequence_step():
    """A >= number of masks, B = 0, R = 1: every step is the no-pruning full-sequence step."""
    cfg = synth.get_config("llada8b", **dict(SMALL_BF16, A=80, B=0, R=1, T=0, k=4))
    logs = run(cfg, 3)
    assert all(l["info"]["is_refresh"] for l in logs)
    assert logs[0]["info"]["n_rows"] == 120 and logs[0]["info"]["n_active"] == 80


def test_non_prefix_decoded_pattern_uses_index_lists():
    cfg = synth.get_config("llada8b", **SMALL_BF16)
    ids = synth.make_prompts(cfg)
    S = ids.shape[1]
    dec = synth.random_decoded_pattern(S, 0.4, 5)[None, :]
    rng = np.random.default_rng(3)
    ids = np.where(dec == 1, rng.integers(0, cfg["V"] - 1, size=ids.shape), cfg["mask_id"]).astype(np.int32)
    logs = run(cfg, 6, ids=ids, decoded=dec)
    assert not logs[0]["plans"][0]["vis_contiguous"]


def test_late_state_and_finish():
    """Fast-forwarded state near the end: runs to WD_DONE, last phases have fewer tokens than A."""
    cfg = synth.get_config("llada8b", **SMALL_BF16)
    ids, dec = synth.fast_forward(cfg, synth.make_prompts(cfg), 70)
    logs = run(cfg, 20, ids=ids, decoded=dec)
    assert len(logs) == 10                          # 10 masks left, one per step
    assert logs[-1]["info"]["n_active"] == 1


def test_adaptive_termination_on_gpu():
    """Take the id the model generates at the third step as the end-of-sequence id: the rerun
    must follow the oracle step by step and finish early (Section 4.2, adaptive termination)."""
    cfg = synth.get_config("llada8b", **SMALL_BF16)
    w = synth.make_weights(cfg, DEV, gain_jitter=0.1)
    ids = synth.make_prompts(cfg)
    p = Parity(cfg, w, ids)
    toks = [p.step(cfg["A"], cfg["B"], cfg["R"], cfg["T"], 1)["res"] for _ in range(3)]
    p.close()
    eos = int(toks[2]["token_ids"][0, 0])
    p = Parity(cfg, w, ids, eos_id=eos)
    n = 0
    while p.step(cfg["A"], cfg["B"], cfg["R"], cfg["T"], 1) is not None:
        n += 1
        assert n <= cfg["G"]
    p.check_state_mirror()
    st = p.st.read(0)
    p.close()
    # (the harness has checked every step against the oracle, which carries the same eos id)
    gen = np.flatnonzero(st["decoded"] & (st["ids"] == eos) & (st["dec_step"] >= 0))
    assert n < cfg["G"] and len(gen) > 0
    e = int(gen.min())                                       # first generated eos in position order
    assert st["decoded"][: e + 1].all()                      # everything before it was decoded ...
    assert not st["decoded"][e + 1:].all()                   # ... and the tail was left alone


@pytest.mark.parametrize("shape", [SMALL_BF16, DH128])
def test_far_field_and_refresh_independence_on_gpu(shape):
    """Changing ids at far-field positions and poisoning the K/V cache before a refresh
    changes nothing, bit for bit (with head_dim 128 the attention tiles cover poisoned
    far-field cache rows, which must stay masked)."""
    cfg = synth.get_config("llada8b", **shape)
    w = synth.make_weights(cfg, DEV)
    ids = synth.make_prompts(cfg)
    S = ids.shape[1]
    outs = []
    for variant in range(2):
        ctx = wd.Context(cfg, w, 1, S, S, S)
        ids_v = ids.copy()
        if variant:
            ids_v[0, cfg["P"] + cfg["A"] + cfg["B"]:] = 17
        st = wd.State(ctx, ids_v, (ids != cfg["mask_id"]).astype(np.uint8))
        # state memory = ids | K cache | V cache | device planner state (flags, steps, window)
        up = lambda v: (v + 255) // 256 * 256
        tail = (up(S) + 2 * up(4 * S)) // 2
        st.mem.view(torch.int16)[S * 2 + 128: -tail].fill_(0x7FC0 if variant else 0)      # NaN / zero K/V cache
        torch.cuda.synchronize()
        lg = torch.zeros(S * cfg["V"], device=DEV)
        st.set_taps(logits=lg)
        res = []
        for _ in range(3):
            _, info = st.step(cfg["A"], cfg["B"], cfg["R"], cfg["T"], 1)
            r = st.sync()
            res.append((lg[: info["n_active"] * cfg["V"]].clone(), r["positions"].copy(), r["token_ids"].copy()))
        outs.append(res)
        st.close(); ctx.close()
    for a, b in zip(*outs):
        assert torch.equal(a[0], b[0]) and (a[1] == b[1]).all() and (a[2] == b[2]).all()


@pytest.mark.parametrize("shape,batch,mode", [(SMALL_BF16, 1, 0), (DH128, 2, 0), (DH128, 2, 1)])
def test_steps_enqueued_back_to_back_match_stepwise_sync(shape, batch, mode):
    """With a prompt-prefix state the device plans the steps itself: a whole run enqueued without
    a host round trip gives exactly the results of the same run with a sync after every step,
    and the host mirror ends up identical."""
    cfg = synth.get_config("llada8b", **dict(shape, batch=batch))
    w = synth.make_weights(cfg, DEV)
    ids = synth.make_prompts(cfg)
    S = ids.shape[1]
    n_steps = 11
    ctx = wd.Context(cfg, w, batch, S, batch * S, batch * cfg["A"])
    runs = []
    for queued in (False, True):
        st = wd.State(ctx, ids)
        st.set_refresh_mode(mode)
        res = []
        for i in range(n_steps):
            st.step(cfg["A"], cfg["B"], cfg["R"], cfg["T"], cfg["k"])
            if not queued:
                res.append(st.sync())
        if queued:
            res = st.sync_all()
            assert len(res) == n_steps
        runs.append((res, [st.read(b) for b in range(batch)]))
        st.close()
    for a, b in zip(*[r[0] for r in runs]):
        assert (a["n_unmasked"] == b["n_unmasked"]).all()
        assert (a["positions"] == b["positions"]).all() and (a["token_ids"] == b["token_ids"]).all()
        assert (a["confidence"] == b["confidence"]).all()
    for ma, mb in zip(runs[0][1], runs[1][1]):
        assert (ma["ids"] == mb["ids"]).all() and (ma["decoded"] == mb["decoded"]).all()
        assert (ma["dec_step"] == mb["dec_step"]).all() and ma["t"] == mb["t"] == n_steps and ma["since"] == mb["since"]
    # the queue holds 32 steps; the 33rd needs a sync first
    st = wd.State(ctx, ids)
    for i in range(32):
        st.step(cfg["A"], cfg["B"], cfg["R"], cfg["T"], cfg["k"])
    with pytest.raises(wd.WdError) as e:
        st.step(cfg["A"], cfg["B"], cfg["R"], cfg["T"], cfg["k"])
    assert e.value.status == wd.WD_ERR_PENDING
    with pytest.raises(wd.WdError) as e:
        st.plan(0, cfg["A"], cfg["B"], cfg["R"], cfg["T"])
    assert e.value.status == wd.WD_ERR_PENDING
    st.sync()
    assert st.read(0)["t"] == 32
    st.close(); ctx.close()


@pytest.mark.parametrize("eos", [False, True])
def test_generate_runs_the_whole_decoding_loop(eos):
    """wd_generate = the same steps as a hand-written loop of wd_step + wd_step_sync: identical
    final tokens, decode steps and counters (device-planned queue without adaptive termination,
    host-planned one step at a time with it)."""
    cfg = synth.get_config("llada8b", **DH128)
    w = synth.make_weights(cfg, DEV)
    ids = synth.make_prompts(cfg)
    S = ids.shape[1]
    A, B, R, T, k = (cfg[x] for x in ("A", "B", "R", "T", "k"))
    ctx = wd.Context(cfg, w, 1, S, S, A)
    finals = []
    for use_generate in (False, True):
        st = wd.State(ctx, ids)
        if eos:
            st.set_eos(3)
        if use_generate:
            status, n_steps, n_tok = st.generate(A, B, R, T, k)
            assert status == wd.WD_DONE
        else:
            n_steps = n_tok = 0
            while True:
                status, _ = st.step(A, B, R, T, k)
                if status == wd.WD_DONE:
                    break
                n_tok += int(st.sync()["n_unmasked"].sum())
                n_steps += 1
        finals.append((st.read(0), n_steps, n_tok))
        st.close()
    (ma, sa, ta), (mb, sb, tb) = finals
    assert sa == sb and ta == tb and sa > 0
    assert (ma["ids"] == mb["ids"]).all() and (ma["decoded"] == mb["decoded"]).all()
    assert (ma["dec_step"] == mb["dec_step"]).all() and ma["t"] == mb["t"] == sa
    if not eos:
        assert ma["decoded"].all() and ta == cfg["G"]
    # max_steps stops early with WD_OK and leaves a consistent state
    st = wd.State(ctx, ids)
    status, n_steps, n_tok = st.generate(A, B, R, T, k, max_steps=5)
    assert status == wd.WD_OK and n_steps == 5 and n_tok == 5 * k and st.read(0)["t"] == 5
    st.close(); ctx.close()


def test_non_prefix_state_needs_a_sync_between_steps():
    cfg = synth.get_config("llada8b", **SMALL_BF16)
    w = synth.make_weights(cfg, DEV)
    ids = synth.make_prompts(cfg)
    S = ids.shape[1]
    dec = synth.random_decoded_pattern(S, 0.4, 5)[None, :]
    ctx = wd.Context(cfg, w, 1, S, S, S)
    st = wd.State(ctx, ids, dec)
    st.step(cfg["A"], cfg["B"], cfg["R"], cfg["T"], 1)
    with pytest.raises(wd.WdError) as e:
        st.step(cfg["A"], cfg["B"], cfg["R"], cfg["T"], 1)
    assert e.value.status == wd.WD_ERR_PENDING
    st.sync()
    st.close(); ctx.close()


def test_step_error_codes():
    cfg = synth.get_config("llada8b", **SMALL_BF16)
    w = synth.make_weights(cfg, DEV)
    ids = synth.make_prompts(cfg)
    S = ids.shape[1]
    ctx = wd.Context(cfg, w, 1, S, 64, 16)            # max_rows 64 < a refresh over 72 rows
    st = wd.State(ctx, ids)
    with pytest.raises(wd.WdError) as e:
        st.step(8, 24, 4, 2, 1)
    assert e.value.status == wd.WD_ERR_CAPACITY
    with pytest.raises(wd.WdError) as e:
        st.step(0, 24, 4, 2, 1)
    assert e.value.status == wd.WD_ERR_BAD_PARAM
    with pytest.raises(wd.WdError) as e:
        st.sync()
    assert e.value.status == wd.WD_ERR_NOT_PENDING
    status, _ = st.step(8, 8, 4, 2, 1)                # 40 + 16 = 56 rows fits
    assert status == wd.WD_OK
    st.sync()
    st.close(); ctx.close()
    with pytest.raises(wd.WdError) as e:
        wd.Context(synth.get_config("llada8b", **dict(SMALL_BF16, d=500)), w, 1, S, S, S)
    assert e.value.status == wd.WD_ERR_INVALID_DIMS


def _small_state(cfg, w, ids):
    S = ids.shape[1]
    ctx = wd.Context(cfg, w, ids.shape[0], S, ids.shape[0] * S, ids.shape[0] * cfg["A"])
    return ctx, wd.State(ctx, ids)


def _steps(st, cfg, n, stream=None):
    out = []
    for _ in range(n):
        status, info = st.step(cfg["A"], cfg["B"], cfg["R"], cfg["T"], cfg["k"], stream)
        if status == wd.WD_DONE:
            break
        r = st.sync()
        out.append((info["is_refresh"], info["n_rows"], r["positions"].tolist(), r["token_ids"].tolist(),
                    r["confidence"].tolist()))
    return out


@pytest.mark.parametrize("queued", [False, True])
def test_device_index_check_reports_bounds_and_the_state_waits_for_a_reset(queued):
    """A token id outside the vocabulary in the DEVICE copy of the ids (put there through the test hook; the
    host entry points reject such ids) is never used as an index: the embedding kernel skips the row and
    records WD_ERR_BOUNDS, wd_step_sync reports it, the state refuses further steps (WD_ERR_POISONED) until
    it is reset, and after the reset the same context produces exactly what a fresh state produces."""
    cfg = synth.get_config("llada8b", **SMALL_BF16)
    w = synth.make_weights(cfg, DEV)
    ids = synth.make_prompts(cfg)
    ctx, st = _small_state(cfg, w, ids)
    want = _steps(st, cfg, 6)
    st.reset(ids)
    _steps(st, cfg, 2)
    first_active = st.plan(0, cfg["A"], cfg["B"], cfg["R"], cfg["T"])["active"][0]
    st.poke_id(0, first_active, cfg["V"] + 5)
    n_enq = 3 if queued else 1
    for _ in range(n_enq):
        st.step(cfg["A"], cfg["B"], cfg["R"], cfg["T"], cfg["k"])
    with pytest.raises(wd.WdError) as e:
        st.sync()
    assert e.value.status == wd.WD_ERR_BOUNDS
    for call in (lambda: st.step(cfg["A"], cfg["B"], cfg["R"], cfg["T"], cfg["k"]),
                 lambda: st.plan(0, cfg["A"], cfg["B"], cfg["R"], cfg["T"]),
                 lambda: st.generate(cfg["A"], cfg["B"], cfg["R"], cfg["T"], cfg["k"])):
        with pytest.raises(wd.WdError) as e:
            call()
        assert e.value.status == wd.WD_ERR_POISONED
    st.reset(ids)
    assert _steps(st, cfg, 6) == want
    st.close(); ctx.close()


def test_state_export_import_resumes_the_trajectory():
    """Checkpoint / resume: the blob holds the sequence state and phase bookkeeping, the caller copies the
    state memory (K/V cache).  Resumed with its cache, a second state continues bit for bit; resumed without
    it, the next step is a refresh step over the same index sets the oracle's planner gives for a state whose
    external window was dropped, and generation runs to the end."""
    from oracle import wd_oracle as wo
    cfg = synth.get_config("llada8b", **dict(SMALL_BF16, batch=2, k=2))
    w = synth.make_weights(cfg, DEV)
    ids = synth.make_prompts(cfg)
    ctx, st = _small_state(cfg, w, ids)
    _steps(st, cfg, 6)                                    # stops mid-phase (R = 4: steps 4, 5 of the second phase done)
    blob = st.export()
    mem = st.mem.clone()
    snap = [st.read(b) for b in range(2)]
    rest = _steps(st, cfg, 7)
    assert [r[0] for r in rest[:3]] == [0, 0, 1]
    # with the cache: identical continuation
    st2 = wd.State(ctx, ids)
    st2.mem.copy_(mem)
    st2.import_(blob, True)
    for b in range(2):
        got = st2.read(b)
        assert all((got[k] == snap[b][k]).all() if hasattr(got[k], "all") else got[k] == snap[b][k] for k in got)
    assert _steps(st2, cfg, 7) == rest
    # without the cache: a refresh first, planned like the oracle plans a state without a stored window
    st3 = wd.State(ctx, ids)
    st3.import_(blob, False)
    for b in range(2):
        ost = wo.SeqState(ids=snap[b]["ids"], decoded=snap[b]["decoded"], t=snap[b]["t"], since=snap[b]["since"],
                          dec_step=np.where(snap[b]["dec_step"] == -(1 << 31), wo.NEVER, snap[b]["dec_step"]), wex=[])
        op = wo.oracle_plan(ost, cfg["A"], cfg["B"], cfg["R"], cfg["T"])
        p = st3.plan(b, cfg["A"], cfg["B"], cfg["R"], cfg["T"])
        assert p["refresh"] and op["refresh"] and p["rows"] == op["rows"] == op["vis"] and p["active"] == op["active"]
        assert p["ext_window"] == op["wex"] and p["transient"] == []
    tail = _steps(st3, cfg, 200)
    assert tail[0][0] == 1 and tail[0][1] == sum(int(s["decoded"].sum()) + cfg["A"] + cfg["B"] for s in snap)
    assert all((st3.read(b)["decoded"]).all() for b in range(2))
    # foreign or damaged blobs change nothing
    for bad in (blob[:40], b"x" * len(blob), blob[:-4]):
        with pytest.raises(wd.WdError) as e:
            st2.import_(bad, True)
        assert e.value.status == wd.WD_ERR_BAD_PARAM
    for s_ in (st, st2, st3):
        s_.close()
    ctx.close()


@pytest.mark.parametrize("shape,batch,R", [(SMALL_BF16, 4, 4), (DH128, 3, 4), (DH128, 8, 3)])
def test_staggered_refresh_variant_matches_its_oracle(shape, batch, R):
    """wd_state_set_stagger (not in the paper): sequence i of the batch shifts its phase clock by i * R / n
    steps, so one call of wd_step carries refresh steps of some sequences (hundreds of rows, all K/V written)
    and normal steps of the others (a few rows, cached K/V read).  Index sets, layer outputs, logits and
    unmask choices follow the oracle run in the same mode; the steps are planned on the device."""
    cfg = synth.get_config("llada8b", **dict(shape, batch=batch, R=R))
    logs = run(cfg, 3 * R + 2, stagger=True)
    for t, l in enumerate(logs):
        kinds = [p["refresh"] for p in l["plans"]]
        want = [t == 0 or (t >= (i * R) // batch and (t - (i * R) // batch) % R == 0) for i in range(batch)]
        assert kinds == want, (t, kinds)
    mixed = [l for l in logs[1:] if any(p["refresh"] for p in l["plans"]) and not all(p["refresh"] for p in l["plans"])]
    assert len(mixed) >= 2 * R                     # refresh and normal steps really share calls
    # the rows of a mixed call: the visible positions of the refreshing sequences plus a few rows of the others
    l = mixed[0]
    assert l["info"]["n_rows"] == sum(len(p["vis"]) if p["refresh"] else len(p["active"]) + len(p["transient"]) for p in l["plans"])


def test_staggered_refresh_queued_steps_match_stepwise_sync():
    """Steps enqueued back to back (planned by the device kernel from counts that now differ per sequence in
    kind) give the same tokens as stepping with a sync after every step."""
    cfg = synth.get_config("llada8b", **dict(DH128, batch=4, R=4))
    w = synth.make_weights(cfg, DEV)
    ids = synth.make_prompts(cfg)
    ctx, st = _small_state(cfg, w, ids)
    st.set_stagger(True)
    want = _steps(st, cfg, 12)
    st.reset(ids)
    got = []
    for _ in range(12):
        st.step(cfg["A"], cfg["B"], cfg["R"], cfg["T"], cfg["k"])
    for r in st.sync_all(32):
        got.append((r["positions"].tolist(), r["token_ids"].tolist(), r["confidence"].tolist()))
    assert got == [(w_[2], w_[3], w_[4]) for w_ in want]
    st.close(); ctx.close()
