"""Parity at the benchmark configurations' full widths (GPU required).

The five configurations are run with their real model width, head layout, FFN
width, vocabulary, sequence lengths, window sizes and batch, but with ONE
transformer block instead of 28/32: the fp64 oracle needs 5-110 TFLOP for a
full-depth refresh step, and depth only repeats the same kernels with the same
launch configuration.  Steps compared per config: the first refresh, the normal
steps of the phase (transients appear), the next refresh; for batches the
oracle follows a subset of the sequences (they are independent)."""
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


def run_cfg(cfg, n_steps, oracle_seqs=None, ids=None, decoded=None, refresh_mode=0, fp8=False, tol=None, fp4=False):
    w = synth.make_weights(cfg, DEV)
    ids = synth.make_prompts(cfg) if ids is None else ids
    batch, S = ids.shape
    p = Parity(cfg, w, ids, decoded, oracle_seqs=oracle_seqs, max_rows=batch * S, max_active=batch * cfg["A"],
               refresh_mode=refresh_mode, fp8=fp8, fp4=fp4)
    logs = []
    for _ in range(n_steps):
        if tol is None:
            logs.append(p.step(cfg["A"], cfg["B"], cfg["R"], cfg["T"], cfg["k"]))
        else:
            logs.append(p.step(cfg["A"], cfg["B"], cfg["R"], cfg["T"], cfg["k"], tol_layer=tol[0], tol_attn=tol[1]))
    p.check_state_mirror()
    p.close()
    del w
    torch.cuda.empty_cache()
    return logs


def test_cfg2_llada8b_shape():
    """LLaDA-8B width, prompt 256 + 256 masks, A=32 B=64 R=8 T=2, one token per step."""
    cfg = synth.get_config("llada8b", L=1)
    logs = run_cfg(cfg, 9)
    assert [l["info"]["is_refresh"] for l in logs] == [1, 0, 0, 0, 0, 0, 0, 0, 1]
    assert logs[0]["info"]["n_rows"] == 352 and logs[3]["info"]["n_rows"] == 34
    assert sum(l["worst"]["ambiguous"] for l in logs) == 0


def test_cfg3_llada8b_long_two_tokens_and_full_sequence_step():
    """prompt 512 + 1024 masks, A=64 B=128, two tokens per step; then the no-pruning step."""
    cfg = synth.get_config("llada8b_long", L=1)
    logs = run_cfg(cfg, 3)
    assert logs[0]["info"]["n_rows"] == 704 and logs[1]["info"]["n_rows"] == 64 + 2
    assert all(l["res"]["n_unmasked"][0] == 2 for l in logs)
    full = dict(cfg, A=cfg["G"], B=0, R=1, T=0)
    logs = run_cfg(full, 1)
    assert logs[0]["info"]["n_rows"] == 1536 and logs[0]["info"]["n_active"] == 1024


def test_cfg4_dream7b_shape_gqa_batch8():
    """Dream-7B width (28 query heads over 4 KV heads), batch 8 with independent windows."""
    cfg = synth.get_config("dream7b", L=1)
    logs = run_cfg(cfg, 5, oracle_seqs=[0, 5])
    assert [l["info"]["is_refresh"] for l in logs] == [1, 0, 0, 0, 1]
    assert logs[0]["info"]["n_rows"] == 8 * 672 and logs[3]["info"]["n_rows"] == 8 * 35
    pos = logs[0]["res"]["positions"][:, 0]
    assert len(set(pos.tolist())) > 1                     # the windows really are independent


def test_cfg4_gate_up_launch_writes_swiglu_itself():
    """At the Dream-7B width every CTA pair gets two whole (gate tile, up tile) units, so the gate/up
    GEMM's epilogue writes h = silu(gate) * up and no SwiGLU kernel runs: one launch fewer per block
    than at the LLaDA-8B width with 352 rows (96 units for 74 pairs: partial sums + SwiGLU kernel).
    The parity of that path is what test_cfg4_dream7b_shape_gqa_batch8 checks."""
    if any(os.environ.get(k) == "0" for k in ("WD_GEMM_DUAL", "WD_GEMM_SWIGLU", "WD_GEMM_PAIR_FROM")):
        pytest.skip("the SwiGLU epilogue is switched off by a tuning knob")
    counts = {}
    for name in ("llada8b", "dream7b"):
        cfg = synth.get_config(name, L=1)
        w = synth.make_weights(cfg, DEV)
        ids = synth.make_prompts(cfg)
        batch, S = ids.shape
        ctx = wd.Context(cfg, w, batch, S, batch * S, batch * cfg["A"])
        st = wd.State(ctx, ids)
        _, info = st.step(cfg["A"], cfg["B"], cfg["R"], cfg["T"], cfg["k"])
        st.sync()
        assert info["is_refresh"] == 1 and info["n_rows"] > 256
        counts[name] = info["n_launches"]
        del st, ctx, w
        torch.cuda.empty_cache()
    assert counts["dream7b"] == counts["llada8b"] - 1


def test_cfg5_sweep_corner_late_state():
    """Window sweep corner A=128 B=256 R=4, prompt 1024 + 2048 masks, batch 2, from a
    half-decoded state (2048 visible positions)."""
    cfg = synth.get_config("llada8b_sweep", L=1, A=128, B=256, R=4, batch=2)
    ids, dec = synth.fast_forward(cfg, synth.make_prompts(cfg), 640)
    logs = run_cfg(cfg, 3, oracle_seqs=[1], ids=ids, decoded=dec)
    assert logs[0]["info"]["n_rows"] == 2 * (1024 + 640 + 384)
    assert logs[1]["info"]["n_rows"] == 2 * 129 and logs[1]["info"]["n_vis"] == 2 * 2048


def test_cfg5_sweep_batch8_small_window_many_key_tiles():
    """Sweep point A=16 B=64 R=16 at batch 8: 256 attention CTAs (two waves) of nine key tiles with 17
    valid query rows each, K/V streamed from HBM.  The softmax warps run a tile ahead of the MMA thread
    here (it waits for V first), which a single 'P written' barrier did not survive."""
    cfg = synth.get_config("llada8b_sweep", L=1, A=16, B=64, R=16, batch=8)
    logs = run_cfg(cfg, 3, oracle_seqs=[3])
    assert [l["info"]["is_refresh"] for l in logs] == [1, 0, 0]
    assert logs[1]["info"]["n_rows"] == 8 * 17 and logs[1]["info"]["n_vis"] == 8 * 1104


def test_cfg2_window_only_refresh_variant_at_full_width():
    """The variant outside the paper at the LLaDA-8B width: the second refresh computes the new
    window and the previous phase's tokens only (104 rows instead of 360)."""
    cfg = synth.get_config("llada8b", L=1)
    logs = run_cfg(cfg, 9, refresh_mode=wd.WD_REFRESH_WINDOW)
    assert [l["info"]["is_refresh"] for l in logs] == [1, 0, 0, 0, 0, 0, 0, 0, 1]
    assert logs[0]["info"]["n_rows"] == 352 and logs[8]["info"]["n_rows"] == 96 + 8 and logs[8]["info"]["n_vis"] == 360


def test_cfg2_and_cfg4_fp8_projections_at_full_width():
    """FP8 mode (outside the paper) at the real widths: LLaDA-8B shape (vocabulary 126464 through
    the FP8 LM-head epilogue) and the Dream-7B shape (GQA, batch 8, d_ffn 18944, two-CTA FP8
    GEMMs at 5376 rows); tolerances as derived in test_gpu_step."""
    logs = run_cfg(synth.get_config("llada8b", L=1), 3, fp8=True, tol=(5e-2, 1e-1))
    assert logs[0]["info"]["n_rows"] == 352 and logs[1]["info"]["n_rows"] == 33
    logs = run_cfg(synth.get_config("dream7b", L=1), 2, oracle_seqs=[3], fp8=True, tol=(5e-2, 1e-1))
    assert logs[0]["info"]["n_rows"] == 8 * 672 and logs[1]["info"]["n_rows"] == 8 * 33


def test_cfg2_and_cfg4_nvfp4_projections_at_full_width():
    """NVFP4 mode (outside the paper) at the real layer widths: the LLaDA-8B block (d 4096, d_ffn 12288,
    refresh at 352 rows and a normal step at 33) and the Dream-7B block's refresh (GQA, batch 8, d 3584, d_ffn 18944,
    5376 rows: several token tiles per weight tile).  The vocabulary is cut to 16384 rows to keep the
    oracle's block-by-block product within seconds; tolerances as derived in test_gpu_step."""
    logs = run_cfg(synth.get_config("llada8b", L=1, V=16384), 2, fp4=True, tol=(1.5e-1, 1e-1))
    assert logs[0]["info"]["n_rows"] == 352 and logs[1]["info"]["n_rows"] == 33
    assert max(l["worst"]["logits"] for l in logs) < 2.5e-1
    logs = run_cfg(synth.get_config("dream7b", L=1, V=16384), 1, oracle_seqs=[3], fp4=True, tol=(1.5e-1, 1e-1))
    assert logs[0]["info"]["n_rows"] == 8 * 672
    assert max(l["worst"]["logits"] for l in logs) < 2.5e-1
