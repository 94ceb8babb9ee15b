"""Parity at the benchmark configurations' full DEPTH (GPU required).

The other GPU tests compare one to three transformer blocks; rounding error of the bf16 path
(bf16 GEMM inputs, Q, K/V cache, attention output and FFN hidden; fp32 residual stream) grows
with depth, so the stated tolerances (relative RMS 1e-2 per layer output, 2e-2 max-rel per
attention output, index sets and unmask choices exact) are checked here on the LLaDA-8B-shaped
model with all 32 blocks and on the Dream-7B-shaped model with all 28, teacher-forced, with
the launch configuration the benchmark times.  The fp64 oracle needs about half a minute per
step at these sizes, so the steps are few: the first refresh, the normal steps that follow
(the second one has a transient row), and a refresh from a fast-forwarded late state.

Set WD_DEPTH_CURVE=<file> to also write the per-block error curves as JSON."""
import json
import os

import numpy as np
import pytest
import torch

from paper_2601_20332_b200 import build as wd_build
from paper_2601_20332_b200 import synth
from wd_harness import Parity, TOL_ATTN, TOL_LAYER

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.fixture(scope="module", autouse=True)
def built():
    wd_build.build()


def _dump(name, logs):
    path = os.environ.get("WD_DEPTH_CURVE")
    if not path:
        return
    try:
        old = json.load(open(path))
    except Exception:
        old = {}
    old[name] = [dict(is_refresh=l["info"]["is_refresh"], n_rows=l["info"]["n_rows"], layer=l["curve"]["layer"],
                      attn=l["curve"]["attn"], logits=l["worst"]["logits"]) for l in logs]
    json.dump(old, open(path, "w"))


def _run(cfg, w, ids, decoded, n_steps, oracle_seqs):
    batch, S = ids.shape
    p = Parity(cfg, w, ids, decoded, oracle_seqs=oracle_seqs, max_rows=batch * S, max_active=batch * cfg["A"])
    logs = [p.step(cfg["A"], cfg["B"], cfg["R"], cfg["T"], cfg["k"]) for _ in range(n_steps)]
    p.check_state_mirror()
    p.close()
    return logs


def _check_curve(logs, L):
    for l in logs:
        assert len(l["curve"]["layer"]) == L
        assert max(l["curve"]["layer"]) <= TOL_LAYER and max(l["curve"]["attn"]) <= TOL_ATTN
        assert l["worst"]["ambiguous"] == 0


def test_cfg2_llada8b_all_32_blocks():
    """LLaDA-8B shape at full depth: refresh (352 rows), two normal steps (33 and 34 rows: the second
    recomputes the token the first one unmasked), then a refresh from a state with 100 generated
    tokens (452 rows, 452 visible positions)."""
    cfg = synth.get_config("llada8b")
    assert cfg["L"] == 32
    w = synth.make_weights(cfg, DEV)
    ids = synth.make_prompts(cfg)
    logs = _run(cfg, w, ids, None, 3, [0])
    assert [l["info"]["is_refresh"] for l in logs] == [1, 0, 0]
    assert [l["info"]["n_rows"] for l in logs] == [352, 33, 34]
    _check_curve(logs, 32)
    ids2, dec2 = synth.fast_forward(cfg, ids, 100)
    late = _run(cfg, w, ids2, dec2, 1, [0])
    assert late[0]["info"]["is_refresh"] == 1 and late[0]["info"]["n_rows"] == 256 + 100 + 96
    _check_curve(late, 32)
    _dump("llada8b", logs + late)
    del w
    torch.cuda.empty_cache()


def test_cfg4_dream7b_all_28_blocks():
    """Dream-7B shape (28 query heads over 4 KV heads) at full depth and batch 8; the oracle follows
    sequence 5 through the first refresh (8 x 672 rows on the GPU) and two normal steps (8 x 33, 8 x 34)."""
    cfg = synth.get_config("dream7b")
    assert cfg["L"] == 28
    w = synth.make_weights(cfg, DEV)
    ids = synth.make_prompts(cfg)
    logs = _run(cfg, w, ids, None, 3, [5])
    assert [l["info"]["is_refresh"] for l in logs] == [1, 0, 0]
    assert [l["info"]["n_rows"] for l in logs] == [8 * 672, 8 * 33, 8 * 34]
    _check_curve(logs, 28)
    _dump("dream7b", logs)
    del w
    torch.cuda.empty_cache()
