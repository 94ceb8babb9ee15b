"""Micro-benchmarks of single kernels through the C ABI (CUDA-event timing).

    python -m paper_2601_20332_b200.microbench gemm --rows 34 --n 24576 --k 4096 [--iters 20]
    python -m paper_2601_20332_b200.microbench gemm-suite [--rows 34]
    python -m paper_2601_20332_b200.microbench step --config llada8b --layers 4 [--steps 16]

`gemm` times y = x w^T for one shape (weights larger than L2 unless the shape is
small; a ring of distinct weight buffers keeps every launch cold).  `step` runs
the windowed step on a depth-truncated model.  Both print one JSON line per
measurement; they are also the small cases profiled under ncu.
"""
from __future__ import annotations

import argparse
import json

import numpy as np
import torch

from . import binding as wd
from . import build as wd_build
from . import synth

LLADA_GEMMS = [("qkv", 12288, 4096), ("o", 4096, 4096), ("gate_up", 24576, 4096), ("down", 4096, 12288),
               ("lm_head", 126464, 4096)]


def time_gemm(rows, n, k, iters=20, impl=wd.WD_GEMM_TCGEN05, ring_bytes=600 << 20):
    dev = "cuda:0"
    g = torch.Generator(device=dev).manual_seed(1)
    wbytes = n * k * 2
    n_ring = max(2, min(8, ring_bytes // wbytes + 1))
    ws = [(torch.randn(n, k, device=dev, generator=g) * 0.02).to(torch.bfloat16) for _ in range(n_ring)]
    x = torch.randn(rows, k, device=dev, generator=g).to(torch.bfloat16)
    nb = wd.lib().wd_op_gemm_scratch_bytes(rows, n, k)
    scratch = torch.empty(max(nb, 256), dtype=torch.uint8, device=dev)
    for i in range(3):
        wd.op_gemm(x, ws[i % n_ring], impl, scratch=scratch)
    torch.cuda.synchronize()
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(iters + 1)]
    ev[0].record()
    for i in range(iters):
        wd.op_gemm(x, ws[i % n_ring], impl, scratch=scratch)
        ev[i + 1].record()
    torch.cuda.synchronize()
    assert wd.op_status() == 0
    ts = np.array([ev[i].elapsed_time(ev[i + 1]) for i in range(iters)])
    by = wbytes + rows * k * 2 + rows * n * 4
    return dict(rows=rows, n=n, k=k, us_median=float(np.median(ts) * 1e3), us_min=float(ts.min() * 1e3),
                algorithmic_bytes=by, gbs_median=by / (np.median(ts) * 1e-3) / 1e9,
                note="includes the split-K reduce kernel of the single-op entry point")


def run_step(config, layers, steps, warmup, impl):
    dev = "cuda:0"
    cfg = synth.get_config(config, L=layers)
    A, B, R, T, k, batch = (cfg[x] for x in ("A", "B", "R", "T", "k", "batch"))
    S = cfg["P"] + cfg["G"]
    w = synth.make_weights(cfg, dev)
    ids = synth.make_prompts(cfg)
    ctx = wd.Context(cfg, w, batch, S, batch * S, batch * A)
    ctx.set_gemm_impl(impl)
    st = wd.State(ctx, ids)
    stream = torch.cuda.Stream(device=dev)
    out = []
    for i in range(warmup + steps):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        _, info = st.step(A, B, R, T, k, stream)
        e1.record(stream)
        st.sync()
        torch.cuda.synchronize()
        if i >= warmup:
            out.append((info, e0.elapsed_time(e1)))
    normal = [t for i, t in out if not i["is_refresh"]]
    refresh = [t for i, t in out if i["is_refresh"]]
    return dict(config=config, layers=layers, normal_ms=float(np.median(normal)) if normal else None,
                refresh_ms=float(np.median(refresh)) if refresh else None, launches=out[-1][0]["n_launches"],
                rows=out[-1][0]["n_rows"])


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("mode", choices=["gemm", "gemm-suite", "step"])
    ap.add_argument("--rows", type=int, default=34)
    ap.add_argument("--n", type=int, default=24576)
    ap.add_argument("--k", type=int, default=4096)
    ap.add_argument("--iters", type=int, default=20)
    ap.add_argument("--config", default="llada8b")
    ap.add_argument("--layers", type=int, default=4)
    ap.add_argument("--steps", type=int, default=16)
    ap.add_argument("--warmup", type=int, default=8)
    ap.add_argument("--plain", action="store_true")
    a = ap.parse_args()
    wd_build.build()
    impl = wd.WD_GEMM_PLAIN if a.plain else wd.WD_GEMM_TCGEN05
    if a.mode == "gemm":
        print(json.dumps(time_gemm(a.rows, a.n, a.k, a.iters, impl)))
    elif a.mode == "gemm-suite":
        for name, n, k in LLADA_GEMMS:
            r = time_gemm(a.rows, n, k, a.iters, impl)
            r["name"] = name
            print(json.dumps(r))
    else:
        print(json.dumps(run_step(a.config, a.layers, a.steps, a.warmup, impl)))


if __name__ == "__main__":
    main()
