"""Micro-benchmarks of single kernels through the C ABI (CUDA-event timing).

    python -m paper_2601_20332_b200.microbench gemm --rows 34 --n 24576 --k 4096 [--iters 20]
    python -m paper_2601_20332_b200.microbench gemm-fp4 --rows 34 --n 24576 --k 4096 [--iters 20]
    python -m paper_2601_20332_b200.microbench gemm-suite [--rows 34]
    python -m paper_2601_20332_b200.microbench step --config llada8b --layers 4 [--steps 16]
    python -m paper_2601_20332_b200.microbench sweep [--A 16,32,64,128 --B 64,128,256 --R 1,4,16 --batch 1,16]
    python -m paper_2601_20332_b200.microbench stamps --layers 4 --steps 6      (a -DWD_GEMM_TRACE build)

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
                tflops_median=2.0 * rows * n * k / (np.median(ts) * 1e-3) / 1e12,
                note="includes the split-K reduce kernel of the single-op entry point")


def time_gemm_fp4(rows, n, k, iters=20, ring_bytes=600 << 20):
    """The NVFP4 GEMM alone on operands quantised beforehand (a ring of distinct weights keeps every launch cold)."""
    dev = "cuda:0"
    g = torch.Generator(device=dev).manual_seed(1)
    wbytes = n * k * 9 // 16
    n_ring = max(2, min(8, ring_bytes // wbytes + 1))
    wqs = []
    for _ in range(n_ring):
        w = (torch.randn(n, k, device=dev, generator=g) * 0.02).to(torch.bfloat16)
        wqs.append(wd.op_nvfp4_quantize(w))
        del w
    xq = wd.op_nvfp4_quantize(torch.randn(rows, k, device=dev, generator=g).to(torch.bfloat16))
    nb = wd.lib().wd_op_gemm_scratch_bytes(rows, n, k)
    scratch = torch.empty(max(nb, 256), dtype=torch.uint8, device=dev)
    for i in range(3):
        wd.op_gemm_nvfp4(xq, wqs[i % n_ring], rows, n, k, scratch=scratch)
    torch.cuda.synchronize()
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(iters + 1)]
    ev[0].record()
    for i in range(iters):
        wd.op_gemm_nvfp4(xq, wqs[i % n_ring], rows, n, k, scratch=scratch)
        ev[i + 1].record()
    torch.cuda.synchronize()
    assert wd.op_status() == 0
    ts = np.array([ev[i].elapsed_time(ev[i + 1]) for i in range(iters)])
    by = (n + rows) * k * 9 // 16 + rows * n * 4
    return dict(kind="nvfp4", rows=rows, n=n, k=k, us_median=float(np.median(ts) * 1e3), us_min=float(ts.min() * 1e3),
                algorithmic_bytes=by, gbs_median=by / (np.median(ts) * 1e-3) / 1e9,
                tflops_median=2.0 * rows * n * k / (np.median(ts) * 1e-3) / 1e12,
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


def run_stamps(config, layers, steps):
    """Clock stamps of the last block's GEMM launches (a library built with -DWD_GEMM_TRACE: `WD_NVCC_FLAGS=-DWD_GEMM_TRACE
    python -m paper_2601_20332_b200.build`): per launch and event the minimum, median and maximum over the CTAs, in
    nanoseconds after the first CTA's dependency wait returned (output projection: after the attention kernel's last
    CTA left)."""
    import ctypes as C
    lib = wd.lib()
    if not hasattr(lib, "wd_debug_gemm_trace"):
        raise SystemExit("this libwd.so was built without -DWD_GEMM_TRACE")
    dev = "cuda:0"
    cfg = synth.get_config(config, L=layers)
    A, B, R, T, k, batch = (cfg[x] for x in ("A", "B", "R", "T", "k", "batch"))
    S = cfg["P"] + cfg["G"]
    w = synth.make_weights(cfg, dev)
    ctx = wd.Context(cfg, w, batch, S, batch * S, batch * A)
    st = wd.State(ctx, synth.make_prompts(cfg))
    stream = torch.cuda.Stream(device=dev)
    for _ in range(steps):
        st.step(A, B, R, T, k, stream)
        st.sync()
    torch.cuda.synchronize()
    buf = np.zeros((8, 160, 8), np.uint64)
    lib.wd_debug_gemm_trace(buf.ctypes.data_as(C.c_void_p))
    ab = np.zeros(64, np.uint64)
    lib.wd_debug_attn_trace(ab.ctypes.data_as(C.c_void_p))
    names = ["qkv", "o", "gate_up", "down"]
    events = ["entry", "ring filled (before the wait)", "wait returned", "first stage complete", "last MMA issued",
              "last accumulator ready", "epilogue done", "exit"]
    out = {}
    for slot, name in enumerate(names):
        t = buf[slot, :148, :].astype(np.int64)
        t = t[t[:, 0] > 0]
        if not len(t):
            continue
        ref = int(ab[layers - 1]) if name == "o" and ab[layers - 1] else int(t[:, 2].min())
        out[name] = {e: [int((t[:, i] - ref).min()), int(np.median(t[:, i] - ref)), int((t[:, i] - ref).max())]
                     for i, e in enumerate(events)}
    return dict(config=config, layers=layers, ctas=148, ns_min_median_max=out)


def run_sweep(config, layers, A_list, B_list, R_list, batch_list, repeats, out_path):
    """Window sweep (benchmark configuration 5): for every (A, B, R, batch) one full phase
    (R steps) from three fast-forwarded states (0 %, 50 %, ~100 % of the masks decoded), with the
    per-step window-token counts and K/V-cache bytes logged next to each timing (JSON lines)."""
    dev = "cuda:0"
    cfg = synth.get_config(config) if layers is None else synth.get_config(config, L=layers)
    S, G, P, T, k = cfg["P"] + cfg["G"], cfg["G"], cfg["P"], cfg["T"], cfg["k"]
    w = synth.make_weights(cfg, dev)
    max_b, max_a = max(batch_list), max(A_list)
    ctx = wd.Context(cfg, w, max_b, S, max_b * S, max_b * max_a)
    stream = torch.cuda.Stream(device=dev)
    kv_tok = 2 * cfg["Hkv"] * cfg["dh"] * 2 * cfg["L"]
    lines = []
    for batch in batch_list:
        base_ids = synth.make_prompts(cfg, batch=batch)
        st = None
        for A in A_list:
            for B in B_list:
                for R in R_list:
                    for frac in (0.0, 0.5, 1.0):
                        n_dec = min(int(G * frac), G - (A + B))         # keep a full window undecoded
                        ids, dec = synth.fast_forward(cfg, base_ids, max(n_dec, 0))
                        if st is None:
                            st = wd.State(ctx, ids, dec)
                        best = None
                        for rep in range(repeats):
                            st.reset(ids, dec, stream)
                            steps = []
                            for i in range(R):
                                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                                e0.record(stream)
                                _, info = st.step(A, B, R, T, k, stream)
                                e1.record(stream)
                                st.sync()
                                torch.cuda.synchronize()
                                steps.append(dict(us=e0.elapsed_time(e1) * 1e3, refresh=info["is_refresh"],
                                                  rows=info["n_rows"], active=info["n_active"], vis=info["n_vis"]))
                            tot = sum(x["us"] for x in steps)
                            if best is None or tot < best[0]:
                                best = (tot, steps)
                        tot, steps = best
                        rec = dict(config=config, layers=cfg["L"], A=A, B=B, R=R, T=T, k=k, batch=batch,
                                   decoded_frac=frac, phase_us=tot, us_per_step=tot / R,
                                   tokens_per_s=batch * k * R / (tot * 1e-6),
                                   window_tokens_per_seq=A + B, kv_cache_bytes_resident=batch * S * kv_tok,
                                   steps=[dict(s, kv_bytes_read=s["vis"] * kv_tok, kv_bytes_written=s["rows"] * kv_tok)
                                          for s in steps])
                        lines.append(rec)
                        print(json.dumps(rec), flush=True)
        if st is not None:
            st.close()
    if out_path:
        with open(out_path, "w") as f:
            for r in lines:
                f.write(json.dumps(r) + "\n")


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("mode", choices=["gemm", "gemm-fp4", "gemm-suite", "step", "sweep", "stamps"])
    ap.add_argument("--rows", type=int, default=34)
    ap.add_argument("--n", type=int, default=24576)
    ap.add_argument("--k", type=int, default=4096)
    ap.add_argument("--iters", type=int, default=20)
    ap.add_argument("--config", default="llada8b")
    ap.add_argument("--layers", type=int, default=4)
    ap.add_argument("--steps", type=int, default=16)
    ap.add_argument("--warmup", type=int, default=8)
    ap.add_argument("--plain", action="store_true")
    ap.add_argument("--A", default="16,32,64,128")
    ap.add_argument("--B", default="64,128,256")
    ap.add_argument("--R", default="1,4,16")
    ap.add_argument("--batch", default="1,16")
    ap.add_argument("--repeats", type=int, default=3)
    ap.add_argument("--out", default=None)
    a = ap.parse_args()
    wd_build.build()
    impl = wd.WD_GEMM_PLAIN if a.plain else wd.WD_GEMM_TCGEN05
    if a.mode == "gemm":
        print(json.dumps(time_gemm(a.rows, a.n, a.k, a.iters, impl)))
    elif a.mode == "stamps":
        print(json.dumps(run_stamps(a.config, a.layers, a.steps)))
    elif a.mode == "gemm-fp4":
        print(json.dumps(time_gemm_fp4(a.rows, a.n, a.k, a.iters)))
    elif a.mode == "gemm-suite":
        for name, n, k in LLADA_GEMMS:
            r = time_gemm(a.rows, n, k, a.iters, impl)
            r["name"] = name
            print(json.dumps(r))
    elif a.mode == "sweep":
        ints = lambda v: [int(x) for x in v.split(",")]
        run_sweep(a.config if a.config != "llada8b" else "llada8b_sweep", None if a.layers == 4 else a.layers,
                  ints(a.A), ints(a.B), ints(a.R), ints(a.batch), a.repeats, a.out)
    else:
        print(json.dumps(run_step(a.config, a.layers, a.steps, a.warmup, impl)))


if __name__ == "__main__":
    main()
