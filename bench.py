#!/usr/bin/env python
"""Benchmark of the windowed denoising step on B200.

Default workload: the LLaDA-8B-shaped bf16 configuration (32 layers, d 4096,
32 heads x 128, FFN 12288, vocab 126464; prompt 256 + 256 masks; A=32, B=64,
R=8, T=2, one token per step, batch 1) with seeded random-init weights and
uniform-random prompt ids.  A "step" is one wd_step + wd_step_sync of the
generation trajectory (one refresh step then R-1 normal steps per phase).

Prints ONE JSON line.  `value` is generated tokens/s with the state resident
on the GPU; `e2e` is a whole generation through the library's own driver on the
host clock from host buffers (prompt ids uploaded, every step's result block
copied down, final ids read back; `e2e.per_step_sync` = the timed steps with a
host sync after each); `roofline` is the tensor-core GEMM kernel's algorithmic bytes over its
CUDA-event time; `cpu_baseline` is the fp64 oracle timed on the host cores.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference] [--config NAME]
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np
import torch

from paper_2601_20332_b200 import synth

METRIC = "generated tokens/s (windowed denoising steps, LLaDA-8B shape, 1 B200)"
UNIT = "tokens/s"


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return dict(hbm_gbs=float(d["hbm_gbs"]), bf16_tflops=float(d["bf16_tflops"]),
                    bf16_tflops_sustained=float(d.get("bf16_tflops_sustained", d["bf16_tflops"])), source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, source="fallback")


class ClockSampler:
    """nvidia-smi clocks and throttle reasons sampled while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu, self.proc, self.path = gpu_index, None, None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.gpu}", f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "50"],
                                         stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self) -> dict:
        out = dict(sm_mhz=None, sm_max_mhz=None, reasons=[], samples=0)
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        try:
            for line in open(self.path):
                f = [c.strip() for c in line.split(",")]
                if len(f) < 9:
                    continue
                try:
                    sm.append(float(f[1])); mx.append(float(f[2]))
                except ValueError:
                    continue
                for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[5:9]):
                    if v.lower().startswith("active"):
                        reasons.add(name)
            os.unlink(self.path)
        except Exception:
            pass
        if sm:
            out.update(sm_mhz=float(np.median(sm)), sm_max_mhz=float(max(mx)), reasons=sorted(reasons), samples=len(sm))
        return out


def weight_bytes(cfg) -> float:
    """Bytes of all matrices a step reads once: the transformer blocks and the LM head."""
    L, d, Hq, Hkv, dh, F, V = (cfg[k] for k in ("L", "d", "Hq", "Hkv", "dh", "F", "V"))
    w = 2 if cfg["dtype"] == "bf16" else 4
    return float((d * (Hq + 2 * Hkv) * dh + Hq * dh * d + 3 * d * F) * L * w + V * d * w)


def shape_name(cfg) -> str:
    kind = {"llada8b": "LLaDA-8B-shaped", "llada8b_long": "LLaDA-8B-shaped", "llada8b_sweep": "LLaDA-8B-shaped",
            "dream7b": "Dream-7B-shaped", "tiny": "tiny"}.get(cfg.get("name", ""), cfg.get("name", "model"))
    heads = f"{cfg['Hq']} heads" if cfg["Hq"] == cfg["Hkv"] else f"{cfg['Hq']} query / {cfg['Hkv']} KV heads"
    return (f"{kind} {cfg['dtype']} ({cfg['L']} layers, d {cfg['d']}, {heads} x {cfg['dh']}, FFN {cfg['F']}, "
            f"vocab {cfg['V']})")


def algorithmic_step(cfg, rows, n_act, vis, batch=1):
    """Bytes and FLOPs the method itself must move / compute in one step
    (weights once, K/V of the visible positions read, fresh K/V written)."""
    L, d, Hq, Hkv, dh, F, V = (cfg[k] for k in ("L", "d", "Hq", "Hkv", "dh", "F", "V"))
    w = 2 if cfg["dtype"] == "bf16" else 4
    per_layer = d * (Hq + 2 * Hkv) * dh + Hq * dh * d + 3 * d * F
    kv_tok = 2 * Hkv * dh * w * L
    by = per_layer * L * w + V * d * w + vis * kv_tok + rows * kv_tok
    fl = 2 * rows * per_layer * L + 2 * n_act * d * V + 4 * rows * (vis / max(batch, 1)) * Hq * dh * L
    return by, fl


def phase_amortised(normal_ms, refresh_ms, R, tokens_per_step):
    """A phase is one refresh step and R-1 normal steps; the K timed steps need not hold refresh steps in
    that proportion, so the per-step time of a whole phase is also given: (refresh + (R-1) normal) / R
    from the medians of the two kinds."""
    if not refresh_ms or (R > 1 and not normal_ms):
        return None
    r = float(np.median(refresh_ms))
    n = float(np.median(normal_ms)) if normal_ms else 0.0
    ms = (r + (R - 1) * n) / R
    return {"ms_per_step": ms, "value": tokens_per_step / (ms * 1e-3), "unit": UNIT}


def max_over_ranks(ms: float, world: int, device) -> float:
    """A multi-rank run is as slow as its slowest rank: all-reduce MAX of the device-timed region
    (NCCL between GPUs; the CPU tests run the same code over gloo)."""
    if world <= 1:
        return float(ms)
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    torch.distributed.all_reduce(t, op=torch.distributed.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(units_per_rank: float, world: int, total_ms: float) -> float:
    """Replicas only: every rank processes the same number of units, no data-path collective."""
    return units_per_rank * world / (total_ms * 1e-3)


def run_ours(args, rank, world):
    from paper_2601_20332_b200 import binding as wd
    from paper_2601_20332_b200 import build as wd_build
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dev = f"cuda:{local}"
    wd_build.build()
    wd.lib()
    cfg = synth.get_config(args.config)
    A, B, R, T, k, batch = (cfg[x] for x in ("A", "B", "R", "T", "k", "batch"))
    S = cfg["P"] + cfg["G"]
    K, W = args.steps, args.warmup
    w = synth.make_weights(cfg, dev)
    ids = synth.make_prompts(cfg)
    ctx = wd.Context(cfg, w, batch, S, batch * S, batch * max(A, cfg["G"]))
    stream = torch.cuda.Stream(device=dev)
    peaks = measured_peaks()

    def trajectory(n_warm, n_timed, state, per_step_cb=None, queued=False):
        """queued: steps are enqueued back to back (the device plans them) and drained every
        `QUEUE` steps; otherwise every step is followed by a sync."""
        QUEUE = 16
        infos, per_step = [], []
        pending = [False]

        def one_step():
            # a generation that runs out of masks starts again from the prompt (the first step of
            # the new generation is a refresh like any other)
            status, info = state.step(A, B, R, T, k, stream)
            if status == wd.WD_DONE:
                if pending[0]:
                    state.sync()
                    pending[0] = False
                state.reset(ids, None, stream)
                status, info = state.step(A, B, R, T, k, stream)
            pending[0] = True
            return info

        for i in range(n_warm):
            one_step()
            state.sync()
            pending[0] = False
        if world > 1:
            torch.distributed.barrier()
        torch.cuda.synchronize()
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(n_timed + 1)]
        t0 = time.perf_counter()
        ev[0].record(stream)
        for i in range(n_timed):
            info = one_step()
            ev[i + 1].record(stream)
            if not queued or (i + 1) % QUEUE == 0 or i + 1 == n_timed:
                state.sync()
                pending[0] = False
            infos.append(info)
            if per_step_cb:
                per_step_cb(info)
        torch.cuda.synchronize()
        wall = time.perf_counter() - t0
        if world > 1:
            torch.distributed.barrier()
        per_step = [ev[i].elapsed_time(ev[i + 1]) for i in range(n_timed)]
        return infos, per_step, ev[0].elapsed_time(ev[n_timed]), wall

    # ---- device-resident run: the headline value
    state = wd.State(ctx, ids)
    sampler = ClockSampler(local)
    sampler.start()
    infos, per_step, total_ms, _ = trajectory(W, K, state, queued=True)
    # ---- same trajectory again with GEMM events: roofline of the dominant kernel
    state.reset(ids, None, stream)
    ctx.profile_enable(True)
    kinds = {0: dict(gemm_ms=0.0, gemm_bytes=0.0, gemm_launches=0, flops=0.0),
             1: dict(gemm_ms=0.0, gemm_bytes=0.0, gemm_launches=0, flops=0.0)}
    last = dict(gemm_ms=0.0, gemm_bytes=0.0, gemm_launches=0)
    per_layer = cfg["d"] * (cfg["Hq"] + 2 * cfg["Hkv"]) * cfg["dh"] + cfg["Hq"] * cfg["dh"] * cfg["d"] + 3 * cfg["d"] * cfg["F"]

    def on_step(info):
        now = ctx.profile_read()
        kk = kinds[1 if info["is_refresh"] else 0]
        for key in last:
            kk[key] += now[key] - last[key]
            last[key] = now[key]
        kk["flops"] += 2.0 * info["n_rows"] * per_layer * cfg["L"] + 2.0 * info["n_active"] * cfg["d"] * cfg["V"]

    def step_sync(state):
        status, _ = state.step(A, B, R, T, k, stream)
        if status == wd.WD_DONE:                      # out of masks: start again from the prompt
            state.reset(ids, None, stream)
            state.step(A, B, R, T, k, stream)
        state.sync()

    def warm_then_time(n_warm, n_timed, state):
        # warm-up steps must not count: reset the totals after them
        for i in range(n_warm):
            step_sync(state)
        now = ctx.profile_read()
        last.update({key: now[key] for key in last})
        return trajectory(0, n_timed, state, on_step)

    warm_then_time(W, K, state)
    prof = kinds[0] if kinds[0]["gemm_launches"] else kinds[1]
    prof_refresh = kinds[1]
    ctx.profile_enable(False)
    clocks = sampler.stop()
    # ---- end to end from host buffers on the host clock
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    state.reset(ids, None, stream)
    for i in range(W + K):
        step_sync(state)
    torch.cuda.synchronize()
    e2e_wall = time.perf_counter() - t0
    # ---- the window-only refresh variant (NOT the paper's method; reported beside the headline, never as it)
    state.reset(ids, None, stream)
    state.set_refresh_mode(wd.WD_REFRESH_WINDOW)
    v_infos, v_per_step, v_total_ms, _ = trajectory(W, K, state, queued=True)
    v_total_ms = max_over_ranks(v_total_ms, world, dev)
    v_refresh = [t for t, i in zip(v_per_step, v_infos) if i["is_refresh"]]
    state.set_refresh_mode(wd.WD_REFRESH_FULL)
    # ---- FP8 projections (an option outside the paper; never the headline, which stays bf16)
    fp8_line = None
    if cfg["dtype"] == "bf16":
        ctx.fp8_enable(stream)
        state.reset(ids, None, stream)
        f_infos, f_per_step, f_total_ms, _ = trajectory(W, K, state, queued=True)
        f_total_ms = max_over_ranks(f_total_ms, world, dev)
        f_normal = [t for t, i in zip(f_per_step, f_infos) if not i["is_refresh"]]
        f_refresh = [t for t, i in zip(f_per_step, f_infos) if i["is_refresh"]]
        fp8_line = {"note": "NOT the headline precision: e4m3 weights and activations with per-row scales for q/k/v, "
                            "gate/up, down and the LM head (fp32 accumulation); everything else as in the bf16 run",
                    "value": whole_job_value(batch * k * K, world, f_total_ms), "unit": UNIT,
                    "normal_step_ms": float(np.median(f_normal)) if f_normal else None,
                    "refresh_step_ms": float(np.median(f_refresh)) if f_refresh else None}
        ctx.fp8_set(False)
    # ---- NVFP4 projections (outside the paper too; 4-bit codes with block scales on the block-scaled tensor-core path)
    fp4_line = None
    if cfg["dtype"] == "bf16" and cfg["d"] % 256 == 0 and cfg["F"] % 256 == 0:
        ctx.fp4_enable(stream)
        state.reset(ids, None, stream)
        q_infos, q_per_step, q_total_ms, _ = trajectory(W, K, state, queued=True)
        q_total_ms = max_over_ranks(q_total_ms, world, dev)
        q_normal = [t for t, i in zip(q_per_step, q_infos) if not i["is_refresh"]]
        q_refresh = [t for t, i in zip(q_per_step, q_infos) if i["is_refresh"]]
        fp4_line = {"note": "NOT the headline precision: NVFP4 (e2m1 codes, e4m3 scale per 16 elements, float scale per row) "
                            "weights and activations for q/k/v, gate/up, down and the LM head (fp32 accumulation); "
                            "everything else as in the bf16 run",
                    "value": whole_job_value(batch * k * K, world, q_total_ms), "unit": UNIT,
                    "normal_step_ms": float(np.median(q_normal)) if q_normal else None,
                    "refresh_step_ms": float(np.median(q_refresh)) if q_refresh else None}
        ctx.fp4_set(False)
    # ---- a whole generation through the library's own driver: host prompt in, host tokens out
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    state.reset(ids, None, stream)
    _, gen_steps, gen_tokens = state.generate(A, B, R, T, k, 0, stream)
    final_ids = [state.read(b)["ids"] for b in range(batch)]
    gen_wall = time.perf_counter() - t0
    assert gen_tokens == batch * cfg["G"] and all((f != cfg["mask_id"]).all() for f in final_ids)
    # ---- the full-sequence no-pruning step at the same starting state, for context
    state.reset(ids, None, stream)
    full_ms = []
    for i in range(4):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        state.step(cfg["G"], 0, 1, 0, k, stream)
        e1.record(stream)
        state.sync()
        torch.cuda.synchronize()
        full_ms.append(e0.elapsed_time(e1))
    state.close()

    total_ms = max_over_ranks(total_ms, world, dev)
    value = whole_job_value(batch * k * K, world, total_ms)
    normal = [t for t, i in zip(per_step, infos) if not i["is_refresh"]]
    refresh = [t for t, i in zip(per_step, infos) if i["is_refresh"]]
    # roofline of the GEMM kernel: algorithmic bytes per launch / average launch time
    n_l = max(prof["gemm_launches"], 1)
    gemm_gbs = prof["gemm_bytes"] / (prof["gemm_ms"] * 1e-3) / 1e9 if prof["gemm_ms"] > 0 else 0.0
    # whole-step roofline for the normal step (HBM bound)
    ni = [i for i in infos if not i["is_refresh"]]
    step_by, step_fl = algorithmic_step(cfg, np.mean([i["n_rows"] for i in ni]) if ni else 0,
                                        np.mean([i["n_active"] for i in ni]) if ni else 0,
                                        np.mean([i["n_vis"] for i in ni]) if ni else 0, batch)
    normal_ms = float(np.median(normal)) if normal else None
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": W,
        "ms_per_step": total_ms / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": cfg["dtype"], "data": "synthetic",
        "config": {"workload": f"{args.config}: {shape_name(cfg)}, prompt {cfg['P']} + {cfg['G']} masks, A={A} B={B} R={R} "
                               f"T={T} k={k} batch {batch}; steps {W}..{W + K - 1} of the generation; replicas only at N>1",
                   "l2": f"inputs larger than L2: every step streams {weight_bytes(cfg) / 1e9:.1f} GB of weights",
                   "normal_step_ms": normal_ms, "refresh_step_ms": float(np.median(refresh)) if refresh else None,
                   "normal_step_algorithmic_gb": step_by / 1e9,
                   "normal_step_frac_of_hbm_roofline_measured": (step_by / (normal_ms * 1e-3) / 1e9 / peaks["hbm_gbs"])
                   if normal_ms else None,
                   "normal_step_frac_of_hbm_roofline_nominal_8TBs": (step_by / (normal_ms * 1e-3) / 8e12) if normal_ms else None,
                   "phase_amortised": phase_amortised(normal, refresh, R, batch * k * world),
                   "full_sequence_step_ms": float(np.median(full_ms)),
                   "rows_normal": float(np.mean([i["n_rows"] for i in ni])) if ni else None,
                   "stepping": "queued: steps enqueued back to back, index lists planned on the device, drained every 16 steps",
                   "gemm_impl": infos[-1]["gemm_impl"],
                   "variant_fp8_projections": fp8_line,
                   "variant_nvfp4_projections": fp4_line,
                   "variant_window_only_refresh": {
                       "note": "NOT the paper's refresh: after the first step a refresh recomputes only the new window "
                               "and the previous phase's tokens (an approximation beyond one block); same steps otherwise",
                       "value": whole_job_value(batch * k * K, world, v_total_ms), "unit": UNIT,
                       "refresh_step_ms": float(np.median(v_refresh)) if v_refresh else None,
                       "refresh_rows": float(np.mean([i["n_rows"] for i in v_infos if i["is_refresh"]])) if v_refresh else None}},
        "clocks": {"sm_mhz": clocks["sm_mhz"], "sm_max_mhz": clocks["sm_max_mhz"], "reasons": clocks["reasons"],
                   "samples": clocks["samples"]},
        # end to end = the call a user makes for a generation: host prompt in (wd_state_reset), the library's own
        # decoding loop (wd_generate: every step copies its result block to pinned host memory, the host commits
        # them as they arrive), host tokens out (wd_state_read), on the host clock
        "e2e": {"value": gen_tokens * world / gen_wall, "unit": UNIT, "steps": gen_steps, "tokens": gen_tokens,
                "seconds": gen_wall,
                "call": "wd_state_reset + wd_generate + wd_state_read on the host clock (the whole generation)",
                "per_step_sync": {"value": batch * k * (W + K) * world / e2e_wall, "unit": UNIT,
                                  "stepping": "the bench's W + K steps as one wd_step + wd_step_sync per step (every "
                                              "step's tokens reach the host before the next is enqueued)"},
                "h2d_bytes_per_step": float(batch * S * 5 / max(gen_steps, 1)),
                "d2h_bytes_per_step": float((1 + batch + 3 * batch * k) * 4 + batch * S * 4 / max(gen_steps, 1))},
        "gpu_launches": int(sum(i["n_launches"] for i in infos)),
        "roofline": {"bound": "hbm", "kernel": "gemm_tc_kernel (launches of the normal, weight-streaming steps)",
                     "achieved": gemm_gbs, "peak": peaks["hbm_gbs"],
                     "unit": "GB/s", "frac": gemm_gbs / peaks["hbm_gbs"], "peak_source": peaks["source"],
                     "traffic": prof["gemm_bytes"] / n_l * 1.03,
                     "traffic_note": "ncu small case (gate/up shape): DRAM bytes = 1.03 x algorithmic, scaled by bytes",
                     "launches": int(prof["gemm_launches"]),
                     "avg_launch_us": prof["gemm_ms"] * 1e3 / n_l, "bytes_per_launch": prof["gemm_bytes"] / n_l,
                     "timing": "CUDA events around every launch on the step's stream (serialises the stream: isolated "
                               "launch time, without the programmatic overlap the timed value has)",
                     # the claim for the hot path as a whole: all algorithmic bytes of a normal step over its time
                     "whole_normal_step": {"achieved": (step_by / (normal_ms * 1e-3) / 1e9) if normal_ms else None,
                                           "unit": "GB/s", "bytes": step_by,
                                           "frac": (step_by / (normal_ms * 1e-3) / 1e9 / peaks["hbm_gbs"]) if normal_ms else None,
                                           "note": "the step-level figure is the claim; the kernel-level figure above is "
                                                   "the same kernel timed in isolation"}},
    }
    if prof_refresh["gemm_launches"] and prof_refresh["gemm_ms"] > 0:
        tf = prof_refresh["flops"] / (prof_refresh["gemm_ms"] * 1e-3) / 1e12
        line["roofline_refresh_steps"] = {"bound": "tensor", "kernel": "gemm_tc_kernel (launches of the refresh steps)",
                                          "achieved": tf, "peak": peaks["bf16_tflops_sustained"], "unit": "TFLOP/s",
                                          "frac": tf / peaks["bf16_tflops_sustained"], "peak_source": peaks["source"],
                                          "launches": int(prof_refresh["gemm_launches"])}
    if rank == 0:
        line["cpu_baseline"] = cpu_baseline(cfg, w, ids, budget_s=args.cpu_seconds)
        print(json.dumps(line))
    ctx.close()


def cpu_baseline(cfg, w, ids, budget_s=25.0):
    """The oracle as it stands, timed on the host cores on a bounded sample:
    one refresh step and one normal step of the same workload truncated to 1
    and to 2 layers, extrapolated linearly in depth to the full model."""
    from oracle import wd_oracle as wo
    try:
        from threadpoolctl import threadpool_info
        cores = max([p.get("num_threads", 1) for p in threadpool_info()] + [1])
    except Exception:
        cores = os.cpu_count() or 1
    S = cfg["P"] + cfg["G"]
    A, B, R, T, k = (cfg[x] for x in ("A", "B", "R", "T", "k"))

    class Truncated(synth.OracleModelView):
        def __init__(self, w, n_layers):
            super().__init__(w)
            self.dims = dict(self.dims, L=n_layers)

    times = {}
    for nl in (1, 2):
        model = Truncated(w, nl)
        st = [wo.SeqState(ids=ids[0], decoded=np.arange(S) < cfg["P"])]
        cache = [wo.KVCache.empty(model.dims, S)]
        t0 = time.perf_counter()
        wo.oracle_step(model, st, cache, A, B, R, T, k)
        t1 = time.perf_counter()
        wo.oracle_step(model, st, cache, A, B, R, T, k)
        t2 = time.perf_counter()
        times[nl] = (t1 - t0, t2 - t1)
    L = cfg["L"]
    per_layer_r, per_layer_n = times[2][0] - times[1][0], times[2][1] - times[1][1]
    t_refresh = times[1][0] + (L - 1) * max(per_layer_r, 0.0)
    t_normal = times[1][1] + (L - 1) * max(per_layer_n, 0.0)
    phase = t_refresh + (R - 1) * t_normal
    return {"value": k * R / phase, "unit": UNIT, "cores": int(cores), "kind": "oracle",
            "sample": f"one refresh + one normal step of batch-1 sequence 0 at 1 and 2 of {L} layers, extrapolated linearly "
                      f"in depth; refresh {t_refresh:.1f} s, normal {t_normal:.1f} s per step; most of either is the oracle's "
                      f"weight access (each layer's matrices copied from the device and widened bf16 -> fp64 every step), "
                      f"not its arithmetic, which is why the normal step is not faster than the refresh"}


def run_reference(args, rank, world):
    """The reference arm is the CPU oracle (there is no reference implementation)."""
    if rank != 0:
        return
    cfg = synth.get_config(args.config)
    dev = "cuda:0" if torch.cuda.is_available() else "cpu"
    w = synth.make_weights(cfg, dev)
    ids = synth.make_prompts(cfg)
    vals = []
    for i in range(args.warmup + args.steps):
        cb = cpu_baseline(cfg, w, ids)
        if i >= args.warmup:
            vals.append(cb["value"])
    v = float(np.mean(vals))
    R, k = cfg["R"], cfg["k"]
    cb["value"] = v
    print(json.dumps({"impl": "reference", "metric": METRIC, "value": v, "unit": UNIT, "n_gpus": world,
                      "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * k / v, "higher_is_better": True,
                      "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
                      "config": {"workload": f"{args.config}: fp64 CPU oracle on a bounded sample of the same workload"},
                      "cpu_baseline": cb,
                      "e2e": {"value": v, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}))


def run_plumbing_check(args, rank, world):
    """`--plumbing-check` (used by the CPU tests of the launcher): the rank plumbing of a run without its
    GPU work.  Every rank joins the process group the launcher set up, contributes a made-up local
    time, and rank 0 prints a line whose n_gpus is the world size and whose value is the work of all
    ranks over the slowest rank's time."""
    local_ms = 10.0 * (rank + 1)
    total = max_over_ranks(local_ms, world, "cpu")
    if world > 1:
        torch.distributed.barrier()
    if rank == 0:
        print(json.dumps({"metric": METRIC, "value": whole_job_value(args.steps, world, total), "unit": UNIT,
                          "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": total / args.steps,
                          "scaling": "weak", "config": {"workload": "plumbing check: no GPU work"}}))


def launch_ranks(args, argv) -> int:
    """`bench.py --gpus N` started as a plain process: start N ranks of this same command, one per
    GPU, under torch.distributed.run on this node (rendezvous on 127.0.0.1, a free port) and hand
    their output through.  Replicas only: NCCL carries the barrier and the MAX of the timings."""
    import socket
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + list(argv)
    return subprocess.call(cmd)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", default="llada8b")
    ap.add_argument("--cpu-seconds", type=float, default=25.0)
    ap.add_argument("--plumbing-check", action="store_true",
                    help="rank plumbing only, over gloo, no GPU work (CPU test of the --gpus launcher)")
    args = ap.parse_args()
    if args.gpus < 1:
        ap.error("--gpus must be at least 1")
    if "WORLD_SIZE" not in os.environ and args.gpus > 1:
        # not under a launcher yet: become N ranks (the reference arm too, whose ranks > 0 exit at once)
        if not args.plumbing_check and torch.cuda.device_count() < args.gpus:
            sys.stderr.write(f"bench.py: --gpus {args.gpus} but {torch.cuda.device_count()} CUDA devices are visible\n")
            sys.exit(2)
        sys.exit(launch_ranks(args, sys.argv[1:]))
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if world != args.gpus:
        sys.stderr.write(f"bench.py: --gpus {args.gpus} disagrees with WORLD_SIZE={world}\n")
        sys.exit(2)
    if args.plumbing_check:
        args.steps = 64 if args.steps is None else args.steps
        args.warmup = 8 if args.warmup is None else args.warmup
        if world > 1:
            torch.distributed.init_process_group("gloo")
        try:
            run_plumbing_check(args, rank, world)
        finally:
            if world > 1:
                torch.distributed.destroy_process_group()
        return
    if args.impl == "reference":
        args.steps = 1 if args.steps is None else min(args.steps, 3)
        args.warmup = 0 if args.warmup is None else min(args.warmup, 1)
        run_reference(args, rank, world)
        return
    args.steps = 64 if args.steps is None else args.steps
    args.warmup = 8 if args.warmup is None else max(args.warmup, 3)
    if world > 1:
        torch.distributed.init_process_group("nccl", device_id=torch.device(f"cuda:{int(os.environ.get('LOCAL_RANK', 0))}"))
    try:
        run_ours(args, rank, world)
    finally:
        if world > 1:
            torch.distributed.destroy_process_group()


if __name__ == "__main__":
    main()
