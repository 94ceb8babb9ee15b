"""Seeded synthetic inputs shared by the tests and the benchmark.

This module only *generates and marshals data*: model shapes, random-init
weights, prompts, decoded-flag patterns.  It contains none of the method's
arithmetic (no planner, no forward pass, no unmask rule) so that the CUDA
library and the CPU oracle can both be fed from it without sharing code.

Shapes follow the five benchmark configurations: a tiny fp32 model, an
LLaDA-8B-shaped and a Dream-7B-shaped bf16 model.  The paper's own workloads
(LLaDA / Dream checkpoints on GSM8K, MATH, HumanEval, MBPP prompts, Section
5.1 and the hyper-parameter tables of the appendix) need trained weights and
datasets; here every weight matrix is N(0, 0.02) from a seeded generator and
every prompt is uniform-random token ids, which reproduces the shapes, sizes
and length mix but not the text.
"""
from __future__ import annotations

import copy
from dataclasses import dataclass, field

import numpy as np
import torch

# --------------------------------------------------------------------------
# model shapes and window settings
# --------------------------------------------------------------------------

_TINY = dict(dtype="f32", L=2, d=256, Hq=4, Hkv=4, dh=64, F=688, V=1024,
             theta=1.0e4, eps=1.0e-5)
_LLADA = dict(dtype="bf16", L=32, d=4096, Hq=32, Hkv=32, dh=128, F=12288,
              V=126464, theta=5.0e5, eps=1.0e-5)
_DREAM = dict(dtype="bf16", L=28, d=3584, Hq=28, Hkv=4, dh=128, F=18944,
              V=152064, theta=1.0e6, eps=1.0e-6)

CONFIGS = {
    # cfg 1: correctness config, runs everywhere
    "tiny": dict(_TINY, P=32, G=64, batch=1, A=8, B=16, R=4, T=2, k=1,
                 wseed=0, iseed=1),
    # cfg 2: the configuration the headline metric is quoted on
    "llada8b": dict(_LLADA, P=256, G=256, batch=1, A=32, B=64, R=8, T=2, k=1,
                    wseed=0, iseed=2),
    # cfg 3: long generation, two tokens per step
    "llada8b_long": dict(_LLADA, P=512, G=1024, batch=1, A=64, B=128, R=8,
                         T=2, k=2, wseed=0, iseed=3),
    # cfg 4: GQA, batch of independent windows
    "dream7b": dict(_DREAM, P=512, G=512, batch=8, A=32, B=128, R=4, T=3,
                    k=1, wseed=0, iseed=4),
    # cfg 5: base point of the window sweep (A, B, R, batch are swept)
    "llada8b_sweep": dict(_LLADA, P=1024, G=2048, batch=1, A=32, B=128, R=4,
                          T=2, k=1, wseed=0, iseed=5),
}


def get_config(name: str, **overrides) -> dict:
    """Return a copy of a named configuration with fields overridden."""
    cfg = copy.deepcopy(CONFIGS[name])
    cfg.update(overrides)
    cfg["name"] = name
    cfg.setdefault("mask_id", cfg["V"] - 1)
    return cfg


def torch_dtype(cfg: dict) -> torch.dtype:
    return torch.float32 if cfg["dtype"] == "f32" else torch.bfloat16


# --------------------------------------------------------------------------
# weights
# --------------------------------------------------------------------------

@dataclass
class Weights:
    """Random-init weights as torch tensors (row-major, K contiguous)."""
    cfg: dict
    tok_embed: torch.Tensor                    # [V, d]
    wq: list = field(default_factory=list)      # L x [Hq*dh, d]
    wk: list = field(default_factory=list)      # L x [Hkv*dh, d]
    wv: list = field(default_factory=list)      # L x [Hkv*dh, d]
    wo: list = field(default_factory=list)      # L x [d, Hq*dh]
    w_gate: list = field(default_factory=list)  # L x [F, d]
    w_up: list = field(default_factory=list)    # L x [F, d]
    w_down: list = field(default_factory=list)  # L x [d, F]
    attn_norm: list = field(default_factory=list)  # L x [d] fp32
    ffn_norm: list = field(default_factory=list)   # L x [d] fp32
    final_norm: torch.Tensor = None             # [d] fp32
    lm_head: torch.Tensor = None                # [V, d]


def make_weights(cfg: dict, device="cpu", gain_jitter: float = 0.0) -> Weights:
    """All matrices N(0, 0.02) sampled in fp32 then rounded to the model dtype.

    Norm gains are 1 (plus ``gain_jitter`` * N(0,1) when a test wants the
    gains to matter).  One generator, fixed tensor order, so the same seed
    gives the same bits on the same device type.
    """
    dev = torch.device(device)
    gen = torch.Generator(device=dev)
    gen.manual_seed(int(cfg["wseed"]))
    dt = torch_dtype(cfg)
    L, d, Hq, Hkv, dh, F, V = (cfg[k] for k in ("L", "d", "Hq", "Hkv", "dh", "F", "V"))

    def mat(rows, cols):
        t = torch.empty(rows, cols, dtype=torch.float32, device=dev)
        t.normal_(0.0, 0.02, generator=gen)
        return t.to(dt).contiguous()

    def gain():
        g = torch.ones(d, dtype=torch.float32, device=dev)
        if gain_jitter:
            g += gain_jitter * torch.randn(d, dtype=torch.float32, device=dev, generator=gen)
        return g.contiguous()

    w = Weights(cfg=cfg, tok_embed=mat(V, d))
    for _ in range(L):
        w.wq.append(mat(Hq * dh, d))
        w.wk.append(mat(Hkv * dh, d))
        w.wv.append(mat(Hkv * dh, d))
        w.wo.append(mat(d, Hq * dh))
        w.w_gate.append(mat(F, d))
        w.w_up.append(mat(F, d))
        w.w_down.append(mat(d, F))
        w.attn_norm.append(gain())
        w.ffn_norm.append(gain())
    w.final_norm = gain()
    w.lm_head = mat(V, d)
    return w


def to_f64(t: torch.Tensor) -> np.ndarray:
    """Exact widening of an fp32 / bf16 tensor to a float64 numpy array."""
    return t.detach().to(torch.float32).cpu().numpy().astype(np.float64)


class OracleModelView:
    """Hands the weights to the CPU oracle as float64 numpy arrays, one layer
    at a time (an 8B-parameter model does not fit in host memory as fp64)."""

    def __init__(self, w: Weights):
        self.w = w
        c = w.cfg
        self.dims = dict(L=c["L"], d=c["d"], Hq=c["Hq"], Hkv=c["Hkv"], dh=c["dh"],
                         F=c["F"], V=c["V"], theta=float(c["theta"]), eps=float(c["eps"]))

    def embed_rows(self, ids) -> np.ndarray:
        idx = torch.as_tensor(np.asarray(ids, dtype=np.int64), device=self.w.tok_embed.device)
        return to_f64(self.w.tok_embed.index_select(0, idx))

    def layer(self, l: int) -> dict:
        w = self.w
        return dict(wq=to_f64(w.wq[l]), wk=to_f64(w.wk[l]), wv=to_f64(w.wv[l]),
                    wo=to_f64(w.wo[l]), w_gate=to_f64(w.w_gate[l]), w_up=to_f64(w.w_up[l]),
                    w_down=to_f64(w.w_down[l]), attn_norm=to_f64(w.attn_norm[l]),
                    ffn_norm=to_f64(w.ffn_norm[l]))

    def final_norm(self) -> np.ndarray:
        return to_f64(self.w.final_norm)

    def lm_head(self) -> np.ndarray:
        return to_f64(self.w.lm_head)


# --------------------------------------------------------------------------
# sequences
# --------------------------------------------------------------------------

def make_prompts(cfg: dict, batch: int | None = None, P: int | None = None,
                 G: int | None = None) -> np.ndarray:
    """[batch, P+G] int32: P uniform-random ids (never the mask id) followed by
    G mask placeholders.  Each sequence of a batch gets different ids."""
    batch = cfg["batch"] if batch is None else batch
    P = cfg["P"] if P is None else P
    G = cfg["G"] if G is None else G
    rng = np.random.default_rng(int(cfg["iseed"]))
    V, mask_id = cfg["V"], cfg["mask_id"]
    ids = np.full((batch, P + G), mask_id, dtype=np.int32)
    draw = rng.integers(0, V - 1, size=(batch, P), dtype=np.int64)
    draw = np.where(draw >= mask_id, draw + 1, draw)      # skip mask_id
    ids[:, :P] = draw.astype(np.int32)
    return ids


def fast_forward(cfg: dict, ids: np.ndarray, n_decoded: int, seed: int = 1234):
    """Late-generation state: mark the first ``n_decoded`` masks of every
    sequence as decoded with seeded random ids.  Returns (ids, decoded)."""
    rng = np.random.default_rng(seed)
    ids = ids.copy()
    P = cfg["P"]
    V, mask_id = cfg["V"], cfg["mask_id"]
    decoded = np.zeros(ids.shape, dtype=np.uint8)
    decoded[:, :P] = 1
    n = min(n_decoded, ids.shape[1] - P)
    if n > 0:
        draw = rng.integers(0, V - 1, size=(ids.shape[0], n), dtype=np.int64)
        draw = np.where(draw >= mask_id, draw + 1, draw)
        ids[:, P:P + n] = draw.astype(np.int32)
        decoded[:, P:P + n] = 1
    return ids, decoded


def random_decoded_pattern(S: int, frac: float, seed: int) -> np.ndarray:
    """Arbitrary (non-prefix) decoded flags for planner property tests."""
    rng = np.random.default_rng(seed)
    return (rng.random(S) < frac).astype(np.uint8)
