"""Independent dense full-sequence forward, used only to pin the oracle.

TEST INFRASTRUCTURE ONLY.  Section 3.1 of the paper: a masked diffusion LM
step is a transformer forward over the entire sequence with no causal mask.
Section 4.3 says a refresh step is such a forward over everything that takes
part in the phase, so when the external window covers every undecoded token
and every step is a refresh, the windowed step must reduce to this function.

It is written separately from ``wd_oracle.py`` on purpose: whole-sequence
matrices, no cache, no index lists, torch float64 library routines
(``rms_norm``, ``scaled_dot_product_attention``, ``silu``) and rotary
embedding as a complex multiplication, so a mistake in the oracle (a dropped
term, a transposed operand, a wrong sign or head mapping) does not repeat
here.  Neither file imports the other.
"""
from __future__ import annotations

import numpy as np
import torch
import torch.nn.functional as F


def dense_full_forward(model, ids) -> dict:
    """ids: [S] token ids.  Returns per-layer outputs [L][S, d], attention
    outputs [L][S, Hq*dh] and logits [S, V] as float64 numpy arrays."""
    dm = model.dims
    L, d, Hq, Hkv, dh = dm["L"], dm["d"], dm["Hq"], dm["Hkv"], dm["dh"]
    S = len(ids)
    t = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(torch.float64)
    x = t(model.embed_rows(np.asarray(ids)))
    # e^{i * pos * theta^{-2j/dh}} for every (position, frequency)
    inv_freq = 1.0 / (dm["theta"] ** (torch.arange(0, dh, 2, dtype=torch.float64) / dh))
    phase = torch.polar(torch.ones(S, dh // 2, dtype=torch.float64),
                        torch.outer(torch.arange(S, dtype=torch.float64), inv_freq))

    def rotate(u):                       # u: [S, H, dh], pairs (j, j + dh/2)
        z = torch.complex(u[..., : dh // 2], u[..., dh // 2:]) * phase[:, None, :]
        return torch.cat([z.real, z.imag], dim=-1)

    layer_out, attn_out = [], []
    for l in range(L):
        w = {k: t(v) for k, v in model.layer(l).items()}
        a = F.rms_norm(x, (d,), weight=w["attn_norm"], eps=dm["eps"])
        q = rotate(F.linear(a, w["wq"]).view(S, Hq, dh))
        k = rotate(F.linear(a, w["wk"]).view(S, Hkv, dh))
        v = F.linear(a, w["wv"]).view(S, Hkv, dh)
        # [1, H, S, dh]; expand KV heads so that query head h reads KV head h // group
        qh = q.permute(1, 0, 2).unsqueeze(0)
        kh = k.permute(1, 0, 2).repeat_interleave(Hq // Hkv, dim=0).unsqueeze(0)
        vh = v.permute(1, 0, 2).repeat_interleave(Hq // Hkv, dim=0).unsqueeze(0)
        o = F.scaled_dot_product_attention(qh, kh, vh, attn_mask=None, is_causal=False)
        o = o.squeeze(0).permute(1, 0, 2).reshape(S, Hq * dh)
        h = x + F.linear(o, w["wo"])
        f = F.rms_norm(h, (d,), weight=w["ffn_norm"], eps=dm["eps"])
        x = h + F.linear(F.silu(F.linear(f, w["w_gate"])) * F.linear(f, w["w_up"]), w["w_down"])
        layer_out.append(x.numpy().copy())
        attn_out.append(o.numpy().copy())
    xf = F.rms_norm(x, (d,), weight=t(model.final_norm()), eps=dm["eps"])
    logits = F.linear(xf, t(model.lm_head()))
    return dict(layer_out=layer_out, attn_out=attn_out, logits=logits.numpy())
