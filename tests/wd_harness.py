"""Teacher-forced GPU-vs-oracle trajectory comparison used by the GPU tests.

Both sides start from the same seeded state.  At every step the library's
index sets must equal the oracle's exactly; per-layer outputs, attention
outputs and logits are compared within the stated tolerances; the unmask rule
is checked bit-exactly by feeding the GPU's own float32 logits to the oracle's
unmask routine; then both sides advance with the GPU's choice, because
random-init confidences are nearly uniform and free-running trajectories would
split at the first bf16-level difference.
"""
from __future__ import annotations

import numpy as np
import torch

from oracle import wd_oracle as wo
from paper_2601_20332_b200 import binding as wd
from paper_2601_20332_b200 import synth

TOL_LAYER = 1e-2      # relative RMS of a layer's output over [rows, d]
TOL_ATTN = 2e-2       # max |a-b| / max |b| of a layer's attention output
GAP = 1e-8            # below this relative confidence gap a rank decision is rounding-ambiguous
                      # (the GPU sums single-precision exponentials of the same float logits in double: ~1e-9)


def rel_rms(a, b):
    return float(np.linalg.norm(a - b) / max(np.linalg.norm(b), 1e-300))


def max_rel(a, b):
    return float(np.abs(a - b).max() / max(np.abs(b).max(), 1e-300))


class Parity:
    def __init__(self, cfg, weights, ids, decoded=None, gemm_impl=wd.WD_GEMM_AUTO, oracle_seqs=None,
                 max_rows=None, max_active=None, fusion=wd.WD_FUSION_AUTO, eos_id=None, refresh_mode=0, fp8=False,
                 follow_rounded=False, stagger=False, fp4=False):
        """follow_rounded: a second oracle follower per sequence runs in the bfloat16 storage-points mode
        (the same teacher-forced trajectory); `step` then also records, per block, the GPU's distance to it
        and its own distance to the plain float64 follower: what the storage format alone costs at that
        depth, the yardstick for the GPU's error in a deep model."""
        self.cfg = cfg
        self.batch, self.S = ids.shape
        dev = weights.tok_embed.device
        max_rows = self.batch * self.S if max_rows is None else max_rows
        max_active = max_rows if max_active is None else max_active
        self.ctx = wd.Context(cfg, weights, self.batch, self.S, max_rows, max_active)
        self.ctx.set_gemm_impl(gemm_impl)
        self.ctx.set_fusion(fusion)
        if fp8:
            self.ctx.fp8_enable()
        if fp4:
            self.ctx.fp4_enable()
        self.st = wd.State(self.ctx, ids, decoded)
        if eos_id is not None:
            self.st.set_eos(eos_id)
        if refresh_mode:
            self.st.set_refresh_mode(refresh_mode)
        if stagger:
            self.st.set_stagger(True)
        L, d, hq, V = cfg["L"], cfg["d"], cfg["Hq"] * cfg["dh"], cfg["V"]
        self.t_layer = torch.zeros(L * max_rows * d, dtype=torch.float32, device=dev)
        self.t_attn = torch.zeros(L * max_rows * hq, dtype=torch.float32, device=dev)
        self.t_logits = torch.zeros(max_active * V, dtype=torch.float32, device=dev)
        self.st.set_taps(self.t_layer, self.t_attn, self.t_logits)
        self.model = synth.OracleModelView(weights)
        if fp8:
            self.model.dims = dict(self.model.dims, fp8=True)
        if fp4:
            self.model.dims = dict(self.model.dims, nvfp4=True)
        self.oracle_seqs = list(range(self.batch)) if oracle_seqs is None else list(oracle_seqs)
        dec = (ids != cfg["mask_id"]) if decoded is None else decoded.astype(bool)
        stg = (lambda b: (b, self.batch)) if stagger else (lambda b: None)
        self.ost = [wo.SeqState(ids=ids[b], decoded=dec[b], eos_id=eos_id, refresh_mode=refresh_mode, stagger=stg(b))
                    for b in self.oracle_seqs]
        self.follow_rounded = follow_rounded
        if follow_rounded:      # followers n .. 2n-1: the same sequences with bfloat16 storage points
            self.ost += [wo.SeqState(ids=ids[b], decoded=dec[b], eos_id=eos_id, refresh_mode=refresh_mode, bf16_points=True,
                                     stagger=stg(b)) for b in self.oracle_seqs]
        self.oc = [wo.KVCache.empty(self.model.dims, self.S) for _ in self.ost]
        self.log = []

    def step(self, A, B, R, T, k, tol_layer=TOL_LAYER, tol_attn=TOL_ATTN, check=True, envelope=None):
        """envelope: optional function block index -> (layer tolerance, attention tolerance) for the comparison
        with the plain float64 oracle (default: tol_layer, tol_attn for every block)."""
        cfg = self.cfg
        L, d, hq, V = cfg["L"], cfg["d"], cfg["Hq"] * cfg["dh"], cfg["V"]
        plans = [self.st.plan(b, A, B, R, T) for b in range(self.batch)]
        status, info = self.st.step(A, B, R, T, k)
        if status == wd.WD_DONE:
            for st in self.ost:
                assert wo.oracle_plan(st, A, B, R, T)["done"]
            return None
        res = self.st.sync()
        n_rows, n_act = info["n_rows"], info["n_active"]
        assert n_rows == sum(len(p["rows"]) for p in plans if not p["done"])
        lay = self.t_layer[: L * n_rows * d].view(L, n_rows, d).cpu().numpy().astype(np.float64)
        att = self.t_attn[: L * n_rows * hq].view(L, n_rows, hq).cpu().numpy().astype(np.float64)
        lg = self.t_logits[: n_act * V].view(n_act, V).cpu().numpy()
        row_off = np.cumsum([0] + [0 if p["done"] else len(p["rows"]) for p in plans])
        act_off = np.cumsum([0] + [0 if p["done"] else len(p["active"]) for p in plans])
        forced = []
        for b in self.oracle_seqs:
            nb = int(res["n_unmasked"][b])
            forced.append((res["positions"][b, :nb].tolist(), res["token_ids"][b, :nb].tolist()))
        if self.follow_rounded:
            forced = forced + forced
        outs = wo.oracle_step(self.model, self.ost, self.oc, A, B, R, T, k, forced=forced)
        worst = dict(layer=0.0, attn=0.0, logits=0.0, ambiguous=0, layer_rounded=0.0, attn_rounded=0.0, logits_rounded=0.0)
        # worst error of each block over the followed sequences (and against the bf16 storage-points followers)
        curve = dict(layer=[0.0] * L, attn=[0.0] * L, layer_rounded=[0.0] * L, attn_rounded=[0.0] * L,
                     layer_format=[0.0] * L, attn_format=[0.0] * L)    # *_format: storage-points oracle against the plain one
        for j, b in enumerate(self.oracle_seqs):
            o, p = outs[j], plans[b]
            assert p["done"] == o["done"]
            if o["done"]:
                continue
            op = o["plan"]
            # index sets: bit-exact
            assert p["refresh"] == op["refresh"]
            for name, oname in (("active", "active"), ("buffer", "buffer"), ("decoded", "decoded"),
                                ("transient", "transient"), ("far_field", "far_field"), ("rows", "rows"),
                                ("vis", "vis"), ("ext_window", "wex")):
                assert p[name] == op[oname], (name, b)
            r0, r1 = row_off[b], row_off[b + 1]
            a0, a1 = act_off[b], act_off[b + 1]
            for l in range(L):
                e_l = rel_rms(lay[l, r0:r1], o["layer_out"][l])
                e_a = max_rel(att[l, r0:r1], o["attn_out"][l])
                worst["layer"] = max(worst["layer"], e_l)
                worst["attn"] = max(worst["attn"], e_a)
                curve["layer"][l] = max(curve["layer"][l], e_l)
                curve["attn"][l] = max(curve["attn"][l], e_a)
                tl, ta = envelope(l) if envelope else (tol_layer, tol_attn)
                if check:
                    assert np.isfinite(lay[l, r0:r1]).all()
                    assert e_l <= tl, f"seq {b} layer {l}: rel-RMS {e_l:.3e}"
                    assert e_a <= ta, f"seq {b} layer {l}: attention max-rel {e_a:.3e}"
                if self.follow_rounded:
                    orr = outs[len(self.oracle_seqs) + j]
                    r_l = rel_rms(lay[l, r0:r1], orr["layer_out"][l])
                    r_a = max_rel(att[l, r0:r1], orr["attn_out"][l])
                    worst["layer_rounded"] = max(worst["layer_rounded"], r_l)
                    worst["attn_rounded"] = max(worst["attn_rounded"], r_a)
                    curve["layer_rounded"][l] = max(curve["layer_rounded"][l], r_l)
                    curve["attn_rounded"][l] = max(curve["attn_rounded"][l], r_a)
                    curve["layer_format"][l] = max(curve["layer_format"][l], rel_rms(orr["layer_out"][l], o["layer_out"][l]))
                    curve["attn_format"][l] = max(curve["attn_format"][l], max_rel(orr["attn_out"][l], o["attn_out"][l]))
            glg = lg[a0:a1]
            e_lg = rel_rms(glg.astype(np.float64), o["logits"])
            worst["logits"] = max(worst["logits"], e_lg)
            if check:
                assert e_lg <= 2 * (envelope(L - 1)[0] if envelope else tol_layer), f"seq {b}: logits rel-RMS {e_lg:.3e}"
            if self.follow_rounded:
                r_lg = rel_rms(glg.astype(np.float64), outs[len(self.oracle_seqs) + j]["logits"])
                worst["logits_rounded"] = max(worst["logits_rounded"], r_lg)
            # the unmask rule on the GPU's own logits: token ids exact, ranking exact unless the
            # confidence gap at the cut is below rounding
            um = wo.oracle_unmask(glg, op["active"], k)
            nb = int(res["n_unmasked"][b])
            assert nb == min(k, len(op["active"]))
            got_pos = res["positions"][b, :nb].tolist()
            got_tok = res["token_ids"][b, :nb].tolist()
            conf_sorted = sorted(um["conf"], reverse=True)
            ambiguous = any(abs(conf_sorted[i] - conf_sorted[i + 1]) <= GAP * conf_sorted[i]
                            for i in range(min(nb, len(conf_sorted) - 1)))
            tok_of = dict(zip(op["active"], um["ids"].tolist()))
            assert got_tok == [tok_of[q] for q in got_pos]
            if ambiguous:
                worst["ambiguous"] += 1
                assert set(got_pos) <= set(op["active"])
            else:
                assert got_pos == um["positions"], (got_pos, um["positions"])
            np.testing.assert_allclose(res["confidence"][b, :nb], [um["conf"][op["active"].index(q)] for q in got_pos],
                                       rtol=1e-4)
        self.log.append(dict(info=info, worst=worst, curve=curve))
        return dict(info=info, res=res, worst=worst, curve=curve, plans=plans, outs=outs)

    def check_state_mirror(self):
        """The library's host mirror equals the oracle's state."""
        for j, b in enumerate(self.oracle_seqs):
            got = self.st.read(b)
            st = self.ost[j]
            assert (got["ids"] == st.ids).all()
            assert (got["decoded"] == st.decoded).all()
            assert got["t"] == st.t and got["since"] == st.since
            gs = np.where(got["dec_step"] == -(1 << 31), wo.NEVER, got["dec_step"])
            assert (gs == st.dec_step).all()

    def close(self):
        self.st.close()
        self.ctx.close()
