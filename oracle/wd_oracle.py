"""CPU oracle for one windowed denoising step (Window-Diffusion).

TEST INFRASTRUCTURE ONLY.  This is a plain, slow, float64 numpy statement of
what the step computes, written from the paper's text.  It shares no code with
the CUDA library and must never be on a product path: only the tests, the
smoke check and the benchmark's CPU-baseline leg may import it.

What each part follows
  * planner            Section 4.2 (dual-window sets, the buffer-set equation),
                       Section 4.3 (one refresh step then normal steps per
                       phase; newly decoded tokens keep being recomputed for a
                       few steps), Section 5.3 "Effect of Cache Refresh Cycle"
                       (in the authors' implementation that transient lasts
                       until the next refresh).
  * forward            Section 3.1 (bidirectional transformer forward, no
                       causal mask) restricted to the rows Section 4.3 says
                       are computed, reading K/V written at the refresh step
                       (the cache-write equation of Section 4.3) for the rest.
  * unmask             Section 3.2 Observation 1 / Section 4.1: decoding is
                       decided by prediction confidence on the active tokens.

The paper uses the pretrained models unmodified and does not restate their
internals, so the block structure is the benchmark configurations' reading:
pre-norm residual blocks, RMSNorm, rotary embedding at the absolute position
(half-split pairing), grouped-query bidirectional attention with scale
1/sqrt(dh), SwiGLU feed-forward, final RMSNorm, untied LM head, no biases.

Parity pins: the forward is pinned to an independently written dense
full-sequence forward (``dense_ref.py``) through the paper's reduction "window
covers everything and every step is a refresh"; attention, RoPE, RMSNorm and
the unmask rule are pinned to closed forms and brute force; the planner is
pinned to the set identities of Section 4.2 and to a hand-traced trajectory.
The readings the paper does not fix (transient length capped by T and reset at
a refresh, forced early refresh when the window is exhausted, every model
constant) are **parity unpinned against the paper**: they are only checked for
internal consistency.

Precision modes.  The default is plain float64 with no intermediate rounding.
Two optional modes restate a reduced-precision pipeline's *storage formats* (and
nothing else of it) so that a deep model can be compared layer by layer without
the formats' own rounding noise hiding everything else: ``dims["fp8"]`` (e4m3
projections) and ``SeqState.bf16_points`` (activations stored as bfloat16 at the
points a "bf16 in, fp32 accumulate" pipeline stores them).  Both are pinned to
the formats' definitions by brute force.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np

NEVER = -(1 << 30)          # decode step of tokens that were given, not generated


# ---------------------------------------------------------------------------
# sequence state and planner (Sections 4.2 and 4.3)
# ---------------------------------------------------------------------------

@dataclass
class SeqState:
    """x^(t) of Section 3.1 plus the phase bookkeeping of Section 4.3."""
    ids: np.ndarray                       # [S] token ids (mask id where undecoded)
    decoded: np.ndarray                   # [S] bool
    dec_step: np.ndarray = None           # [S] step at which a token was unmasked
    t: int = 0                            # diffusion step index
    since: int = 0                        # steps since the last refresh
    phase_start: int = 0
    wex: list = field(default_factory=list)   # external window of the current phase
    eos_id: int = None                    # adaptive termination (Section 4.2), None = off
    refresh_mode: int = 0                 # 0: the paper's refresh (Section 4.3); 1: window-only variant (see oracle_plan)
    bf16_points: bool = False             # activations rounded to bfloat16 where a bf16 pipeline stores them (see oracle_layer)
    stagger: tuple = None                 # (i, n): sequence i of a batch of n with staggered refresh steps (see oracle_plan)

    def __post_init__(self):
        self.ids = np.array(self.ids, dtype=np.int64)
        self.decoded = np.array(self.decoded, dtype=bool)
        if self.dec_step is None:
            self.dec_step = np.full(self.ids.shape, NEVER, dtype=np.int64)


def oracle_plan(st: SeqState, A: int, B: int, R: int, T: int) -> dict:
    """Index sets for the step that comes next.  Does not modify ``st``.

    Section 4.2: the external window is a fixed-length prefix of the undecoded
    region, fixed within a phase; the internal (active) window is the front of
    what is still undecoded inside it; buffer = external \\ (active ∪ decoded in
    phase); undecoded tokens outside the external window are far-field.
    Section 4.3: a phase is one refresh step followed by normal steps.

    ``st.refresh_mode == 1`` selects a VARIANT that is not in the paper (Section 4.3 recomputes
    everything visible at a refresh): from the second phase on, a refresh step computes only the
    new external window and the tokens decoded during the phase that just ended; every other
    visible position (prompt, tokens of earlier phases) keeps the K/V it already has in the
    cache.  The first step of a state always computes everything (nothing is cached yet).

    ``st.stagger = (i, n)`` selects a second VARIANT that is not in the paper, which never discusses
    batches: sequence i of a batch of n shifts its phase clock by o = i * R // n steps, so that the
    refresh steps of the batch's sequences fall on different steps instead of all on the same one.
    Every sequence still refreshes at step 0 (nothing is cached yet); a sequence with 0 < o < R then
    refreshes again at step o, which makes its first phase o steps long, and every later phase has
    the paper's R steps (Section 4.3).  Each phase is a phase of the paper; only where the phases of
    different sequences begin is new.
    """
    if A < 1 or B < 0 or R < 1 or T < 0:
        raise ValueError("bad window parameters")
    S = len(st.ids)
    # Adaptive termination (Section 4.2): once an end-of-sequence token has been generated the
    # internal window stops advancing: undecoded positions after it are never activated again,
    # they stay in the far field, and generation ends when nothing undecoded is left before it.
    # (Reading: "generated" = unmasked by a step; an eos id inside the given prompt does not count,
    # and the first generated eos in position order is the one that ends the text.)
    limit = S
    if st.eos_id is not None:
        for i in range(S):
            if st.decoded[i] and st.ids[i] == st.eos_id and st.dec_step[i] != NEVER:
                limit = i
                break
    undecoded_all = [i for i in range(S) if not st.decoded[i]]
    U = [i for i in undecoded_all if i < limit]
    if not U:
        return dict(done=True)
    Uset = set(U)
    refresh = (st.t == 0) or (st.since >= R) or not any(i in Uset for i in st.wex)
    if st.stagger is not None:
        offset = (st.stagger[0] * R) // st.stagger[1]
        refresh = refresh or (0 < offset < R and st.t == offset)
    if refresh:
        wex = U[: min(A + B, len(U))]
        phase_start = st.t
    else:
        wex = list(st.wex)
        phase_start = st.phase_start
    W = [i for i in wex if i in Uset]                    # still undecoded part
    act = W[: min(A, len(W))]
    buf = W[len(act):]
    dp = [i for i in wex if i not in Uset]               # decoded within this phase
    trans = [i for i in dp if 1 <= st.t - int(st.dec_step[i]) <= T]
    live = set(W)
    far = [i for i in undecoded_all if i not in live]
    dec = [i for i in range(S) if st.decoded[i]]
    vis = sorted(set(dec) | set(W))
    if not refresh:
        rows = sorted(set(act) | set(trans))
    elif st.refresh_mode == 1 and st.t > 0:
        # st.phase_start is still the start of the phase that just ended
        prev = [i for i in dec if st.dec_step[i] != NEVER and st.dec_step[i] >= st.phase_start]
        rows = sorted(set(W) | set(prev))
    else:
        rows = list(vis)
    return dict(done=False, refresh=refresh, wex=wex, phase_start=phase_start,
                active=act, buffer=buf, in_phase_decoded=dp, transient=trans,
                far_field=far, decoded=dec, vis=vis, rows=rows)


def oracle_commit(st: SeqState, plan: dict, positions, token_ids) -> None:
    """Apply the step's update set U^(t) (Section 3.1) and advance the phase
    counters (Section 4.3)."""
    if plan["refresh"]:
        st.wex = list(plan["wex"])
        st.phase_start = plan["phase_start"]
        st.since = 0
    for p, v in zip(positions, token_ids):
        st.ids[p] = v
        st.decoded[p] = True
        st.dec_step[p] = st.t
    st.t += 1
    st.since += 1


# ---------------------------------------------------------------------------
# model pieces
# ---------------------------------------------------------------------------

def rmsnorm(x: np.ndarray, g: np.ndarray, eps: float) -> np.ndarray:
    ms = np.mean(x * x, axis=-1, keepdims=True)
    return g * x / np.sqrt(ms + eps)


def rope(x: np.ndarray, pos: np.ndarray, theta: float) -> np.ndarray:
    """x: [n, H, dh]; rotate pair (j, j + dh/2) by pos * theta^(-2j/dh)."""
    n, H, dh = x.shape
    half = dh // 2
    j = np.arange(half, dtype=np.float64)
    ang = np.asarray(pos, dtype=np.float64)[:, None] * theta ** (-2.0 * j / dh)[None, :]
    c, s = np.cos(ang)[:, None, :], np.sin(ang)[:, None, :]
    a, b = x[..., :half], x[..., half:]
    return np.concatenate([a * c - b * s, b * c + a * s], axis=-1)


def silu(z: np.ndarray) -> np.ndarray:
    return z / (1.0 + np.exp(-z))


def attention_rows(q: np.ndarray, K: np.ndarray, V: np.ndarray, group: int):
    """Bidirectional attention of n query rows over m visible positions.

    q: [n, Hq, dh]; K, V: [m, Hkv, dh].  Query head h uses KV head h // group.
    Returns (out [n, Hq, dh], probs [n, Hq, m]).  No mask (Section 3.1).
    """
    n, Hq, dh = q.shape
    out = np.empty_like(q)
    probs = np.empty((n, Hq, K.shape[0]), dtype=np.float64)
    for h in range(Hq):
        kv = h // group
        s = q[:, h, :] @ K[:, kv, :].T / np.sqrt(dh)
        s = s - s.max(axis=-1, keepdims=True)
        p = np.exp(s)
        p /= p.sum(axis=-1, keepdims=True)
        probs[:, h, :] = p
        out[:, h, :] = p @ V[:, kv, :]
    return out, probs


@dataclass
class KVCache:
    """Per-sequence fp64 K/V of every layer, indexed by absolute position."""
    K: np.ndarray      # [L, S, Hkv, dh]
    V: np.ndarray

    @staticmethod
    def empty(dims: dict, S: int, fill=np.nan) -> "KVCache":
        shape = (dims["L"], S, dims["Hkv"], dims["dh"])
        return KVCache(np.full(shape, fill), np.full(shape, fill))


# ---------------------------------------------------------------------------
# FP8 mode (an option outside the paper, which calls quantisation orthogonal to the method)
# ---------------------------------------------------------------------------
# With dims["fp8"] set, the projections q/k/v, gate/up, down and the LM head take both operands
# in 8-bit floating point e4m3 (4 exponent bits, 3 mantissa bits, largest finite value 448, no
# infinities): every weight row and every activation row is divided by its own scale
# s = fl32(max |row| / 448) (1 for an all-zero row), rounded to the nearest e4m3 value (ties to
# even), and the product is scaled back by the two row scales.  The output projection, attention,
# the residual stream and the K/V cache are unchanged.

E4M3_MAX = 448.0


def e4m3_round(v32: np.ndarray) -> np.ndarray:
    """Nearest e4m3 value of each float32 (round to nearest even), returned as float64."""
    import torch
    t = torch.from_numpy(np.ascontiguousarray(v32, dtype=np.float32)).to(torch.float8_e4m3fn)
    return t.to(torch.float64).numpy()


def fp8_quant_rows(x: np.ndarray):
    """Per-row e4m3 quantisation of a [n, K] matrix: (values on the e4m3 grid as float64, float32 scales).
    The value that is quantised is the float32 rounding of the input (what a float32 pipeline holds)."""
    x32 = np.asarray(x).astype(np.float32)
    amax = np.abs(x32).max(axis=1) if x32.shape[1] else np.zeros(x32.shape[0], np.float32)
    s = np.where(amax > 0, (amax / np.float32(E4M3_MAX)).astype(np.float32), np.float32(1.0)).astype(np.float32)
    q = e4m3_round((x32 / s[:, None]).astype(np.float32))
    return q, s


def fp8_matmul(x: np.ndarray, w: np.ndarray) -> np.ndarray:
    """x w^T with both operands quantised row by row (see above)."""
    qx, sx = fp8_quant_rows(x)
    qw, sw = fp8_quant_rows(w)
    return (qx @ qw.T) * sx.astype(np.float64)[:, None] * sw.astype(np.float64)[None, :]


# ---------------------------------------------------------------------------
# NVFP4 mode (a second option outside the paper: 4-bit block-scaled operands)
# ---------------------------------------------------------------------------
# With dims["nvfp4"] set, the same projections take both operands in the NVFP4 format: elements are
# 4-bit floats e2m1 (1 sign, 2 exponent, 1 mantissa bit: 0, 0.5, 1, 1.5, 2, 3, 4, 6 and their
# negatives), every block of 16 consecutive elements along the reduction dimension shares one scale
# stored as an unsigned e4m3 number, and every row has one float32 scale on top:
#   g   = fl32(max|row| / (6 * 448))                 (1 for an all-zero row)
#   s_b = e4m3(fl32(fl32(max|block| / 6) / g))       (round to nearest even; at most 448 by construction)
#   q_i = e2m1(fl32(x_i / fl32(s_b * g)))            (round to nearest even, saturating at 6; 0 if s_b = 0)
# and x_i is represented by q_i * s_b * g.  The value that is quantised is the bfloat16 rounding of the
# activation (the pipeline stores its normalised rows as bfloat16 before quantising them); weights are
# bfloat16 already.  The product is the exact sum over blocks of (s_a s_w) * sum_i q_a,i q_w,i, times the
# two row scales.

E2M1_GRID = np.array([0.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0])


def e2m1_round(v32: np.ndarray) -> np.ndarray:
    """Nearest e2m1 value of each float32 (ties to the even code, saturating at +-6), as float64."""
    v = np.asarray(v32, dtype=np.float32).astype(np.float64)
    a = np.abs(v)
    # midpoints between neighbours; a tie goes to the neighbour whose code (index in the grid) is even
    out = np.zeros_like(a)
    for i in range(1, 8):
        mid = (E2M1_GRID[i - 1] + E2M1_GRID[i]) / 2.0
        up = (a > mid) | ((a == mid) & (i % 2 == 0))
        out = np.where(up, E2M1_GRID[i], out)
    return np.copysign(out, v)


def nvfp4_quant_rows(x: np.ndarray):
    """NVFP4 quantisation of a [n, K] matrix, K a multiple of 16: (q on the e2m1 grid [n, K] as float64,
    block scales [n, K / 16] as float64 on the e4m3 grid, row scales [n] float32)."""
    x32 = bf16_round(np.asarray(x)).astype(np.float32)
    n, K = x32.shape
    blocks = x32.reshape(n, K // 16, 16)
    amax = np.abs(x32).max(axis=1) if K else np.zeros(n, np.float32)
    g = np.where(amax > 0, (amax / np.float32(6.0 * 448.0)).astype(np.float32), np.float32(1.0)).astype(np.float32)
    bmax = np.abs(blocks).max(axis=2).astype(np.float32)
    s = e4m3_round(((bmax / np.float32(6.0)).astype(np.float32) / g[:, None]).astype(np.float32))          # float64, on the grid
    d = (s.astype(np.float32) * g[:, None]).astype(np.float32)                                             # fl32(s_b * g)
    safe = np.where(d > 0, d, np.float32(1.0)).astype(np.float32)
    q = e2m1_round((blocks / safe[:, :, None]).astype(np.float32))
    q = np.where(d[:, :, None] > 0, q, 0.0)
    return q.reshape(n, K), s, g


def nvfp4_matmul(x: np.ndarray, w: np.ndarray) -> np.ndarray:
    """x w^T with both operands in NVFP4 (see above)."""
    qx, sx, gx = nvfp4_quant_rows(x)
    qw, sw, gw = nvfp4_quant_rows(w)
    n, K = qx.shape
    m = qw.shape[0]
    out = np.zeros((n, m))
    for b in range(K // 16):
        part = qx[:, 16 * b:16 * b + 16] @ qw[:, 16 * b:16 * b + 16].T
        out += part * sx[:, b][:, None] * sw[:, b][None, :]
    return out * gx.astype(np.float64)[:, None] * gw.astype(np.float64)[None, :]


def _proj(dims: dict, x: np.ndarray, w: np.ndarray) -> np.ndarray:
    if dims.get("nvfp4"):
        return nvfp4_matmul(x, w)
    return fp8_matmul(x, w) if dims.get("fp8") else x @ w.T


# ---------------------------------------------------------------------------
# bfloat16 storage points (a precision mode, not part of the method)
# ---------------------------------------------------------------------------
# bfloat16: 1 sign bit, 8 exponent bits, 7 mantissa bits = the upper half of a float32.  A
# "bf16 in, fp32 accumulate" pipeline holds a value in float32 and stores it as the nearest
# bfloat16 (ties to even).  With dims["bf16_points"] the oracle rounds the same stored values
# in the same way: the normalised rows that feed q/k/v and the feed-forward projections,
# q and k after the rotation, v (i.e. the K/V cache), the attention output that feeds the
# output projection, the SwiGLU product that feeds the down projection, and the normalised
# active rows that feed the LM head.  Everything else stays float64: products, sums, softmax,
# the residual stream, the logits.


def bf16_round(x: np.ndarray) -> np.ndarray:
    """Nearest bfloat16 (ties to even) of the float32 rounding of each value, as float64.
    Written out on the bit pattern: add half of the dropped 16 bits' range minus one, plus the
    lowest kept bit (which breaks ties towards an even mantissa), then clear the dropped bits."""
    b = np.ascontiguousarray(np.asarray(x, dtype=np.float64).astype(np.float32)).view(np.uint32).astype(np.uint64)
    r = ((b + np.uint64(0x7FFF) + ((b >> np.uint64(16)) & np.uint64(1))) & np.uint64(0xFFFF0000)).astype(np.uint32)
    return r.view(np.float32).astype(np.float64).reshape(np.shape(x))


def _store(dims: dict, x: np.ndarray) -> np.ndarray:
    return bf16_round(x) if dims.get("bf16_points") else x


def oracle_layer(dims: dict, lw: dict, x: np.ndarray, pos, vis, cache: KVCache, l: int,
                 want_probs: bool = False) -> dict:
    """One transformer block over the computed rows ``pos`` (ascending
    positions) whose inputs are ``x`` [n, d].  All fresh K/V are written to the
    cache before any row attends; attention then reads every visible position
    from the cache (fresh rows included).  Returns the block output and the
    attention output (before the output projection)."""
    Hq, Hkv, dh = dims["Hq"], dims["Hkv"], dims["dh"]
    n = x.shape[0]
    pos = np.asarray(pos, dtype=np.int64)
    a = _store(dims, rmsnorm(x, lw["attn_norm"], dims["eps"]))
    q = _proj(dims, a, lw["wq"]).reshape(n, Hq, dh)
    k = _proj(dims, a, lw["wk"]).reshape(n, Hkv, dh)
    v = _proj(dims, a, lw["wv"]).reshape(n, Hkv, dh)
    q = _store(dims, rope(q, pos, dims["theta"]))
    k = _store(dims, rope(k, pos, dims["theta"]))
    cache.K[l, pos] = k
    cache.V[l, pos] = _store(dims, v)
    vis = np.asarray(vis, dtype=np.int64)
    o, probs = attention_rows(q, cache.K[l, vis], cache.V[l, vis], Hq // Hkv)
    o = _store(dims, o.reshape(n, Hq * dh))
    h = x + o @ lw["wo"].T
    f = _store(dims, rmsnorm(h, lw["ffn_norm"], dims["eps"]))
    y = h + _proj(dims, _store(dims, silu(_proj(dims, f, lw["w_gate"])) * _proj(dims, f, lw["w_up"])), lw["w_down"])
    res = dict(out=y, attn=o)
    if want_probs:
        res["probs"] = probs
    return res


# ---------------------------------------------------------------------------
# unmask rule
# ---------------------------------------------------------------------------

def oracle_unmask(logits: np.ndarray, positions, k: int) -> dict:
    """Choose which active positions to unmask.

    Per row: token = lowest index among the maximal logits, confidence = the
    softmax probability of that token = 1 / sum_v exp(logit_v - max).  Rows are
    ranked by confidence (descending), equal confidence by position
    (ascending); the first min(k, rows) are unmasked.
    """
    logits = np.asarray(logits, dtype=np.float64)
    n = logits.shape[0]
    ids = np.empty(n, dtype=np.int64)
    conf = np.empty(n, dtype=np.float64)
    for r in range(n):
        m = logits[r].max()
        ids[r] = int(np.flatnonzero(logits[r] == m)[0])
        conf[r] = 1.0 / np.exp(logits[r] - m).sum()
    order = sorted(range(n), key=lambda r: (-conf[r], positions[r]))
    chosen = order[: min(k, n)]
    return dict(ids=ids, conf=conf, order=order,
                positions=[int(positions[r]) for r in chosen],
                token_ids=[int(ids[r]) for r in chosen],
                confidence=[float(conf[r]) for r in chosen])


# ---------------------------------------------------------------------------
# one step
# ---------------------------------------------------------------------------

def _seq_dims(dims: dict, st: SeqState) -> dict:
    """The model dims with this sequence's precision mode switched on."""
    return dict(dims, bf16_points=True) if st.bf16_points else dims


def oracle_step(model, states, caches, A: int, B: int, R: int, T: int, k: int,
                forced=None, want_probs: bool = False, commit: bool = True) -> list:
    """One windowed denoising step for a batch of independent sequences.

    ``model`` supplies float64 weights (``dims``, ``embed_rows``, ``layer``,
    ``final_norm``, ``lm_head``).  ``forced[i]`` = (positions, token_ids)
    replaces sequence i's own unmask choice (teacher forcing).  Returns one
    dict per sequence: the plan, per-layer outputs, attention outputs, logits
    of the active rows, confidences and the chosen update set.
    """
    dims = model.dims
    plans = [oracle_plan(st, A, B, R, T) for st in states]
    outs = []
    xs = []
    for st, pl in zip(states, plans):
        if pl["done"]:
            outs.append(dict(plan=pl, done=True))
            xs.append(None)
            continue
        rows = pl["rows"]
        xs.append(model.embed_rows(st.ids[rows]))
        outs.append(dict(plan=pl, done=False, layer_out=[], attn_out=[], probs=[]))
    for l in range(dims["L"]):
        lw = model.layer(l)
        for i, (pl, cache) in enumerate(zip(plans, caches)):
            if pl["done"]:
                continue
            r = oracle_layer(_seq_dims(dims, states[i]), lw, xs[i], pl["rows"], pl["vis"], cache, l, want_probs)
            xs[i] = r["out"]
            outs[i]["layer_out"].append(r["out"])
            outs[i]["attn_out"].append(r["attn"])
            if want_probs:
                outs[i]["probs"].append(r["probs"])
    g_final = model.final_norm()
    w_lm = None
    for i, (st, pl) in enumerate(zip(states, plans)):
        if pl["done"]:
            continue
        if w_lm is None:
            w_lm = model.lm_head()
        rows = pl["rows"]
        sel = [rows.index(p) for p in pl["active"]]
        sd = _seq_dims(dims, st)
        logits = _proj(sd, _store(sd, rmsnorm(xs[i][sel], g_final, dims["eps"])), w_lm)
        um = oracle_unmask(logits, pl["active"], k)
        outs[i].update(logits=logits, unmask=um)
        if forced is not None and forced[i] is not None:
            pos, tok = forced[i]
        else:
            pos, tok = um["positions"], um["token_ids"]
        outs[i]["committed"] = (list(pos), list(tok))
        if commit:
            oracle_commit(st, pl, pos, tok)
    return outs
