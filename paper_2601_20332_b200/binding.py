"""ctypes binding of libwd.so: the same calls as include/wd.h, argument
marshalling only.  PyTorch appears here for device memory and streams; every
step of the path runs inside the library's CUDA kernels.  There is no CPU
fallback: loading fails loudly if the library has not been built."""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(HERE, "libwd.so")

WD_OK, WD_DONE = 0, 1
WD_ERR_NULL, WD_ERR_INVALID_DIMS, WD_ERR_WORKSPACE_TOO_SMALL, WD_ERR_UNSUPPORTED_ARCH = -1, -2, -3, -4
WD_ERR_BAD_PARAM, WD_ERR_CAPACITY, WD_ERR_PENDING, WD_ERR_CUDA = -5, -6, -7, -8
WD_ERR_DEVICE_TIMEOUT, WD_ERR_BOUNDS, WD_ERR_NOT_PENDING, WD_ERR_MISALIGNED, WD_ERR_INTERNAL = -9, -10, -11, -12, -13
WD_ERR_POISONED = -14
WD_FUSION_AUTO, WD_FUSION_NONE, WD_FUSION_TILE, WD_FUSION_CLUSTER, WD_FUSION_CHAIN = -1, 0, 1, 2, 3
WD_F32, WD_BF16 = 0, 1
WD_GEMM_AUTO, WD_GEMM_PLAIN, WD_GEMM_TCGEN05 = 0, 1, 2

i32, u8p, vp = C.c_int32, C.POINTER(C.c_uint8), C.c_void_p
i32p, f32p = C.POINTER(C.c_int32), C.POINTER(C.c_float)


class wd_model_dims(C.Structure):
    _fields_ = [(n, i32) for n in ("n_layers", "d_model", "n_q_heads", "n_kv_heads", "head_dim", "d_ffn", "vocab")] + \
               [("rope_theta", C.c_float), ("rms_eps", C.c_float)] + \
               [(n, i32) for n in ("dtype", "mask_id", "max_batch", "max_seq", "max_rows", "max_active")]


class wd_weights(C.Structure):
    _fields_ = [("tok_embed", vp)] + [(n, C.POINTER(vp)) for n in ("wq", "wk", "wv", "wo", "w_gate", "w_up", "w_down",
                                                                    "attn_norm", "ffn_norm")] + \
               [("final_norm", vp), ("lm_head", vp)]


class wd_index_sets(C.Structure):
    _fields_ = [("capacity", i32),
                ("active", i32p), ("n_active", i32), ("buffer", i32p), ("n_buffer", i32),
                ("decoded", i32p), ("n_decoded", i32), ("transient", i32p), ("n_transient", i32),
                ("far_field", i32p), ("n_far_field", i32), ("rows", i32p), ("n_rows", i32),
                ("vis", i32p), ("n_vis", i32), ("ext_window", i32p), ("n_ext_window", i32),
                ("is_refresh", i32), ("vis_contiguous", i32), ("done", i32)]


class wd_step_out(C.Structure):
    _fields_ = [("n_unmasked", i32p), ("positions", i32p), ("token_ids", i32p), ("confidence", f32p)]


class wd_debug_taps(C.Structure):
    _fields_ = [("layer_out", vp), ("attn_out", vp), ("logits", vp)]


class wd_step_info(C.Structure):
    _fields_ = [(n, i32) for n in ("is_refresh", "n_rows", "n_active", "n_vis", "n_launches", "gemm_impl")]


# name -> (restype, argtypes); must list every symbol include/wd.h declares
SIGNATURES = {
    "wd_workspace_bytes": (C.c_size_t, [C.POINTER(wd_model_dims)]),
    "wd_state_bytes": (C.c_size_t, [C.POINTER(wd_model_dims), i32, i32]),
    "wd_version": (i32, []),
    "wd_kv_bytes": (C.c_size_t, [C.POINTER(wd_model_dims), i32, i32]),
    "wd_last_error": (C.c_char_p, []),
    "wd_state_export_bytes": (C.c_size_t, [vp]),
    "wd_state_export": (C.c_int, [vp, vp, C.c_size_t]),
    "wd_state_import": (C.c_int, [vp, vp, C.c_size_t, i32, vp]),
    "wd_debug_poke_id": (C.c_int, [vp, i32, i32, i32, vp]),
    "wd_status_string": (C.c_char_p, [C.c_int]),
    "wd_create": (C.c_int, [C.POINTER(wd_model_dims), C.POINTER(wd_weights), vp, C.c_size_t, C.POINTER(vp)]),
    "wd_destroy": (C.c_int, [vp]),
    "wd_set_gemm_impl": (C.c_int, [vp, i32]),
    "wd_set_fusion": (C.c_int, [vp, i32]),
    "wd_profile_enable": (C.c_int, [vp, i32]),
    "wd_profile_read": (C.c_int, [vp, C.POINTER(C.c_double), C.POINTER(C.c_double), C.POINTER(C.c_int64)]),
    "wd_state_create": (C.c_int, [vp, i32, i32, i32p, u8p, vp, C.c_size_t, C.POINTER(vp)]),
    "wd_state_reset": (C.c_int, [vp, i32p, u8p, vp]),
    "wd_state_destroy": (C.c_int, [vp]),
    "wd_state_read": (C.c_int, [vp, i32, i32p, u8p, i32p, i32p, i32p]),
    "wd_debug_taps_set": (C.c_int, [vp, C.POINTER(wd_debug_taps)]),
    "wd_plan": (C.c_int, [vp, i32, i32, i32, i32, i32, C.POINTER(wd_index_sets)]),
    "wd_plan_raw": (C.c_int, [u8p, i32p, i32p, i32, i32, i32, i32, i32p, i32, i32, i32, i32, i32, i32, i32, i32,
                              C.POINTER(wd_index_sets)]),
    "wd_set_graphs": (C.c_int, [vp, i32]),
    "wd_debug_graph_stats": (C.c_int, [vp, C.POINTER(i32), C.POINTER(i32)]),
    "wd_fp8_bytes": (C.c_size_t, [C.POINTER(wd_model_dims)]),
    "wd_fp8_enable": (C.c_int, [vp, vp, C.c_size_t, vp]),
    "wd_fp8_set": (C.c_int, [vp, i32]),
    "wd_fp4_bytes": (C.c_size_t, [C.POINTER(wd_model_dims)]),
    "wd_fp4_enable": (C.c_int, [vp, vp, C.c_size_t, vp]),
    "wd_fp4_set": (C.c_int, [vp, i32]),
    "wd_state_set_eos": (C.c_int, [vp, i32]),
    "wd_state_set_refresh_mode": (C.c_int, [vp, i32]),
    "wd_state_set_stagger": (C.c_int, [vp, i32]),
    "wd_step": (C.c_int, [vp, i32, i32, i32, i32, i32, vp, C.POINTER(wd_step_info)]),
    "wd_step_sync": (C.c_int, [vp, C.POINTER(wd_step_out)]),
    "wd_step_sync_all": (C.c_int, [vp, C.POINTER(wd_step_out), i32, i32p]),
    "wd_generate": (C.c_int, [vp, i32, i32, i32, i32, i32, i32, vp, i32p, i32p]),
    "wd_op_gemm": (C.c_int, [i32, i32, vp, vp, vp, i32, i32, i32, vp, C.c_size_t, vp]),
    "wd_op_gemm_scratch_bytes": (C.c_size_t, [i32, i32, i32]),
    "wd_op_gemm_fp8": (C.c_int, [vp, vp, vp, i32, i32, i32, vp, C.c_size_t, vp]),
    "wd_op_gemm_fp8_scratch_bytes": (C.c_size_t, [i32, i32, i32]),
    "wd_op_gemm_fp4": (C.c_int, [vp, vp, vp, i32, i32, i32, vp, C.c_size_t, vp]),
    "wd_op_gemm_fp4_scratch_bytes": (C.c_size_t, [i32, i32, i32]),
    "wd_op_nvfp4_bytes": (C.c_size_t, [i32, i32]),
    "wd_op_nvfp4_quantize": (C.c_int, [vp, i32, i32, vp, C.c_size_t, vp]),
    "wd_op_gemm_nvfp4": (C.c_int, [vp, vp, vp, i32, i32, i32, vp, C.c_size_t, vp]),
    "wd_op_gemm_noalloc": (C.c_int, [vp, vp, vp, i32, i32, i32, vp]),
    "wd_op_gemm_noalloc_max_floats": (C.c_size_t, []),
    "wd_op_attention": (C.c_int, [i32, vp, vp, vp, vp, vp, i32, i32, i32, i32, i32, i32, vp]),
    "wd_op_unmask": (C.c_int, [vp, vp, i32, i32, i32, vp, vp, vp, vp, vp, vp, vp, vp, C.c_size_t, vp]),
    "wd_op_unmask_scratch_bytes": (C.c_size_t, [i32, i32]),
    "wd_op_attention_tc": (C.c_int, [vp, vp, vp, vp, i32, i32, i32, i32, i32, i32, vp, C.c_size_t, vp]),
    "wd_op_attention_tc_scratch_bytes": (C.c_size_t, [i32]),
    "wd_op_lm_unmask": (C.c_int, [vp, vp, vp, i32, i32, i32, i32, vp, vp, vp, vp, vp, vp, vp, vp, vp, C.c_size_t, vp]),
    "wd_op_lm_unmask_scratch_bytes": (C.c_size_t, [i32, i32]),
    "wd_op_status": (C.c_int, []),
    "wd_debug_wait_expire": (C.c_int, [vp]),
}

_lib = None


def lib():
    """Load libwd.so (once).  Raises if it is missing: there is no other path."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} not found: build it with `python -m paper_2601_20332_b200.build` "
                               "(there is no CPU fallback)")
        L = C.CDLL(LIB_PATH)
        for name, (res, args) in SIGNATURES.items():
            fn = getattr(L, name)
            fn.restype, fn.argtypes = res, args
        _lib = L
    return _lib


class WdError(RuntimeError):
    def __init__(self, status, where):
        self.status = status
        super().__init__(f"{where}: {lib().wd_status_string(status).decode()} ({status})")


def check(status, where):
    if status < 0:
        raise WdError(status, where)
    return status


def _np_i32p(a):
    return a.ctypes.data_as(i32p)


def _stream_ptr(stream):
    return None if stream is None else C.c_void_p(stream.cuda_stream)


def _ptr(t):
    return None if t is None else C.c_void_p(t.data_ptr())


def make_dims(cfg: dict, max_batch: int, max_seq: int, max_rows: int, max_active: int) -> wd_model_dims:
    return wd_model_dims(cfg["L"], cfg["d"], cfg["Hq"], cfg["Hkv"], cfg["dh"], cfg["F"], cfg["V"],
                         float(cfg["theta"]), float(cfg["eps"]), WD_F32 if cfg["dtype"] == "f32" else WD_BF16,
                         cfg["mask_id"], max_batch, max_seq, max_rows, max_active)


_LISTS = ("active", "buffer", "decoded", "transient", "far_field", "rows", "vis", "ext_window")


def _index_sets(cap: int):
    bufs = {n: np.empty(max(cap, 1), np.int32) for n in _LISTS}
    s = wd_index_sets()
    s.capacity = cap
    for n, b in bufs.items():
        setattr(s, n, _np_i32p(b))
    return s, bufs


def _index_sets_dict(s, bufs) -> dict:
    out = {n: bufs[n][: getattr(s, "n_" + n)].tolist() for n in bufs}
    out.update(refresh=bool(s.is_refresh), vis_contiguous=bool(s.vis_contiguous), done=bool(s.done))
    return out


WD_REFRESH_FULL, WD_REFRESH_WINDOW = 0, 1


def plan_raw(decoded, dec_step, t: int, since: int, ext_window, A: int, B: int, R: int, T: int,
             token_ids=None, eos_id: int = -1, refresh_mode: int = WD_REFRESH_FULL, stagger=None) -> dict:
    """wd_plan_raw: the host planner on explicit state arrays (needs no GPU)."""
    dec = np.ascontiguousarray(decoded, dtype=np.uint8)
    ds = np.ascontiguousarray(dec_step, dtype=np.int32)
    wex = np.ascontiguousarray(ext_window, dtype=np.int32)
    ids = None if token_ids is None else np.ascontiguousarray(token_ids, dtype=np.int32)
    s, bufs = _index_sets(len(dec))
    check(lib().wd_plan_raw(dec.ctypes.data_as(u8p), _np_i32p(ds), None if ids is None else _np_i32p(ids), eos_id,
                            len(dec), t, since, _np_i32p(wex) if len(wex) else None, len(wex), A, B, R, T,
                            refresh_mode, stagger[0] if stagger else 0, stagger[1] if stagger else 0, C.byref(s)), "wd_plan_raw")
    return _index_sets_dict(s, bufs)


class Context:
    """wd_create / wd_destroy.  `weights` is a synth.Weights on the CUDA device."""

    def __init__(self, cfg: dict, weights, max_batch: int, max_seq: int, max_rows: int, max_active: int):
        import torch
        self.cfg, self.weights = cfg, weights
        self.dims = make_dims(cfg, max_batch, max_seq, max_rows, max_active)
        nbytes = lib().wd_workspace_bytes(C.byref(self.dims))
        if nbytes == 0:
            raise WdError(WD_ERR_INVALID_DIMS, "wd_workspace_bytes")
        self.workspace = torch.empty(nbytes, dtype=torch.uint8, device=weights.tok_embed.device)
        L = cfg["L"]

        def arr(tensors):
            return (vp * L)(*[t.data_ptr() for t in tensors])

        self._arrays = [arr(getattr(weights, n)) for n in ("wq", "wk", "wv", "wo", "w_gate", "w_up", "w_down",
                                                           "attn_norm", "ffn_norm")]
        w = wd_weights(weights.tok_embed.data_ptr(), *self._arrays, weights.final_norm.data_ptr(),
                       weights.lm_head.data_ptr())
        self.handle = vp()
        check(lib().wd_create(C.byref(self.dims), C.byref(w), _ptr(self.workspace), nbytes, C.byref(self.handle)),
              "wd_create")

    def set_gemm_impl(self, impl: int):
        check(lib().wd_set_gemm_impl(self.handle, impl), "wd_set_gemm_impl")

    def set_fusion(self, mode: int):
        """A WD_FUSION_* mode: where the consumers of the GEMMs run (same results within rounding)."""
        check(lib().wd_set_fusion(self.handle, int(mode)), "wd_set_fusion")

    def profile_enable(self, on: bool):
        check(lib().wd_profile_enable(self.handle, 1 if on else 0), "wd_profile_enable")

    def set_graphs(self, on: bool):
        check(lib().wd_set_graphs(self.handle, 1 if on else 0), "wd_set_graphs")

    def graph_stats(self):
        """(graphs recorded, steps replayed) since the context was created."""
        a, b = i32(0), i32(0)
        check(lib().wd_debug_graph_stats(self.handle, C.byref(a), C.byref(b)), "wd_debug_graph_stats")
        return a.value, b.value

    def fp8_enable(self, stream=None):
        """wd_fp8_enable: quantise the weights to e4m3 and run the projections in FP8 from now on."""
        import torch
        nbytes = lib().wd_fp8_bytes(C.byref(self.dims))
        if nbytes == 0:
            raise WdError(WD_ERR_BAD_PARAM, "wd_fp8_bytes")
        self._fp8_mem = torch.empty(nbytes, dtype=torch.uint8, device=self.workspace.device)
        check(lib().wd_fp8_enable(self.handle, _ptr(self._fp8_mem), nbytes, _stream_ptr(stream)), "wd_fp8_enable")

    def fp8_set(self, on: bool):
        check(lib().wd_fp8_set(self.handle, 1 if on else 0), "wd_fp8_set")

    def fp4_enable(self, stream=None):
        """wd_fp4_enable: quantise the weights to NVFP4 and run the projections in NVFP4 from now on."""
        import torch
        nbytes = lib().wd_fp4_bytes(C.byref(self.dims))
        if nbytes == 0:
            raise WdError(WD_ERR_BAD_PARAM, "wd_fp4_bytes")
        self._fp4_mem = torch.empty(nbytes, dtype=torch.uint8, device=self.workspace.device)
        check(lib().wd_fp4_enable(self.handle, _ptr(self._fp4_mem), nbytes, _stream_ptr(stream)), "wd_fp4_enable")

    def fp4_set(self, on: bool):
        check(lib().wd_fp4_set(self.handle, 1 if on else 0), "wd_fp4_set")

    def profile_read(self) -> dict:
        ms, by, n = C.c_double(), C.c_double(), C.c_int64()
        check(lib().wd_profile_read(self.handle, C.byref(ms), C.byref(by), C.byref(n)), "wd_profile_read")
        return dict(gemm_ms=ms.value, gemm_bytes=by.value, gemm_launches=n.value)

    def close(self):
        if self.handle:
            lib().wd_destroy(self.handle)
            self.handle = vp()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


class State:
    """wd_state_* / wd_plan / wd_step / wd_step_sync for one batch of sequences."""

    def __init__(self, ctx: Context, token_ids: np.ndarray, decoded: np.ndarray | None = None):
        import torch
        self.ctx = ctx
        ids = np.ascontiguousarray(token_ids, dtype=np.int32)
        self.batch, self.S = ids.shape
        nbytes = lib().wd_state_bytes(C.byref(ctx.dims), self.batch, self.S)
        if nbytes == 0:
            raise WdError(WD_ERR_BAD_PARAM, "wd_state_bytes")
        self.mem = torch.empty(nbytes, dtype=torch.uint8, device=ctx.workspace.device)
        dec = None if decoded is None else np.ascontiguousarray(decoded, dtype=np.uint8)
        self.handle = vp()
        check(lib().wd_state_create(ctx.handle, self.batch, self.S, _np_i32p(ids),
                                    None if dec is None else dec.ctypes.data_as(u8p), _ptr(self.mem), nbytes,
                                    C.byref(self.handle)), "wd_state_create")
        self._taps = None
        self._k = 1

    def reset(self, token_ids: np.ndarray, decoded: np.ndarray | None = None, stream=None):
        ids = np.ascontiguousarray(token_ids, dtype=np.int32)
        dec = None if decoded is None else np.ascontiguousarray(decoded, dtype=np.uint8)
        check(lib().wd_state_reset(self.handle, _np_i32p(ids), None if dec is None else dec.ctypes.data_as(u8p),
                                   _stream_ptr(stream)), "wd_state_reset")

    def read(self, seq: int = 0) -> dict:
        ids = np.empty(self.S, np.int32); dec = np.empty(self.S, np.uint8); ds = np.empty(self.S, np.int32)
        t, since = i32(), i32()
        check(lib().wd_state_read(self.handle, seq, _np_i32p(ids), dec.ctypes.data_as(u8p), _np_i32p(ds),
                                  C.byref(t), C.byref(since)), "wd_state_read")
        return dict(ids=ids, decoded=dec.astype(bool), dec_step=ds, t=t.value, since=since.value)

    def export(self) -> bytes:
        """wd_state_export: the sequence state and phase bookkeeping as one blob (the K/V cache is not in it)."""
        n = lib().wd_state_export_bytes(self.handle)
        buf = C.create_string_buffer(n)
        check(lib().wd_state_export(self.handle, buf, n), "wd_state_export")
        return buf.raw

    def import_(self, blob: bytes, cache_valid: bool, stream=None):
        """wd_state_import: resume from a blob; cache_valid=False makes the next step a refresh."""
        check(lib().wd_state_import(self.handle, blob, len(blob), 1 if cache_valid else 0, _stream_ptr(stream)),
              "wd_state_import")

    def poke_id(self, seq: int, pos: int, token_id: int, stream=None):
        """wd_debug_poke_id: overwrite one entry of the device copy of the ids, unchecked (test hook)."""
        check(lib().wd_debug_poke_id(self.handle, seq, pos, token_id, _stream_ptr(stream)), "wd_debug_poke_id")

    def plan(self, seq: int, A: int, B: int, R: int, T: int) -> dict:
        s, bufs = _index_sets(self.S)
        check(lib().wd_plan(self.handle, seq, A, B, R, T, C.byref(s)), "wd_plan")
        return _index_sets_dict(s, bufs)

    def set_eos(self, eos_id: int):
        """Adaptive termination: stop extending the window past a generated eos token (-1 = off)."""
        check(lib().wd_state_set_eos(self.handle, eos_id), "wd_state_set_eos")

    def set_refresh_mode(self, mode: int):
        """WD_REFRESH_FULL (the paper's refresh) or WD_REFRESH_WINDOW (variant outside the paper)."""
        check(lib().wd_state_set_refresh_mode(self.handle, mode), "wd_state_set_refresh_mode")

    def set_stagger(self, on: bool):
        """Staggered refresh steps across the sequences of the batch (variant outside the paper)."""
        check(lib().wd_state_set_stagger(self.handle, 1 if on else 0), "wd_state_set_stagger")

    def set_taps(self, layer_out=None, attn_out=None, logits=None):
        """Device float tensors that receive intermediates of later steps (None = off)."""
        self._taps = (layer_out, attn_out, logits)
        if layer_out is None and attn_out is None and logits is None:
            check(lib().wd_debug_taps_set(self.handle, None), "wd_debug_taps_set")
        else:
            t = wd_debug_taps(_ptr(layer_out), _ptr(attn_out), _ptr(logits))
            check(lib().wd_debug_taps_set(self.handle, C.byref(t)), "wd_debug_taps_set")

    def step(self, A: int, B: int, R: int, T: int, k: int, stream=None) -> tuple:
        """Enqueue one step.  Returns (status, info dict)."""
        info = wd_step_info()
        st = check(lib().wd_step(self.handle, A, B, R, T, k, _stream_ptr(stream), C.byref(info)), "wd_step")
        self._k = k
        return st, {n: getattr(info, n) for n, _ in wd_step_info._fields_}

    def sync(self) -> dict:
        k = max(self._k, 1)
        n = np.zeros(self.batch, np.int32)
        pos = np.full(self.batch * k, -1, np.int32); tok = np.full(self.batch * k, -1, np.int32)
        conf = np.zeros(self.batch * k, np.float32)
        out = wd_step_out(_np_i32p(n), _np_i32p(pos), _np_i32p(tok), conf.ctypes.data_as(f32p))
        check(lib().wd_step_sync(self.handle, C.byref(out)), "wd_step_sync")
        return dict(n_unmasked=n, positions=pos.reshape(self.batch, k), token_ids=tok.reshape(self.batch, k),
                    confidence=conf.reshape(self.batch, k))

    def sync_all(self, max_steps: int = 32) -> list:
        """wd_step_sync_all: results of every enqueued step, oldest first (all enqueued with the same k)."""
        k = max(self._k, 1)
        bufs, outs = [], (wd_step_out * max_steps)()
        for i in range(max_steps):
            n = np.zeros(self.batch, np.int32)
            pos = np.full(self.batch * k, -1, np.int32); tok = np.full(self.batch * k, -1, np.int32)
            conf = np.zeros(self.batch * k, np.float32)
            bufs.append((n, pos, tok, conf))
            outs[i] = wd_step_out(_np_i32p(n), _np_i32p(pos), _np_i32p(tok), conf.ctypes.data_as(f32p))
        done = i32()
        check(lib().wd_step_sync_all(self.handle, outs, max_steps, C.byref(done)), "wd_step_sync_all")
        return [dict(n_unmasked=n, positions=pos.reshape(self.batch, k), token_ids=tok.reshape(self.batch, k),
                     confidence=conf.reshape(self.batch, k)) for (n, pos, tok, conf) in bufs[: done.value]]

    def generate(self, A: int, B: int, R: int, T: int, k: int, max_steps: int = 0, stream=None) -> tuple:
        """wd_generate: run steps until done (or max_steps).  Returns (status, steps, tokens unmasked)."""
        n_steps, n_tok = i32(), i32()
        st = check(lib().wd_generate(self.handle, A, B, R, T, k, max_steps, _stream_ptr(stream), C.byref(n_steps),
                                     C.byref(n_tok)), "wd_generate")
        return st, n_steps.value, n_tok.value

    def close(self):
        if self.handle:
            lib().wd_state_destroy(self.handle)
            self.handle = vp()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


# ---- single operations ------------------------------------------------------

def _dtype_code(t):
    import torch
    return WD_F32 if t.dtype == torch.float32 else WD_BF16


def op_gemm(x, w, impl: int = WD_GEMM_AUTO, stream=None, scratch=None):
    """y[rows, n] (float32) = x[rows, k] @ w[n, k]^T on the GPU."""
    import torch
    rows, k = x.shape
    n = w.shape[0]
    y = torch.empty(rows, n, dtype=torch.float32, device=x.device)
    if scratch is None:
        nb = lib().wd_op_gemm_scratch_bytes(rows, n, k)
        scratch = torch.empty(max(nb, 256), dtype=torch.uint8, device=x.device)
    check(lib().wd_op_gemm(_dtype_code(x), impl, _ptr(x), _ptr(w), _ptr(y), rows, n, k, _ptr(scratch),
                           scratch.numel(), _stream_ptr(stream)), "wd_op_gemm")
    return y


def op_gemm_fp8(x, w, stream=None):
    """y[rows, n] (float32) = FP8 product of the bf16 operands (per-row e4m3 quantisation of both)."""
    import torch
    rows, k = x.shape
    n = w.shape[0]
    y = torch.empty(rows, n, dtype=torch.float32, device=x.device)
    nb = lib().wd_op_gemm_fp8_scratch_bytes(rows, n, k)
    scratch = torch.empty(max(nb, 256), dtype=torch.uint8, device=x.device)
    check(lib().wd_op_gemm_fp8(_ptr(x), _ptr(w), _ptr(y), rows, n, k, _ptr(scratch), nb, _stream_ptr(stream)), "wd_op_gemm_fp8")
    return y


def op_gemm_fp4(x, w, stream=None):
    """y[rows, n] (float32) = NVFP4 product of the bf16 operands (e2m1 codes, e4m3 block scales, float row scales)."""
    import torch
    rows, k = x.shape
    n = w.shape[0]
    y = torch.empty(rows, n, dtype=torch.float32, device=x.device)
    nb = lib().wd_op_gemm_fp4_scratch_bytes(rows, n, k)
    scratch = torch.empty(max(nb, 256), dtype=torch.uint8, device=x.device)
    check(lib().wd_op_gemm_fp4(_ptr(x), _ptr(w), _ptr(y), rows, n, k, _ptr(scratch), nb, _stream_ptr(stream)), "wd_op_gemm_fp4")
    return y


def op_nvfp4_quantize(x, stream=None):
    """The NVFP4 form of a bf16 matrix [rows, k] as one uint8 device tensor (codes | block scales | row scales)."""
    import torch
    rows, k = x.shape
    nb = lib().wd_op_nvfp4_bytes(rows, k)
    if nb == 0:
        raise WdError(WD_ERR_BAD_PARAM, "wd_op_nvfp4_bytes")
    out = torch.empty(nb, dtype=torch.uint8, device=x.device)
    check(lib().wd_op_nvfp4_quantize(_ptr(x), rows, k, _ptr(out), nb, _stream_ptr(stream)), "wd_op_nvfp4_quantize")
    return out


def op_gemm_nvfp4(xq, wq, rows, n, k, scratch=None, stream=None):
    """y[rows, n] (float32) from two operands quantised by op_nvfp4_quantize."""
    import torch
    y = torch.empty(rows, n, dtype=torch.float32, device=xq.device)
    nb = lib().wd_op_gemm_scratch_bytes(rows, n, k)
    if scratch is None:
        scratch = torch.empty(max(nb, 256), dtype=torch.uint8, device=xq.device)
    check(lib().wd_op_gemm_nvfp4(_ptr(xq), _ptr(wq), _ptr(y), rows, n, k, _ptr(scratch), scratch.numel(), _stream_ptr(stream)),
          "wd_op_gemm_nvfp4")
    return y


def op_gemm_noalloc(x, w, y=None, stream=None):
    """wd_op_gemm_noalloc: bf16 GEMM whose scratch is a fixed array inside the library, for
    callers that may not allocate.  Pass a preallocated float32 `y` to keep this wrapper
    allocation-free as well."""
    import torch
    rows, k = x.shape
    n = w.shape[0]
    if y is None:
        y = torch.empty(rows, n, dtype=torch.float32, device=x.device)
    check(lib().wd_op_gemm_noalloc(_ptr(x), _ptr(w), _ptr(y), rows, n, k, _stream_ptr(stream)), "wd_op_gemm_noalloc")
    return y


def op_attention(q, kcache, vcache, vis, stream=None):
    """q: [rows, Hq, dh]; kcache: [Hkv, S, dh]; vcache transposed: [Hkv, dh, S]; vis: int32 [n_vis] (device)."""
    import torch
    rows, Hq, dh = q.shape
    Hkv, S, _ = kcache.shape
    out = torch.empty_like(q)
    check(lib().wd_op_attention(_dtype_code(q), _ptr(q), _ptr(kcache), _ptr(vcache), _ptr(vis), _ptr(out), rows,
                                vis.numel(), Hq, Hkv, dh, S, _stream_ptr(stream)), "wd_op_attention")
    return out


def op_attention_tc(q, kcache, vcache_t, n_vis: int, max_vis: int = 0, stream=None):
    """Tensor-core attention over positions [0, n_vis).  q: [rows, Hq, 128] bf16; kcache: [Hkv, S, 128];
    vcache_t transposed: [Hkv, 128, S]; max_vis (default n_vis) sizes the key split."""
    import torch
    rows, Hq, dh = q.shape
    Hkv, S, _ = kcache.shape
    assert dh == 128
    out = torch.empty_like(q)
    nb = lib().wd_op_attention_tc_scratch_bytes(rows)
    scratch = torch.empty(nb, dtype=torch.uint8, device=q.device)
    check(lib().wd_op_attention_tc(_ptr(q), _ptr(kcache), _ptr(vcache_t), _ptr(out), rows, n_vis, max(max_vis, n_vis), Hq,
                                   Hkv, S, _ptr(scratch), nb, _stream_ptr(stream)), "wd_op_attention_tc")
    return out


def op_lm_unmask(x, w, positions, k: int, stream=None) -> dict:
    """x: bf16 [n, K] normalised rows; w: bf16 [V, K] LM head; positions: int32 [n] ascending (all device).
    Returns the per-row statistics, the selection and the logits the tensor-core GEMM produced."""
    import torch
    n, K = x.shape
    V = w.shape[0]
    dev = x.device
    kk = max(k, 1)
    logits = torch.empty(n, V, dtype=torch.float32, device=dev)
    row_token = torch.empty(n, dtype=torch.int32, device=dev)
    row_sumexp = torch.empty(n, dtype=torch.float64, device=dev)
    row_conf = torch.empty(n, dtype=torch.float32, device=dev)
    sel_pos = torch.full((kk,), -1, dtype=torch.int32, device=dev)
    sel_tok = torch.full((kk,), -1, dtype=torch.int32, device=dev)
    sel_conf = torch.zeros(kk, dtype=torch.float32, device=dev)
    n_sel = torch.zeros(1, dtype=torch.int32, device=dev)
    nb = lib().wd_op_lm_unmask_scratch_bytes(n, V)
    scratch = torch.empty(nb, dtype=torch.uint8, device=dev)
    check(lib().wd_op_lm_unmask(_ptr(x), _ptr(w), _ptr(positions), n, V, K, k, _ptr(logits), _ptr(row_token),
                                _ptr(row_sumexp), _ptr(row_conf), _ptr(sel_pos), _ptr(sel_tok), _ptr(sel_conf), _ptr(n_sel),
                                _ptr(scratch), nb, _stream_ptr(stream)), "wd_op_lm_unmask")
    ns = int(n_sel.item())
    return dict(logits=logits, row_token=row_token.cpu().numpy(), row_sumexp=row_sumexp.cpu().numpy(),
                row_conf=row_conf.cpu().numpy(), positions=sel_pos.cpu().numpy()[:ns].tolist(),
                token_ids=sel_tok.cpu().numpy()[:ns].tolist(), confidence=sel_conf.cpu().numpy()[:ns].tolist())


def op_unmask(logits, positions, k: int, stream=None) -> dict:
    """logits: float32 [n, V] (device); positions: int32 [n] ascending (device)."""
    import torch
    n, V = logits.shape
    dev = logits.device
    kk = max(k, 1)
    row_token = torch.empty(n, dtype=torch.int32, device=dev)
    row_sumexp = torch.empty(n, dtype=torch.float64, device=dev)
    row_conf = torch.empty(n, dtype=torch.float32, device=dev)
    sel_pos = torch.full((kk,), -1, dtype=torch.int32, device=dev)
    sel_tok = torch.full((kk,), -1, dtype=torch.int32, device=dev)
    sel_conf = torch.zeros(kk, dtype=torch.float32, device=dev)
    n_sel = torch.zeros(1, dtype=torch.int32, device=dev)
    scratch = torch.empty(lib().wd_op_unmask_scratch_bytes(n, V), dtype=torch.uint8, device=dev)
    check(lib().wd_op_unmask(_ptr(logits), _ptr(positions), n, V, k, _ptr(row_token), _ptr(row_sumexp),
                             _ptr(row_conf), _ptr(sel_pos), _ptr(sel_tok), _ptr(sel_conf), _ptr(n_sel),
                             _ptr(scratch), scratch.numel(), _stream_ptr(stream)), "wd_op_unmask")
    ns = int(n_sel.item())
    return dict(row_token=row_token.cpu().numpy(), row_sumexp=row_sumexp.cpu().numpy(),
                row_conf=row_conf.cpu().numpy(), positions=sel_pos.cpu().numpy()[:ns].tolist(),
                token_ids=sel_tok.cpu().numpy()[:ns].tolist(), confidence=sel_conf.cpu().numpy()[:ns].tolist())


def op_status() -> int:
    return lib().wd_op_status()


def debug_wait_expire(stream=None) -> None:
    """Launch the kernel whose bounded wait runs out (see wd_debug_wait_expire)."""
    check(lib().wd_debug_wait_expire(_stream_ptr(stream)), "wd_debug_wait_expire")
