"""ctypes binding over the C ABI of ``libdkv.so`` (see ``include/dkv.h``).

Argument marshalling only: every function has the name and the meaning of its
C counterpart, takes torch tensors where the C function takes device pointers,
and raises ``DkvError`` on a non-zero status.  torch is used for device memory
and streams; no step of the method runs here.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Dict, List, Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libdkv.so")

DKV_OK = 0
DKV_F32, DKV_BF16, DKV_F16 = 0, 1, 2
DKV_POLICY_NONE, DKV_POLICY_DECODE, DKV_POLICY_PREFILL, DKV_POLICY_PD, DKV_POLICY_GREEDY = 0, 1, 2, 3, 4
DKV_CENTER_PREV, DKV_CENTER_CUR = 0, 1
DKV_REFRESH_ALL, DKV_REFRESH_DECODED_ONLY = 0, 1
DKV_SCORE_MAXPROB, DKV_SCORE_MARGIN, DKV_SCORE_NEG_ENTROPY = 0, 1, 2
DKV_PROF_CLASSES = 16

EXPORTS = [
    "dkv_strerror", "dkv_model_bytes", "dkv_model_create", "dkv_model_destroy", "dkv_cache_bytes", "dkv_init_cache",
    "dkv_cache_destroy", "dkv_step", "dkv_refresh", "dkv_select_unmask", "dkv_step_host", "dkv_generate",
    "dkv_get_stats", "dkv_get_provenance", "dkv_get_index_maps", "dkv_status", "dkv_cache_slots",
    "dkv_profile_enable", "dkv_profile_read", "dkv_gemm_workspace_bytes", "dkv_op_gemm", "dkv_op_attention",
    "dkv_static_scratch_bytes", "dkv_op_gemm_static", "dkv_trace_set", "dkv_debug_tail_wait",
    "dkv_cache_state_bytes", "dkv_cache_export", "dkv_cache_import", "dkv_op_stream_probe",
]


class DkvError(RuntimeError):
    def __init__(self, fn: str, status: int):
        self.status = status
        msg = _lib.dkv_strerror(status).decode() if _lib is not None else "?"
        super().__init__(f"{fn} failed: {status} ({msg})")


class dkv_model_desc(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("n_layers", "d_model", "n_q_heads", "n_kv_heads", "head_dim", "d_ffn",
                                         "vocab", "mask_id")] + \
               [("rope_theta", C.c_float), ("rms_eps", C.c_float), ("dtype", C.c_int32), ("act_dtype", C.c_int32)]


class dkv_layer_weights(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("wqkv", "wo", "wgu", "wd", "attn_norm", "ffn_norm")]


class dkv_weights(C.Structure):
    _fields_ = [("embed", C.c_void_p), ("head", C.c_void_p), ("final_norm", C.c_void_p),
                ("layers", C.POINTER(dkv_layer_weights))]


class dkv_policy(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("kind", "refresh_interval", "delay", "window", "window_center",
                                         "max_head_rows", "max_k", "shift", "score",
                                         "isolated_prefill")]


class dkv_stats(C.Structure):
    _fields_ = [("steps", C.c_int64), ("refresh_steps", C.c_int64), ("active_rows", C.c_int64),
                ("total_rows", C.c_int64), ("cache_ratio", C.c_double), ("cache_bytes", C.c_int64),
                ("kernel_launches", C.c_int64)]


class dkv_profile_entry(C.Structure):
    _fields_ = [("name", C.c_char * 32), ("launches", C.c_int64), ("ms", C.c_double), ("bytes", C.c_double),
                ("flops", C.c_double)]


_lib = None


def load():
    """Load libdkv.so; raises if it has not been built (there is no fallback)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2505_15781_b200.build` "
                           "(there is no CPU or PyTorch fallback for the CUDA path)")
    lib = C.CDLL(LIB_PATH)
    vp, i32, sz = C.c_void_p, C.c_int, C.c_size_t
    lib.dkv_strerror.restype = C.c_char_p
    lib.dkv_strerror.argtypes = [i32]
    lib.dkv_model_bytes.restype = sz
    lib.dkv_model_bytes.argtypes = [C.POINTER(dkv_model_desc)]
    lib.dkv_model_create.argtypes = [C.POINTER(dkv_model_desc), C.POINTER(dkv_weights), vp, sz, vp, C.POINTER(vp)]
    lib.dkv_model_destroy.argtypes = [vp]
    lib.dkv_cache_bytes.restype = sz
    lib.dkv_cache_bytes.argtypes = [vp, i32, i32, C.POINTER(dkv_policy)]
    lib.dkv_init_cache.argtypes = [vp, i32, i32, i32, C.POINTER(dkv_policy), vp, sz, vp, C.POINTER(vp)]
    lib.dkv_cache_destroy.argtypes = [vp]
    lib.dkv_step.argtypes = [vp, vp, vp, vp, i32, i32, i32, i32, vp, vp, vp, vp]
    lib.dkv_refresh.argtypes = [vp, i32]
    lib.dkv_select_unmask.argtypes = [vp, vp, i32, i32, i32, i32, i32, vp, vp, vp, vp, vp]
    lib.dkv_step_host.argtypes = [vp, vp, vp, vp, i32, i32, i32, i32, vp, vp]
    lib.dkv_generate.argtypes = [vp, vp, vp, vp, i32, i32, i32, vp, vp]
    lib.dkv_get_stats.argtypes = [vp, C.POINTER(dkv_stats)]
    lib.dkv_get_provenance.argtypes = [vp, vp, vp]
    lib.dkv_get_index_maps.argtypes = [vp, vp, vp, vp, vp]
    lib.dkv_status.argtypes = [vp, C.POINTER(C.c_int32)]
    lib.dkv_cache_slots.argtypes = [vp, i32, C.POINTER(vp), C.POINTER(vp)]
    lib.dkv_cache_state_bytes.restype = sz
    lib.dkv_cache_state_bytes.argtypes = [vp]
    lib.dkv_cache_export.argtypes = [vp, vp, sz, vp]
    lib.dkv_cache_import.argtypes = [vp, vp, sz, vp]
    lib.dkv_profile_enable.argtypes = [vp, i32]
    lib.dkv_profile_read.argtypes = [vp, C.POINTER(dkv_profile_entry), C.POINTER(C.c_int)]
    lib.dkv_gemm_workspace_bytes.restype = sz
    lib.dkv_gemm_workspace_bytes.argtypes = [i32, i32]
    lib.dkv_op_gemm.argtypes = [vp, vp, vp, i32, i32, i32, i32, i32, vp, sz, vp]
    lib.dkv_op_attention.argtypes = [vp, vp, vp, vp, vp, i32, i32, i32, i32, i32, i32, i32, vp]
    lib.dkv_trace_set.argtypes = [vp, i32]
    lib.dkv_debug_tail_wait.argtypes = [vp, C.c_longlong, i32]
    lib.dkv_static_scratch_bytes.restype = sz
    lib.dkv_static_scratch_bytes.argtypes = []
    lib.dkv_op_gemm_static.argtypes = [vp, vp, vp, i32, i32, i32, i32, i32, vp]
    lib.dkv_op_stream_probe.argtypes = [vp, C.c_longlong, vp, C.c_longlong, i32, i32, i32, i32, vp, vp]
    for name in EXPORTS:
        if name not in ("dkv_strerror", "dkv_model_bytes", "dkv_cache_bytes", "dkv_gemm_workspace_bytes",
                        "dkv_static_scratch_bytes", "dkv_cache_state_bytes"):
            getattr(lib, name).restype = C.c_int
    _lib = lib
    return lib


def _check(fn: str, status: int):
    if status != DKV_OK:
        raise DkvError(fn, status)


def _ptr(t) -> Optional[int]:
    if t is None:
        return None
    if isinstance(t, np.ndarray):
        return t.ctypes.data
    return t.data_ptr()


def _stream(stream=None) -> int:
    import torch
    s = stream if stream is not None else torch.cuda.current_stream()
    return s.cuda_stream


# ------------------------------------------------------------------ handles

class Model:
    """Owns the device tensors a dkv_model points to, and the handle."""

    def __init__(self, handle: int, desc: dkv_model_desc, keep: list):
        self.handle, self.desc, self._keep = handle, desc, keep

    def __del__(self):
        if getattr(self, "handle", None) and _lib is not None:
            _lib.dkv_model_destroy(self.handle)
            self.handle = None


class Cache:
    """Owns the arena a dkv_cache lives in, and the handle."""

    def __init__(self, handle: int, model: Model, arena, batch: int, seq_len: int, prompt_len: int,
                 policy: dkv_policy):
        self.handle, self.model, self.arena = handle, model, arena
        self.batch, self.seq_len, self.prompt_len, self.policy = batch, seq_len, prompt_len, policy

    def __del__(self):
        if getattr(self, "handle", None) and _lib is not None:
            _lib.dkv_cache_destroy(self.handle)
            self.handle = None


def make_policy(kind: int, refresh_interval: int = 0, delay: int = 1, window: int = 0,
                window_center: int = DKV_CENTER_PREV, max_head_rows: int = 0, max_k: int = 1,
                shift: int = 0, score: int = 0, isolated_prefill: int = 0) -> dkv_policy:
    return dkv_policy(kind, refresh_interval, delay, window, window_center, max_head_rows, max_k, shift, score,
                      isolated_prefill)


def dkv_model_create(shape, weights: Dict, dtype: int, act_dtype: Optional[int] = None, stream=None) -> Model:
    """shape: synth.ModelShape-like; weights: dict as made by synth.make_weights
    with torch tensors already on the CUDA device in the model dtype.  The
    stacked [Wq;Wk;Wv] and [Wg;Wu] matrices the C ABI wants are assembled here
    (a copy, nothing else)."""
    import torch
    lib = load()
    if act_dtype is None:
        act_dtype = DKV_F32 if dtype == DKV_F32 else DKV_F16
    keep: list = []
    n_layers = len(weights["layers"])
    arr = (dkv_layer_weights * n_layers)()
    for l, lw in enumerate(weights["layers"]):
        wqkv = torch.cat([lw["wq"], lw["wk"], lw["wv"]], dim=0).contiguous()
        wgu = torch.cat([lw["wg"], lw["wu"]], dim=0).contiguous()
        wo, wd = lw["wo"].contiguous(), lw["wd"].contiguous()
        an, fn = lw["attn_norm"].float().contiguous(), lw["ffn_norm"].float().contiguous()
        keep += [wqkv, wgu, wo, wd, an, fn]
        arr[l] = dkv_layer_weights(wqkv.data_ptr(), wo.data_ptr(), wgu.data_ptr(), wd.data_ptr(), an.data_ptr(),
                                   fn.data_ptr())
    embed, head = weights["embed"].contiguous(), weights["head"].contiguous()
    fnorm = weights["final_norm"].float().contiguous()
    keep += [embed, head, fnorm, arr]
    w = dkv_weights(embed.data_ptr(), head.data_ptr(), fnorm.data_ptr(), arr)
    desc = dkv_model_desc(n_layers, shape.d_model, shape.n_q_heads, shape.n_kv_heads, shape.head_dim, shape.d_ffn,
                          shape.vocab, shape.mask_id, shape.rope_theta, shape.rms_eps, dtype, act_dtype)
    out = C.c_void_p()
    need = lib.dkv_model_bytes(C.byref(desc))
    arena, aligned = None, None
    if need:
        arena = torch.empty(need + 256, dtype=torch.uint8, device=embed.device)
        aligned = (arena.data_ptr() + 255) // 256 * 256
    _check("dkv_model_create", lib.dkv_model_create(C.byref(desc), C.byref(w), aligned, need, _stream(stream),
                                                    C.byref(out)))
    if need:
        # the library now reads its fp16 copies; only embed and the norm gains of the originals stay in use
        torch.cuda.current_stream().synchronize()
        keep = [t for t in keep if not (hasattr(t, "dim") and t.dim() == 2 and t is not embed)] + [arena]
    return Model(out.value, desc, keep)


def dkv_cache_bytes(model: Model, batch: int, seq_len: int, policy: dkv_policy) -> int:
    return load().dkv_cache_bytes(model.handle, batch, seq_len, C.byref(policy))


def dkv_init_cache(model: Model, batch: int, seq_len: int, prompt_len: int, policy: dkv_policy, arena=None,
                   stream=None) -> Cache:
    import torch
    lib = load()
    need = dkv_cache_bytes(model, batch, seq_len, policy)
    if need == 0:
        raise DkvError("dkv_cache_bytes", -2)
    if arena is None:
        arena = torch.empty(need + 256, dtype=torch.uint8, device="cuda")
    base = arena.data_ptr()
    aligned = (base + 255) // 256 * 256
    out = C.c_void_p()
    _check("dkv_init_cache", lib.dkv_init_cache(model.handle, batch, seq_len, prompt_len, C.byref(policy), aligned,
                                                arena.numel() - (aligned - base), _stream(stream), C.byref(out)))
    return Cache(out.value, model, arena, batch, seq_len, prompt_len, policy)


def dkv_step(cache: Cache, tokens, masked, next_pos, k: int, cand_lo: int, cand_hi: int, rows_bound: int, conf,
             pred, logits_dbg=None, stream=None):
    _check("dkv_step", load().dkv_step(cache.handle, _ptr(tokens), _ptr(masked), _ptr(next_pos), k, cand_lo,
                                       cand_hi, rows_bound, _ptr(conf), _ptr(pred), _ptr(logits_dbg),
                                       _stream(stream)))


def dkv_refresh(cache: Cache, scope: int = DKV_REFRESH_ALL):
    _check("dkv_refresh", load().dkv_refresh(cache.handle, scope))


def dkv_select_unmask(conf, pred, batch: int, seq_len: int, cand_lo: int, cand_hi: int, k: int, tokens, masked,
                      chosen_pos, status=None, stream=None):
    _check("dkv_select_unmask", load().dkv_select_unmask(_ptr(conf), _ptr(pred), batch, seq_len, cand_lo, cand_hi,
                                                         k, _ptr(tokens), _ptr(masked), _ptr(chosen_pos),
                                                         _ptr(status), _stream(stream)))


def dkv_step_host(cache: Cache, tokens_host, masked_host, next_pos_host, k: int, cand_lo: int, cand_hi: int,
                  rows_bound: int, chosen_host, stream=None):
    """Host buffers: numpy arrays or CPU (ideally pinned) torch tensors, updated in place."""
    _check("dkv_step_host", load().dkv_step_host(cache.handle, _ptr(tokens_host), _ptr(masked_host),
                                                 _ptr(next_pos_host), k, cand_lo, cand_hi, rows_bound,
                                                 _ptr(chosen_host), _stream(stream)))


def dkv_generate(cache: Cache, tokens, masked, order_dev, k: int, block_len: int = 0, n_steps: int = 0,
                 chosen_dev=None, stream=None):
    _check("dkv_generate", load().dkv_generate(cache.handle, _ptr(tokens), _ptr(masked), _ptr(order_dev), k,
                                               block_len, n_steps, _ptr(chosen_dev), _stream(stream)))


def dkv_get_stats(cache: Cache) -> dkv_stats:
    s = dkv_stats()
    _check("dkv_get_stats", load().dkv_get_stats(cache.handle, C.byref(s)))
    return s


def dkv_get_provenance(cache: Cache, written_step, stream=None):
    _check("dkv_get_provenance", load().dkv_get_provenance(cache.handle, _ptr(written_step), _stream(stream)))


def dkv_get_index_maps(cache: Cache, act_idx=None, row_off=None, inv=None, stream=None):
    _check("dkv_get_index_maps", load().dkv_get_index_maps(cache.handle, _ptr(act_idx), _ptr(row_off), _ptr(inv),
                                                           _stream(stream)))


def dkv_status(cache: Cache) -> int:
    """Synchronises; returns the device status word (0 = clean)."""
    w = C.c_int32(0)
    rc = load().dkv_status(cache.handle, C.byref(w))
    if rc not in (0, -7):
        raise DkvError("dkv_status", rc)
    return w.value


def dkv_cache_slots(cache: Cache, layer: int):
    k, v = C.c_void_p(), C.c_void_p()
    _check("dkv_cache_slots", load().dkv_cache_slots(cache.handle, layer, C.byref(k), C.byref(v)))
    return k.value, v.value


def dkv_cache_state_bytes(cache: Cache) -> int:
    return load().dkv_cache_state_bytes(cache.handle)


def dkv_cache_export(cache: Cache, state_host, stream=None):
    """state_host: a CPU uint8 tensor of at least dkv_cache_state_bytes(cache) bytes."""
    _check("dkv_cache_export", load().dkv_cache_export(cache.handle, _ptr(state_host), state_host.numel(),
                                                       _stream(stream)))


def dkv_cache_import(cache: Cache, state_host, stream=None):
    _check("dkv_cache_import", load().dkv_cache_import(cache.handle, _ptr(state_host), state_host.numel(),
                                                       _stream(stream)))


def dkv_profile_enable(cache: Cache, on: bool):
    _check("dkv_profile_enable", load().dkv_profile_enable(cache.handle, 1 if on else 0))


def dkv_profile_read(cache: Cache) -> List[dict]:
    arr = (dkv_profile_entry * DKV_PROF_CLASSES)()
    n = C.c_int(0)
    _check("dkv_profile_read", load().dkv_profile_read(cache.handle, arr, C.byref(n)))
    return [dict(name=arr[i].name.decode(), launches=arr[i].launches, ms=arr[i].ms, bytes=arr[i].bytes,
                 flops=arr[i].flops) for i in range(n.value)]


def dkv_op_stream_probe(streamed, reread, ctas: int, chunk_bytes: int, reread_chunk_bytes: int, stages: int,
                        status=None, stream=None):
    """streamed / reread: CUDA uint8 tensors (reread may be None when reread_chunk_bytes is 0)."""
    _check("dkv_op_stream_probe", load().dkv_op_stream_probe(
        _ptr(streamed), streamed.numel(), _ptr(reread), reread.numel() if reread is not None else 0, ctas,
        chunk_bytes, reread_chunk_bytes, stages, _ptr(status), _stream(stream)))


def dkv_gemm_workspace_bytes(rows: int, n: int) -> int:
    return load().dkv_gemm_workspace_bytes(rows, n)


def dkv_op_gemm(x, w, out, dtype: int, splits: int = 0, workspace=None, stream=None):
    import torch
    rows, k = x.shape
    n = w.shape[0]
    if workspace is None and dtype != DKV_F32:
        workspace = torch.empty(dkv_gemm_workspace_bytes(rows, n), dtype=torch.uint8, device=x.device)
    _check("dkv_op_gemm", load().dkv_op_gemm(_ptr(x), _ptr(w), _ptr(out), rows, n, k, dtype, splits,
                                             _ptr(workspace), workspace.numel() if workspace is not None else 0,
                                             _stream(stream)))
    return workspace


def dkv_op_attention(q, k_slots, v_slots, o, row_off, batch: int, rows_per_seq_bound: int, seq_len: int,
                     n_q_heads: int, n_kv_heads: int, head_dim: int, dtype: int, stream=None):
    _check("dkv_op_attention", load().dkv_op_attention(_ptr(q), _ptr(k_slots), _ptr(v_slots), _ptr(o),
                                                       _ptr(row_off), batch, rows_per_seq_bound, seq_len, n_q_heads,
                                                       n_kv_heads, head_dim, dtype, _stream(stream)))


def dkv_static_scratch_bytes() -> int:
    return load().dkv_static_scratch_bytes()


def dkv_op_gemm_static(x, w, out, dtype: int, splits: int = 0, stream=None):
    """The GEMM for callers that cannot allocate: pointers in, pointers out.
    Nothing is allocated here either (no torch tensor is created)."""
    rows, k = x.shape
    n = w.shape[0]
    _check("dkv_op_gemm_static", load().dkv_op_gemm_static(_ptr(x), _ptr(w), _ptr(out), rows, n, k, dtype, splits,
                                                           _stream(stream)))


def dkv_debug_tail_wait(cache: Cache, wait_cycles: int, never_complete: bool):
    _check("dkv_debug_tail_wait", load().dkv_debug_tail_wait(cache.handle, wait_cycles, 1 if never_complete else 0))


def dkv_trace_set(records, capacity: int):
    """records: torch uint8 tensor of capacity * 24 bytes on the device, or None to switch the trace off."""
    _check("dkv_trace_set", load().dkv_trace_set(_ptr(records), capacity))
