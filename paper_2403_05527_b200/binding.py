"""ctypes binding of libgear_b200.so: the C entry points of include/gear.h under
the same names.  Only argument marshalling happens here -- torch supplies device
memory and the stream handle; every step of the method runs in the CUDA library.

The library is loaded on first use; if it is missing the call raises (there is
no CPU fallback).
"""
from __future__ import annotations

import ctypes as C
import os

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libgear_b200.so")

GEAR_OK, GEAR_FLUSHED = 0, 1
GEAR_ERR_ARG, GEAR_ERR_SHAPE, GEAR_ERR_ALIGN, GEAR_ERR_CAPACITY = -1, -2, -3, -4
GEAR_ERR_ALLOC, GEAR_ERR_CUDA, GEAR_ERR_TIMEOUT, GEAR_ERR_STATE = -5, -6, -7, -8
GEAR_FLAG_KEEP_FP32_FACTORS = 1

EXP = dict(K_CODES=0, V_CODES=1, K_SCALE=2, V_SCALE=3, K_ZERO=4, V_ZERO=5, K_OUT_IDX=6, V_OUT_IDX=7,
           K_OUT_VAL=8, V_OUT_VAL=9, K_A=10, V_A=11, K_B=12, V_B=13, K_A_FP32=14, V_A_FP32=15,
           K_B_FP32=16, V_B_FP32=17, K_BUFFER=18, V_BUFFER=19)


class GearConfig(C.Structure):
    _fields_ = [("batch", C.c_int32), ("n_q_heads", C.c_int32), ("n_kv_heads", C.c_int32), ("head_dim", C.c_int32),
                ("bits", C.c_int32), ("group", C.c_int32), ("outlier_pct", C.c_float), ("buffer_cap", C.c_int32),
                ("rank_flush", C.c_int32), ("rank_max", C.c_int32), ("power_iters", C.c_int32),
                ("max_tokens", C.c_int64), ("seed", C.c_uint64), ("flags", C.c_uint32), ("max_queries", C.c_uint32)]


class GearInfo(C.Structure):
    _fields_ = [("n_segments", C.c_int32), ("buffer_len", C.c_int32), ("n_compressed", C.c_int64)]


class GearSegmentInfo(C.Structure):
    _fields_ = [("n_c", C.c_int64), ("rank", C.c_int32), ("g_k", C.c_int32), ("g_v", C.c_int32),
                ("k_k", C.c_int32), ("k_v", C.c_int32)]


class GearBytes(C.Structure):
    _fields_ = [(n, C.c_int64) for n in ("codes", "scale_zero", "outliers", "lowrank_a", "lowrank_b", "buffer",
                                         "stored_total", "alloc_total")]


class GearError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {strerror(status)} ({status})")


_lib = None

# every symbol include/gear.h declares, with its C signature
_SIGNATURES = {
    "gear_create": (C.c_int32, [C.POINTER(C.c_void_p), C.POINTER(GearConfig)]),
    "gear_compress": (C.c_int32, [C.POINTER(C.c_void_p), C.POINTER(GearConfig), C.c_void_p, C.c_void_p, C.c_int64,
                                  C.c_int32, C.c_void_p, C.c_void_p]),
    "gear_append_buffer": (C.c_int32, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]),
    "gear_decode_attn": (C.c_int32, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_float, C.c_void_p]),
    "gear_decode_attn_multi": (C.c_int32, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_float, C.c_void_p]),
    "gear_free": (None, [C.c_void_p]),
    "gear_release_workspace": (C.c_int32, []),
    "gear_append_buffer_host": (C.c_int32, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]),
    "gear_decode_attn_host": (C.c_int32, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_float, C.c_void_p]),
    "gear_decode_attn_host_async": (C.c_int32, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_float, C.c_void_p]),
    "gear_cache_wait": (C.c_int32, [C.c_void_p]),
    "gear_step_host": (C.c_int32, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_float, C.c_void_p]),
    "gear_fp16_decode_attn": (C.c_int32, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_int32,
                                          C.c_int32, C.c_int32, C.c_int64, C.c_int64, C.c_float, C.c_void_p,
                                          C.c_size_t, C.c_void_p]),
    "gear_fp16_attn_scratch_bytes": (C.c_size_t, [C.c_int32, C.c_int32, C.c_int32]),
    "gear_fp16_decode_attn_static": (C.c_int32, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_int32,
                                                 C.c_int32, C.c_int32, C.c_int64, C.c_int64, C.c_float, C.c_void_p]),
    "gear_export": (C.c_int32, [C.c_void_p, C.c_int32, C.c_int32, C.c_void_p, C.c_size_t]),
    "gear_cache_info": (C.c_int32, [C.c_void_p, C.POINTER(GearInfo)]),
    "gear_segment_info_get": (C.c_int32, [C.c_void_p, C.c_int32, C.POINTER(GearSegmentInfo)]),
    "gear_cache_bytes": (C.c_int32, [C.c_void_p, C.POINTER(GearBytes)]),
    "gear_last_device_status": (C.c_int32, [C.c_void_p, C.POINTER(C.c_int32)]),
    "gear_fp16_attn_status": (C.c_int32, [C.c_void_p, C.POINTER(C.c_int32)]),
    "gear_fp16_attn_static_status": (C.c_int32, [C.POINTER(C.c_int32)]),
    "gear_test_dead_wait": (C.c_int32, [C.c_void_p, C.c_int32]),
    "gear_set_allocator": (C.c_int32, [C.c_void_p, C.c_void_p, C.c_void_p]),
    "gear_strerror": (C.c_char_p, [C.c_int32]),
    "gear_kernel_launches": (C.c_uint64, []),
}


def lib():
    """The loaded shared library (raises if it has not been built)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: run `python -m paper_2403_05527_b200.build` "
                               "(there is no CPU fallback)")
        handle = C.CDLL(LIB_PATH)
        for name, (res, args) in _SIGNATURES.items():
            fn = getattr(handle, name)
            fn.restype, fn.argtypes = res, args
        _lib = handle
    return _lib


def strerror(status: int) -> str:
    return lib().gear_strerror(status).decode()


def _ptr(t):
    """Device / host address of a torch tensor or numpy array (None -> NULL)."""
    if t is None:
        return None
    if hasattr(t, "data_ptr"):
        if not t.is_contiguous():
            raise ValueError("tensor must be contiguous")
        return C.c_void_p(t.data_ptr())
    if not t.flags["C_CONTIGUOUS"]:
        raise ValueError("array must be contiguous")
    return C.c_void_p(t.ctypes.data)


def _stream(stream):
    if stream is None:
        import torch
        return C.c_void_p(torch.cuda.current_stream().cuda_stream)
    return C.c_void_p(int(stream))


def make_config(batch, n_q_heads, n_kv_heads, bits, group, outlier_pct, buffer_cap, rank_flush, max_tokens,
                rank_max=None, power_iters=3, head_dim=128, seed=0, flags=0, max_queries=1) -> GearConfig:
    return GearConfig(batch, n_q_heads, n_kv_heads, head_dim, bits, group, float(outlier_pct), buffer_cap, rank_flush,
                      rank_flush if rank_max is None else rank_max, power_iters, int(max_tokens), seed, flags, max_queries)


def _check(status: int, where: str) -> int:
    if status < 0:
        raise GearError(status, where)
    return status


def gear_create(cfg: GearConfig) -> C.c_void_p:
    h = C.c_void_p()
    _check(lib().gear_create(C.byref(h), C.byref(cfg)), "gear_create")
    return h


def gear_compress(cache, cfg, K, V, n: int, rank: int, B0=None, stream=None) -> C.c_void_p:
    """cache may be None (created from cfg).  K, V: device fp16 [B, H, n, d_H].  Returns the cache handle."""
    h = cache if cache is not None else C.c_void_p()
    cfgp = C.byref(cfg) if cfg is not None else None
    _check(lib().gear_compress(C.byref(h), cfgp, _ptr(K), _ptr(V), n, rank, _ptr(B0), _stream(stream)), "gear_compress")
    return h


def gear_append_buffer(cache, k_new, v_new, B0_flush=None, stream=None) -> int:
    return _check(lib().gear_append_buffer(cache, _ptr(k_new), _ptr(v_new), _ptr(B0_flush), _stream(stream)),
                  "gear_append_buffer")


def gear_decode_attn(cache, q, out, softmax_scale: float = 0.0, stream=None) -> int:
    return _check(lib().gear_decode_attn(cache, _ptr(q), _ptr(out), softmax_scale, _stream(stream)), "gear_decode_attn")


def gear_decode_attn_multi(cache, q, out, n_queries: int, softmax_scale: float = 0.0, stream=None) -> int:
    """q, out: [B, H_q, n_queries, d_H]; every query row attends to the whole cache."""
    return _check(lib().gear_decode_attn_multi(cache, _ptr(q), _ptr(out), n_queries, softmax_scale, _stream(stream)),
                  "gear_decode_attn_multi")


def gear_append_buffer_host(cache, k_new_host, v_new_host, B0_flush_host=None, stream=None) -> int:
    return _check(lib().gear_append_buffer_host(cache, _ptr(k_new_host), _ptr(v_new_host), _ptr(B0_flush_host),
                                                _stream(stream)), "gear_append_buffer_host")


def gear_decode_attn_host(cache, q_host, out_host, softmax_scale: float = 0.0, stream=None) -> int:
    return _check(lib().gear_decode_attn_host(cache, _ptr(q_host), _ptr(out_host), softmax_scale, _stream(stream)),
                  "gear_decode_attn_host")


def gear_decode_attn_host_async(cache, q_host, out_host, softmax_scale: float = 0.0, stream=None) -> int:
    return _check(lib().gear_decode_attn_host_async(cache, _ptr(q_host), _ptr(out_host), softmax_scale,
                                                    _stream(stream)), "gear_decode_attn_host_async")


def gear_step_host(cache, k_new_host, v_new_host, q_host, out_host, softmax_scale: float = 0.0, stream=None) -> int:
    return _check(lib().gear_step_host(cache, _ptr(k_new_host), _ptr(v_new_host), _ptr(q_host), _ptr(out_host),
                                       softmax_scale, _stream(stream)), "gear_step_host")


def gear_cache_wait(cache) -> int:
    return _check(lib().gear_cache_wait(cache), "gear_cache_wait")


def gear_fp16_attn_scratch_bytes(batch, n_q_heads, head_dim=128) -> int:
    return lib().gear_fp16_attn_scratch_bytes(batch, n_q_heads, head_dim)


def gear_fp16_decode_attn(K, V, q, out, batch, n_q_heads, n_kv_heads, n, n_alloc, scratch, softmax_scale=0.0,
                          head_dim=128, stream=None) -> int:
    return _check(lib().gear_fp16_decode_attn(_ptr(K), _ptr(V), _ptr(q), _ptr(out), batch, n_q_heads, n_kv_heads,
                                              head_dim, n, n_alloc, softmax_scale, _ptr(scratch),
                                              scratch.numel() * scratch.element_size(), _stream(stream)),
                  "gear_fp16_decode_attn")


def gear_fp16_decode_attn_static(K, V, q, out, batch, n_q_heads, n_kv_heads, n, n_alloc, softmax_scale=0.0,
                                 head_dim=128, stream=None) -> int:
    """gear_fp16_decode_attn without a scratch argument: the library's built-in device array is used, nothing is
    allocated.  Calls that may overlap on the GPU must be ordered by the caller (they share that array)."""
    return _check(lib().gear_fp16_decode_attn_static(_ptr(K), _ptr(V), _ptr(q), _ptr(out), batch, n_q_heads, n_kv_heads,
                                                     head_dim, n, n_alloc, softmax_scale, _stream(stream)),
                  "gear_fp16_decode_attn_static")


def gear_free(cache) -> None:
    if cache is not None:
        lib().gear_free(cache)


def gear_release_workspace() -> int:
    return _check(lib().gear_release_workspace(), "gear_release_workspace")


def gear_cache_info(cache) -> GearInfo:
    info = GearInfo()
    _check(lib().gear_cache_info(cache, C.byref(info)), "gear_cache_info")
    return info


def gear_segment_info_get(cache, segment: int) -> GearSegmentInfo:
    info = GearSegmentInfo()
    _check(lib().gear_segment_info_get(cache, segment, C.byref(info)), "gear_segment_info_get")
    return info


def gear_cache_bytes(cache) -> GearBytes:
    b = GearBytes()
    _check(lib().gear_cache_bytes(cache, C.byref(b)), "gear_cache_bytes")
    return b


def gear_last_device_status(cache) -> int:
    code = C.c_int32()
    _check(lib().gear_last_device_status(cache, C.byref(code)), "gear_last_device_status")
    return code.value


def gear_fp16_attn_status(scratch) -> int:
    code = C.c_int32()
    _check(lib().gear_fp16_attn_status(_ptr(scratch), C.byref(code)), "gear_fp16_attn_status")
    return code.value


def gear_fp16_attn_static_status() -> int:
    code = C.c_int32()
    _check(lib().gear_fp16_attn_static_status(C.byref(code)), "gear_fp16_attn_static_status")
    return code.value


def gear_test_dead_wait(cache, on: bool) -> None:
    _check(lib().gear_test_dead_wait(cache, 1 if on else 0), "gear_test_dead_wait")


ALLOC_FN = C.CFUNCTYPE(C.c_void_p, C.c_size_t, C.c_void_p)
FREE_FN = C.CFUNCTYPE(None, C.c_void_p, C.c_void_p)


def gear_set_allocator(alloc_fn, free_fn) -> None:
    """Install a device allocator pair (ctypes callbacks of type ALLOC_FN / FREE_FN, kept alive by the caller), or
    None, None for cudaMalloc / cudaFree."""
    a = C.cast(alloc_fn, C.c_void_p) if alloc_fn is not None else None
    f = C.cast(free_fn, C.c_void_p) if free_fn is not None else None
    _check(lib().gear_set_allocator(a, f, None), "gear_set_allocator")


def gear_kernel_launches() -> int:
    return int(lib().gear_kernel_launches())


def gear_export(cache, segment: int, what: str, batch: int, n_kv_heads: int):
    """One piece of a segment as a numpy array in the canonical layout of include/gear.h."""
    import numpy as np
    code = EXP[what]
    if what.endswith("BUFFER"):
        n = gear_cache_info(cache).buffer_len
        arr = np.empty((batch, n_kv_heads, n, 128), np.float16)
    else:
        si = gear_segment_info_get(cache, segment)
        n_c, r = int(si.n_c), si.rank
        side_k = what.startswith("K_")
        base = what[2:]
        if base == "CODES":
            arr = np.empty((batch, n_kv_heads, n_c, 128), np.uint8)
        elif base in ("SCALE", "ZERO"):
            arr = np.empty((batch, n_kv_heads, n_c // si.g_k, 128) if side_k else (batch, n_kv_heads, n_c, 128 // si.g_v),
                           np.float16)
        elif base in ("OUT_IDX", "OUT_VAL"):
            shape = ((batch, n_kv_heads, n_c // si.g_k, 128, 2 * si.k_k) if side_k
                     else (batch, n_kv_heads, n_c, 128 // si.g_v, 2 * si.k_v))
            # a key group longer than 128 tokens (per-vector grouping): token indices come as 32-bit integers
            idx_t = np.int32 if side_k and si.g_k > 128 else np.uint8
            arr = np.empty(shape, idx_t if base == "OUT_IDX" else np.float16)
        elif base in ("A", "A_FP32"):
            arr = np.empty((batch, n_kv_heads, n_c, r), np.float32)
        elif base in ("B", "B_FP32"):
            arr = np.empty((batch, n_kv_heads, 128, r), np.float32)
        else:
            raise ValueError(what)
    _check(lib().gear_export(cache, segment, code, _ptr(arr), arr.nbytes), f"gear_export({what})")
    return arr
