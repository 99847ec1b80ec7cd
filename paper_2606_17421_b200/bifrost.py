"""ctypes binding of libbifrost's C ABI (include/bifrost.h): argument marshalling only.

Every function has the name and the argument order of its C counterpart.  Device buffers are
passed as torch CUDA tensors (or raw integer addresses); PyTorch is used for nothing but device
memory and streams.  There is no fallback: if the CUDA library has not been built, load() raises.
"""
from __future__ import annotations

import ctypes
import os

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(HERE, "libbifrost.so")

BF_OK = 0
BF_ERR_INVALID_ARG = -1
BF_ERR_BAD_PRIME = -2
BF_ERR_SHAPE = -3
BF_ERR_LEVEL = -4
BF_ERR_MISSING_KEY = -5
BF_ERR_OOM = -6
BF_ERR_CUDA = -7
BF_ERR_RANGE = -8
BF_ERR_TOO_LARGE = -9
BF_ERR_TIMEOUT = -10


BF_PLAN_COMPLEX_PACK = 1
BF_PLAN_MODDOWN_PER_OUTPUT = 2
BF_PLAN_DOUBLE_HOIST = 4


class bf_plan(ctypes.Structure):
    """bf_plan(tile_D, tau, bsgs_b, bsgs_g[, flags]); flags = BF_PLAN_* bits, 0 by default."""
    _fields_ = [("tile_D", ctypes.c_uint32), ("tau", ctypes.c_uint32),
                ("bsgs_b", ctypes.c_uint32), ("bsgs_g", ctypes.c_uint32), ("flags", ctypes.c_uint32)]


class BifrostError(RuntimeError):
    def __init__(self, code: int, where: str, detail: str = ""):
        self.code = code
        super().__init__(f"{where}: {bf_strerror(code)} ({code}) {detail}".strip())


_vp = ctypes.c_void_p
_u32 = ctypes.c_uint32
_u64 = ctypes.c_uint64
_lib = None

_SIGNATURES = {
    "bf_ctx_create": (ctypes.c_int, [ctypes.POINTER(_vp), _u32, ctypes.POINTER(_u64), _u32, ctypes.c_double,
                                     ctypes.POINTER(bf_plan), _vp]),
    "bf_ctx_destroy": (None, [_vp]),
    "bf_load_eval_keys": (ctypes.c_int, [_vp, ctypes.POINTER(_u32), _u32, _vp]),
    "bf_set_cache_budget": (ctypes.c_int, [_vp, _u64]),
    "bf_cache_bytes_used": (_u64, [_vp]),
    "bf_weights_bytes": (_u64, [_vp, _u32, _u32]),
    "bf_encode_weights": (ctypes.c_int, [_vp, _vp, _u32, _u32, ctypes.POINTER(_vp)]),
    "bf_encode_weights_split": (ctypes.c_int, [_vp, _vp, _u32, _u32, _u32, _u32, ctypes.POINTER(_vp)]),
    "bf_weights_free": (None, [_vp, _vp]),
    "bf_linear": (ctypes.c_int, [_vp, _vp, _u32, _vp, _vp, _u32, _u32, _vp, _u32]),
    "bf_linear_rescaled": (ctypes.c_int, [_vp, _vp, _u32, _vp, _vp, _u32, _u32, _vp, _u32, ctypes.POINTER(ctypes.c_double)]),
    "bf_device_status": (ctypes.c_int, [_vp]),
    "bf_set_graph_replay": (ctypes.c_int, [_vp, ctypes.c_int]),
    "bf_set_dependent_launch": (ctypes.c_int, [_vp, ctypes.c_int]),
    "bf_set_lanes": (ctypes.c_int, [_vp, ctypes.c_int]),
    "bf_set_compact_cache": (ctypes.c_int, [_vp, ctypes.c_int]),
    "bf_set_coefficient_cache": (ctypes.c_int, [_vp, ctypes.c_int]),
    "bf_set_encode_scratch": (ctypes.c_int, [_vp, _u64]),
    "bf_rescale": (ctypes.c_int, [_vp, _vp, _vp, _u32, _u32, ctypes.POINTER(ctypes.c_double)]),
    "bf_fold": (ctypes.c_int, [_vp, _vp, _u32]),
    "bf_linear_host": (ctypes.c_int, [_vp, _vp, _u32, _vp, _vp, _u32, _u32, _vp, _u32]),
    "bf_rotate": (ctypes.c_int, [_vp, _vp, _u32, _vp]),
    "bf_negacyclic_mul": (ctypes.c_int, [_vp, _vp, _vp, _vp, _u32]),
    "bf_negacyclic_mul_noalloc": (ctypes.c_int, [_vp, _vp, _vp, _vp, _u32]),
    "bf_noalloc_max_words": (_u64, []),
    "bf_weights_export": (ctypes.c_int, [_vp, _vp, _u32, _u32, _u32, _u32, _vp]),
    "bf_set_stage_timing": (ctypes.c_int, [_vp, ctypes.c_int]),
    "bf_get_stage_ms": (ctypes.c_int, [_vp, ctypes.POINTER(ctypes.c_float)]),
    "bf_set_kernel_timing": (ctypes.c_int, [_vp, ctypes.c_int]),
    "bf_kernel_categories": (ctypes.c_int, []),
    "bf_kernel_category_name": (ctypes.c_char_p, [ctypes.c_int]),
    "bf_get_kernel_stats": (ctypes.c_int, [_vp, ctypes.POINTER(_u64), ctypes.POINTER(ctypes.c_float)]),
    "bf_measure_imad_rate": (ctypes.c_int, [_vp, ctypes.POINTER(ctypes.c_double)]),
    "bf_measure_fma64_rate": (ctypes.c_int, [_vp, ctypes.POINTER(ctypes.c_double)]),
    "bf_get_key_stream_bytes": (ctypes.c_int, [_vp, ctypes.POINTER(_u64), ctypes.POINTER(_u64)]),
    "bf_strerror": (ctypes.c_char_p, [ctypes.c_int]),
    "bf_last_cuda_error": (ctypes.c_char_p, [_vp]),
}


def exported_symbols() -> list[str]:
    return sorted(_SIGNATURES)


def load():
    """Load libbifrost.so.  Raises if it is missing: there is no other implementation to fall back to."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} not found: build it with `python -m paper_2606_17421_b200.build` "
                               "(there is no CPU fallback)")
        lib = ctypes.CDLL(LIB_PATH)
        for name, (res, args) in _SIGNATURES.items():
            fn = getattr(lib, name)
            fn.restype = res
            fn.argtypes = args
        _lib = lib
    return _lib


def _ptr(x):
    """Device or host address of a torch tensor / numpy array / int / None."""
    if x is None:
        return None
    if isinstance(x, int):
        return x
    if hasattr(x, "data_ptr"):
        return x.data_ptr()
    if hasattr(x, "ctypes"):
        return x.ctypes.data
    raise TypeError(type(x))


def _check(code: int, where: str, ctx=None):
    if code != BF_OK:
        detail = ""
        if code == BF_ERR_CUDA and ctx:
            detail = (load().bf_last_cuda_error(ctx) or b"").decode()
        raise BifrostError(code, where, detail)


def bf_strerror(code: int) -> str:
    return load().bf_strerror(code).decode()


def bf_ctx_create(N: int, primes, n_ct_primes: int, scale: float, plan: bf_plan, cuda_stream: int = 0):
    arr = (_u64 * len(primes))(*primes)
    out = _vp()
    _check(load().bf_ctx_create(ctypes.byref(out), N, arr, n_ct_primes, scale, ctypes.byref(plan), cuda_stream),
           "bf_ctx_create")
    return out


def bf_ctx_destroy(ctx):
    load().bf_ctx_destroy(ctx)


def bf_load_eval_keys(ctx, rot_steps, n_keys: int, keys):
    arr = (_u32 * max(1, len(rot_steps)))(*rot_steps)
    _check(load().bf_load_eval_keys(ctx, arr, n_keys, _ptr(keys)), "bf_load_eval_keys", ctx)


def bf_set_cache_budget(ctx, nbytes: int):
    _check(load().bf_set_cache_budget(ctx, nbytes), "bf_set_cache_budget", ctx)


def bf_cache_bytes_used(ctx) -> int:
    return load().bf_cache_bytes_used(ctx)


def bf_weights_bytes(ctx, d_out: int, d_in: int) -> int:
    return load().bf_weights_bytes(ctx, d_out, d_in)


def bf_encode_weights(ctx, W, d_out: int, d_in: int):
    out = _vp()
    _check(load().bf_encode_weights(ctx, _ptr(W), d_out, d_in, ctypes.byref(out)), "bf_encode_weights", ctx)
    return out


def bf_encode_weights_split(ctx, W, d_out: int, d_in: int, bsgs_b: int, bsgs_g: int):
    out = _vp()
    _check(load().bf_encode_weights_split(ctx, _ptr(W), d_out, d_in, bsgs_b, bsgs_g, ctypes.byref(out)),
           "bf_encode_weights_split", ctx)
    return out


def bf_weights_free(ctx, w):
    load().bf_weights_free(ctx, w)


def bf_linear(ctx, ct_in, n_in: int, pt_weights, W_raw, d_out: int, d_in: int, ct_out, n_out: int):
    _check(load().bf_linear(ctx, _ptr(ct_in), n_in, pt_weights, _ptr(W_raw), d_out, d_in, _ptr(ct_out), n_out),
           "bf_linear", ctx)


def bf_device_status(ctx):
    """Synchronises; raises if a device-side wait gave up or the on-the-fly encoder overflowed."""
    _check(load().bf_device_status(ctx), "bf_device_status", ctx)


def bf_set_graph_replay(ctx, on: bool):
    _check(load().bf_set_graph_replay(ctx, 1 if on else 0), "bf_set_graph_replay", ctx)


def bf_set_compact_cache(ctx, on: bool):
    _check(load().bf_set_compact_cache(ctx, 1 if on else 0), "bf_set_compact_cache", ctx)


def bf_set_coefficient_cache(ctx, bits: int):
    _check(load().bf_set_coefficient_cache(ctx, bits), "bf_set_coefficient_cache", ctx)


def bf_set_encode_scratch(ctx, n_bytes: int):
    _check(load().bf_set_encode_scratch(ctx, n_bytes), "bf_set_encode_scratch", ctx)


def bf_set_lanes(ctx, n_lanes: int):
    _check(load().bf_set_lanes(ctx, n_lanes), "bf_set_lanes", ctx)


def bf_set_dependent_launch(ctx, on: bool):
    _check(load().bf_set_dependent_launch(ctx, 1 if on else 0), "bf_set_dependent_launch", ctx)


def bf_rescale(ctx, ct_in, ct_out, n_ct: int, level: int, scale: float | None = None):
    """Returns the new scale when `scale` is given."""
    s = ctypes.c_double(scale if scale is not None else 0.0)
    _check(load().bf_rescale(ctx, _ptr(ct_in), _ptr(ct_out), n_ct, level,
                             ctypes.byref(s) if scale is not None else None), "bf_rescale", ctx)
    return s.value if scale is not None else None


def bf_linear_rescaled(ctx, ct_in, n_in: int, pt_weights, W_raw, d_out: int, d_in: int, ct_low, n_out: int,
                       scale: float | None = None):
    """Returns the new scale when `scale` is given."""
    s = ctypes.c_double(scale if scale is not None else 0.0)
    _check(load().bf_linear_rescaled(ctx, _ptr(ct_in), n_in, pt_weights, _ptr(W_raw), d_out, d_in, _ptr(ct_low), n_out,
                                     ctypes.byref(s) if scale is not None else None), "bf_linear_rescaled", ctx)
    return s.value if scale is not None else None


def bf_linear_host(ctx, host_ct_in, n_in: int, pt_weights, W_raw, d_out: int, d_in: int, host_ct_out, n_out: int):
    _check(load().bf_linear_host(ctx, _ptr(host_ct_in), n_in, pt_weights, _ptr(W_raw), d_out, d_in,
                                 _ptr(host_ct_out), n_out), "bf_linear_host", ctx)


def bf_rotate(ctx, ct_in, steps: int, ct_out):
    _check(load().bf_rotate(ctx, _ptr(ct_in), steps, _ptr(ct_out)), "bf_rotate", ctx)


def bf_fold(ctx, ct, n_ct: int):
    """Sums the tau partial results inside n_ct full-level ciphertexts, in place."""
    _check(load().bf_fold(ctx, _ptr(ct), n_ct), "bf_fold", ctx)


def bf_negacyclic_mul(ctx, a, b, out, n_polys: int):
    _check(load().bf_negacyclic_mul(ctx, _ptr(a), _ptr(b), _ptr(out), n_polys), "bf_negacyclic_mul", ctx)


def bf_negacyclic_mul_noalloc(ctx, a, b, out, n_polys: int):
    """bf_negacyclic_mul without any device allocation: scratch is a fixed array in the library image."""
    _check(load().bf_negacyclic_mul_noalloc(ctx, _ptr(a), _ptr(b), _ptr(out), n_polys), "bf_negacyclic_mul_noalloc", ctx)


def bf_noalloc_max_words() -> int:
    return load().bf_noalloc_max_words()


def bf_weights_export(ctx, w, p: int, q: int, j: int, k: int, out):
    _check(load().bf_weights_export(ctx, w, p, q, j, k, _ptr(out)), "bf_weights_export", ctx)


def bf_set_stage_timing(ctx, on: bool):
    _check(load().bf_set_stage_timing(ctx, 1 if on else 0), "bf_set_stage_timing", ctx)


def bf_get_stage_ms(ctx) -> list[float]:
    arr = (ctypes.c_float * 4)()
    _check(load().bf_get_stage_ms(ctx, arr), "bf_get_stage_ms", ctx)
    return list(arr)


def bf_set_kernel_timing(ctx, on: bool):
    _check(load().bf_set_kernel_timing(ctx, 1 if on else 0), "bf_set_kernel_timing", ctx)


def bf_kernel_categories() -> int:
    return load().bf_kernel_categories()


def bf_kernel_category_name(cat: int) -> str:
    return load().bf_kernel_category_name(cat).decode()


def bf_get_kernel_stats(ctx) -> dict:
    """{category name: (launches, summed event ms)} since the previous call."""
    n = bf_kernel_categories()
    launches = (_u64 * n)()
    ms = (ctypes.c_float * n)()
    _check(load().bf_get_kernel_stats(ctx, launches, ms), "bf_get_kernel_stats", ctx)
    return {bf_kernel_category_name(c): (int(launches[c]), float(ms[c])) for c in range(n)}


def bf_measure_imad_rate(ctx) -> float:
    out = ctypes.c_double(0.0)
    _check(load().bf_measure_imad_rate(ctx, ctypes.byref(out)), "bf_measure_imad_rate", ctx)
    return out.value


def bf_measure_fma64_rate(ctx) -> float:
    out = ctypes.c_double(0.0)
    _check(load().bf_measure_fma64_rate(ctx, ctypes.byref(out)), "bf_measure_fma64_rate", ctx)
    return out.value


def bf_get_key_stream_bytes(ctx) -> tuple[int, int]:
    """(bytes counted once per distinct key of each launch, bytes counted once per rotation) since the previous call."""
    a, b = _u64(0), _u64(0)
    _check(load().bf_get_key_stream_bytes(ctx, ctypes.byref(a), ctypes.byref(b)), "bf_get_key_stream_bytes", ctx)
    return int(a.value), int(b.value)
