"""ctypes binding of libslim.so: same names as the C ABI, argument marshalling
only.  Every step of the decode path runs inside the library's CUDA kernels;
torch is used by callers for device memory and streams.  If the shared library
is missing or cannot be loaded this module raises -- there is no fallback."""
from __future__ import annotations

import ctypes
import os
from ctypes import POINTER, byref, c_char_p, c_double, c_int, c_longlong, c_size_t, c_void_p

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libslim.so")

SLIM_OK, SLIM_ERR_INVALID_ARG, SLIM_ERR_UNSUPPORTED, SLIM_ERR_SINGULAR, SLIM_ERR_CAPACITY, \
    SLIM_ERR_OOM, SLIM_ERR_CUDA, SLIM_ERR_TIMEOUT, SLIM_ERR_NO_WEIGHTS, SLIM_ERR_STATIC_WS = range(10)
SLIM_F32, SLIM_BF16, SLIM_FP8 = 0, 1, 2
SLIM_HOST_F32, SLIM_HOST_F64 = 0, 1
SLIM_PATH_AUTO, SLIM_PATH_GENERIC, SLIM_PATH_TC = 0, 1, 2
SLIM_Q_PATH_IN_USE, SLIM_Q_LAUNCHES_PER_DECODE, SLIM_Q_MAX_UNITS, SLIM_Q_NUM_SMS, SLIM_Q_WORKERS = range(5)

# name -> (restype, argtypes); mirrors include/slim.h
SIGNATURES = {
    "slim_create": (c_int, [POINTER(c_void_p), c_int, c_int, c_int, c_double, c_int]),
    "slim_destroy": (None, [c_void_p]),
    "slim_set_weights": (c_int, [c_void_p, c_void_p, c_void_p, c_int, c_void_p, POINTER(c_double)]),
    "slim_set_weights_nonsquare": (c_int, [c_void_p, c_void_p, c_void_p, c_int, c_int, c_void_p, POINTER(c_double)]),
    "slim_set_wkv": (c_int, [c_void_p, c_void_p, c_int]),
    "slim_cache_bytes": (c_size_t, [c_void_p, c_int, c_int]),
    "slim_workspace_bytes": (c_size_t, [c_void_p, c_int, c_int]),
    "slim_cache_create": (c_int, [c_void_p, POINTER(c_void_p), c_void_p, c_int, c_int]),
    "slim_cache_create_paged": (c_int, [c_void_p, POINTER(c_void_p), c_void_p, c_int, c_int, c_void_p, c_int, c_int]),
    "slim_cache_destroy": (None, [c_void_p]),
    "slim_values_from_keys": (c_int, [c_void_p, c_void_p, c_int, c_void_p, c_void_p]),
    "slim_prefill": (c_int, [c_void_p, c_void_p, c_void_p, c_void_p, c_int, c_void_p, c_void_p]),
    "slim_append_k": (c_int, [c_void_p, c_void_p, c_void_p, c_void_p, c_int, c_void_p]),
    "slim_decode": (c_int, [c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p]),
    "slim_decode_step": (c_int, [c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p]),
    "slim_static_workspace_max": (c_size_t, []),
    "slim_decode_static_ws": (c_int, [c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p]),
    "slim_xcache_create": (c_int, [POINTER(c_void_p), c_int, c_int, c_int, c_int]),
    "slim_xcache_set_weights": (c_int, [c_void_p, c_void_p, c_void_p, c_int]),
    "slim_xcache_workspace_bytes": (c_size_t, [c_void_p, c_int, c_int]),
    "slim_xcache_decode": (c_int, [c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p]),
    "slim_reserve_positions": (c_int, [c_void_p, c_int]),
    "slim_decode_partial": (c_int, [c_void_p] * 10),
    "slim_combine_project": (c_int, [c_void_p, c_void_p, c_void_p, c_int, c_void_p, c_int, c_void_p, c_void_p, c_void_p]),
    "slim_device_status": (c_int, [c_void_p, c_void_p]),
    "slim_selftest_bounded_wait": (c_int, [c_void_p, c_void_p]),
    "slim_profile_enable": (c_int, [c_void_p, c_int]),
    "slim_profile_read": (c_int, [c_void_p, POINTER(ctypes.c_float), POINTER(ctypes.c_float)]),
    "slim_set_trace": (c_int, [c_void_p, c_void_p]),
    "slim_set_path": (c_int, [c_void_p, c_int]),
    "slim_query": (c_longlong, [c_void_p, c_int]),
    "slim_strerror": (c_char_p, [c_int]),
}

_lib = None


class SlimError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {strerror(status)} (status {status})")


def lib() -> ctypes.CDLL:
    """Load libslim.so (once).  Raises if it has not been built.  SLIM_LIBRARY names another build of the
    library (the instrumented one of trace.py)."""
    global _lib
    if _lib is None:
        path = os.environ.get("SLIM_LIBRARY", LIB_PATH)
        if not os.path.exists(path):
            raise RuntimeError(f"{path} is missing: run `python -m paper_2503_05840_b200.build` "
                               "(there is no CPU fallback)")
        L = ctypes.CDLL(path)
        for name, (res, args) in SIGNATURES.items():
            fn = getattr(L, name)
            fn.restype = res
            fn.argtypes = args
        _lib = L
    return _lib


def strerror(status: int) -> str:
    return lib().slim_strerror(int(status)).decode()


def _check(status: int, where: str) -> None:
    if status != SLIM_OK:
        raise SlimError(status, where)


def _ptr(x) -> c_void_p:
    """Raw address of a torch tensor / numpy array / int / None."""
    if x is None:
        return c_void_p(0)
    if isinstance(x, int):
        return c_void_p(x)
    if isinstance(x, np.ndarray):
        return c_void_p(x.ctypes.data)
    return c_void_p(x.data_ptr())        # torch.Tensor


def _host_mat(a):
    a = np.ascontiguousarray(a)
    if a.dtype == np.float64:
        return a, SLIM_HOST_F64
    if a.dtype == np.float32:
        return a, SLIM_HOST_F32
    return np.ascontiguousarray(a, dtype=np.float64), SLIM_HOST_F64


# ---- thin wrappers, same names as the C ABI ---------------------------------
def slim_create(d: int, H: int, d_k: int, rope_theta: float, dtype: int) -> int:
    h = c_void_p()
    _check(lib().slim_create(byref(h), d, H, d_k, float(rope_theta), dtype), "slim_create")
    return h.value


def slim_destroy(ctx: int) -> None:
    lib().slim_destroy(c_void_p(ctx))


def slim_set_weights(ctx: int, W_K, W_V, want_wkv: bool = False):
    """Returns (residual, W_KV float64 or None)."""
    a, dt = _host_mat(W_K)
    b, dt2 = _host_mat(W_V)
    if dt != dt2:
        a = np.ascontiguousarray(a, dtype=np.float64); b = np.ascontiguousarray(b, dtype=np.float64)
        dt = SLIM_HOST_F64
    out = np.empty(a.shape, dtype=np.float64) if want_wkv else None
    res = c_double(0.0)
    _check(lib().slim_set_weights(c_void_p(ctx), _ptr(a), _ptr(b), dt, _ptr(out), byref(res)), "slim_set_weights")
    return res.value, out


def slim_set_weights_nonsquare(ctx: int, W_K, W_V, want_wkv: bool = False):
    """W_K, W_V: [d_model, e] with e = H d_k > d_model.  Returns (residual, W_KV [e, e] float64 or None)."""
    a = np.ascontiguousarray(W_K, dtype=np.float64)
    b = np.ascontiguousarray(W_V, dtype=np.float64)
    assert a.shape == b.shape and a.ndim == 2
    d_model, e = a.shape
    out = np.empty((e, e), dtype=np.float64) if want_wkv else None
    res = c_double(0.0)
    _check(lib().slim_set_weights_nonsquare(c_void_p(ctx), _ptr(a), _ptr(b), d_model, SLIM_HOST_F64, _ptr(out), byref(res)),
           "slim_set_weights_nonsquare")
    return res.value, out


def slim_set_wkv(ctx: int, W_KV) -> None:
    a, dt = _host_mat(W_KV)
    _check(lib().slim_set_wkv(c_void_p(ctx), _ptr(a), dt), "slim_set_wkv")


def slim_cache_bytes(ctx: int, batch: int, t_cap: int) -> int:
    return lib().slim_cache_bytes(c_void_p(ctx), batch, t_cap)


def slim_workspace_bytes(ctx: int, batch: int, t_cap: int) -> int:
    return lib().slim_workspace_bytes(c_void_p(ctx), batch, t_cap)


def slim_cache_create(ctx: int, k_storage, batch: int, t_cap: int) -> int:
    h = c_void_p()
    _check(lib().slim_cache_create(c_void_p(ctx), byref(h), _ptr(k_storage), batch, t_cap), "slim_cache_create")
    return h.value


def slim_cache_create_paged(ctx: int, pool, num_pages: int, page_rows: int, block_table, batch: int, max_pages: int) -> int:
    h = c_void_p()
    _check(lib().slim_cache_create_paged(c_void_p(ctx), byref(h), _ptr(pool), num_pages, page_rows, _ptr(block_table), batch,
                                         max_pages), "slim_cache_create_paged")
    return h.value


def slim_cache_destroy(cache: int) -> None:
    lib().slim_cache_destroy(c_void_p(cache))


def slim_values_from_keys(ctx: int, K, n: int, V, stream: int = 0) -> None:
    _check(lib().slim_values_from_keys(c_void_p(ctx), _ptr(K), n, _ptr(V), c_void_p(stream)), "slim_values_from_keys")


def slim_prefill(ctx: int, cache: int, k_new, positions, n_new: int, V, stream: int = 0) -> None:
    """Prompt phase: store the prompt's keys and return V = K W_KV in one call."""
    _check(lib().slim_prefill(c_void_p(ctx), c_void_p(cache), _ptr(k_new), _ptr(positions), n_new, _ptr(V),
                              c_void_p(stream)), "slim_prefill")


def slim_append_k(ctx: int, cache: int, k_new, positions, n_new: int, stream: int = 0) -> None:
    _check(lib().slim_append_k(c_void_p(ctx), c_void_p(cache), _ptr(k_new), _ptr(positions), n_new,
                               c_void_p(stream)), "slim_append_k")


def slim_decode(ctx: int, q, cache: int, lengths, o, workspace, stream: int = 0) -> None:
    _check(lib().slim_decode(c_void_p(ctx), _ptr(q), c_void_p(cache), _ptr(lengths), _ptr(o), _ptr(workspace),
                             c_void_p(stream)), "slim_decode")


def slim_decode_step(ctx: int, q, k_new, cache: int, lengths, o, workspace, stream: int = 0) -> None:
    """Cache update (k_new at row lengths[b]-1) and decode in one call."""
    _check(lib().slim_decode_step(c_void_p(ctx), _ptr(q), _ptr(k_new), c_void_p(cache), _ptr(lengths), _ptr(o),
                                  _ptr(workspace), c_void_p(stream)), "slim_decode_step")


def slim_static_workspace_max() -> int:
    return lib().slim_static_workspace_max()


def slim_decode_static_ws(ctx: int, q, cache: int, lengths, o, stream: int = 0) -> None:
    """slim_decode with the library's built-in scratch: for callers that must not allocate."""
    _check(lib().slim_decode_static_ws(c_void_p(ctx), _ptr(q), c_void_p(cache), _ptr(lengths), _ptr(o),
                                       c_void_p(stream)), "slim_decode_static_ws")


def slim_xcache_create(d_model: int, H: int, d_k: int, dtype: int) -> int:
    """X-cache context whose cache rows are d_model wide while queries and outputs are H*d_k wide."""
    h = c_void_p()
    _check(lib().slim_xcache_create(byref(h), d_model, H, d_k, dtype), "slim_xcache_create")
    return h.value


def slim_xcache_set_weights(ctx: int, W_K, W_V) -> None:
    a = np.ascontiguousarray(W_K, dtype=np.float64)
    b = np.ascontiguousarray(W_V, dtype=np.float64)
    _check(lib().slim_xcache_set_weights(c_void_p(ctx), _ptr(a), _ptr(b), SLIM_HOST_F64), "slim_xcache_set_weights")


def slim_xcache_workspace_bytes(ctx: int, batch: int, t_cap: int) -> int:
    return lib().slim_xcache_workspace_bytes(c_void_p(ctx), batch, t_cap)


def slim_xcache_decode(ctx: int, q, cache: int, lengths, o, workspace, stream: int = 0) -> None:
    _check(lib().slim_xcache_decode(c_void_p(ctx), _ptr(q), c_void_p(cache), _ptr(lengths), _ptr(o), _ptr(workspace),
                                    c_void_p(stream)), "slim_xcache_decode")


def slim_reserve_positions(ctx: int, max_position: int) -> None:
    _check(lib().slim_reserve_positions(c_void_p(ctx), int(max_position)), "slim_reserve_positions")


def slim_decode_partial(ctx: int, q, cache: int, lengths, first_tile, q_pos, lse_out, u_out, workspace, stream: int = 0) -> None:
    _check(lib().slim_decode_partial(c_void_p(ctx), _ptr(q), c_void_p(cache), _ptr(lengths), _ptr(first_tile), _ptr(q_pos),
                                     _ptr(lse_out), _ptr(u_out), _ptr(workspace), c_void_p(stream)), "slim_decode_partial")


def slim_combine_project(ctx: int, lse_all, u_all, ranks: int, total_lengths, batch: int, o, workspace, stream: int = 0) -> None:
    _check(lib().slim_combine_project(c_void_p(ctx), _ptr(lse_all), _ptr(u_all), ranks, _ptr(total_lengths), batch, _ptr(o),
                                      _ptr(workspace), c_void_p(stream)), "slim_combine_project")


def slim_device_status(ctx: int, stream: int = 0) -> int:
    return lib().slim_device_status(c_void_p(ctx), c_void_p(stream))


def slim_selftest_bounded_wait(ctx: int, stream: int = 0) -> None:
    _check(lib().slim_selftest_bounded_wait(c_void_p(ctx), c_void_p(stream)), "slim_selftest_bounded_wait")


def slim_profile_enable(ctx: int, enable: bool) -> None:
    _check(lib().slim_profile_enable(c_void_p(ctx), 1 if enable else 0), "slim_profile_enable")


def slim_profile_read(ctx: int):
    """(main_ms, tail_ms) of the last slim_decode of this ctx."""
    a, b = ctypes.c_float(0), ctypes.c_float(0)
    _check(lib().slim_profile_read(c_void_p(ctx), byref(a), byref(b)), "slim_profile_read")
    return a.value, b.value


def slim_set_trace(ctx: int, device_buffer) -> None:
    _check(lib().slim_set_trace(c_void_p(ctx), _ptr(device_buffer)), "slim_set_trace")


def slim_set_path(ctx: int, path: int) -> None:
    _check(lib().slim_set_path(c_void_p(ctx), path), "slim_set_path")


def slim_query(ctx: int, key: int) -> int:
    return lib().slim_query(c_void_p(ctx), key)


def slim_strerror(status: int) -> str:
    return strerror(status)
