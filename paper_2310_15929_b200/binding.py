"""ctypes binding of libesparse.so: same names as include/esparse.h, argument marshalling only.

PyTorch supplies device memory and streams; every step of the path runs in the library's kernels.
There is no fallback: if the shared library is missing the import of this module fails.
"""
from __future__ import annotations

import ctypes
import os
from ctypes import POINTER, c_char_p, c_double, c_int, c_long, c_longlong, c_size_t, c_void_p

from .build import LIB_PATH

ESP_OK = 0
ESP_ERR_INVALID_ARG, ESP_ERR_SHAPE, ESP_ERR_ALIGNMENT, ESP_ERR_WORKSPACE = 1, 2, 3, 4
ESP_ERR_UNSUPPORTED, ESP_ERR_CUDA, ESP_ERR_TIMEOUT = 5, 6, 7
ESP_ERR_STATIC_LIMIT = 8
ESP_STATIC_SCRATCH_BYTES = 8 << 20
ESP_X_TOKEN_MAJOR, ESP_X_CHANNEL_MAJOR = 0, 1
ESP_OUT_F16, ESP_OUT_F32 = 0, 1
ESP_ACT_NONE, ESP_ACT_RELU = 0, 1
ESP_KERNEL_AUTO, ESP_KERNEL_GATHER, ESP_KERNEL_TMA, ESP_KERNEL_STREAM, ESP_KERNEL_PAIR, ESP_KERNEL_PAIR_TILED = 0, 1, 2, 4, 5, 6
ESP_KERNEL_QUAD_TILED, ESP_KERNEL_PAIR_PERSIST, ESP_KERNEL_QUAD_MULTICAST, ESP_KERNEL_STREAM_IMAGES = 7, 8, 9, 10


class esp_prune_opts(ctypes.Structure):
    _fields_ = [("struct_size", c_size_t), ("alpha", c_double), ("bins", c_int), ("n_keep", c_int),
                ("m_group", c_int), ("lbs_block", c_int), ("lbs_max_swaps", c_int), ("use_entropy", c_int),
                ("use_norm", c_int), ("use_gns", c_int), ("use_lbs", c_int), ("score_override", c_void_p),
                ("global_bin_range", c_int), ("perm_override", c_void_p)]


class esp_prune_stats(ctypes.Structure):
    _fields_ = [("struct_size", c_size_t), ("near_tie_groups", c_longlong), ("near_tie_sort", c_longlong),
                ("near_tie_swaps", c_longlong), ("lbs_swaps_total", c_longlong), ("obj_identity", c_double),
                ("obj_after_gns", c_double), ("obj_after_lbs", c_double)]


class esp_gemm_opts(ctypes.Structure):
    _fields_ = [("struct_size", c_size_t), ("x_layout", c_int), ("out_dtype", c_int), ("split_k", c_int),
                ("force_kernel", c_int), ("token_tile", c_int), ("static_weights", c_int), ("pipeline_stages", c_int), ("activation", c_int),
                ("bias", c_void_p)]


class EsparseError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = int(status)
        super().__init__(f"{where}: {esp_status_string(status)} (status {int(status)})")


if not os.path.exists(LIB_PATH):
    raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2310_15929_b200.build` "
                      "(there is no CPU or PyTorch fallback)")
_lib = ctypes.CDLL(LIB_PATH)

EXPORTS = ("esp_status_string", "esp_version", "esp_prune_opts_default", "esp_gemm_opts_default",
           "esp_metric_prune_workspace_bytes", "esp_packed_bytes", "esp_metric_prune", "esp_pack",
           "esp_decompress", "esp_spgemm_workspace_bytes", "esp_spgemm", "esp_last_device_status",
           "esp_spgemm_static", "esp_spgemm_plan", "esp_selftest_wait_timeout", "esp_calib_state_bytes", "esp_calib_reset",
           "esp_calib_range", "esp_calib_histogram", "esp_calib_finish", "esp_spgemm_tune", "esp_spgemm_grouped",
           "esp_multicast_available")

_lib.esp_status_string.restype = c_char_p
_lib.esp_status_string.argtypes = [c_int]
_lib.esp_version.restype = c_int
_lib.esp_prune_opts_default.argtypes = [POINTER(esp_prune_opts)]
_lib.esp_gemm_opts_default.argtypes = [POINTER(esp_gemm_opts)]
_lib.esp_metric_prune_workspace_bytes.restype = c_size_t
_lib.esp_metric_prune_workspace_bytes.argtypes = [c_int, c_int, c_int, POINTER(esp_prune_opts)]
_lib.esp_packed_bytes.restype = c_size_t
_lib.esp_packed_bytes.argtypes = [c_int, c_int]
_lib.esp_metric_prune.restype = c_int
_lib.esp_metric_prune.argtypes = [c_void_p, c_int, c_int, c_long, c_void_p, c_int, c_long, POINTER(esp_prune_opts),
                                  c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p,
                                  POINTER(esp_prune_stats), c_void_p, c_size_t, c_void_p]
_lib.esp_pack.restype = c_int
_lib.esp_pack.argtypes = [c_void_p, c_void_p, c_int, c_int, c_void_p, c_void_p]
_lib.esp_decompress.restype = c_int
_lib.esp_decompress.argtypes = [c_void_p, c_void_p, c_void_p, c_int, c_int, c_void_p, c_long, c_void_p]
_lib.esp_spgemm_workspace_bytes.restype = c_size_t
_lib.esp_spgemm_workspace_bytes.argtypes = [c_int, c_int, c_int, POINTER(esp_gemm_opts)]
_lib.esp_spgemm.restype = c_int
_lib.esp_spgemm.argtypes = [c_void_p, c_int, c_int, c_long, c_void_p, c_void_p, c_int, c_void_p, c_long,
                            POINTER(esp_gemm_opts), c_void_p, c_size_t, c_void_p]
_lib.esp_last_device_status.restype = c_int
_lib.esp_multicast_available.restype = c_int
_lib.esp_selftest_wait_timeout.restype = c_int
_lib.esp_selftest_wait_timeout.argtypes = [c_void_p]
_lib.esp_spgemm_plan.restype = c_int
_lib.esp_spgemm_plan.argtypes = [c_int, c_int, c_int, POINTER(esp_gemm_opts), c_int, POINTER(c_int), POINTER(c_int),
                                 POINTER(c_int), POINTER(c_int)]
_lib.esp_spgemm_static.restype = c_int
_lib.esp_spgemm_static.argtypes = [c_void_p, c_int, c_int, c_long, c_void_p, c_void_p, c_int, c_void_p, c_long,
                                   c_int, c_void_p]


def _ptr(t):
    """Device (or host) address of a torch tensor / raw int / None."""
    if t is None:
        return None
    if isinstance(t, int):
        return t
    return t.data_ptr()


def _stream(stream):
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)


def esp_status_string(status: int) -> str:
    return _lib.esp_status_string(int(status)).decode()


def esp_version() -> int:
    return int(_lib.esp_version())


def esp_prune_opts_default() -> esp_prune_opts:
    o = esp_prune_opts()
    _lib.esp_prune_opts_default(ctypes.byref(o))
    return o


def esp_gemm_opts_default() -> esp_gemm_opts:
    o = esp_gemm_opts()
    _lib.esp_gemm_opts_default(ctypes.byref(o))
    return o


def esp_metric_prune_workspace_bytes(No: int, C: int, T: int, opts: esp_prune_opts) -> int:
    return int(_lib.esp_metric_prune_workspace_bytes(No, C, T, ctypes.byref(opts)))


def esp_packed_bytes(No: int, C: int) -> int:
    return int(_lib.esp_packed_bytes(No, C))


def esp_metric_prune_raw(W, No, C, ldw, Xcal, T, ldx, opts, vals, meta, perm, packed, chan_norm, chan_entropy,
                         chan_score, stats, workspace, workspace_bytes, stream) -> int:
    """The C call with raw addresses; returns the status code without raising (used by error-path tests)."""
    return int(_lib.esp_metric_prune(_ptr(W), No, C, ldw, _ptr(Xcal), T, ldx,
                                     ctypes.byref(opts) if opts is not None else None,
                                     _ptr(vals), _ptr(meta), _ptr(perm), _ptr(packed), _ptr(chan_norm),
                                     _ptr(chan_entropy), _ptr(chan_score),
                                     ctypes.byref(stats) if stats is not None else None,
                                     _ptr(workspace), workspace_bytes, stream))


def esp_metric_prune(W, Xcal, opts, vals, meta, perm, packed=None, chan_norm=None, chan_entropy=None,
                     chan_score=None, stats=None, workspace=None, stream=None):
    """W [No,C] f16, Xcal [T,C] f16 (or None with opts.score_override) -> vals, meta, perm (, packed)."""
    No, C = W.shape
    T = 0 if Xcal is None else Xcal.shape[0]
    ldx = C if Xcal is None else Xcal.stride(0)
    if stats is not None:
        stats.struct_size = ctypes.sizeof(esp_prune_stats)
    st = esp_metric_prune_raw(W, No, C, W.stride(0), Xcal, T, ldx, opts, vals, meta, perm, packed, chan_norm,
                              chan_entropy, chan_score, stats, workspace,
                              0 if workspace is None else workspace.numel() * workspace.element_size(),
                              _stream(stream))
    if st != ESP_OK:
        raise EsparseError(st, "esp_metric_prune")


def esp_pack(vals, meta, No, C, packed, stream=None):
    st = int(_lib.esp_pack(_ptr(vals), _ptr(meta), No, C, _ptr(packed), _stream(stream)))
    if st != ESP_OK:
        raise EsparseError(st, "esp_pack")


def esp_decompress(vals, meta, perm, No, C, W_out, stream=None):
    st = int(_lib.esp_decompress(_ptr(vals), _ptr(meta), _ptr(perm), No, C, _ptr(W_out), W_out.stride(0),
                                 _stream(stream)))
    if st != ESP_OK:
        raise EsparseError(st, "esp_decompress")


def esp_spgemm_workspace_bytes(M: int, N: int, K: int, opts: esp_gemm_opts) -> int:
    return int(_lib.esp_spgemm_workspace_bytes(M, N, K, ctypes.byref(opts)))


def esp_spgemm_plan(M: int, N: int, K: int, opts: esp_gemm_opts, have_workspace: bool = True) -> dict:
    """The launch configuration esp_spgemm would use (needs the device; launches nothing)."""
    k, t, s, g = c_int(), c_int(), c_int(), c_int()
    st = int(_lib.esp_spgemm_plan(M, N, K, ctypes.byref(opts), 1 if have_workspace else 0, ctypes.byref(k),
                                  ctypes.byref(t), ctypes.byref(s), ctypes.byref(g)))
    if st != ESP_OK:
        raise EsparseError(st, "esp_spgemm_plan")
    return {"kernel": k.value, "token_tile": t.value, "split_k": s.value, "stages": g.value}


def esp_spgemm_raw(X, M, K, ldx, packed, perm, N, Y, ldy, opts, workspace, workspace_bytes, stream) -> int:
    return int(_lib.esp_spgemm(_ptr(X), M, K, ldx, _ptr(packed), _ptr(perm), N, _ptr(Y), ldy,
                               ctypes.byref(opts) if opts is not None else None, _ptr(workspace), workspace_bytes,
                               stream))


def esp_spgemm(X, packed, perm, Y, opts, workspace=None, stream=None):
    """Y [M,N] = X . P . W_s^T.  X is [M,K] (token-major) or [K,M] (channel-major) per opts.x_layout."""
    M, N = Y.shape
    if opts.x_layout == ESP_X_CHANNEL_MAJOR:
        K = X.shape[0]
    else:
        K = X.shape[1]
    st = esp_spgemm_raw(X, M, K, X.stride(0), packed, perm, N, Y, Y.stride(0), opts, workspace,
                        0 if workspace is None else workspace.numel() * workspace.element_size(), _stream(stream))
    if st != ESP_OK:
        raise EsparseError(st, "esp_spgemm")


_lib.esp_spgemm_tune.restype = c_int
_lib.esp_spgemm_tune.argtypes = [c_void_p, c_int, c_int, c_long, c_void_p, c_void_p, c_int, c_void_p, c_long,
                                 POINTER(esp_gemm_opts), c_void_p, c_size_t, c_int, POINTER(ctypes.c_float),
                                 POINTER(ctypes.c_float), c_void_p]


def esp_spgemm_tune(X, packed, perm, Y, opts, workspace=None, reps=5, stream=None) -> dict:
    """Times the admissible launch configurations on these buffers and writes the fastest into `opts` (see the header).
    Returns {"kernel", "token_tile", "split_k", "best_us", "planned_us"}."""
    M, N = Y.shape
    K = X.shape[0] if opts.x_layout == ESP_X_CHANNEL_MAJOR else X.shape[1]
    best, planned = ctypes.c_float(), ctypes.c_float()
    st = int(_lib.esp_spgemm_tune(_ptr(X), M, K, X.stride(0), _ptr(packed), _ptr(perm), N, _ptr(Y), Y.stride(0),
                                  ctypes.byref(opts), _ptr(workspace),
                                  0 if workspace is None else workspace.numel() * workspace.element_size(), reps,
                                  ctypes.byref(best), ctypes.byref(planned), _stream(stream)))
    if st != ESP_OK:
        raise EsparseError(st, "esp_spgemm_tune")
    return {"kernel": opts.force_kernel, "token_tile": opts.token_tile, "split_k": opts.split_k,
            "pipeline_stages": opts.pipeline_stages, "best_us": best.value, "planned_us": planned.value}


_lib.esp_spgemm_grouped.restype = c_int
_lib.esp_spgemm_grouped.argtypes = [c_int, POINTER(c_void_p), c_int, c_int, c_long, POINTER(c_void_p), POINTER(c_void_p),
                                    POINTER(c_int), POINTER(c_void_p), POINTER(c_long), POINTER(esp_gemm_opts), c_void_p,
                                    c_size_t, c_void_p]


def esp_spgemm_grouped(Xs, packeds, perms, Ys, opts, workspace=None, stream=None):
    """Ys[i] = Xs[i] . P[i] . W_s[i]^T for up to 4 problems with common M and K in one call (one launch up to 256 tokens)."""
    n = len(Ys)
    M = Ys[0].shape[0]
    K = Xs[0].shape[0] if opts.x_layout == ESP_X_CHANNEL_MAJOR else Xs[0].shape[1]
    arr = lambda items: (c_void_p * n)(*[_ptr(t) for t in items])
    Ns = (c_int * n)(*[y.shape[1] for y in Ys])
    ldys = (c_long * n)(*[y.stride(0) for y in Ys])
    st = int(_lib.esp_spgemm_grouped(n, arr(Xs), M, K, Xs[0].stride(0), arr(packeds), arr(perms), Ns, arr(Ys), ldys,
                                     ctypes.byref(opts), _ptr(workspace),
                                     0 if workspace is None else workspace.numel() * workspace.element_size(), _stream(stream)))
    if st != ESP_OK:
        raise EsparseError(st, "esp_spgemm_grouped")


def plan_key(M: int, N: int, K: int, opts: esp_gemm_opts) -> str:
    return f"{M}x{N}x{K}:layout{opts.x_layout}:out{opts.out_dtype}:static{opts.static_weights}"


def save_plan_table(path: str, table: dict) -> None:
    """Persists tuned configurations: {plan_key(...): {"kernel": .., "token_tile": .., "split_k": ..}} as JSON."""
    import json
    with open(path, "w") as f:
        json.dump({k: {"kernel": int(v["kernel"]), "token_tile": int(v["token_tile"]), "split_k": int(v["split_k"]),
                       "pipeline_stages": int(v.get("pipeline_stages", 0))}
                   for k, v in table.items()}, f, indent=1, sort_keys=True)


def load_plan_table(path: str) -> dict:
    import json
    with open(path) as f:
        return json.load(f)


def apply_plan(opts: esp_gemm_opts, table: dict, M: int, N: int, K: int) -> bool:
    """Sets opts.force_kernel / token_tile / split_k from the table's entry for these sizes; False if there is none."""
    e = table.get(plan_key(M, N, K, opts))
    if e is None:
        return False
    opts.force_kernel, opts.token_tile, opts.split_k = e["kernel"], e["token_tile"], e["split_k"]
    opts.pipeline_stages = e.get("pipeline_stages", 0)
    return True


def esp_spgemm_static_raw(X, M, K, ldx, packed, perm, N, Y, ldy, out_dtype, stream) -> int:
    return int(_lib.esp_spgemm_static(_ptr(X), M, K, ldx, _ptr(packed), _ptr(perm), N, _ptr(Y), ldy, out_dtype,
                                      stream))


def esp_spgemm_static(X, packed, perm, Y, stream=None):
    """Y [M,N] = X . P . W_s^T for token-major X [M,K] with the library's built-in scratch: no workspace and
    no allocation (for callers that cannot allocate device memory).  Y's dtype picks fp16 or fp32 output."""
    import torch
    M, N = Y.shape
    K = X.shape[1]
    out = ESP_OUT_F32 if Y.dtype == torch.float32 else ESP_OUT_F16
    st = esp_spgemm_static_raw(X, M, K, X.stride(0), packed, perm, N, Y, Y.stride(0), out, _stream(stream))
    if st != ESP_OK:
        raise EsparseError(st, "esp_spgemm_static")


def esp_selftest_wait_timeout(stream=None) -> None:
    """Launches the kernel whose bounded wait runs out (see include/esparse.h); check esp_last_device_status() after."""
    st = int(_lib.esp_selftest_wait_timeout(_stream(stream)))
    if st != ESP_OK:
        raise EsparseError(st, "esp_selftest_wait_timeout")


_lib.esp_calib_state_bytes.restype = c_size_t
_lib.esp_calib_state_bytes.argtypes = [c_int, c_int]
_lib.esp_calib_reset.restype = c_int
_lib.esp_calib_reset.argtypes = [c_void_p, c_int, c_int, c_void_p]
_lib.esp_calib_range.restype = c_int
_lib.esp_calib_range.argtypes = [c_void_p, c_void_p, c_int, c_int, c_long, c_int, c_void_p]
_lib.esp_calib_histogram.restype = c_int
_lib.esp_calib_histogram.argtypes = [c_void_p, c_void_p, c_int, c_int, c_long, c_int, c_void_p]
_lib.esp_calib_finish.restype = c_int
_lib.esp_calib_finish.argtypes = [c_void_p, c_int, c_longlong, POINTER(esp_prune_opts), c_void_p, c_void_p, c_void_p, c_void_p]


def esp_calib_state_bytes(C: int, bins: int) -> int:
    return int(_lib.esp_calib_state_bytes(C, bins))


def _calib_call(fn, name, *args):
    st = int(fn(*args))
    if st != ESP_OK:
        raise EsparseError(st, name)


def esp_calib_reset(state, C, bins, stream=None):
    _calib_call(_lib.esp_calib_reset, "esp_calib_reset", _ptr(state), C, bins, _stream(stream))


def esp_calib_range(state, X, bins, stream=None):
    _calib_call(_lib.esp_calib_range, "esp_calib_range", _ptr(state), _ptr(X), X.shape[0], X.shape[1], X.stride(0), bins,
                _stream(stream))


def esp_calib_histogram(state, X, bins, stream=None):
    _calib_call(_lib.esp_calib_histogram, "esp_calib_histogram", _ptr(state), _ptr(X), X.shape[0], X.shape[1], X.stride(0),
                bins, _stream(stream))


def esp_calib_finish(state, C, T_total, opts, chan_norm, chan_entropy, chan_score, stream=None):
    _calib_call(_lib.esp_calib_finish, "esp_calib_finish", _ptr(state), C, T_total, ctypes.byref(opts), _ptr(chan_norm),
                _ptr(chan_entropy), _ptr(chan_score), _stream(stream))


def esp_last_device_status() -> int:
    return int(_lib.esp_last_device_status())


def esp_multicast_available() -> bool:
    """True when the optional companion library (ESP_KERNEL_QUAD_MULTICAST) lies beside the main one and loads."""
    return bool(_lib.esp_multicast_available())
