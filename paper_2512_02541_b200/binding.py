"""ctypes binding of libavggt.so: same names as the C ABI, argument marshalling only.

Every step of the path runs inside the library's CUDA kernels.  There is no
fallback: if the shared library is missing and cannot be built, importing the
entry points raises.
"""

import ctypes
import os

from . import build as _build

AVGGT_OK = 0
AVGGT_ERR_INVALID_ARG = -1
AVGGT_ERR_UNSUPPORTED = -2
AVGGT_ERR_WORKSPACE_TOO_SMALL = -3
AVGGT_ERR_ALIGNMENT = -4
AVGGT_ERR_CUDA = -5
AVGGT_ERR_DEVICE_TIMEOUT = -6
AVGGT_ERR_STATIC_SCRATCH = -7

AVGGT_FLAG_KEEP_FIRST_FRAME = 1
AVGGT_MEAN_OFF, AVGGT_MEAN_UNIT, AVGGT_MEAN_FILL = 0, 1, 2

# every symbol include/avggt.h declares
EXPORTS = (
    "avggt_kv_count", "avggt_workspace_bytes", "avggt_build_kv", "avggt_build_kv_noalloc", "avggt_global_attn",
    "avggt_frame_attn", "avggt_build_kv_indexed", "avggt_global_attn_indexed", "avggt_global_attn_shard",
    "avggt_build_kv_shard", "avggt_shard_assemble", "avggt_project_workspace_bytes", "avggt_project_build_kv",
    "avggt_check_status", "avggt_strerror", "avggt_last_cuda_error", "avggt_version",
)


class AvggtParams(ctypes.Structure):
    """Mirror of ``avggt_params`` in include/avggt.h."""

    _fields_ = [
        ("batch", ctypes.c_int32),
        ("n_frames", ctypes.c_int32),
        ("tokens_per_frame", ctypes.c_int32),
        ("grid_h", ctypes.c_int32),
        ("grid_w", ctypes.c_int32),
        ("n_special", ctypes.c_int32),
        ("n_heads", ctypes.c_int32),
        ("head_dim", ctypes.c_int32),
        ("sigma", ctypes.c_int32),
        ("diag", ctypes.c_int32),
        ("mean_fill", ctypes.c_int32),
        ("softmax_scale", ctypes.c_float),
        ("flags", ctypes.c_uint32),
    ]


class AvggtError(RuntimeError):
    def __init__(self, code, where):
        self.code = code
        msg = lib().avggt_strerror(code).decode()
        if code == AVGGT_ERR_CUDA:
            msg += ": " + lib().avggt_last_cuda_error().decode()
        super().__init__(f"{where}: {msg} ({code})")


_LIB = None


def load_library(path):
    """ctypes handle of a build of the library at ``path`` with every entry point's signature declared."""
    L = ctypes.CDLL(path)
    vp, i64p, szp = ctypes.c_void_p, ctypes.POINTER(ctypes.c_int64), ctypes.POINTER(ctypes.c_size_t)
    pp = ctypes.POINTER(AvggtParams)
    sz, i64 = ctypes.c_size_t, ctypes.c_int64
    signatures = {
        "avggt_kv_count": [pp, i64p, i64p],
        "avggt_workspace_bytes": [pp, szp, szp],
        "avggt_build_kv": [pp, vp, vp, vp, vp, vp, vp, vp, vp, sz, vp],
        "avggt_build_kv_noalloc": [pp, vp, vp, vp, vp, vp, vp, vp, vp],
        "avggt_global_attn": [pp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, sz, vp],
        "avggt_frame_attn": [pp, vp, vp, vp, vp, vp, vp, sz, vp],
        "avggt_build_kv_indexed": [pp, vp, i64, vp, vp, vp, vp, vp, vp, vp, vp, sz, vp],
        "avggt_global_attn_indexed": [pp, i64, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, sz, vp],
        "avggt_global_attn_shard": [pp, i64, i64, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, sz, vp],
        "avggt_build_kv_shard": [pp, vp, vp, vp, i64, vp, vp, vp, sz, vp],
        "avggt_shard_assemble": [pp, vp, ctypes.c_int32, i64p, i64, vp, i64, vp, vp, vp, vp, vp],
        "avggt_project_workspace_bytes": [pp, ctypes.c_int32, szp],
        "avggt_project_build_kv": [pp, ctypes.c_int32, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, sz, vp],
        "avggt_check_status": [vp, ctypes.POINTER(ctypes.c_uint32)],
        "avggt_strerror": [ctypes.c_int],
        "avggt_last_cuda_error": [],
        "avggt_version": [],
    }
    assert set(signatures) == set(EXPORTS)
    for name, argtypes in signatures.items():
        f = getattr(L, name)
        f.argtypes = argtypes
        f.restype = ctypes.c_char_p if name in ("avggt_strerror", "avggt_last_cuda_error", "avggt_version") else ctypes.c_int
    return L


def lib():
    """The loaded shared library (built in-tree on first use if stale or absent)."""
    global _LIB
    if _LIB is None:
        path = _build.LIB
        if _build.needs_build():
            try:
                path = _build.build()
            except Exception:
                if not os.path.exists(_build.LIB):
                    raise
                path = _build.LIB      # no compiler on this machine: use the library that shipped
        _LIB = load_library(path)
    return _LIB


def make_params(n_frames, grid_h, grid_w, n_special, n_heads, head_dim, sigma, diag=1, mean_fill=AVGGT_MEAN_FILL,
                softmax_scale=0.0, keep_first_frame=False, batch=1):
    return AvggtParams(batch, n_frames, n_special + grid_h * grid_w, grid_h, grid_w, n_special, n_heads, head_dim,
                       sigma, int(diag), int(mean_fill), float(softmax_scale),
                       AVGGT_FLAG_KEEP_FIRST_FRAME if keep_first_frame else 0)


def _check(code, where):
    if code != AVGGT_OK:
        raise AvggtError(code, where)


def _ptr(t):
    """Device (or host) address of a tensor-like object, or None."""
    if t is None:
        return None
    if isinstance(t, int):
        return t
    return t.data_ptr()


def avggt_kv_count(params):
    """-> (M, n_dropped)."""
    m, nd = ctypes.c_int64(), ctypes.c_int64()
    _check(lib().avggt_kv_count(ctypes.byref(params), ctypes.byref(m), ctypes.byref(nd)), "avggt_kv_count")
    return m.value, nd.value


def avggt_workspace_bytes(params):
    """-> (build_ws_bytes, attn_ws_bytes) on the current CUDA device."""
    b, a = ctypes.c_size_t(), ctypes.c_size_t()
    _check(lib().avggt_workspace_bytes(ctypes.byref(params), ctypes.byref(b), ctypes.byref(a)), "avggt_workspace_bytes")
    return b.value, a.value


def avggt_build_kv(params, K, V, Kc, Vc, idx, kmean, vmean, ws, ws_bytes, stream=None):
    """Enqueue the K/V compaction + mean reduction.  Arguments are tensors (or raw addresses)."""
    _check(lib().avggt_build_kv(ctypes.byref(params), _ptr(K), _ptr(V), _ptr(Kc), _ptr(Vc), _ptr(idx), _ptr(kmean),
                                _ptr(vmean), _ptr(ws), ws_bytes, stream), "avggt_build_kv")


def avggt_build_kv_noalloc(params, K, V, Kc, Vc, idx, kmean, vmean, stream=None):
    """avggt_build_kv without a workspace, for callers that cannot allocate device memory (a host
    whose memory manager owns the whole GPU, a plugin under a fixed budget, a loop that must not
    call cudaMalloc).  The scratch is a fixed array inside the library: n_heads * head_dim <= 1024,
    calls that overlap on the GPU race, and the first call on a device should precede any stream
    capture.  This binding allocates nothing either."""
    _check(lib().avggt_build_kv_noalloc(ctypes.byref(params), _ptr(K), _ptr(V), _ptr(Kc), _ptr(Vc), _ptr(idx),
                                        _ptr(kmean), _ptr(vmean), stream), "avggt_build_kv_noalloc")


def avggt_global_attn(params, Q, K, V, Kc, Vc, kmean, vmean, O, lse, ws, ws_bytes, stream=None):
    """Enqueue the subsampled global attention."""
    _check(lib().avggt_global_attn(ctypes.byref(params), _ptr(Q), _ptr(K), _ptr(V), _ptr(Kc), _ptr(Vc), _ptr(kmean),
                                   _ptr(vmean), _ptr(O), _ptr(lse), _ptr(ws), ws_bytes, stream), "avggt_global_attn")


def avggt_build_kv_indexed(params, idx, n_kept, K, V, Kc, Vc, slot_of_token, kmean, vmean, ws, ws_bytes, stream=None):
    """Enqueue the compaction + mean reduction for a caller-chosen retained set (ascending int32 token indices)."""
    _check(lib().avggt_build_kv_indexed(ctypes.byref(params), _ptr(idx), n_kept, _ptr(K), _ptr(V), _ptr(Kc), _ptr(Vc),
                                        _ptr(slot_of_token), _ptr(kmean), _ptr(vmean), _ptr(ws), ws_bytes, stream),
           "avggt_build_kv_indexed")


def avggt_global_attn_indexed(params, n_kept, slot_of_token, Q, K, V, Kc, Vc, kmean, vmean, O, lse, ws, ws_bytes,
                              stream=None):
    """Enqueue the attention over a caller-chosen retained set."""
    _check(lib().avggt_global_attn_indexed(ctypes.byref(params), n_kept, _ptr(slot_of_token), _ptr(Q), _ptr(K), _ptr(V),
                                           _ptr(Kc), _ptr(Vc), _ptr(kmean), _ptr(vmean), _ptr(O), _ptr(lse), _ptr(ws),
                                           ws_bytes, stream), "avggt_global_attn_indexed")


def avggt_global_attn_shard(params, n_kept_total, n_dropped_total, Q, K, V, Kc, Vc, kmean, vmean, O, lse, ws, ws_bytes,
                            stream=None):
    """Enqueue the attention of one frame shard against the whole sequence's compact keys and mean pair."""
    _check(lib().avggt_global_attn_shard(ctypes.byref(params), n_kept_total, n_dropped_total, _ptr(Q), _ptr(K), _ptr(V),
                                         _ptr(Kc), _ptr(Vc), _ptr(kmean), _ptr(vmean), _ptr(O), _ptr(lse), _ptr(ws),
                                         ws_bytes, stream), "avggt_global_attn_shard")


def avggt_build_kv_shard(params, K, V, slot, slot_rows, idx, sums, ws, ws_bytes, stream=None):
    """Enqueue the compaction of one frame shard into its slot [2][H][slot_rows][d] of the exchange buffer;
    ``sums`` [2][H][d] receives the un-normalised sums over the shard's dropped tokens."""
    _check(lib().avggt_build_kv_shard(ctypes.byref(params), _ptr(K), _ptr(V), _ptr(slot), slot_rows, _ptr(idx), _ptr(sums),
                                      _ptr(ws), ws_bytes, stream), "avggt_build_kv_shard")


def avggt_shard_assemble(params, gathered, kept, slot_rows, sums, n_dropped_total, Kc, Vc, kmean, vmean, stream=None):
    """Enqueue the assembly of the gathered slots [n_ranks][2][H][slot_rows][d] into Kc, Vc [H][sum(kept)][d] and
    the division of the all-reduced sums by the total dropped count.  ``kept``: M of every rank (host ints)."""
    arr = (ctypes.c_int64 * len(kept))(*[int(k) for k in kept])
    _check(lib().avggt_shard_assemble(ctypes.byref(params), _ptr(gathered), len(kept), arr, slot_rows, _ptr(sums),
                                      n_dropped_total, _ptr(Kc), _ptr(Vc), _ptr(kmean), _ptr(vmean), stream),
           "avggt_shard_assemble")


def avggt_project_workspace_bytes(params, model_dim):
    """-> workspace bytes of avggt_project_build_kv on the current CUDA device."""
    b = ctypes.c_size_t()
    _check(lib().avggt_project_workspace_bytes(ctypes.byref(params), model_dim, ctypes.byref(b)), "avggt_project_workspace_bytes")
    return b.value


def avggt_project_build_kv(params, model_dim, X, Wk, Wv, bias_k, bias_v, K, V, Kc, Vc, idx, kmean, vmean, ws, ws_bytes,
                           stream=None):
    """Enqueue K = X Wk^T + bias_k, V = X Wv^T + bias_v with the K/V compaction and the mean reduction in the
    projection's epilogue.  K, V (the full arrays) may both be None."""
    _check(lib().avggt_project_build_kv(ctypes.byref(params), model_dim, _ptr(X), _ptr(Wk), _ptr(Wv), _ptr(bias_k),
                                        _ptr(bias_v), _ptr(K), _ptr(V), _ptr(Kc), _ptr(Vc), _ptr(idx), _ptr(kmean),
                                        _ptr(vmean), _ptr(ws), ws_bytes, stream), "avggt_project_build_kv")


def avggt_frame_attn(params, Q, K, V, O, lse, ws, ws_bytes, stream=None):
    """Enqueue the frame attention of a converted early global block (every frame on its own)."""
    _check(lib().avggt_frame_attn(ctypes.byref(params), _ptr(Q), _ptr(K), _ptr(V), _ptr(O), _ptr(lse), _ptr(ws),
                                  ws_bytes, stream), "avggt_frame_attn")


def avggt_check_status(attn_ws):
    """After a stream synchronise: raises AvggtError if a device-side wait gave up."""
    detail = (ctypes.c_uint32 * 4)()
    code = lib().avggt_check_status(_ptr(attn_ws), detail)
    if code != AVGGT_OK:
        err = AvggtError(code, "avggt_check_status")
        err.detail = tuple(detail)
        raise err


def avggt_version():
    return lib().avggt_version().decode()
