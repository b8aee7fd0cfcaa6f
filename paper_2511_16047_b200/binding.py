"""ctypes binding of libamskv.so: the same names as the C ABI, argument marshalling only.

Every step of the hot path runs inside the library's CUDA kernels.  There is no Python or
CPU implementation behind these calls: if the shared library is missing the import fails,
and without a CUDA device the compute calls return AMSKV_ERR_CUDA.
torch is used by callers for device memory and streams; this module accepts raw addresses
(ints) or torch tensors (their data_ptr is taken).
"""
from __future__ import annotations

import ctypes
import os
from typing import List, Optional, Sequence, Tuple

_HERE = os.path.dirname(os.path.abspath(__file__))
# AMSKV_LIBRARY names another build of the same library (a debug build, say); default: the in-tree one
LIB_PATH = os.environ.get("AMSKV_LIBRARY") or os.path.join(_HERE, "libamskv.so")

OK = 0
ERR_INVALID, ERR_ORDER, ERR_NOMEM, ERR_UNSUPPORTED, ERR_CUDA, ERR_DEVICE_TIMEOUT = -1, -2, -3, -4, -5, -6
MAX_SCALES = 32
FLAG_PLAN_ONLY = 1
FLAG_BULK_APPEND = 2
FLAG_TRANSIENT_LAST_SCALE = 4
FLAG_NVTX = 8
PATH_AUTO, PATH_SIMT, PATH_TENSOR, PATH_TENSOR_PAIR, PATH_SMALL = 0, 1, 2, 3, 4
LAYER_EFFICIENT, LAYER_DEMANDING, LAYER_PROMOTABLE = 0, 1, 2


class LayerPolicy(ctypes.Structure):
    _fields_ = [("n_condensed", ctypes.c_int32), ("n_local", ctypes.c_int32), ("cache_demanding", ctypes.c_int32)]


class TokenBudget(ctypes.Structure):
    _fields_ = [("budget_tokens", ctypes.c_int32), ("condensed_tokens", ctypes.c_int32),
                ("promoted_budget_tokens", ctypes.c_int32)]


class Desc(ctypes.Structure):
    _fields_ = [("layers", ctypes.c_int32), ("heads", ctypes.c_int32), ("head_dim", ctypes.c_int32),
                ("rows", ctypes.c_int32), ("n_scales", ctypes.c_int32),
                ("scale_sides", ctypes.POINTER(ctypes.c_int32)), ("policy", ctypes.POINTER(LayerPolicy)),
                ("softmax_scale", ctypes.c_float), ("flags", ctypes.c_uint32),
                ("token_budget", ctypes.POINTER(TokenBudget))]


class AmskvError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__("%s: %s (%d)" % (where, strerror(code), code))


def _load() -> ctypes.CDLL:
    if not os.path.exists(LIB_PATH):
        raise ImportError("libamskv.so is not built: run `python paper_2511_16047_b200/build.py` "
                          "(there is no fallback implementation)")
    lib = ctypes.CDLL(LIB_PATH)
    vp, i, sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_size_t
    i64p, i32p, szp = ctypes.POINTER(ctypes.c_int64), ctypes.POINTER(ctypes.c_int32), ctypes.POINTER(ctypes.c_size_t)
    dp = ctypes.POINTER(ctypes.c_double)
    sig = {
        "amskv_cache_required_bytes": ([ctypes.POINTER(Desc), szp], i),
        "amskv_cache_create": ([ctypes.POINTER(Desc), vp, sz, ctypes.POINTER(vp)], i),
        "amskv_cache_destroy": ([vp], i),
        "amskv_cache_reset": ([vp], i),
        "amskv_append": ([vp, i, i, vp, vp, i64p, vp], i),
        "amskv_attend": ([vp, i, i, vp, vp, i64p, i64p, vp], i),
        "amskv_append_attend": ([vp, i, i, vp, vp, i64p, vp, vp, i64p, i64p, vp], i),
        "amskv_attention_density": ([vp, i, i, vp, i64p, vp, sz, vp], i),
        "amskv_attend_density": ([vp, i, i, vp, vp, i64p, i64p, vp, sz, vp], i),
        "amskv_set_attend_path": ([vp, i], i),
        "amskv_first_overflow_scale": ([vp, i, ctypes.POINTER(i)], i),
        "amskv_promote_layer": ([vp, i], i),
        "amskv_step_host": ([vp, i, i, vp, vp, vp, vp, vp, sz, vp], i),
        "amskv_step_staging_bytes": ([vp, szp], i),
        "amskv_layer_similarity": ([vp, i, vp, i, i, i, i, vp, vp, sz, vp], i),
        "amskv_similarity_workspace_bytes": ([], sz),
        "amskv_layer_similarity_static": ([vp, i, vp, i, i, i, i, vp, vp], i),
        "amskv_classify_by_threshold": ([dp, i, ctypes.c_double, i32p], i),
        "amskv_classify_lowest": ([dp, i, i, i32p], i),
        "amskv_kept_segments": ([vp, i, i, i32p, i32p], i),
        "amskv_evicted_at": ([vp, i, i, i32p, i32p], i),
        "amskv_resident_ranges": ([vp, i, i, i32p, i32p], i),
        "amskv_attended_tokens": ([vp, i, i, i32p, i32p], i),
        "amskv_append_copies": ([vp, i, i, i32p, i32p], i),
        "amskv_cache_bytes": ([vp, szp, szp, szp], i),
        "amskv_status": ([vp, ctypes.POINTER(i)], i),
        "amskv_selftest_wait_timeout": ([vp, ctypes.c_uint32, vp], i),
        "amskv_launch_count": ([], ctypes.c_int64),
        "amskv_strerror": ([i], ctypes.c_char_p),
    }
    for name, (args, res) in sig.items():
        fn = getattr(lib, name)
        fn.argtypes = args
        fn.restype = res
    return lib


lib = _load()
EXPORTS = ("amskv_cache_required_bytes amskv_cache_create amskv_cache_destroy amskv_cache_reset amskv_append "
           "amskv_attend amskv_append_attend amskv_attention_density amskv_attend_density amskv_first_overflow_scale amskv_promote_layer amskv_set_attend_path amskv_step_host amskv_step_staging_bytes amskv_layer_similarity "
           "amskv_similarity_workspace_bytes amskv_layer_similarity_static amskv_classify_by_threshold amskv_classify_lowest "
           "amskv_kept_segments amskv_evicted_at amskv_resident_ranges amskv_attended_tokens amskv_append_copies "
           "amskv_cache_bytes amskv_status amskv_selftest_wait_timeout "
           "amskv_launch_count amskv_strerror").split()


def strerror(code: int) -> str:
    return lib.amskv_strerror(int(code)).decode()


def _check(code: int, where: str) -> None:
    if code != OK:
        raise AmskvError(code, where)


def _addr(x) -> Optional[int]:
    if x is None:
        return None
    if hasattr(x, "data_ptr"):
        return int(x.data_ptr())
    return int(x)


def _strides(x) -> Optional[ctypes.Array]:
    """Element strides (row, head, token) of a [rows, heads, T, D] tensor, or None if contiguous/raw."""
    if x is None or not hasattr(x, "stride"):
        return None
    if x.is_contiguous():
        return None
    s = x.stride()
    assert x.dim() == 4 and s[3] == 1, "expected [rows, heads, T, D] with contiguous channels"
    return (ctypes.c_int64 * 3)(s[0], s[1], s[2])


def _stream(stream) -> Optional[int]:
    if stream is None:
        return None
    if hasattr(stream, "cuda_stream"):
        return int(stream.cuda_stream)
    return int(stream)


def make_desc(layers: int, heads: int, head_dim: int, rows: int, sides: Sequence[int],
              policies: Sequence[Tuple[int, int, bool]], softmax_scale: float = 0.0, flags: int = 0,
              token_budgets: Optional[Sequence[Tuple[int, int]]] = None):
    """Returns (Desc, keepalive) -- keepalive holds the arrays the descriptor points to.

    token_budgets: optional per-layer (budget_tokens, condensed_tokens[, promoted_budget_tokens]); a layer
    with budget 0 follows its entry of `policies`."""
    sides_arr = (ctypes.c_int32 * len(sides))(*[int(s) for s in sides])
    # the class is False / True, or LAYER_PROMOTABLE
    pol_arr = (LayerPolicy * len(policies))(*[LayerPolicy(int(c), int(w), int(d)) for c, w, d in policies])
    bud_arr = None
    if token_budgets is not None:
        assert len(token_budgets) == len(policies)
        bud_arr = (TokenBudget * len(token_budgets))(*[TokenBudget(int(t[0]), int(t[1]), int(t[2]) if len(t) > 2 else 0)
                                                       for t in token_budgets])
    d = Desc(layers, heads, head_dim, rows, len(sides), sides_arr, pol_arr, float(softmax_scale), flags,
             bud_arr if bud_arr is not None else ctypes.cast(None, ctypes.POINTER(TokenBudget)))
    return d, (sides_arr, pol_arr, bud_arr)


def amskv_cache_required_bytes(desc: Desc) -> int:
    n = ctypes.c_size_t(0)
    _check(lib.amskv_cache_required_bytes(ctypes.byref(desc), ctypes.byref(n)), "amskv_cache_required_bytes")
    return int(n.value)


def amskv_cache_create(desc: Desc, dev_mem=None, dev_bytes: int = 0) -> int:
    handle = ctypes.c_void_p(None)
    _check(lib.amskv_cache_create(ctypes.byref(desc), _addr(dev_mem), int(dev_bytes), ctypes.byref(handle)),
           "amskv_cache_create")
    return handle.value


def amskv_cache_destroy(cache: int) -> None:
    _check(lib.amskv_cache_destroy(cache), "amskv_cache_destroy")


def amskv_first_overflow_scale(cache: int, layer: int) -> int:
    k = ctypes.c_int(0)
    _check(lib.amskv_first_overflow_scale(cache, layer, ctypes.byref(k)), "amskv_first_overflow_scale")
    return int(k.value)


def amskv_promote_layer(cache: int, layer: int) -> None:
    _check(lib.amskv_promote_layer(cache, layer), "amskv_promote_layer")


def amskv_cache_reset(cache: int) -> None:
    _check(lib.amskv_cache_reset(cache), "amskv_cache_reset")


def amskv_append(cache: int, layer: int, scale: int, K, V, stream=None) -> None:
    ks, vs = _strides(K), _strides(V)
    if (ks is None) != (vs is None) or (ks is not None and list(ks) != list(vs)):
        raise ValueError("K and V must share one stride triple")
    _check(lib.amskv_append(cache, layer, scale, _addr(K), _addr(V), ks, _stream(stream)), "amskv_append")


def amskv_attend(cache: int, layer: int, scale: int, Q, out, stream=None) -> None:
    _check(lib.amskv_attend(cache, layer, scale, _addr(Q), _addr(out), _strides(Q), _strides(out), _stream(stream)),
           "amskv_attend")


def amskv_append_attend(cache: int, layer: int, scale: int, K, V, Q, out, stream=None) -> None:
    """append(layer, scale, K, V) then attend(layer, scale, Q, out), as one launch where possible."""
    ks, vs = _strides(K), _strides(V)
    if (ks is None) != (vs is None) or (ks is not None and list(ks) != list(vs)):
        raise ValueError("K and V must share one stride triple")
    _check(lib.amskv_append_attend(cache, layer, scale, _addr(K), _addr(V), ks, _addr(Q), _addr(out), _strides(Q),
                                   _strides(out), _stream(stream)), "amskv_append_attend")


def amskv_attention_density(cache: int, layer: int, scale: int, Q, out, out_entries: int, stream=None) -> None:
    """Attention density per (head, run of amskv_attended_tokens) into `out` (device doubles)."""
    _check(lib.amskv_attention_density(cache, layer, scale, _addr(Q), _strides(Q), _addr(out), int(out_entries),
                                       _stream(stream)), "amskv_attention_density")


def amskv_attend_density(cache: int, layer: int, scale: int, Q, out, density, density_entries: int, stream=None) -> None:
    """amskv_attend plus the attention density of the same queries, from one launch where the paired kernel serves."""
    _check(lib.amskv_attend_density(cache, layer, scale, _addr(Q), _addr(out), _strides(Q), _strides(out), _addr(density),
                                    int(density_entries), _stream(stream)), "amskv_attend_density")


def amskv_set_attend_path(cache: int, path: int) -> None:
    _check(lib.amskv_set_attend_path(cache, path), "amskv_set_attend_path")


def amskv_step_staging_bytes(cache: int) -> int:
    n = ctypes.c_size_t(0)
    _check(lib.amskv_step_staging_bytes(cache, ctypes.byref(n)), "amskv_step_staging_bytes")
    return int(n.value)


def amskv_step_host(cache: int, layer: int, scale: int, K_host, V_host, Q_host, out_host, staging,
                    staging_bytes: int, stream=None) -> None:
    _check(lib.amskv_step_host(cache, layer, scale, _addr(K_host), _addr(V_host), _addr(Q_host), _addr(out_host),
                               _addr(staging), int(staging_bytes), _stream(stream)), "amskv_step_host")


def amskv_similarity_workspace_bytes() -> int:
    return int(lib.amskv_similarity_workspace_bytes())


def amskv_layer_similarity(K_prev, side_prev: int, K_cur, side_cur: int, rows: int, heads: int, head_dim: int,
                           out_ss, workspace, workspace_bytes: int, stream=None) -> None:
    _check(lib.amskv_layer_similarity(_addr(K_prev), side_prev, _addr(K_cur), side_cur, rows, heads, head_dim,
                                      _addr(out_ss), _addr(workspace), int(workspace_bytes), _stream(stream)),
           "amskv_layer_similarity")


def amskv_layer_similarity_static(K_prev, side_prev: int, K_cur, side_cur: int, rows: int, heads: int, head_dim: int,
                                  out_ss, stream=None) -> None:
    """amskv_layer_similarity without a workspace argument, for callers that cannot allocate
    device memory (fixed memory pools, plug-ins, loops where cudaMalloc is off limits): the
    partial sums live in a 16 KB array inside the library.  Calls on one device share that
    array, so they must not overlap on the GPU; problems above 2^30 16-byte chunks are refused."""
    _check(lib.amskv_layer_similarity_static(_addr(K_prev), side_prev, _addr(K_cur), side_cur, rows, heads, head_dim,
                                             _addr(out_ss), _stream(stream)), "amskv_layer_similarity_static")


def amskv_classify_by_threshold(scores: Sequence[float], theta: float) -> List[bool]:
    n = len(scores)
    s = (ctypes.c_double * n)(*scores)
    out = (ctypes.c_int32 * n)()
    _check(lib.amskv_classify_by_threshold(s, n, float(theta), out), "amskv_classify_by_threshold")
    return [bool(v) for v in out]


def amskv_classify_lowest(scores: Sequence[float], n_demanding: int) -> List[bool]:
    n = len(scores)
    s = (ctypes.c_double * n)(*scores)
    out = (ctypes.c_int32 * n)()
    _check(lib.amskv_classify_lowest(s, n, int(n_demanding), out), "amskv_classify_lowest")
    return [bool(v) for v in out]


def _ids(fn, where: str, cache: int, layer: int, scale: int, width: int = 1) -> List[int]:
    buf = (ctypes.c_int32 * (2 * MAX_SCALES))()
    n = ctypes.c_int32(0)
    _check(fn(cache, layer, scale, buf, ctypes.byref(n)), where)
    return [int(buf[j]) for j in range(n.value * width)]


def amskv_kept_segments(cache: int, layer: int, scale: int) -> List[int]:
    return _ids(lib.amskv_kept_segments, "amskv_kept_segments", cache, layer, scale)


def amskv_evicted_at(cache: int, layer: int, scale: int) -> List[int]:
    return _ids(lib.amskv_evicted_at, "amskv_evicted_at", cache, layer, scale)


def amskv_resident_ranges(cache: int, layer: int, scale: int) -> List[Tuple[int, int]]:
    flat = _ids(lib.amskv_resident_ranges, "amskv_resident_ranges", cache, layer, scale, width=2)
    return [(flat[2 * j], flat[2 * j + 1]) for j in range(len(flat) // 2)]


def _triples(fn, where: str, cache: int, layer: int, scale: int) -> List[Tuple[int, int, int]]:
    buf = (ctypes.c_int32 * (3 * 2 * MAX_SCALES))()
    n = ctypes.c_int32(0)
    _check(fn(cache, layer, scale, buf, ctypes.byref(n)), where)
    return [(int(buf[3 * j]), int(buf[3 * j + 1]), int(buf[3 * j + 2])) for j in range(n.value)]


def amskv_attended_tokens(cache: int, layer: int, scale: int) -> List[Tuple[int, int, int]]:
    """Runs (segment, first token, count) the queries of `scale` attend to."""
    return _triples(lib.amskv_attended_tokens, "amskv_attended_tokens", cache, layer, scale)


def amskv_append_copies(cache: int, layer: int, scale: int) -> List[Tuple[int, int, int]]:
    """Copies (first source token, destination position, tokens) that append(layer, scale) performs."""
    return _triples(lib.amskv_append_copies, "amskv_append_copies", cache, layer, scale)


def amskv_cache_bytes(cache: int) -> Tuple[int, int, int]:
    a, r, p = ctypes.c_size_t(0), ctypes.c_size_t(0), ctypes.c_size_t(0)
    _check(lib.amskv_cache_bytes(cache, ctypes.byref(a), ctypes.byref(r), ctypes.byref(p)), "amskv_cache_bytes")
    return int(a.value), int(r.value), int(p.value)


def amskv_status(cache: int) -> int:
    """Device status word (0 = fine); the call clears it.  Synchronises the device."""
    w = ctypes.c_int(0)
    rc = lib.amskv_status(cache, ctypes.byref(w))
    if rc not in (OK, ERR_DEVICE_TIMEOUT):
        raise AmskvError(rc, "amskv_status")
    return int(w.value)


def amskv_selftest_wait_timeout(cache: int, iterations: int, stream=None) -> None:
    """Enqueues the diagnostic kernel whose bounded wait runs out after `iterations` polls."""
    _check(lib.amskv_selftest_wait_timeout(cache, int(iterations), _stream(stream)), "amskv_selftest_wait_timeout")


def amskv_launch_count() -> int:
    return int(lib.amskv_launch_count())
