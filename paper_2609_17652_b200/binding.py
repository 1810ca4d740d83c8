"""ctypes binding of libfathom.so: argument marshalling only, every step runs in the CUDA kernels.

The function names are those of the C ABI (include/fathom.h).  Tensors are torch tensors used as
plain device (or pinned host) buffers; their data pointers are passed through unchanged.  There is
no CPU fallback: if the library cannot be loaded, importing raises.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libfathom.so")

F32, BF16 = 0, 1
DEPTH_WATERFILL, DEPTH_FIXED_TOP_R, DEPTH_UNIFORM = 0, 1, 2
MAX_K = 16384
DEV_TOPK_SHORT, DEV_WAIT_EXPIRED = 0x1, 0x2

EXPORTS = ["fathom_create", "fathom_destroy", "fathom_scratch_bytes", "fathom_strerror", "fathom_last_cuda_error",
           "fathom_device_status", "fathom_version", "fathom_build_planes", "fathom_alloc_depth", "fathom_scan",
           "fathom_topk", "fathom_sparse_attend", "fathom_sparse_attend_static", "fathom_gather_union",
           "fathom_scan_topk", "fathom_calibrate", "fathom_rotate_keys", "fathom_rotate_query",
           "fathom_channel_variance", "fathom_plan_layer_budgets", "fathom_topk_passes", "fathom_build_planes_rotated", "fathom_scan_batch",
           "fathom_scan_set_ctas_per_plan", "fathom_selftest_wait_expiry", "fathom_klt_basis"]


class Layout(C.Structure):
    _fields_ = [("n_kv_heads", C.c_int32), ("n_q_heads", C.c_int32), ("d", C.c_int32), ("reserved", C.c_int32),
                ("n", C.c_int64), ("plane_stride_words", C.c_int64), ("scale_stride", C.c_int64),
                ("score_stride", C.c_int64)]


def make_layout(Hkv: int, Hq: int, n: int, d: int = 128, row_align_bytes: int = 128) -> Layout:
    """Strides rounded up so that every (head, channel, plane) row of words, every row of scales and every score row
    starts on a `row_align_bytes` boundary (default 128: a row's 128-byte runs then never straddle a memory line, which
    matters most when the store is read over the host link).  row_align_bytes = 16 gives the tightest strides the
    layout allows."""
    nb = (n + 63) // 64
    a = max(16, row_align_bytes)
    rnd = lambda x, m: (x + m - 1) // m * m
    return Layout(Hkv, Hq, d, 0, n, rnd(nb, a // 8), rnd(nb, a // 2), rnd(n, a // 4))


def _load() -> C.CDLL:
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is missing: run `python -m paper_2609_17652_b200.build` (needs nvcc); "
                          "there is no fallback path")
    lib = C.CDLL(LIB_PATH)
    vp, i32, i64 = C.c_void_p, C.c_int, C.c_int64
    LP = C.POINTER(Layout)
    lib.fathom_create.argtypes = [C.POINTER(vp), i32, C.c_size_t]
    lib.fathom_destroy.argtypes = [vp]
    lib.fathom_scratch_bytes.argtypes = [LP, i32]
    lib.fathom_scratch_bytes.restype = C.c_size_t
    lib.fathom_strerror.argtypes = [i32]
    lib.fathom_strerror.restype = C.c_char_p
    lib.fathom_last_cuda_error.argtypes = [vp]
    lib.fathom_last_cuda_error.restype = C.c_char_p
    lib.fathom_device_status.argtypes = [vp, vp, C.POINTER(C.c_uint32)]
    lib.fathom_version.argtypes = []
    lib.fathom_build_planes.argtypes = [vp, LP, vp, i32, vp, vp, vp]
    lib.fathom_alloc_depth.argtypes = [vp, LP, vp, vp, i32, i32, i32, vp, vp]
    lib.fathom_scan.argtypes = [vp, LP, vp, vp, vp, vp, i32, vp, vp]
    lib.fathom_topk.argtypes = [vp, LP, vp, i32, i32, i32, vp, vp]
    lib.fathom_sparse_attend.argtypes = [vp, LP, vp, vp, vp, i32, vp, i32, C.c_float, vp, vp]
    lib.fathom_calibrate.argtypes = [vp, LP, vp, i32, vp, vp, vp]
    lib.fathom_rotate_keys.argtypes = [vp, LP, vp, i32, vp, vp, vp, vp]
    lib.fathom_rotate_query.argtypes = [vp, LP, vp, vp, vp, vp]
    lib.fathom_klt_basis.argtypes = [vp, LP, vp, vp, vp, vp]
    lib.fathom_channel_variance.argtypes = [vp, LP, vp, i32, vp, vp, vp]
    lib.fathom_plan_layer_budgets.argtypes = [vp, i32, i32, vp, C.c_double, vp]
    lib.fathom_topk_passes.argtypes = [LP, i32, i32, i32]
    lib.fathom_scan_batch.argtypes = [vp, vp, i32, i32, vp]
    lib.fathom_scan_set_ctas_per_plan.argtypes = [i32]
    lib.fathom_selftest_wait_expiry.argtypes = [vp, i32, vp]
    lib.fathom_build_planes_rotated.argtypes = [vp, LP, vp, i32, vp, vp, vp, vp, vp]
    lib.fathom_scan_topk.argtypes = [vp, LP, vp, vp, vp, vp, i32, i32, i32, i32, vp, vp]
    lib.fathom_gather_union.argtypes = [vp, LP, vp, i32, vp, vp, i32, vp, vp, vp, vp, vp]
    lib.fathom_sparse_attend_static.argtypes = [LP, vp, vp, vp, i32, vp, i32, C.c_float, vp, vp]
    for name in EXPORTS:
        if name not in ("fathom_scratch_bytes", "fathom_strerror", "fathom_last_cuda_error"):
            getattr(lib, name).restype = C.c_int
    return lib


lib = _load()


class ScanItem(C.Structure):
    _fields_ = [("layout", Layout), ("planes", C.c_void_p), ("scales", C.c_void_p), ("q", C.c_void_p),
                ("depth", C.c_void_p), ("scores", C.c_void_p)]


class FathomError(RuntimeError):
    def __init__(self, status: int, ctx=None):
        msg = lib.fathom_strerror(status).decode()
        if status == -5 and ctx is not None:
            msg += ": " + lib.fathom_last_cuda_error(ctx).decode()
        super().__init__(f"fathom status {status}: {msg}")
        self.status = status


def _ptr(t) -> int:
    if t is None:
        return 0
    if isinstance(t, int):
        return t
    return t.data_ptr()


def _stream(stream) -> int:
    if stream is None:
        return torch.cuda.current_stream().cuda_stream
    if isinstance(stream, int):
        return stream
    return stream.cuda_stream


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return F32
    if t.dtype == torch.bfloat16:
        return BF16
    raise TypeError(f"unsupported dtype {t.dtype}")


class Context:
    """Owns one fathom_ctx (scratch arena + status word) on one device."""

    def __init__(self, device: int = 0, scratch_bytes: int = 0):
        self._h = C.c_void_p()
        rc = lib.fathom_create(C.byref(self._h), device, scratch_bytes)
        if rc != 0:
            raise FathomError(rc)
        self.device, self.scratch_bytes = device, scratch_bytes

    def close(self):
        if self._h:
            lib.fathom_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _check(self, rc: int):
        if rc != 0:
            raise FathomError(rc, self._h)

    # ---- the five calls (raw status returned by the *_rc variants is used by the error-path tests)
    def fathom_build_planes(self, layout, K, planes, scales, stream=None, k_dtype=None):
        self._check(lib.fathom_build_planes(self._h, C.byref(layout), _ptr(K), _dtype_code(K) if k_dtype is None else k_dtype,
                                            _ptr(planes), _ptr(scales), _stream(stream)))

    def fathom_alloc_depth(self, layout, q, var, mode, budget, heads_per_plan, depth, stream=None):
        self._check(lib.fathom_alloc_depth(self._h, C.byref(layout), _ptr(q), _ptr(var), mode, budget, heads_per_plan,
                                           _ptr(depth), _stream(stream)))

    def fathom_scan(self, layout, planes, scales, q, depth, heads_per_plan, scores, stream=None):
        self._check(lib.fathom_scan(self._h, C.byref(layout), _ptr(planes), _ptr(scales), _ptr(q), _ptr(depth),
                                    heads_per_plan, _ptr(scores), _stream(stream)))

    def fathom_scan_batch(self, items, heads_per_plan, stream=None):
        """items: sequence of (layout, planes, scales, q, depth, scores)."""
        arr = (ScanItem * len(items))()
        for i, (lay, planes, scales, q, depth, scores) in enumerate(items):
            arr[i].layout = lay
            arr[i].planes, arr[i].scales, arr[i].q = _ptr(planes), _ptr(scales), _ptr(q)
            arr[i].depth, arr[i].scores = _ptr(depth), _ptr(scores)
        self._check(lib.fathom_scan_batch(self._h, arr, len(items), heads_per_plan, _stream(stream)))

    def fathom_topk(self, layout, scores, k, n_sink, n_local, idx, stream=None):
        self._check(lib.fathom_topk(self._h, C.byref(layout), _ptr(scores), k, n_sink, n_local, _ptr(idx), _stream(stream)))

    def fathom_sparse_attend(self, layout, q, Krows, Vrows, idx, k, softmax_scale, out, stream=None, row_dtype=None):
        self._check(lib.fathom_sparse_attend(self._h, C.byref(layout), _ptr(q), _ptr(Krows), _ptr(Vrows),
                                             _dtype_code(Krows) if row_dtype is None else row_dtype, _ptr(idx), k,
                                             C.c_float(softmax_scale), _ptr(out), _stream(stream)))

    def fathom_calibrate(self, layout, K, mean, cov, stream=None):
        self._check(lib.fathom_calibrate(self._h, C.byref(layout), _ptr(K), _dtype_code(K), _ptr(mean), _ptr(cov), _stream(stream)))

    def fathom_channel_variance(self, layout, K, mean, var, stream=None):
        self._check(lib.fathom_channel_variance(self._h, C.byref(layout), _ptr(K), _dtype_code(K), _ptr(mean), _ptr(var), _stream(stream)))

    def fathom_klt_basis(self, layout, cov, basis, eigenvalues, stream=None):
        self._check(lib.fathom_klt_basis(self._h, C.byref(layout), _ptr(cov), _ptr(basis), _ptr(eigenvalues), _stream(stream)))

    def fathom_rotate_keys(self, layout, K, mean, basis, K_rot, stream=None):
        self._check(lib.fathom_rotate_keys(self._h, C.byref(layout), _ptr(K), _dtype_code(K), _ptr(mean), _ptr(basis),
                                           _ptr(K_rot), _stream(stream)))

    def fathom_build_planes_rotated(self, layout, K, mean, basis, planes, scales, stream=None):
        self._check(lib.fathom_build_planes_rotated(self._h, C.byref(layout), _ptr(K), _dtype_code(K), _ptr(mean), _ptr(basis),
                                                    _ptr(planes), _ptr(scales), _stream(stream)))

    def fathom_rotate_query(self, layout, q, basis, q_rot, stream=None):
        self._check(lib.fathom_rotate_query(self._h, C.byref(layout), _ptr(q), _ptr(basis), _ptr(q_rot), _stream(stream)))

    def fathom_scan_topk(self, layout, planes, scales, q, depth, heads_per_plan, k, n_sink, n_local, idx, stream=None):
        self._check(lib.fathom_scan_topk(self._h, C.byref(layout), _ptr(planes), _ptr(scales), _ptr(q), _ptr(depth),
                                         heads_per_plan, k, n_sink, n_local, _ptr(idx), _stream(stream)))

    def fathom_gather_union(self, layout, idx, k, Krows, Vrows, K_stage, V_stage, idx_local, union_count, stream=None,
                            row_dtype=None):
        self._check(lib.fathom_gather_union(self._h, C.byref(layout), _ptr(idx), k, _ptr(Krows), _ptr(Vrows),
                                            _dtype_code(Krows) if row_dtype is None else row_dtype, _ptr(K_stage),
                                            _ptr(V_stage), _ptr(idx_local), _ptr(union_count), _stream(stream)))

    def fathom_selftest_wait_expiry(self, tries: int = 200, stream=None):
        self._check(lib.fathom_selftest_wait_expiry(self._h, tries, _stream(stream)))

    def fathom_device_status(self, stream=None) -> int:
        st = C.c_uint32(0)
        self._check(lib.fathom_device_status(self._h, _stream(stream), C.byref(st)))
        return st.value


ATTEND_STATIC_MAX_CHUNKS = 2048


def fathom_sparse_attend_static(layout, q, Krows, Vrows, idx, k, softmax_scale, out, stream=None, row_dtype=None):
    """Attention over the selected rows for callers that cannot allocate device memory: no context, no
    scratch arena.  The partial results live in an array built into the library (limit:
    n_q_heads * ceil(k / 128) <= ATTEND_STATIC_MAX_CHUNKS).  The current device must be the stream's; the
    first call on a device looks up the array's address and should come before any stream capture; calls
    that may overlap on the device share the array and must be ordered by the caller."""
    rc = lib.fathom_sparse_attend_static(C.byref(layout), _ptr(q), _ptr(Krows), _ptr(Vrows),
                                         _dtype_code(Krows) if row_dtype is None else row_dtype, _ptr(idx), k,
                                         C.c_float(softmax_scale), _ptr(out), _stream(stream))
    if rc != 0:
        raise FathomError(rc)


def fathom_plan_layer_budgets(err, levels, target_mean: float):
    """Host-side greedy per-layer plan: err [L][n_levels] (any nested sequence of floats), levels ascending ints.
    Returns the chosen level index per layer (marshalling only: the plan is computed inside the library)."""
    L, nlev = len(err), len(levels)
    flat = (C.c_double * (L * nlev))(*[float(x) for row in err for x in row])
    lev = (C.c_int * nlev)(*[int(b) for b in levels])
    out = (C.c_int * L)()
    rc = lib.fathom_plan_layer_budgets(flat, L, nlev, lev, C.c_double(target_mean), out)
    if rc != 0:
        raise FathomError(rc)
    return list(out)


def fathom_topk_passes(layout: Layout, k: int, n_sink: int = 0, n_local: int = 0) -> int:
    rc = int(lib.fathom_topk_passes(C.byref(layout), k, n_sink, n_local))
    if rc < 0:
        raise FathomError(rc)
    return rc


def fathom_scan_set_ctas_per_plan(ctas: int) -> None:
    """Process-wide tuning knob: CTAs per plan of every later scan launch; 0 = automatic."""
    lib.fathom_scan_set_ctas_per_plan(int(ctas))


def fathom_scratch_bytes(layout: Layout, k: int) -> int:
    return int(lib.fathom_scratch_bytes(C.byref(layout), k))


def fathom_version() -> int:
    return int(lib.fathom_version())
