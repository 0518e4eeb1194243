"""Thin Python binding of libmosaic.so (the C ABI declared in include/mosaic.h).

Argument marshalling only: every function takes torch tensors that already
live on the CUDA device (torch is used for device memory and streams), passes
their raw pointers and sizes through ctypes, and raises `MosaicError` on a
non-zero status.  All arithmetic of the method runs inside the library's CUDA
kernels; there is no CPU fallback - if the library cannot be loaded the import
of a function here fails loudly.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libmosaic.so")

F32, BF16 = 0, 1
RESET_ACCUM = 1
GLOBAL_NORM, PER_CATEGORY_NORM = 0, 1
WEIGHTED_MEAN = 2        # flag, or-ed into the mode
REDISTRIBUTE = 4         # flag, or-ed into the mode: clamp and redistribute
ROWS_GIVEN, COLS_GIVEN, RANK_ONLY, SCORES_ONLY, SCORES_ACCUM = 1, 2, 4, 8, 16
OK, ERR_INFEASIBLE = 0, -9

# every symbol include/mosaic.h declares
SYMBOLS = (
    "mosaic_version", "mosaic_status_string",
    "mosaic_act_norms_workspace_bytes", "mosaic_act_norms",
    "mosaic_score",
    "mosaic_outlier_ratio_workspace_bytes", "mosaic_outlier_ratio", "mosaic_ratio_from_count",
    "mosaic_outlier_ratio_static_max_workspace_bytes", "mosaic_outlier_ratio_static",
    "mosaic_outlier_ratio_batch_workspace_bytes", "mosaic_outlier_ratio_batch", "mosaic_outlier_ratio_grouped",
    "mosaic_allocate_sparsity",
    "mosaic_prune_unstructured_workspace_bytes", "mosaic_prune_unstructured",
    "mosaic_prune_unstructured_batch_workspace_bytes", "mosaic_prune_unstructured_batch",
    "mosaic_prune_structured_compact_workspace_bytes", "mosaic_prune_structured_compact",
    "mosaic_rank_units", "mosaic_sum_unit_scores",
    "mosaic_unit_scores_batch_workspace_bytes", "mosaic_unit_scores_batch", "mosaic_add_unit_scores_batch",
    "mosaic_rank_units_batch", "mosaic_compact_batch",
    "mosaic_gram_accumulate", "mosaic_bounded_wait_selftest",
)


class MosaicError(RuntimeError):
    def __init__(self, status: int, what: str):
        self.status = status
        super().__init__(f"{what}: {status_string(status)} ({status})")


_lib = None


def lib() -> C.CDLL:
    """Load libmosaic.so (once).  Raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(
                f"{LIB_PATH} is missing: build it with `python -m paper_2504_06323_b200.build` "
                "(there is no fallback path)")
        L = C.CDLL(LIB_PATH)
        i64, vp, sz, ci, dbl, flt = C.c_int64, C.c_void_p, C.c_size_t, C.c_int, C.c_double, C.c_float
        L.mosaic_version.restype = ci
        L.mosaic_status_string.restype = C.c_char_p
        L.mosaic_status_string.argtypes = [ci]
        L.mosaic_bounded_wait_selftest.restype = ci
        L.mosaic_bounded_wait_selftest.argtypes = [i64, vp, vp]
        L.mosaic_gram_accumulate.restype = ci
        L.mosaic_gram_accumulate.argtypes = [vp, i64, i64, i64, ci, vp, i64, ci, vp, vp]
        L.mosaic_act_norms_workspace_bytes.restype = sz
        L.mosaic_act_norms_workspace_bytes.argtypes = [i64, i64]
        L.mosaic_act_norms.restype = ci
        L.mosaic_act_norms.argtypes = [vp, i64, i64, i64, ci, vp, vp, ci, vp, sz, vp]
        L.mosaic_score.restype = ci
        L.mosaic_score.argtypes = [vp, i64, i64, i64, ci, vp, vp, vp]
        L.mosaic_outlier_ratio_workspace_bytes.restype = sz
        L.mosaic_outlier_ratio_workspace_bytes.argtypes = [i64, i64]
        L.mosaic_outlier_ratio.restype = ci
        L.mosaic_outlier_ratio.argtypes = [vp, i64, i64, i64, ci, vp, flt, vp, vp, vp, sz, vp]
        L.mosaic_outlier_ratio_static_max_workspace_bytes.restype = sz
        L.mosaic_outlier_ratio_static_max_workspace_bytes.argtypes = []
        L.mosaic_outlier_ratio_static.restype = ci
        L.mosaic_outlier_ratio_static.argtypes = [vp, i64, i64, i64, ci, vp, flt, vp, vp, vp]
        L.mosaic_outlier_ratio_batch_workspace_bytes.restype = sz
        L.mosaic_outlier_ratio_batch_workspace_bytes.argtypes = [vp, i64]
        L.mosaic_outlier_ratio_batch.restype = ci
        L.mosaic_outlier_ratio_batch.argtypes = [vp, i64, ci, flt, vp, sz, vp]
        L.mosaic_outlier_ratio_grouped.restype = ci
        L.mosaic_outlier_ratio_grouped.argtypes = [vp, vp, i64, ci, flt, vp, sz, vp]
        L.mosaic_ratio_from_count.restype = dbl
        L.mosaic_ratio_from_count.argtypes = [i64, i64]
        L.mosaic_allocate_sparsity.restype = ci
        L.mosaic_allocate_sparsity.argtypes = [vp, vp, vp, ci, ci, dbl, dbl, ci, vp, vp]
        L.mosaic_prune_unstructured_workspace_bytes.restype = sz
        L.mosaic_prune_unstructured_workspace_bytes.argtypes = [i64, i64]
        L.mosaic_prune_unstructured.restype = ci
        L.mosaic_prune_unstructured.argtypes = [vp, vp, i64, i64, i64, ci, vp, i64, vp, vp, sz, vp]
        L.mosaic_prune_unstructured_batch_workspace_bytes.restype = sz
        L.mosaic_prune_unstructured_batch_workspace_bytes.argtypes = [vp, i64, ci]
        L.mosaic_prune_unstructured_batch.restype = ci
        L.mosaic_prune_unstructured_batch.argtypes = [vp, i64, ci, vp, sz, vp]
        L.mosaic_prune_structured_compact_workspace_bytes.restype = sz
        L.mosaic_prune_structured_compact_workspace_bytes.argtypes = [i64, i64]
        L.mosaic_prune_structured_compact.restype = ci
        L.mosaic_prune_structured_compact.argtypes = [vp, i64, i64, i64, ci, vp, i64, i64, i64, i64, vp, vp, ci, vp,
                                                      vp, vp, sz, vp]
        L.mosaic_rank_units.restype = ci
        L.mosaic_rank_units.argtypes = [vp, i64, i64, vp, vp]
        L.mosaic_sum_unit_scores.restype = ci
        L.mosaic_sum_unit_scores.argtypes = [vp, vp, i64, vp]
        L.mosaic_unit_scores_batch_workspace_bytes.restype = sz
        L.mosaic_unit_scores_batch_workspace_bytes.argtypes = [vp, i64]
        L.mosaic_unit_scores_batch.restype = ci
        L.mosaic_unit_scores_batch.argtypes = [vp, i64, ci, vp, sz, vp]
        L.mosaic_add_unit_scores_batch.restype = ci
        L.mosaic_add_unit_scores_batch.argtypes = [vp, i64, vp]
        L.mosaic_rank_units_batch.restype = ci
        L.mosaic_rank_units_batch.argtypes = [vp, i64, vp]
        L.mosaic_compact_batch.restype = ci
        L.mosaic_compact_batch.argtypes = [vp, i64, ci, vp]
        _lib = L
    return _lib


def status_string(status: int) -> str:
    return lib().mosaic_status_string(int(status)).decode()


def _check(status: int, what: str, allow=()):
    if status != OK and status not in allow:
        raise MosaicError(status, what)
    return status


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.bfloat16:
        return BF16
    if t.dtype == torch.float32:
        return F32
    raise TypeError(f"unsupported dtype {t.dtype}: the library takes float32 or bfloat16")


def _dev(t: torch.Tensor, name: str, dtype=None, ndim=None) -> torch.Tensor:
    if not isinstance(t, torch.Tensor) or not t.is_cuda:
        raise TypeError(f"{name} must be a CUDA tensor (no CPU path exists)")
    if dtype is not None and t.dtype != dtype:
        raise TypeError(f"{name} must be {dtype}, got {t.dtype}")
    if ndim is not None and t.dim() != ndim:
        raise ValueError(f"{name} must have {ndim} dims")
    return t


def _mat(t: torch.Tensor, name: str):
    _dev(t, name, ndim=2)
    if t.stride(1) != 1:
        raise ValueError(f"{name} must be row-major (unit stride along columns)")
    return t.data_ptr(), t.shape[0], t.shape[1], (t.stride(0) if t.shape[0] > 1 else max(t.stride(0), t.shape[1]))


def _ptr(t):
    return None if t is None else t.data_ptr()


def _stream(stream) -> int | None:
    s = torch.cuda.current_stream() if stream is None else stream
    return s.cuda_stream or None


class Workspace:
    """A caller-owned, growable scratch buffer (the library itself allocates nothing)."""

    def __init__(self, device="cuda"):
        self.device = torch.device(device)
        self.buf = None

    def get(self, nbytes: int) -> tuple[int, int]:
        nbytes = max(int(nbytes), 256)
        if self.buf is None or self.buf.numel() < nbytes:
            self.buf = torch.empty(nbytes, dtype=torch.uint8, device=self.device)
        assert self.buf.data_ptr() % 256 == 0
        return self.buf.data_ptr(), self.buf.numel()


_default_ws: dict[int, Workspace] = {}


def _ws(ws: Workspace | None, device) -> Workspace:
    if ws is not None:
        return ws
    idx = torch.device(device).index
    idx = torch.cuda.current_device() if idx is None else idx
    if idx not in _default_ws:
        _default_ws[idx] = Workspace(torch.device("cuda", idx))
    return _default_ws[idx]


# --------------------------------------------------------------------------- calls
def mosaic_version() -> int:
    return int(lib().mosaic_version())


def mosaic_act_norms(X: torch.Tensor, sumsq_accum: torch.Tensor, norms_out: torch.Tensor | None = None,
                     flags: int = 0, ws: Workspace | None = None, stream=None) -> None:
    """sumsq_accum[j] += sum_t X[t,j]^2 (fp64); optionally norms_out = sqrt (Eq. 5's norm term)."""
    xp, tokens, cols, ldx = _mat(X, "X")
    _dev(sumsq_accum, "sumsq_accum", torch.float64)
    if sumsq_accum.numel() != cols or (norms_out is not None and norms_out.numel() != cols):
        raise ValueError("sumsq_accum / norms_out must have one entry per column of X")
    if norms_out is not None:
        _dev(norms_out, "norms_out", torch.float32)
    L = lib()
    wp, wn = _ws(ws, X.device).get(L.mosaic_act_norms_workspace_bytes(tokens, cols))
    _check(L.mosaic_act_norms(xp, tokens, cols, ldx, _dtype_code(X), sumsq_accum.data_ptr(), _ptr(norms_out),
                              int(flags), wp, wn, _stream(stream)), "mosaic_act_norms")


def mosaic_gram_accumulate(X: torch.Tensor, G: torch.Tensor, flags: int = 0, status: torch.Tensor | None = None,
                           stream=None) -> None:
    """G[j,l] += sum_t X[t,j] X[t,l] (fp32, both triangles): the second moments of a projection's
    input, from which the inverse-Hessian back-end forms H = (2/T) G.  `status` (one int32 on the
    device) reads 1 after synchronisation if a bounded wait of the kernel ran out."""
    xp, tokens, cols, ldx = _mat(X, "X")
    _dev(G, "G", torch.float32)
    if G.dim() != 2 or tuple(G.shape) != (cols, cols) or G.stride(1) != 1:
        raise ValueError("G must be a [cols, cols] fp32 matrix with unit column stride")
    if status is not None:
        _dev(status, "status", torch.int32)
    _check(lib().mosaic_gram_accumulate(xp, tokens, cols, ldx, _dtype_code(X), G.data_ptr(), G.stride(0), int(flags),
                                        _ptr(status), _stream(stream)), "mosaic_gram_accumulate")


def mosaic_bounded_wait_selftest(budget_cycles: int, status: torch.Tensor, stream=None) -> None:
    """Diagnostic: the bounded mbarrier wait of the tensor-core kernel on its own, on a barrier that
    nothing completes.  `status` (one int32 on the device) reads 1 after synchronisation if the wait
    gave up after `budget_cycles` and raised the error word, as it must."""
    _dev(status, "status", torch.int32)
    _check(lib().mosaic_bounded_wait_selftest(int(budget_cycles), status.data_ptr(), _stream(stream)),
           "mosaic_bounded_wait_selftest")


def mosaic_score(W: torch.Tensor, norms: torch.Tensor, score_out: torch.Tensor, stream=None) -> None:
    """score_out[i,j] = norms[j] * |W[i,j]| in fp32 (Eq. 5, materialised)."""
    p, rows, cols, ldw = _mat(W, "W")
    _dev(norms, "norms", torch.float32)
    _dev(score_out, "score_out", torch.float32)
    if norms.numel() != cols or tuple(score_out.shape) != (rows, cols) or not score_out.is_contiguous():
        raise ValueError("norms must be [cols] and score_out a contiguous [rows, cols]")
    _check(lib().mosaic_score(p, rows, cols, ldw, _dtype_code(W), norms.data_ptr(), score_out.data_ptr(),
                              _stream(stream)), "mosaic_score")


def mosaic_outlier_ratio(W: torch.Tensor, norms: torch.Tensor, alpha: float, outlier_count_out: torch.Tensor,
                         score_sum_out: torch.Tensor | None = None, ws: Workspace | None = None, stream=None) -> None:
    """Eq. 6: outlier_count_out[0] = #{score > alpha*mean(score)}; score_sum_out[0] = fp64 sum of scores."""
    p, rows, cols, ldw = _mat(W, "W")
    _dev(norms, "norms", torch.float32)
    _dev(outlier_count_out, "outlier_count_out", torch.int64)
    if score_sum_out is not None:
        _dev(score_sum_out, "score_sum_out", torch.float64)
    if norms.numel() != cols:
        raise ValueError("norms must be [cols]")
    L = lib()
    wp, wn = _ws(ws, W.device).get(L.mosaic_outlier_ratio_workspace_bytes(rows, cols))
    _check(L.mosaic_outlier_ratio(p, rows, cols, ldw, _dtype_code(W), norms.data_ptr(), float(alpha),
                                  outlier_count_out.data_ptr(), _ptr(score_sum_out), wp, wn, _stream(stream)),
           "mosaic_outlier_ratio")


def mosaic_outlier_ratio_static(W: torch.Tensor, norms: torch.Tensor, alpha: float, outlier_count_out: torch.Tensor,
                                score_sum_out: torch.Tensor | None = None, stream=None) -> None:
    """mosaic_outlier_ratio for callers that cannot allocate device memory: no workspace is
    passed, the library uses the fixed scratch array it carries on the device.  Calls on one
    device share that array, so do not let two of them overlap on the GPU."""
    p, rows, cols, ldw = _mat(W, "W")
    _dev(norms, "norms", torch.float32)
    _dev(outlier_count_out, "outlier_count_out", torch.int64)
    if score_sum_out is not None:
        _dev(score_sum_out, "score_sum_out", torch.float64)
    if norms.numel() != cols:
        raise ValueError("norms must be [cols]")
    _check(lib().mosaic_outlier_ratio_static(p, rows, cols, ldw, _dtype_code(W), norms.data_ptr(), float(alpha),
                                             outlier_count_out.data_ptr(), _ptr(score_sum_out), _stream(stream)),
           "mosaic_outlier_ratio_static")


class OutlierJob(C.Structure):
    """mosaic_outlier_job of include/mosaic.h."""
    _fields_ = [("W", C.c_void_p), ("rows", C.c_int64), ("cols", C.c_int64), ("ldw", C.c_int64),
                ("norms", C.c_void_p), ("outlier_count_out", C.c_void_p), ("score_sum_out", C.c_void_p)]


class OutlierBatch:
    """The marshalled job list of mosaic_outlier_ratio_batch for a list of
    (W, norms, outlier_count_out[1], score_sum_out[1] or None); the count tensors may be
    one-element views of a larger int64 tensor.  Checked and laid out once; run() only makes
    the call, so a caller that repeats the sweep over matrices that stay where they are pays
    the per-job Python work once.  The tensors are kept alive by the object."""

    def __init__(self, jobs):
        self.jobs = list(jobs)
        if not self.jobs:
            raise ValueError("empty batch")
        self.arr = (OutlierJob * len(self.jobs))()
        dtype = self.jobs[0][0].dtype
        for i, (W, norms, cnt, ssum) in enumerate(self.jobs):
            p, rows, cols, ldw = _mat(W, "W")
            if W.dtype != dtype:
                raise TypeError("one dtype per batch")
            _dev(norms, "norms", torch.float32)
            _dev(cnt, "outlier_count_out", torch.int64)
            if ssum is not None:
                _dev(ssum, "score_sum_out", torch.float64)
            if norms.numel() != cols:
                raise ValueError("norms must be [cols]")
            self.arr[i] = OutlierJob(p, rows, cols, ldw, norms.data_ptr(), cnt.data_ptr(), _ptr(ssum))
        self.code = _dtype_code(self.jobs[0][0])
        self.device = self.jobs[0][0].device
        self.ws_bytes = lib().mosaic_outlier_ratio_batch_workspace_bytes(C.addressof(self.arr), len(self.jobs))

    def run(self, alpha: float, ws: Workspace | None = None, stream=None, group_of=None) -> None:
        """group_of: None (every matrix against its own mean, Eq. 6) or one group id per job - adjacent jobs
        with equal ids are counted against the mean over the whole group (Eq. 3-4, layer outlier distribution)."""
        wp, wn = _ws(ws, self.device).get(self.ws_bytes)
        if group_of is None:
            _check(lib().mosaic_outlier_ratio_batch(C.addressof(self.arr), len(self.jobs), self.code, float(alpha), wp, wn,
                                                    _stream(stream)), "mosaic_outlier_ratio_batch")
            return
        if len(group_of) != len(self.jobs):
            raise ValueError("one group id per job")
        g = (C.c_int32 * len(self.jobs))(*[int(v) for v in group_of])
        _check(lib().mosaic_outlier_ratio_grouped(C.addressof(self.arr), C.addressof(g), len(self.jobs), self.code, float(alpha),
                                                  wp, wn, _stream(stream)), "mosaic_outlier_ratio_grouped")


def mosaic_outlier_ratio_batch(jobs, alpha: float, ws: Workspace | None = None, stream=None) -> None:
    """mosaic_outlier_ratio over a list of (W, norms, outlier_count_out[1], score_sum_out[1] or None)
    in a handful of launches (bf16: one sweep over the weights); the count tensors may be one-element
    views of a larger int64 tensor."""
    if jobs:
        OutlierBatch(jobs).run(alpha, ws, stream)


def mosaic_outlier_ratio_grouped(jobs, group_of, alpha: float, ws: Workspace | None = None, stream=None) -> None:
    """Eq. 3-4: as mosaic_outlier_ratio_batch, with adjacent jobs of equal group id sharing one threshold."""
    if jobs:
        OutlierBatch(jobs).run(alpha, ws, stream, group_of=group_of)


def mosaic_ratio_from_count(outlier_count: int, numel: int) -> float:
    return float(lib().mosaic_ratio_from_count(int(outlier_count), int(numel)))


def mosaic_allocate_sparsity(outlier_counts, numels, cols, n_layers: int, n_proj: int, p: float,
                             lam: float = 0.08, mode: int = GLOBAL_NORM):
    """Host call: (sparsity[N*M] fp64, k[N*M] int64, infeasible flag) from the outlier counts."""
    n = n_layers * n_proj
    oc, ne, cl = (np.ascontiguousarray(v, dtype=np.int64) for v in (outlier_counts, numels, cols))
    if not (oc.shape == ne.shape == cl.shape == (n,)):
        raise ValueError("outlier_counts, numels and cols need one entry per projection")
    s, k = np.empty(n, dtype=np.float64), np.empty(n, dtype=np.int64)
    st = _check(lib().mosaic_allocate_sparsity(oc.ctypes.data, ne.ctypes.data, cl.ctypes.data, n_layers, n_proj,
                                               float(p), float(lam), int(mode), s.ctypes.data, k.ctypes.data),
                "mosaic_allocate_sparsity", allow=(ERR_INFEASIBLE,))
    return s.tolist(), k.tolist(), st == ERR_INFEASIBLE


def _out_ptr(W_in: torch.Tensor, W_out: torch.Tensor | None, rows: int, cols: int, ldw: int):
    """Pointer of the pruned-weights output, or None for mask-only mode."""
    if W_out is None:
        return None
    po, r2, c2, ld2 = _mat(W_out, "W_out")
    if (r2, c2) != (rows, cols) or W_out.dtype != W_in.dtype or (rows > 1 and ld2 != ldw):
        raise ValueError("W_out must match W_in in shape, dtype and leading dimension")
    return po


def mosaic_prune_unstructured(W_in: torch.Tensor, W_out: torch.Tensor | None, norms: torch.Tensor, k: int,
                              mask_out: torch.Tensor | None = None, ws: Workspace | None = None, stream=None) -> None:
    """Per row, zero the k entries first under (score asc, column asc); optional keep bitmask.
    W_out None: mask-only mode (mask_out is then the only output)."""
    p, rows, cols, ldw = _mat(W_in, "W_in")
    po = _out_ptr(W_in, W_out, rows, cols, ldw)
    if W_out is None and mask_out is None:
        raise ValueError("mask-only mode needs mask_out")
    _dev(norms, "norms", torch.float32)
    if norms.numel() != cols:
        raise ValueError("norms must be [cols]")
    if mask_out is not None:
        _dev(mask_out, "mask_out", torch.int32)
        if tuple(mask_out.shape) != (rows, (cols + 31) // 32) or not mask_out.is_contiguous():
            raise ValueError("mask_out must be a contiguous int32 [rows, ceil(cols/32)]")
    _check(lib().mosaic_prune_unstructured(p, po, rows, cols, ldw, _dtype_code(W_in), norms.data_ptr(), int(k),
                                           _ptr(mask_out), None, 0, _stream(stream)), "mosaic_prune_unstructured")


class PruneJob(C.Structure):
    """mosaic_prune_job of include/mosaic.h."""
    _fields_ = [("W_in", C.c_void_p), ("W_out", C.c_void_p), ("rows", C.c_int64), ("cols", C.c_int64),
                ("ldw", C.c_int64), ("norms", C.c_void_p), ("k", C.c_int64), ("mask_out", C.c_void_p)]


class PruneBatch:
    """The marshalled job list of mosaic_prune_unstructured_batch for a list of
    (W_in, W_out or None, norms, k, mask_out or None).  Checked and laid out once; run() may replace
    the per-row prune counts and then only makes the call.  The tensors are kept alive by the object."""

    def __init__(self, jobs):
        self.jobs = list(jobs)
        if not self.jobs:
            raise ValueError("empty batch")
        self.arr = (PruneJob * len(self.jobs))()
        dtype = self.jobs[0][0].dtype
        for i, (W_in, W_out, norms, k, mask_out) in enumerate(self.jobs):
            p, rows, cols, ldw = _mat(W_in, "W_in")
            po = _out_ptr(W_in, W_out, rows, cols, ldw)
            if W_in.dtype != dtype:
                raise TypeError("one dtype per batch")
            if W_out is None and mask_out is None:
                raise ValueError("mask-only mode needs mask_out")
            _dev(norms, "norms", torch.float32)
            if norms.numel() != cols:
                raise ValueError("norms must be [cols]")
            if mask_out is not None:
                _dev(mask_out, "mask_out", torch.int32)
                if tuple(mask_out.shape) != (rows, (cols + 31) // 32) or not mask_out.is_contiguous():
                    raise ValueError("mask_out must be a contiguous int32 [rows, ceil(cols/32)]")
            self.arr[i] = PruneJob(p, po, rows, cols, ldw, norms.data_ptr(), int(k), _ptr(mask_out))
        self.code = _dtype_code(self.jobs[0][0])
        self.device = self.jobs[0][0].device
        self.ws_bytes = lib().mosaic_prune_unstructured_batch_workspace_bytes(C.addressof(self.arr), len(self.jobs), self.code)

    def run(self, k=None, ws: Workspace | None = None, stream=None) -> None:
        """k: None (the counts given at construction) or one prune count per job."""
        if k is not None:
            if len(k) != len(self.jobs):
                raise ValueError("one k per job")
            # (the k fields of all jobs in one strided write: a job is 8 words, k the seventh)
            np.frombuffer(self.arr, dtype=np.int64).reshape(len(self.jobs), 8)[:, 6] = np.asarray(k, dtype=np.int64)
            self.ws_bytes = lib().mosaic_prune_unstructured_batch_workspace_bytes(C.addressof(self.arr), len(self.jobs), self.code)
        wp, wn = _ws(ws, self.device).get(self.ws_bytes)
        _check(lib().mosaic_prune_unstructured_batch(C.addressof(self.arr), len(self.jobs), self.code, wp, wn, _stream(stream)),
               "mosaic_prune_unstructured_batch")


def mosaic_prune_unstructured_batch(jobs, ws: Workspace | None = None, stream=None) -> None:
    """mosaic_prune_unstructured over a list of (W_in, W_out, norms, k, mask_out or None) in few launches."""
    if jobs:
        PruneBatch(jobs).run(None, ws, stream)


def mosaic_prune_structured_compact(W_in: torch.Tensor, norms: torch.Tensor | None, row_group: int, col_group: int,
                                    row_units_keep: int, col_units_keep: int, row_keep_units: torch.Tensor | None,
                                    col_keep_units: torch.Tensor | None, flags: int = 0,
                                    W_out: torch.Tensor | None = None, unit_scores_out: torch.Tensor | None = None,
                                    ws: Workspace | None = None, stream=None) -> None:
    """Unit scores -> ranked keep lists -> dense compacted W_out (see include/mosaic.h)."""
    p, rows, cols, ldw = _mat(W_in, "W_in")
    if norms is not None:
        _dev(norms, "norms", torch.float32)
    for t, nm, n in ((row_keep_units, "row_keep_units", row_units_keep), (col_keep_units, "col_keep_units", col_units_keep)):
        if t is not None:
            _dev(t, nm, torch.int32)
            if t.numel() < n:
                raise ValueError(f"{nm} is shorter than the number of kept units")
    if W_out is not None:
        _dev(W_out, "W_out", W_in.dtype)
        if not W_out.is_contiguous() or W_out.numel() < row_units_keep * row_group * col_units_keep * col_group:
            raise ValueError("W_out must be contiguous and hold the compacted matrix")
    if unit_scores_out is not None:
        _dev(unit_scores_out, "unit_scores_out", torch.float32)
        if unit_scores_out.numel() < rows // row_group + cols // col_group:
            raise ValueError("unit_scores_out too short")
    L = lib()
    wp, wn = _ws(ws, W_in.device).get(L.mosaic_prune_structured_compact_workspace_bytes(rows, cols))
    _check(L.mosaic_prune_structured_compact(p, rows, cols, ldw, _dtype_code(W_in), _ptr(norms), int(row_group),
                                             int(col_group), int(row_units_keep), int(col_units_keep),
                                             _ptr(row_keep_units), _ptr(col_keep_units), int(flags), _ptr(W_out),
                                             _ptr(unit_scores_out), wp, wn, _stream(stream)),
           "mosaic_prune_structured_compact")


def mosaic_rank_units(scores: torch.Tensor, keep: int, keep_out: torch.Tensor, stream=None) -> None:
    """Ascending indices of the `keep` units that survive removal of the lowest-scored ones."""
    _dev(scores, "scores", torch.float32)
    _dev(keep_out, "keep_out", torch.int32)
    if keep_out.numel() < keep:
        raise ValueError("keep_out too short")
    _check(lib().mosaic_rank_units(scores.data_ptr(), scores.numel(), int(keep), keep_out.data_ptr(), _stream(stream)),
           "mosaic_rank_units")


def mosaic_sum_unit_scores(dst: torch.Tensor, src: torch.Tensor, stream=None) -> None:
    """dst[u] += src[u] in fp32: running total of the unit scores of coupled projections."""
    _dev(dst, "dst", torch.float32)
    _dev(src, "src", torch.float32)
    if dst.numel() != src.numel() or not dst.is_contiguous() or not src.is_contiguous():
        raise ValueError("dst and src must be contiguous and of equal length")
    _check(lib().mosaic_sum_unit_scores(dst.data_ptr(), src.data_ptr(), dst.numel(), _stream(stream)),
           "mosaic_sum_unit_scores")


# --------------------------------------------------------------------------- batched structured steps
class UnitScoreJob(C.Structure):
    """mosaic_unit_score_job of include/mosaic.h."""
    _fields_ = [("W", C.c_void_p), ("rows", C.c_int64), ("cols", C.c_int64), ("ldw", C.c_int64), ("norms", C.c_void_p),
                ("row_group", C.c_int64), ("col_group", C.c_int64), ("row_scores_out", C.c_void_p),
                ("col_scores_out", C.c_void_p)]


class AddJob(C.Structure):
    """mosaic_add_job of include/mosaic.h."""
    _fields_ = [("dst", C.c_void_p), ("a", C.c_void_p), ("b", C.c_void_p), ("n", C.c_int64)]


class RankJob(C.Structure):
    """mosaic_rank_job of include/mosaic.h."""
    _fields_ = [("scores", C.c_void_p), ("n_units", C.c_int64), ("keep", C.c_int64), ("keep_out", C.c_void_p)]


class CompactJob(C.Structure):
    """mosaic_compact_job of include/mosaic.h."""
    _fields_ = [("W_in", C.c_void_p), ("rows", C.c_int64), ("cols", C.c_int64), ("ldw", C.c_int64),
                ("row_keep_units", C.c_void_p), ("row_units_keep", C.c_int64), ("row_group", C.c_int64),
                ("col_keep_units", C.c_void_p), ("col_units_keep", C.c_int64), ("col_group", C.c_int64),
                ("W_out", C.c_void_p)]


class UnitScoreBatch:
    """The marshalled job list of mosaic_unit_scores_batch for a list of (W, norms or None, row_group,
    col_group, row_scores_out or None, col_scores_out or None).  Checked and laid out once; run() only
    makes the call.  The tensors are kept alive by the object."""

    def __init__(self, jobs):
        self.jobs = list(jobs)
        if not self.jobs:
            raise ValueError("empty batch")
        self.arr = (UnitScoreJob * len(self.jobs))()
        dtype = self.jobs[0][0].dtype
        for i, (W, norms, rg, cg, rs, cs) in enumerate(self.jobs):
            p, rows, cols, ldw = _mat(W, "W")
            if W.dtype != dtype:
                raise TypeError("one dtype per batch")
            if norms is not None:
                _dev(norms, "norms", torch.float32)
            for t, nm, n in ((rs, "row_scores_out", rows // rg), (cs, "col_scores_out", cols // cg)):
                if t is not None:
                    _dev(t, nm, torch.float32)
                    if t.numel() < n or not t.is_contiguous():
                        raise ValueError(f"{nm} must be contiguous with one entry per unit")
            self.arr[i] = UnitScoreJob(p, rows, cols, ldw, _ptr(norms), int(rg), int(cg), _ptr(rs), _ptr(cs))
        self.code = _dtype_code(self.jobs[0][0])
        self.device = self.jobs[0][0].device
        self.ws_bytes = lib().mosaic_unit_scores_batch_workspace_bytes(C.addressof(self.arr), len(self.jobs))

    def run(self, ws: Workspace | None = None, stream=None) -> None:
        wp, wn = _ws(ws, self.device).get(self.ws_bytes)
        _check(lib().mosaic_unit_scores_batch(C.addressof(self.arr), len(self.jobs), self.code, wp, wn, _stream(stream)),
               "mosaic_unit_scores_batch")


class AddBatch:
    """The marshalled list of mosaic_add_unit_scores_batch for (dst, a, b) fp32 vectors of equal length."""

    def __init__(self, jobs):
        self.jobs = list(jobs)
        if not self.jobs:
            raise ValueError("empty batch")
        self.arr = (AddJob * len(self.jobs))()
        for i, (dst, a, b) in enumerate(self.jobs):
            for t, nm in ((dst, "dst"), (a, "a"), (b, "b")):
                _dev(t, nm, torch.float32)
                if not t.is_contiguous() or t.numel() != dst.numel():
                    raise ValueError("dst, a and b must be contiguous and of equal length")
            self.arr[i] = AddJob(dst.data_ptr(), a.data_ptr(), b.data_ptr(), dst.numel())

    def run(self, stream=None) -> None:
        _check(lib().mosaic_add_unit_scores_batch(C.addressof(self.arr), len(self.jobs), _stream(stream)),
               "mosaic_add_unit_scores_batch")


class RankBatch:
    """The marshalled list of mosaic_rank_units_batch for (scores, keep, keep_out)."""

    def __init__(self, jobs):
        self.jobs = list(jobs)
        if not self.jobs:
            raise ValueError("empty batch")
        self.arr = (RankJob * len(self.jobs))()
        for i, (scores, keep, keep_out) in enumerate(self.jobs):
            _dev(scores, "scores", torch.float32)
            _dev(keep_out, "keep_out", torch.int32)
            if keep_out.numel() < keep or not scores.is_contiguous():
                raise ValueError("keep_out too short or scores not contiguous")
            self.arr[i] = RankJob(scores.data_ptr(), scores.numel(), int(keep), keep_out.data_ptr())

    def run(self, stream=None) -> None:
        _check(lib().mosaic_rank_units_batch(C.addressof(self.arr), len(self.jobs), _stream(stream)), "mosaic_rank_units_batch")


class CompactBatch:
    """The marshalled list of mosaic_compact_batch for (W_in, row_keep_units, row_units_keep, row_group,
    col_keep_units, col_units_keep, col_group, W_out)."""

    def __init__(self, jobs):
        self.jobs = list(jobs)
        if not self.jobs:
            raise ValueError("empty batch")
        self.arr = (CompactJob * len(self.jobs))()
        dtype = self.jobs[0][0].dtype
        for i, (W_in, rk, n_rk, rg, ck, n_ck, cg, W_out) in enumerate(self.jobs):
            p, rows, cols, ldw = _mat(W_in, "W_in")
            if W_in.dtype != dtype:
                raise TypeError("one dtype per batch")
            _dev(rk, "row_keep_units", torch.int32)
            _dev(ck, "col_keep_units", torch.int32)
            _dev(W_out, "W_out", W_in.dtype)
            if rk.numel() < n_rk or ck.numel() < n_ck:
                raise ValueError("keep list shorter than the number of kept units")
            if not W_out.is_contiguous() or W_out.numel() < n_rk * rg * n_ck * cg:
                raise ValueError("W_out must be contiguous and hold the compacted matrix")
            self.arr[i] = CompactJob(p, rows, cols, ldw, rk.data_ptr(), int(n_rk), int(rg), ck.data_ptr(), int(n_ck), int(cg),
                                     W_out.data_ptr())
        self.code = _dtype_code(self.jobs[0][0])

    def run(self, stream=None) -> None:
        _check(lib().mosaic_compact_batch(C.addressof(self.arr), len(self.jobs), self.code, _stream(stream)),
               "mosaic_compact_batch")


def mosaic_unit_scores_batch(jobs, ws: Workspace | None = None, stream=None) -> None:
    """Unit scores of a list of (W, norms or None, row_group, col_group, row_scores_out or None,
    col_scores_out or None) in two launches."""
    if jobs:
        UnitScoreBatch(jobs).run(ws, stream)


def mosaic_add_unit_scores_batch(jobs, stream=None) -> None:
    """dst[u] = fl32(a[u] + b[u]) for a list of (dst, a, b): fp32 vectors of equal length."""
    if jobs:
        AddBatch(jobs).run(stream)


def mosaic_rank_units_batch(jobs, stream=None) -> None:
    """mosaic_rank_units for a list of (scores, keep, keep_out) in one launch."""
    if jobs:
        RankBatch(jobs).run(stream)


def mosaic_compact_batch(jobs, stream=None) -> None:
    """Dense compaction of a list of (W_in, row_keep_units, row_units_keep, row_group, col_keep_units,
    col_units_keep, col_group, W_out) in one launch."""
    if jobs:
        CompactBatch(jobs).run(stream)
