"""TEST INFRASTRUCTURE - not part of the product.

ctypes front end of ``mosaic_oracle.c``, the plain CPU statement of Mosaic's
pruning hot path (Eq. 5, Eq. 6, Algorithm 1, Section 3.3 components 4-9).
Only the tests, the smoke check and the benchmark's CPU-baseline leg may
import this module; the CUDA library and its Python binding never do.

Arrays are numpy.  A bf16 matrix is passed as a ``uint16`` array holding the
raw bit patterns together with ``dtype="bf16"``; an fp32 matrix as ``float32``.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "mosaic_oracle.c")
_SO = os.path.join(_HERE, "libmosaic_oracle.so")

F32, BF16 = 0, 1
MODE_GLOBAL_NORM, MODE_PER_CATEGORY_NORM = 0, 1
MODE_WEIGHTED_MEAN = 2      # flag, or-ed into the mode
MODE_REDISTRIBUTE = 4       # flag, or-ed into the mode: clamp and redistribute


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (strict IEEE flags) if it is missing or stale."""
    if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-std=c11", "-ffp-contract=off", "-fno-fast-math", "-fopenmp",
               "-shared", "-fPIC", "-o", _SO, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _SO


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.oracle_norm_certify.restype = C.c_int64
        _lib.oracle_unit_scores_certify.restype = C.c_int64
        _lib.oracle_allocate_sparsity.restype = C.c_int
        _lib.oracle_num_threads.restype = C.c_int
    return _lib


def _code(a: np.ndarray, dtype: str | None) -> int:
    if dtype in ("bf16", BF16):
        assert a.dtype == np.uint16, "bf16 data is passed as raw uint16 bit patterns"
        return BF16
    assert a.dtype == np.float32
    return F32


def _p(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _i64(v):
    return C.c_int64(int(v))


def _ld(a: np.ndarray) -> int:
    assert a.ndim == 2 and a.strides[1] == a.itemsize
    return a.strides[0] // a.itemsize


def num_threads() -> int:
    return int(lib().oracle_num_threads())


def set_num_threads(n: int) -> None:
    """Threads of the oracle's parallel loops (for timing; results never depend on it)."""
    lib().oracle_set_num_threads(C.c_int(int(n)))


def act_sumsq(X: np.ndarray, sumsq: np.ndarray | None = None, dtype=None) -> np.ndarray:
    """sumsq[j] += sum_t X[t,j]^2 in fp64, t in order (the norm term of Eq. 5)."""
    code = _code(X, dtype)
    T, cols = X.shape
    if sumsq is None:
        sumsq = np.zeros(cols, np.float64)
    assert sumsq.dtype == np.float64 and sumsq.shape == (cols,)
    lib().oracle_act_sumsq(_p(X), _i64(T), _i64(cols), _i64(_ld(X)), code, _p(sumsq))
    return sumsq


def norm_finalize(sumsq: np.ndarray) -> np.ndarray:
    out = np.empty(sumsq.shape[0], np.float32)
    lib().oracle_norm_finalize(_p(sumsq), _i64(sumsq.shape[0]), _p(out))
    return out


def act_norms(X: np.ndarray, dtype=None) -> np.ndarray:
    return norm_finalize(act_sumsq(X, None, dtype))


def norm_certify(X: np.ndarray, dtype=None) -> np.ndarray:
    """Per column: True if no fp64 summation order can change the fp32 norm."""
    code = _code(X, dtype)
    T, cols = X.shape
    ok = np.zeros(cols, np.uint8)
    lib().oracle_norm_certify(_p(X), _i64(T), _i64(cols), _i64(_ld(X)), code, _p(ok))
    return ok.astype(bool)


def score(W: np.ndarray, norms: np.ndarray, dtype=None) -> np.ndarray:
    """Eq. 5 materialised: fp32 [rows, cols]."""
    code = _code(W, dtype)
    rows, cols = W.shape
    norms = np.ascontiguousarray(norms, np.float32)
    out = np.empty((rows, cols), np.float32)
    lib().oracle_score(_p(W), _i64(rows), _i64(cols), _i64(_ld(W)), code, _p(norms), _p(out))
    return out


def outlier_ratio(W: np.ndarray, norms: np.ndarray, alpha: float = 5.0, dtype=None) -> dict:
    """Eq. 6 / Algorithm 1's count and rank steps: outlier count O, fp64 score sum, R = 100*O/C."""
    code = _code(W, dtype)
    rows, cols = W.shape
    norms = np.ascontiguousarray(norms, np.float32)
    O = C.c_int64(0)
    s = C.c_double(0.0)
    r = C.c_double(0.0)
    cert = C.c_int(0)
    lib().oracle_outlier_ratio(_p(W), _i64(rows), _i64(cols), _i64(_ld(W)), code, _p(norms),
                               C.c_float(alpha), C.byref(O), C.byref(s), C.byref(r), C.byref(cert))
    return {"count": int(O.value), "sum": float(s.value), "ratio": float(r.value),
            "certified": bool(cert.value), "numel": rows * cols}


def outlier_ratio_group(Ws, norms, alpha: float = 5.0, dtype=None) -> dict:
    """Eq. 3-4 (layer outlier distribution): one threshold alpha * mean over all matrices of the
    group; per-matrix counts, their total, the fp64 score sum and R = 100*O/C of the group."""
    n = len(Ws)
    code = _code(Ws[0], dtype)
    for W in Ws:
        assert _code(W, dtype) == code
    norms = [np.ascontiguousarray(x, np.float32) for x in norms]
    PW = (C.c_void_p * n)(*[W.ctypes.data for W in Ws])
    PN = (C.c_void_p * n)(*[x.ctypes.data for x in norms])
    I64 = C.c_int64 * n
    rows, cols, lds = I64(*[W.shape[0] for W in Ws]), I64(*[W.shape[1] for W in Ws]), I64(*[_ld(W) for W in Ws])
    counts = I64()
    s, r, cert = C.c_double(0.0), C.c_double(0.0), C.c_int(0)
    lib().oracle_outlier_ratio_group(PW, rows, cols, lds, code, PN, C.c_int(n), C.c_float(alpha), counts, C.byref(s),
                                     C.byref(r), C.byref(cert))
    return {"counts": [int(v) for v in counts], "count": int(sum(counts)), "sum": float(s.value), "ratio": float(r.value),
            "certified": bool(cert.value), "numel": int(sum(W.size for W in Ws))}


def allocate_sparsity(outlier_counts, numels, cols, n_layers: int, n_proj: int, p: float,
                      lam: float = 0.08, mode: int = MODE_GLOBAL_NORM):
    """normalize(R_LLM) + Projection Planner.  Returns (sparsity[N*M], k[N*M], clamped)."""
    oc = np.ascontiguousarray(outlier_counts, np.int64)
    ne = np.ascontiguousarray(numels, np.int64)
    cl = np.ascontiguousarray(cols, np.int64)
    n = n_layers * n_proj
    assert oc.shape == ne.shape == cl.shape == (n,)
    s = np.empty(n, np.float64)
    k = np.empty(n, np.int64)
    clamped = lib().oracle_allocate_sparsity(_p(oc), _p(ne), _p(cl), C.c_int(n_layers),
                                             C.c_int(n_proj), C.c_double(p), C.c_double(lam),
                                             C.c_int(mode), _p(s), _p(k))
    return s, k, bool(clamped)


def prune_unstructured(W: np.ndarray, norms: np.ndarray, k: int, dtype=None):
    """Per row, zero the k entries first under (score asc, column asc).  Returns (W', mask)."""
    code = _code(W, dtype)
    rows, cols = W.shape
    norms = np.ascontiguousarray(norms, np.float32)
    W = np.ascontiguousarray(W)
    out = np.empty_like(W)
    mask = np.empty((rows, (cols + 31) // 32), np.uint32)
    lib().oracle_prune_unstructured(_p(W), _p(out), _i64(rows), _i64(cols), _i64(_ld(W)), code,
                                    _p(norms), _i64(k), _p(mask))
    return out, mask


def unit_scores(W: np.ndarray, norms, row_group: int = 1, col_group: int = 1, dtype=None):
    """fp32 scores of row units and column units (sum of Eq. 5 over the unit)."""
    code = _code(W, dtype)
    rows, cols = W.shape
    assert rows % row_group == 0 and cols % col_group == 0
    if norms is not None:
        norms = np.ascontiguousarray(norms, np.float32)
    rs = np.empty(rows // row_group, np.float32)
    cs = np.empty(cols // col_group, np.float32)
    lib().oracle_unit_scores(_p(W), _i64(rows), _i64(cols), _i64(_ld(W)), code, _p(norms),
                             _i64(row_group), _i64(col_group), _p(rs), _p(cs))
    return rs, cs


def unit_scores_certify(W: np.ndarray, norms, row_group: int = 1, col_group: int = 1, dtype=None):
    """Per row unit and per column unit: True if no fp64 summation order can change the fp32 score."""
    code = _code(W, dtype)
    rows, cols = W.shape
    assert rows % row_group == 0 and cols % col_group == 0
    if norms is not None:
        norms = np.ascontiguousarray(norms, np.float32)
    r_ok = np.zeros(rows // row_group, np.uint8)
    c_ok = np.zeros(cols // col_group, np.uint8)
    lib().oracle_unit_scores_certify(_p(W), _i64(rows), _i64(cols), _i64(_ld(W)), code, _p(norms),
                                     _i64(row_group), _i64(col_group), _p(r_ok), _p(c_ok))
    return r_ok.astype(bool), c_ok.astype(bool)


def gram(X: np.ndarray, G: np.ndarray | None = None, dtype=None, with_abs: bool = False):
    """G[j,l] += sum_t X[t,j] X[t,l] in fp64, t in order (second moments of a projection's input;
    the back-end's layer Hessian is 2/T times it).  with_abs: also sum_t |X[t,j]| |X[t,l]|."""
    code = _code(X, dtype)
    tokens, cols = X.shape
    G = np.zeros((cols, cols), dtype=np.float64) if G is None else G
    assert G.dtype == np.float64 and G.shape == (cols, cols) and G.flags.c_contiguous
    Ga = np.zeros((cols, cols), dtype=np.float64) if with_abs else None
    lib().oracle_gram(_p(X), _i64(tokens), _i64(cols), _i64(_ld(X)), code, _p(G), _p(Ga) if with_abs else None)
    return (G, Ga) if with_abs else G


def gram_pairs(X: np.ndarray, js, ls, dtype=None):
    """(sum_t X[t,j] X[t,l], sum_t |X[t,j]| |X[t,l]|) for the listed (j, l) pairs, fp64."""
    code = _code(X, dtype)
    js = np.ascontiguousarray(js, dtype=np.int64)
    ls = np.ascontiguousarray(ls, dtype=np.int64)
    assert js.shape == ls.shape and js.ndim == 1
    out = np.zeros(js.shape[0], dtype=np.float64)
    out_abs = np.zeros(js.shape[0], dtype=np.float64)
    lib().oracle_gram_pairs(_p(X), _i64(X.shape[0]), _i64(_ld(X)), code, _i64(js.shape[0]), _p(js), _p(ls), _p(out), _p(out_abs))
    return out, out_abs


def hessian(X: np.ndarray, dtype=None) -> np.ndarray:
    """Layer Hessian of the inverse-Hessian back-end: (2 / T) * sum_t x_t x_t^T, fp64."""
    return gram(X, None, dtype) * (2.0 / X.shape[0])


def rank_units(scores: np.ndarray, keep: int) -> np.ndarray:
    """Ascending list of the `keep` units that survive removal of the lowest-scored ones."""
    scores = np.ascontiguousarray(scores, np.float32)
    out = np.empty(keep, np.int32)
    lib().oracle_rank_units(_p(scores), _i64(scores.shape[0]), _i64(keep), _p(out))
    return out


def compact(W: np.ndarray, row_keep, col_keep, row_group: int = 1, col_group: int = 1, dtype=None):
    """Dense gather of the kept row units x kept column units, bit for bit."""
    code = _code(W, dtype)
    rk = np.ascontiguousarray(row_keep, np.int32)
    ck = np.ascontiguousarray(col_keep, np.int32)
    out = np.empty((rk.shape[0] * row_group, ck.shape[0] * col_group), W.dtype)
    lib().oracle_compact(_p(W), _i64(_ld(W)), code, _p(rk), _i64(rk.shape[0]), _i64(row_group),
                         _p(ck), _i64(ck.shape[0]), _i64(col_group), _p(out))
    return out
