"""CPU pins of the oracle: every oracle function is checked against something
other than itself - exact rational brute force on tiny inputs, closed forms,
invariants the paper states, and special cases that reduce to a library
routine.  No GPU, no CUDA library.
"""
from fractions import Fraction
import math

import numpy as np
import pytest
import torch

import oracle
from paper_2504_06323_b200 import workloads as wl


# ----------------------------------------------------------------- helpers
def bf16_bits(a: np.ndarray) -> np.ndarray:
    """float32 array -> bf16 bit patterns (RN-even), via torch's conversion."""
    return wl.to_numpy(torch.from_numpy(np.ascontiguousarray(a, np.float32)).to(torch.bfloat16))


def bf16_value(bits: np.ndarray) -> np.ndarray:
    return (bits.astype(np.uint32) << 16).view(np.float32)


def as_f32(W, dtype):
    return bf16_value(W) if dtype == "bf16" else W


def exact_score(norm, w) -> np.float32:
    """Eq. 5 for one element from exact rational arithmetic: the product of two
    fp32 values has <= 48 significant bits, so it is exact in a double, and the
    single conversion to fp32 is the one RN rounding the definition allows."""
    prod = Fraction(float(norm)) * abs(Fraction(float(w)))
    d = float(prod)
    assert Fraction(d) == prod
    return np.float32(d)


def rand_matrix(rng, rows, cols, dtype):
    W = (rng.standard_normal((rows, cols)) * 0.02).astype(np.float32)
    return bf16_bits(W) if dtype == "bf16" else W


DTYPES = ["f32", "bf16"]


# ----------------------------------------------------------------- norms
@pytest.mark.parametrize("dtype", DTYPES)
def test_norms_closed_forms(dtype):
    T, cols = 96, 7
    X = np.zeros((T, cols), np.float32)
    X[:, 0] = 3.0                     # constant column: |c| * sqrt(T)
    X[:, 1] = -0.5
    X[17, 2] = -2.5                   # one-hot column: |x|
    X[:, 3] = 0.0                     # zero column
    X[::2, 4] = 1.0                   # T/2 ones: sqrt(T/2)
    X[:, 5] = np.where(np.arange(T) % 2 == 0, 4.0, -4.0)  # sign must not matter
    X[0, 6], X[1, 6] = 3.0, 4.0       # 3-4-5
    Xd = bf16_bits(X) if dtype == "bf16" else X
    n = oracle.act_norms(Xd, dtype)
    want = [3.0 * math.sqrt(T), 0.5 * math.sqrt(T), 2.5, 0.0, math.sqrt(T / 2), 4.0 * math.sqrt(T), 5.0]
    assert n.dtype == np.float32
    np.testing.assert_array_equal(n, np.array(want, np.float64).astype(np.float32))


@pytest.mark.parametrize("dtype", DTYPES)
def test_norms_exact_rational(dtype):
    rng = np.random.default_rng(1)
    T, cols = 53, 9                   # non-square: a transposed reduction would fail
    X = rng.standard_normal((T, cols)).astype(np.float32) * np.float32(3.0)
    Xd = bf16_bits(X) if dtype == "bf16" else X
    Xv = as_f32(Xd, dtype)
    ss = oracle.act_sumsq(Xd, None, dtype)
    n = oracle.norm_finalize(ss)
    for j in range(cols):
        exact = sum(Fraction(float(x)) ** 2 for x in Xv[:, j])
        assert abs(Fraction(float(ss[j])) - exact) <= exact * Fraction(T, 2 ** 52)
        # correctly rounded sqrt of the exact sum, then one rounding to fp32
        root = math.sqrt(float(exact))
        assert abs(float(n[j]) - root) <= abs(root) * 2.0 ** -23
        assert n[j] == np.float32(math.sqrt(ss[j]))


def test_norms_accumulate_in_chunks_and_ld():
    rng = np.random.default_rng(2)
    T, cols, ld = 40, 12, 16
    buf = rng.standard_normal((T, ld)).astype(np.float32)
    X = buf[:, :cols]                 # strided view: ld != cols
    whole = oracle.act_sumsq(np.ascontiguousarray(X))
    acc = np.zeros(cols)
    oracle.act_sumsq(X[:13], acc)
    oracle.act_sumsq(X[13:], acc)
    np.testing.assert_array_equal(acc, whole)      # sequential in t: chunking cannot change it
    np.testing.assert_allclose(whole, (X.astype(np.float64) ** 2).sum(0), rtol=1e-14)


def test_norm_certify_flags_a_rounding_boundary():
    # S = 1 + 2^-23 + 2^-48 = (1 + 2^-24)^2 exactly, so sqrt(S) sits exactly half way
    # between the fp32 neighbours 1 and 1 + 2^-23: any perturbation of S flips the
    # rounding, and the column must not be certified.  The benign columns must be.
    X = np.zeros((4, 3), np.float32)
    X[:, 0] = [1.0, 2.0 ** -12, 2.0 ** -12, 2.0 ** -24]
    X[:, 1] = [3.0, 4.0, 0.0, 0.0]
    X[:, 2] = 1.0
    ok = oracle.norm_certify(X)
    assert list(ok) == [False, True, True]
    assert oracle.act_norms(X)[0] == np.float32(1.0)          # the tie rounds to even


# ----------------------------------------------------------------- score
@pytest.mark.parametrize("dtype", DTYPES)
def test_score_special_cases_and_exact(dtype):
    rng = np.random.default_rng(3)
    rows, cols = 5, 11
    W = rand_matrix(rng, rows, cols, dtype)
    Wv = as_f32(W, dtype)
    ones = np.ones(cols, np.float32)
    np.testing.assert_array_equal(oracle.score(W, ones, dtype), np.abs(Wv))       # norm = 1 -> |W|
    norms = (rng.random(cols).astype(np.float32) + np.float32(0.5)) * np.float32(30)
    pm = np.where(rng.random((rows, cols)) < 0.5, -1.0, 1.0).astype(np.float32)
    pm_d = bf16_bits(pm) if dtype == "bf16" else pm
    np.testing.assert_array_equal(oracle.score(pm_d, norms, dtype),               # W = +-1 -> norm
                                  np.broadcast_to(norms, (rows, cols)))
    S = oracle.score(W, norms, dtype)
    for i in range(rows):
        for j in range(cols):
            assert S[i, j] == exact_score(norms[j], Wv[i, j])   # norm indexed by COLUMN


# ----------------------------------------------------------------- outlier ratio
def brute_outliers(Wv, norms, alpha):
    rows, cols = Wv.shape
    sc = [[Fraction(float(exact_score(norms[j], Wv[i, j]))) for j in range(cols)] for i in range(rows)]
    total = sum(sum(r) for r in sc)
    tau = Fraction(float(np.float32(alpha))) * total / (rows * cols)
    return sum(1 for r in sc for s in r if s > tau), total


@pytest.mark.parametrize("dtype", DTYPES)
@pytest.mark.parametrize("alpha", [1.0, 2.5, 5.0])
def test_outlier_count_vs_exact_enumeration(dtype, alpha):
    rng = np.random.default_rng(4)
    for rows, cols in [(16, 32), (7, 13), (1, 5)]:
        W = rand_matrix(rng, rows, cols, dtype)
        W_f = as_f32(W, dtype).copy()
        W_f[rng.random((rows, cols)) < 0.05] *= 40          # plant some outliers
        W = bf16_bits(W_f) if dtype == "bf16" else W_f
        norms = (rng.random(cols).astype(np.float32) + np.float32(0.1)) * np.float32(20)
        O, total = brute_outliers(as_f32(W, dtype), norms, alpha)
        r = oracle.outlier_ratio(W, norms, alpha, dtype)
        assert r["count"] == O
        assert abs(Fraction(r["sum"]) - total) <= total * Fraction(rows * cols, 2 ** 52)
        assert r["ratio"] == 100.0 * O / (rows * cols)
        assert r["numel"] == rows * cols


@pytest.mark.parametrize("dtype", DTYPES)
def test_outlier_planted_closed_form(dtype):
    # score = 1 everywhere except m entries equal to v:  mean = (C - m + m v)/C,
    # O = m exactly when 1 <= alpha*mean < v;  O = 0 when alpha*mean >= v.
    rows, cols, m, v = 8, 64, 5, 64.0
    W = np.ones((rows, cols), np.float32)
    flat = W.reshape(-1)
    flat[[3, 77, 200, 301, 511]] = -v            # sign must not matter
    Wd = bf16_bits(W) if dtype == "bf16" else W
    ones = np.ones(cols, np.float32)
    C = rows * cols
    mean = (C - m + m * v) / C
    r = oracle.outlier_ratio(Wd, ones, 5.0, dtype)
    assert 1.0 <= 5.0 * mean < v
    assert r["count"] == m and r["sum"] == C - m + m * v and r["certified"]
    r = oracle.outlier_ratio(Wd, ones, 50.0, dtype)          # threshold above v
    assert 50.0 * mean >= v and r["count"] == 0
    r = oracle.outlier_ratio(Wd, ones, 0.5, dtype)           # threshold below 1: everything
    assert 0.5 * mean < 1.0 and r["count"] == C
    # constant matrix: score == mean everywhere, strict '>' with alpha = 1 gives none
    Wc = np.full((rows, cols), 0.25, np.float32)
    Wc = bf16_bits(Wc) if dtype == "bf16" else Wc
    assert oracle.outlier_ratio(Wc, ones, 1.0, dtype)["count"] == 0


def test_outlier_certified_flags_a_score_on_or_next_to_the_threshold():
    # four scores (1, 1, 1, x), alpha = 2: tau = (3 + x) / 2.
    # x = 3 sits exactly on tau: not an outlier (strict), but any downward move of tau makes it
    # one, so the count must NOT be certified.  x = the next fp32 above 3 clears tau by 2^-23,
    # far more than the admissible C*2^-52: certified, one outlier.
    ones = np.ones(4, np.float32)
    r = oracle.outlier_ratio(np.array([[1, 1, 1, 3]], np.float32), ones, 2.0)
    assert r["count"] == 0 and not r["certified"]
    x = np.nextafter(np.float32(3), np.float32(4))
    r = oracle.outlier_ratio(np.array([[1, 1, 1, x]], np.float32), ones, 2.0)
    assert r["count"] == 1 and r["certified"]


@pytest.mark.parametrize("log2_t,certified", [(-13, False), (-10, True)])
def test_outlier_certified_margin_is_numel_times_2_pow_minus_52(log2_t, certified):
    # C = 2^20 scores: all 1 except one 2 and one t = 2^log2_t, alpha = 2, so the sum C + t is
    # exact in fp64 and tau = 2 (1 + t/C) lies t/C above the score 2 (relative).  The stated
    # margin is C * 2^-52 = 2^-32: t/C = 2^-33 is inside it (not certified - a margin four times
    # smaller would certify wrongly), t/C = 2^-30 is outside (certified - a margin four times
    # larger would refuse wrongly).  Either way 2 is not above tau: no outliers.
    n = 1024
    W = np.ones((n, n), np.float32)
    W[5, 7] = 2.0
    W[900, 33] = np.float32(2.0 ** log2_t)
    r = oracle.outlier_ratio(W, np.ones(n, np.float32), 2.0)
    assert r["sum"] == float(n * n) + 2.0 ** log2_t
    assert r["count"] == 0 and r["certified"] == certified


def test_unit_scores_certify_flags_a_rounding_boundary():
    # row 0: 1 + 2^-24 is exactly half way between the fp32 neighbours 1 and 1 + 2^-23 (the tie
    # rounds to even, 1.0): any change of the fp64 sum flips the rounding - not certified.
    # row 1: 1 + 2^-23 is an fp32 number: certified.  Columns: {1, 1}, {2^-24, 2^-23}, {0, 0}: exact.
    W = np.array([[1.0, 2.0 ** -24, 0.0], [1.0, 2.0 ** -23, 0.0]], np.float32)
    rs, cs = oracle.unit_scores(W, None)
    r_ok, c_ok = oracle.unit_scores_certify(W, None)
    assert rs[0] == np.float32(1.0) and rs[1] == np.float32(1.0 + 2.0 ** -23)
    assert list(r_ok) == [False, True] and list(c_ok) == [True, True, True]
    # as one row unit of two rows the sum is 2 + 3*2^-24 = 2 + 0.75 ulp(2): clear of a boundary
    r_ok, c_ok = oracle.unit_scores_certify(W, None, 2, 3)
    assert list(r_ok) == [True] and list(c_ok) == [True]
    # norms enter the scores that are summed: with norm_1 = 1/2 row 0 is 1 + 2^-25 (clear of the
    # boundary) and row 1 is 1 + 2^-24 (on it)
    r_ok, _ = oracle.unit_scores_certify(W, np.array([1, 0.5, 1], np.float32))
    assert list(r_ok) == [True, False]


def test_outlier_uses_column_norms_not_row_norms():
    # 2 x 3 matrix of ones; norms (1, 1, 100): the outliers are the third COLUMN.
    W = np.ones((2, 3), np.float32)
    r = oracle.outlier_ratio(W, np.array([1, 1, 100], np.float32), 2.0)
    assert r["count"] == 2 and r["sum"] == 204.0


# ----------------------------------------------------------------- allocation
def test_allocation_hand_cases():
    cols = [1000, 1000]
    # two projections: s = p +- lambda, the one with more outliers pruned less
    s, k, clamped = oracle.allocate_sparsity([10, 30], [1000, 1000], cols, 1, 2, 0.5, 0.1)
    np.testing.assert_allclose(s, [0.6, 0.4], rtol=0, atol=1e-15)
    assert list(k) == [600, 400] or list(k) == [599, 400] or list(k) == [600, 399]
    assert list(k) == [math.floor(s[0] * 1000), math.floor(s[1] * 1000)] and not clamped
    # three projections, R = 0, 1, 3 %: r = 0, 1/3, 1; dbar = 2*lam*4/9
    lam, p = 0.09, 0.7
    s, k, _ = oracle.allocate_sparsity([0, 10, 30], [1000] * 3, [1000] * 3, 3, 1, p, lam)
    want = [p + 2 * lam * (4 / 9 - r) for r in (0, 1 / 3, 1)]
    np.testing.assert_allclose(s, want, rtol=0, atol=1e-15)


@pytest.mark.parametrize("mode", [oracle.MODE_GLOBAL_NORM, oracle.MODE_PER_CATEGORY_NORM])
@pytest.mark.parametrize("p,lam", [(0.5, 0.08), (0.8, 0.15), (0.3, 0.0)])
def test_allocation_invariants(mode, p, lam):
    rng = np.random.default_rng(5)
    N, M = 6, 7
    numel = rng.integers(1000, 5000, N * M) * 64
    O = (numel * rng.random(N * M) * 0.03).astype(np.int64)
    cols = rng.choice([256, 688, 4096], N * M)
    s, k, clamped = oracle.allocate_sparsity(O, numel, cols, N, M, p, lam, mode)
    assert not clamped
    R = 100.0 * O / numel
    groups = [np.arange(N * M)] if mode == 0 else [np.arange(N) * M + m for m in range(M)]
    for g in groups:
        assert abs(s[g].mean() - p) < 1e-14                       # Eq. 1-2: targets average to p
        if lam > 0:
            assert abs((s[g].max() - s[g].min()) - 2 * lam) < 1e-14
            for a in g:
                for b in g:
                    if R[a] > R[b]:
                        assert s[a] < s[b]                        # more outliers => pruned less
        else:
            np.testing.assert_array_equal(s[g], p)                # uniform = global pruning
    np.testing.assert_array_equal(k, np.floor(s * cols).astype(np.int64))


def test_allocation_equal_ranks_and_clamp():
    s, k, clamped = oracle.allocate_sparsity([5] * 4, [100] * 4, [64] * 4, 2, 2, 0.37, 0.2)
    np.testing.assert_array_equal(s, 0.37)
    assert not clamped and list(k) == [math.floor(0.37 * 64)] * 4
    s, k, clamped = oracle.allocate_sparsity([0, 50], [100, 100], [64, 64], 1, 2, 0.95, 0.2)
    assert clamped and s[0] == 1 - 1 / 64 and k[0] == 63 and 0 <= s[1] <= 1


# ----------------------------------------------------------------- unstructured
def brute_prune(Wv, norms, k):
    rows, cols = Wv.shape
    pruned = np.zeros((rows, cols), bool)
    for i in range(rows):
        sc = [(float(exact_score(norms[j], Wv[i, j])), j) for j in range(cols)]
        for _, j in sorted(sc)[:k]:
            pruned[i, j] = True
    return pruned


def unpack_mask(mask, cols):
    bits = (mask[:, :, None] >> np.arange(32, dtype=np.uint32)[None, None, :]) & 1
    return bits.reshape(mask.shape[0], -1)[:, :cols].astype(bool), bits.reshape(mask.shape[0], -1)[:, cols:]


@pytest.mark.parametrize("dtype", DTYPES)
def test_unstructured_vs_full_sort_every_k(dtype):
    rng = np.random.default_rng(6)
    rows, cols = 6, 37                          # ragged: not a multiple of 32
    W = rand_matrix(rng, rows, cols, dtype)
    norms = (rng.random(cols).astype(np.float32) + np.float32(0.1)) * np.float32(10)
    Wv = as_f32(W, dtype)
    prev = None
    for k in range(cols + 1):
        Wp, mask = oracle.prune_unstructured(W, norms, k, dtype)
        pruned = brute_prune(Wv, norms, k)
        kept, pad = unpack_mask(mask, cols)
        np.testing.assert_array_equal(kept, ~pruned)
        assert not pad.any()                                        # padding bits are 0
        assert (kept.sum(1) == cols - k).all()                      # exact per-row sparsity
        np.testing.assert_array_equal(Wp[~pruned], W[~pruned])      # kept entries bit-identical
        assert (Wp[pruned] == 0).all()
        if prev is not None:
            assert (pruned | ~prev).all()                           # nested across increasing k
        prev = pruned


@pytest.mark.parametrize("dtype", DTYPES)
def test_unstructured_ties_lowest_index_first(dtype):
    cols = 40
    W = np.full((3, cols), 0.5, np.float32)
    W[1, ::2] = -0.5                              # same magnitude, other sign: still all tied
    W[2, 5] = 0.25                                # one strictly smaller entry goes first
    Wd = bf16_bits(W) if dtype == "bf16" else W
    ones = np.ones(cols, np.float32)
    for k in (0, 1, 7, cols):
        Wp, mask = oracle.prune_unstructured(Wd, ones, k, dtype)
        kept, _ = unpack_mask(mask, cols)
        assert (~kept[0, :k]).all() and kept[0, k:].all()
        assert (~kept[1, :k]).all() and kept[1, k:].all()
        if 0 < k < cols:
            assert not kept[2, 5]
            others = [j for j in range(cols) if j != 5]
            assert (~kept[2, others[:k - 1]]).all() and kept[2, others[k - 1:]].all()


def test_unstructured_unit_norms_is_magnitude_pruning():
    rng = np.random.default_rng(7)
    rows, cols, k = 9, 128, 50
    W = rand_matrix(rng, rows, cols, "bf16")
    Wp, mask = oracle.prune_unstructured(W, np.ones(cols, np.float32), k, "bf16")
    mag = np.abs(bf16_value(W))
    order = np.argsort(mag, axis=1, kind="stable")        # library routine: stable sort of |W|
    kept, _ = unpack_mask(mask, cols)
    for i in range(rows):
        want = np.ones(cols, bool)
        want[order[i, :k]] = False
        np.testing.assert_array_equal(kept[i], want)


def test_unstructured_scaling_activations_changes_nothing():
    # a positive per-projection constant in the norm changes neither the outlier
    # predicate nor any per-row order (power-of-two scale: exact in fp32)
    rng = np.random.default_rng(8)
    W = rand_matrix(rng, 8, 96, "bf16")
    norms = (rng.random(96).astype(np.float32) + np.float32(0.1))
    a = oracle.prune_unstructured(W, norms, 31, "bf16")
    b = oracle.prune_unstructured(W, norms * np.float32(4), 31, "bf16")
    np.testing.assert_array_equal(a[1], b[1])
    assert oracle.outlier_ratio(W, norms, 5.0, "bf16")["count"] == \
        oracle.outlier_ratio(W, norms * np.float32(4), 5.0, "bf16")["count"]


# ----------------------------------------------------------------- structured
@pytest.mark.parametrize("dtype", DTYPES)
@pytest.mark.parametrize("rg,cg", [(1, 1), (4, 2), (2, 8)])
def test_unit_scores_exact(dtype, rg, cg):
    rng = np.random.default_rng(9)
    rows, cols = 8, 16
    W = rand_matrix(rng, rows, cols, dtype)
    Wv = as_f32(W, dtype)
    norms = (rng.random(cols).astype(np.float32) + np.float32(0.1)) * np.float32(7)
    for nv in (norms, None):
        rs, cs = oracle.unit_scores(W, nv, rg, cg, dtype)
        nn = norms if nv is not None else np.ones(cols, np.float32)
        sc = [[Fraction(float(exact_score(nn[j], Wv[i, j]))) for j in range(cols)] for i in range(rows)]
        for u in range(rows // rg):
            exact = sum(sc[i][j] for i in range(u * rg, (u + 1) * rg) for j in range(cols))
            assert abs(Fraction(float(rs[u])) - exact) <= exact * Fraction(1, 2 ** 23)
        for v in range(cols // cg):
            exact = sum(sc[i][j] for i in range(rows) for j in range(v * cg, (v + 1) * cg))
            assert abs(Fraction(float(cs[v])) - exact) <= exact * Fraction(1, 2 ** 23)
    # norms=None is pure magnitude: row score = sum |W|
    rs, _ = oracle.unit_scores(W, None, 1, 1, dtype)
    np.testing.assert_allclose(rs, np.abs(Wv).astype(np.float64).sum(1).astype(np.float32), rtol=2e-7)


def test_rank_units_vs_sort_and_nesting():
    rng = np.random.default_rng(10)
    n = 50
    scores = rng.random(n).astype(np.float32)
    scores[[4, 9, 30]] = scores[2]                   # ties
    order = sorted(range(n), key=lambda u: (float(scores[u]), u))
    prev = None
    for keep in range(n, -1, -1):
        got = oracle.rank_units(scores, keep)
        want = sorted(order[n - keep:])
        assert list(got) == want
        assert all(a < b for a, b in zip(got[:-1], got[1:]))       # strictly ascending
        if prev is not None:
            assert set(got) <= prev                                 # nested keep sets
        prev = set(got)
    assert list(oracle.rank_units(scores, n)) == list(range(n))    # removing nothing = identity
    eq = np.full(6, 2.0, np.float32)
    assert list(oracle.rank_units(eq, 4)) == [2, 3, 4, 5]          # ties: lowest index removed first


@pytest.mark.parametrize("dtype", DTYPES)
def test_compact_equals_fancy_indexing(dtype):
    rng = np.random.default_rng(11)
    rows, cols, rg, cg = 12, 24, 3, 4
    W = rand_matrix(rng, rows, cols, dtype)
    rk, ck = np.array([0, 2, 3], np.int32), np.array([1, 2, 5], np.int32)
    Wc = oracle.compact(W, rk, ck, rg, cg, dtype)
    ri = np.concatenate([np.arange(u * rg, (u + 1) * rg) for u in rk])
    ci = np.concatenate([np.arange(u * cg, (u + 1) * cg) for u in ck])
    assert Wc.shape == (len(rk) * rg, len(ck) * cg)                # shape = retained counts
    np.testing.assert_array_equal(Wc, W[ri][:, ci])
    full = oracle.compact(W, np.arange(rows // rg, dtype=np.int32), np.arange(cols // cg, dtype=np.int32), rg, cg, dtype)
    np.testing.assert_array_equal(full, W)                         # keep everything = identity


def test_composite_order_matters():
    # unstructured first, then structured ranking on the masked matrix (Section 3.3 (c)):
    # row 0 = many small entries, row 1 = one big entry.  Unmasked row sums: row0 > row1.
    # After zeroing the 6 smallest entries of every row, row 0 collapses and is removed.
    W = np.zeros((2, 8), np.float32)
    W[0, :] = 0.3
    W[0, 0] = 0.35
    W[1, 3] = 2.0
    ones = np.ones(8, np.float32)
    rs_raw, _ = oracle.unit_scores(W, ones)
    assert rs_raw[0] > rs_raw[1]
    Wp, _ = oracle.prune_unstructured(W, ones, 6)
    rs_masked, _ = oracle.unit_scores(Wp, ones)
    assert rs_masked[0] < rs_masked[1]
    assert list(oracle.rank_units(rs_raw, 1)) == [0]
    assert list(oracle.rank_units(rs_masked, 1)) == [1]
    # zeros inside the compacted matrix are exactly the mask's zeros on kept rows/cols
    Wc = oracle.compact(Wp, oracle.rank_units(rs_masked, 1), np.arange(8, dtype=np.int32))
    np.testing.assert_array_equal(Wc, Wp[1:2])


# ----------------------------------------------------------------- config-1 sanity
def test_tiny_config_outliers_sit_in_planted_columns():
    cfg = wl.CONFIGS["tiny"]
    for proj in ("q", "gate", "down"):
        W = wl.to_numpy(wl.gen_weight(cfg, 0, proj))
        X = wl.to_numpy(wl.gen_activation(cfg, 0, cfg.x_key(proj)))
        norms = oracle.act_norms(X)
        assert oracle.norm_certify(X).all()
        r = oracle.outlier_ratio(W, norms, cfg.alpha)
        assert r["certified"]
        S = oracle.score(W, norms)
        tau = cfg.alpha * r["sum"] / r["numel"]
        cols = wl.outlier_columns(cfg, 0, cfg.x_key(proj), W.shape[1], cfg.x_outlier_frac).numpy()
        inside = (S[:, cols] > tau).sum()
        assert (S > tau).sum() == r["count"]
        assert inside >= 0.99 * r["count"] > 0


@pytest.mark.parametrize("base", [oracle.MODE_GLOBAL_NORM, oracle.MODE_PER_CATEGORY_NORM])
def test_allocation_weighted_mean_prunes_exactly_p_of_the_parameters(base):
    # with the parameter-weighted mean the pruned share of all parameters (of each normalisation
    # group) is p; the spread, the order and the equal-size special case are unchanged
    rng = np.random.default_rng(7)
    N, M, p, lam = 6, 7, 0.6, 0.1
    numel = np.tile(np.array([16, 16, 16, 16, 43, 43, 43]) * 1_000_000, N).astype(np.int64)
    cols = np.tile(np.array([4096] * 6 + [11008]), N).astype(np.int64)
    O = (numel * rng.uniform(0.001, 0.03, N * M)).astype(np.int64)
    s, k, clamped = oracle.allocate_sparsity(O, numel, cols, N, M, p, lam, base | oracle.MODE_WEIGHTED_MEAN)
    assert not clamped
    groups = [np.arange(N * M)] if base == 0 else [np.arange(N) * M + m for m in range(M)]
    R = 100.0 * O / numel
    for g in groups:
        assert abs(np.sum(s[g] * numel[g]) / np.sum(numel[g]) - p) < 1e-12
        assert abs((s[g].max() - s[g].min()) - 2 * lam) < 1e-12
        order = np.argsort(R[g])
        assert (np.diff(s[g][order]) <= 1e-15).all()
    s_plain, _, _ = oracle.allocate_sparsity(O, numel, cols, N, M, p, lam, base)
    if base == 0:
        assert abs(np.mean(s_plain) - p) < 1e-12 and abs(np.sum(s_plain * numel) / np.sum(numel) - p) > 1e-6
    # equal sizes: the weighted and the plain mean coincide
    same = np.full(N * M, 1 << 20, np.int64)
    a, _, _ = oracle.allocate_sparsity(O % (1 << 20), same, cols, N, M, p, lam, base | oracle.MODE_WEIGHTED_MEAN)
    b, _, _ = oracle.allocate_sparsity(O % (1 << 20), same, cols, N, M, p, lam, base)
    np.testing.assert_allclose(a, b, rtol=0, atol=1e-15)


# ----------------------------------------------------------------- layer outlier distribution (Eq. 3-4)
@pytest.mark.parametrize("dtype", DTYPES)
def test_group_outlier_count_vs_exact_enumeration(dtype):
    # three matrices of different shapes under ONE threshold alpha * mean over all their scores
    rng = np.random.default_rng(14)
    shapes = [(6, 16), (3, 40), (9, 8)]
    Ws, Wv, norms = [], [], []
    for rows, cols in shapes:
        W = rand_matrix(rng, rows, cols, dtype)
        W_f = as_f32(W, dtype).copy()
        W_f[rng.random((rows, cols)) < 0.08] *= 30
        Ws.append(bf16_bits(W_f) if dtype == "bf16" else W_f)
        Wv.append(as_f32(Ws[-1], dtype))
        norms.append((rng.random(cols).astype(np.float32) + np.float32(0.1)) * np.float32(10 ** rng.integers(0, 3)))
    for alpha in (1.0, 3.0, 5.0):
        sc = [[[Fraction(float(exact_score(n[j], W[i, j]))) for j in range(W.shape[1])] for i in range(W.shape[0])]
              for W, n in zip(Wv, norms)]
        C = sum(W.size for W in Wv)
        total = sum(s for m in sc for r in m for s in r)
        tau = Fraction(float(np.float32(alpha))) * total / C
        want = [sum(1 for r in m for s in r if s > tau) for m in sc]
        got = oracle.outlier_ratio_group(Ws, norms, alpha, dtype)
        assert got["counts"] == want and got["count"] == sum(want) and got["numel"] == C
        assert abs(Fraction(got["sum"]) - total) <= total * Fraction(C, 2 ** 52)
        assert got["ratio"] == 100.0 * sum(want) / C


def test_group_of_one_is_the_projection_statistic_and_groups_differ_from_projections():
    rng = np.random.default_rng(15)
    W = rand_matrix(rng, 12, 24, "f32")
    n = rng.random(24).astype(np.float32) + np.float32(0.5)
    one = oracle.outlier_ratio_group([W], [n], 4.0)
    ref = oracle.outlier_ratio(W, n, 4.0)
    assert one["counts"] == [ref["count"]] and one["sum"] == ref["sum"] and one["ratio"] == ref["ratio"]
    # hand case: A = all ones (4 entries), B = all 100s (4 entries), alpha = 1.5.  Per projection nothing exceeds
    # 1.5 x its own mean; in the group the mean is 50.5, tau = 75.75: every entry of B is an outlier, none of A.
    A, B = np.ones((2, 2), np.float32), np.full((2, 2), 100.0, np.float32)
    ones = np.ones(2, np.float32)
    assert oracle.outlier_ratio(A, ones, 1.5)["count"] == 0 and oracle.outlier_ratio(B, ones, 1.5)["count"] == 0
    g = oracle.outlier_ratio_group([A, B], [ones, ones], 1.5)
    assert g["counts"] == [0, 4] and g["sum"] == 404.0 and g["ratio"] == 50.0 and g["certified"]
    # a score exactly on the group threshold: not an outlier, and not certified
    g = oracle.outlier_ratio_group([np.array([[1, 1]], np.float32), np.array([[1, 3]], np.float32)], [ones, ones], 2.0)
    assert g["counts"] == [0, 0] and not g["certified"]


# ----------------------------------------------------------------- clamp and redistribute
def _wmean(s, w):
    return float(np.dot(s, w) / np.sum(w))


@pytest.mark.parametrize("weighted", [False, True])
def test_redistribution_keeps_the_mean_at_p_after_clamping(weighted):
    # ranks spread so widely (lambda = 0.6) that several targets fall below 0 or above 1 - 1/cols
    counts = [0, 5, 10, 200, 400, 0, 900, 20]
    numels = [1000, 4000, 1000, 2000, 1000, 8000, 1000, 3000]
    cols = [10, 40, 10, 20, 10, 80, 10, 30]
    mode = oracle.MODE_REDISTRIBUTE | (oracle.MODE_WEIGHTED_MEAN if weighted else 0)
    w = np.array(numels, np.float64) if weighted else np.ones(8)
    for p in (0.3, 0.5, 0.7):
        s0, _, clamped0 = oracle.allocate_sparsity(counts, numels, cols, 4, 2, p, 0.6, mode & ~oracle.MODE_REDISTRIBUTE)
        assert clamped0 and abs(_wmean(s0, w) - p) > 1e-3            # plain clamping leaves the mean off p
        s, k, infeasible = oracle.allocate_sparsity(counts, numels, cols, 4, 2, p, 0.6, mode)
        assert not infeasible
        assert abs(_wmean(s, w) - p) < 1e-14                          # the (weighted) mean is p again
        smax = 1.0 - 1.0 / np.array(cols)
        assert (s >= 0).all() and (s <= smax).all()
        on_bound = (s == 0) | (s == smax)
        assert on_bound.any() and not on_bound.all()
        free = ~on_bound                                              # the free targets keep their mutual distances
        np.testing.assert_allclose(np.diff(s[free]), np.diff(s0_unclamped(counts, numels, cols, p, 0.6, weighted)[free]), atol=1e-15)
        assert list(k) == [math.floor(a * c) for a, c in zip(s, cols)]


def s0_unclamped(counts, numels, cols, p, lam, weighted):
    R = 100.0 * np.array(counts, np.float64) / np.array(numels, np.float64)
    r = (R - R.min()) / (R.max() - R.min())
    d = 2 * lam * r
    w = np.array(numels, np.float64) if weighted else np.ones(len(counts))
    return p + np.dot(w, d) / w.sum() - d


def test_redistribution_changes_nothing_without_a_clamp_and_flags_the_impossible():
    counts, numels, cols = [10, 30, 20, 25], [1000] * 4, [100] * 4
    a = oracle.allocate_sparsity(counts, numels, cols, 2, 2, 0.5, 0.08, 0)
    b = oracle.allocate_sparsity(counts, numels, cols, 2, 2, 0.5, 0.08, oracle.MODE_REDISTRIBUTE)
    assert np.array_equal(a[0].view(np.uint64), b[0].view(np.uint64)) and list(a[1]) == list(b[1]) and not b[2]
    # hand case, two projections, p = 0.5, lambda = 0.8: targets 1.3 and -0.3 -> both on their bounds (0.9 and 0): the
    # mean 0.45 cannot be brought to 0.5, which is reported
    s, k, infeasible = oracle.allocate_sparsity([0, 10], [100, 100], [10, 10], 1, 2, 0.5, 0.8, oracle.MODE_REDISTRIBUTE)
    np.testing.assert_allclose(s, [0.9, 0.0], atol=1e-15)
    assert infeasible
    # three projections, R = 0, 50, 100 %, p = 0.5, lambda = 0.5: b = (1.0, 0.5, 0.0) with bounds [0, 0.9]:
    # the first clamps to 0.9, the others shift by t = (1.5 - 0.9 - 0.5) / 2 = 0.05
    s, k, infeasible = oracle.allocate_sparsity([0, 50, 100], [100] * 3, [10] * 3, 1, 3, 0.5, 0.5, oracle.MODE_REDISTRIBUTE)
    np.testing.assert_allclose(s, [0.9, 0.55, 0.05], atol=1e-15)
    assert not infeasible and list(k) == [9, 5, 0]


# ----------------------------------------------------------------- second moments / Hessian (calibration side, Section 4.1.3)
@pytest.mark.parametrize("dtype", DTYPES)
def test_gram_exact_rational_brute_force(dtype):
    """Every entry against sum_t x_tj x_tl in exact rational arithmetic (the fp64 sums are exact
    here: a handful of products of 8- or 24-bit mantissas with close exponents)."""
    rng = np.random.default_rng(11)
    X = (rng.integers(-8, 9, size=(7, 5)) * 0.25).astype(np.float32)
    Xd = bf16_bits(X) if dtype == "bf16" else X
    G, Ga = oracle.gram(Xd, None, dtype, with_abs=True)
    Xv = as_f32(Xd, dtype)
    for j in range(5):
        for l in range(5):
            exact = sum(Fraction(float(Xv[t, j])) * Fraction(float(Xv[t, l])) for t in range(7))
            exact_abs = sum(abs(Fraction(float(Xv[t, j])) * Fraction(float(Xv[t, l]))) for t in range(7))
            assert Fraction(float(G[j, l])) == exact, (j, l)
            assert Fraction(float(Ga[j, l])) == exact_abs, (j, l)


@pytest.mark.parametrize("dtype", DTYPES)
def test_gram_closed_forms(dtype):
    # constant columns c_j: G[j,l] = T c_j c_l (all values powers of two: exact)
    T, c = 64, np.array([1.0, -2.0, 0.5, 4.0, 0.0, -0.25], np.float32)
    X = np.tile(c, (T, 1))
    Xd = bf16_bits(X) if dtype == "bf16" else X
    G = oracle.gram(Xd, None, dtype)
    assert np.array_equal(G, T * np.outer(c, c).astype(np.float64))
    # one non-zero per token (token t excites channel t mod cols with value v_t): G is diagonal
    cols = 5
    v = (np.arange(1, 21) * 0.5).astype(np.float32)
    X = np.zeros((20, cols), np.float32)
    X[np.arange(20), np.arange(20) % cols] = v
    Xd = bf16_bits(X) if dtype == "bf16" else X
    G = oracle.gram(Xd, None, dtype)
    expect = np.zeros((cols, cols))
    for t in range(20):
        expect[t % cols, t % cols] += float(v[t]) ** 2
    assert np.array_equal(G, expect)
    # the back-end's Hessian is 2/T times it
    assert np.array_equal(oracle.hessian(Xd, dtype), expect * (2.0 / 20))


@pytest.mark.parametrize("dtype", DTYPES)
def test_gram_against_library_matmul_and_invariants(dtype):
    rng = np.random.default_rng(12)
    T, cols = 300, 24
    X = rng.standard_normal((T, cols)).astype(np.float32)
    X[:, 3] *= 50.0                                   # an outlier channel
    Xd = bf16_bits(X) if dtype == "bf16" else X
    Xv = as_f32(Xd, dtype).astype(np.float64)
    G, Ga = oracle.gram(Xd, None, dtype, with_abs=True)
    ref = Xv.T @ Xv                                    # the textbook definition through BLAS (another summation order)
    assert np.allclose(G, ref, rtol=0, atol=1e-12 * np.abs(Xv).T @ np.abs(Xv))
    assert np.array_equal(G, G.T)                      # symmetric, bit for bit (products commute)
    assert np.linalg.eigvalsh(G).min() > -1e-9 * np.trace(G)          # positive semi-definite
    assert (Ga >= np.abs(G)).all() and np.allclose(Ga, np.abs(Xv).T @ np.abs(Xv), rtol=1e-12)
    # the diagonal is the squared norm of Eq. 5
    assert np.allclose(np.diag(G), oracle.act_sumsq(Xd, None, dtype), rtol=1e-14)
    # scaling the activations by 2 scales every second moment by exactly 4
    X2 = (2.0 * as_f32(Xd, dtype)).astype(np.float32)
    X2d = bf16_bits(X2) if dtype == "bf16" else X2
    assert np.array_equal(oracle.gram(X2d, None, dtype), 4.0 * G)
    # a transposed or mis-strided read shows on a view with a leading dimension larger than cols
    wide = np.zeros((T, cols + 8), Xd.dtype)
    wide[:, :cols] = Xd
    wide[:, cols:] = Xd[:, :8]                         # junk beyond the columns
    assert np.array_equal(oracle.gram(wide[:, :cols], None, dtype), G)


@pytest.mark.parametrize("dtype", DTYPES)
def test_gram_accumulates_over_token_chunks_and_pairs_agree(dtype):
    rng = np.random.default_rng(13)
    T, cols = 257, 16
    X = rng.standard_normal((T, cols)).astype(np.float32)
    Xd = bf16_bits(X) if dtype == "bf16" else X
    G = oracle.gram(Xd, None, dtype)
    acc = np.zeros((cols, cols))
    for a, b in [(0, 100), (100, 101), (101, 257)]:
        oracle.gram(np.ascontiguousarray(Xd[a:b]), acc, dtype)
    assert np.allclose(acc, G, rtol=0, atol=1e-13 * np.abs(G).max())
    js, ls = np.array([0, 3, 15, 7, 7]), np.array([0, 9, 2, 7, 8])
    out, out_abs = oracle.gram_pairs(Xd, js, ls, dtype)
    assert np.array_equal(out, G[js, ls])
    assert (out_abs >= np.abs(out)).all()
