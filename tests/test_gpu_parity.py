"""GPU parity: every device call of the C ABI against the CPU oracle, element by
element, on the same seeded inputs.  Masks, pruned weights, keep lists,
compacted weights and outlier counts must be bit-exact; norms and scores are
required within 1e-5 relative and are additionally expected bit-exact wherever
the oracle certifies that fp64 summation order cannot matter.
"""
import numpy as np
import pytest
import torch

import oracle
import oracle_pipeline as op
from paper_2504_06323_b200 import api, workloads as wl

pytestmark = pytest.mark.gpu
DEV = "cuda"
REL = 1e-5   # relative tolerance required of norms and scores in fp32


def make(rows, cols, dtype, seed, ld=None, scale=0.02, heavy=False):
    """Random matrix on the device with optional padded leading dimension."""
    g = torch.Generator(device="cpu").manual_seed(seed)
    ld = cols if ld is None else ld
    buf = torch.randn(rows, ld, generator=g) * scale
    if heavy:
        buf = buf * torch.exp(2.0 * torch.randn(rows, ld, generator=g))
    buf = buf.to(torch.float32 if dtype == "f32" else torch.bfloat16).to(DEV)
    return buf[:, :cols]


def host(t):
    return wl.to_numpy(t)


def norms_for(cols, seed):
    g = torch.Generator(device="cpu").manual_seed(seed)
    n = (torch.rand(cols, generator=g) + 0.05) * 40.0
    n[::97] *= 50.0
    return n.to(torch.float32).to(DEV)


def assert_bits_equal(a: np.ndarray, b: np.ndarray):
    assert a.shape == b.shape and a.dtype == b.dtype
    a, b = np.ascontiguousarray(a), np.ascontiguousarray(b)
    assert np.array_equal(a.view(np.uint8), b.view(np.uint8))


# ------------------------------------------------------------------ act norms
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("T,cols,ld", [(1024, 256, None), (1000, 688, None), (4100, 1000, 1008), (33, 8, 16), (70000, 520, None)])
def test_act_norms(dtype, T, cols, ld):
    X = make(T, cols, dtype, seed=T + cols, ld=ld, scale=1.0)
    X[:, 3] *= 100.0
    Xh = host(X)
    ss_ref = oracle.act_sumsq(Xh, None, dtype)
    n_ref = oracle.norm_finalize(ss_ref)
    ok = oracle.norm_certify(Xh, dtype)
    ss = torch.full((cols,), 123.0, dtype=torch.float64, device=DEV)     # RESET must ignore this
    n = torch.empty(cols, dtype=torch.float32, device=DEV)
    api.mosaic_act_norms(X, ss, n, api.RESET_ACCUM)
    np.testing.assert_allclose(ss.cpu().numpy(), ss_ref, rtol=1e-13)
    np.testing.assert_allclose(n.cpu().numpy(), n_ref, rtol=REL)
    assert ok.mean() > 0.999
    assert_bits_equal(n.cpu().numpy()[ok], n_ref[ok])


def test_act_norms_accumulates_over_chunks_and_handles_empty_chunk():
    X = make(3000, 300, "bf16", seed=5, ld=304, scale=1.0)
    Xh = host(X)
    n_ref = oracle.act_norms(Xh, "bf16")
    ss = torch.zeros(300, dtype=torch.float64, device=DEV)
    n = torch.empty(300, dtype=torch.float32, device=DEV)
    api.mosaic_act_norms(X[:1111], ss, None, api.RESET_ACCUM)
    api.mosaic_act_norms(X[1111:1111], ss, None)                 # tokens == 0 is legal
    api.mosaic_act_norms(X[1111:], ss, n)
    ok = oracle.norm_certify(Xh, "bf16")
    np.testing.assert_allclose(n.cpu().numpy(), n_ref, rtol=REL)
    assert_bits_equal(n.cpu().numpy()[ok], n_ref[ok])
    n2 = torch.empty_like(n)
    api.mosaic_act_norms(X[:0], ss, n2)                          # finalise only
    assert_bits_equal(n2.cpu().numpy(), n.cpu().numpy())


def test_act_norms_zero_denormal_and_closed_forms():
    T = 96
    X = torch.zeros(T, 8, dtype=torch.bfloat16, device=DEV)
    X[:, 0] = 3.0
    X[17, 1] = -2.5
    X[:, 2] = 2.0 ** -130          # bf16 denormal: squares underflow fp32 but not fp64
    X[0, 3], X[1, 3] = 3.0, 4.0
    ss = torch.zeros(8, dtype=torch.float64, device=DEV)
    n = torch.empty(8, dtype=torch.float32, device=DEV)
    api.mosaic_act_norms(X, ss, n, api.RESET_ACCUM)
    n_ref = oracle.act_norms(host(X), "bf16")
    assert_bits_equal(n.cpu().numpy(), n_ref)
    assert n[0].item() == np.float32(3.0 * np.sqrt(96.0)) and n[1].item() == 2.5 and n[3].item() == 5.0
    assert n[4].item() == 0.0 and n[2].item() > 0.0


# ------------------------------------------------------------------ score
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("rows,cols,ld", [(256, 256, None), (300, 1000, 1008), (7, 13, 16)])
def test_score_bit_exact(dtype, rows, cols, ld):
    W = make(rows, cols, dtype, seed=rows * cols, ld=ld)
    norms = norms_for(cols, 1)
    out = torch.empty(rows, cols, dtype=torch.float32, device=DEV)
    api.mosaic_score(W, norms, out)
    ref = oracle.score(host(W), norms.cpu().numpy(), dtype)
    assert_bits_equal(out.cpu().numpy(), ref)


# ------------------------------------------------------------------ outlier ratio
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("rows,cols,ld,alpha", [(256, 256, None, 5.0), (688, 256, None, 5.0), (256, 688, None, 3.0),
                                                (1000, 1000, 1008, 5.0), (3, 5, 8, 1.0), (2048, 4096, None, 5.0),
                                                (517, 11008, None, 7.5)])
def test_outlier_ratio(dtype, rows, cols, ld, alpha):
    W = make(rows, cols, dtype, seed=rows + 3 * cols, ld=ld, heavy=True)
    norms = norms_for(cols, 2)
    cnt = torch.full((1,), -7, dtype=torch.int64, device=DEV)
    ssum = torch.zeros(1, dtype=torch.float64, device=DEV)
    api.mosaic_outlier_ratio(W, norms, alpha, cnt, ssum)
    ref = oracle.outlier_ratio(host(W), norms.cpu().numpy(), alpha, dtype)
    assert ref["certified"]
    assert cnt.item() == ref["count"] and ref["count"] > 0
    np.testing.assert_allclose(ssum.item(), ref["sum"], rtol=1e-13)
    assert api.mosaic_ratio_from_count(cnt.item(), rows * cols) == ref["ratio"]
    cnt2 = torch.zeros(1, dtype=torch.int64, device=DEV)
    api.mosaic_outlier_ratio(W, norms, alpha, cnt2, None)             # sum output is optional; rerun is identical
    assert cnt2.item() == cnt.item()


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_outlier_ratio_batch_matches_oracle_job_by_job(dtype):
    shapes = [(256, 256), (688, 256), (300, 1000), (7, 13), (1100, 4096), (64, 11008), (65, 1024), (1, 8)]
    jobs, refs = [], []
    counts = torch.full((len(shapes),), -5, dtype=torch.int64, device=DEV)
    sums = torch.full((len(shapes),), -1.0, dtype=torch.float64, device=DEV)
    for i, (rows, cols) in enumerate(shapes):
        ld = cols if cols % 8 == 0 else (cols + 7) // 8 * 8
        W = make(rows, cols, dtype, seed=900 + i, ld=ld, heavy=(i % 2 == 1))
        norms = norms_for(cols, 60 + i)
        refs.append(oracle.outlier_ratio(host(W), norms.cpu().numpy(), 4.0, dtype))
        jobs.append((W, norms, counts[i:i + 1], sums[i:i + 1] if i != 2 else None))
    api.mosaic_outlier_ratio_batch(jobs, 4.0)
    for i, ref in enumerate(refs):
        assert ref["certified"]
        assert counts[i].item() == ref["count"], shapes[i]
        if i != 2:
            np.testing.assert_allclose(sums[i].item(), ref["sum"], rtol=1e-12)
    assert sums[2].item() == -1.0
    # the single call gives the same bits as the batch
    for i, (W, norms, _, _) in enumerate(jobs):
        c1 = torch.zeros(1, dtype=torch.int64, device=DEV)
        s1 = torch.zeros(1, dtype=torch.float64, device=DEV)
        api.mosaic_outlier_ratio(W, norms, 4.0, c1, s1)
        assert c1.item() == counts[i].item()
        if i != 2:
            assert s1.cpu().numpy().tobytes() == sums[i:i + 1].cpu().numpy().tobytes()


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_outlier_ratio_uneven_rows_and_dense_threshold(dtype):
    # rows of very different scale (a sample of rows would misjudge the mean), and a matrix whose
    # scores all sit within 3 % of the threshold
    rows, cols = 1100, 2048
    W = make(rows, cols, dtype, seed=321).clone()
    W[::3] *= 40.0                      # every third row is large; the sample sees a different mix
    W[5::7, ::5] *= 300.0
    norms = norms_for(cols, 70)
    for alpha in (2.0, 5.0, 9.0):
        ref = oracle.outlier_ratio(host(W), norms.cpu().numpy(), alpha, dtype)
        cnt = torch.zeros(1, dtype=torch.int64, device=DEV)
        api.mosaic_outlier_ratio(W, norms, alpha, cnt)
        assert ref["certified"] and cnt.item() == ref["count"], alpha
    # all weights equal up to 3 %, alpha = 1: the threshold cuts through the bulk of the scores
    g = torch.Generator(device="cpu").manual_seed(5)
    W2 = ((1.0 + 0.03 * torch.rand(600, 2048, generator=g)) * 0.5).to(W.dtype).to(DEV)
    ones = torch.ones(2048, dtype=torch.float32, device=DEV)
    ref = oracle.outlier_ratio(host(W2), ones.cpu().numpy(), 1.0, dtype)
    cnt = torch.zeros(1, dtype=torch.int64, device=DEV)
    api.mosaic_outlier_ratio(W2, ones, 1.0, cnt)
    assert ref["certified"] and cnt.item() == ref["count"] and 0 < ref["count"] < 600 * 2048


def test_outlier_batch_single_sweep_and_its_fallback():
    """The batched bf16 call counts in ONE sweep from an estimate of the threshold taken on a sample of
    rows (about every rows/128-th), and falls back to the count sweep where the estimate misleads it.
    Matrices whose sampled rows are unlike the rest, in both directions, non-finite weights, dead
    channels and a constant matrix must all give the oracle's count and the single call's sum."""
    cols = 2048
    cases = []
    for kind in ("plain", "sample_small", "sample_large", "inf", "nan", "dead_channels", "constant", "tall"):
        rows = 3000 if kind == "tall" else 512
        W = make(rows, cols, "bf16", seed=4000 + len(cases), heavy=(kind == "tall")).clone()
        n = norms_for(cols, 400 + len(cases))
        step = max(rows // 128, 1)
        if kind == "sample_small":
            W[step // 2::step] *= 0.001          # the sampled rows say "small scores": the ladders sit far too low
        elif kind == "sample_large":
            W[step // 2::step] *= 1000.0         # ... "large scores": far too high
        elif kind == "inf":
            W[7, 9] = float("inf")
        elif kind == "nan":
            W[300, 2000] = float("nan")
        elif kind == "dead_channels":
            n = n * (torch.rand(cols, device=DEV) > 0.5)
        elif kind == "constant":
            W.fill_(0.5)
            n = torch.ones(cols, device=DEV)
        cases.append((kind, W, n))
    counts = torch.full((len(cases),), -5, dtype=torch.int64, device=DEV)
    sums = torch.full((len(cases),), -1.0, dtype=torch.float64, device=DEV)
    api.mosaic_outlier_ratio_batch([(W, n, counts[i:i + 1], sums[i:i + 1]) for i, (_, W, n) in enumerate(cases)], 4.0)
    torch.cuda.synchronize()
    for i, (kind, W, n) in enumerate(cases):
        ref = oracle.outlier_ratio(host(W), n.cpu().numpy(), 4.0, "bf16")
        assert counts[i].item() == ref["count"], kind
        if kind not in ("inf", "nan"):
            assert ref["certified"], kind
            c1 = torch.zeros(1, dtype=torch.int64, device=DEV)
            s1 = torch.zeros(1, dtype=torch.float64, device=DEV)
            api.mosaic_outlier_ratio(W, n, 4.0, c1, s1)
            assert c1.item() == counts[i].item(), kind
            assert s1.cpu().numpy().tobytes() == sums[i:i + 1].cpu().numpy().tobytes(), kind   # same partial sums, same order
    assert counts[[k for k, _, _ in cases].index("constant")].item() == 0


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_outlier_ratio_grouped_matches_oracle(dtype):
    # Eq. 3-4: the matrices of a group are counted against ONE threshold; three groups of different sizes
    shapes = [(256, 256), (688, 256), (256, 688), (300, 1000), (1100, 4096), (64, 11008), (65, 1024), (1, 8), (40, 2048)]
    groups = [0, 0, 0, 1, 1, 2, 2, 2, 2]
    Ws, norms = [], []
    for i, (rows, cols) in enumerate(shapes):
        W = make(rows, cols, dtype, seed=1300 + i, heavy=(i % 2 == 1), scale=0.02 * (1 + 3 * (i % 3)))
        Ws.append(W)
        norms.append(norms_for(cols, 110 + i))
    counts = torch.full((len(shapes),), -5, dtype=torch.int64, device=DEV)
    sums = torch.full((len(shapes),), -1.0, dtype=torch.float64, device=DEV)
    jobs = [(W, n, counts[i:i + 1], sums[i:i + 1]) for i, (W, n) in enumerate(zip(Ws, norms))]
    api.mosaic_outlier_ratio_grouped(jobs, groups, 4.0)
    got = counts.cpu().tolist()
    for g in sorted(set(groups)):
        idx = [i for i, x in enumerate(groups) if x == g]
        ref = oracle.outlier_ratio_group([host(Ws[i]) for i in idx], [norms[i].cpu().numpy() for i in idx], 4.0, dtype)
        assert ref["certified"] and ref["count"] > 0
        assert [got[i] for i in idx] == ref["counts"], g
        np.testing.assert_allclose(sum(sums[i].item() for i in idx), ref["sum"], rtol=1e-12)
    # the grouped count differs from the per-matrix one somewhere (else the test shows nothing)
    api.mosaic_outlier_ratio_batch(jobs, 4.0)
    assert counts.cpu().tolist() != got
    # groups of one matrix each are the per-matrix statistic
    per_matrix = counts.cpu().tolist()
    api.mosaic_outlier_ratio_grouped(jobs, list(range(len(shapes))), 4.0)
    assert counts.cpu().tolist() == per_matrix


def test_outlier_planted_and_constant():
    rows, cols = 64, 1024
    W = torch.ones(rows, cols, dtype=torch.bfloat16, device=DEV)
    W.view(-1)[[3, 77, 2000, 30100, 65535]] = -64.0
    ones = torch.ones(cols, dtype=torch.float32, device=DEV)
    cnt = torch.zeros(1, dtype=torch.int64, device=DEV)
    api.mosaic_outlier_ratio(W, ones, 5.0, cnt)
    assert cnt.item() == 5
    api.mosaic_outlier_ratio(W, ones, 0.5, cnt)
    assert cnt.item() == rows * cols
    Wc = torch.full((rows, cols), 0.25, dtype=torch.bfloat16, device=DEV)
    api.mosaic_outlier_ratio(Wc, ones, 1.0, cnt)                      # score == mean: strict '>' gives none
    assert cnt.item() == 0


# ------------------------------------------------------------------ unstructured
def run_prune(W, norms, k, inplace=False):
    rows, cols = W.shape
    if inplace:
        out = W
    else:   # same leading dimension as the input
        ld = W.stride(0) if rows > 1 else cols
        out = torch.full((rows, ld), 7.0, dtype=W.dtype, device=DEV)[:, :cols]
    mask = torch.full((rows, (cols + 31) // 32), -1, dtype=torch.int32, device=DEV)
    api.mosaic_prune_unstructured(W, out, norms, k, mask)
    return out, mask


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("rows,cols,ld", [(64, 256, None), (40, 688, None), (33, 1000, 1008), (9, 37, 40),
                                          (24, 4096, None), (10, 5120, None), (6, 11008, None), (5, 13824, None),
                                          (5, 14336, None), (300, 2048, None)])
def test_prune_unstructured_bit_exact(dtype, rows, cols, ld):
    W = make(rows, cols, dtype, seed=cols + rows, ld=ld, heavy=True)
    norms = norms_for(cols, 3)
    Wh, nh = host(W), norms.cpu().numpy()
    for k in sorted({0, 1, cols // 3, cols // 2, cols - 1, cols}):
        out, mask = run_prune(W, norms, k)
        ref_W, ref_mask = oracle.prune_unstructured(Wh, nh, k, dtype)
        assert_bits_equal(host(out), ref_W)
        assert_bits_equal(mask.cpu().numpy().view(np.uint32), ref_mask)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_prune_ties_everywhere(dtype):
    # unit norms on low-precision weights: massive ties, resolved by lowest column index
    rows, cols = 16, 4096
    g = torch.Generator(device="cpu").manual_seed(9)
    W = (torch.randint(-3, 4, (rows, cols), generator=g).float() * 0.25).to(
        torch.float32 if dtype == "f32" else torch.bfloat16).to(DEV)
    W[3] = 0.5                                          # a fully tied row
    ones = torch.ones(cols, dtype=torch.float32, device=DEV)
    for k in (1, 5, 1000, 2048, 4095):
        out, mask = run_prune(W, ones, k)
        ref_W, ref_mask = oracle.prune_unstructured(host(W), ones.cpu().numpy(), k, dtype)
        assert_bits_equal(host(out), ref_W)
        assert_bits_equal(mask.cpu().numpy().view(np.uint32), ref_mask)
    m = mask.cpu().numpy().view(np.uint32)[3]
    bits = ((m[:, None] >> np.arange(32, dtype=np.uint32)) & 1).reshape(-1)
    assert (bits[:4095] == 0).all() and bits[4095] == 1


def test_prune_in_place_nested_and_deterministic():
    rows, cols = 128, 4096
    W = make(rows, cols, "bf16", seed=11, heavy=True)
    norms = norms_for(cols, 4)
    prev = None
    for k in (400, 1200, 2048, 2900):
        out, mask = run_prune(W, norms, k)
        out2, mask2 = run_prune(W, norms, k)
        assert torch.equal(out.view(torch.int16), out2.view(torch.int16)) and torch.equal(mask, mask2)
        kept = mask.cpu().numpy().view(np.uint32)
        assert (np.unpackbits(kept.view(np.uint8), axis=1).sum(1) == cols - k).all()     # exact per-row sparsity
        if prev is not None:
            assert ((kept & ~prev) == 0).all()                                           # masks nested in k
        prev = kept
    Wc = W.clone()
    inp, mask3 = run_prune(Wc, norms, 2900, inplace=True)
    assert torch.equal(inp.view(torch.int16), out.view(torch.int16)) and torch.equal(mask3, mask)


def test_prune_writes_only_its_outputs():
    rows, cols = 16, 1000
    buf = torch.full((rows + 2, 1008), 3.0, dtype=torch.bfloat16, device=DEV)
    W = make(rows, cols, "bf16", seed=12, ld=1008)
    out = buf[1:rows + 1, :cols]
    words = (cols + 31) // 32
    mbuf = torch.full((rows + 2, words), 0x5A5A5A5A, dtype=torch.int32, device=DEV)
    api.mosaic_prune_unstructured(W, out, norms_for(cols, 5), 500, mbuf[1:rows + 1])
    assert (buf[0] == 3.0).all() and (buf[-1] == 3.0).all() and (buf[:, cols:] == 3.0).all()     # canaries intact
    assert (mbuf[0] == 0x5A5A5A5A).all() and (mbuf[-1] == 0x5A5A5A5A).all()


def _check_prune(W, norms, k, dtype):
    out, mask = run_prune(W, norms, k)
    ref_W, ref_mask = oracle.prune_unstructured(host(W), norms.cpu().numpy(), k, dtype)
    assert_bits_equal(host(out), ref_W)
    assert_bits_equal(mask.cpu().numpy().view(np.uint32), ref_mask)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("rows,cols", [(2500, 4096), (1300, 5120), (700, 11008), (640, 14336)])
def test_prune_many_rows_per_cta(dtype, rows, cols):
    # more rows than resident CTAs: every CTA carries its threshold estimate from row to row
    W = make(rows, cols, dtype, seed=rows + cols, heavy=False)
    norms = norms_for(cols, 31)
    for k in (cols // 2, cols // 10):
        _check_prune(W, norms, k, dtype)


@pytest.mark.parametrize("cols", [2048, 2056, 2560, 3072, 3584, 4104, 5120, 5128, 6152, 7168, 8192, 8200, 10248, 11264, 11272,
                                  12296, 13824, 14336, 16384, 16392])
def test_prune_bf16_every_cta_shape_with_a_ragged_last_vector_slot(cols):
    # one row length per shape of the row-group kernel (1, 2, 4 or 8 warps per row; 8 ... 20 vectors per thread) and
    # just past each limit, so that some threads own vector slots beyond the end of the row; 16392 columns is beyond
    # the kernel and takes the general one.  Single and batched calls.
    rows = 700
    W = make(rows, cols, "bf16", seed=cols, heavy=(cols % 16 == 0))
    norms = norms_for(cols, cols % 97)
    for k in (cols // 2, 1, cols - 1):
        _check_prune(W, norms, k, "bf16")
    k = (3 * cols) // 10
    out = torch.full_like(W, 3.0)
    mask = torch.full((rows, (cols + 31) // 32), -1, dtype=torch.int32, device=DEV)
    api.mosaic_prune_unstructured_batch([(W, out, norms, k, mask)])
    ref_W, ref_mask = oracle.prune_unstructured(host(W), norms.cpu().numpy(), k, "bf16")
    assert_bits_equal(host(out), ref_W)
    assert_bits_equal(mask.cpu().numpy().view(np.uint32), ref_mask)


@pytest.mark.parametrize("dtype,rows,cols", [("bf16", 300, 4096), ("bf16", 90, 11008), ("bf16", 40, 688), ("f32", 64, 1000),
                                             ("bf16", 50, 16392)])
def test_prune_mask_only_mode(dtype, rows, cols):
    # W_out == NULL: the keep bitmask is the only output, the input stays as it was
    W = make(rows, cols, dtype, seed=rows + cols, heavy=True)
    before = W.clone()
    norms = norms_for(cols, 44)
    for k in (0, cols // 2, cols - 1):
        ref_W, ref_mask = oracle.prune_unstructured(host(W), norms.cpu().numpy(), k, dtype)
        mask = torch.full((rows, (cols + 31) // 32), -1, dtype=torch.int32, device=DEV)
        api.mosaic_prune_unstructured(W, None, norms, k, mask)
        assert_bits_equal(mask.cpu().numpy().view(np.uint32), ref_mask)
        mask2 = torch.full_like(mask, -1)
        api.mosaic_prune_unstructured_batch([(W, None, norms, k, mask2)])
        assert_bits_equal(mask2.cpu().numpy().view(np.uint32), ref_mask)
        assert torch.equal(W.view(torch.int16 if dtype == "bf16" else torch.int32),
                           before.view(torch.int16 if dtype == "bf16" else torch.int32))
    L = api.lib()
    rc = L.mosaic_prune_unstructured(W.data_ptr(), None, rows, cols, W.stride(0), api.BF16 if dtype == "bf16" else api.F32,
                                     norms.data_ptr(), 1, None, None, 0, None)
    assert rc == -2                                     # no output at all: refused


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_prune_rows_of_very_different_scale(dtype):
    # consecutive rows of a CTA differ by orders of magnitude, some are constant, some all zero,
    # some half zero: the carried estimate is useless and every fallback of the selection runs
    rows, cols = 3000, 4096
    W = make(rows, cols, dtype, seed=77, heavy=True).clone()
    g = torch.Generator(device="cpu").manual_seed(78)
    scale = torch.exp2(torch.randint(-20, 21, (rows, 1), generator=g).float()).to(DEV)
    W = (W.float() * scale).to(W.dtype)
    W[5::97] = 0.0
    W[7::89] = 0.125
    W[11::83, ::2] = 0.0
    W[13::79, 100:] = -3.0
    norms = norms_for(cols, 32)
    for k in (1, 1500, 2048, 4000, 4096):
        _check_prune(W, norms, k, dtype)


@pytest.mark.parametrize("cols", [4096, 11008])
def test_prune_thresholds_across_and_beyond_the_window(cols):
    # rows of one matrix scaled by factors that rise smoothly over +-8 %: their thresholds sweep through the
    # matrix's whole window of score keys, sit on its edges and fall just outside it (the kernel's window holds
    # about +-3 sigma of the rank scatter of equally scaled rows, a few per cent in score)
    rows = 640 if cols == 4096 else 320
    W = make(rows, cols, "bf16", seed=cols + 5)
    scale = (1.0 + 0.16 * (torch.arange(rows, device=DEV).float() / rows - 0.5))[:, None]
    W = (W.float() * scale).to(torch.bfloat16)
    for norms in (norms_for(cols, 51), torch.full((cols,), 37.5, dtype=torch.float32, device=DEV)):
        for k in (cols // 2, (3 * cols) // 10):
            _check_prune(W, norms, k, "bf16")
            out = torch.full_like(W, 3.0)
            mask = torch.full((rows, (cols + 31) // 32), -1, dtype=torch.int32, device=DEV)
            api.mosaic_prune_unstructured_batch([(W, out, norms, k, mask)])
            ref_W, ref_mask = oracle.prune_unstructured(host(W), norms.cpu().numpy(), k, "bf16")
            assert_bits_equal(host(out), ref_W)
            assert_bits_equal(mask.cpu().numpy().view(np.uint32), ref_mask)


def test_prune_already_pruned_matrix():
    # half of every row is exactly zero (a matrix pruned before): thousands of tied keys at +0
    rows, cols = 1200, 4096
    W = make(rows, cols, "bf16", seed=91)
    norms = norms_for(cols, 33)
    half, _ = run_prune(W, norms, 2048)
    half = half.contiguous()
    for k in (100, 2047, 2048, 2049, 3000):
        _check_prune(half, norms, k, "bf16")


def _adversarial_norms(case, cols):
    """Norm vectors that reach the corners of the selection: columns whose scores are all zero,
    subnormal, near overflow, infinite or NaN, and norms on and next to powers of two."""
    g = torch.Generator(device="cpu").manual_seed(len(case) + cols)
    n = norms_for(cols, 41).cpu()
    if case == "zeros":
        n[::3] = 0.0                                   # every score of these columns is +0: ties by column
    elif case == "all_zero":
        n[:] = 0.0
    elif case == "tiny":
        n[0::5], n[1::5], n[2::5] = 2.0 ** -110, 2.0 ** -101, 2.0 ** -100
    elif case == "huge":
        n[0::5], n[1::5], n[2::5] = 2.0 ** 110, 2.0 ** 101, 2.0 ** 100
    elif case == "subnormal_scores":
        n[:] = (torch.rand(cols, generator=g) + 0.5) * 2.0 ** -122      # every score is an fp32 subnormal or zero
    elif case == "overflowing_scores":
        n[:] = (torch.rand(cols, generator=g) + 0.5) * 2.0 ** 126       # large weights overflow to +inf: tied keys
    elif case == "inf":
        n[7::211] = float("inf")                       # inf * 0 = NaN for zero weights, +inf otherwise
    elif case == "nan":
        n[9::199] = float("nan")
        n[100] = float("inf")
    elif case == "pow2":
        e = torch.randint(-3, 9, (cols,), generator=g).float()
        n = torch.exp2(e)
        up = torch.nextafter(n, torch.full_like(n, 1e30))
        dn = torch.nextafter(n, torch.zeros_like(n))
        sel = torch.randint(0, 3, (cols,), generator=g)
        n = torch.where(sel == 0, n, torch.where(sel == 1, up, dn))
    else:
        raise KeyError(case)
    return n.to(torch.float32).to(DEV)


@pytest.mark.parametrize("case", ["zeros", "all_zero", "tiny", "huge", "subnormal_scores", "overflowing_scores", "inf", "nan",
                                  "pow2"])
@pytest.mark.parametrize("cols", [2048, 4096, 11008])
def test_prune_bf16_adversarial_norms(case, cols):
    rows = 96 if cols < 8192 else 40
    W = make(rows, cols, "bf16", seed=cols + len(case), heavy=True).clone()
    W[3, ::2] = 0.0                                    # zero weights meet the infinite norms
    W[5] = W[5].abs() * 512.0                          # a row of large weights
    norms = _adversarial_norms(case, cols)
    Wh, nh = host(W), norms.cpu().numpy()
    for k in (cols // 2, cols // 10, cols - cols // 10):
        ref_W, ref_mask = oracle.prune_unstructured(Wh, nh, k, "bf16")
        out, mask = run_prune(W, norms, k)                                           # windows sampled row by row
        assert_bits_equal(host(out), ref_W)
        assert_bits_equal(mask.cpu().numpy().view(np.uint32), ref_mask)
        out2 = torch.full_like(W, 3.0)
        mask2 = torch.full((rows, (cols + 31) // 32), -1, dtype=torch.int32, device=DEV)
        api.mosaic_prune_unstructured_batch([(W, out2, norms, k, mask2)])             # windows planned per matrix
        assert_bits_equal(host(out2), ref_W)
        assert_bits_equal(mask2.cpu().numpy().view(np.uint32), ref_mask)


@pytest.mark.parametrize("spread", [0.0, 0.004, 0.03])
def test_prune_bf16_scores_crowded_around_the_threshold(spread):
    # every score of a row within a few bf16 steps of every other: all weights are candidates of any
    # window (more than a warp's queue holds) and single histogram bins hold hundreds of equal keys
    rows, cols = 64, 4096
    g = torch.Generator(device="cpu").manual_seed(int(spread * 1000))
    W = ((1.0 + spread * torch.rand(rows, cols, generator=g)) * 0.5).to(torch.bfloat16).to(DEV)
    W[::2] = -W[::2]
    ones = torch.ones(cols, dtype=torch.float32, device=DEV)
    norms = norms_for(cols, 43)
    for nrm in (ones, norms):
        for k in (1, 700, 2048, 4000):
            _check_prune(W, nrm, k, "bf16")
    out = torch.full_like(W, 3.0)
    mask = torch.full((rows, cols // 32), -1, dtype=torch.int32, device=DEV)
    api.mosaic_prune_unstructured_batch([(W, out, ones, 1500, mask)])
    ref_W, ref_mask = oracle.prune_unstructured(host(W), ones.cpu().numpy(), 1500, "bf16")
    assert_bits_equal(host(out), ref_W)
    assert_bits_equal(mask.cpu().numpy().view(np.uint32), ref_mask)


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_prune_batch_matches_oracle_job_by_job(dtype):
    # several projections of different shapes in one call: rows long enough for the bf16-domain
    # kernel (planned from three sample rows), short ones, k = 0 and k = cols, one job in place
    shapes = [(700, 4096, 2048), (300, 4096, 400), (260, 11008, 5504), (50, 688, 300), (40, 4096, 0), (33, 4096, 4096),
              (500, 4096, 3000), (128, 5120, 2560), (1, 4096, 2048)]
    jobs, refs = [], []
    for i, (rows, cols, k) in enumerate(shapes):
        W = make(rows, cols, dtype, seed=500 + i, heavy=(i % 2 == 0))
        if i == 6:
            W = (W.float() * torch.exp2(torch.arange(rows, device=DEV).remainder(9).float() - 4.0)[:, None]).to(W.dtype)
        norms = norms_for(cols, 40 + i)
        ref_W, ref_mask = oracle.prune_unstructured(host(W), norms.cpu().numpy(), k, dtype)
        out = W if i == 3 else torch.full_like(W, 7.0)
        mask = None if i == 1 else torch.full((rows, (cols + 31) // 32), -1, dtype=torch.int32, device=DEV)
        jobs.append((W, out, norms, k, mask))
        refs.append((ref_W, ref_mask))
    api.mosaic_prune_unstructured_batch(jobs)
    for (W, out, norms, k, mask), (ref_W, ref_mask) in zip(jobs, refs):
        assert_bits_equal(host(out), ref_W)
        if mask is not None:
            assert_bits_equal(mask.cpu().numpy().view(np.uint32), ref_mask)


def test_prune_batch_reused_with_new_counts():
    # one marshalled job list run three times with different per-row prune counts (k = 0 <-> k > 0 changes
    # which kernel a job takes and how much workspace the call needs)
    shapes = [(300, 4096), (120, 11008), (64, 688), (200, 8192)]
    Ws = [make(r, c, "bf16", seed=900 + i, heavy=(i == 1)) for i, (r, c) in enumerate(shapes)]
    norms = [norms_for(c, 70 + i) for i, (r, c) in enumerate(shapes)]
    outs = [torch.empty_like(W) for W in Ws]
    masks = [torch.empty(r, (c + 31) // 32, dtype=torch.int32, device=DEV) for r, c in shapes]
    batch = api.PruneBatch([(W, o, n, 0, m) for W, o, n, m in zip(Ws, outs, norms, masks)])
    ws = api.Workspace(DEV)
    for ks in ([0, 0, 0, 0], [2048, 5504, 300, 4096], [1000, 0, 688, 8191], [2048, 5504, 300, 4096]):
        for o, m in zip(outs, masks):
            o.fill_(7.0)
            m.fill_(-1)
        batch.run(ks, ws)
        for W, o, n, m, k in zip(Ws, outs, norms, masks, ks):
            ref_W, ref_mask = oracle.prune_unstructured(host(W), n.cpu().numpy(), k, "bf16")
            assert_bits_equal(host(o), ref_W)
            assert_bits_equal(m.cpu().numpy().view(np.uint32), ref_mask)


def test_outlier_batch_reused():
    shapes = [(300, 4096), (64, 688), (130, 11008)]
    Ws = [make(r, c, "bf16", seed=950 + i, heavy=True) for i, (r, c) in enumerate(shapes)]
    norms = [norms_for(c, 80 + i) for i, (r, c) in enumerate(shapes)]
    counts = torch.full((len(shapes),), -5, dtype=torch.int64, device=DEV)
    batch = api.OutlierBatch([(W, n, counts[i:i + 1], None) for i, (W, n) in enumerate(zip(Ws, norms))])
    ws = api.Workspace(DEV)
    for alpha in (5.0, 2.0, 5.0):
        batch.run(alpha, ws)
        got = counts.cpu().tolist()
        for i, (W, n) in enumerate(zip(Ws, norms)):
            ref = oracle.outlier_ratio(host(W), n.cpu().numpy(), alpha, "bf16")
            assert ref["certified"] and got[i] == ref["count"], (alpha, i)


# ------------------------------------------------------------------ structured
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("rows,cols,rg,cg,fr,fc", [(256, 688, 1, 1, 0.3, 0.3), (512, 1024, 64, 1, 0.25, 0.5),
                                                   (96, 4096, 1, 128, 0.1, 0.25), (1000, 520, 1, 1, 0.5, 0.1),
                                                   (64, 64, 1, 1, 0.0, 0.0)])
def test_structured_compact(dtype, rows, cols, rg, cg, fr, fc):
    W = make(rows, cols, dtype, seed=rows + cols + rg, heavy=True)
    norms = norms_for(cols, 6)
    Wh, nh = host(W), norms.cpu().numpy()
    n_ru, n_cu = rows // rg, cols // cg
    keep_r, keep_c = n_ru - int(fr * n_ru), n_cu - int(fc * n_cu)
    for use_norms in (True, False):
        rk = torch.full((keep_r,), -1, dtype=torch.int32, device=DEV)
        ck = torch.full((keep_c,), -1, dtype=torch.int32, device=DEV)
        out = torch.empty(keep_r * rg, keep_c * cg, dtype=W.dtype, device=DEV)
        sc = torch.empty(n_ru + n_cu, dtype=torch.float32, device=DEV)
        api.mosaic_prune_structured_compact(W, norms if use_norms else None, rg, cg, keep_r, keep_c, rk, ck, 0, out, sc)
        rs_ref, cs_ref = oracle.unit_scores(Wh, nh if use_norms else None, rg, cg, dtype)
        sc_h = sc.cpu().numpy()
        np.testing.assert_allclose(sc_h[:n_ru], rs_ref, rtol=REL)
        np.testing.assert_allclose(sc_h[n_ru:], cs_ref, rtol=REL)
        # bit-equal wherever no order of the fp64 additions can move the fp32 rounding (one step off at most elsewhere)
        r_ok, c_ok = oracle.unit_scores_certify(Wh, nh if use_norms else None, rg, cg, dtype)
        rs_ref = op.reconcile_fp32(rs_ref, sc_h[:n_ru], r_ok)
        cs_ref = op.reconcile_fp32(cs_ref, sc_h[n_ru:], c_ok)
        rk_ref, ck_ref = oracle.rank_units(rs_ref, keep_r), oracle.rank_units(cs_ref, keep_c)
        assert_bits_equal(rk.cpu().numpy(), rk_ref)
        assert_bits_equal(ck.cpu().numpy(), ck_ref)
        assert out.shape == (keep_r * rg, keep_c * cg)
        assert_bits_equal(host(out), oracle.compact(Wh, rk_ref, ck_ref, rg, cg, dtype))


def test_structured_given_lists_and_score_accumulation():
    # coupled MLP channel pruning: rows of gate and up and columns of down share one keep list,
    # ranked by the sum of the three unit scores
    hidden, inter = 256, 688
    gate, up = make(inter, hidden, "bf16", 21, heavy=True), make(inter, hidden, "bf16", 22, heavy=True)
    down = make(hidden, inter, "bf16", 23, heavy=True)
    n_in, n_mid = norms_for(hidden, 7), norms_for(inter, 8)
    tot = torch.zeros(inter, dtype=torch.float32, device=DEV)
    s_gate = torch.zeros(inter + hidden, dtype=torch.float32, device=DEV)
    s_up = torch.zeros_like(s_gate)
    s_down = torch.zeros(hidden + inter, dtype=torch.float32, device=DEV)
    api.mosaic_prune_structured_compact(gate, n_in, 1, 1, 0, 0, None, None, api.SCORES_ONLY, None, s_gate)
    api.mosaic_prune_structured_compact(up, n_in, 1, 1, 0, 0, None, None, api.SCORES_ONLY | api.SCORES_ACCUM, None, s_gate)
    api.mosaic_prune_structured_compact(down, n_mid, 1, 1, 0, 0, None, None, api.SCORES_ONLY, None, s_down)
    g_r, _ = oracle.unit_scores(host(gate), n_in.cpu().numpy(), 1, 1, "bf16")
    u_r, _ = oracle.unit_scores(host(up), n_in.cpu().numpy(), 1, 1, "bf16")
    _, d_c = oracle.unit_scores(host(down), n_mid.cpu().numpy(), 1, 1, "bf16")
    assert_bits_equal(s_gate[:inter].cpu().numpy(), g_r + u_r)                          # fp32 add, same order
    total = (s_gate[:inter] + s_down[hidden:]).contiguous()
    total_ref = (g_r + u_r) + d_c
    assert_bits_equal(total.cpu().numpy(), total_ref)
    keep = inter - int(0.2 * inter)
    ch = torch.empty(keep, dtype=torch.int32, device=DEV)
    api.mosaic_rank_units(total, keep, ch)
    ch_ref = oracle.rank_units(total_ref, keep)
    assert_bits_equal(ch.cpu().numpy(), ch_ref)
    allh = torch.arange(hidden, dtype=torch.int32, device=DEV)
    g_out = torch.empty(keep, hidden, dtype=torch.bfloat16, device=DEV)
    d_out = torch.empty(hidden, keep, dtype=torch.bfloat16, device=DEV)
    api.mosaic_prune_structured_compact(gate, None, 1, 1, keep, hidden, ch, allh, api.ROWS_GIVEN | api.COLS_GIVEN, g_out)
    api.mosaic_prune_structured_compact(down, None, 1, 1, hidden, keep, allh, ch, api.ROWS_GIVEN | api.COLS_GIVEN, d_out)
    assert_bits_equal(host(g_out), host(gate)[ch_ref])
    assert_bits_equal(host(d_out), host(down)[:, ch_ref])
    del tot, s_up


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_structured_batched_calls_match_the_oracle(dtype):
    # several matrices of different shapes and unit sizes through each batched step, against the oracle step by step
    shapes = [(256, 688, 1, 1), (512, 1024, 64, 1), (96, 4096, 1, 128), (1000, 520, 1, 1), (300, 1000, 1, 8), (64, 64, 1, 1)]
    Ws, norms, refs = [], [], []
    for i, (rows, cols, rg, cg) in enumerate(shapes):
        ld = cols if cols % 8 == 0 else (cols + 7) // 8 * 8
        W = make(rows, cols, dtype, seed=700 + i, ld=ld, heavy=True)
        n = norms_for(cols, 90 + i) if i % 2 == 0 else None
        Ws.append(W)
        norms.append(n)
    rs = [torch.full((r // rg,), -1.0, dtype=torch.float32, device=DEV) for r, c, rg, cg in shapes]
    cs = [torch.full((c // cg,), -1.0, dtype=torch.float32, device=DEV) for r, c, rg, cg in shapes]
    jobs = [(W, n, rg, cg, rs[i] if i != 4 else None, cs[i]) for i, (W, n, (r, c, rg, cg)) in enumerate(zip(Ws, norms, shapes))]
    api.mosaic_unit_scores_batch(jobs)
    agreed = []
    for i, (W, n, (rows, cols, rg, cg)) in enumerate(zip(Ws, norms, shapes)):
        nh = None if n is None else n.cpu().numpy()
        r_ref, c_ref = oracle.unit_scores(host(W), nh, rg, cg, dtype)
        r_ok, c_ok = oracle.unit_scores_certify(host(W), nh, rg, cg, dtype)
        c_ag = op.reconcile_fp32(c_ref, cs[i].cpu().numpy(), c_ok)
        if i != 4:
            r_ag = op.reconcile_fp32(r_ref, rs[i].cpu().numpy(), r_ok)
        else:
            assert (rs[i] == -1.0).all()                         # a NULL output is left alone
            r_ag = r_ref
        agreed.append((r_ag, c_ag))
    # sums of coupled scores: dst = a + b in fp32, dst may be a
    tot = rs[0].clone()
    api.mosaic_add_unit_scores_batch([(tot, tot, rs[0]), (cs[5], cs[5], rs[5])])
    assert_bits_equal(tot.cpu().numpy(), agreed[0][0] + agreed[0][0])
    assert_bits_equal(cs[5].cpu().numpy(), agreed[5][1] + agreed[5][0])
    # ranking of every list in one launch
    fr = [0.3, 0.25, 0.1, 0.5, 0.2, 0.0]
    keep_r = [len(a[0]) - int(f * len(a[0])) for a, f in zip(agreed, fr)]
    keep_c = [len(a[1]) - int(f * len(a[1])) for a, f in zip(agreed, fr)]
    sc_r = [torch.from_numpy(a[0]).to(DEV) for a in agreed]
    sc_c = [torch.from_numpy(a[1]).to(DEV) for a in agreed]
    rk = [torch.full((k,), -1, dtype=torch.int32, device=DEV) for k in keep_r]
    ck = [torch.full((k,), -1, dtype=torch.int32, device=DEV) for k in keep_c]
    api.mosaic_rank_units_batch([(s, k, o) for s, k, o in zip(sc_r + sc_c, keep_r + keep_c, rk + ck)])
    for i, a in enumerate(agreed):
        assert_bits_equal(rk[i].cpu().numpy(), oracle.rank_units(a[0], keep_r[i]))
        assert_bits_equal(ck[i].cpu().numpy(), oracle.rank_units(a[1], keep_c[i]))
    # compaction of every matrix in one launch (staged gather, whole vectors of a column unit, whole rows)
    outs = [torch.full((keep_r[i] * rg, keep_c[i] * cg), 7.0, dtype=Ws[i].dtype, device=DEV) for i, (r, c, rg, cg) in enumerate(shapes)]
    api.mosaic_compact_batch([(Ws[i], rk[i], keep_r[i], rg, ck[i], keep_c[i], cg, outs[i]) for i, (r, c, rg, cg) in enumerate(shapes)])
    for i, (rows, cols, rg, cg) in enumerate(shapes):
        ref = oracle.compact(host(Ws[i]), rk[i].cpu().numpy(), ck[i].cpu().numpy(), rg, cg, dtype)
        assert_bits_equal(host(outs[i]), ref)


def test_rank_units_ties_and_sizes():
    for n, keep in [(8, 7), (50, 20), (1024, 1000), (14336, 11469), (5000, 1), (3000, 3000)]:
        g = torch.Generator(device="cpu").manual_seed(n)
        s = torch.rand(n, generator=g)
        s[::7] = s[0]                        # ties
        sd = s.to(DEV)
        out = torch.empty(keep, dtype=torch.int32, device=DEV)
        api.mosaic_rank_units(sd, keep, out)
        assert_bits_equal(out.cpu().numpy(), oracle.rank_units(s.numpy(), keep))
