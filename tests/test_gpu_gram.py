"""GPU parity of mosaic_gram_accumulate (second moments of a projection's input, the matrix the
inverse-Hessian back-end of Section 4.1.2 is built from) against the fp64 oracle.

The kernel sums exact bf16 products in fp32 on the tensor cores, so parity is a tolerance, derived
from the arithmetic: every 16-token MMA step adds 16 exact products to the running sum and
truncates - allow 2 units in the last place of the largest operand, i.e. 2^-22 of
sum_t |x_tj| |x_tl| (which the oracle returns beside the sum) per step - plus the rounded add into G.
Observed on sums of one sign (the diagonal): about a quarter of that, always low.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2504_06323_b200 import api, workloads as wl

pytestmark = pytest.mark.gpu
DEV = "cuda"
ERR_INVALID_ARG, ERR_NULL_PTR, ERR_BAD_DTYPE, ERR_MISALIGNED, ERR_ALIASING = -1, -2, -3, -4, -6   # include/mosaic.h


def bound(tokens_per_call, calls, G_abs):
    return (tokens_per_call / 4.0 + 2.0) * calls * 2.0 ** -24 * G_abs


def synth(tokens, cols, seed, outliers=True):
    g = torch.Generator(device=DEV).manual_seed(seed)
    X = torch.randn(tokens, cols, generator=g, device=DEV, dtype=torch.float32)
    if outliers and cols >= 16:
        X[:, torch.randperm(cols, generator=g, device=DEV)[: max(1, cols // 200)]] *= 100.0   # outlier channels
    return X.to(torch.bfloat16)


def run(X, G=None, flags=api.RESET_ACCUM):
    cols = X.shape[1]
    if G is None:
        G = torch.full((cols, cols), float("nan"), device=DEV, dtype=torch.float32)
    status = torch.full((1,), 7, device=DEV, dtype=torch.int32)
    api.mosaic_gram_accumulate(X, G, flags, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0, "a bounded wait of the kernel ran out"
    return G


@pytest.mark.parametrize("tokens,cols", [(300, 520), (64, 256), (1, 8), (129, 264), (1000, 768)])
def test_gram_whole_matrix_against_oracle(tokens, cols):
    X = synth(tokens, cols, seed=tokens * 7 + cols)
    G = run(X).cpu().numpy()
    ref, ref_abs = oracle.gram(wl.to_numpy(X), None, "bf16", with_abs=True)
    assert np.isfinite(G).all()
    assert (np.abs(G - ref) <= bound(tokens, 1, ref_abs) + 1e-30).all()
    assert np.array_equal(G, G.T)                      # both triangles hold the same bits
    # diag(G) is the squared norm of Eq. 5
    ss = oracle.act_sumsq(wl.to_numpy(X), None, "bf16")
    assert np.allclose(np.diag(G), ss, rtol=(tokens / 4.0 + 2.0) * 2.0 ** -24)


def test_gram_accumulates_over_chunks_and_respects_ld():
    tokens, cols = 700, 328
    wide = synth(tokens, cols + 24, seed=3)
    X = wide[:, :cols]                                  # leading dimension 352 > cols
    G = run(X[:256])                                    # reset
    run(X[256:320], G, 0)
    run(X[320:], G, 0)
    Xh = np.ascontiguousarray(wl.to_numpy(wide)[:, :cols])
    ref, ref_abs = oracle.gram(Xh, None, "bf16", with_abs=True)
    assert (np.abs(G.cpu().numpy() - ref) <= bound(380, 3, ref_abs)).all()
    # G inside a wider buffer: only [cols, cols] is touched
    buf = torch.full((cols, cols + 12), -3.0, device=DEV, dtype=torch.float32)
    run(X, buf[:, :cols])
    assert (buf[:, cols:] == -3.0).all()
    assert (np.abs(buf[:, :cols].cpu().numpy() - ref) <= bound(tokens, 1, ref_abs)).all()


def test_gram_exact_cases():
    # powers of two: every partial sum is exact in fp32, so the result must equal the oracle's bit for bit
    tokens, cols = 512, 272
    g = torch.Generator(device=DEV).manual_seed(5)
    e = torch.randint(-3, 4, (tokens, cols), generator=g, device=DEV)
    sgn = torch.randint(0, 2, (tokens, cols), generator=g, device=DEV) * 2 - 1
    X = (sgn * torch.pow(2.0, e.float())).to(torch.bfloat16)
    G = run(X).cpu().numpy()
    ref = oracle.gram(wl.to_numpy(X), None, "bf16")
    assert np.array_equal(G.astype(np.float64), ref)
    # no tokens: reset gives zeros, accumulate leaves G alone
    Z = run(X[:0])
    assert (Z == 0).all()
    keep = torch.full((cols, cols), 2.5, device=DEV)
    run(X[:0], keep, 0)
    assert (keep == 2.5).all()


def test_gram_many_blocks_sampled_pairs():
    """cols = 1280 (5 blocks, 15 of them computed), 8192 tokens: pairs across every block border."""
    tokens, cols = 8192, 1280
    X = synth(tokens, cols, seed=9)
    G = run(X).cpu().numpy()
    rng = np.random.default_rng(0)
    edge = np.array([0, 1, 127, 128, 255, 256, 257, 511, 512, 1023, 1024, 1279])
    js = np.concatenate([np.repeat(edge, len(edge)), rng.integers(0, cols, 3000)])
    ls = np.concatenate([np.tile(edge, len(edge)), rng.integers(0, cols, 3000)])
    ref, ref_abs = oracle.gram_pairs(wl.to_numpy(X), js, ls, "bf16")
    assert (np.abs(G[js, ls] - ref) <= bound(tokens, 1, ref_abs)).all()
    assert np.array_equal(G, G.T)


def test_gram_llama_width_sampled_pairs():
    """One projection input at the LLaMA-7B width, 32768 calibration tokens in two calls."""
    cfg = wl.CONFIGS["llama7b"]
    X = wl.gen_activation(cfg, 0, cfg.x_keys()[0], DEV, tokens=32768)
    tokens, cols = X.shape
    assert cols == 4096
    G = run(X[:16384])
    run(X[16384:], G, 0)
    G = G.cpu().numpy()
    rng = np.random.default_rng(1)
    js = np.concatenate([np.arange(0, cols, 97), rng.integers(0, cols, 2000)])
    ls = np.concatenate([np.arange(0, cols, 97), rng.integers(0, cols, 2000)])      # the first part is the diagonal
    ref, ref_abs = oracle.gram_pairs(wl.to_numpy(X), js, ls, "bf16")
    assert (np.abs(G[js, ls] - ref) <= bound(16384, 2, ref_abs)).all()
    assert np.array_equal(G[:512, 2048:2560], G[2048:2560, :512].T)


def test_gram_full_size_widest_input_sampled_pairs():
    """The widest projection input of the LLaMA-7B shape (11008 channels) at the full calibration
    size (262144 tokens), accumulated the way the benchmark does it (calls of 32768 tokens)."""
    from paper_2504_06323_b200 import driver
    cfg = wl.CONFIGS["llama7b"]
    X = wl.gen_activation(cfg, 0, "mlp_mid", DEV)
    tokens, cols = X.shape
    assert (tokens, cols) == (262144, 11008)
    G = torch.empty(cols, cols, device=DEV)
    status = torch.zeros(1, device=DEV, dtype=torch.int32)
    n = driver.accumulate_second_moments(G, X, reset=True, status=status, chunk_tokens=32768)
    torch.cuda.synchronize()
    assert n == 8 and int(status.item()) == 0
    rng = np.random.default_rng(2)
    js = np.concatenate([np.array([0, 255, 256, 11007, 10752, 5000]), rng.integers(0, cols, 300)])
    ls = np.concatenate([np.array([0, 256, 255, 11007, 17, 5000]), rng.integers(0, cols, 300)])
    Gs = G[torch.from_numpy(js).to(DEV), torch.from_numpy(ls).to(DEV)].cpu().numpy()
    Gt = G[torch.from_numpy(ls).to(DEV), torch.from_numpy(js).to(DEV)].cpu().numpy()
    ref, ref_abs = oracle.gram_pairs(wl.to_numpy(X), js, ls, "bf16")
    assert (np.abs(Gs - ref) <= bound(32768, 8, ref_abs)).all()
    assert np.array_equal(Gs, Gt)


def test_bounded_wait_gives_up_and_reports():
    """The mbarrier wait every role of the kernel uses, alone, on a barrier nothing completes: it must
    return after its cycle budget (2e6 cycles, about a millisecond) with the error word raised, and the
    context must stay usable."""
    import time
    status = torch.full((1,), 7, device=DEV, dtype=torch.int32)
    t0 = time.perf_counter()
    api.mosaic_bounded_wait_selftest(2_000_000, status)
    torch.cuda.synchronize()
    assert time.perf_counter() - t0 < 5.0
    assert int(status.item()) == 1
    # the context is intact: a regular call still works
    X = synth(64, 64, seed=2)
    G = run(X)
    assert torch.isfinite(G).all()
    L = api.lib()
    assert L.mosaic_bounded_wait_selftest(0, status.data_ptr(), None) == ERR_INVALID_ARG
    assert L.mosaic_bounded_wait_selftest(3_000_000_000, status.data_ptr(), None) == ERR_INVALID_ARG
    assert L.mosaic_bounded_wait_selftest(1000, None, None) == ERR_NULL_PTR


def test_gram_argument_errors():
    L = api.lib()
    X = synth(64, 64, seed=1)
    G = torch.zeros(64, 64, device=DEV)
    args = lambda **kw: [kw.get("X", X.data_ptr()), kw.get("tokens", 64), kw.get("cols", 64), kw.get("ldx", 64), kw.get("dtype", api.BF16),
                         kw.get("G", G.data_ptr()), kw.get("ldg", 64), 0, None, None]
    assert L.mosaic_gram_accumulate(*args(dtype=api.F32)) == ERR_BAD_DTYPE
    assert L.mosaic_gram_accumulate(*args(G=None)) == ERR_NULL_PTR
    assert L.mosaic_gram_accumulate(*args(G=G.data_ptr() + 4)) == ERR_MISALIGNED
    assert L.mosaic_gram_accumulate(*args(ldg=62)) == ERR_INVALID_ARG
    assert L.mosaic_gram_accumulate(*args(cols=60, ldx=64)) == ERR_INVALID_ARG
    both = torch.zeros(64 * 64 * 2, device=DEV, dtype=torch.float32)
    assert L.mosaic_gram_accumulate(*args(X=both.data_ptr(), G=both.data_ptr() + 64)) == ERR_ALIASING
