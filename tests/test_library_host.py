"""CPU-only checks of the C-ABI library: it loads, exports every symbol the
header declares, validates arguments before touching the device, and its host
function mosaic_allocate_sparsity agrees bit for bit with the oracle."""
import os
import re

import numpy as np
import pytest

import oracle
from paper_2504_06323_b200 import api, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build_library()
    return api.lib()


def header_symbols():
    text = open(os.path.join(ROOT, "include", "mosaic.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(mosaic_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = header_symbols()
    assert len(names) >= 12
    for n in names:
        assert hasattr(lib, n), n
    assert set(api.SYMBOLS) == set(names)
    assert lib.mosaic_version() == 100


def test_outlier_batch_workspace_holds_partials_and_ladders(lib):
    # per matrix: one fp64 partial per 64 x 1024 tile (256-byte aligned) + a bookkeeping block and
    # 32 counters of 4 bytes per column for the single-sweep count
    jobs = (api.OutlierJob * 2)()
    jobs[0].rows, jobs[0].cols = 4096, 4096
    jobs[1].rows, jobs[1].cols = 11008, 4096
    import ctypes as C
    got = lib.mosaic_outlier_ratio_batch_workspace_bytes(C.addressof(jobs), 2)
    want = 256
    for rows, cols in ((4096, 4096), (11008, 4096)):
        want += lib.mosaic_outlier_ratio_workspace_bytes(rows, cols)
        want += (256 + 128 * cols + 255) // 256 * 256
    assert got == want
    assert lib.mosaic_outlier_ratio_workspace_bytes(4096, 4096) == 8 * 64 * 4     # 64 bands x 4 chunks of doubles


def test_status_strings(lib):
    seen = set()
    for s in range(0, -11, -1):
        txt = api.status_string(s)
        assert txt and txt != "unknown status"
        seen.add(txt)
    assert len(seen) == 11
    assert api.status_string(-99) == "unknown status"


def test_argument_validation_needs_no_device(lib):
    # every one of these is rejected before any CUDA call is made
    assert lib.mosaic_act_norms(None, 4, 4, 4, 7, None, None, 0, None, 0, None) == -3       # bad dtype
    assert lib.mosaic_act_norms(None, 4, 4, 4, 0, None, None, 0, None, 0, None) == -2       # null accum
    assert lib.mosaic_score(None, 4, 4, 4, 1, None, None, None) == -2
    assert lib.mosaic_score(16, 4, 4, 3, 1, 16, 16, None) == -1                              # ld < cols
    assert lib.mosaic_score(8, 4, 8, 8, 1, 16, 16, None) == -4                               # misaligned base
    assert lib.mosaic_score(16, 4, 8, 12, 1, 16, 16, None) == -4                             # ld not 16 B multiple
    assert lib.mosaic_prune_unstructured(16, 16, 4, 8, 8, 1, 16, 9, None, None, 0, None) == -1   # k > cols
    assert lib.mosaic_prune_unstructured(16, 32, 4, 8, 8, 1, 16, 1, None, None, 0, None) == -6   # partial overlap
    assert lib.mosaic_outlier_ratio(16, 4, 8, 8, 1, 16, 5.0, 16, None, 256, 16, None) == -5      # workspace too small
    assert lib.mosaic_prune_structured_compact(16, 4, 8, 8, 1, None, 3, 1, 1, 1, 16, 16, 0, 4096, None, 256, 1 << 20,
                                               None) == -1                                   # rows % row_group
    assert lib.mosaic_rank_units(16, 4, 5, 16, None) == -1                                   # keep > n
    # mosaic_gram_accumulate(X, tokens, cols, ldx, dtype, G, ldg, flags, status, stream)
    assert lib.mosaic_gram_accumulate(16, 64, 64, 64, 0, 4096, 64, 0, None, None) == -3         # fp32 input: products not exact
    assert lib.mosaic_gram_accumulate(None, 64, 64, 64, 1, 4096, 64, 0, None, None) == -2        # tokens but no X
    assert lib.mosaic_gram_accumulate(16, 64, 64, 64, 1, None, 64, 0, None, None) == -2          # no G
    assert lib.mosaic_gram_accumulate(16, 64, 60, 64, 1, 1 << 20, 64, 0, None, None) == -1       # cols % 8
    assert lib.mosaic_gram_accumulate(16, 64, 64, 64, 1, 1 << 20, 60, 0, None, None) == -1       # ldg < cols
    assert lib.mosaic_gram_accumulate(16, 64, 64, 64, 1, (1 << 20) + 4, 64, 0, None, None) == -4  # G not 16-byte aligned
    assert lib.mosaic_gram_accumulate(16, 64, 64, 64, 1, 1 << 20, 64, 0, 6, None) == -4          # status word not 4-byte aligned
    assert lib.mosaic_gram_accumulate(1 << 20, 64, 64, 64, 1, (1 << 20) + 4096, 64, 0, None, None) == -6   # G inside X
    assert lib.mosaic_ratio_from_count(3, 200) == 1.5
    assert lib.mosaic_act_norms_workspace_bytes(262144, 4096) % 256 == 0


@pytest.mark.parametrize("mode", [api.GLOBAL_NORM, api.PER_CATEGORY_NORM, api.GLOBAL_NORM | api.WEIGHTED_MEAN,
                                  api.PER_CATEGORY_NORM | api.WEIGHTED_MEAN, api.REDISTRIBUTE,
                                  api.REDISTRIBUTE | api.WEIGHTED_MEAN, api.REDISTRIBUTE | api.PER_CATEGORY_NORM,
                                  api.REDISTRIBUTE | api.PER_CATEGORY_NORM | api.WEIGHTED_MEAN])
@pytest.mark.parametrize("p,lam", [(0.5, 0.08), (0.8, 0.15), (0.1, 0.0), (0.7, 0.3), (0.9, 0.6), (0.05, 0.5)])
def test_allocate_sparsity_bit_exact_vs_oracle(lib, mode, p, lam):
    rng = np.random.default_rng(42)
    for N, M in [(1, 7), (32, 7), (40, 7), (3, 2)]:
        numel = rng.integers(1 << 16, 1 << 26, N * M)
        O = (numel * rng.random(N * M) * 0.02).astype(np.int64)
        cols = rng.choice([256, 688, 4096, 5120, 11008, 14336], N * M)
        s_ref, k_ref, clamp_ref = oracle.allocate_sparsity(O, numel, cols, N, M, p, lam, mode)
        s, k, clamp = api.mosaic_allocate_sparsity(O, numel, cols, N, M, p, lam, mode)
        assert np.array_equal(np.array(s).view(np.uint64), s_ref.view(np.uint64))     # bit-exact fp64
        assert list(k) == list(k_ref) and clamp == clamp_ref


def test_allocate_sparsity_errors(lib):
    with pytest.raises(api.MosaicError):
        api.mosaic_allocate_sparsity([1], [10], [8], 1, 1, 1.0)          # p must be < 1
    with pytest.raises(api.MosaicError):
        api.mosaic_allocate_sparsity([11], [10], [8], 1, 1, 0.5)         # more outliers than elements
    s, k, infeasible = api.mosaic_allocate_sparsity([0, 50], [100, 100], [64, 64], 1, 2, 0.95, 0.2)
    assert infeasible and k[0] == 63


def test_binding_refuses_cpu_tensors(lib):
    import torch
    with pytest.raises(TypeError):
        api.mosaic_score(torch.zeros(4, 8), torch.zeros(8), torch.zeros(4, 8))
