"""Randomised GPU parity: seeded draws of shapes, prune counts, weight and norm distributions and
output modes for the unstructured prune, of unit groups and keep lists for the compaction, and of
token counts and widths for the second moments - each case compared with the oracle (bits for the
first two, the fp32 bound for the third).  The fixed cases elsewhere cover the paper's shapes; this
file walks the ground between them (row lengths of every group size of the selection kernel,
k = 1 and cols - 1, tie-heavy and already sparse rows, zero and many-octave norms, ragged widths)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2504_06323_b200 import api, workloads as wl

pytestmark = pytest.mark.gpu
DEV = "cuda"


def rand_weights(rng, rows, cols, kind):
    g = torch.Generator(device=DEV).manual_seed(int(rng.integers(1 << 30)))
    if kind == "t3":            # the workloads' heavy-tailed weights
        z = torch.randn(4, rows, cols, generator=g, device=DEV)
        W = 0.02 * z[0] / torch.sqrt((z[1] ** 2 + z[2] ** 2 + z[3] ** 2) / 3) / 3 ** 0.5
    elif kind == "ties":        # thirteen distinct values: most scores of a column pair are equal
        W = torch.randint(-6, 7, (rows, cols), generator=g, device=DEV).float() * 0.0078125
    elif kind == "sparse":      # half of the weights already zero
        W = torch.randn(rows, cols, generator=g, device=DEV) * 0.02
        W = W * (torch.rand(rows, cols, generator=g, device=DEV) > 0.5)
    else:                       # rows of very different scale
        W = torch.randn(rows, cols, generator=g, device=DEV) * 0.02 * torch.exp(torch.randn(rows, 1, generator=g, device=DEV))
    return W.to(torch.bfloat16)


def rand_norms(rng, cols, kind):
    g = torch.Generator(device=DEV).manual_seed(int(rng.integers(1 << 30)))
    if kind == "spread":
        n = torch.rand(cols, generator=g, device=DEV) * 500 + 100
    elif kind == "equal":
        n = 512.0 * (1 + 0.002 * torch.randn(cols, generator=g, device=DEV))
    elif kind == "ones":
        n = torch.ones(cols, device=DEV)
    elif kind == "zeros":       # a third of the channels never fired
        n = (torch.rand(cols, generator=g, device=DEV) * 10) * (torch.rand(cols, generator=g, device=DEV) > 0.3)
    else:                       # many octaves
        n = torch.exp(torch.randn(cols, generator=g, device=DEV) * 6)
    if kind in ("spread", "equal"):
        n[torch.randperm(cols, generator=g, device=DEV)[: max(1, cols // 200)]] *= 100
    return n.float()


@pytest.mark.parametrize("seed", [0, 1, 2])
def test_prune_unstructured_random_cases(seed):
    rng = np.random.default_rng(100 + seed)
    for _ in range(40):
        cols = int(rng.choice([2048, 2056, 3072, 4096, 4104, 5120, 6144, 8192, 8200, 11008, 13824, 14336, 16384,
                               int(rng.integers(256, 2048)) * 8]))
        rows = int(rng.integers(20, 300))
        k = int(rng.choice([1, cols - 1, cols // 2, int(rng.integers(1, cols)), int(cols * rng.choice([0.1, 0.3, 0.7]))]))
        wk = str(rng.choice(["t3", "ties", "sparse", "scales"]))
        nk = str(rng.choice(["spread", "equal", "ones", "zeros", "octaves"]))
        mode = int(rng.integers(3))
        W, n = rand_weights(rng, rows, cols, wk), rand_norms(rng, cols, nk)
        ref_W, ref_m = oracle.prune_unstructured(wl.to_numpy(W), n.cpu().numpy(), k, "bf16")
        m = torch.full((rows, (cols + 31) // 32), -1, dtype=torch.int32, device=DEV)
        if mode == 0:           # separate output
            o = torch.full_like(W, 3.0)
            api.mosaic_prune_unstructured(W, o, n, k, m)
        elif mode == 1:         # in place
            o = W.clone()
            api.mosaic_prune_unstructured(o, o, n, k, m)
        else:                   # keep mask only
            o = None
            api.mosaic_prune_unstructured(W, None, n, k, m)
        torch.cuda.synchronize()
        case = dict(cols=cols, rows=rows, k=k, weights=wk, norms=nk, mode=mode)
        assert np.array_equal(m.cpu().numpy().view(np.uint32), ref_m), case
        assert o is None or np.array_equal(wl.to_numpy(o), ref_W), case


@pytest.mark.parametrize("seed", [0, 1])
def test_compact_random_cases(seed):
    rng = np.random.default_rng(200 + seed)
    for _ in range(60):
        rg = int(rng.choice([1, 1, 2]))
        cg = int(rng.choice([1, 1, 1, 2, 4, 8, 16]))
        rows = max(rg, int(rng.integers(3, 300)) // rg * rg)
        cols = int(rng.choice([int(rng.integers(1, 700)) * 8, 4096, 11008, int(rng.integers(8, 3000))]))
        cols = max(8 * cg, cols // (8 * cg) * (8 * cg))
        W = rand_weights(rng, rows, cols, "t3")
        n_ru, n_cu = rows // rg, cols // cg
        kr = int(rng.integers(1, n_ru + 1))
        kc = int(rng.choice([n_cu, int(rng.integers(1, n_cu + 1))]))
        rk = np.sort(rng.choice(n_ru, kr, replace=False)).astype(np.int32)
        ck = np.sort(rng.choice(n_cu, kc, replace=False)).astype(np.int32)
        out = torch.full((kr * rg, kc * cg), 9.0, dtype=torch.bfloat16, device=DEV)
        api.mosaic_compact_batch([(W, torch.from_numpy(rk).to(DEV), kr, rg, torch.from_numpy(ck).to(DEV), kc, cg, out)])
        torch.cuda.synchronize()
        ref = oracle.compact(wl.to_numpy(W), rk, ck, rg, cg, "bf16")
        assert np.array_equal(wl.to_numpy(out), ref), dict(rows=rows, cols=cols, rg=rg, cg=cg, kr=kr, kc=kc)


@pytest.mark.parametrize("seed", [0, 1])
def test_gram_random_cases(seed):
    rng = np.random.default_rng(300 + seed)
    torch.manual_seed(300 + seed)
    for _ in range(60):
        tokens, cols = int(rng.integers(0, 700)), int(rng.integers(1, 130)) * 8
        X = (torch.randn(max(tokens, 1), cols, device=DEV) * torch.exp(torch.randn(cols, device=DEV)))[:tokens].to(torch.bfloat16)
        G = torch.full((cols, cols), float("nan"), device=DEV)
        status = torch.zeros(1, dtype=torch.int32, device=DEV)
        api.mosaic_gram_accumulate(X, G, api.RESET_ACCUM, status)
        torch.cuda.synchronize()
        if tokens > 0:
            ref, ref_abs = oracle.gram(wl.to_numpy(X), None, "bf16", with_abs=True)
        else:
            ref = ref_abs = np.zeros((cols, cols))
        assert int(status.item()) == 0
        assert (np.abs(G.cpu().numpy() - ref) <= (tokens / 4.0 + 2.0) * 2.0 ** -24 * ref_abs + 1e-30).all(), dict(tokens=tokens, cols=cols)


@pytest.mark.parametrize("seed", [0, 1, 2])
def test_outlier_batch_random_cases(seed):
    """The batched call (one sweep with per-column ladders, count sweep as the fallback) over lists of
    random matrices, each with its own threshold or grouped: counts equal to the oracle's wherever it
    certifies them, sums within what the order of fp64 additions can move them."""
    rng = np.random.default_rng(400 + seed)
    for _ in range(6):
        n_jobs = int(rng.integers(1, 7))
        alpha = float(rng.choice([1.0, 2.5, 5.0, 9.0]))
        grouped = bool(rng.integers(2))
        Ws, ns = [], []
        for _j in range(n_jobs):
            rows = int(rng.choice([1, 7, 64, 65, 255, 256, 257, int(rng.integers(1, 1500))]))
            cols = int(rng.choice([8, 1024, 1032, 2048, 4096, int(rng.integers(1, 700)) * 8]))
            Ws.append(rand_weights(rng, rows, cols, str(rng.choice(["t3", "ties", "sparse", "scales"]))))
            ns.append(rand_norms(rng, cols, str(rng.choice(["spread", "equal", "ones", "zeros", "octaves"]))))
        counts = torch.full((n_jobs,), -3, dtype=torch.int64, device=DEV)
        sums = torch.full((n_jobs,), -1.0, dtype=torch.float64, device=DEV)
        jobs = [(W, n, counts[i:i + 1], sums[i:i + 1]) for i, (W, n) in enumerate(zip(Ws, ns))]
        if grouped:
            groups = np.sort(rng.integers(0, 3, n_jobs)).tolist()
            api.mosaic_outlier_ratio_grouped(jobs, groups, alpha)
        else:
            groups = list(range(n_jobs))
            api.mosaic_outlier_ratio_batch(jobs, alpha)
        torch.cuda.synchronize()
        got_c, got_s = counts.cpu().tolist(), sums.cpu().numpy()
        for g in sorted(set(groups)):
            idx = [i for i in range(n_jobs) if groups[i] == g]
            ref = oracle.outlier_ratio_group([wl.to_numpy(Ws[i]) for i in idx], [ns[i].cpu().numpy() for i in idx], alpha, "bf16")
            for pos, i in enumerate(idx):
                case = dict(seed=seed, shape=tuple(Ws[i].shape), alpha=alpha, grouped=grouped)
                own = oracle.outlier_ratio(wl.to_numpy(Ws[i]), ns[i].cpu().numpy(), alpha, "bf16")["sum"]   # a matrix's own score sum
                # another order of the fp64 additions: at most numel * 2^-53 of the sum of these non-negative terms
                assert abs(got_s[i] - own) <= Ws[i].numel() * 2.0 ** -52 * abs(own) + 1e-300 or not np.isfinite(own), case
                if ref["certified"]:
                    assert got_c[i] == ref["counts"][pos], case
