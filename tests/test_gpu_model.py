"""GPU parity of the whole path over a model, driver vs oracle pipeline: the five
workload configurations (the tiny one at full size, the LLaMA-shaped ones scaled
down so the oracle finishes in seconds but every row still spans several tiles
and ragged tails)."""
import numpy as np
import pytest
import torch

import oracle
import oracle_pipeline as op
from paper_2504_06323_b200 import api, driver, workloads as wl
from paper_2504_06323_b200.workloads import PROJECTIONS

pytestmark = pytest.mark.gpu
DEV = "cuda"


def bits_equal(a, b):
    a, b = np.ascontiguousarray(a), np.ascontiguousarray(b)
    return a.shape == b.shape and a.dtype == b.dtype and np.array_equal(a.view(np.uint8), b.view(np.uint8))


def small(name, **kw):
    base = wl.CONFIGS[name]
    d = dict(n_layers=2, hidden=512, n_heads=8, n_kv_heads=8, head_dim=64, intermediate=1376, tokens=3000)
    d.update(kw)
    return wl.scaled(base, **d)


def run_phase_a(cfg):
    st = driver.alloc_model(cfg, DEV)
    Wh, Xh = {}, {}
    for layer in st.layers:
        X = driver.make_activations(cfg, layer, DEV)
        # two chunks through the accumulating call
        cut = cfg.tokens // 3
        driver.accumulate_norms(st, layer, {k: v[:cut] for k, v in X.items()}, first=True, last=False)
        driver.accumulate_norms(st, layer, {k: v[cut:] for k, v in X.items()}, first=False, last=True)
        driver.count_outliers(st, layer)
        for xk, x in X.items():
            Xh[layer, xk] = wl.to_numpy(x)
        for pr in PROJECTIONS:
            Wh[layer, pr] = wl.to_numpy(st.W[layer, pr])
    counts = driver.exchange_counts(st.counts, cfg.n_layers, 0, 1)
    norms_ref, counts_ref = op.phase_a(cfg, Wh, Xh, st.layers)
    for key, n in st.norms.items():
        ok = oracle.norm_certify(Xh[key], cfg.dtype)
        got = n.cpu().numpy()
        np.testing.assert_allclose(got, norms_ref[key], rtol=1e-5)
        assert ok.all(), "re-seed: a column sits on an fp32 rounding boundary"
        assert bits_equal(got, norms_ref[key])
    assert counts == counts_ref
    st.counts.fill_(-3)                     # and the batched call over every projection gives the same counts
    driver.count_outliers_all(st)
    assert driver.exchange_counts(st.counts, cfg.n_layers, 0, 1) == counts_ref
    return st, Wh, Xh, norms_ref, counts


@pytest.mark.parametrize("name,kw", [("tiny", None), ("llama7b", {}), ("llama2_13b", dict(hidden=640, n_heads=10, n_kv_heads=10,
                                                                                        intermediate=1728))])
def test_unstructured_model(name, kw):
    cfg = wl.CONFIGS[name] if kw is None else small(name, **kw)
    st, Wh, Xh, norms_ref, counts = run_phase_a(cfg)
    sweep = cfg.extra.get("p_sweep", (cfg.p,))
    prev = {}
    for p in sweep:
        s, k, infeasible = driver.plan_sparsity(cfg, counts, p=p)
        s_ref, k_ref, inf_ref = op.plan(cfg, counts, cfg.n_layers, p=p)
        assert np.array_equal(np.array(s).view(np.uint64), s_ref.view(np.uint64)) and list(k) == list(k_ref)
        assert infeasible == inf_ref
        assert abs(np.mean(s) - p) < 1e-12                      # targets average to p
        assert len(set(k)) > 1                                  # allocation is non-uniform
        for layer in st.layers:
            driver.prune_unstructured_layer(st, layer, k)
            ref = op.unstructured(cfg, Wh, norms_ref, layer, k_ref)
            for pr in PROJECTIONS:
                assert bits_equal(wl.to_numpy(st.W_out[layer, pr]), ref[pr][0]), (layer, pr)
                m = st.mask[layer, pr].cpu().numpy().view(np.uint32)
                assert bits_equal(m, ref[pr][1]), (layer, pr)
                if (layer, pr) in prev:
                    assert ((m & ~prev[layer, pr]) == 0).all()  # masks nested across the sweep
                prev[layer, pr] = m
        # the batched call over all projections must give the same bits
        for key in st.W_out:
            st.W_out[key].fill_(3.0)
            st.mask[key].fill_(-1)
        driver.prune_unstructured_all(st, k)
        for layer in st.layers:
            ref = op.unstructured(cfg, Wh, norms_ref, layer, k_ref)
            for pr in PROJECTIONS:
                assert bits_equal(wl.to_numpy(st.W_out[layer, pr]), ref[pr][0]), (layer, pr)
                assert bits_equal(st.mask[layer, pr].cpu().numpy().view(np.uint32), ref[pr][1]), (layer, pr)


@pytest.mark.parametrize("name,kw", [("tiny", None), ("llama3_8b", dict(hidden=640, n_heads=10, n_kv_heads=5, head_dim=64, intermediate=1728))])
def test_composite_model(name, kw):
    cfg = wl.CONFIGS[name] if kw is None else small(name, **kw)
    frac = cfg.extra.get("structured_frac", 0.2)
    st, Wh, Xh, norms_ref, counts = run_phase_a(cfg)
    _, k, _ = driver.plan_sparsity(cfg, counts)
    for layer in st.layers:
        driver.prune_unstructured_layer(st, layer, k)
        masked = {pr: st.W_out[layer, pr] for pr in PROJECTIONS}
        got = driver.prune_structured_coupled_layer(st, layer, frac, source=masked)
        ref_u = op.unstructured(cfg, Wh, norms_ref, layer, k)
        ref = op.structured_coupled(cfg, {pr: ref_u[pr][0] for pr in PROJECTIONS}, norms_ref, layer, frac)
        assert bits_equal(got["mlp_keep"].cpu().numpy(), ref["mlp_keep"])
        assert bits_equal(got["attn_keep"].cpu().numpy(), ref["attn_keep"])
        assert len(ref["mlp_keep"]) == cfg.intermediate - int(frac * cfg.intermediate)
        for pr in PROJECTIONS:
            assert bits_equal(wl.to_numpy(got["W"][pr]), ref["W"][pr]), (layer, pr)


@pytest.mark.parametrize("frac", [0.1, 0.3, 0.5])
def test_structured_independent_model(frac):
    cfg = small("llama7b_structured", n_layers=1)
    st, Wh, Xh, norms_ref, counts = run_phase_a(cfg)
    for pr in PROJECTIONS:
        out, rk, ck = driver.prune_structured_independent(st, 0, pr, frac)
        ref, rk_ref, ck_ref = op.structured_independent(cfg, Wh[0, pr], norms_ref[0, cfg.x_key(pr)], frac)
        assert bits_equal(rk.cpu().numpy(), rk_ref) and bits_equal(ck.cpu().numpy(), ck_ref)
        rows, cols = cfg.shape(pr)
        assert tuple(out.shape) == (rows - int(frac * rows), cols - int(frac * cols))
        assert bits_equal(wl.to_numpy(out), ref)


def test_full_size_rows_sampled_against_oracle():
    # the headline launch configuration: full LLaMA-7B projection shapes, checked on sampled rows
    cfg = wl.CONFIGS["llama7b"]
    for pr in ("q", "gate", "down"):
        rows, cols = cfg.shape(pr)
        W = wl.gen_weight(cfg, 0, pr, DEV)
        g = torch.Generator(device="cpu").manual_seed(rows + cols)
        norms = (torch.rand(cols, generator=g) * 500 + 100).to(DEV)
        norms[wl.outlier_columns(cfg, 0, cfg.x_key(pr), cols, cfg.x_outlier_frac).to(DEV)] *= 100
        out = torch.empty_like(W)
        mask = torch.empty(rows, (cols + 31) // 32, dtype=torch.int32, device=DEV)
        k = cols // 2
        api.mosaic_prune_unstructured(W, out, norms, k, mask)
        cnt = torch.zeros(1, dtype=torch.int64, device=DEV)
        ssum = torch.zeros(1, dtype=torch.float64, device=DEV)
        api.mosaic_outlier_ratio(W, norms, cfg.alpha, cnt, ssum)
        sample = torch.randperm(rows, generator=g)[:48].sort().values
        Ws, nh = wl.to_numpy(W[sample.to(DEV)]), norms.cpu().numpy()
        ref_W, ref_mask = oracle.prune_unstructured(Ws, nh, k, "bf16")
        assert bits_equal(wl.to_numpy(out[sample.to(DEV)]), ref_W)
        assert bits_equal(mask[sample.to(DEV)].cpu().numpy().view(np.uint32), ref_mask)
        # properties that hold at any size
        kept = mask.cpu().numpy().view(np.uint8)
        assert (np.unpackbits(kept, axis=1).sum(1) == cols - k).all()
        assert int((out == 0).sum().item()) >= rows * k
        ref = oracle.outlier_ratio(wl.to_numpy(W), nh, cfg.alpha, "bf16")     # whole matrix: a second or two
        assert ref["certified"] and cnt.item() == ref["count"]
        np.testing.assert_allclose(ssum.item(), ref["sum"], rtol=1e-12)


def test_full_size_batched_model_pass_sampled_against_oracle():
    # two full LLaMA-7B-shaped layers through the batched call, as the benchmark launches it:
    # sampled rows of every projection against the oracle, exact per-row sparsity everywhere
    cfg = wl.scaled(wl.CONFIGS["llama7b"], n_layers=2)
    st = driver.alloc_model(cfg, DEV)
    g = torch.Generator(device="cpu").manual_seed(5)
    for layer in st.layers:
        for xk in cfg.x_keys():
            c = cfg.x_cols(xk)
            n = (torch.rand(c, generator=g) * 500 + 100)
            n[wl.outlier_columns(cfg, layer, xk, c, cfg.x_outlier_frac)] *= 100
            st.norms[layer, xk].copy_(n)
    M = len(PROJECTIONS)
    k = [int(cfg.shape(pr)[1] * (0.42 + 0.02 * ((l * M + m) % 9))) for l in st.layers for m, pr in enumerate(PROJECTIONS)]
    driver.prune_unstructured_all(st, k)
    for layer in st.layers:
        for m, pr in enumerate(PROJECTIONS):
            rows, cols = cfg.shape(pr)
            kk = k[layer * M + m]
            sample = torch.randperm(rows, generator=g)[:24].sort().values.to(DEV)
            nh = st.norms[layer, cfg.x_key(pr)].cpu().numpy()
            ref_W, ref_mask = oracle.prune_unstructured(wl.to_numpy(st.W[layer, pr][sample]), nh, kk, "bf16")
            assert bits_equal(wl.to_numpy(st.W_out[layer, pr][sample]), ref_W), (layer, pr)
            assert bits_equal(st.mask[layer, pr][sample].cpu().numpy().view(np.uint32), ref_mask), (layer, pr)
            kept = st.mask[layer, pr].cpu().numpy().view(np.uint8)
            assert (np.unpackbits(kept, axis=1).sum(1) == cols - kk).all(), (layer, pr)


def test_norm_calls_on_side_streams_match_the_serial_order():
    # the same layers three ways: one stream, two side streams joined after every layer, joined once at the end
    cfg = small("llama7b", n_layers=3, tokens=2500)
    X = {layer: driver.make_activations(cfg, layer, DEV) for layer in range(cfg.n_layers)}
    results = []
    for mode in ("serial", "join_each", "join_last"):
        st = driver.alloc_model(cfg, DEV, outputs=False, masks=False)
        for n in st.norms.values():
            n.fill_(-1.0)
        for layer in st.layers:
            if mode == "serial":
                driver.accumulate_norms(st, layer, X[layer], overlap=False)
            else:
                driver.accumulate_norms(st, layer, X[layer], join=(mode == "join_each"))
        if mode == "join_last":
            driver.join_side(st)
        torch.cuda.current_stream().synchronize()      # the current stream alone: it must already cover the side streams
        results.append({k: v.cpu().numpy() for k, v in st.norms.items()})
    for key, ref in results[0].items():
        assert (ref > 0).all()
        assert bits_equal(results[1][key], ref) and bits_equal(results[2][key], ref), key


def test_structured_model_through_batched_calls_matches_layer_by_layer():
    cfg = small("llama3_8b", hidden=640, n_heads=10, n_kv_heads=5, head_dim=64, intermediate=1728, n_layers=5, tokens=1500)
    st = driver.alloc_model(cfg, DEV, outputs=False, masks=False)
    for layer in st.layers:
        driver.accumulate_norms(st, layer, driver.make_activations(cfg, layer, DEV))
    for rep in range(2):   # the second pass rebuilds the plan over the same matrices
        got = driver.prune_structured_model(st, 0.2, coupled=True)
        torch.cuda.current_stream().synchronize()
        for layer in st.layers:
            ref = driver.prune_structured_coupled_layer(st, layer, 0.2)
            assert torch.equal(got[layer]["mlp_keep"], ref["mlp_keep"]) and torch.equal(got[layer]["attn_keep"], ref["attn_keep"])
            for pr in PROJECTIONS:
                assert bits_equal(wl.to_numpy(got[layer]["W"][pr]), wl.to_numpy(ref["W"][pr])), (rep, layer, pr)
        got = driver.prune_structured_model(st, 0.3, coupled=False)
        torch.cuda.current_stream().synchronize()
        for layer in st.layers:
            for pr in PROJECTIONS:
                out, rk, ck = driver.prune_structured_independent(st, layer, pr, 0.3)
                g = got[layer, pr]
                assert torch.equal(g[1], rk) and torch.equal(g[2], ck)
                assert bits_equal(wl.to_numpy(g[0]), wl.to_numpy(out)), (rep, layer, pr)


def test_layer_pruning_baseline_model():
    # Eq. 3-4 / the layer method of Section 4.1.3: one outlier statistic and one target per layer
    cfg = small("llama7b", n_layers=3)
    st, Wh, Xh, norms_ref, _ = run_phase_a(cfg)
    driver.count_outliers_by_layer(st)
    counts = driver.exchange_counts(st.counts, cfg.n_layers, 0, 1)
    M = len(PROJECTIONS)
    layer_counts = []
    for layer in st.layers:
        ref = oracle.outlier_ratio_group([Wh[layer, pr] for pr in PROJECTIONS], [norms_ref[layer, cfg.x_key(pr)] for pr in PROJECTIONS],
                                         cfg.alpha, cfg.dtype)
        assert ref["certified"] and counts[layer * M:(layer + 1) * M] == ref["counts"]
        layer_counts.append(ref["count"])
    s, k, infeasible = driver.plan_sparsity_by_layer(cfg, counts, lam=0.15)
    per_layer = sum(r * c for r, c in (cfg.shape(pr) for pr in PROJECTIONS))
    min_cols = min(cfg.shape(pr)[1] for pr in PROJECTIONS)
    s_ref, _, inf_ref = oracle.allocate_sparsity(layer_counts, [per_layer] * cfg.n_layers, [min_cols] * cfg.n_layers, cfg.n_layers, 1,
                                                 cfg.p, 0.15)
    assert np.array_equal(np.array(s).view(np.uint64), s_ref.view(np.uint64)) and infeasible == inf_ref
    assert abs(np.mean(s) - cfg.p) < 1e-12 and len(set(s)) == cfg.n_layers          # one target per layer, mean p
    assert k == [int(np.floor(s_ref[n] * cfg.shape(pr)[1])) for n in range(cfg.n_layers) for pr in PROJECTIONS]
    driver.prune_unstructured_all(st, k)
    for layer in st.layers:
        ref = op.unstructured(cfg, Wh, norms_ref, layer, k)
        for pr in PROJECTIONS:
            assert bits_equal(wl.to_numpy(st.W_out[layer, pr]), ref[pr][0]), (layer, pr)
            assert bits_equal(st.mask[layer, pr].cpu().numpy().view(np.uint32), ref[pr][1]), (layer, pr)
