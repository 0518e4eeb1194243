"""GPU parity at the stated sizes of the LLaMA-shaped workload configurations: ONE whole
layer of each, at the configuration's own shapes and calibration token count, every output
compared with the CPU oracle element by element.

  * activation norms of every projection input at the full token count (128 x 2048, or 64 x 2048
    for the compaction stress), certified against summation order, bit-equal;
  * outlier counts of all seven projections from THOSE norms, through the batched call;
  * the allocation;
  * every row of every projection through the batched unstructured call (the 13B shape at
    10/30/50/70 % with nested masks);
  * the composite path at the GQA shapes (14336 MLP channels, 8 KV groups, 20 % structured after
    50 % unstructured) with coupled units;
  * independent row + column compaction of every projection at 10/30/50 %.

One activation tensor is resident at a time (2 - 7 GB), so the largest layer fits easily.
"""
import numpy as np
import pytest
import torch

import oracle
import oracle_pipeline as op
from paper_2504_06323_b200 import api, driver, workloads as wl
from paper_2504_06323_b200.workloads import PROJECTIONS

pytestmark = pytest.mark.gpu
DEV = "cuda"
LAYER = 0


def bits_equal(a, b):
    a, b = np.ascontiguousarray(a), np.ascontiguousarray(b)
    return a.shape == b.shape and a.dtype == b.dtype and np.array_equal(a.view(np.uint8), b.view(np.uint8))


def phase_a_full_layer(name):
    """Norms (full token count) and outlier counts of one layer, GPU vs oracle.  Returns the
    model state, the host copies of the weights, the oracle norms and the counts."""
    cfg = wl.scaled(wl.CONFIGS[name], n_layers=1)
    st = driver.alloc_model(cfg, DEV)
    norms_ref = {}
    for xk in cfg.x_keys():
        x = wl.gen_activation(cfg, LAYER, xk, DEV)                      # [tokens, cols] at the full token count
        assert x.shape[0] == wl.CONFIGS[name].tokens
        # two unequal chunks through the accumulating call, the second one finalises
        cut = (x.shape[0] // 3) | 1
        api.mosaic_act_norms(x[:cut], st.sumsq[LAYER, xk], None, api.RESET_ACCUM, st.ws)
        api.mosaic_act_norms(x[cut:], st.sumsq[LAYER, xk], st.norms[LAYER, xk], 0, st.ws)
        torch.cuda.synchronize()
        xh = wl.to_numpy(x)
        del x
        ss_ref = oracle.act_sumsq(xh, None, cfg.dtype)
        n_ref = oracle.norm_finalize(ss_ref)
        ok = oracle.norm_certify(xh, cfg.dtype)
        del xh
        np.testing.assert_allclose(st.sumsq[LAYER, xk].cpu().numpy(), ss_ref, rtol=1e-12)
        got = st.norms[LAYER, xk].cpu().numpy()
        np.testing.assert_allclose(got, n_ref, rtol=1e-5)
        # bit-equal wherever no order of the fp64 additions can move the fp32 rounding; a column whose
        # sum sits within tokens*2^-52 of a rounding boundary (a handful at this token count) may come
        # out one fp32 step away and is then taken as the library has it, on both sides, downstream
        assert ok.mean() > 0.99
        norms_ref[LAYER, xk] = op.reconcile_fp32(n_ref, got, ok)
    Wh = {(LAYER, pr): wl.to_numpy(st.W[LAYER, pr]) for pr in PROJECTIONS}
    driver.count_outliers_all(st)
    counts = driver.exchange_counts(st.counts, 1, 0, 1)
    for m, pr in enumerate(PROJECTIONS):
        ref = oracle.outlier_ratio(Wh[LAYER, pr], norms_ref[LAYER, cfg.x_key(pr)], cfg.alpha, cfg.dtype)
        assert ref["certified"], (name, pr)
        assert counts[m] == ref["count"] and ref["count"] > 0, (name, pr)
    return cfg, st, Wh, norms_ref, counts


def check_unstructured_layer(cfg, st, Wh, norms_ref, counts, p, prev=None):
    """Allocation + every row of the layer through the batched call, against the oracle."""
    s, k, infeasible = driver.plan_sparsity(cfg, counts, p=p)
    s_ref, k_ref, inf_ref = op.plan(cfg, counts, 1, p=p)
    assert np.array_equal(np.array(s).view(np.uint64), s_ref.view(np.uint64)) and list(k) == list(k_ref)
    assert infeasible == inf_ref and abs(np.mean(s) - p) < 1e-12
    for key in st.W_out:
        st.W_out[key].fill_(3.0)
        st.mask[key].fill_(-1)
    driver.prune_unstructured_all(st, k)
    torch.cuda.synchronize()
    ref = op.unstructured(cfg, Wh, norms_ref, LAYER, k_ref)
    masks = {}
    for m, pr in enumerate(PROJECTIONS):
        rows, cols = cfg.shape(pr)
        assert bits_equal(wl.to_numpy(st.W_out[LAYER, pr]), ref[pr][0]), (cfg.name, pr, p)
        mk = st.mask[LAYER, pr].cpu().numpy().view(np.uint32)
        assert bits_equal(mk, ref[pr][1]), (cfg.name, pr, p)
        assert (np.unpackbits(mk.view(np.uint8), axis=1).sum(1) == cols - int(k[m])).all()   # exact per-row sparsity
        if prev is not None:
            assert ((mk & ~prev[pr]) == 0).all(), (cfg.name, pr, p)                          # nested in p
        masks[pr] = mk
    return k, masks


def test_llama7b_layer_unstructured():
    cfg, st, Wh, norms_ref, counts = phase_a_full_layer("llama7b")
    check_unstructured_layer(cfg, st, Wh, norms_ref, counts, cfg.p)


def test_llama2_13b_layer_unstructured_sweep():
    cfg, st, Wh, norms_ref, counts = phase_a_full_layer("llama2_13b")
    prev = None
    for p in cfg.extra["p_sweep"]:
        _, prev = check_unstructured_layer(cfg, st, Wh, norms_ref, counts, p, prev)


def agreed_unit_scores(W_dev, Wm, norms_dev, nrm, row_group, col_group, dtype):
    """(row_scores, col_scores) both sides rank on: the oracle's fp32 unit scores, bit-equal to the
    library's wherever the oracle certifies them against summation order; the few units whose fp64
    sum sits within n*2^-52 of an fp32 rounding boundary take the library's value, which must be
    the neighbouring fp32 number at most."""
    rows, cols = Wm.shape
    n_ru = rows // row_group
    sc = torch.empty(n_ru + cols // col_group, dtype=torch.float32, device=DEV)
    api.mosaic_prune_structured_compact(W_dev, norms_dev, row_group, col_group, 0, 0, None, None, api.SCORES_ONLY, None, sc)
    got = sc.cpu().numpy()
    rs, cs = oracle.unit_scores(Wm, nrm, row_group, col_group, dtype)
    r_ok, c_ok = oracle.unit_scores_certify(Wm, nrm, row_group, col_group, dtype)
    assert r_ok.mean() > 0.99 and c_ok.mean() > 0.99
    return op.reconcile_fp32(rs, got[:n_ru], r_ok), op.reconcile_fp32(cs, got[n_ru:], c_ok)


def test_llama3_8b_layer_composite():
    cfg, st, Wh, norms_ref, counts = phase_a_full_layer("llama3_8b")
    frac = cfg.extra["structured_frac"]
    k, _ = check_unstructured_layer(cfg, st, Wh, norms_ref, counts, cfg.p)
    masked = {pr: st.W_out[LAYER, pr] for pr in PROJECTIONS}
    got = driver.prune_structured_coupled_layer(st, LAYER, frac, source=masked)
    torch.cuda.synchronize()
    ref_u = op.unstructured(cfg, Wh, norms_ref, LAYER, k)
    src = {pr: ref_u[pr][0] for pr in PROJECTIONS}
    # the keep lists rest on fp32 unit scores: both sides rank on scores agreed unit by unit
    def scores(pr, rg, cg):
        return agreed_unit_scores(masked[pr], src[pr], st.norms[LAYER, cfg.x_key(pr)], norms_ref[LAYER, cfg.x_key(pr)],
                                  rg, cg, cfg.dtype)
    ref = op.structured_coupled(cfg, src, norms_ref, LAYER, frac, scores=scores)
    assert len(ref["mlp_keep"]) == cfg.intermediate - int(frac * cfg.intermediate) == 14336 - 2867
    assert len(ref["attn_keep"]) == cfg.n_kv_heads - int(frac * cfg.n_kv_heads) == 7
    assert bits_equal(got["mlp_keep"].cpu().numpy(), ref["mlp_keep"])
    assert bits_equal(got["attn_keep"].cpu().numpy(), ref["attn_keep"])
    for pr in PROJECTIONS:
        assert bits_equal(wl.to_numpy(got["W"][pr]), ref["W"][pr]), pr
    # the batched calls (scores, sums, ranking and compaction of all matrices in a launch or two each) give the same bits
    got_b = driver.prune_structured_model(st, frac, coupled=True, sources={LAYER: masked})[LAYER]
    torch.cuda.synchronize()
    assert bits_equal(got_b["mlp_keep"].cpu().numpy(), ref["mlp_keep"]) and bits_equal(got_b["attn_keep"].cpu().numpy(), ref["attn_keep"])
    for pr in PROJECTIONS:
        assert bits_equal(wl.to_numpy(got_b["W"][pr]), ref["W"][pr]), pr
    # zeros inside the compacted matrices are the mask's zeros restricted to the kept rows / columns
    ch = ref["mlp_keep"]
    assert bits_equal(wl.to_numpy(got["W"]["gate"]), src["gate"][ch])
    assert bits_equal(wl.to_numpy(got["W"]["down"]), src["down"][:, ch])


def test_llama7b_structured_layer_rows_and_columns():
    cfg, st, Wh, norms_ref, counts = phase_a_full_layer("llama7b_structured")
    assert cfg.tokens == 64 * 2048
    for pr in PROJECTIONS:
        Wm, nrm = Wh[LAYER, pr], norms_ref[LAYER, cfg.x_key(pr)]
        rows, cols = cfg.shape(pr)
        rs, cs = agreed_unit_scores(st.W[LAYER, pr], Wm, st.norms[LAYER, cfg.x_key(pr)], nrm, 1, 1, cfg.dtype)
        prev_r = prev_c = None
        for frac in sorted(cfg.extra["structured_sweep"], reverse=True):          # 50 %, 30 %, 10 %: keep sets grow
            out, rk, ck = driver.prune_structured_independent(st, LAYER, pr, frac)
            torch.cuda.synchronize()
            rk_ref = oracle.rank_units(rs, rows - int(frac * rows))
            ck_ref = oracle.rank_units(cs, cols - int(frac * cols))
            assert bits_equal(rk.cpu().numpy(), rk_ref) and bits_equal(ck.cpu().numpy(), ck_ref), (pr, frac)
            assert tuple(out.shape) == (rows - int(frac * rows), cols - int(frac * cols))
            assert bits_equal(wl.to_numpy(out), oracle.compact(Wm, rk_ref, ck_ref, 1, 1, cfg.dtype)), (pr, frac)
            if prev_r is not None:                                                  # nested keep sets
                assert set(prev_r.tolist()) <= set(rk_ref.tolist()) and set(prev_c.tolist()) <= set(ck_ref.tolist())
            prev_r, prev_c = rk_ref, ck_ref
    # all seven projections at once through the batched calls
    got = driver.prune_structured_model(st, 0.3, coupled=False)
    torch.cuda.synchronize()
    for pr in PROJECTIONS:
        out, rk, ck = driver.prune_structured_independent(st, LAYER, pr, 0.3)
        assert torch.equal(got[LAYER, pr][1], rk) and torch.equal(got[LAYER, pr][2], ck), pr
        assert bits_equal(wl.to_numpy(got[LAYER, pr][0]), wl.to_numpy(out)), pr
