"""The whole path over a model, written with oracle calls only (test helper).

Mirrors what the product's driver does with library calls, so the two can be
compared output by output on the same seeded inputs.
"""
import numpy as np

import oracle
from paper_2504_06323_b200.workloads import PROJECTIONS


def phase_a(cfg, W, X, layers):
    """W[(layer, proj)], X[(layer, x_key)] numpy -> norms[(layer, x_key)], counts in (layer, proj) order."""
    dt = cfg.dtype
    norms, counts = {}, []
    for layer in layers:
        for xk in cfg.x_keys():
            norms[layer, xk] = oracle.act_norms(X[layer, xk], dt)
        for pr in PROJECTIONS:
            counts.append(oracle.outlier_ratio(W[layer, pr], norms[layer, cfg.x_key(pr)], cfg.alpha, dt)["count"])
    return norms, counts


def plan(cfg, counts, n_layers, p=None, lam=None, mode=0):
    numels, cols = [], []
    for _ in range(n_layers):
        for pr in PROJECTIONS:
            r, c = cfg.shape(pr)
            numels.append(r * c)
            cols.append(c)
    return oracle.allocate_sparsity(counts, numels, cols, n_layers, len(PROJECTIONS), cfg.p if p is None else p,
                                    cfg.lam if lam is None else lam, mode)


def unstructured(cfg, W, norms, layer, k):
    out = {}
    for m, pr in enumerate(PROJECTIONS):
        out[pr] = oracle.prune_unstructured(W[layer, pr], norms[layer, cfg.x_key(pr)], int(k[layer * len(PROJECTIONS) + m]),
                                            cfg.dtype)
    return out


def structured_coupled(cfg, src, norms, layer, frac, use_norms=True, scores=None):
    """src[proj] numpy matrices of one layer -> compacted matrices + keep lists (coupled units).
    `scores(proj, row_group, col_group) -> (row_scores, col_scores)` replaces the oracle's unit
    scores where a caller has reconciled them (units whose fp32 rounding depends on the order of
    the fp64 additions); ranking and compaction are the oracle's either way."""
    dt = cfg.dtype
    nrm = {pr: (norms[layer, cfg.x_key(pr)] if use_norms else None) for pr in PROJECTIONS}
    hd, n_kv = cfg.head_dim, cfg.n_kv_heads
    n_rep = cfg.n_heads // n_kv
    h, it = cfg.hidden, cfg.intermediate

    class _U:   # oracle.unit_scores, or the caller's reconciled scores
        @staticmethod
        def unit_scores(W, n, rg, cg, dtype, pr):
            return oracle.unit_scores(W, n, rg, cg, dtype) if scores is None else scores(pr, rg, cg)
    g_r, _ = _U.unit_scores(src["gate"], nrm["gate"], 1, 1, dt, "gate")
    u_r, _ = _U.unit_scores(src["up"], nrm["up"], 1, 1, dt, "up")
    _, d_c = _U.unit_scores(src["down"], nrm["down"], 1, 1, dt, "down")
    total = (g_r + u_r) + d_c                                   # fp32 adds, in this order
    ch = oracle.rank_units(total, it - int(frac * it))
    all_h = np.arange(h, dtype=np.int32)
    out = {"W": {}, "mlp_keep": ch}
    out["W"]["gate"] = oracle.compact(src["gate"], ch, all_h, 1, 1, dt)
    out["W"]["up"] = oracle.compact(src["up"], ch, all_h, 1, 1, dt)
    out["W"]["down"] = oracle.compact(src["down"], all_h, ch, 1, 1, dt)
    gq = n_rep * hd
    q_r, _ = _U.unit_scores(src["q"], nrm["q"], gq, 1, dt, "q")
    k_r, _ = _U.unit_scores(src["k"], nrm["k"], hd, 1, dt, "k")
    v_r, _ = _U.unit_scores(src["v"], nrm["v"], hd, 1, dt, "v")
    _, o_c = _U.unit_scores(src["o"], nrm["o"], 1, gq, dt, "o")
    tot_a = (q_r + (k_r + v_r)) + o_c
    grp = oracle.rank_units(tot_a, n_kv - int(frac * n_kv))
    out["attn_keep"] = grp
    out["W"]["q"] = oracle.compact(src["q"], grp, all_h, gq, 1, dt)
    out["W"]["k"] = oracle.compact(src["k"], grp, all_h, hd, 1, dt)
    out["W"]["v"] = oracle.compact(src["v"], grp, all_h, hd, 1, dt)
    out["W"]["o"] = oracle.compact(src["o"], all_h, grp, 1, gq, dt)
    return out


def reconcile_fp32(ref, got, ok):
    """fp32 values rounded once from an fp64 sum (norms, unit scores) that the two sides must agree
    on: the oracle's where it certifies that no order of the fp64 additions can move the fp32
    rounding (there `got` must be bit-equal), the compared side's elsewhere (there it must be a
    neighbouring fp32 value at most).  Everything downstream (scores, rankings, masks) is then
    computed by the oracle from this one array, so both sides decide on the same numbers."""
    ref, got = np.asarray(ref, np.float32), np.asarray(got, np.float32)
    assert ref.shape == got.shape == ok.shape
    assert np.array_equal(ref[ok].view(np.uint32), got[ok].view(np.uint32)), "certified values differ"
    if not ok.all():
        d = np.abs(ref[~ok].view(np.int32).astype(np.int64) - got[~ok].view(np.int32).astype(np.int64))
        assert (d <= 1).all(), "uncertified value is more than one fp32 step away"
    out = ref.copy()
    out[~ok] = got[~ok]
    return out


def structured_independent(cfg, Wm, nrm, frac):
    rows, cols = Wm.shape
    rs, cs = oracle.unit_scores(Wm, nrm, 1, 1, cfg.dtype)
    rk = oracle.rank_units(rs, rows - int(frac * rows))
    ck = oracle.rank_units(cs, cols - int(frac * cols))
    return oracle.compact(Wm, rk, ck, 1, 1, cfg.dtype), rk, ck
