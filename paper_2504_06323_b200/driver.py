"""Runs the pruning hot path over a whole LLaMA-shaped model.

Host-side orchestration only: it owns the device buffers (through torch),
decides the order of the library calls, moves the <= N*M outlier counts to the
host for the allocation, and - when several processes each own a share of the
layers - exchanges those counts.  All arithmetic happens inside the library.

Two phases separated by one tiny global dependency:
  phase A (per projection, independent): activation norms, outlier counts;
  host: every projection's count is needed before any target is known
        (normalize(R_LLM) ranks each projection against all others);
  phase B (per projection, independent): unstructured selection + zeroing,
        and / or structured ranking + compaction.
The phase-A result (counts) does not depend on the pruning target p, so one
calibration serves any number of targets.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np
import torch

from . import api
from .workloads import PROJECTIONS, ModelConfig, gen_activation, gen_weight


def layers_of_rank(n_layers: int, rank: int, world: int) -> list[int]:
    """Round-robin ownership of whole layers (coupled structured units stay inside a layer)."""
    return [l for l in range(n_layers) if l % world == rank]


def exchange_counts(local_counts: torch.Tensor, n_layers: int, rank: int, world: int, group=None) -> list[int]:
    """All ranks' outlier counts in global (layer, projection) order.

    local_counts: int64 [len(layers_of_rank) * M], host or device.  With world == 1
    this is only the device->host read.  Otherwise one all_gather of equal-sized int64
    blocks (layers are padded to the largest share) - the only data-path exchange.
    """
    M = len(PROJECTIONS)
    mine = layers_of_rank(n_layers, rank, world)
    assert local_counts.numel() == len(mine) * M
    if world == 1:
        return [int(v) for v in local_counts.cpu().tolist()]
    import torch.distributed as dist
    share = (n_layers + world - 1) // world
    block = torch.full((share * M,), -1, dtype=torch.int64, device=local_counts.device)
    block[: local_counts.numel()] = local_counts
    out = [torch.empty_like(block) for _ in range(world)]
    dist.all_gather(out, block, group=group)
    counts = [0] * (n_layers * M)
    for r in range(world):
        vals = out[r].cpu().tolist()
        for i, layer in enumerate(layers_of_rank(n_layers, r, world)):
            counts[layer * M:(layer + 1) * M] = [int(v) for v in vals[i * M:(i + 1) * M]]
    return counts


def plan_sparsity(cfg: ModelConfig, counts: list[int], p: float | None = None, lam: float | None = None,
                  mode: int = api.GLOBAL_NORM, n_layers: int | None = None):
    """normalize(R_LLM) + Projection Planner through the library's host call."""
    n_layers = cfg.n_layers if n_layers is None else n_layers
    shapes = [cfg.shape(pr) for pr in PROJECTIONS]
    numels = np.tile(np.array([r * c for r, c in shapes], dtype=np.int64), n_layers)
    cols = np.tile(np.array([c for _, c in shapes], dtype=np.int64), n_layers)
    return api.mosaic_allocate_sparsity(counts, numels, cols, n_layers, len(PROJECTIONS),
                                        cfg.p if p is None else p, cfg.lam if lam is None else lam, mode)


@dataclass
class ModelState:
    cfg: ModelConfig
    device: torch.device
    layers: list[int]                                  # global ids of the layers this process owns
    W: dict = field(default_factory=dict)              # (layer, proj) -> weights
    W_out: dict = field(default_factory=dict)          # (layer, proj) -> pruned weights
    mask: dict = field(default_factory=dict)           # (layer, proj) -> keep bitmask
    sumsq: dict = field(default_factory=dict)          # (layer, x_key) -> fp64 accumulator
    norms: dict = field(default_factory=dict)          # (layer, x_key) -> fp32 norms
    counts: torch.Tensor | None = None                 # int64 [len(layers)*M]
    ws: api.Workspace | None = None
    ws_batch: api.Workspace | None = None             # holds the plans of the batched pruning call
    batches: dict = field(default_factory=dict)        # name -> (identity of the tensors, marshalled batch)
    side: list | None = None                           # two (stream, workspace) pairs for independent calls

    def q_local(self, layer: int, proj: str) -> int:
        return self.layers.index(layer) * len(PROJECTIONS) + PROJECTIONS.index(proj)


def alloc_model(cfg: ModelConfig, device="cuda", layers: list[int] | None = None, outputs: bool = True,
                masks: bool = True, generate: bool = True) -> ModelState:
    """Allocate (and fill with the seeded synthetic weights) the buffers of the owned layers."""
    device = torch.device(device)
    st = ModelState(cfg, device, list(range(cfg.n_layers)) if layers is None else list(layers))
    st.ws = api.Workspace(device)
    st.counts = torch.zeros(len(st.layers) * len(PROJECTIONS), dtype=torch.int64, device=device)
    for layer in st.layers:
        for pr in PROJECTIONS:
            rows, cols = cfg.shape(pr)
            st.W[layer, pr] = gen_weight(cfg, layer, pr, device) if generate else \
                torch.empty(rows, cols, dtype=cfg.torch_dtype, device=device)
            if outputs:
                st.W_out[layer, pr] = torch.empty(rows, cols, dtype=cfg.torch_dtype, device=device)
            if masks:
                st.mask[layer, pr] = torch.empty(rows, (cols + 31) // 32, dtype=torch.int32, device=device)
        for xk in cfg.x_keys():
            c = cfg.x_cols(xk)
            st.sumsq[layer, xk] = torch.zeros(c, dtype=torch.float64, device=device)
            st.norms[layer, xk] = torch.empty(c, dtype=torch.float32, device=device)
    return st


def make_activations(cfg: ModelConfig, layer: int, device="cuda", tokens: int | None = None) -> dict:
    """One layer's calibration activations, one tensor per distinct projection input."""
    return {xk: gen_activation(cfg, layer, xk, device, tokens) for xk in cfg.x_keys()}


# ------------------------------------------------------------------ phase A
def accumulate_norms(st: ModelState, layer: int, X: dict, first: bool = True, last: bool = True,
                     overlap: bool = True, join: bool = True) -> int:
    """Add one chunk of calibration tokens per input; `last` also finalises the fp32 norms.
    Returns the number of library calls made.

    The inputs of a layer are independent, so with `overlap` their calls alternate between two side
    streams (each with a workspace of its own): the start-up and the finishing kernel of one input
    then run under the streaming of the next.  With `join` the current stream waits for both before
    returning; a caller that runs several layers in a row joins on the last one only (join_side())
    so that the layers overlap as well."""
    if not overlap or st.device.type != "cuda" or len(X) < 2:
        for xk, x in X.items():
            api.mosaic_act_norms(x, st.sumsq[layer, xk], st.norms[layer, xk] if last else None,
                                 api.RESET_ACCUM if first else 0, st.ws)
        return len(X)
    _side_streams(st, 2)
    need = max(api.lib().mosaic_act_norms_workspace_bytes(x.shape[0], x.shape[1]) for x in X.values())
    cur = torch.cuda.current_stream(st.device)
    fork = torch.cuda.Event()
    fork.record(cur)
    for s, ws in st.side[:2]:
        if ws.buf is None or ws.buf.numel() < need:   # grown before anything is in flight on the side stream
            s.synchronize()
            ws.get(need)
        s.wait_event(fork)
    for i, (xk, x) in enumerate(X.items()):
        s, ws = st.side[i % 2]
        api.mosaic_act_norms(x, st.sumsq[layer, xk], st.norms[layer, xk] if last else None,
                             api.RESET_ACCUM if first else 0, ws, stream=s)
    if join:
        join_side(st)
    return len(X)


def _side_streams(st: ModelState, n: int) -> list:
    """At least n (stream, workspace) pairs for calls that do not depend on one another."""
    if st.side is None:
        st.side = []
    while len(st.side) < n:
        st.side.append((torch.cuda.Stream(st.device), api.Workspace(st.device)))
    return st.side[:n]


def join_side(st: ModelState) -> None:
    """Make the current stream wait for everything issued on the side streams so far."""
    if st.side is None:
        return
    cur = torch.cuda.current_stream(st.device)
    for s, _ in st.side:
        done = torch.cuda.Event()
        done.record(s)
        cur.wait_event(done)


def count_outliers(st: ModelState, layer: int, alpha: float | None = None) -> int:
    cfg = st.cfg
    a = cfg.alpha if alpha is None else alpha
    for pr in PROJECTIONS:
        q = st.q_local(layer, pr)
        api.mosaic_outlier_ratio(st.W[layer, pr], st.norms[layer, cfg.x_key(pr)], a, st.counts[q:q + 1], None, st.ws)
    return len(PROJECTIONS)


def _cached_batch(st: ModelState, name: str, jobs: list, make):
    """The marshalled batch for `jobs`, rebuilt only when one of the tensors has been replaced."""
    ident = tuple(id(t) for job in jobs for t in job if isinstance(t, torch.Tensor))
    hit = st.batches.get(name)
    if hit is None or hit[0] != ident:
        hit = (ident, make(jobs))
        st.batches[name] = hit
    return hit[1]


def count_outliers_all(st: ModelState, alpha: float | None = None) -> int:
    """Outlier counts of every owned projection through the batched call (a handful of launches).  The job
    list is marshalled once and reused while the tensors of the ModelState stay the same objects."""
    cfg = st.cfg
    a = cfg.alpha if alpha is None else alpha
    if "count_views" not in st.batches or st.batches["count_views"][0] is not st.counts:
        st.batches["count_views"] = (st.counts, [st.counts[q:q + 1] for q in range(st.counts.numel())])
    views = st.batches["count_views"][1]
    jobs = [(st.W[layer, pr], st.norms[layer, cfg.x_key(pr)], views[st.q_local(layer, pr)], None)
            for layer in st.layers for pr in PROJECTIONS]
    if st.ws_batch is None:
        st.ws_batch = api.Workspace(st.device)
    _cached_batch(st, "outlier", jobs, api.OutlierBatch).run(a, st.ws_batch)
    return len(jobs)


def accumulate_second_moments(G: torch.Tensor, X: torch.Tensor, reset: bool = True, status: torch.Tensor | None = None,
                              chunk_tokens: int = 32768) -> int:
    """G (+)= X^T X over the tokens of X (fp32, both triangles): the second moments of a projection's
    input, from which the inverse-Hessian back-end forms H = (2/T) G.  `chunk_tokens` tokens per call:
    the fp32 error bound of a call grows with its tokens.  Returns the number of kernel launches.
    `status` (one int32) is overwritten by every call: check it after the last one only if the calls
    before cannot have failed, or pass chunk_tokens >= tokens."""
    tokens = X.shape[0]
    launches, first = 0, True
    for t0 in range(0, max(tokens, 1), chunk_tokens):
        api.mosaic_gram_accumulate(X[t0:t0 + chunk_tokens], G, api.RESET_ACCUM if (reset and first) else 0, status)
        first = False
        launches += 1 if tokens > 0 else 0
    return launches


def count_outliers_by_layer(st: ModelState, alpha: float | None = None) -> int:
    """Layer outlier distribution (Eq. 3-4, the layer-pruning baseline): every projection of a layer
    is counted against alpha times the mean score of the WHOLE layer.  st.counts receives the
    per-projection counts (their sum over a layer is the layer's outlier count)."""
    cfg = st.cfg
    a = cfg.alpha if alpha is None else alpha
    if "count_views" not in st.batches or st.batches["count_views"][0] is not st.counts:
        st.batches["count_views"] = (st.counts, [st.counts[q:q + 1] for q in range(st.counts.numel())])
    views = st.batches["count_views"][1]
    jobs = [(st.W[layer, pr], st.norms[layer, cfg.x_key(pr)], views[st.q_local(layer, pr)], None)
            for layer in st.layers for pr in PROJECTIONS]
    groups = [i for i, _ in enumerate(st.layers) for _ in PROJECTIONS]
    if st.ws_batch is None:
        st.ws_batch = api.Workspace(st.device)
    _cached_batch(st, "outlier", jobs, api.OutlierBatch).run(a, st.ws_batch, group_of=groups)
    return len(jobs)


def plan_sparsity_by_layer(cfg: ModelConfig, counts: list[int], p: float | None = None, lam: float | None = None,
                           mode: int = api.GLOBAL_NORM, n_layers: int | None = None):
    """One target per layer from the layers' outlier counts (normalize + planner over N entries, one
    "projection" per layer); every projection of layer n gets k = floor(s_n * cols).  Returns
    (s per layer, k per (layer, projection), infeasible)."""
    import math
    n_layers = cfg.n_layers if n_layers is None else n_layers
    M = len(PROJECTIONS)
    per_layer = sum(r * c for r, c in (cfg.shape(pr) for pr in PROJECTIONS))
    layer_counts = [sum(counts[n * M:(n + 1) * M]) for n in range(n_layers)]
    # the clamp bound needs a column count: the shortest row of the layer is the binding one
    min_cols = min(cfg.shape(pr)[1] for pr in PROJECTIONS)
    s, _, infeasible = api.mosaic_allocate_sparsity(layer_counts, [per_layer] * n_layers, [min_cols] * n_layers, n_layers, 1,
                                                    cfg.p if p is None else p, cfg.lam if lam is None else lam, mode)
    k = [int(math.floor(s[n] * cfg.shape(pr)[1])) for n in range(n_layers) for pr in PROJECTIONS]
    return s, k, infeasible


# ------------------------------------------------------------------ phase B
def prune_unstructured_layer(st: ModelState, layer: int, k_global: list[int], in_place: bool = False) -> int:
    cfg = st.cfg
    M = len(PROJECTIONS)
    for m, pr in enumerate(PROJECTIONS):
        W = st.W[layer, pr]
        out = W if in_place else st.W_out[layer, pr]
        api.mosaic_prune_unstructured(W, out, st.norms[layer, cfg.x_key(pr)], int(k_global[layer * M + m]),
                                      st.mask.get((layer, pr)), st.ws)
    return M


def prune_unstructured_all(st: ModelState, k_global: list[int], in_place: bool = False) -> int:
    """Phase B for every owned projection through the batched call: one planning launch and one
    pruning launch per distinct row length instead of one launch per projection.  The job list is
    marshalled once and reused, with the new prune counts, while the tensors of the ModelState stay
    the same objects.  Returns the number of jobs."""
    cfg = st.cfg
    M = len(PROJECTIONS)
    jobs = [(st.W[layer, pr], st.W[layer, pr] if in_place else st.W_out[layer, pr], st.norms[layer, cfg.x_key(pr)], 0,
             st.mask.get((layer, pr))) for layer in st.layers for pr in PROJECTIONS]
    if st.ws_batch is None:
        st.ws_batch = api.Workspace(st.device)
    ks = [int(k_global[layer * M + m]) for layer in st.layers for m in range(M)]
    _cached_batch(st, "prune_in_place" if in_place else "prune", jobs, api.PruneBatch).run(ks, st.ws_batch)
    return len(ks)


def _scores(W, norms, row_group, col_group, out, accumulate, ws):
    flags = api.SCORES_ONLY | (api.SCORES_ACCUM if accumulate else 0)
    api.mosaic_prune_structured_compact(W, norms, row_group, col_group, 0, 0, None, None, flags, None, out, ws)


def prune_structured_coupled_layer(st: ModelState, layer: int, frac: float, source: dict | None = None,
                                   use_norms: bool = True, ws: api.Workspace | None = None) -> dict:
    """Structured stage with the projections of a layer coupled the way the model's shapes require
    (Fig. "composite": nodes between projections are pruned as a group):
      * MLP channel c = row c of gate and up + column c of down, scored by the sum of the three;
      * attention unit = one KV head with its query heads: rows of q (n_rep*head_dim), k and v
        (head_dim), columns of o (n_rep*head_dim), scored by the sum of the four;
      * the hidden (residual) dimension is never removed.
    floor(frac * n_units) units are removed.  `source` gives the matrices to read (the masked
    weights in composite mode); returns {"W": {proj: compacted}, "mlp_keep", "attn_keep"}.
    """
    cfg, dev, ws = st.cfg, st.device, (st.ws if ws is None else ws)
    src = {pr: (source[pr] if source is not None else st.W[layer, pr]) for pr in PROJECTIONS}
    nrm = {pr: (st.norms[layer, cfg.x_key(pr)] if use_norms else None) for pr in PROJECTIONS}
    hd, n_kv = cfg.head_dim, cfg.n_kv_heads
    n_rep = cfg.n_heads // n_kv
    h, it = cfg.hidden, cfg.intermediate
    out: dict = {"W": {}}

    # MLP channels
    s_gu = torch.empty(it + h, dtype=torch.float32, device=dev)       # row units first, then column units
    s_d = torch.empty(h + it, dtype=torch.float32, device=dev)
    _scores(src["gate"], nrm["gate"], 1, 1, s_gu, False, ws)
    _scores(src["up"], nrm["up"], 1, 1, s_gu, True, ws)
    _scores(src["down"], nrm["down"], 1, 1, s_d, False, ws)
    total = s_gu[:it]                                                 # (gate + up) + down, fp32
    api.mosaic_sum_unit_scores(total, s_d[h:])
    keep_n = it - int(frac * it)
    ch = torch.empty(keep_n, dtype=torch.int32, device=dev)
    api.mosaic_rank_units(total, keep_n, ch)
    all_h = torch.arange(h, dtype=torch.int32, device=dev)
    given = api.ROWS_GIVEN | api.COLS_GIVEN
    for pr in ("gate", "up"):
        o = torch.empty(keep_n, h, dtype=cfg.torch_dtype, device=dev)
        api.mosaic_prune_structured_compact(src[pr], None, 1, 1, keep_n, h, ch, all_h, given, o, None, ws)
        out["W"][pr] = o
    o = torch.empty(h, keep_n, dtype=cfg.torch_dtype, device=dev)
    api.mosaic_prune_structured_compact(src["down"], None, 1, 1, h, keep_n, all_h, ch, given, o, None, ws)
    out["W"]["down"] = o
    out["mlp_keep"] = ch

    # attention KV groups
    gq = n_rep * hd
    s_q = torch.empty(n_kv + h, dtype=torch.float32, device=dev)
    s_k = torch.empty(n_kv + h, dtype=torch.float32, device=dev)
    s_o = torch.empty(h + n_kv, dtype=torch.float32, device=dev)
    _scores(src["q"], nrm["q"], gq, 1, s_q, False, ws)
    _scores(src["k"], nrm["k"], hd, 1, s_k, False, ws)
    _scores(src["v"], nrm["v"], hd, 1, s_k, True, ws)
    _scores(src["o"], nrm["o"], 1, gq, s_o, False, ws)
    tot_a = s_q[:n_kv]                                                # (q + (k + v)) + o, fp32
    api.mosaic_sum_unit_scores(tot_a, s_k[:n_kv])
    api.mosaic_sum_unit_scores(tot_a, s_o[h:])
    keep_a = n_kv - int(frac * n_kv)
    grp = torch.empty(keep_a, dtype=torch.int32, device=dev)
    api.mosaic_rank_units(tot_a, keep_a, grp)
    for pr, g in (("q", gq), ("k", hd), ("v", hd)):
        o = torch.empty(keep_a * g, h, dtype=cfg.torch_dtype, device=dev)
        api.mosaic_prune_structured_compact(src[pr], None, g, 1, keep_a, h, grp, all_h, given, o, None, ws)
        out["W"][pr] = o
    o = torch.empty(h, keep_a * gq, dtype=cfg.torch_dtype, device=dev)
    api.mosaic_prune_structured_compact(src["o"], None, 1, gq, h, keep_a, all_h, grp, given, o, None, ws)
    out["W"]["o"] = o
    out["attn_keep"] = grp
    return out


def prune_structured_independent(st: ModelState, layer: int, proj: str, frac: float, use_norms: bool = True,
                                 ws: api.Workspace | None = None):
    """Every projection on its own: remove floor(frac*rows) rows and floor(frac*cols) columns
    (group 1) and write the dense compacted matrix.  Returns (W_compact, row_keep, col_keep)."""
    cfg, dev = st.cfg, st.device
    W = st.W[layer, proj]
    rows, cols = W.shape
    kr, kc = rows - int(frac * rows), cols - int(frac * cols)
    rk = torch.empty(kr, dtype=torch.int32, device=dev)
    ck = torch.empty(kc, dtype=torch.int32, device=dev)
    out = torch.empty(kr, kc, dtype=cfg.torch_dtype, device=dev)
    api.mosaic_prune_structured_compact(W, st.norms[layer, cfg.x_key(proj)] if use_norms else None, 1, 1, kr, kc, rk,
                                        ck, 0, out, None, st.ws if ws is None else ws)
    return out, rk, ck


class _StructuredPlan:
    """Buffers and marshalled job lists of the structured stage over every owned layer, built once
    per (fraction, coupling, source matrices) and reused: the stage is then a handful of library
    calls (scores, sums of coupled scores, ranking, compaction - each one launch or two over all
    matrices) with no per-projection host work."""

    def __init__(self, st: ModelState, frac: float, coupled: bool, sources: dict | None, use_norms: bool):
        cfg, dev = st.cfg, st.device
        f32, i32 = torch.float32, torch.int32
        self.steps: list = []          # objects with run(...), in order
        self.out: dict = {}
        self.ws = api.Workspace(dev)
        src = {(layer, pr): (sources[layer][pr] if sources is not None else st.W[layer, pr])
               for layer in st.layers for pr in PROJECTIONS}
        nrm = {(layer, pr): (st.norms[layer, cfg.x_key(pr)] if use_norms else None) for layer in st.layers for pr in PROJECTIONS}
        self.keepalive = (src, nrm)
        score_jobs, rank_jobs, compact_jobs = [], [], []
        add_steps: list[list] = [[], [], []]
        if not coupled:
            for layer in st.layers:
                for pr in PROJECTIONS:
                    W = src[layer, pr]
                    rows, cols = W.shape
                    kr, kc = rows - int(frac * rows), cols - int(frac * cols)
                    rs, cs = torch.empty(rows, dtype=f32, device=dev), torch.empty(cols, dtype=f32, device=dev)
                    rk, ck = torch.empty(kr, dtype=i32, device=dev), torch.empty(kc, dtype=i32, device=dev)
                    out = torch.empty(kr, kc, dtype=cfg.torch_dtype, device=dev)
                    score_jobs.append((W, nrm[layer, pr], 1, 1, rs, cs))
                    rank_jobs += [(rs, kr, rk), (cs, kc, ck)]
                    compact_jobs.append((W, rk, kr, 1, ck, kc, 1, out))
                    self.out[layer, pr] = (out, rk, ck)
        else:
            hd, n_kv = cfg.head_dim, cfg.n_kv_heads
            gq = (cfg.n_heads // n_kv) * hd
            h, it = cfg.hidden, cfg.intermediate
            keep_n, keep_a = it - int(frac * it), n_kv - int(frac * n_kv)
            all_h = torch.arange(h, dtype=i32, device=dev)
            for layer in st.layers:
                def vec(n):
                    return torch.empty(n, dtype=f32, device=dev)
                g_r, u_r, d_c, q_r, k_r, v_r, o_c = vec(it), vec(it), vec(it), vec(n_kv), vec(n_kv), vec(n_kv), vec(n_kv)
                S = {pr: src[layer, pr] for pr in PROJECTIONS}
                N = {pr: nrm[layer, pr] for pr in PROJECTIONS}
                score_jobs += [(S["gate"], N["gate"], 1, 1, g_r, None), (S["up"], N["up"], 1, 1, u_r, None),
                               (S["down"], N["down"], 1, 1, None, d_c), (S["q"], N["q"], gq, 1, q_r, None),
                               (S["k"], N["k"], hd, 1, k_r, None), (S["v"], N["v"], hd, 1, v_r, None),
                               (S["o"], N["o"], 1, gq, None, o_c)]
                # (gate + up) + down  and  (q + (k + v)) + o, in fp32, in this order
                add_steps[0] += [(g_r, g_r, u_r), (k_r, k_r, v_r)]
                add_steps[1] += [(g_r, g_r, d_c), (q_r, q_r, k_r)]
                add_steps[2] += [(q_r, q_r, o_c)]
                ch, grp = torch.empty(keep_n, dtype=i32, device=dev), torch.empty(keep_a, dtype=i32, device=dev)
                rank_jobs += [(g_r, keep_n, ch), (q_r, keep_a, grp)]
                Wc = {}
                for pr in ("gate", "up"):
                    Wc[pr] = torch.empty(keep_n, h, dtype=cfg.torch_dtype, device=dev)
                    compact_jobs.append((S[pr], ch, keep_n, 1, all_h, h, 1, Wc[pr]))
                Wc["down"] = torch.empty(h, keep_n, dtype=cfg.torch_dtype, device=dev)
                compact_jobs.append((S["down"], all_h, h, 1, ch, keep_n, 1, Wc["down"]))
                for pr, g in (("q", gq), ("k", hd), ("v", hd)):
                    Wc[pr] = torch.empty(keep_a * g, h, dtype=cfg.torch_dtype, device=dev)
                    compact_jobs.append((S[pr], grp, keep_a, g, all_h, h, 1, Wc[pr]))
                Wc["o"] = torch.empty(h, keep_a * gq, dtype=cfg.torch_dtype, device=dev)
                compact_jobs.append((S["o"], all_h, h, 1, grp, keep_a, gq, Wc["o"]))
                self.out[layer] = {"W": Wc, "mlp_keep": ch, "attn_keep": grp}
        self.score = api.UnitScoreBatch(score_jobs)
        self.adds = [api.AddBatch(a) for a in add_steps if a]
        self.rank = api.RankBatch(rank_jobs)
        self.compact = api.CompactBatch(compact_jobs)
        self.launches = 3 * ((len(score_jobs) + 127) // 128) + len(self.adds) + (len(rank_jobs) + 511) // 512 + \
            (len(compact_jobs) + 127) // 128

    def run(self) -> dict:
        self.score.run(self.ws)
        for a in self.adds:
            a.run()
        self.rank.run()
        self.compact.run()
        return self.out


def prune_structured_model(st: ModelState, frac: float, coupled: bool = True, sources: dict | None = None,
                           use_norms: bool = True) -> dict:
    """The structured stage over every owned layer through the batched calls: unit scores of all
    matrices, (coupled) the sums of the coupled units' scores, all rankings, all compactions - a
    launch or two per step for the whole model.  `sources[layer]`, if given, holds the matrices to
    read (the masked weights in composite mode).  Returns {layer: {"W": {proj: compacted},
    "mlp_keep", "attn_keep"}} (coupled, as prune_structured_coupled_layer) or {(layer, proj):
    (W_compact, row_keep, col_keep)}.  Buffers and job lists are built on the first call with a
    given (frac, coupled, sources) and reused by later ones: the returned tensors are overwritten
    by the next call with the same arguments."""
    ident = (float(frac), bool(coupled), bool(use_norms),
             None if sources is None else tuple(id(sources[layer][pr]) for layer in st.layers for pr in PROJECTIONS),
             tuple(id(st.W[layer, pr]) for layer in st.layers for pr in PROJECTIONS))
    hit = st.batches.get("structured")
    if hit is None or hit[0] != ident:
        hit = (ident, _StructuredPlan(st, frac, coupled, sources, use_norms))
        st.batches["structured"] = hit
    return hit[1].run()
