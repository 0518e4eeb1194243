#!/usr/bin/env python
"""Benchmark of the Mosaic pruning hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl native|reference]

A step is one pass of the whole path over a LLaMA-7B-shaped model (32 layers,
bf16, 128 x 2048 calibration tokens per projection input): activation norms
for every projection input, outlier count of every projection, the host
allocation of the 224 sparsity targets, and the per-row unstructured
selection + zeroing (+ keep bitmask) of every projection at 50 % average
sparsity.  The metric is weight GB/s: bytes of weights scored and pruned per
second of step time.  One JSON line is printed by rank 0.

With N > 1 every rank (one process per GPU) owns 32 layers of a 32*N-layer
model (weak scaling); the only exchange is one all_gather of the outlier
counts between the two phases.  Started as a single process with --gpus N,
the script starts its N ranks itself (torch.distributed.run on 127.0.0.1);
started by a launcher it finds RANK / WORLD_SIZE in the environment.

After the headline region (N = 1 only) two more arms are timed and appended
to the same JSON line: `structured` - rows and columns of every projection of
the compaction-stress configuration ranked and compacted at f = 0.3 - and
`composite` - one pass over the LLaMA-3-8B-shaped configuration: outlier
sweeps, allocation, 50 % unstructured, then the coupled 20 % structured stage -
and `hessian` - the second-moment matrices X^T X of one layer's projection
inputs on the tensor cores (the calibration-side companion of the norms).
--blocks chooses the arms (default: all).

--impl reference times the CPU oracle (as it stands) on the host cores over a
bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2504_06323_b200 import workloads as wl  # noqa: E402
from paper_2504_06323_b200.workloads import PROJECTIONS  # noqa: E402

METRIC = "weight_GBps_scored_and_pruned"
UNIT = "GB/s"

# DRAM traffic of the dominant kernel from an ncu capture of a smaller launch (profiles/
# col_partial_kernel_act_norms_small.md): reads = 1.00005 x the bytes of X (they scale with the
# token count), writes = the split partials, about 1240 B per column whatever the token count.
NCU_TRAFFIC = {"col_partial_kernel": {"read_ratio": 1.00005, "write_bytes_per_col": 1240.0}}


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return float(d["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


def measured_tensor_peaks():
    """(burst, sustained) dense bf16 TFLOP/s of the library GEMM on this machine, and where they come from."""
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return float(d["bf16_tflops"]), float(d.get("bf16_tflops_sustained", d["bf16_tflops"])), "measured"
    return 1590.0, 1400.0, "fallback"


class ClockSampler:
    """nvidia-smi clocks and throttle reasons sampled every 200 ms while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.proc, self.path = index, None, None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "200", "-f", self.path], stdout=subprocess.DEVNULL, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self) -> dict:
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": []}
        if self.proc is None:
            return out
        time.sleep(0.25)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        try:
            rows = [l.strip().split(", ") for l in open(self.path) if l.strip()]
            os.unlink(self.path)
            sm = [float(r[0]) for r in rows if len(r) >= 7]
            if sm:
                busy = [s for s, r in zip(sm, rows) if float(r[2]) > 250.0] or sm
                out["sm_mhz"] = statistics.median(busy)
                out["sm_max_mhz"] = float(rows[0][1])
                names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
                out["reasons"] = [n for i, n in enumerate(names) if any(r[3 + i].strip() == "Active" for r in rows)]
                out["samples"] = len(sm)
        except Exception:
            pass
        return out


def cpu_model() -> str:
    try:
        with open("/proc/cpuinfo") as f:
            for line in f:
                if line.lower().startswith("model name"):
                    return line.split(":", 1)[1].strip()
    except OSError:
        pass
    return "unknown"


# --------------------------------------------------------------------------- CPU oracle sample
def oracle_sample_inputs(cfg, frac_div: int, device):
    """1/frac_div of one layer: tokens/frac_div calibration tokens per input and rows/frac_div rows
    of each of the seven projections (so activation and weight work keep the model's ratio)."""
    T = cfg.tokens // frac_div
    X = {xk: wl.to_numpy(wl.gen_activation(cfg, 0, xk, device, tokens=T)) for xk in cfg.x_keys()}
    W = {}
    for pr in PROJECTIONS:
        rows, cols = cfg.shape(pr)
        W[pr] = wl.to_numpy(wl.gen_weight(cfg, 0, pr, device, shape=(max(rows // frac_div, 1), cols)))
    return X, W


def oracle_sample_step(cfg, X, W):
    """The path on the sample, oracle calls only.  Returns weight bytes processed."""
    import oracle
    norms = {xk: oracle.act_norms(x, cfg.dtype) for xk, x in X.items()}
    counts, numels, cols = [], [], []
    for pr in PROJECTIONS:
        r = oracle.outlier_ratio(W[pr], norms[cfg.x_key(pr)], cfg.alpha, cfg.dtype)
        counts.append(r["count"])
        numels.append(r["numel"])
        cols.append(W[pr].shape[1])
    _, k, _ = oracle.allocate_sparsity(counts, numels, cols, 1, len(PROJECTIONS), cfg.p, cfg.lam)
    for m, pr in enumerate(PROJECTIONS):
        oracle.prune_unstructured(W[pr], norms[cfg.x_key(pr)], int(k[m]), cfg.dtype)
    return sum(w.size * w.itemsize for w in W.values())


def run_reference(args, cfg):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    device = "cuda" if torch.cuda.is_available() else "cpu"
    frac_div = 32
    X, W = oracle_sample_inputs(cfg, frac_div, device)
    for _ in range(args.warmup):
        oracle_sample_step(cfg, X, W)
    t0 = time.perf_counter()
    nbytes = 0
    for _ in range(args.steps):
        nbytes += oracle_sample_step(cfg, X, W)
    dt = time.perf_counter() - t0
    value = nbytes / dt / 1e9
    sample = f"1/{frac_div} of one layer per step: {cfg.tokens // frac_div} tokens per input, rows/{frac_div} of each projection"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": "llama7b: 32 layers, hidden 4096, MLP 11008, bf16, 128x2048 calibration tokens, "
                               "unstructured 50% (oracle on a bounded sample)", "inputs": "larger than L2"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# --------------------------------------------------------------------------- native arm
def run_native(args, cfg):
    import torch.distributed as dist
    from paper_2504_06323_b200 import api, build, driver

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
    if world != args.gpus:
        raise SystemExit(f"bench.py --gpus {args.gpus} is running as {world} rank(s): start it plainly (it launches its "
                         f"ranks itself) or with --nproc-per-node equal to --gpus")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    if not os.path.exists(api.LIB_PATH):
        if rank == 0:
            build.build_library()
        if world > 1:
            dist.barrier()
    api.lib()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    n_layers = args.layers or cfg.n_layers
    total_cfg = wl.scaled(cfg, n_layers=n_layers * world)            # weak scaling: each rank owns n_layers layers
    mine = driver.layers_of_rank(total_cfg.n_layers, rank, world)
    st = driver.alloc_model(total_cfg, dev, mine)
    # One layer's calibration activations, resident in HBM and reused for every layer
    # (12.2 GB for the 7B shape: far larger than L2; a whole model's 391 GB would not fit).
    X = driver.make_activations(cfg, 0, dev, tokens=args.tokens or cfg.tokens)
    M = len(PROJECTIONS)
    w_bytes = sum(st.W[l, p].numel() * cfg.itemsize for l in mine for p in PROJECTIONS)
    x_bytes_layer = sum(x.numel() * cfg.itemsize for x in X.values())

    blocks = set(args.blocks.split(","))
    if world == 1 and "headline" not in blocks:
        # only the other arms (for profiling them alone): norms of one layer serve every layer
        driver.accumulate_norms(st, mine[0], X)
        for layer in mine[1:]:
            for xk in cfg.x_keys():
                st.norms[layer, xk].copy_(st.norms[mine[0], xk])
        peak, _ = measured_peaks()
        line = {"metric": METRIC, "n_gpus": 1, "note": "headline arm skipped (--blocks)"}
        if "structured" in blocks:
            line["structured"] = run_structured_block(args, st, peak)
        if "hessian" in blocks:
            line["hessian"] = run_hessian_block(args, cfg, X, dev, local)
        del st, X
        torch.cuda.empty_cache()
        if "composite" in blocks:
            line["composite"] = run_composite_block(args, dev, peak)
        print(json.dumps(line), flush=True)
        return

    def step(ev=None):
        """One pass of the whole path.  `ev`: five CUDA events recorded at the phase boundaries."""
        launches = 0
        if ev: ev[0].record()
        for layer in mine:
            launches += 2 * driver.accumulate_norms(st, layer, X, join=(layer == mine[-1]))
        if ev: ev[1].record()
        driver.count_outliers_all(st)
        launches += 4                                                   # estimate, summing sweep with ladders, finish, fallback count sweep
        if ev: ev[2].record()
        counts = driver.exchange_counts(st.counts, total_cfg.n_layers, rank, world)
        _, k, _ = driver.plan_sparsity(total_cfg, counts)
        if ev: ev[3].record()
        driver.prune_unstructured_all(st, k)
        launches += sum(prune_launches(c) for c in {cfg.shape(p)[1] for p in PROJECTIONS})
        if ev: ev[4].record()
        return launches

    for _ in range(max(args.warmup, 3)):
        step()
    barrier()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    # phase boundaries are marked inside the timed region (an event record costs nothing on the device)
    events = [[torch.cuda.Event(enable_timing=True) for _ in range(5)] for _ in range(args.steps)]
    start, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    start.record()
    launches = 0
    for s in range(args.steps):
        launches += step(events[s])
    end.record()
    barrier()
    total_ms = start.elapsed_time(end)
    phase_ms = [sum(ev[i].elapsed_time(ev[i + 1]) for ev in events) / args.steps for i in range(4)]
    # per-step times: from one step's first event to the next step's (the last step ends at `end`)
    step_ms = [events[i][0].elapsed_time(events[i + 1][0]) for i in range(args.steps - 1)] + [events[-1][0].elapsed_time(end)]
    weight_ms = [ev[1].elapsed_time(ev[4]) for ev in events]
    clocks = sampler.stop() if rank == 0 else None

    t = torch.tensor([total_ms], dtype=torch.float64, device=dev)
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    ms_per_step = t.item() / args.steps
    value = w_bytes * world / (ms_per_step * 1e-3) / 1e9

    # ---- end to end from pinned host buffers (weights and activations in, pruned weights out)
    e2e = None
    if not args.no_e2e:
        e2e = run_e2e(args, cfg, total_cfg, st, mine, dev, rank, world, barrier)

    # ---- CPU oracle on a bounded sample (rank 0, N = 1 only)
    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu:
        import oracle
        frac_div, reps = 2, 4
        Xs, Ws = oracle_sample_inputs(cfg, frac_div, dev)
        threads = oracle.num_threads()
        t0 = time.perf_counter()
        nb = sum(oracle_sample_step(cfg, Xs, Ws) for _ in range(reps))
        dt = time.perf_counter() - t0
        del Xs, Ws
        # the same oracle on one thread, on a sample 16 times smaller
        Xs, Ws = oracle_sample_inputs(cfg, 32, dev)
        oracle.set_num_threads(1)
        t1 = time.perf_counter()
        nb1 = oracle_sample_step(cfg, Xs, Ws)
        dt1 = time.perf_counter() - t1
        oracle.set_num_threads(threads)
        del Xs, Ws
        cpu = {"value": nb / dt / 1e9, "unit": UNIT, "cores": threads, "kind": "oracle", "cpu_model": cpu_model(),
               "sample": f"{reps} passes over 1/{frac_div} of one layer: {cfg.tokens // frac_div} calibration tokens "
                         f"per input and rows/{frac_div} of each of the 7 projections ({nb / 1e6:.1f} MB of weights "
                         f"in {dt:.1f} s)",
               "one_thread": {"value": nb1 / dt1 / 1e9, "unit": UNIT, "cores": 1,
                              "sample": f"1 pass over 1/32 of one layer ({nb1 / 1e6:.1f} MB of weights in {dt1:.1f} s)"}}

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return
    peak, peak_kind = measured_peaks()
    n_act_launch = len(mine) * len(X)
    act_bytes = x_bytes_layer * len(mine)
    act_gbs = act_bytes / (phase_ms[0] * 1e-3) / 1e9
    tr = NCU_TRAFFIC["col_partial_kernel"]
    avg_cols = sum(x.shape[1] for x in X.values()) / len(X)
    roofline = {
        "kernel": "col_partial_kernel<bf16, square> (activation norms)", "bound": "hbm", "achieved": act_gbs,
        "peak": peak, "peak_kind": f"of {peak_kind}", "unit": "GB/s", "frac": act_gbs / peak,
        "traffic": tr["read_ratio"] * act_bytes / n_act_launch + tr["write_bytes_per_col"] * avg_cols,
        "traffic_note": "bytes per launch, scaled from an ncu capture of a 32768-token launch (reads scale with tokens, "
                        "partial-sum writes do not)",
        "algorithmic_bytes_per_launch": act_bytes / n_act_launch, "launches_per_step": n_act_launch,
        "avg_launch_ms": phase_ms[0] / n_act_launch,
        "note": "duration = the phase's CUDA-event time / launches (a layer's launches alternate between two streams, so "
                "the finishing kernel of one runs under the next); the peak is a copy (read + write): a read-only "
                "stream like this one can exceed it by a few per cent",
    }
    outl_gbs = w_bytes / (phase_ms[1] * 1e-3) / 1e9
    prune_gbs = w_bytes * 4.125 / 2 / (phase_ms[3] * 1e-3) / 1e9
    weight_pass_ms = phase_ms[1] + phase_ms[2] + phase_ms[3]
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3),
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
        "data": "synthetic",
        "ms_per_step_spread": {"min": min(step_ms), "median": statistics.median(step_ms), "max": max(step_ms),
                               "note": "rank 0, CUDA events per step"},
        "config": {"workload": f"{cfg.name}: {n_layers} layers/GPU, hidden {cfg.hidden}, MLP {cfg.intermediate}, bf16 "
                               f"Student-t weights, {args.tokens or cfg.tokens} calibration tokens per projection input "
                               f"(one layer's activations resident and reused by every layer), alpha {cfg.alpha}, "
                               f"unstructured p={cfg.p}, lambda={cfg.lam}",
                   "inputs": "larger than L2 (25.1 GB per step vs 126 MB)", "parallelism": f"layers sharded over {world} GPU(s)"},
        "clocks": clocks, "e2e": e2e, "gpu_launches": launches,
        "roofline": roofline, "cpu_baseline": cpu,
        "phases_ms": {"act_norms": phase_ms[0], "outlier_ratio": phase_ms[1], "counts_d2h_allocate": phase_ms[2],
                      "prune_unstructured": phase_ms[3]},
        "weight_pass": {"ms": weight_pass_ms, "ms_min": min(weight_ms), "ms_median": statistics.median(weight_ms),
                        "ms_max": max(weight_ms), "weight_GBps": w_bytes / (weight_pass_ms * 1e-3) / 1e9,
                        "compulsory_GBps": w_bytes * 6.125 / 2 / (weight_pass_ms * 1e-3) / 1e9,
                        "frac_of_peak": w_bytes * 6.125 / 2 / (weight_pass_ms * 1e-3) / 1e9 / peak,
                        "frac_of_8TBps": w_bytes * 6.125 / 2 / (weight_pass_ms * 1e-3) / 1e9 / 8000.0},
        "roofline_other": [
            {"kernel": "score_sum_ladder_kernel (+ estimate, finish and fallback launches; all projections per launch)", "bound": "hbm",
             "achieved": outl_gbs, "peak": peak, "unit": "GB/s", "frac": outl_gbs / peak,
             "algorithmic_bytes": "2 B/weight (one sweep: the count comes from per-column ladders of bf16 patterns)"},
            {"kernel": "prune_rows_warp_kernel (one launch per row length)", "bound": "hbm",
             "achieved": prune_gbs, "peak": peak, "unit": "GB/s", "frac": prune_gbs / peak,
             "algorithmic_bytes": "4.125 B/weight"}],
    }
    # ---- the structured and the composite arm (N = 1): appended to the same line
    if world == 1:
        if "structured" in blocks:
            line["structured"] = run_structured_block(args, st, peak)
        if "hessian" in blocks:
            line["hessian"] = run_hessian_block(args, cfg, X, dev, local)
        del st, X
        torch.cuda.empty_cache()
        if "composite" in blocks:
            line["composite"] = run_composite_block(args, dev, peak)
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def prune_launches(cols: int) -> int:
    """Kernel launches mosaic_prune_unstructured_batch makes for the (<= 256) jobs of one row length:
    one launch of the row-group kernel (bf16 rows of 2048..16384 columns)."""
    return 1


def _median_ms(fn, warmup=3, reps=5):
    for _ in range(warmup):
        fn()
    torch.cuda.synchronize()
    ts = []
    for _ in range(reps):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        fn()
        e1.record()
        torch.cuda.synchronize()
        ts.append(e0.elapsed_time(e1))
    return {"min": min(ts), "median": statistics.median(ts), "max": max(ts)}


def run_structured_block(args, st, peak):
    """Structured stage alone (steps C1-C3) on the compaction-stress shape: every projection of the
    model on its own, floor(f*rows) rows and floor(f*cols) columns removed, dense compacted bf16 out.
    Algorithmic bytes per weight: 2 (scores: W read once) + 2(1-f) (kept rows read) + 2(1-f)^2 (written)."""
    from paper_2504_06323_b200 import driver
    f = 0.3
    t = _median_ms(lambda: driver.prune_structured_model(st, f, coupled=False))
    w = sum(x.numel() for x in st.W.values())
    nbytes = w * (2.0 + 2.0 * (1 - f) + 2.0 * (1 - f) ** 2)
    gbs = nbytes / (t["median"] * 1e-3) / 1e9
    return {"workload": f"llama7b_structured shape: {len(st.layers)} layers x 7 projections, rows and columns of every "
                        f"projection independently, f = {f}", "ms": t["median"], "ms_min": t["min"], "ms_max": t["max"],
            "algorithmic_bytes": nbytes, "bytes_per_weight": nbytes / w, "achieved": gbs, "unit": "GB/s", "peak": peak,
            "frac": gbs / peak, "projections": len(st.W)}


def run_hessian_block(args, cfg, X, dev, local):
    """Calibration-side companion: the second-moment matrix G = X^T X of every projection input of one
    layer (the matrix the inverse-Hessian back-end is built from), on the tensor cores, over the resident
    calibration activations in calls of 32768 tokens.  Algorithmic flops: tokens * cols * (cols + 1) per
    input (G is symmetric: the blocks on or above the diagonal are computed, the rest mirrored)."""
    from paper_2504_06323_b200 import driver
    chunk = 32768
    G = {xk: torch.empty(x.shape[1], x.shape[1], device=dev, dtype=torch.float32) for xk, x in X.items()}
    status = torch.zeros(1, device=dev, dtype=torch.int32)
    timed_out = []

    def one_pass():
        launches = 0
        for xk, x in X.items():
            launches += driver.accumulate_second_moments(G[xk], x, reset=True, status=status, chunk_tokens=chunk)
        return launches

    one_pass()
    torch.cuda.synchronize()
    timed_out.append(int(status.item()))
    sampler = ClockSampler(local)
    sampler.start()
    t = _median_ms(one_pass, warmup=1, reps=5)
    clocks = sampler.stop()
    timed_out.append(int(status.item()))
    launches = one_pass()
    torch.cuda.synchronize()
    alg = sum(float(x.shape[0]) * x.shape[1] * (x.shape[1] + 1) for x in X.values())
    exe = 0.0
    for x in X.values():
        nb = (x.shape[1] + 255) // 256
        exe += 2.0 * x.shape[0] * 256.0 * 256.0 * nb * (nb + 1) / 2
    burst, sustained, kind = measured_tensor_peaks()
    tf = alg / (t["median"] * 1e-3) / 1e12
    return {"workload": f"{cfg.name}: G = X^T X of the {len(X)} projection inputs of one layer "
                        f"({', '.join(str(x.shape[1]) for x in X.values())} columns, {next(iter(X.values())).shape[0]} tokens, "
                        f"bf16 in, fp32 out, {chunk} tokens per call)",
            "kernel": "gram_kernel (tcgen05.mma, TMA-staged MN-major tiles, 256x256 fp32 blocks in tensor memory)",
            "bound": "tensor", "ms": t["median"], "ms_min": t["min"], "ms_max": t["max"], "gpu_launches": launches,
            "algorithmic_flops": alg, "executed_flops": exe, "achieved": tf, "achieved_executed": exe / (t["median"] * 1e-3) / 1e12,
            "unit": "TFLOP/s", "peak": burst, "peak_sustained": sustained, "peak_kind": f"of {kind} (library bf16 GEMM; burst / sustained)",
            "frac": tf / burst, "frac_of_sustained": tf / sustained, "dtype": "bf16 x bf16 -> fp32", "clocks": clocks,
            "bounded_wait_ran_out": any(timed_out),
            "vs_full_square_gemm": "a library GEMM of X^T X computes both triangles: twice the flops counted here"}


def run_composite_block(args, dev, peak):
    """One pass over the LLaMA-3-8B-shaped configuration (GQA, MLP 14336) with the norms in place:
    outlier sweeps, allocation, 50 % unstructured, coupled 20 % structured (MLP channels; KV groups)."""
    from paper_2504_06323_b200 import driver
    cfg = wl.CONFIGS["llama3_8b"]
    n_layers = args.layers or cfg.n_layers
    cfg_n = wl.scaled(cfg, n_layers=n_layers)
    st = driver.alloc_model(cfg_n, dev)
    X = driver.make_activations(cfg, 0, dev, tokens=min(args.tokens or 32768, 32768))   # norms only have to be realistic
    driver.accumulate_norms(st, 0, X)
    del X
    for layer in st.layers[1:]:
        for xk in cfg.x_keys():
            st.norms[layer, xk].copy_(st.norms[0, xk])
    frac = cfg.extra["structured_frac"]
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(5)]

    def one_pass(record=False):
        if record: ev[0].record()
        driver.count_outliers_all(st)
        if record: ev[1].record()
        counts = driver.exchange_counts(st.counts, cfg_n.n_layers, 0, 1)
        _, k, _ = driver.plan_sparsity(cfg_n, counts)
        if record: ev[2].record()
        driver.prune_unstructured_all(st, k)
        if record: ev[3].record()
        sources = {layer: {pr: st.W_out[layer, pr] for pr in PROJECTIONS} for layer in st.layers}
        out = driver.prune_structured_model(st, frac, coupled=True, sources=sources)
        if record: ev[4].record()
        return out

    for _ in range(3):
        one_pass()
    torch.cuda.synchronize()
    runs = []
    for _ in range(5):
        one_pass(record=True)
        torch.cuda.synchronize()
        runs.append([ev[i].elapsed_time(ev[i + 1]) for i in range(4)])
    med = [statistics.median(r[i] for r in runs) for i in range(4)]
    w = sum(x.numel() for x in st.W.values())
    # structured stage: scores read every weight once; compaction reads the kept rows whole and writes the kept part
    keep = 1.0 - int(frac * cfg.intermediate) / cfg.intermediate
    keep_a = 1.0 - int(frac * cfg.n_kv_heads) / cfg.n_kv_heads
    c_bytes = 0.0
    for layer in st.layers:
        for pr in PROJECTIONS:
            n = st.W[layer, pr].numel()
            kr, kc = {"gate": (keep, 1.0), "up": (keep, 1.0), "down": (1.0, keep), "q": (keep_a, 1.0), "k": (keep_a, 1.0),
                      "v": (keep_a, 1.0), "o": (1.0, keep_a)}[pr]
            c_bytes += n * (2.0 + 2.0 * kr + 2.0 * kr * kc)
    total = sum(med)
    return {"workload": f"llama3_8b shape: {n_layers} layers, GQA 32/8 heads, MLP 14336; norms in place; p = {cfg.p}, "
                        f"structured f = {frac} (coupled MLP channels and KV groups)",
            "ms": total, "phases_ms": {"outlier_ratio": med[0], "counts_d2h_allocate": med[1], "prune_unstructured": med[2],
                                       "structured_coupled": med[3]},
            "algorithmic_bytes": {"outlier_ratio": 2.0 * w, "prune_unstructured": 4.125 * w, "structured_coupled": c_bytes},
            "achieved": {"outlier_ratio": 2.0 * w / (med[0] * 1e-3) / 1e9, "prune_unstructured": 4.125 * w / (med[2] * 1e-3) / 1e9,
                         "structured_coupled": c_bytes / (med[3] * 1e-3) / 1e9}, "unit": "GB/s", "peak": peak,
            "frac": {"outlier_ratio": 2.0 * w / (med[0] * 1e-3) / 1e9 / peak,
                     "prune_unstructured": 4.125 * w / (med[2] * 1e-3) / 1e9 / peak,
                     "structured_coupled": c_bytes / (med[3] * 1e-3) / 1e9 / peak}}


def run_e2e(args, cfg, total_cfg, st, mine, dev, rank, world, barrier):
    """Same step, but every input starts in pinned host memory and the pruned weights end there:
    weights H2D once per step, calibration activations streamed H2D in token chunks through two
    device staging slots (copy stream) while the previous chunk is reduced (compute stream),
    counts D2H, allocation, pruning, pruned weights D2H."""
    import torch.distributed as dist
    from paper_2504_06323_b200 import api, driver
    M = len(PROJECTIONS)
    tokens = args.tokens or cfg.tokens
    chunk = min(args.e2e_chunk, tokens)
    n_chunks = (tokens + chunk - 1) // chunk
    host_x = {xk: torch.randn(chunk, cfg.x_cols(xk), dtype=torch.float32).to(cfg.torch_dtype).pin_memory()
              for xk in cfg.x_keys()}
    stage = {xk: [torch.empty(chunk, cfg.x_cols(xk), dtype=cfg.torch_dtype, device=dev) for _ in range(2)]
             for xk in cfg.x_keys()}
    host_w = {key: torch.empty(w.shape, dtype=w.dtype).pin_memory() for key, w in st.W.items()}
    for key, w in st.W.items():
        host_w[key].copy_(w)
    host_out = {key: torch.empty(w.shape, dtype=w.dtype).pin_memory() for key, w in st.W.items()}
    copy_s = torch.cuda.Stream(dev)
    comp_s = torch.cuda.current_stream(dev)
    h2d = sum(w.numel() * w.element_size() for w in host_w.values()) + \
        len(mine) * n_chunks * sum(x.numel() * x.element_size() for x in host_x.values())
    d2h = sum(w.numel() * w.element_size() for w in host_out.values()) + st.counts.numel() * 8
    free_ev = {(xk, s): None for xk in host_x for s in range(2)}

    def e2e_step():
        with torch.cuda.stream(copy_s):
            for key in st.W:
                st.W[key].copy_(host_w[key], non_blocking=True)
            w_ready = torch.cuda.Event()
            w_ready.record(copy_s)
        i = 0
        for layer in mine:
            for c in range(n_chunks):
                slot = i % 2
                i += 1
                t = min(chunk, tokens - c * chunk)
                for xk in host_x:
                    if free_ev[xk, slot] is not None:
                        copy_s.wait_event(free_ev[xk, slot])
                    with torch.cuda.stream(copy_s):
                        stage[xk][slot][:t].copy_(host_x[xk][:t], non_blocking=True)
                        ready = torch.cuda.Event()
                        ready.record(copy_s)
                    comp_s.wait_event(ready)
                    api.mosaic_act_norms(stage[xk][slot][:t], st.sumsq[layer, xk],
                                         st.norms[layer, xk] if c == n_chunks - 1 else None,
                                         api.RESET_ACCUM if c == 0 else 0, st.ws)
                    done = torch.cuda.Event()
                    done.record(comp_s)
                    free_ev[xk, slot] = done
        comp_s.wait_event(w_ready)
        driver.count_outliers_all(st)                      # the batched calls, as in the device-resident step
        counts = driver.exchange_counts(st.counts, total_cfg.n_layers, rank, world)
        _, k, _ = driver.plan_sparsity(total_cfg, counts)
        driver.prune_unstructured_all(st, k)
        done = torch.cuda.Event()
        done.record(comp_s)
        copy_s.wait_event(done)
        with torch.cuda.stream(copy_s):
            for layer in mine:
                for pr in PROJECTIONS:
                    host_out[layer, pr].copy_(st.W_out[layer, pr], non_blocking=True)
        fin = torch.cuda.Event()
        fin.record(copy_s)
        comp_s.wait_event(fin)

    for _ in range(args.e2e_warmup):
        e2e_step()
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(args.e2e_steps):
        e2e_step()
    e1.record()
    barrier()
    t = torch.tensor([e0.elapsed_time(e1)], dtype=torch.float64, device=dev)
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    ms = t.item() / args.e2e_steps
    w_bytes = sum(w.numel() * w.element_size() for w in host_w.values())
    return {"value": w_bytes * world / (ms * 1e-3) / 1e9, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
            "ms_per_step": ms, "steps": args.e2e_steps, "warmup": args.e2e_warmup,
            "note": "weights + calibration activations from pinned host memory, pruned weights back to it; bound by the "
                    "host link (about 400 GB of activations per step), not by the kernels"}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="native", choices=["native", "reference"])
    ap.add_argument("--config", default="llama7b")
    ap.add_argument("--layers", type=int, default=0, help="layers per GPU (default: the model's)")
    ap.add_argument("--tokens", type=int, default=0, help="calibration tokens (default: the config's)")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu", action="store_true")
    ap.add_argument("--e2e-steps", type=int, default=1)
    ap.add_argument("--e2e-warmup", type=int, default=1)
    ap.add_argument("--e2e-chunk", type=int, default=16384)
    ap.add_argument("--blocks", default="headline,structured,composite,hessian",
                    help="arms appended to the line at N = 1: headline, structured, composite")
    args = ap.parse_args()
    cfg = wl.CONFIGS[args.config]
    if args.impl == "reference":
        run_reference(args, cfg)
        return
    from paper_2504_06323_b200 import launch
    if args.gpus > 1 and not launch.under_launcher():
        # started plainly: become the launcher of our own N ranks (rank 0 prints the line)
        sys.exit(launch.spawn_ranks(args.gpus, os.path.abspath(__file__), sys.argv[1:]))
    run_native(args, cfg)


if __name__ == "__main__":
    main()
