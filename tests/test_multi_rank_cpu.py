"""The multi-process path on CPU (gloo, world_size 2): layers are sharded
round-robin, each rank computes the outlier counts of its own layers, one
all_gather of the counts is the only exchange, and every rank then derives the
same allocation as a single process does."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import oracle
import oracle_pipeline as op
from paper_2504_06323_b200 import build, driver, workloads as wl
from paper_2504_06323_b200.workloads import PROJECTIONS


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _cfg():
    return wl.scaled(wl.CONFIGS["tiny"], n_layers=5, hidden=64, n_heads=2, n_kv_heads=2, head_dim=32,
                     intermediate=160, tokens=200)


def _counts_for(cfg, layers):
    W, X = {}, {}
    for layer in layers:
        for pr in PROJECTIONS:
            W[layer, pr] = wl.to_numpy(wl.gen_weight(cfg, layer, pr))
        for xk in cfg.x_keys():
            X[layer, xk] = wl.to_numpy(wl.gen_activation(cfg, layer, xk))
    return op.phase_a(cfg, W, X, layers)[1]


def _worker(rank, world, port, q):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        cfg = _cfg()
        mine = driver.layers_of_rank(cfg.n_layers, rank, world)
        local = torch.tensor(_counts_for(cfg, mine), dtype=torch.int64)
        counts = driver.exchange_counts(local, cfg.n_layers, rank, world)
        s, k, _ = driver.plan_sparsity(cfg, counts)
        q.put((rank, mine, counts, list(s), list(k)))
    finally:
        dist.destroy_process_group()


def test_layer_sharding_covers_every_layer_once():
    for n, world in [(32, 1), (32, 2), (40, 8), (5, 2), (3, 4)]:
        seen = sorted(l for r in range(world) for l in driver.layers_of_rank(n, r, world))
        assert seen == list(range(n))


def test_two_ranks_agree_with_one_process():
    build.build_library()
    cfg = _cfg()
    want_counts = _counts_for(cfg, list(range(cfg.n_layers)))
    s_ref, k_ref, _ = op.plan(cfg, want_counts, cfg.n_layers)
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    results = [q.get(timeout=120) for _ in procs]
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert sorted(r[0] for r in results) == [0, 1]
    for rank, mine, counts, s, k in results:
        assert mine == [l for l in range(cfg.n_layers) if l % 2 == rank]
        assert counts == want_counts
        assert np.array_equal(np.array(s).view(np.uint64), s_ref.view(np.uint64))
        assert k == list(k_ref)
    assert len(set(results[0][4])) > 1


def test_launcher_starts_two_ranks_that_agree_with_one_process(tmp_path):
    # the launcher bench.py --gpus N uses (torch.distributed.run on 127.0.0.1), here with gloo ranks on CPU
    import json
    from paper_2504_06323_b200 import launch
    build.build_library()
    worker = os.path.join(os.path.dirname(os.path.abspath(__file__)), "rank_worker.py")
    rc = launch.spawn_ranks(2, worker, [str(tmp_path)], timeout=300)
    assert rc == 0
    cfg = _cfg()
    want_counts = _counts_for(cfg, list(range(cfg.n_layers)))
    s_ref, k_ref, _ = op.plan(cfg, want_counts, cfg.n_layers)
    for rank in range(2):
        with open(tmp_path / f"rank{rank}.json") as f:
            r = json.load(f)
        assert r["world"] == 2 and r["mine"] == [l for l in range(cfg.n_layers) if l % 2 == rank]
        assert r["counts"] == want_counts and r["k"] == list(k_ref)
        assert np.array_equal(np.array(r["s"]).view(np.uint64), s_ref.view(np.uint64))
