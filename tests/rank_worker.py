"""One rank of the multi-process CPU test (started through paper_2504_06323_b200.launch): gloo
process group, outlier counts of the rank's own layers from the oracle pipeline, the one
all-gather of counts, the allocation; the result goes to a JSON file per rank."""
import json
import os
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
sys.path.insert(0, os.path.join(ROOT, "tests"))

import torch                          # noqa: E402
import torch.distributed as dist      # noqa: E402

import oracle_pipeline as op          # noqa: E402
from paper_2504_06323_b200 import driver, workloads as wl   # noqa: E402
from paper_2504_06323_b200.workloads import PROJECTIONS     # noqa: E402


def tiny_cfg():
    return wl.scaled(wl.CONFIGS["tiny"], n_layers=5, hidden=64, n_heads=2, n_kv_heads=2, head_dim=32,
                     intermediate=160, tokens=200)


def counts_for(cfg, layers):
    W, X = {}, {}
    for layer in layers:
        for pr in PROJECTIONS:
            W[layer, pr] = wl.to_numpy(wl.gen_weight(cfg, layer, pr))
        for xk in cfg.x_keys():
            X[layer, xk] = wl.to_numpy(wl.gen_activation(cfg, layer, xk))
    return op.phase_a(cfg, W, X, layers)[1]


def main(out_dir):
    rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
    dist.init_process_group("gloo")
    try:
        cfg = tiny_cfg()
        mine = driver.layers_of_rank(cfg.n_layers, rank, world)
        local = torch.tensor(counts_for(cfg, mine), dtype=torch.int64)
        counts = driver.exchange_counts(local, cfg.n_layers, rank, world)
        s, k, _ = driver.plan_sparsity(cfg, counts)
        with open(os.path.join(out_dir, f"rank{rank}.json"), "w") as f:
            json.dump({"rank": rank, "world": world, "mine": mine, "counts": counts, "s": list(s), "k": list(k)}, f)
    finally:
        dist.destroy_process_group()


if __name__ == "__main__":
    main(sys.argv[1])
