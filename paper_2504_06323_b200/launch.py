"""Starts one process per rank on this node (torch.distributed.run, rendezvous on 127.0.0.1).

The path shards by whole layers with one all-gather of the outlier counts as its only exchange
(driver.layers_of_rank / driver.exchange_counts); this module is just the launcher: a program
that was started as a single process re-runs itself as `world` ranks through it.
"""
from __future__ import annotations

import os
import socket
import subprocess
import sys


def free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def under_launcher() -> bool:
    """True inside a rank that torch.distributed.run (or a compatible launcher) started."""
    return "WORLD_SIZE" in os.environ and "RANK" in os.environ


def rank_command(world: int, script: str, args: list[str], port: int | None = None) -> list[str]:
    return [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={world}",
            "--master-addr", "127.0.0.1", "--master-port", str(free_port() if port is None else port), script, *args]


def spawn_ranks(world: int, script: str, args: list[str], env: dict | None = None, timeout: float | None = None) -> int:
    """Run `script args...` as `world` ranks and return the launcher's exit code.  The ranks find
    RANK / LOCAL_RANK / WORLD_SIZE / MASTER_ADDR / MASTER_PORT in their environment."""
    if world < 1:
        raise ValueError("world must be >= 1")
    full_env = dict(os.environ)
    for k in ("RANK", "LOCAL_RANK", "WORLD_SIZE", "MASTER_ADDR", "MASTER_PORT"):
        full_env.pop(k, None)
    if env:
        full_env.update(env)
    return subprocess.run(rank_command(world, script, args), env=full_env, timeout=timeout).returncode
