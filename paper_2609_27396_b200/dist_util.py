"""Host-side helpers for running the draft step on several GPUs of one node.

Requests are independent in both calls (each has its own context, spine, branches and logits), so the
batch shards across ranks with no data-path collective; torch.distributed is used only to bracket the
timed region and to take the maximum time over ranks.
"""
from __future__ import annotations

import os
import socket
import subprocess
import sys
from typing import Dict, List, Optional, Sequence, Tuple


def free_port() -> int:
    """A TCP port that is free on 127.0.0.1 right now."""
    with socket.socket(socket.AF_INET, socket.SOCK_STREAM) as s:
        s.bind(("127.0.0.1", 0))
        return int(s.getsockname()[1])


def rank_environments(n: int, port: int, base: Optional[Dict[str, str]] = None) -> List[Dict[str, str]]:
    """The environments of n ranks of one node, one rank per GPU: what a launcher such as torch.distributed.run
    would set (RANK, LOCAL_RANK, WORLD_SIZE, LOCAL_WORLD_SIZE, MASTER_ADDR = 127.0.0.1, MASTER_PORT), on top of
    `base` (default: this process's environment)."""
    if n < 1:
        raise ValueError("need at least one rank")
    base = dict(os.environ if base is None else base)
    envs = []
    for r in range(n):
        e = dict(base)
        e.update(RANK=str(r), LOCAL_RANK=str(r), WORLD_SIZE=str(n), LOCAL_WORLD_SIZE=str(n),
                 MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        envs.append(e)
    return envs


def launch_ranks(argv: Sequence[str], n: int, timeout: Optional[float] = None) -> int:
    """Runs `python argv...` as n ranks (one child process per GPU) and waits for them.  Rank 0 inherits this
    process's stdout (it prints the result line); every rank inherits stderr.  Returns the largest exit code;
    if a rank fails or the timeout passes, the remaining children (exactly those started here) are terminated."""
    envs = rank_environments(n, free_port())
    procs = []
    for r, e in enumerate(envs):
        procs.append(subprocess.Popen([sys.executable] + list(argv), env=e,
                                      stdout=None if r == 0 else subprocess.DEVNULL))
    rc = 0
    try:
        for p in procs:
            rc = max(rc, abs(p.wait(timeout=timeout)))
    except subprocess.TimeoutExpired:
        rc = 124
    finally:
        for p in procs:
            if p.poll() is None:
                p.terminate()
    return rc


def shard_requests(ctx_lens: Sequence[int], world: int) -> List[List[int]]:
    """Partition request indices over `world` ranks, balancing the summed context length (longest first,
    each to the currently lightest rank).  Every request lands on exactly one rank."""
    order = sorted(range(len(ctx_lens)), key=lambda i: (-int(ctx_lens[i]), i))
    loads = [0] * world
    parts: List[List[int]] = [[] for _ in range(world)]
    for i in order:
        r = min(range(world), key=lambda k: (loads[k], k))
        parts[r].append(i)
        loads[r] += int(ctx_lens[i]) + 1
    return [sorted(p) for p in parts]


def rank_seed(base_seed: int, rank: int) -> int:
    """Seed of rank's own synthetic batch under weak scaling (rank 0 keeps the single-GPU batch)."""
    return base_seed + 1000 * rank


def max_over_ranks(value: float, device="cpu") -> float:
    """Maximum of a host float over all ranks (identity when torch.distributed is not initialised)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def gather_results(accept_len, bonus) -> Tuple[list, list]:
    """All ranks' (accept_len, bonus) lists on every rank: 8 bytes per request, the only exchange a caller
    that wants the whole batch's outcome on one rank needs."""
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return [list(accept_len)], [list(bonus)]
    a = [None] * dist.get_world_size()
    b = [None] * dist.get_world_size()
    dist.all_gather_object(a, list(accept_len))
    dist.all_gather_object(b, list(bonus))
    return a, b
