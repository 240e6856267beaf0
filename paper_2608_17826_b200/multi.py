"""Multi-GPU plumbing: one process per GPU, rank slices are independent units.

A TP rank slice has its own tier objects, ring, block tables and paged pools, so a restore shards
over GPUs with no data exchange at all.  The single step that spans processes is the commit
predicate (Eq. 6 is an AND over all ranks): one integer per process, combined with a MIN
all-reduce.  Works on any torch.distributed backend (NCCL over NVLink on GPUs, gloo on CPU).
"""
from __future__ import annotations

import torch
import torch.distributed as dist


def slices_of(process_rank: int, world: int, n_slices: int) -> list[int]:
    """The TP rank slices process `process_rank` restores: slice r lives on process r mod world."""
    return [r for r in range(n_slices) if r % world == process_rank]


def commit_across_ranks(exposed_local: int, n_adv: int, device=None, group=None) -> int:
    """Request-level commit over all processes: the prefix is exposed (n_adv) only if every
    process exposed it; otherwise every process reports 0 and must invalidate its slices."""
    ok = 1 if exposed_local == n_adv else 0
    if dist.is_available() and dist.is_initialized() and dist.get_world_size(group) > 1:
        flag = torch.tensor([ok], dtype=torch.int32, device=device)
        dist.all_reduce(flag, op=dist.ReduceOp.MIN, group=group)
        ok = int(flag.item())
    return n_adv if ok else 0


def max_over_ranks(value: float, device=None, group=None) -> float:
    """Slowest process's figure (device-timed milliseconds are compared, never wall clocks)."""
    if dist.is_available() and dist.is_initialized() and dist.get_world_size(group) > 1:
        t = torch.tensor([value], dtype=torch.float64, device=device)
        dist.all_reduce(t, op=dist.ReduceOp.MAX, group=group)
        return float(t.item())
    return float(value)


def cpu_share(allowed: list[int], node_cpus_of_rank: list[list[int] | None], local_rank: int) -> list[int]:
    """The host CPUs local rank `local_rank` keeps for its fill threads when several processes
    feed their GPUs from one host.

    allowed: CPUs this job may use (its affinity mask).  node_cpus_of_rank[l]: the CPUs of the NUMA
    node GPU l hangs off, or None where the platform does not say.  Ranks whose GPUs share a node
    split that node's allowed CPUs evenly, in rank order; ranks without a known node split what no
    known node claims (all allowed CPUs when no node is known at all).  Every rank gets at least one CPU."""
    allowed = sorted(allowed)
    key = [None if c is None else tuple(sorted(set(c) & set(allowed))) or None for c in node_cpus_of_rank]
    mine = key[local_rank]
    if mine is None:
        claimed = set().union(*[set(k) for k in key if k is not None]) if any(k is not None for k in key) else set()
        pool = [c for c in allowed if c not in claimed] or allowed
    else:
        pool = list(mine)
    peers = [l for l, k in enumerate(key) if k == mine]
    n, at = len(peers), peers.index(local_rank)
    lo, hi = at * len(pool) // n, (at + 1) * len(pool) // n
    return pool[lo:hi] or [pool[min(lo, len(pool) - 1)]]
