"""Host-side plumbing for running the path on several GPUs, one process per GPU.

The path shards by matrix: every weight matrix is an independent problem with its own bit budget
(Algorithm 3 takes one matrix; Section 5.1 quantises a model layer by layer), so ranks exchange
no data on the data path.  What is left for the host is to deal the matrices out, and to turn the
per-rank device times into one job-wide figure (slowest rank, summed work).

Nothing here touches the method's arithmetic; the functions work with any torch.distributed
backend (NCCL on GPUs, gloo in the CPU tests).
"""
from __future__ import annotations

import torch
import torch.distributed as dist


def assign_matrices(sizes, world):
    """Deals matrices to ranks so that the element counts are balanced.

    sizes: list of (rows, cols).  Returns a list of `world` lists of matrix indices.  Largest
    matrix first, each to the rank with the least work so far (lowest rank on ties), so the
    result is deterministic and every rank computes the same table without communication.
    """
    if world < 1:
        raise ValueError("world must be >= 1")
    order = sorted(range(len(sizes)), key=lambda i: (-int(sizes[i][0]) * int(sizes[i][1]), i))
    load = [0] * world
    out = [[] for _ in range(world)]
    for i in order:
        r = min(range(world), key=lambda q: (load[q], q))
        out[r].append(i)
        load[r] += int(sizes[i][0]) * int(sizes[i][1])
    for lst in out:
        lst.sort()
    return out


def matrix_seed(base_seed, matrix_index):
    """Seed of a matrix of the job: independent of which rank ends up clustering it."""
    return int(base_seed) + int(matrix_index)


def max_over_ranks(value, device="cpu"):
    """Largest `value` (a float, e.g. milliseconds of device time) over all ranks; identity without a group."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(value, device="cpu"):
    """Sum of an integer count (rows, launches) over all ranks."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return int(value)
    t = torch.tensor([int(value)], dtype=torch.int64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return int(t.item())


def job_throughput(units_this_rank, ms_this_rank, device="cpu"):
    """Whole-job units per second: all ranks' units over the slowest rank's time.

    Returns (units per second, total units, max milliseconds)."""
    total = sum_over_ranks(units_this_rank, device)
    ms = max_over_ranks(ms_this_rank, device)
    return total / (ms * 1e-3), total, ms
