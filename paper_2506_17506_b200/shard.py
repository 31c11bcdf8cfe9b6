"""Host-side plumbing for running the verifier on several GPUs, one process per GPU.

Candidates are independent (Section 3.4 checks each sampled allocation on its own), so the rows are
split across ranks and no data-path collective is needed: the only exchanges are the reductions of
the timing (max over ranks), of the counts (sum over ranks) that a report needs, and of the first
passing row of the re-sampling statistics (min over ranks).
Nothing here computes any part of the check.
"""
from __future__ import annotations

from typing import Optional, Tuple

import torch
import torch.distributed as dist


def row_range(rank: int, world: int, n_rows: int, align: int = 32) -> Tuple[int, int]:
    """Rows [lo, hi) of a job of n_rows that rank `rank` of `world` checks.

    Shards are contiguous, cover every row once, differ by fewer than 2 * `align` rows, and all but the last
    non-empty one start and end on a multiple of `align` (the verify kernels take candidates 32 at a time).
    """
    if world < 1 or not 0 <= rank < world or n_rows < 0 or align < 1:
        raise ValueError("bad shard request")
    units = (n_rows + align - 1) // align
    base, extra = divmod(units, world)
    lo_u = rank * base + min(rank, extra)
    hi_u = lo_u + base + (1 if rank < extra else 0)
    return min(lo_u * align, n_rows), min(hi_u * align, n_rows)


def weak_rows(rank: int, rows_per_rank: int) -> Tuple[int, int]:
    """Rows of the seeded candidate stream that rank `rank` checks when every rank takes rows_per_rank."""
    return rank * rows_per_rank, (rank + 1) * rows_per_rank


def job_totals(rows_local: int, ms_local: float, passing_local: int = 0,
               device: Optional[torch.device] = None) -> Tuple[int, float, int]:
    """(rows of all ranks, slowest rank's time in ms, passing rows of all ranks).

    Without an initialised process group this is the identity, so a single process needs no launcher.
    """
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return int(rows_local), float(ms_local), int(passing_local)
    dev = device if device is not None else torch.device("cpu")
    s = torch.tensor([rows_local, passing_local], dtype=torch.int64, device=dev)
    t = torch.tensor([ms_local], dtype=torch.float64, device=dev)
    dist.all_reduce(s, op=dist.ReduceOp.SUM)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return int(s[0].item()), float(t[0].item()), int(s[1].item())


def job_sample_stats(first_pass_local: int, n_pass_local: int, rows_local: int, row_offset: int, rows_total: int,
                     device: Optional[torch.device] = None) -> Tuple[int, int]:
    """(first passing row of the whole job, passing rows of the whole job) from every rank's record of
    its own shard (as vl_resample_stats wrote it: first_pass_local == rows_local when the shard has no
    passing row).  row_offset is the job row of the shard's row 0.  The job's first passing row is the
    minimum over ranks of offset + local first (rows_total if no shard has one): one MIN and one SUM
    all-reduce of a single number each.  Identity without a process group."""
    first = row_offset + first_pass_local if first_pass_local < rows_local else rows_total
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return int(first), int(n_pass_local)
    dev = device if device is not None else torch.device("cpu")
    f = torch.tensor([first], dtype=torch.int64, device=dev)
    n = torch.tensor([n_pass_local], dtype=torch.int64, device=dev)
    dist.all_reduce(f, op=dist.ReduceOp.MIN)
    dist.all_reduce(n, op=dist.ReduceOp.SUM)
    return int(f.item()), int(n.item())


def throughput(rows_total: int, ms: float) -> float:
    """Verifications per second of the whole job."""
    return rows_total / (ms * 1e-3) if ms > 0 else 0.0
