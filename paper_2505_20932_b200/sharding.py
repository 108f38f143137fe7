"""Multi-GPU plumbing: the hot path shards over rows (tokens).

Forward: rows are independent and the per-token scales are row-local, so every rank runs the fused layer
on its own rows with replicated W / fscale / fbias -- no collective.
Calibration: the five per-channel sums of Eq. 4-5 are additive over row shards, so every rank reduces its
rows with qwt_cwac_stats_accumulate, ONE all-reduce(sum) of 5*C doubles combines them, and every rank solves.
"""
from __future__ import annotations

from typing import Tuple


def shard_rows(total_rows: int, world: int, rank: int, align: int = 1) -> Tuple[int, int]:
    """Contiguous row range (start, count) of `rank`; shard sizes are multiples of `align` except the last
    non-empty one, shards differ by at most `align` rows and cover [0, total_rows) exactly."""
    if world < 1 or not (0 <= rank < world) or total_rows < 0 or align < 1:
        raise ValueError("bad shard request")
    units = -(-total_rows // align)
    base, extra = divmod(units, world)
    u0 = rank * base + min(rank, extra)
    u1 = u0 + base + (1 if rank < extra else 0)
    start = min(u0 * align, total_rows)
    stop = min(u1 * align, total_rows)
    return start, stop - start


def allreduce_stats_(stats) -> None:
    """In-place sum over ranks of a [5*C] float64 statistics tensor (NCCL on GPUs, gloo on CPU)."""
    import torch.distributed as dist
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(stats, op=dist.ReduceOp.SUM)


def max_over_ranks(seconds: float, device=None) -> float:
    """Largest value of a host float over all ranks (timing of a multi-GPU step)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(seconds)
    t = torch.tensor([seconds], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def calibrate_sharded(B, fp_out, q_out, rows_local: int, channels: int, ld: int, a, b, stats, workspace,
                      workspace_bytes: int, stream=None) -> None:
    """CWAC calibration over row shards: local statistics -> all-reduce(sum) -> solve.  `B` is the binding;
    fp_out/q_out hold this rank's rows; `stats` is a zeroed float64 [5*channels] device tensor."""
    import torch
    if rows_local > 0:
        B.qwt_cwac_stats_accumulate(fp_out, q_out, rows_local, channels, ld, stats, workspace, workspace_bytes, stream)
    # The collective is ordered with the CURRENT stream; when the library calls run on a side stream the all-reduce
    # must wait for the local statistics and the solve must wait for the sum over ranks.
    side = stream is not None and getattr(stats, "is_cuda", False)
    if side:
        torch.cuda.current_stream().wait_stream(stream)
    allreduce_stats_(stats)
    if side:
        stream.wait_stream(torch.cuda.current_stream())
    B.qwt_cwac_solve(stats, channels, a, b, None, stream)
