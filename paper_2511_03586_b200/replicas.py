"""Data-parallel plumbing for running the layer on several GPUs.

Rows, GEMM row blocks and whole sequences are independent (attention mixes only
within a sequence) and the weights are small enough to replicate, so the path
shards with no exchange step: every rank runs the same kernels on its own
sequences.  The only communication is the bookkeeping here - who owns which
sequences, and the max-over-ranks step time of a measurement - done with
``torch.distributed`` on whatever backend the process group has (NCCL on GPUs,
gloo in the CPU tests).  Nothing in this module touches the CUDA library.
"""
from __future__ import annotations

import torch
import torch.distributed as dist


def shard_sequences(n_sequences: int, rank: int, world: int) -> range:
    """Contiguous block of sequence indices owned by ``rank`` (sizes differ by at most one)."""
    if not (0 <= rank < world):
        raise ValueError("rank out of range")
    base, extra = divmod(n_sequences, world)
    start = rank * base + min(rank, extra)
    return range(start, start + base + (1 if rank < extra else 0))


def max_over_ranks(values, device="cpu", group=None):
    """Element-wise maximum of a list of floats over all ranks (identity when not distributed)."""
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size(group) > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX, group=group)
    return [float(v) for v in t]


def whole_job_rate(units_per_rank_step: float, ms_per_step_local: float, device="cpu", group=None) -> dict:
    """Whole-job throughput of a weak-scaling run: every rank does ``units_per_rank_step`` units per step;
    the job's step time is the slowest rank's."""
    world = dist.get_world_size(group) if dist.is_available() and dist.is_initialized() else 1
    (ms,) = max_over_ranks([ms_per_step_local], device=device, group=group)
    return {"world": world, "ms_per_step": ms, "units_per_s": world * units_per_rank_step / (ms * 1e-3)}
