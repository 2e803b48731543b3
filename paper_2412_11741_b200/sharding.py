"""Host-side helpers for running the codec on several GPUs of one node.

Every input vector is encoded independently and the dictionary is a few MB, so the path
shards by rows with no exchange step: each rank owns a contiguous block of rows, keeps
its own copy of the dictionary and writes its own block of codes.  The only
communication is the bookkeeping below (who owns which rows; the job-wide rate) and one
broadcast when a dictionary is installed or replaced.
"""
from __future__ import annotations

from typing import Tuple

import torch
import torch.distributed as dist

ROW_ALIGN = 256  # one CTA works on 256 rows at a time; blocks start on that boundary


def shard_rows(M: int, rank: int, world: int) -> Tuple[int, int]:
    """[begin, end) of the rows rank owns: blocks of ROW_ALIGN rows dealt as evenly as
    possible, earlier ranks taking the extra block; the last block may be ragged."""
    if not (0 <= rank < world) or M < 0:
        raise ValueError("bad rank/world/M")
    blocks = (M + ROW_ALIGN - 1) // ROW_ALIGN
    base, extra = divmod(blocks, world)
    b0 = rank * base + min(rank, extra)
    b1 = b0 + base + (1 if rank < extra else 0)
    return min(b0 * ROW_ALIGN, M), min(b1 * ROW_ALIGN, M)


def job_rate(units_local: int, seconds_local: float, device: torch.device | str = "cpu") -> float:
    """Whole-job throughput: all ranks' units divided by the slowest rank's time."""
    t = torch.tensor([float(units_local), float(seconds_local)], dtype=torch.float64, device=device)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        units = t[0:1].clone()
        secs = t[1:2].clone()
        dist.all_reduce(units, op=dist.ReduceOp.SUM)
        dist.all_reduce(secs, op=dist.ReduceOp.MAX)
        return float(units.item() / secs.item())
    return float(t[0].item() / t[1].item())


def install_dictionary(D: torch.Tensor, src: int = 0) -> torch.Tensor:
    """Every rank ends up with rank `src`'s dictionary: one broadcast at install time (a new
    prompt's online atoms, a newly trained dictionary), never on the encode path.  D must have
    the same shape and dtype on every rank and is overwritten in place on the others."""
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.broadcast(D, src=src)
    return D
