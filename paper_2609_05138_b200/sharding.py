"""Host-side logic of the multi-GPU path: documents are independent, so rank r
searches its own contiguous range of documents against a replica of the
codebook and nothing crosses ranks on the data path.  Only timing (max over
ranks) and, if wanted, the final outputs travel through torch.distributed.
Runs on any backend (NCCL on GPUs, gloo in the CPU tests)."""
from __future__ import annotations

import torch
import torch.distributed as dist


def shard_range(n_docs: int, rank: int, world: int):
    """Contiguous range [lo, hi) of documents for `rank`; sizes differ by at most one."""
    if not (0 <= rank < world):
        raise ValueError("rank %d outside world of %d" % (rank, world))
    base, extra = divmod(n_docs, world)
    lo = rank * base + min(rank, extra)
    return lo, lo + base + (1 if rank < extra else 0)


def shard_csr(rowptr: torch.Tensor, colidx: torch.Tensor, rank: int, world: int):
    """The CSR of this rank's documents, re-based so that rowptr[0] == 0."""
    lo, hi = shard_range(rowptr.numel() - 1, rank, world)
    e0, e1 = int(rowptr[lo]), int(rowptr[hi])
    return (rowptr[lo:hi + 1] - rowptr[lo]).contiguous(), colidx[e0:e1].contiguous()


def job_throughput(units_local: int, seconds_local: float, device="cpu") -> float:
    """Whole-job units per second: all ranks' units over the slowest rank's time."""
    t = torch.tensor([float(seconds_local)], dtype=torch.float64, device=device)
    u = torch.tensor([float(units_local)], dtype=torch.float64, device=device)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(u.item() / t.item())


def gather_outputs(out_local: torch.Tensor, n_docs: int) -> torch.Tensor:
    """All ranks' per-document outputs in the original document order, on every rank."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return out_local
    world = dist.get_world_size()
    sizes = [shard_range(n_docs, r, world) for r in range(world)]
    width = max(hi - lo for lo, hi in sizes)
    padded = torch.zeros(width, dtype=out_local.dtype, device=out_local.device)
    padded[:out_local.numel()] = out_local
    parts = [torch.empty_like(padded) for _ in range(world)]
    dist.all_gather(parts, padded)
    return torch.cat([p[:hi - lo] for p, (lo, hi) in zip(parts, sizes)])
