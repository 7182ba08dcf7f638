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


# ---- neuron-axis sharding: a codebook too large for one GPU ---------------------
# Rank r holds the columns [j_lo, j_hi) of W, searches every document against its own
# slice and gets (distance, local index) per document.  One exchange step merges them:
# an all-reduce MIN over a 64-bit key whose order is the lexicographic order of
# (distance, global index) -- the same key the kernels use across neuron chunks -- so the
# lowest index still wins a tie.  N x 8 bytes cross NVLink once.
def neuron_range(M: int, rank: int, world: int, multiple: int = 512):
    """Columns [j_lo, j_hi) of rank `rank`: whole multiples of `multiple`, the last rank takes
    the ragged end."""
    if not (0 <= rank < world):
        raise ValueError("rank %d outside world of %d" % (rank, world))
    per = -(-M // world)
    per = -(-per // multiple) * multiple
    lo = min(M, rank * per)
    return lo, min(M, lo + per)


def pack_keys(dist_local: torch.Tensor, bmu_local: torch.Tensor, j_lo: int) -> torch.Tensor:
    """int64 keys ordered like (distance, j_lo + bmu_local); float bits mapped so that integer
    order is float order, then the sign bit flipped so that signed MIN is unsigned MIN."""
    b = dist_local.contiguous().view(torch.int32).to(torch.int64) & 0xFFFFFFFF
    ordered = torch.where(b >= 0x80000000, (~b) & 0xFFFFFFFF, b | 0x80000000)
    key = (ordered << 32) | (bmu_local.to(torch.int64) + int(j_lo))
    return key ^ (-0x8000000000000000)


def unpack_keys(key: torch.Tensor):
    """(distance float32, global index int32) of packed keys."""
    key = key ^ (-0x8000000000000000)
    idx = (key & 0xFFFFFFFF).to(torch.int32)
    ordered = (key >> 32) & 0xFFFFFFFF
    b = torch.where(ordered >= 0x80000000, ordered & 0x7FFFFFFF, (~ordered) & 0xFFFFFFFF)
    b = torch.where(b >= 0x80000000, b - 0x100000000, b).to(torch.int32)
    return b.view(torch.float32), idx


def merge_neuron_shards(dist_local: torch.Tensor, bmu_local: torch.Tensor, j_lo: int):
    """Best unit over all ranks' neuron slices: (distance, global index) on every rank."""
    key = pack_keys(dist_local, bmu_local, j_lo)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(key, op=dist.ReduceOp.MIN)
    return unpack_keys(key)
