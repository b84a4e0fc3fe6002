"""Multi-GPU plumbing.

Default: the path shards over independent layers, one per rank, with no data-path collective (the paper
computes Hessians of different layers / groups on different GPUs, Section 3.2 and Appendix C); the only
communication is the reduction of timings and of per-rank scalar results.

Token sharding of ONE layer (H_k is a sum over tokens, Algorithm 1, Hessian step): every rank accumulates the chunks
`chunks_for_rank` gives it into its own H, then `exchange_hessian` adds the partial matrices with the library's
reduce / gather kernels over peer memory, the ranks meeting at host barriers in between."""
from __future__ import annotations

from typing import Sequence

import torch
import torch.distributed as dist


def layer_seed_for_rank(base_seed: int, rank: int) -> int:
    """Every rank works on its own synthetic layer: distinct seeds, same shape."""
    return int(base_seed) + int(rank)


def max_over_ranks(values: Sequence[float], device="cpu") -> list:
    """Element-wise maximum over all ranks of a few host scalars (timings)."""
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t.cpu()]


def gather_scalars(value: float, device="cpu") -> list:
    """All ranks' values of one host scalar, in rank order (e.g. each layer's objective)."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return [float(value)]
    t = torch.tensor([value], dtype=torch.float64, device=device)
    out = [torch.zeros_like(t) for _ in range(dist.get_world_size())]
    dist.all_gather(out, t)
    return [float(o.item()) for o in out]


def whole_job_throughput(units_per_rank: int, steps: int, max_seconds: float, world: int) -> float:
    """Units all ranks processed divided by the slowest rank's time."""
    return float(units_per_rank) * world * steps / max_seconds


def chunks_for_rank(n_chunks: int, rank: int, world: int) -> list:
    """Token chunks of one layer that rank `rank` accumulates (round-robin: every chunk exactly once)."""
    return list(range(int(rank), int(n_chunks), int(world)))


def allocate_symmetric_hessian(g: int, d_in: int, device, group=None):
    """H of this rank in memory every rank of `group` can address, zeroed, and all ranks' pointers to it
    (index = rank) as this process sees them."""
    import torch.distributed._symmetric_memory as symm_mem
    H = symm_mem.empty((g, d_in, d_in), dtype=torch.float32, device=device)
    H.zero_()
    handle = symm_mem.rendezvous(H, group=group if group is not None else dist.group.WORLD)
    return H, [int(p) for p in handle.buffer_ptrs]


def exchange_hessian(H: torch.Tensor, rank_ptrs: Sequence, rank: int, group=None, ops=None) -> torch.Tensor:
    """After every rank has accumulated its chunks into its H: make every rank's H the full sum and complete
    it (finalize).  `rank_ptrs[r]` is rank r's H as addressable from this GPU (`rank_ptrs[rank]` is `H`).
    `ops` supplies gq_hessian_reduce_share / gq_hessian_gather_shares / gq_hessian_finalize (default: the
    library binding); the sequence of calls and meeting points is what this function owns."""
    if ops is None:
        from . import api as ops
    g, d_in = int(H.shape[0]), int(H.shape[1])

    def meet():
        if H.is_cuda:
            torch.cuda.current_stream(H.device).synchronize()
        if dist.is_available() and dist.is_initialized() and dist.get_world_size(group) > 1:
            dist.barrier(group)

    if len(rank_ptrs) > 1:
        meet()                                            # all partial matrices are complete
        ops.gq_hessian_reduce_share(rank_ptrs, rank, d_in, g)
        meet()                                            # all shares are reduced
        ops.gq_hessian_gather_shares(rank_ptrs, rank, d_in, g)
        meet()                                            # nobody reads this rank's H any more
    ops.gq_hessian_finalize(H)
    return H


def exchange_bytes_per_rank(d_in: int, g: int, world: int, block: int = 128) -> int:
    """Bytes one rank reads from its peers in the two steps of `exchange_hessian` together: in the reduce step its
    own share of the 128 x 128 blocks of the upper triangle from the other world - 1 matrices, in the gather step
    the other ranks' shares; each is (world - 1) / world of the blocks."""
    nb = (int(d_in) + block - 1) // block
    blocks = int(g) * nb * (nb + 1) // 2
    return 2 * (blocks * (int(world) - 1) // int(world)) * block * block * 4
