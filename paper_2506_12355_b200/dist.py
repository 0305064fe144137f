"""Multi-GPU plumbing: one process per GPU, no data-path collective.

Every (batch, head) pair is an independent attention problem, so the operator shards with
no exchange step: a fixed problem is split by heads (`shard_heads`), and the benchmark's
weak-scaling mode gives every rank its own batch of the same configuration.  The only
communication is the timing protocol (a barrier and a max/sum reduction of scalars).
"""
from __future__ import annotations

import os

import torch
import torch.distributed as dist


def env_world():
    """(rank, local_rank, world_size) from the torchrun environment; (0, 0, 1) when absent."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")),
            int(os.environ.get("WORLD_SIZE", "1")))


def init(backend: str) -> tuple:
    rank, local_rank, world = env_world()
    if world > 1 and not dist.is_initialized():
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        os.environ.setdefault("MASTER_PORT", "29500")
        dist.init_process_group(backend=backend, rank=rank, world_size=world)
    return rank, local_rank, world


def shard_heads(n_heads_total: int, world: int, rank: int) -> tuple:
    """[begin, end) of the flattened (batch*head) axis that `rank` owns: contiguous, balanced to
    within one head, empty for ranks beyond the number of heads."""
    if world <= 0 or not (0 <= rank < world):
        raise ValueError("bad rank/world")
    base, extra = divmod(n_heads_total, world)
    begin = rank * base + min(rank, extra)
    return begin, begin + base + (1 if rank < extra else 0)


def shard_keys(n_keys: int, world: int, rank: int) -> tuple:
    """[begin, end) of the key axis that `rank` owns when K/V are sharded by sequence: contiguous,
    balanced to within one key.  `begin` is the k_offset to hand to attn_fwd_partial."""
    return shard_heads(n_keys, world, rank)


def kv_sharded_attention(q, k_shard, v_shard, scale: float, causal: bool, k_offset: int, stream=None):
    """Attention when every rank holds the full Q but only its own slice of the keys/values.

    Each rank computes the partial result of its shard (attn_fwd_partial), the partial (O_r, LSE_r)
    pairs are all-gathered into this GPU's own memory (NCCL; the one exchange step of this path), and
    attn_combine merges them.  Peer memory is never read by a kernel.  Without a process group the
    single shard is merged alone, which reproduces attn_fwd_gqa.
    """
    from . import api
    o_r, lse_r = api.attn_fwd_partial(q, k_shard, v_shard, scale, causal, k_offset, stream=stream)
    if dist.is_initialized() and dist.get_world_size() > 1:
        world = dist.get_world_size()
        o_parts = torch.empty((world,) + tuple(o_r.shape), dtype=o_r.dtype, device=o_r.device)
        l_parts = torch.empty((world,) + tuple(lse_r.shape), dtype=lse_r.dtype, device=lse_r.device)
        dist.all_gather_into_tensor(o_parts, o_r)
        dist.all_gather_into_tensor(l_parts, lse_r)
    else:
        o_parts, l_parts = o_r.unsqueeze(0), lse_r.unsqueeze(0)
    return api.attn_combine(o_parts.contiguous(), l_parts.contiguous(), stream=stream)


def rank_seed(base_seed: int, rank: int) -> int:
    """Seed of a rank's own batch in weak-scaling runs (rank 0 keeps the single-GPU inputs)."""
    return base_seed + 7919 * rank


def barrier():
    if dist.is_initialized():
        dist.barrier()


def reduce_scalar(x: float, op: str, device) -> float:
    """max or sum of a python float over all ranks (identity without a process group)."""
    if not dist.is_initialized():
        return float(x)
    t = torch.tensor([x], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX if op == "max" else dist.ReduceOp.SUM)
    return float(t.item())
