"""Multi-GPU plumbing: one process per GPU.

Every (batch, head) pair is an independent attention problem, so the operator shards with
no exchange step: a fixed problem is split by heads (`shard_heads`), and the benchmark's
weak-scaling mode gives every rank its own batch of the same configuration; the only
communication there is the timing protocol (a barrier and a max/sum reduction of scalars).
When heads run out, the keys are sharded instead (`kv_sharded_attention`), which has one
exchange step: the partial results, gathered by NCCL or read in place by the merge kernel.
"""
from __future__ import annotations

import datetime
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
        # a bounded rendezvous / collective timeout: a rank that never joins ends the others with an error
        dist.init_process_group(backend=backend, rank=rank, world_size=world,
                                timeout=datetime.timedelta(seconds=int(os.environ.get("ATTN_DIST_TIMEOUT_S", "300"))))
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


_peer_buffers = {}   # (shape, dtype, device) -> (o_buf, lse_buf, o_handle, lse_handle): rendezvous is done once per shape


def _peer_partials(o_shape, lse_shape, dtype, device):
    """Partial-result buffers in symmetric memory, with every rank's pointers to them (cached per shape)."""
    import torch.distributed._symmetric_memory as symm_mem
    key = (tuple(o_shape), dtype, str(device))
    if key not in _peer_buffers:
        o_buf = symm_mem.empty(tuple(o_shape), dtype=dtype, device=device)
        l_buf = symm_mem.empty(tuple(lse_shape), dtype=torch.float32, device=device)
        group = dist.group.WORLD
        _peer_buffers[key] = (o_buf, l_buf, symm_mem.rendezvous(o_buf, group), symm_mem.rendezvous(l_buf, group))
    return _peer_buffers[key]


def _all_gather_stacked(out, x):
    """out[r] = rank r's x.  NCCL gathers straight into the stacked tensor; other backends (the CPU tests run on
    gloo, which has no single-tensor all-gather) receive into its slices."""
    if dist.get_backend() == "nccl":
        dist.all_gather_into_tensor(out, x)
    else:
        dist.all_gather(list(out.unbind(0)), x)


def _on_stream(stream):
    """Context that makes `stream` torch's current stream (a no-op for None or CPU tensors), so that torch's
    collectives, the symmetric-memory barriers and the library's kernels are all ordered on ONE stream."""
    import contextlib
    if stream is None or not torch.cuda.is_available():
        return contextlib.nullcontext()
    return torch.cuda.stream(stream)


def kv_sharded_attention(q, k_shard, v_shard, scale: float, causal: bool, k_offset: int, stream=None,
                         exchange: str = "nccl"):
    """Attention when every rank holds the full Q but only its own slice of the keys/values.

    Each rank computes the partial result of its shard (attn_fwd_partial); the partial (O_r, LSE_r) pairs are
    then merged.  exchange="nccl": they are all-gathered into this GPU's own memory (the process group's
    collective; the one exchange step of this path) and attn_combine merges them; no kernel reads peer memory.
    exchange="peer": the partial results are written into symmetric memory and ONE kernel (attn_combine_gather)
    reads every rank's partial result in place over NVLink with plain loads and merges: exchange and merge fused,
    nothing gathered first (needs torch's symmetric memory and peer access between the GPUs; a barrier across the
    ranks orders it after the partial kernels, a second one keeps the partial results alive until every rank has
    read them).  Without a process group the single shard is merged alone, which reproduces attn_fwd_gqa.

    Everything is enqueued on `stream` (default: torch's current stream), which is made the current stream for
    the duration of the call: the collectives and the symmetric-memory barriers are ordered against torch's
    current stream, so they and the kernels must share it.
    """
    from . import api
    if exchange not in ("nccl", "peer"):
        raise ValueError("exchange must be 'nccl' or 'peer'")
    multi = dist.is_initialized() and dist.get_world_size() > 1
    with _on_stream(stream):
        if multi and exchange == "peer":
            B, H, Sq, D = q.shape
            o_buf, l_buf, o_hdl, l_hdl = _peer_partials((B, H, Sq, D), (B, H, Sq), q.dtype, q.device)
            api.attn_fwd_partial(q, k_shard, v_shard, scale, causal, k_offset, out=o_buf, lse=l_buf, stream=stream)
            o_hdl.barrier()          # every rank's partial result is complete
            out = torch.empty_like(o_buf)
            lse = torch.empty_like(l_buf)
            api.attn_combine_gather(list(o_hdl.buffer_ptrs), list(l_hdl.buffer_ptrs), (B, H, Sq, D), q.dtype, out,
                                    lse, stream=stream)
            o_hdl.barrier()          # nobody overwrites its partial result while a peer still reads it
            return out, lse
        o_r, lse_r = api.attn_fwd_partial(q, k_shard, v_shard, scale, causal, k_offset, stream=stream)
        if multi:
            world = dist.get_world_size()
            o_parts = torch.empty((world,) + tuple(o_r.shape), dtype=o_r.dtype, device=o_r.device)
            l_parts = torch.empty((world,) + tuple(lse_r.shape), dtype=lse_r.dtype, device=lse_r.device)
            _all_gather_stacked(o_parts, o_r)
            _all_gather_stacked(l_parts, lse_r)
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
