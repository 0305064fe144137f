"""The multi-rank path on CPU: two gloo ranks split one problem by heads (no collective on the data
path), each computes its shard, and the gathered result equals the unsharded one."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2506_12355_b200 import dist as adist
from paper_2506_12355_b200 import inputs


def test_shard_heads_partitions_exactly():
    for total in (0, 1, 5, 32, 33, 128):
        for world in (1, 2, 3, 8):
            spans = [adist.shard_heads(total, world, r) for r in range(world)]
            assert spans[0][0] == 0 and spans[-1][1] == total
            for a, b in zip(spans, spans[1:]):
                assert a[1] == b[0]
            sizes = [e - b for b, e in spans]
            assert max(sizes) - min(sizes) <= 1
    with pytest.raises(ValueError):
        adist.shard_heads(4, 2, 2)


def test_rank_seed_distinct():
    assert adist.rank_seed(100, 0) == 100
    assert len({adist.rank_seed(100, r) for r in range(8)}) == 8


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank, world, port, out_path):
    from oracle import attn_oracle as orc
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    r, _, w = adist.init("gloo")
    assert (r, w) == (rank, world)
    B, H, Sq, Sk, D = 1, 5, 24, 40, 16
    q, k, v = inputs.make_qkv(B, H, Sq, Sk, D, inputs.DTYPE_FP16, seed=11)
    qf, kf, vf = (orc.widen(inputs.bits(t), 0).reshape(B * H, -1, D) for t in (q, k, v))
    b, e = adist.shard_heads(B * H, world, rank)
    o, lse = orc.attention(qf[None, b:e], kf[None, b:e], vf[None, b:e], 0.25, True)
    # gather the shards (the caller's job; the operator itself needs no exchange)
    gathered = [None] * world
    dist.all_gather_object(gathered, (b, e, o[0], lse[0]))
    t_max = adist.reduce_scalar(float(rank + 1), "max", "cpu")
    t_sum = adist.reduce_scalar(float(rank + 1), "sum", "cpu")
    adist.barrier()
    if rank == 0:
        full_o = np.concatenate([g[2] for g in sorted(gathered, key=lambda g: g[0])])
        full_l = np.concatenate([g[3] for g in sorted(gathered, key=lambda g: g[0])])
        ref_o, ref_l = orc.attention(qf[None], kf[None], vf[None], 0.25, True)
        ok = (np.array_equal(full_o, ref_o[0]) and np.array_equal(full_l, ref_l[0])
              and t_max == world and t_sum == world * (world + 1) / 2)
        open(out_path, "w").write("ok" if ok else "mismatch")
    dist.destroy_process_group()


def test_two_gloo_ranks_shard_by_heads(tmp_path):
    out = str(tmp_path / "result.txt")
    mp.spawn(_worker, args=(2, _free_port(), out), nprocs=2, join=True)
    assert open(out).read() == "ok"


def _kv_worker(rank, world, port, out_path):
    """Key/value sharding on CPU: every rank evaluates its own key slice with the oracle's shard entry
    (global key offset from shard_keys), the partial (O, LSE) pairs are exchanged, and the merge equals
    the unsharded result."""
    from oracle import attn_oracle as orc
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    adist.init("gloo")
    B, H, Sq, Sk, D = 1, 2, 37, 53, 8
    q, k, v = inputs.make_qkv(B, H, Sq, Sk, D, inputs.DTYPE_FP16, seed=21)
    qf, kf, vf = (orc.widen(inputs.bits(t), 0) for t in (q, k, v))
    b, e = adist.shard_keys(Sk, world, rank)
    o_r, l_r = orc.attention_shard(qf, kf[:, :, b:e], vf[:, :, b:e], 0.3, True, b)
    got_o = [torch.zeros(B, H, Sq, D, dtype=torch.float64) for _ in range(world)]
    got_l = [torch.zeros(B, H, Sq, dtype=torch.float64) for _ in range(world)]
    dist.all_gather(got_o, torch.from_numpy(o_r))
    dist.all_gather(got_l, torch.from_numpy(l_r))
    o, lse = orc.combine(np.stack([t.numpy() for t in got_o]), np.stack([t.numpy() for t in got_l]))
    o_ref, l_ref = orc.attention(qf, kf, vf, 0.3, True)
    ok = np.allclose(o, o_ref, atol=1e-12) and np.allclose(lse, l_ref, atol=1e-12)
    flags = [None] * world
    dist.all_gather_object(flags, bool(ok))
    if rank == 0:
        open(out_path, "w").write("ok" if all(flags) else "mismatch")
    dist.destroy_process_group()


def test_two_gloo_ranks_shard_by_keys_and_merge(tmp_path):
    out = str(tmp_path / "result_kv.txt")
    mp.spawn(_kv_worker, args=(2, _free_port(), out), nprocs=2, join=True)
    assert open(out).read() == "ok"


def _kv_glue_worker(rank, world, port, out_path):
    """Drives dist.kv_sharded_attention itself (exchange="nccl" shape of the control flow: partial call, two
    all-gathers into the rank's own memory, merge) on two gloo ranks, with the two library calls replaced by the
    shard and merge arithmetic of the oracle on CPU tensors.  Checks the glue: offsets, gather order, shapes."""
    from oracle import attn_oracle as orc
    from paper_2506_12355_b200 import api
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    adist.init("gloo")
    calls = []

    def fake_partial(q, k, v, scale, causal, k_offset, out=None, lse=None, stream=None):
        calls.append(("partial", k_offset, tuple(k.shape)))
        o, l = orc.attention_shard(q.numpy(), k.numpy(), v.numpy(), scale, causal, k_offset)
        return torch.from_numpy(o), torch.from_numpy(l)

    def fake_combine(o_parts, lse_parts, out=None, lse=None, stream=None):
        calls.append(("combine", tuple(o_parts.shape)))
        o, l = orc.combine(o_parts.numpy(), lse_parts.numpy())
        return torch.from_numpy(o), torch.from_numpy(l)

    api.attn_fwd_partial, api.attn_combine = fake_partial, fake_combine
    B, H, Sq, Sk, D = 2, 2, 19, 45, 8
    q, k, v = inputs.make_qkv(B, H, Sq, Sk, D, inputs.DTYPE_FP16, seed=31)
    qf, kf, vf = (torch.from_numpy(orc.widen(inputs.bits(t), 0)) for t in (q, k, v))
    b, e = adist.shard_keys(Sk, world, rank)
    o, lse = adist.kv_sharded_attention(qf, kf[:, :, b:e].contiguous(), vf[:, :, b:e].contiguous(), 0.3, True, b,
                                        exchange="nccl")
    o_ref, l_ref = orc.attention(qf.numpy(), kf.numpy(), vf.numpy(), 0.3, True)
    ok = (np.allclose(o.numpy(), o_ref, atol=1e-12) and np.allclose(lse.numpy(), l_ref, atol=1e-12)
          and calls == [("partial", b, (B, H, e - b, D)), ("combine", (world, B, H, Sq, D))])
    flags = [None] * world
    dist.all_gather_object(flags, bool(ok))
    if rank == 0:
        open(out_path, "w").write("ok" if all(flags) else "mismatch")
    dist.destroy_process_group()


def test_two_gloo_ranks_drive_kv_sharded_attention_glue(tmp_path):
    out = str(tmp_path / "result_glue.txt")
    mp.spawn(_kv_glue_worker, args=(2, _free_port(), out), nprocs=2, join=True)
    assert open(out).read() == "ok"


def test_kv_sharded_attention_rejects_unknown_exchange():
    with pytest.raises(ValueError):
        adist.kv_sharded_attention(None, None, None, 1.0, False, 0, exchange="carrier pigeon")


def test_shard_keys_offsets():
    assert [adist.shard_keys(10, 3, r) for r in range(3)] == [(0, 4), (4, 7), (7, 10)]
