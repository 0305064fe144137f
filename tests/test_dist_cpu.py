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
