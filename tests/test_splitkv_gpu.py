"""GPU parity of the split-KV entry point (key ranges as concurrent launches + merge) against the fp64 CPU
oracle of the whole problem.  The ranges' partial outputs are stored in the 16-bit type before the merge, so O
carries two 16-bit roundings instead of one: the O bar is 1.5 x that of attn_fwd (1.5e-2 fp16, 3e-2 bf16);
LSE 1e-3."""
import numpy as np
import pytest
import torch

from oracle import attn_oracle as orc
from paper_2506_12355_b200 import api, inputs

pytestmark = pytest.mark.gpu

O_TOL = {inputs.DTYPE_FP16: 1.5e-2, inputs.DTYPE_BF16: 3e-2}
LSE_TOL = 1e-3

CASES = [
    # D, dtype, causal, B, H, Hkv, Sq, Sk, n_splits
    (128, 1, False, 2, 8, 2, 1, 5000, 8),      # decoding: one query per head, grouped K/V heads
    (128, 1, False, 1, 4, 4, 1, 5000, 3),
    (64, 0, False, 1, 6, 2, 64, 4173, 5),      # a few queries, ragged last range
    (256, 0, False, 1, 2, 1, 130, 1500, 4),
    (128, 0, True, 1, 3, 3, 1000, 1000, 4),    # causal: early rows see no key of the later ranges
    (64, 1, True, 2, 2, 1, 300, 700, 64),      # more ranges asked for than there are 128-key tiles
    (128, 1, False, 1, 2, 2, 200, 100, 4),     # a single tile: falls back to the plain call
]


@pytest.mark.parametrize("D,dt,causal,B,H,Hkv,Sq,Sk,n", CASES)
def test_splitkv_against_oracle(D, dt, causal, B, H, Hkv, Sq, Sk, n):
    dev = torch.device("cuda:0")
    q = inputs.randn16((B, H, Sq, D), 8100 + Sk, dt)
    k = inputs.randn16((B, Hkv, Sk, D), 8200 + Sk, dt)
    v = inputs.randn16((B, Hkv, Sk, D), 8300 + Sk, dt)
    scale = D ** -0.5
    o, lse = api.attn_fwd_splitkv(q.to(dev), k.to(dev), v.to(dev), scale, causal, n)
    assert api.attn_last_device_status() == 0
    qf, kf, vf = (orc.widen(inputs.bits(t), dt) for t in (q, k, v))
    o_ref, lse_ref = orc.attention_gqa(qf, kf, vf, scale, causal)
    o64 = o.cpu().to(torch.float64).numpy()
    l64 = lse.cpu().to(torch.float64).numpy()
    assert not np.isnan(o64).any()
    assert np.abs(o64 - o_ref).max() <= O_TOL[dt], "max |dO| = %g" % np.abs(o64 - o_ref).max()
    assert np.abs(l64 - lse_ref).max() <= LSE_TOL


def test_splitkv_one_range_is_the_plain_call_and_reuse_of_the_workspace():
    dev = torch.device("cuda:0")
    q, k, v = inputs.make_qkv(1, 4, 3, 3000, 128, 1, seed=8400)
    qd, kd, vd = q.to(dev), k.to(dev), v.to(dev)
    o1, l1 = api.attn_fwd_splitkv(qd, kd, vd, 0.1, False, 1)
    o0, l0 = api.attn_fwd(qd, kd, vd, 0.1, False)
    assert torch.equal(o1, o0) and torch.equal(l1, l0)
    ws = torch.empty(api.attn_fwd_splitkv_workspace_bytes(1, 4, 3, 128, 6), dtype=torch.uint8, device=dev)
    a = api.attn_fwd_splitkv(qd, kd, vd, 0.1, False, 6, workspace=ws)
    b = api.attn_fwd_splitkv(qd, kd, vd, 0.1, False, 6, workspace=ws)   # same stream, same workspace: ordered
    torch.cuda.synchronize()
    assert api.attn_last_device_status() == 0
    assert torch.equal(a[0], b[0]) and torch.equal(a[1], b[1])
    assert (a[0].float() - o0.float()).abs().max().item() <= 3e-2 and (a[1] - l0).abs().max().item() <= 1e-3


def test_splitkv_rejects_bad_arguments():
    dev = torch.device("cuda:0")
    q, k, v = inputs.make_qkv(1, 2, 1, 1024, 128, 1, seed=8500)
    qd, kd, vd = q.to(dev), k.to(dev), v.to(dev)
    for n in (0, 65, -3):
        with pytest.raises(api.AttnError) as e:
            api.attn_fwd_splitkv(qd, kd, vd, 0.1, False, n, workspace=torch.empty(1 << 20, dtype=torch.uint8, device=dev))
        assert e.value.status == 2
    with pytest.raises(api.AttnError) as e:
        api.attn_fwd_splitkv(qd, kd, vd, 0.1, False, 4, workspace=torch.empty(256, dtype=torch.uint8, device=dev))
    assert e.value.status == 10


def test_splitkv_in_a_cuda_graph():
    # the concurrent launches on the library's own streams fork from and join the capturing stream, so the whole
    # call (counter resets, partial launches, merge) is one graph; a decoding loop replays it
    dev = torch.device("cuda:0")
    q, k, v = inputs.make_qkv(1, 8, 1, 8192, 128, 1, seed=8600)
    qd, kd, vd = q.to(dev), k.to(dev), v.to(dev)
    ws = torch.empty(api.attn_fwd_splitkv_workspace_bytes(1, 8, 1, 128, 8), dtype=torch.uint8, device=dev)
    ref_o, ref_l = api.attn_fwd_splitkv(qd, kd, vd, 0.09, False, 8, workspace=ws)   # one-time set-up outside capture
    torch.cuda.synchronize()
    o = torch.empty_like(ref_o)
    lse = torch.empty_like(ref_l)
    g = torch.cuda.CUDAGraph()
    st = torch.cuda.Stream(device=dev)
    with torch.cuda.stream(st):
        with torch.cuda.graph(g, stream=st):
            api.attn_fwd_splitkv(qd, kd, vd, 0.09, False, 8, workspace=ws, out=o, lse=lse, stream=st)
    for _ in range(3):
        o.zero_()
        g.replay()
    torch.cuda.synchronize()
    assert api.attn_last_device_status() == 0
    assert torch.equal(o.view(torch.int16), ref_o.view(torch.int16)) and torch.equal(lse, ref_l)


def test_bench_kv_sharded_check_single_rank():
    # the check that bench.py adds to its line at N > 1, driven here with one rank (no process group: the single
    # shard is merged alone): its input recipe, both exchange branches and the oracle comparison run end to end
    import os
    import sys
    sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
    import bench
    res = bench.kv_sharded_check(api, torch.device("cuda:0"), 0, 1)
    for exchange in ("nccl", "peer"):
        assert isinstance(res[exchange], dict), res[exchange]
        assert res[exchange]["max_abs_o"] <= 2e-2 and res[exchange]["max_abs_lse"] <= 1e-3
