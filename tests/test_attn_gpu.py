"""GPU parity: the CUDA path (through the C ABI) against the fp64 CPU oracle, element by element
on the same seeded inputs.  Tolerances (max-abs): O 1e-2 for fp16, 2e-2 for bf16; LSE 1e-3."""
import json
import math
import os

import numpy as np
import pytest
import torch

from oracle import attn_oracle as orc
from paper_2506_12355_b200 import api, inputs

pytestmark = pytest.mark.gpu

O_TOL = {inputs.DTYPE_FP16: 1e-2, inputs.DTYPE_BF16: 2e-2}
LSE_TOL = 1e-3
GUARD = 4096  # canary elements on both sides of every output buffer


def guarded(shape, dtype, device):
    n = int(np.prod(shape))
    buf = torch.full((n + 2 * GUARD,), float("nan"), dtype=dtype, device=device)
    return buf, buf[GUARD:GUARD + n].view(shape)


def guards_intact(buf):
    return bool(torch.isnan(buf[:GUARD]).all()) and bool(torch.isnan(buf[-GUARD:]).all())


def f32_scale(D):
    """1/sqrt(D) as the fp32 value that crosses the C ABI, widened to a Python float: the oracle
    is given exactly the number the kernels see."""
    return float(np.float32(1.0) / np.sqrt(np.float32(D)))


def run_gpu(fn, q, k, v, scale, causal):
    dev = torch.device("cuda:0")
    qd, kd, vd = q.to(dev), k.to(dev), v.to(dev)
    B, H, Sq, D = q.shape
    obuf, o = guarded((B, H, Sq, D), q.dtype, dev)
    lbuf, lse = guarded((B, H, Sq), torch.float32, dev)
    fn(qd, kd, vd, scale, causal, out=o, lse=lse)
    assert api.attn_last_device_status() == 0, "a kernel reported a timed-out wait"
    assert guards_intact(obuf) and guards_intact(lbuf), "write outside the output buffers"
    return o.cpu(), lse.cpu()


def check_against_oracle(fn, q, k, v, dtype, scale, causal, o_tol=None):
    o, lse = run_gpu(fn, q, k, v, scale, causal)
    qf, kf, vf = (orc.widen(inputs.bits(t), dtype) for t in (q, k, v))
    o_ref, lse_ref = orc.attention(qf, kf, vf, scale, causal)
    o64 = o.to(torch.float64).numpy()
    assert not np.isnan(o64).any(), "NaN in O (unwritten canary or arithmetic NaN)"
    err_o = np.abs(o64 - o_ref)
    where = np.unravel_index(err_o.argmax(), err_o.shape) if err_o.size else None
    tol = O_TOL[dtype] if o_tol is None else o_tol
    assert err_o.size == 0 or err_o.max() <= tol, "max |dO| = %g at %s" % (err_o.max(), where)
    l64 = lse.to(torch.float64).numpy()
    inf = np.isneginf(lse_ref)
    assert np.array_equal(np.isneginf(l64), inf)
    err_l = np.abs(l64[~inf] - lse_ref[~inf])
    assert err_l.size == 0 or err_l.max() <= LSE_TOL, "max |dLSE| = %g" % err_l.max()


IMPLS = {"tc": api.attn_fwd, "simt": api.attn_fwd_simt}


# ------------------------------------------------------------------ small shapes, full comparison

SMALL = [
    # B, H, Sq, Sk
    (1, 2, 128, 128),
    (1, 1, 1, 1),
    (1, 3, 17, 17),
    (2, 1, 127, 127),
    (1, 1, 129, 129),
    (1, 2, 255, 255),
    (1, 1, 100, 333),
    (1, 1, 257, 129),
    (1, 1, 384, 640),
]


@pytest.mark.parametrize("impl", ["tc", "simt"])
@pytest.mark.parametrize("causal", [False, True])
@pytest.mark.parametrize("dtype", [inputs.DTYPE_FP16, inputs.DTYPE_BF16])
@pytest.mark.parametrize("D", [64, 128, 256])
@pytest.mark.parametrize("shape", SMALL)
def test_small_shapes(shape, D, dtype, causal, impl):
    B, H, Sq, Sk = shape
    if impl == "simt" and (D == 256 or Sq * Sk > 70000) and dtype == inputs.DTYPE_BF16:
        pytest.skip("cross-check kernel: subset only")
    q, k, v = inputs.make_qkv(B, H, Sq, Sk, D, dtype, seed=1000 + Sq * 7 + Sk + D)
    check_against_oracle(IMPLS[impl], q, k, v, dtype, f32_scale(D), causal)


def test_config_c1_full():
    cfg = inputs.CONFIGS["C1"]
    q, k, v = inputs.make_config_inputs(cfg)
    check_against_oracle(api.attn_fwd, q, k, v, cfg.dtype, cfg.scale, cfg.causal)


@pytest.mark.parametrize("D,dtype,causal", [(64, 0, False), (128, 1, True), (256, 0, False), (128, 0, True),
                                            (64, 1, True)])
def test_several_tiles_and_ragged_tail(D, dtype, causal):
    # several 128-row Q tiles and K/V tiles plus a ragged tail, several heads
    q, k, v = inputs.make_qkv(2, 3, 128 * 3 + 37, 128 * 4 + 91, D, dtype, seed=4242 + D)
    check_against_oracle(api.attn_fwd, q, k, v, dtype, f32_scale(D), causal)


# ------------------------------------------------------------------ hand-derived cases on the GPU

def test_hand_case_2x2_padded_into_d64():
    # the 2x2 case of tests/golden/hand_cases.json: exactly representable in fp16, zero-padded to D = 64
    c = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "hand_cases.json")))["case_2x2"]
    e = math.e
    for causal, want_o, want_l in (
            (False, [[(e + 3) / (e + 1), (2 * e + 4) / (e + 1)], [(1 + 3 * e) / (e + 1), (2 + 4 * e) / (e + 1)]],
             [math.log(e + 1)] * 2),
            (True, [[1.0, 2.0], [(1 + 3 * e) / (e + 1), (2 + 4 * e) / (e + 1)]], [1.0, math.log(e + 1)])):
        for dt in (torch.float16, torch.bfloat16):
            q = torch.zeros(1, 1, 2, 64, dtype=dt)
            k = torch.zeros(1, 1, 2, 64, dtype=dt)
            v = torch.zeros(1, 1, 2, 64, dtype=dt)
            q[0, 0, :, :2] = torch.tensor(c["Q"], dtype=dt)
            k[0, 0, :, :2] = torch.tensor(c["K"], dtype=dt)
            v[0, 0, :, :2] = torch.tensor(c["V"], dtype=dt)
            o, lse = run_gpu(api.attn_fwd, q, k, v, 1.0, causal)
            tol = 1e-2 if dt == torch.float16 else 2e-2
            np.testing.assert_allclose(o[0, 0, :, :2].double().numpy(), np.array(want_o), atol=tol)
            assert float(o[0, 0, :, 2:].abs().max()) == 0.0
            np.testing.assert_allclose(lse[0, 0].double().numpy(), np.array(want_l), atol=1e-3)


# ------------------------------------------------------------------ structured inputs (layout mistakes)

@pytest.mark.parametrize("D", [64, 128, 256])
def test_constant_v_and_distinct_columns(D):
    # V column d holds the value d/8 in every row -> O[:, d] = d/8 exactly representable
    B, H, Sq, Sk = 1, 2, 200, 300
    q, k, _ = inputs.make_qkv(B, H, Sq, Sk, D, inputs.DTYPE_FP16, seed=99)
    v = (torch.arange(D, dtype=torch.float32) / 8).to(torch.float16).expand(B, H, Sk, D).contiguous()
    o, _ = run_gpu(api.attn_fwd, q, k, v, 0.125, False)
    want = (torch.arange(D, dtype=torch.float64) / 8).expand(B, H, Sq, D)
    assert float((o.double() - want).abs().max()) <= 2e-2   # |O| up to 32: fp16 spacing there is 1/64..1/32


@pytest.mark.parametrize("D", [64, 128, 256])
def test_one_hot_selection_follows_key_index(D):
    # query i matches key perm[i] strongly -> O row i must be V[perm[i]]: catches transposed or
    # permuted K/V/P tiles
    Sq = Sk = 256
    g = torch.Generator().manual_seed(7)
    perm = torch.randperm(Sk, generator=g)
    basis = torch.zeros(Sk, D)
    # distinct +-1 codes per key: code of key j = binary digits of j spread over the first 16 dims
    for bit in range(8):
        basis[:, bit] = ((torch.arange(Sk) >> bit) & 1).float() * 2 - 1
    k = basis.to(torch.float16).view(1, 1, Sk, D).contiguous()
    q = basis[perm].to(torch.float16).view(1, 1, Sq, D).contiguous()
    v = inputs.randn16((1, 1, Sk, D), 5, inputs.DTYPE_FP16)
    o, lse = run_gpu(api.attn_fwd, q, k, v, 16.0, False)   # score gap between best and next: 2*16
    want = v[0, 0, perm].double()
    assert float((o[0, 0].double() - want).abs().max()) <= 1e-2
    np.testing.assert_allclose(lse[0, 0].numpy(), np.full(Sq, 8 * 16.0), atol=1e-3)


def test_zero_scale_and_no_keys():
    q, k, v = inputs.make_qkv(1, 2, 150, 150, 64, inputs.DTYPE_BF16, seed=31)
    check_against_oracle(api.attn_fwd, q, k, v, inputs.DTYPE_BF16, 0.0, True)
    # Sk == 0: O = 0, LSE = -inf
    k0 = torch.empty(1, 2, 0, 64, dtype=torch.bfloat16)
    o, lse = run_gpu(api.attn_fwd, q, k0, k0, 0.125, False)
    assert float(o.abs().max()) == 0.0 and bool(torch.isneginf(lse).all())


def test_large_logits_do_not_overflow():
    q, k, v = inputs.make_qkv(1, 1, 256, 256, 128, inputs.DTYPE_FP16, seed=32)
    check_against_oracle(api.attn_fwd, q, k, v, inputs.DTYPE_FP16, 8.0, False)


def test_bitwise_deterministic():
    q, k, v = inputs.make_qkv(2, 4, 512, 512, 128, inputs.DTYPE_BF16, seed=33)
    o1, l1 = run_gpu(api.attn_fwd, q, k, v, 0.09, True)
    o2, l2 = run_gpu(api.attn_fwd, q, k, v, 0.09, True)
    assert torch.equal(o1.view(torch.int16), o2.view(torch.int16)) and torch.equal(l1, l2)


# ------------------------------------------------------------------ host-buffer entry point

def test_host_entry_matches_device_entry():
    cfg = inputs.CONFIGS["C1"]
    q, k, v = inputs.make_config_inputs(cfg)
    o_dev, lse_dev = run_gpu(api.attn_fwd, q, k, v, cfg.scale, cfg.causal)
    qp, kp, vp = q.pin_memory(), k.pin_memory(), v.pin_memory()
    o = torch.empty_like(q).pin_memory()
    lse = torch.empty(cfg.B, cfg.H, cfg.Sq, dtype=torch.float32).pin_memory()
    ws = torch.empty(api.attn_fwd_host_workspace_bytes(cfg.B, cfg.H, cfg.Sq, cfg.Sk, cfg.D),
                     dtype=torch.uint8, device="cuda:0")
    api.attn_fwd_host(qp, kp, vp, cfg.scale, cfg.causal, o, lse, ws)
    assert api.attn_last_device_status() == 0
    assert torch.equal(o.view(torch.int16), o_dev.view(torch.int16)) and torch.equal(lse, lse_dev)


@pytest.mark.parametrize("D,dtype,causal,B,H,S", [(128, 1, True, 2, 8, 2048), (64, 0, False, 1, 5, 8192)])
def test_host_entry_pipelined_over_groups_of_heads(D, dtype, causal, B, H, S):
    # large enough (>= 16 MiB of Q, K, V, >= 4 heads) for the copies to run on the library's own streams in
    # groups of heads; two calls in a row on a side stream, the second on other inputs into the same workspace
    dev = torch.device("cuda:0")
    ws = torch.empty(api.attn_fwd_host_workspace_bytes(B, H, S, S, D), dtype=torch.uint8, device=dev)
    stream = torch.cuda.Stream(device=dev)
    outs, refs = [], []
    for rep in range(2):
        q, k, v = inputs.make_qkv(B, H, S, S, D, dtype, seed=4400 + 10 * rep)
        refs.append(run_gpu(api.attn_fwd, q, k, v, D ** -0.5, causal))
        o = torch.full((B, H, S, D), float("nan"), dtype=q.dtype).pin_memory()
        lse = torch.full((B, H, S), float("nan"), dtype=torch.float32).pin_memory()
        outs.append((q.pin_memory(), k.pin_memory(), v.pin_memory(), o, lse))
    with torch.cuda.stream(stream):
        for qp, kp, vp, o, lse in outs:
            api.attn_fwd_host(qp, kp, vp, D ** -0.5, causal, o, lse, ws, stream=stream)
    stream.synchronize()
    assert api.attn_last_device_status() == 0
    for (qp, kp, vp, o, lse), (o_dev, lse_dev) in zip(outs, refs):
        assert torch.equal(o.view(torch.int16), o_dev.view(torch.int16)) and torch.equal(lse, lse_dev)


# ------------------------------------------------------------------ full-size configurations, every row

@pytest.mark.parametrize("name", ["C2", "C3", "C4", "C5"])
def test_full_size_configs_against_oracle_on_every_row(name):
    # the whole output tensor of each benchmark configuration against the fp64 oracle, one (batch, head)
    # at a time so that the fp64 reference of a head (at most 16 MiB) is all that is held at once
    cfg = inputs.CONFIGS[name]
    q, k, v = inputs.make_config_inputs(cfg)
    o, lse = run_gpu(api.attn_fwd, q, k, v, cfg.scale, cfg.causal)
    qb, kb, vb = inputs.bits(q), inputs.bits(k), inputs.bits(v)
    o2, l2 = o.view(-1, cfg.D), lse.view(-1)
    worst_o, worst_l, where, sq_err, sq_ref = 0.0, 0.0, None, 0.0, 0.0
    for bh in range(cfg.B * cfg.H):
        rows = np.arange(bh * cfg.Sq, (bh + 1) * cfg.Sq, dtype=np.int64)
        o_ref, lse_ref = orc.attention_rows_16(qb, kb, vb, cfg.dtype, rows, cfg.scale, cfg.causal)
        err = np.abs(o2[rows[0]:rows[-1] + 1].double().numpy() - o_ref)
        if err.max() > worst_o:
            worst_o = float(err.max())
            where = (bh, int(err.max(axis=1).argmax()))
        worst_l = max(worst_l, float(np.abs(l2[rows[0]:rows[-1] + 1].double().numpy() - lse_ref).max()))
        sq_err += float((err ** 2).sum())
        sq_ref += float((o_ref ** 2).sum())
    print("%s: all %d rows  max|dO| = %.3g at (head, row) %s  max|dLSE| = %.3g  rms dO / rms O = %.3g" % (
        name, cfg.B * cfg.H * cfg.Sq, worst_o, where, worst_l, math.sqrt(sq_err / sq_ref)))
    assert worst_o <= O_TOL[cfg.dtype], "max |dO| = %g at (head, row) %s" % (worst_o, where)
    assert worst_l <= LSE_TOL, "max |dLSE| = %g" % worst_l
    # the absolute bar is loose for long diffuse rows (|O| ~ 0.03): the error must also be small against O itself
    assert math.sqrt(sq_err / sq_ref) <= (2.0 ** -9 if cfg.dtype == inputs.DTYPE_FP16 else 2.0 ** -6)
    # properties that hold at any size: finite outputs, |O| bounded by max |V| per head
    assert bool(torch.isfinite(o.float()).all()) and bool(torch.isfinite(lse).all())
    vmax = v.float().abs().amax(dim=(2, 3), keepdim=True)
    assert bool((o.float().abs() <= vmax * (1 + 1e-2)).all())
    if cfg.causal:   # causal row 0 returns V[0]
        assert torch.equal(o[:, :, 0].view(torch.int16), v[:, :, 0].view(torch.int16))


@pytest.mark.parametrize("name", ["C2", "C3"])
def test_tensor_core_kernel_agrees_with_cross_check_kernel_everywhere(name):
    # all rows of a full-size configuration: the two independent CUDA kernels agree within the
    # sum of their tolerances (the oracle itself covers sampled rows above)
    cfg = inputs.CONFIGS[name]
    q, k, v = inputs.make_config_inputs(cfg)
    o1, l1 = run_gpu(api.attn_fwd, q, k, v, cfg.scale, cfg.causal)
    o2, l2 = run_gpu(api.attn_fwd_simt, q, k, v, cfg.scale, cfg.causal)
    assert float((o1.float() - o2.float()).abs().max()) <= 2 * O_TOL[cfg.dtype]
    assert float((l1 - l2).abs().max()) <= 2 * LSE_TOL


# ------------------------------------------------------------------ grouped-query / multi-query attention

@pytest.mark.parametrize("D,dtype,causal,H,Hkv", [(128, 1, True, 8, 2), (64, 0, False, 6, 1), (256, 0, True, 4, 2),
                                                  (128, 0, False, 4, 4)])
def test_gqa_against_oracle(D, dtype, causal, H, Hkv):
    B, Sq, Sk = 2, 300, 421
    q = inputs.randn16((B, H, Sq, D), 500, dtype)
    k = inputs.randn16((B, Hkv, Sk, D), 501, dtype)
    v = inputs.randn16((B, Hkv, Sk, D), 502, dtype)
    dev = torch.device("cuda:0")
    obuf, o = guarded((B, H, Sq, D), q.dtype, dev)
    lbuf, lse = guarded((B, H, Sq), torch.float32, dev)
    scale = f32_scale(D)
    api.attn_fwd_gqa(q.to(dev), k.to(dev), v.to(dev), scale, causal, out=o, lse=lse)
    assert api.attn_last_device_status() == 0 and guards_intact(obuf) and guards_intact(lbuf)
    o_ref, lse_ref = orc.attention_gqa(*(orc.widen(inputs.bits(t), dtype) for t in (q, k, v)), scale, causal)
    assert np.abs(o.cpu().double().numpy() - o_ref).max() <= O_TOL[dtype]
    assert np.abs(lse.cpu().double().numpy() - lse_ref).max() <= LSE_TOL


def test_gqa_rejects_indivisible_heads():
    q = torch.zeros(1, 5, 128, 64, dtype=torch.float16, device="cuda:0")
    kv = torch.zeros(1, 2, 128, 64, dtype=torch.float16, device="cuda:0")
    with pytest.raises(api.AttnError) as err:
        api.attn_fwd_gqa(q, kv, kv, 0.1, False)
    assert err.value.status == 2


# ------------------------------------------------------------------ separate Q/K and V head dims (192 / 128)

@pytest.mark.parametrize("dtype,causal,H,Hkv,Sq,Sk", [(1, True, 4, 4, 300, 300), (0, False, 4, 2, 257, 515),
                                                      (1, True, 2, 1, 640, 640)])
def test_qk192_v128_against_oracle(dtype, causal, H, Hkv, Sq, Sk):
    B = 2
    q = inputs.randn16((B, H, Sq, 192), 600, dtype)
    k = inputs.randn16((B, Hkv, Sk, 192), 601, dtype)
    v = inputs.randn16((B, Hkv, Sk, 128), 602, dtype)
    dev = torch.device("cuda:0")
    obuf, o = guarded((B, H, Sq, 128), q.dtype, dev)
    lbuf, lse = guarded((B, H, Sq), torch.float32, dev)
    scale = f32_scale(192)
    api.attn_fwd_qkv_dims(q.to(dev), k.to(dev), v.to(dev), scale, causal, out=o, lse=lse)
    assert api.attn_last_device_status() == 0 and guards_intact(obuf) and guards_intact(lbuf)
    o_ref, lse_ref = orc.attention_gqa_dv(*(orc.widen(inputs.bits(t), dtype) for t in (q, k, v)), scale, causal)
    assert np.abs(o.cpu().double().numpy() - o_ref).max() <= O_TOL[dtype]
    assert np.abs(lse.cpu().double().numpy() - lse_ref).max() <= LSE_TOL


def test_qkv_dims_rejects_unsupported_pairs():
    q = torch.zeros(1, 1, 128, 96, dtype=torch.float16, device="cuda:0")
    v = torch.zeros(1, 1, 128, 64, dtype=torch.float16, device="cuda:0")
    with pytest.raises(api.AttnError) as err:
        api.attn_fwd_qkv_dims(q, q, v, 0.1, False)
    assert err.value.status == 3


# ------------------------------------------------------------------ K/V shards (partial results) and their merge

@pytest.mark.parametrize("D,dtype,causal,Hkv", [(128, 1, True, 2), (64, 0, False, 4), (256, 1, True, 4), (128, 0, True, 1)])
def test_kv_shards_and_combine_against_oracle(D, dtype, causal, Hkv):
    B, H, Sq, Sk = 1, 4, 600, 700
    q = inputs.randn16((B, H, Sq, D), 700, dtype)
    k = inputs.randn16((B, Hkv, Sk, D), 701, dtype)
    v = inputs.randn16((B, Hkv, Sk, D), 702, dtype)
    dev = torch.device("cuda:0")
    qd = q.to(dev)
    scale = f32_scale(D)
    cuts = [0, 130, 384, Sk]        # uneven shards, one boundary off the tile grid
    n = len(cuts) - 1
    o_parts = torch.full((n, B, H, Sq, D), float("nan"), dtype=q.dtype, device=dev)
    l_parts = torch.full((n, B, H, Sq), float("nan"), dtype=torch.float32, device=dev)
    qf, kf, vf = (orc.widen(inputs.bits(t), dtype) for t in (q, k, v))
    for r, (a, b) in enumerate(zip(cuts, cuts[1:])):
        api.attn_fwd_partial(qd, k[:, :, a:b].contiguous().to(dev), v[:, :, a:b].contiguous().to(dev), scale, causal, a,
                             out=o_parts[r], lse=l_parts[r])
        # each shard on its own against the oracle's shard entry
        o_ref_r, l_ref_r = orc.attention_shard(qf, kf[:, :, a:b], vf[:, :, a:b], scale, causal, a)
        got_l = l_parts[r].cpu().double().numpy()
        assert np.array_equal(np.isneginf(got_l), np.isneginf(l_ref_r))
        fin = ~np.isneginf(l_ref_r)
        assert np.abs(got_l[fin] - l_ref_r[fin]).max() <= LSE_TOL
        assert np.abs(o_parts[r].cpu().double().numpy() - o_ref_r).max() <= O_TOL[dtype]
    assert api.attn_last_device_status() == 0
    o, lse = api.attn_combine(o_parts, l_parts)
    torch.cuda.synchronize()
    o_ref, lse_ref = orc.attention_gqa(qf, kf, vf, scale, causal)
    assert np.abs(o.cpu().double().numpy() - o_ref).max() <= O_TOL[dtype]
    assert np.abs(lse.cpu().double().numpy() - lse_ref).max() <= LSE_TOL


def test_combine_of_all_empty_rows():
    dev = torch.device("cuda:0")
    o_parts = torch.randn(3, 1, 2, 40, 64, device=dev).to(torch.float16)
    l_parts = torch.full((3, 1, 2, 40), float("-inf"), dtype=torch.float32, device=dev)
    o, lse = api.attn_combine(o_parts, l_parts)
    assert float(o.abs().max()) == 0.0 and bool(torch.isneginf(lse).all())


def test_kv_sharded_attention_single_rank_reduces_to_plain_attention():
    from paper_2506_12355_b200 import dist as adist
    q, k, v = inputs.make_qkv(1, 2, 300, 300, 128, inputs.DTYPE_BF16, seed=77)
    dev = torch.device("cuda:0")
    o1, l1 = adist.kv_sharded_attention(q.to(dev), k.to(dev), v.to(dev), 0.1, True, 0)
    o2, l2 = api.attn_fwd(q.to(dev), k.to(dev), v.to(dev), 0.1, True)
    torch.cuda.synchronize()
    assert torch.equal(o1.view(torch.int16), o2.view(torch.int16)) and float((l1 - l2).abs().max()) <= 1e-5


# ------------------------------------------------------------------ scheduling: many items, streams, graphs

def test_many_short_items_match_cross_check_kernel():
    # 2048 one-pair work items on 148 persistent CTAs: every item must be drawn exactly once
    B, H, S, D = 64, 32, 128, 64
    q, k, v = inputs.make_qkv(B, H, S, S, D, inputs.DTYPE_FP16, seed=88)
    o1, l1 = run_gpu(api.attn_fwd, q, k, v, 0.125, True)
    o2, l2 = run_gpu(api.attn_fwd_simt, q, k, v, 0.125, True)
    assert float((o1.float() - o2.float()).abs().max()) <= 2 * O_TOL[inputs.DTYPE_FP16]
    assert float((l1 - l2).abs().max()) <= 2 * LSE_TOL


@pytest.mark.parametrize("B,H,S,D,dtype", [(3, 25, 1000, 128, 0), (8, 20, 1024, 64, 1), (1, 50, 1000, 128, 1), (5, 31, 300, 64, 0)])
def test_last_wave_cut_into_half_items(B, H, S, D, dtype):
    # Without a mask, when the last wave of equally long work items would occupy at most half of the SMs, its
    # items are cut into their two Q tiles (each half a work item of its own that must leave the other tile's
    # rows alone).  Shapes whose item count modulo the SM count is small, with ragged last tiles; every row of
    # every head against the oracle, outputs pre-filled with NaN.
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    items = B * H * ((S + 255) // 256)
    assert items > sms and 0 < items % sms <= sms // 2, "the shape no longer exercises the half items on this GPU"
    scale = f32_scale(D)
    q, k, v = inputs.make_qkv(B, H, S, S, D, dtype, seed=4242)
    o, lse = run_gpu(api.attn_fwd, q, k, v, scale, False)
    assert not torch.isnan(o.float()).any() and not torch.isnan(lse).any(), "rows left unwritten"
    qb, kb, vb = (inputs.bits(t) for t in (q, k, v))
    worst_o = worst_l = 0.0
    for bh in range(B * H):
        rows = np.arange(bh * S, (bh + 1) * S, dtype=np.int64)
        o_ref, l_ref = orc.attention_rows_16(qb, kb, vb, dtype, rows, scale, False)
        worst_o = max(worst_o, float(np.abs(o.view(-1, D)[rows].double().numpy() - o_ref).max()))
        worst_l = max(worst_l, float(np.abs(lse.view(-1)[rows].double().numpy() - l_ref).max()))
    assert worst_o <= O_TOL[dtype], "max |dO| = %g" % worst_o
    assert worst_l <= LSE_TOL, "max |dLSE| = %g" % worst_l


def test_launches_on_two_streams_do_not_share_a_work_counter():
    dev = torch.device("cuda:0")
    cases = []
    for i, (D, causal) in enumerate(((128, True), (64, False))):
        q, k, v = inputs.make_qkv(2, 8, 1024, 1024, D, inputs.DTYPE_BF16, seed=120 + i)
        qd, kd, vd = q.to(dev), k.to(dev), v.to(dev)
        ref_o, ref_l = api.attn_fwd(qd, kd, vd, 0.1, causal)
        cases.append((qd, kd, vd, causal, ref_o, ref_l))
    torch.cuda.synchronize()
    streams = [torch.cuda.Stream(device=dev) for _ in cases]
    outs = []
    for _ in range(5):
        for (qd, kd, vd, causal, _, _), st in zip(cases, streams):
            outs.append((api.attn_fwd(qd, kd, vd, 0.1, causal, stream=st), len(outs) % len(cases)))
    torch.cuda.synchronize()
    assert api.attn_last_device_status() == 0
    for (o, l), idx in outs:
        assert torch.equal(o.view(torch.int16), cases[idx][4].view(torch.int16)) and torch.equal(l, cases[idx][5])


def test_cuda_graph_capture_and_replay():
    dev = torch.device("cuda:0")
    cfg = inputs.CONFIGS["C1"]
    q, k, v = (t.to(dev) for t in inputs.make_config_inputs(cfg))
    o = torch.empty_like(q)
    lse = torch.empty(cfg.B, cfg.H, cfg.Sq, dtype=torch.float32, device=dev)
    ref_o, ref_l = api.attn_fwd(q, k, v, cfg.scale, cfg.causal)      # first call: one-time set-up outside capture
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    st = torch.cuda.Stream(device=dev)
    with torch.cuda.stream(st):
        with torch.cuda.graph(g, stream=st):
            api.attn_fwd(q, k, v, cfg.scale, cfg.causal, out=o, lse=lse, stream=st)
    for _ in range(3):
        o.zero_()
        g.replay()
    torch.cuda.synchronize()
    assert torch.equal(o.view(torch.int16), ref_o.view(torch.int16)) and torch.equal(lse, ref_l)


def test_many_launches_on_one_stream_while_a_long_launch_runs_on_another():
    # work counters belong to streams: 1100 counted launches on one stream (more than any ring of counters
    # would hold) next to one long launch on another stream; every result must be bit-equal to a quiet run
    dev = torch.device("cuda:0")
    ql, kl, vl = (t.to(dev) for t in inputs.make_qkv(1, 4, 16384, 16384, 128, inputs.DTYPE_BF16, seed=140))
    qs, ks, vs = (t.to(dev) for t in inputs.make_qkv(2, 40, 512, 512, 64, inputs.DTYPE_FP16, seed=141))   # 160 items
    ref_long = api.attn_fwd(ql, kl, vl, 0.09, True)
    ref_short = api.attn_fwd(qs, ks, vs, 0.125, False)
    torch.cuda.synchronize()
    s_long, s_short = torch.cuda.Stream(device=dev), torch.cuda.Stream(device=dev)
    o_long = torch.empty_like(ql)
    l_long = torch.empty(1, 4, 16384, dtype=torch.float32, device=dev)
    o_short = torch.empty_like(qs)
    l_short = torch.empty(2, 40, 512, dtype=torch.float32, device=dev)
    mismatches = torch.zeros(1, dtype=torch.int64, device=dev)
    for rep in range(4):
        for _ in range(3):
            api.attn_fwd(ql, kl, vl, 0.09, True, out=o_long, lse=l_long, stream=s_long)
        with torch.cuda.stream(s_short):
            for i in range(275):
                api.attn_fwd(qs, ks, vs, 0.125, False, out=o_short, lse=l_short, stream=s_short)
                if i % 25 == 0:
                    mismatches += (o_short.view(torch.int16) != ref_short[0].view(torch.int16)).sum() + (l_short != ref_short[1]).sum()
        s_long.synchronize()
        assert torch.equal(o_long.view(torch.int16), ref_long[0].view(torch.int16)) and torch.equal(l_long, ref_long[1])
    torch.cuda.synchronize()
    assert api.attn_last_device_status() == 0
    assert int(mismatches.item()) == 0
    assert torch.equal(o_short.view(torch.int16), ref_short[0].view(torch.int16)) and torch.equal(l_short, ref_short[1])


def test_graph_of_a_counted_launch_replays_next_to_eager_launches():
    # a captured launch with more work items than SMs keeps a work counter of its own: replayed on one stream
    # while eager launches of another problem run on a second stream, all results stay bit-equal
    dev = torch.device("cuda:0")
    cfg = inputs.CONFIGS["C3"]
    q, k, v = (t.to(dev) for t in inputs.make_config_inputs(cfg))
    q2, k2, v2 = (t.to(dev) for t in inputs.make_qkv(2, 40, 512, 512, 64, inputs.DTYPE_FP16, seed=151))
    ref = api.attn_fwd(q, k, v, cfg.scale, cfg.causal)
    ref2 = api.attn_fwd(q2, k2, v2, 0.125, False)
    torch.cuda.synchronize()
    o = torch.empty_like(q)
    lse = torch.empty(cfg.B, cfg.H, cfg.Sq, dtype=torch.float32, device=dev)
    st, st2 = torch.cuda.Stream(device=dev), torch.cuda.Stream(device=dev)
    g = torch.cuda.CUDAGraph()
    with torch.cuda.stream(st):
        with torch.cuda.graph(g, stream=st):
            api.attn_fwd(q, k, v, cfg.scale, cfg.causal, out=o, lse=lse, stream=st)
    o2 = torch.empty_like(q2)
    l2 = torch.empty(2, 40, 512, dtype=torch.float32, device=dev)
    bad = torch.zeros(1, dtype=torch.int64, device=dev)      # one tally per stream
    bad2 = torch.zeros(1, dtype=torch.int64, device=dev)
    for rep in range(20):
        with torch.cuda.stream(st):
            o.zero_()
            g.replay()
            bad += (o.view(torch.int16) != ref[0].view(torch.int16)).sum() + (lse != ref[1]).sum()
        with torch.cuda.stream(st2):
            for _ in range(60):
                api.attn_fwd(q2, k2, v2, 0.125, False, out=o2, lse=l2, stream=st2)
            bad2 += (o2.view(torch.int16) != ref2[0].view(torch.int16)).sum() + (l2 != ref2[1]).sum()
    torch.cuda.synchronize()
    assert api.attn_last_device_status() == 0
    assert int(bad.item()) == 0 and int(bad2.item()) == 0


# ------------------------------------------------------------------ merge of parts behind separate pointers

@pytest.mark.parametrize("n_parts,dtype,D", [(1, 1, 128), (2, 0, 64), (5, 1, 128), (8, 0, 256)])
def test_combine_gather_equals_combine_and_writes_only_its_rows(n_parts, dtype, D):
    # the parts live in separate allocations (as they would on separate GPUs); the merge of a row range must
    # equal attn_combine on the stacked parts for those rows and leave every other row untouched
    dev = torch.device("cuda:0")
    B, H, Sq = 2, 3, 77
    td = inputs.torch_dtype(dtype)
    g = torch.Generator(device="cpu").manual_seed(5500 + n_parts)
    o_parts = [torch.randn((B, H, Sq, D), generator=g).to(td).to(dev) for _ in range(n_parts)]
    l_parts = [torch.randn((B, H, Sq), generator=g).to(dev) for _ in range(n_parts)]
    if n_parts > 1:
        l_parts[1][0, 0, :5] = float("-inf")          # a shard that saw no key for some rows
    ref_o, ref_l = api.attn_combine(torch.stack(o_parts), torch.stack(l_parts))
    rows = B * H * Sq
    for row_begin, row_count in ((0, rows), (100, 211), (rows - 1, 1), (50, 0)):
        out = torch.full((B, H, Sq, D), float("nan"), dtype=td, device=dev)
        lse = torch.full((B, H, Sq), float("nan"), dtype=torch.float32, device=dev)
        api.attn_combine_gather([t.data_ptr() for t in o_parts], [t.data_ptr() for t in l_parts], (B, H, Sq, D), td,
                                out, lse, row_begin, row_count)
        torch.cuda.synchronize()
        sel = torch.zeros(rows, dtype=torch.bool, device=dev)
        sel[row_begin:row_begin + row_count] = True
        o2, l2 = out.view(rows, D), lse.view(rows)
        assert torch.equal(o2[sel].view(torch.int16), ref_o.view(rows, D)[sel].view(torch.int16))
        assert torch.equal(l2[sel], ref_l.view(rows)[sel])
        assert torch.isnan(o2[~sel].float()).all() and torch.isnan(l2[~sel]).all()


def test_combine_gather_rejects_bad_arguments():
    dev = torch.device("cuda:0")
    o = torch.zeros((1, 1, 8, 64), dtype=torch.float16, device=dev)
    l = torch.zeros((1, 1, 8), dtype=torch.float32, device=dev)
    out, lse = torch.empty_like(o), torch.empty_like(l)
    for ptrs_o, ptrs_l, rb, rc, want in (([], [], 0, 8, 2), ([o.data_ptr()] * 33, [l.data_ptr()] * 33, 0, 8, 2),
                                         ([o.data_ptr()], [l.data_ptr()], 4, 8, 2), ([o.data_ptr()], [l.data_ptr()], -1, 2, 2),
                                         ([0], [l.data_ptr()], 0, 8, 1), ([o.data_ptr() + 8], [l.data_ptr()], 0, 8, 5)):
        with pytest.raises(api.AttnError) as e:
            api.attn_combine_gather(ptrs_o, ptrs_l, (1, 1, 8, 64), torch.float16, out, lse, rb, rc)
        assert e.value.status == want


# ------------------------------------------------------------------ very long sequences

@pytest.mark.parametrize("D,dtype,causal,S", [(128, 1, True, 131072), (256, 0, False, 65613)])
def test_very_long_sequence_on_sampled_rows(D, dtype, causal, S):
    # a thousand K/V tiles per row and row indices beyond 2^16: rows of every region against the oracle
    dev = torch.device("cuda:0")
    q, k, v = inputs.make_qkv(1, 1, S, S, D, dtype, seed=6600 + D)
    o, lse = api.attn_fwd(q.to(dev), k.to(dev), v.to(dev), D ** -0.5, causal)
    assert api.attn_last_device_status() == 0
    rows = np.array(sorted({0, 1, 127, 128, 65535, 65536, S // 2, S - 129, S - 128, S - 2, S - 1}), dtype=np.int64)
    o_ref, l_ref = orc.attention_rows_16(inputs.bits(q), inputs.bits(k), inputs.bits(v), dtype, rows, D ** -0.5, causal)
    og = o.cpu().view(-1, D)[rows].to(torch.float64).numpy()
    lg = lse.cpu().view(-1)[rows].to(torch.float64).numpy()
    assert not torch.isnan(o.float()).any()
    assert np.abs(og - o_ref).max() <= O_TOL[dtype]
    assert np.abs(lg - l_ref).max() <= LSE_TOL
