"""GPU parity of the backward pass (attn_bwd through the C ABI) against the fp64 oracle's gradients.

The kernel is given the forward outputs O and LSE of attn_fwd_gqa on the same 16-bit inputs; the oracle
differentiates the definition in fp64 from those inputs alone.  Bars: see O_... below (derived in the test of
the tolerances at the end of this docstring): every gradient tensor is compared on every element with
    |err| <= ATOL[dtype] * max(1, rms(ref)) * max(1, scale * sqrt(D)) + RTOL[dtype] * |ref| ,
RTOL = 2^-7 (bf16) / 2^-10 (fp16): half a unit in the last place of the stored 16-bit result (2^-9 / 2^-12)
plus the rounding of P and dS to the 16-bit type before their second products (2^-9 / 2^-12 each, of sums whose
terms partly cancel); ATOL covers the elements that are small only because their terms cancel, and the one
error the kernel inherits from the forward pass: rowsum(dO o O) is taken from the ROUNDED 16-bit O, so it is off
by about 2^-9 / 2^-12 * sqrt(D) * rms(dO) rms(O); dS = P (dP - rowsum) carries that error wherever P is not
small, and dQ, dK multiply it by scale * |k|, scale * |q|.  With the usual scale = 1 / sqrt(D) that is the ATOL
term as it stands; a larger scale (sharply peaked rows, P near 1) raises it in proportion, hence the last factor.
"""
import math

import numpy as np
import pytest
import torch

from oracle import attn_oracle as orc
from paper_2506_12355_b200 import api, inputs

pytestmark = pytest.mark.gpu

RTOL = {inputs.DTYPE_FP16: 2.0 ** -10, inputs.DTYPE_BF16: 2.0 ** -7}
ATOL = {inputs.DTYPE_FP16: 2.0 ** -9, inputs.DTYPE_BF16: 2.0 ** -6}


def f32_scale(D):
    return float(np.float32(1.0) / np.sqrt(np.float32(D)))


def run_case(B, H, Hkv, Sq, Sk, D, dtype, causal, seed, scale=None, sigma=1.0):
    dev = torch.device("cuda:0")
    scale = f32_scale(D) if scale is None else scale
    q = inputs.randn16((B, H, Sq, D), seed, dtype, sigma)
    k = inputs.randn16((B, Hkv, Sk, D), seed + 1, dtype, sigma)
    v = inputs.randn16((B, Hkv, Sk, D), seed + 2, dtype, sigma)
    dout = inputs.randn16((B, H, Sq, D), seed + 3, dtype, sigma)
    qd, kd, vd, dd = q.to(dev), k.to(dev), v.to(dev), dout.to(dev)
    o, lse = api.attn_fwd_gqa(qd, kd, vd, scale, causal)
    nan = float("nan")
    dq = torch.full_like(qd, nan)
    dk = torch.full_like(kd, nan)
    dv = torch.full_like(vd, nan)
    api.attn_bwd(qd, kd, vd, o, lse, dd, scale, causal, dq=dq, dk=dk, dv=dv)
    assert api.attn_last_device_status() == 0, "a kernel reported a timed-out wait"
    ref = orc.attention_bwd(*(orc.widen(inputs.bits(t), dtype) for t in (q, k, v, dout)), scale, causal)
    worst = {}
    for name, got, want in zip(("dq", "dk", "dv"), (dq, dk, dv), ref):
        g = got.cpu().to(torch.float64).numpy()
        assert not np.isnan(g).any(), "NaN in %s (unwritten or arithmetic)" % name
        err = np.abs(g - want)
        rms = math.sqrt(float((want ** 2).mean())) if want.size else 0.0
        bound = ATOL[dtype] * max(1.0, rms) * max(1.0, scale * math.sqrt(D)) + RTOL[dtype] * np.abs(want)
        worst[name] = (float(err.max()) if err.size else 0.0, rms)
        assert np.all(err <= bound), "%s: max |err| = %g (rms of the reference %g) at %s" % (
            name, err.max(), rms, np.unravel_index((err - bound).argmax(), err.shape))
    return worst


@pytest.mark.parametrize("causal", [False, True])
@pytest.mark.parametrize("dtype", [inputs.DTYPE_FP16, inputs.DTYPE_BF16])
@pytest.mark.parametrize("D", [64, 128])
@pytest.mark.parametrize("shape", [(1, 2, 2, 128, 128), (1, 1, 1, 1, 1), (2, 2, 2, 127, 129), (1, 3, 3, 300, 421),
                                   (1, 2, 2, 513, 257), (1, 4, 2, 384, 640), (2, 4, 1, 200, 200)])
def test_bwd_small_shapes(shape, D, dtype, causal):
    B, H, Hkv, Sq, Sk = shape
    run_case(B, H, Hkv, Sq, Sk, D, dtype, causal, seed=8000 + Sq + 3 * Sk + D)


def test_bwd_hand_case_2x2_padded_into_d64():
    # the pencil-derived gradients of the 2x2 case, zero-padded into the smallest head dim
    dev = torch.device("cuda:0")
    e = math.e
    g, a, b = 2 * e / (e + 1) ** 2, e / (e + 1), 1 / (e + 1)
    for causal, want_dq, want_dk, want_dv in (
            (False, [[-g, g], [-g, g]], [[-g, -g], [g, g]], [[a, b], [b, a]]),
            (True, [[0, 0], [-g, g]], [[0, -g], [0, g]], [[1, b], [0, a]])):
        q = torch.zeros(1, 1, 2, 64, dtype=torch.float16)
        v = torch.zeros(1, 1, 2, 64, dtype=torch.float16)
        dout = torch.zeros(1, 1, 2, 64, dtype=torch.float16)
        q[0, 0, :, :2] = torch.eye(2)
        v[0, 0, :, :2] = torch.tensor([[1.0, 2.0], [3.0, 4.0]])
        dout[0, 0, :, :2] = torch.eye(2)
        qd, vd, dd = q.to(dev), v.to(dev), dout.to(dev)
        o, lse = api.attn_fwd(qd, qd, vd, 1.0, causal)
        dq, dk, dv = api.attn_bwd(qd, qd, vd, o, lse, dd, 1.0, causal)
        assert api.attn_last_device_status() == 0
        for got, want in ((dq, want_dq), (dk, want_dk), (dv, want_dv)):
            np.testing.assert_allclose(got[0, 0, :, :2].cpu().double().numpy(), np.array(want), atol=2e-3)
            assert float(got[0, 0, :, 2:].abs().max()) == 0.0


@pytest.mark.parametrize("D,dtype,causal", [(128, 1, True), (64, 0, False), (128, 0, False), (64, 1, True)])
def test_bwd_many_tiles(D, dtype, causal):
    # 16 x 16 tiles per head and enough heads for several waves of CTAs
    w = run_case(2, 8, 8, 2048, 2048, D, dtype, causal, seed=8100 + D)
    print("bwd D=%d dtype=%d causal=%s: max|err| (rms ref) dq %.3g (%.3g)  dk %.3g (%.3g)  dv %.3g (%.3g)" % (
        D, dtype, causal, *w["dq"], *w["dk"], *w["dv"]))


@pytest.mark.parametrize("name,heads", [("C3", None), ("C5", (0, 31))])
def test_bwd_at_the_benchmark_shapes(name, heads):
    # the two shapes whose backward pass bench.py times, in the same launch configuration: C3 against the oracle's
    # gradients on every head, C5 (3.3 TFLOP of oracle work for all heads) on its first and its last head
    cfg = inputs.CONFIGS[name]
    dev = torch.device("cuda:0")
    q, k, v = inputs.make_config_inputs(cfg)
    dout = inputs.randn16((cfg.B, cfg.H, cfg.Sq, cfg.D), inputs.BASE_SEED + 1000 * cfg.index + 3, cfg.dtype)
    qd, kd, vd, dd = q.to(dev), k.to(dev), v.to(dev), dout.to(dev)
    o, lse = api.attn_fwd(qd, kd, vd, cfg.scale, cfg.causal)
    got = [t.cpu() for t in api.attn_bwd(qd, kd, vd, o, lse, dd, cfg.scale, cfg.causal)]
    assert api.attn_last_device_status() == 0
    flat = lambda t: t.reshape(cfg.B * cfg.H, cfg.Sq, cfg.D)
    sel = list(range(cfg.B * cfg.H)) if heads is None else list(heads)
    pick = lambda t: flat(t)[sel].unsqueeze(0).contiguous()       # the chosen (batch, head) slices as one batch
    ref = orc.attention_bwd(*(orc.widen(inputs.bits(pick(t)), cfg.dtype) for t in (q, k, v, dout)), cfg.scale, cfg.causal)
    for nm, g, want in zip(("dq", "dk", "dv"), got, ref):
        gsel = pick(g).to(torch.float64).numpy()
        assert not np.isnan(gsel).any() and bool(torch.isfinite(g.float()).all())
        err = np.abs(gsel - want)
        rms = math.sqrt(float((want ** 2).mean()))
        bound = ATOL[cfg.dtype] * max(1.0, rms) + RTOL[cfg.dtype] * np.abs(want)
        print("%s %s: max|err| %.3g, rms err / rms %.3g (rms %.3g)" % (name, nm, err.max(), math.sqrt(float((err ** 2).mean())) / rms, rms))
        assert np.all(err <= bound), "%s %s: max |err| = %g" % (name, nm, err.max())
        assert math.sqrt(float((err ** 2).mean())) <= 2.0 ** -6 * rms      # bf16: small against the gradient itself


def test_bwd_long_ragged_sequence_and_no_queries():
    # 65 x 65 tiles per head with ragged tails on both axes (Sq != Sk), grouped heads; then the Sq = 0 corner
    run_case(1, 16, 8, 4133, 4101, 128, inputs.DTYPE_BF16, True, seed=8150)
    dev = torch.device("cuda:0")
    k = torch.randn(1, 2, 300, 64, device=dev).to(torch.float16)
    q0 = torch.empty(1, 2, 0, 64, dtype=torch.float16, device=dev)
    dq, dk, dv = api.attn_bwd(q0, k, k, q0, torch.empty(1, 2, 0, device=dev), q0, 0.1, False,
                              dk=torch.full_like(k, float("nan")), dv=torch.full_like(k, float("nan")))
    torch.cuda.synchronize()
    assert dq.numel() == 0 and float(dk.abs().max()) == 0.0 and float(dv.abs().max()) == 0.0


def test_bwd_keys_that_no_query_sees_and_sharp_scale():
    # Sk > Sq under the causal mask: keys beyond the last query get zero gradients (tiles with and without steps);
    # a large scale makes the softmax rows sharply peaked
    run_case(1, 2, 2, 200, 700, 64, inputs.DTYPE_BF16, True, seed=8200)
    run_case(1, 2, 1, 256, 256, 128, inputs.DTYPE_FP16, False, seed=8201, scale=1.0)


def test_bwd_in_a_cuda_graph_and_on_two_streams():
    # the three launches of a call captured once and replayed; two calls in flight on two streams
    dev = torch.device("cuda:0")
    cases = []
    for i, (D, causal) in enumerate(((128, True), (64, False))):
        q, k, v = (t.to(dev) for t in inputs.make_qkv(2, 4, 700, 700, D, inputs.DTYPE_BF16, seed=8400 + i))
        dout = inputs.randn16((2, 4, 700, D), 8410 + i, inputs.DTYPE_BF16).to(dev)
        o, lse = api.attn_fwd(q, k, v, D ** -0.5, causal)
        ref = api.attn_bwd(q, k, v, o, lse, dout, D ** -0.5, causal)
        cases.append((q, k, v, o, lse, dout, D ** -0.5, causal, ref))
    torch.cuda.synchronize()
    q, k, v, o, lse, dout, scale, causal, ref = cases[0]
    dq, dk, dv = torch.empty_like(q), torch.empty_like(k), torch.empty_like(v)
    ws = torch.empty(api.attn_bwd_workspace_bytes(2, 4, 700), dtype=torch.uint8, device=dev)
    st = torch.cuda.Stream(device=dev)
    g = torch.cuda.CUDAGraph()
    with torch.cuda.stream(st):
        with torch.cuda.graph(g, stream=st):
            api.attn_bwd(q, k, v, o, lse, dout, scale, causal, dq=dq, dk=dk, dv=dv, workspace=ws, stream=st)
    for _ in range(3):
        dq.zero_(); dk.zero_(); dv.zero_()
        g.replay()
    torch.cuda.synchronize()
    for got, want in zip((dq, dk, dv), ref):
        assert torch.equal(got.view(torch.int16), want.view(torch.int16))
    streams = [torch.cuda.Stream(device=dev) for _ in cases]
    outs = []
    for _ in range(4):
        for c, s_ in zip(cases, streams):
            with torch.cuda.stream(s_):
                outs.append((api.attn_bwd(*c[:8], stream=s_), c[8]))
    torch.cuda.synchronize()
    assert api.attn_last_device_status() == 0
    for got, want in outs:
        for a, b in zip(got, want):
            assert torch.equal(a.view(torch.int16), b.view(torch.int16))


def test_bwd_is_bitwise_deterministic_and_validates():
    dev = torch.device("cuda:0")
    q, k, v = (t.to(dev) for t in inputs.make_qkv(2, 4, 640, 640, 128, inputs.DTYPE_BF16, seed=8300))
    dout = inputs.randn16((2, 4, 640, 128), 8303, inputs.DTYPE_BF16).to(dev)
    o, lse = api.attn_fwd(q, k, v, 0.09, True)
    g1 = api.attn_bwd(q, k, v, o, lse, dout, 0.09, True)
    g2 = api.attn_bwd(q, k, v, o, lse, dout, 0.09, True)
    torch.cuda.synchronize()
    for a, b in zip(g1, g2):
        assert torch.equal(a.view(torch.int16), b.view(torch.int16))
    with pytest.raises(api.AttnError) as err:        # head dim 256 has no backward kernel
        x = torch.zeros(1, 1, 128, 256, dtype=torch.float16, device=dev)
        api.attn_bwd(x, x, x, x, torch.zeros(1, 1, 128, device=dev), x, 0.1, False)
    assert err.value.status == 3
    with pytest.raises(api.AttnError) as err:        # workspace too small
        api.attn_bwd(q, k, v, o, lse, dout, 0.09, True, workspace=torch.empty(256, dtype=torch.uint8, device=dev))
    assert err.value.status == 10
    # no keys: dq = 0
    k0 = torch.empty(2, 4, 0, 128, dtype=torch.bfloat16, device=dev)
    dq, dk, dv = api.attn_bwd(q, k0, k0, torch.zeros_like(q), torch.full((2, 4, 640), float("-inf"), device=dev), dout, 0.09, False)
    assert float(dq.abs().max()) == 0.0 and dk.numel() == 0
