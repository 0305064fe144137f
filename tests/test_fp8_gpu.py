"""GPU parity of the 8-bit (E4M3) attention entry point against the fp64 CPU oracle (the definition on the
dequantised tensors), element by element on the same seeded inputs.

Tolerances (sigma = standard deviation of the dequantised inputs).  LSE: 1e-3 absolute for both kernels (the
row sum is taken in fp32 from the un-rounded probabilities).  O of the CUDA-core kernel (fp32 throughout, bf16
output): 2e-2 * sigma, the bf16 bar of the 16-bit path scaled with the values' size.  O of the tensor-core kernel: the probabilities are
rounded to E4M3 for the second product, each with a relative error of at most 2^-4 (half a unit in the last of
3 fraction bits), so elementwise |dO| <= 2^-4 * sum_j p_j |v_j| + bf16 rounding of O (2^-8 |O|) + 1e-3 sigma
of fp32 slack; and because those rounding errors are independent with standard deviation 2^-4 / sqrt(3), the
root-mean-square error over a tensor is ~0.036 of O's own root-mean-square size: the test bar is 0.06, which a
wrong operand, index or scale (relative error ~1) cannot pass."""
import numpy as np
import pytest
import torch

from oracle import attn_oracle as orc
from paper_2506_12355_b200 import api, inputs

pytestmark = pytest.mark.gpu

D = 128
LSE_TOL = 1e-3
GUARD = 4096


def guarded(shape, dtype, device):
    n = int(np.prod(shape))
    buf = torch.full((n + 2 * GUARD,), float("nan"), dtype=dtype, device=device)
    return buf, buf[GUARD:GUARD + n].view(shape)


def guards_intact(buf):
    return bool(torch.isnan(buf[:GUARD]).all()) and bool(torch.isnan(buf[-GUARD:]).all())


def run_gpu(q, k, v, scale, f, causal, impl):
    dev = torch.device("cuda:0")
    B, H, Sq, _ = q.shape
    obuf, o = guarded((B, H, Sq, D), torch.bfloat16, dev)
    lbuf, lse = guarded((B, H, Sq), torch.float32, dev)
    api.attn_fwd_fp8(q.to(dev), k.to(dev), v.to(dev), scale, f[0], f[1], f[2], causal, out=o, lse=lse, impl=impl)
    assert api.attn_last_device_status() == 0, "a kernel reported a timed-out wait"
    assert guards_intact(obuf) and guards_intact(lbuf), "write outside the output buffers"
    return o.cpu().to(torch.float64).numpy(), lse.cpu().to(torch.float64).numpy()


def check_o(o, o_ref, a_ref, f, sigma, impl):
    assert not np.isnan(o).any(), "NaN in O (unwritten canary or arithmetic NaN)"
    err = np.abs(o - o_ref)
    if impl == 1:
        assert err.size == 0 or err.max() <= 2e-2 * sigma, "max |dO| = %g" % err.max()
        return
    bound = 2.0 ** -4 * a_ref + 2.0 ** -8 * np.abs(o_ref) + 1e-3 * sigma
    assert np.all(err <= bound), "elementwise bound exceeded by a factor %g" % (err / bound).max()
    rms_o = np.sqrt(np.mean(o_ref ** 2)) if o_ref.size else 0.0
    if rms_o > 0:
        assert np.sqrt(np.mean(err ** 2)) <= 0.06 * rms_o + 2.0 ** -9 * sigma, \
            "rms error %g of rms(O) %g" % (np.sqrt(np.mean(err ** 2)), rms_o)


def check_lse(lse, lse_ref):
    inf = np.isneginf(lse_ref)
    assert np.array_equal(np.isneginf(lse), inf)
    err = np.abs(lse[~inf] - lse_ref[~inf])
    assert err.size == 0 or err.max() <= LSE_TOL, "max |dLSE| = %g" % err.max()


def check_against_oracle(B, H, Hkv, Sq, Sk, causal, impl, f=(1.0, 1.0, 1.0), sigma=1.0, seed=9001, scale=None):
    q, k, v = inputs.make_qkv_fp8(B, H, Hkv, Sq, Sk, D, seed, sigma, f)
    scale = D ** -0.5 if scale is None else scale
    o, lse = run_gpu(q, k, v, scale, f, causal, impl)
    qn, kn, vn = q.numpy(), k.numpy(), v.numpy()
    o_ref, lse_ref = orc.attention_fp8(qn, kn, vn, f[0], f[1], f[2], scale, causal)
    a_ref, _ = orc.attention_fp8(qn, kn, vn & 0x7f, f[0], f[1], f[2], scale, causal)   # sum_j p_j |v_j|
    check_o(o, o_ref, a_ref, f, sigma, impl)
    check_lse(lse, lse_ref)


SMALL = [
    # B, H, Hkv, Sq, Sk
    (1, 2, 2, 128, 128),
    (1, 1, 1, 1, 1),
    (1, 3, 1, 17, 17),
    (2, 1, 1, 127, 127),
    (1, 1, 1, 129, 129),
    (1, 2, 1, 255, 255),
    (1, 1, 1, 100, 333),
    (1, 1, 1, 257, 129),
    (1, 4, 2, 384, 640),
]


@pytest.mark.parametrize("impl", [0, 1])
@pytest.mark.parametrize("causal", [False, True])
@pytest.mark.parametrize("shape", SMALL)
def test_small_shapes(shape, causal, impl):
    B, H, Hkv, Sq, Sk = shape
    check_against_oracle(B, H, Hkv, Sq, Sk, causal, impl, seed=9100 + Sq + Sk)


@pytest.mark.parametrize("impl", [0, 1])
@pytest.mark.parametrize("f,sigma", [((0.5, 2.0, 0.25), 1.0), ((0.125, 0.125, 8.0), 1.0), ((1.0, 1.0, 1.0), 3.0),
                                     ((2.0 ** -6, 1.0, 2.0 ** -6), 2.0 ** -3)])
def test_dequantisation_factors_and_value_ranges(f, sigma, impl):
    check_against_oracle(2, 4, 2, 300, 515, True, impl, f=f, sigma=sigma, seed=9200)
    check_against_oracle(1, 2, 2, 515, 300, False, impl, f=f, sigma=sigma, seed=9201)


@pytest.mark.parametrize("impl", [0, 1])
def test_several_tiles_ragged_tail_and_peaked_rows(impl):
    # a large scale makes the softmax peaked: the reference maximum moves between tiles
    check_against_oracle(1, 2, 1, 1000, 1500, True, impl, seed=9300, scale=1.0)
    check_against_oracle(1, 2, 2, 777, 2100, False, impl, seed=9301, scale=0.5)


@pytest.mark.parametrize("impl", [0, 1])
def test_one_hot_selection_returns_the_selected_value_row(impl):
    # query i is aligned with key sel[i] only: p = 1 there, (almost) 0 elsewhere, so O_i = V_sel[i]; V's E4M3
    # values are exact in bf16 and p = 1 is exact in E4M3, so the result is exact up to the tiny tail
    Sq, Sk = 200, 400
    rng = np.random.default_rng(77)
    sel = rng.integers(0, Sk, size=Sq)
    one = 0x38                                          # 1.0
    k = np.zeros((1, 1, Sk, D), dtype=np.uint8)
    for j in range(Sk):                                 # key j: a distinct pattern of 9 ones out of 128 slots
        cols = [(j * 7 + 13 * t * (1 + j // 128)) % D for t in range(9)]
        k[0, 0, j, cols] = one
    q = k[:, :, sel, :].copy()
    v = inputs.randn8((1, 1, Sk, D), 78)
    kk = orc.widen_e4m3(k)[0, 0]
    g = kk @ kk.T
    off = g - np.diag(np.diag(g))
    assert off.max() <= np.diag(g).min() - 1            # every other key scores at least 1 lower (before scaling)
    scale = 60.0
    o, lse = run_gpu(torch.from_numpy(q), torch.from_numpy(k), v, scale, (1.0, 1.0, 1.0), False, impl)
    want = orc.widen_e4m3(v.numpy())[0, 0][sel]
    assert np.abs(o[0, 0] - want).max() <= 1e-6
    o_ref, lse_ref = orc.attention_fp8(q, k, v.numpy(), 1.0, 1.0, 1.0, scale, False)
    check_lse(lse, lse_ref)


def test_constant_v_gives_back_the_constant():
    # every value row equal: O = c * (sum of rounded p) / (sum of p), within the rounding statistics
    B, H, Sq, Sk = 1, 2, 256, 384
    q, k, _ = inputs.make_qkv_fp8(B, H, H, Sq, Sk, D, 9400)
    v = torch.full((B, H, Sk, D), 0x3c, dtype=torch.uint8)   # 1.5
    for causal in (False, True):
        o, _ = run_gpu(q, k, v, D ** -0.5, (1.0, 1.0, 2.0), causal, 0)
        assert np.abs(o - 3.0).max() <= 3.0 * 2.0 ** -4
        assert abs(o.mean() - 3.0) <= 0.02
        o1, _ = run_gpu(q, k, v, D ** -0.5, (1.0, 1.0, 2.0), causal, 1)
        assert np.abs(o1 - 3.0).max() <= 3.0 * 2.0 ** -8


def test_zero_scale_no_keys_and_bitwise_determinism():
    q, k, v = inputs.make_qkv_fp8(1, 2, 1, 130, 200, D, 9500)
    o, lse = run_gpu(q, k, v, 0.0, (1.0, 1.0, 1.0), True, 0)
    o_ref, lse_ref = orc.attention_fp8(q.numpy(), k.numpy(), v.numpy(), 1.0, 1.0, 1.0, 0.0, True)
    a_ref, _ = orc.attention_fp8(q.numpy(), k.numpy(), v.numpy() & 0x7f, 1.0, 1.0, 1.0, 0.0, True)
    check_o(o, o_ref, a_ref, (1.0, 1.0, 1.0), 1.0, 0)
    check_lse(lse, lse_ref)
    empty = torch.empty((1, 1, 0, D), dtype=torch.uint8)
    o0, lse0 = run_gpu(q, empty, empty, 0.1, (1.0, 1.0, 1.0), False, 0)
    assert (o0 == 0).all() and np.isneginf(lse0).all()
    a = run_gpu(q, k, v, 0.09, (0.5, 1.0, 1.0), True, 0)
    b = run_gpu(q, k, v, 0.09, (0.5, 1.0, 1.0), True, 0)
    assert np.array_equal(a[0], b[0]) and np.array_equal(a[1], b[1])


@pytest.mark.parametrize("B,H,Hkv,S,causal", [(1, 16, 16, 16384, True), (8, 16, 4, 2048, True), (2, 16, 16, 4096, False)])
def test_paper_grid_cells_on_sampled_rows(B, H, Hkv, S, causal):
    # cells of the benchmark grid of Section 4.1 (batch x sequence = 16k tokens, 16 heads of dim 128), the
    # configuration of Table 6, in the launch configuration the sweep times; rows checked one by one
    f = (0.5, 0.5, 0.25)
    q, k, v = inputs.make_qkv_fp8(B, H, Hkv, S, S, D, 9600 + S, 1.0, f)
    scale = D ** -0.5
    o, lse = run_gpu(q, k, v, scale, f, causal, 0)
    rows = inputs.sample_rows(B * H * S, S, 96, seed=S)
    qn, kn, vn = q.numpy(), k.numpy(), v.numpy()
    o_ref, lse_ref = orc.attention_rows_fp8(qn, kn, vn, f[0], f[1], f[2], rows, scale, causal)
    a_ref, _ = orc.attention_rows_fp8(qn, kn, vn & 0x7f, f[0], f[1], f[2], rows, scale, causal)
    check_o(o.reshape(-1, D)[rows], o_ref, a_ref, f, 1.0, 0)
    check_lse(lse.reshape(-1)[rows], lse_ref)
    assert not np.isnan(o).any() and not np.isnan(lse).any()


def test_tensor_core_kernel_agrees_with_cross_check_kernel_everywhere():
    f = (1.0, 0.5, 2.0)
    q, k, v = inputs.make_qkv_fp8(2, 8, 2, 1024, 1024, D, 9700, 1.0, f)
    o0, lse0 = run_gpu(q, k, v, D ** -0.5, f, True, 0)
    o1, lse1 = run_gpu(q, k, v, D ** -0.5, f, True, 1)
    assert np.abs(lse0 - lse1).max() <= 2e-3
    err = o0 - o1
    assert np.sqrt(np.mean(err ** 2)) <= 0.06 * np.sqrt(np.mean(o1 ** 2))
    # per head too: an error confined to one head or one tile would hide in the global mean
    per_head = np.sqrt(np.mean(err ** 2, axis=(2, 3))) / np.sqrt(np.mean(o1 ** 2, axis=(2, 3)))
    assert per_head.max() <= 0.07
