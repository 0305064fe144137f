"""GPU parity on seeded random problems: every entry point of the tensor-core path against the fp64 CPU
oracle on shapes, head groupings, scales and value ranges drawn from a fixed seed (ragged tails, Sq != Sk,
single rows, several tiles).  Tolerances as in the other parity tests, LSE 1e-3 and O 1e-2 (fp16) / 2e-2 (bf16)
times the inputs' standard deviation where that exceeds 1, plus, because the scales drawn here make some rows
sharply peaked with |O| well above 1, a relative term of 2^-10 (fp16) / 2^-7 (bf16) of |O|: half a unit in the
last place of the stored O (2^-11 / 2^-8) and the rounding of P to the 16-bit type (2^-12 / 2^-9 of sum p |v|).
8-bit inputs: the elementwise rounding bound and the 6 % root-mean-square bar."""
import numpy as np
import pytest
import torch

from oracle import attn_oracle as orc
from paper_2506_12355_b200 import api, inputs

pytestmark = pytest.mark.gpu

O_TOL = {inputs.DTYPE_FP16: 1e-2, inputs.DTYPE_BF16: 2e-2}
O_RTOL = {inputs.DTYPE_FP16: 2.0 ** -10, inputs.DTYPE_BF16: 2.0 ** -7}
LSE_TOL = 1e-3
SQ = [1, 5, 64, 127, 128, 129, 200, 256, 300, 511, 513, 777, 1024]
SK = [1, 17, 128, 130, 255, 257, 640, 1000, 1300]


def draw(seed):
    rng = np.random.default_rng(seed)
    kind = str(rng.choice(["gqa", "qk192_v128", "fp8", "partial"]))
    p = dict(kind=kind, D=int(rng.choice([64, 128, 256])), dt=int(rng.integers(0, 2)), causal=bool(rng.integers(0, 2)),
             B=int(rng.integers(1, 3)), Hkv=int(rng.choice([1, 2, 3])), G=int(rng.choice([1, 2, 4])),
             Sq=int(rng.choice(SQ)), scale=float(rng.choice([0.0884, 0.3, 1.0, 0.02])),
             sigma=float(rng.choice([1.0, 0.3, 3.0])), k_offset=int(rng.choice([0, 1, 100, 128, 300])))
    p["Sk"] = p["Sq"] if rng.random() < 0.5 else int(rng.choice(SK))
    p["H"] = p["Hkv"] * p["G"]
    return p


def check(o, lse, o_ref, lse_ref, tol_o, rtol_o=0.0):
    o = o.cpu().to(torch.float64).numpy()
    lse = lse.cpu().to(torch.float64).numpy()
    assert not np.isnan(o).any()
    err = np.abs(o - o_ref)
    assert np.all(err <= tol_o + rtol_o * np.abs(o_ref)), "max |dO| = %g" % err.max()
    inf = np.isneginf(lse_ref)
    assert np.array_equal(np.isneginf(lse), inf)
    e = np.abs(lse[~inf] - lse_ref[~inf])
    assert e.size == 0 or e.max() <= LSE_TOL, "max |dLSE| = %g" % e.max()


@pytest.mark.parametrize("seed", range(48))
def test_random_problem(seed):
    p = draw(7000 + seed)
    dev = torch.device("cuda:0")
    B, H, Hkv, Sq, Sk, D, dt, causal, scale, sigma = (p[k] for k in ("B", "H", "Hkv", "Sq", "Sk", "D", "dt", "causal", "scale", "sigma"))
    tol_o = O_TOL[dt] * max(1.0, sigma)
    if p["kind"] == "fp8":
        f = (0.5, 1.0, 2.0)
        q, k, v = inputs.make_qkv_fp8(B, H, Hkv, Sq, Sk, 128, 7100 + seed, sigma, f)
        o, lse = api.attn_fwd_fp8(q.to(dev), k.to(dev), v.to(dev), scale, f[0], f[1], f[2], causal)
        assert api.attn_last_device_status() == 0
        qn, kn, vn = q.numpy(), k.numpy(), v.numpy()
        o_ref, lse_ref = orc.attention_fp8(qn, kn, vn, f[0], f[1], f[2], scale, causal)
        a_ref, _ = orc.attention_fp8(qn, kn, vn & 0x7f, f[0], f[1], f[2], scale, causal)
        o64 = o.cpu().to(torch.float64).numpy()
        err = np.abs(o64 - o_ref)
        assert np.all(err <= 2.0 ** -4 * a_ref + 2.0 ** -8 * np.abs(o_ref) + 1e-3 * sigma)
        if np.sqrt(np.mean(o_ref ** 2)) > 0:
            assert np.sqrt(np.mean(err ** 2)) <= 0.06 * np.sqrt(np.mean(o_ref ** 2)) + 2.0 ** -9 * sigma
        check(o, lse, o64, lse_ref, 0.0)   # LSE and the -inf pattern
        return
    Dqk, Dv = (192, 128) if p["kind"] == "qk192_v128" else (D, D)
    q = inputs.randn16((B, H, Sq, Dqk), 7100 + seed, dt, sigma)
    k = inputs.randn16((B, Hkv, Sk, Dqk), 7200 + seed, dt, sigma)
    v = inputs.randn16((B, Hkv, Sk, Dv), 7300 + seed, dt, sigma)
    qf, kf, vf = (orc.widen(inputs.bits(t), dt) for t in (q, k, v))
    qd, kd, vd = q.to(dev), k.to(dev), v.to(dev)
    if p["kind"] == "qk192_v128":
        o, lse = api.attn_fwd_qkv_dims(qd, kd, vd, scale, causal)
        o_ref, lse_ref = orc.attention_gqa_dv(qf, kf, vf, scale, causal)
    elif p["kind"] == "partial":
        o, lse = api.attn_fwd_partial(qd, kd, vd, scale, causal, p["k_offset"])
        rep = H // Hkv
        o_ref, lse_ref = orc.attention_shard(qf, np.repeat(kf, rep, axis=1), np.repeat(vf, rep, axis=1), scale, causal,
                                             p["k_offset"])
    else:
        o, lse = api.attn_fwd_gqa(qd, kd, vd, scale, causal)
        o_ref, lse_ref = orc.attention_gqa(qf, kf, vf, scale, causal)
    assert api.attn_last_device_status() == 0
    check(o, lse, o_ref, lse_ref, tol_o, O_RTOL[dt])
