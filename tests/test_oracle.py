"""Pins for the fp64 CPU oracle (CPU only).

Each test holds the oracle against something other than itself: hand-derived
cases, closed forms, invariants of the definition in Section 2.2 of the paper,
a separately written dense brute force, and torch's fp64 library attention.
A plausible mistake anywhere in the oracle (dropped scale, wrong sign, base-2
log, transposed K, off-by-one causal edge, un-normalised P) fails at least one.
"""
import json
import math
import os

import numpy as np
import pytest
import torch

from oracle import attn_oracle as orc
from paper_2506_12355_b200 import inputs

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "hand_cases.json")


def rand(shape, seed, sigma=1.0):
    return np.random.default_rng(seed).normal(0.0, sigma, size=shape)


# ------------------------------------------------------------------ converters

def test_fp16_widening_all_patterns():
    allbits = np.arange(65536, dtype=np.uint16)
    got = orc.widen(allbits, orc.DTYPE_FP16)
    want = allbits.view(np.float16).astype(np.float64)
    nan = np.isnan(want)
    assert np.array_equal(np.isnan(got), nan)
    assert np.array_equal(got[~nan], want[~nan])
    assert np.array_equal(np.signbit(got[~nan]), np.signbit(want[~nan]))


def test_bf16_widening_all_patterns():
    allbits = np.arange(65536, dtype=np.uint16)
    got = orc.widen(allbits, orc.DTYPE_BF16)
    # a bf16 is the upper half of an fp32
    with np.errstate(invalid="ignore"):
        want = (allbits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    nan = np.isnan(want)
    assert np.array_equal(np.isnan(got), nan)
    assert np.array_equal(got[~nan], want[~nan])
    t = torch.from_numpy(allbits.view(np.int16).copy()).view(torch.bfloat16).to(torch.float64).numpy()
    assert np.array_equal(got[~nan], t[~nan])


# ------------------------------------------------------------------ hand cases

def _ev(x):
    if isinstance(x, (int, float)):
        return float(x)
    env = {"e": math.e, "ln": math.log}
    s = x
    for name in ("ln2", "ln3", "ln4", "ln6", "ln8"):
        s = s.replace(name, "ln(%s)" % name[2:])
    return float(eval(s, {"__builtins__": {}}, env))


def _mat(m):
    return np.array([[_ev(x) for x in row] for row in m], dtype=np.float64)


@pytest.mark.parametrize("case", ["case_2x2", "case_3x3"])
@pytest.mark.parametrize("mode", ["noncausal", "causal"])
def test_hand_cases(case, mode):
    c = json.load(open(GOLDEN))[case]
    q, k, v = (_mat(c[n])[None, None] for n in ("Q", "K", "V"))
    o, lse, rs = orc.attention(q, k, v, c["scale"], mode == "causal", return_rowsum=True)
    np.testing.assert_allclose(o[0, 0], _mat(c[mode]["O"]), rtol=0, atol=1e-14)
    np.testing.assert_allclose(lse[0, 0], [_ev(x) for x in c[mode]["LSE"]], rtol=0, atol=1e-14)
    np.testing.assert_allclose(rs, 1.0, atol=1e-14)


def test_hand_case_2x2_literal_digits():
    # the same 2x2 case against digits worked out separately (e/(e+1) = 0.7310585786300049)
    q = np.eye(2)[None, None]
    v = np.array([[1.0, 2.0], [3.0, 4.0]])[None, None]
    o, lse = orc.attention(q, q, v, 1.0, False)
    np.testing.assert_allclose(o[0, 0, 0], [1.5378828427399902, 2.5378828427399904], atol=1e-14)
    np.testing.assert_allclose(o[0, 0, 1], [2.46211715726001, 3.4621171572600096], atol=1e-14)
    np.testing.assert_allclose(lse[0, 0], [1.3132616875182228] * 2, atol=1e-14)


# ------------------------------------------------------------------ invariants

@pytest.mark.parametrize("causal", [False, True])
def test_probability_rows_sum_to_one(causal):
    q, k, v = rand((2, 3, 37, 16), 1), rand((2, 3, 53, 16), 2), rand((2, 3, 53, 16), 3)
    _, _, rs = orc.attention(q, k, v, 0.25, causal, return_rowsum=True)
    assert np.max(np.abs(rs - 1.0)) <= 1e-12


@pytest.mark.parametrize("causal", [False, True])
def test_constant_v_returns_constant(causal):
    q, k = rand((1, 2, 19, 8), 4), rand((1, 2, 31, 8), 5)
    v = np.full((1, 2, 31, 8), -3.25)
    o, _ = orc.attention(q, k, v, 0.7, causal)
    assert np.max(np.abs(o + 3.25)) <= 1e-12


@pytest.mark.parametrize("causal", [False, True])
def test_identical_keys_give_mean_of_v(causal):
    B, H, Sq, Sk, D = 1, 2, 9, 13, 8
    q, v = rand((B, H, Sq, D), 6), rand((B, H, Sk, D), 7)
    k0 = rand((B, H, 1, D), 8)
    k = np.repeat(k0, Sk, axis=2)
    scale = 0.3
    o, lse = orc.attention(q, k, v, scale, causal)
    for i in range(Sq):
        n = min(i + 1, Sk) if causal else Sk
        np.testing.assert_allclose(o[:, :, i], v[:, :, :n].mean(axis=2), atol=1e-12)
        want = scale * np.einsum("bhd,bhd->bh", q[:, :, i], k0[:, :, 0]) + math.log(n)
        np.testing.assert_allclose(lse[:, :, i], want, atol=1e-12)


def test_zero_queries_and_zero_scale():
    B, H, Sq, Sk, D = 1, 1, 5, 11, 4
    k, v = rand((B, H, Sk, D), 9), rand((B, H, Sk, D), 10)
    o, lse = orc.attention(np.zeros((B, H, Sq, D)), k, v, 1.0, False)
    np.testing.assert_allclose(lse, math.log(Sk), atol=1e-13)
    np.testing.assert_allclose(o, np.broadcast_to(v.mean(axis=2, keepdims=True), o.shape), atol=1e-13)
    o2, lse2 = orc.attention(rand((B, H, Sq, D), 11), k, v, 0.0, True)
    for i in range(Sq):
        np.testing.assert_allclose(lse2[0, 0, i], math.log(i + 1), atol=1e-13)
        np.testing.assert_allclose(o2[0, 0, i], v[0, 0, :i + 1].mean(axis=0), atol=1e-13)


@pytest.mark.parametrize("Sq,Sk", [(7, 7), (5, 9), (9, 5)])
def test_causal_first_row_and_alignment(Sq, Sk):
    q, k, v = rand((1, 2, Sq, 8), 12), rand((1, 2, Sk, 8), 13), rand((1, 2, Sk, 8), 14)
    scale = 0.5
    oc, lc = orc.attention(q, k, v, scale, True)
    on, ln_ = orc.attention(q, k, v, scale, False)
    np.testing.assert_allclose(oc[:, :, 0], v[:, :, 0], atol=1e-14)
    np.testing.assert_allclose(lc[:, :, 0], scale * np.einsum("bhd,bhd->bh", q[:, :, 0], k[:, :, 0]),
                               atol=1e-14)
    # top-left alignment: every row i >= Sk-1 sees all keys, i.e. equals the unmasked result
    for i in range(Sq):
        if i >= Sk - 1:
            np.testing.assert_allclose(oc[:, :, i], on[:, :, i], atol=1e-14)
            np.testing.assert_allclose(lc[:, :, i], ln_[:, :, i], atol=1e-14)
        else:
            # row i equals an unmasked problem over the first i+1 keys
            oi, li = orc.attention(q[:, :, i:i + 1], k[:, :, :i + 1], v[:, :, :i + 1], scale, False)
            np.testing.assert_allclose(oc[:, :, i], oi[:, :, 0], atol=1e-14)
            np.testing.assert_allclose(lc[:, :, i], li[:, :, 0], atol=1e-14)


def test_key_shift_invariance():
    q, k, v = rand((1, 2, 6, 8), 15), rand((1, 2, 10, 8), 16), rand((1, 2, 10, 8), 17)
    u = rand((1, 2, 1, 8), 18)
    scale = 0.4
    o1, l1 = orc.attention(q, k, v, scale, False)
    o2, l2 = orc.attention(q, k + u, v, scale, False)
    np.testing.assert_allclose(o2, o1, atol=1e-12)
    np.testing.assert_allclose(l2 - l1, scale * np.einsum("bhid,bhd->bhi", q, u[:, :, 0]), atol=1e-12)


def test_key_permutation_invariance():
    q, k, v = rand((1, 1, 6, 8), 19), rand((1, 1, 21, 8), 20), rand((1, 1, 21, 8), 21)
    perm = np.random.default_rng(22).permutation(21)
    o1, l1 = orc.attention(q, k, v, 0.35, False)
    o2, l2 = orc.attention(q, k[:, :, perm], v[:, :, perm], 0.35, False)
    np.testing.assert_allclose(o2, o1, atol=1e-12)
    np.testing.assert_allclose(l2, l1, atol=1e-12)


def test_split_combine_identity():
    q, k, v = rand((1, 2, 8, 8), 23), rand((1, 2, 24, 8), 24), rand((1, 2, 24, 8), 25)
    o, lse = orc.attention(q, k, v, 0.3, False)
    oa, la = orc.attention(q, k[:, :, :10], v[:, :, :10], 0.3, False)
    ob, lb = orc.attention(q, k[:, :, 10:], v[:, :, 10:], 0.3, False)
    l = np.logaddexp(la, lb)
    oc = np.exp(la - l)[..., None] * oa + np.exp(lb - l)[..., None] * ob
    np.testing.assert_allclose(l, lse, atol=1e-12)
    np.testing.assert_allclose(oc, o, atol=1e-12)


def test_one_hot_limit_is_overflow_safe():
    q, k, v = rand((1, 1, 4, 8), 26), rand((1, 1, 16, 8), 27), rand((1, 1, 16, 8), 28)
    scale = 1e4
    o, lse = orc.attention(q, k, v, scale, False)
    s = scale * np.einsum("id,jd->ij", q[0, 0], k[0, 0])
    arg = s.argmax(axis=1)
    assert np.all(np.isfinite(o)) and np.all(np.isfinite(lse))
    np.testing.assert_allclose(o[0, 0], v[0, 0, arg], atol=1e-9)
    np.testing.assert_allclose(lse[0, 0], s.max(axis=1), rtol=1e-9)


def test_no_visible_key_convention():
    q = rand((1, 1, 3, 4), 29)
    k = np.zeros((1, 1, 0, 4))
    o, lse = orc.attention(q, k, k, 1.0, False)
    assert np.all(o == 0.0) and np.all(np.isneginf(lse))


# ------------------------------------------------------------------ brute force and library

def dense_brute_force(q, k, v, scale, causal):
    """Builds the full score, mask and probability matrices -- written separately from the oracle."""
    B, H, Sq, D = q.shape
    Sk = k.shape[2]
    o = np.zeros((B, H, Sq, D))
    lse = np.zeros((B, H, Sq))
    for b in range(B):
        for h in range(H):
            S = (q[b, h] @ k[b, h].T) * scale
            if causal:
                mask = np.triu(np.ones((Sq, Sk), dtype=bool), k=1)
                S = np.where(mask, -np.inf, S)
            E = np.exp(S)                       # small inputs: no overflow without max-subtraction
            Z = E.sum(axis=1, keepdims=True)
            o[b, h] = (E / Z) @ v[b, h]
            lse[b, h] = np.log(Z[:, 0])
    return o, lse


@pytest.mark.parametrize("causal", [False, True])
@pytest.mark.parametrize("shape", [(1, 1, 1, 1, 1), (2, 2, 16, 16, 8), (1, 2, 5, 12, 3), (2, 1, 13, 4, 7)])
def test_against_dense_brute_force(shape, causal):
    B, H, Sq, Sk, D = shape
    q, k, v = rand((B, H, Sq, D), 30), rand((B, H, Sk, D), 31), rand((B, H, Sk, D), 32)
    o, lse = orc.attention(q, k, v, 1.0 / math.sqrt(D), causal)
    ob, lb = dense_brute_force(q, k, v, 1.0 / math.sqrt(D), causal)
    np.testing.assert_allclose(o, ob, atol=1e-12)
    np.testing.assert_allclose(lse, lb, atol=1e-12)


@pytest.mark.parametrize("causal", [False, True])
def test_against_torch_sdpa_fp64(causal):
    B, H, Sq, Sk, D = 2, 3, 65, 65, 32
    q, k, v = rand((B, H, Sq, D), 33), rand((B, H, Sk, D), 34), rand((B, H, Sk, D), 35)
    scale = 0.17
    o, lse = orc.attention(q, k, v, scale, causal)
    tq, tk, tv = (torch.from_numpy(x) for x in (q, k, v))
    to = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, is_causal=causal, scale=scale)
    np.testing.assert_allclose(o, to.numpy(), atol=1e-10)
    s = (tq @ tk.transpose(-1, -2)) * scale
    if causal:
        s = s.masked_fill(torch.triu(torch.ones(Sq, Sk, dtype=torch.bool), 1), float("-inf"))
    np.testing.assert_allclose(lse, torch.logsumexp(s, dim=-1).numpy(), atol=1e-10)


# ------------------------------------------------------------------ the 16-bit row-subset entry

@pytest.mark.parametrize("dtype", [inputs.DTYPE_FP16, inputs.DTYPE_BF16])
@pytest.mark.parametrize("causal", [False, True])
def test_row_subset_entry_matches_full(dtype, causal):
    B, H, Sq, Sk, D = 2, 2, 40, 56, 16
    q, k, v = inputs.make_qkv(B, H, Sq, Sk, D, dtype, seed=77)
    qb, kb, vb = inputs.bits(q), inputs.bits(k), inputs.bits(v)
    o, lse = orc.attention(orc.widen(qb, dtype), orc.widen(kb, dtype), orc.widen(vb, dtype), 0.25, causal)
    rows = np.array([0, 1, 39, 40, 79, 100, 159], dtype=np.int64)
    orows, lrows = orc.attention_rows_16(qb, kb, vb, dtype, rows, 0.25, causal)
    np.testing.assert_array_equal(orows, o.reshape(-1, D)[rows])
    np.testing.assert_array_equal(lrows, lse.reshape(-1)[rows])


def test_input_generator_is_seeded_and_rounded():
    a = inputs.randn16((3, 5), 123, inputs.DTYPE_BF16)
    b = inputs.randn16((3, 5), 123, inputs.DTYPE_BF16)
    c = inputs.randn16((3, 5), 124, inputs.DTYPE_BF16)
    assert torch.equal(a, b) and not torch.equal(a, c)
    assert a.dtype == torch.bfloat16
    w = orc.widen(inputs.bits(a), inputs.DTYPE_BF16)
    np.testing.assert_array_equal(w, a.to(torch.float64).numpy())


# ------------------------------------------------------------------ grouped-query attention

@pytest.mark.parametrize("causal", [False, True])
@pytest.mark.parametrize("H,Hkv", [(6, 2), (4, 1), (3, 3)])
def test_gqa_equals_mha_with_repeated_kv_heads(H, Hkv, causal):
    # query head h reads K/V head h // (H // Hkv): the same as plain attention on K/V with every
    # head repeated H // Hkv times (built here with numpy, not with the oracle's index arithmetic)
    B, Sq, Sk, D = 2, 9, 14, 8
    q, k, v = rand((B, H, Sq, D), 40), rand((B, Hkv, Sk, D), 41), rand((B, Hkv, Sk, D), 42)
    o, lse = orc.attention_gqa(q, k, v, 0.3, causal)
    o_ref, lse_ref = orc.attention(q, np.repeat(k, H // Hkv, axis=1), np.repeat(v, H // Hkv, axis=1), 0.3, causal)
    np.testing.assert_array_equal(o, o_ref)
    np.testing.assert_array_equal(lse, lse_ref)
    to = torch.nn.functional.scaled_dot_product_attention(torch.from_numpy(q), torch.from_numpy(k), torch.from_numpy(v),
                                                          is_causal=causal, scale=0.3, enable_gqa=True)
    np.testing.assert_allclose(o, to.numpy(), atol=1e-10)


def test_gqa_rejects_indivisible_heads():
    with pytest.raises(ValueError):
        orc.attention_gqa(rand((1, 5, 2, 4), 1), rand((1, 2, 2, 4), 2), rand((1, 2, 2, 4), 3), 1.0, False)


# ------------------------------------------------------------------ separate Q/K and V head dims

@pytest.mark.parametrize("causal", [False, True])
def test_separate_v_dim_equals_zero_padded_v(causal):
    # O with a narrower V equals the leading columns of plain attention on V padded with zero columns
    B, H, Hkv, Sq, Sk, D, Dv = 2, 4, 2, 7, 11, 12, 8
    q, k, v = rand((B, H, Sq, D), 50), rand((B, Hkv, Sk, D), 51), rand((B, Hkv, Sk, Dv), 52)
    o, lse = orc.attention_gqa_dv(q, k, v, 0.2, causal)
    vpad = np.concatenate([v, np.zeros((B, Hkv, Sk, D - Dv))], axis=3)
    o_ref, lse_ref = orc.attention_gqa(q, k, vpad, 0.2, causal)
    np.testing.assert_array_equal(o, o_ref[..., :Dv])
    assert np.all(o_ref[..., Dv:] == 0.0)
    np.testing.assert_array_equal(lse, lse_ref)
    to = torch.nn.functional.scaled_dot_product_attention(torch.from_numpy(q), torch.from_numpy(k), torch.from_numpy(v),
                                                          is_causal=causal, scale=0.2, enable_gqa=True)
    np.testing.assert_allclose(o, to.numpy(), atol=1e-10)


# ------------------------------------------------------------------ K/V shards and their merge

@pytest.mark.parametrize("causal", [False, True])
def test_shards_merge_to_the_unsharded_result(causal):
    # keys cut into three uneven shards; each shard evaluated with its global key offset; the merge
    # must give the one-shot result (pins the offset convention of the causal mask and the merge)
    B, H, Hkv, Sq, Sk, D = 1, 4, 2, 23, 31, 8
    q, k, v = rand((B, H, Sq, D), 60), rand((B, Hkv, Sk, D), 61), rand((B, Hkv, Sk, D), 62)
    o_ref, lse_ref = orc.attention_gqa(q, k, v, 0.3, causal)
    cuts = [0, 5, 18, Sk]
    parts = [orc.attention_shard(q, k[:, :, a:b], v[:, :, a:b], 0.3, causal, a) for a, b in zip(cuts, cuts[1:])]
    if causal:   # early rows see nothing of the later shards
        assert np.all(np.isneginf(parts[2][1][:, :, :18])) and np.all(parts[2][0][:, :, :18] == 0.0)
        assert np.all(np.isfinite(parts[2][1][:, :, 18:]))
    o, lse = orc.combine(np.stack([p[0] for p in parts]), np.stack([p[1] for p in parts]))
    np.testing.assert_allclose(o, o_ref, atol=1e-12)
    np.testing.assert_allclose(lse, lse_ref, atol=1e-12)
    # the merge against numpy's logaddexp written out separately
    l_np = np.logaddexp.reduce(np.stack([p[1] for p in parts]), axis=0)
    np.testing.assert_allclose(lse, l_np, atol=1e-12)


def test_shard_with_zero_offset_is_plain_attention_and_empty_merge():
    q, k, v = rand((1, 2, 6, 4), 63), rand((1, 2, 9, 4), 64), rand((1, 2, 9, 4), 65)
    o, lse = orc.attention_shard(q, k, v, 0.5, True, 0)
    o_ref, lse_ref = orc.attention(q, k, v, 0.5, True)
    np.testing.assert_array_equal(o, o_ref)
    np.testing.assert_array_equal(lse, lse_ref)
    o2, lse2 = orc.combine(np.zeros((2, 3, 4)), np.full((2, 3), -np.inf))
    assert np.all(o2 == 0.0) and np.all(np.isneginf(lse2))


# ------------------------------------------------------------------ 8-bit (E4M3) inputs, Section 4.4 / Table 6

def test_e4m3_widening_all_patterns():
    allbits = np.arange(256, dtype=np.uint8)
    got = orc.widen_e4m3(allbits)
    want = torch.from_numpy(allbits.copy()).view(torch.float8_e4m3fn).to(torch.float64).numpy()
    nan = np.isnan(want)
    assert nan.sum() == 2 and np.array_equal(nan, np.isnan(got))          # 0x7f and 0xff only
    np.testing.assert_array_equal(got[~nan], want[~nan])
    assert np.array_equal(np.signbit(got[~nan]), np.signbit(want[~nan]))
    # landmarks of the format, from its definition (bias 7, 3 fraction bits, no infinities)
    for code, val in [(0x38, 1.0), (0x7e, 448.0), (0x01, 2.0 ** -9), (0x07, 7 * 2.0 ** -9), (0x08, 2.0 ** -6),
                      (0x40, 2.0), (0x3c, 1.5), (0xc5, -3.25), (0x78, 256.0)]:
        assert got[code] == val
    assert orc.widen_e4m3(np.array([0x3c], dtype=np.uint8), 0.5)[0] == 0.75   # the factor multiplies the value


@pytest.mark.parametrize("causal", [False, True])
def test_fp8_attention_is_the_definition_on_dequantised_tensors(causal):
    B, H, Hkv, Sq, Sk, D = 2, 4, 2, 33, 47, 16
    fq, fk, fv = 0.5, 2.0, 0.125
    q, k, v = inputs.make_qkv_fp8(B, H, Hkv, Sq, Sk, D, seed=311, factors=(fq, fk, fv))
    scale = 0.3
    o, lse = orc.attention_fp8(q.numpy(), k.numpy(), v.numpy(), fq, fk, fv, scale, causal)
    # torch's own 8-bit decoding and fp64 library attention on the dequantised tensors
    tq = q.view(torch.float8_e4m3fn).to(torch.float64) * fq
    tk = (k.view(torch.float8_e4m3fn).to(torch.float64) * fk).repeat_interleave(H // Hkv, dim=1)
    tv = (v.view(torch.float8_e4m3fn).to(torch.float64) * fv).repeat_interleave(H // Hkv, dim=1)
    to = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, is_causal=causal, scale=scale)
    np.testing.assert_allclose(o, to.numpy(), atol=1e-12)
    s = (tq @ tk.transpose(-1, -2)) * scale
    if causal:
        s = s.masked_fill(torch.triu(torch.ones(Sq, Sk, dtype=torch.bool), 1), float("-inf"))
    np.testing.assert_allclose(lse, torch.logsumexp(s, dim=-1).numpy(), atol=1e-12)
    # the factors act as the definition says: q and k factors only through the scores, v's linearly
    o2, lse2 = orc.attention_fp8(q.numpy(), k.numpy(), v.numpy(), 1.0, 1.0, 1.0, scale * fq * fk, causal)
    np.testing.assert_allclose(o2 * fv, o, rtol=1e-13, atol=1e-15)
    np.testing.assert_allclose(lse2, lse, rtol=1e-13, atol=1e-13)


@pytest.mark.parametrize("causal", [False, True])
def test_fp8_row_subset_entry_matches_full(causal):
    B, H, Hkv, Sq, Sk, D = 2, 4, 2, 40, 56, 16
    fq, fk, fv = 0.25, 1.0, 4.0
    q, k, v = inputs.make_qkv_fp8(B, H, Hkv, Sq, Sk, D, seed=312, factors=(fq, fk, fv))
    o, lse = orc.attention_fp8(q.numpy(), k.numpy(), v.numpy(), fq, fk, fv, 0.25, causal)
    rows = np.array([0, 1, 39, 40, 79, 100, 159, 160, 319], dtype=np.int64)
    orows, lrows = orc.attention_rows_fp8(q.numpy(), k.numpy(), v.numpy(), fq, fk, fv, rows, 0.25, causal)
    np.testing.assert_array_equal(orows, o.reshape(-1, D)[rows])
    np.testing.assert_array_equal(lrows, lse.reshape(-1)[rows])


def test_fp8_input_generator_is_seeded_clamped_and_rounded():
    a = inputs.randn8((3, 5, 7), 99, sigma=2.0, factor=0.5)
    b = inputs.randn8((3, 5, 7), 99, sigma=2.0, factor=0.5)
    assert a.dtype == torch.uint8 and torch.equal(a, b)
    g = torch.Generator(device="cpu")
    g.manual_seed(99)
    x = torch.randn((3, 5, 7), generator=g, dtype=torch.float32) * 4.0
    val = orc.widen_e4m3(a.numpy())
    assert not np.isnan(val).any()
    # nearest representable value: the error is at most half a unit in the last place (2^-4 relative, 2^-10 absolute)
    err = np.abs(val - x.numpy().astype(np.float64))
    assert np.all(err <= np.maximum(np.abs(x.numpy()) * 2.0 ** -4, 2.0 ** -10))
    big = inputs.randn8((1000,), 5, sigma=1000.0)
    assert np.nanmax(np.abs(orc.widen_e4m3(big.numpy()))) == 448.0


# ------------------------------------------------------------------ backward pass (gradients of the same operator)

def _loss(q, k, v, dout, scale, causal, gqa):
    """sum(O * dout) through the oracle's FORWARD entries: its gradients are what attention_bwd must return."""
    o, _ = (orc.attention_gqa if gqa else orc.attention)(q, k, v, scale, causal)
    return float((o * dout).sum())


@pytest.mark.parametrize("mode", ["noncausal", "causal"])
def test_bwd_hand_case_2x2(mode):
    g = json.load(open(GOLDEN))
    c, b = g["case_2x2"], g["case_2x2_bwd"]
    q, k, v, dout = (_mat(m)[None, None] for m in (c["Q"], c["K"], c["V"], b["dO"]))
    dq, dk, dv = orc.attention_bwd(q, k, v, dout, c["scale"], mode == "causal")
    np.testing.assert_allclose(dq[0, 0], _mat(b[mode]["dQ"]), rtol=0, atol=1e-14)
    np.testing.assert_allclose(dk[0, 0], _mat(b[mode]["dK"]), rtol=0, atol=1e-14)
    np.testing.assert_allclose(dv[0, 0], _mat(b[mode]["dV"]), rtol=0, atol=1e-14)
    if mode == "noncausal":   # digits worked out separately: 2e/(e+1)^2
        np.testing.assert_allclose(dq[0, 0, 0, 1], b["literal_g"], rtol=0, atol=1e-15)


@pytest.mark.parametrize("causal", [False, True])
@pytest.mark.parametrize("shape", [(1, 1, 1, 3, 5, 4), (2, 2, 2, 4, 4, 3), (1, 4, 2, 5, 3, 2), (1, 2, 1, 3, 7, 4)])
def test_bwd_matches_central_finite_differences(shape, causal):
    # every entry of dq, dk, dv against (L(x + h) - L(x - h)) / 2h of the forward oracle, L = sum(O * dout)
    B, H, Hkv, Sq, Sk, D = shape
    q, k, v, dout = rand((B, H, Sq, D), 1), rand((B, Hkv, Sk, D), 2), rand((B, Hkv, Sk, D), 3), rand((B, H, Sq, D), 4)
    scale = 0.7
    dq, dk, dv = orc.attention_bwd(q, k, v, dout, scale, causal)
    h = 1e-6
    for name, x, grad in (("q", q, dq), ("k", k, dk), ("v", v, dv)):
        num = np.zeros_like(x)
        it = np.nditer(x, flags=["multi_index"])
        for _ in it:
            idx = it.multi_index
            keep = x[idx]
            x[idx] = keep + h
            up = _loss(q, k, v, dout, scale, causal, True)
            x[idx] = keep - h
            dn = _loss(q, k, v, dout, scale, causal, True)
            x[idx] = keep
            num[idx] = (up - dn) / (2 * h)
        np.testing.assert_allclose(grad, num, rtol=0, atol=2e-8, err_msg="d" + name)


@pytest.mark.parametrize("causal", [False, True])
@pytest.mark.parametrize("H,Hkv", [(3, 3), (4, 2), (4, 1)])
def test_bwd_against_torch_autograd_fp64(H, Hkv, causal):
    B, Sq, Sk, D = 2, 33, 47, 16
    q, k, v, dout = rand((B, H, Sq, D), 11), rand((B, Hkv, Sk, D), 12), rand((B, Hkv, Sk, D), 13), rand((B, H, Sq, D), 14)
    scale = 0.31
    dq, dk, dv = orc.attention_bwd(q, k, v, dout, scale, causal)
    tq, tk, tv = (torch.from_numpy(x).clone().requires_grad_(True) for x in (q, k, v))
    # library attention in fp64 with an explicit top-left mask (Sq != Sk), K/V heads repeated for the groups
    rep = H // Hkv
    s = torch.einsum("bhid,bhjd->bhij", tq, tk.repeat_interleave(rep, dim=1)) * scale
    if causal:
        mask = torch.arange(Sk)[None, :] > torch.arange(Sq)[:, None]
        s = s.masked_fill(mask, float("-inf"))
    o = torch.einsum("bhij,bhjd->bhid", torch.softmax(s, dim=-1), tv.repeat_interleave(rep, dim=1))
    o.backward(torch.from_numpy(dout))
    np.testing.assert_allclose(dq, tq.grad.numpy(), rtol=0, atol=1e-12)
    np.testing.assert_allclose(dk, tk.grad.numpy(), rtol=0, atol=1e-12)
    np.testing.assert_allclose(dv, tv.grad.numpy(), rtol=0, atol=1e-12)


def test_bwd_invariants():
    B, H, Sq, Sk, D = 1, 2, 9, 11, 4
    q, k, v, dout = rand((B, H, Sq, D), 21), rand((B, H, Sk, D), 22), rand((B, H, Sk, D), 23), rand((B, H, Sq, D), 24)
    # constant V: O does not depend on the probabilities, so no gradient reaches Q and K, and the
    # probability rows sum to one: sum_j dv_j = sum_i dO_i
    vc = np.broadcast_to(rand((B, H, 1, D), 25), (B, H, Sk, D)).copy()
    dq, dk, dv = orc.attention_bwd(q, k, vc, dout, 0.5, True)
    assert np.abs(dq).max() < 1e-14 and np.abs(dk).max() < 1e-14
    np.testing.assert_allclose(dv.sum(axis=2), dout.sum(axis=2), atol=1e-13)
    # identical keys: the scores of a row are all equal, dq_i = scale * (sum_j ds_j) * k0 = 0
    kc = np.broadcast_to(rand((B, H, 1, D), 26), (B, H, Sk, D)).copy()
    dq, _, dv = orc.attention_bwd(q, kc, v, dout, 0.5, False)
    assert np.abs(dq).max() < 1e-14
    np.testing.assert_allclose(dv, np.broadcast_to(dout.sum(axis=2, keepdims=True) / Sk, dv.shape), atol=1e-13)
    # causal, Sq == Sk: the last key is seen by the last row only; rows see nothing beyond themselves
    q2, d2 = rand((B, H, Sk, D), 27), rand((B, H, Sk, D), 28)
    dq, dk, dv = orc.attention_bwd(q2, k, v, d2, 0.5, True)
    assert np.abs(dq[:, :, 0]).max() < 1e-14          # row 0 sees one key: constant softmax
    # dv of the last key = p(last row, last key) * dO(last row), with p written out here
    s_last = 0.5 * np.einsum("bhd,bhjd->bhj", q2[:, :, -1], k)
    p_last = np.exp(s_last - s_last.max(-1, keepdims=True))
    p_last /= p_last.sum(-1, keepdims=True)
    np.testing.assert_allclose(dv[:, :, -1], p_last[:, :, -1:] * d2[:, :, -1], atol=1e-14)
    # scaling the loss scales every gradient; zero upstream gradient gives zero gradients
    g1 = orc.attention_bwd(q, k, v, dout, 0.5, True)
    g3 = orc.attention_bwd(q, k, v, 3.0 * dout, 0.5, True)
    for a, b3 in zip(g1, g3):
        np.testing.assert_allclose(3.0 * a, b3, atol=1e-13)
    for a in orc.attention_bwd(q, k, v, np.zeros_like(dout), 0.5, True):
        assert np.abs(a).max() == 0.0


def test_bwd_rejects_indivisible_heads_and_handles_no_keys():
    with pytest.raises(ValueError):
        orc.attention_bwd(rand((1, 3, 2, 2), 1), rand((1, 2, 2, 2), 2), rand((1, 2, 2, 2), 3), rand((1, 3, 2, 2), 4), 1.0, False)
    dq, dk, dv = orc.attention_bwd(rand((1, 1, 3, 2), 1), np.zeros((1, 1, 0, 2)), np.zeros((1, 1, 0, 2)), rand((1, 1, 3, 2), 4), 1.0, True)
    assert dq.shape == (1, 1, 3, 2) and np.abs(dq).max() == 0.0 and dk.size == 0 and dv.size == 0
