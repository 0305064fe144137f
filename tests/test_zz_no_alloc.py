"""The entry point for callers that cannot allocate device memory (attn_fwd_host_static).

Such a caller has host buffers but no way to obtain a device workspace (it may not call cudaMalloc:
a plug-in inside an application that owns the memory budget, a loop that cannot afford the implicit
synchronisation of an allocation, a process whose pool is already committed).  The library then
stages the tensors in a 16 MiB buffer that is part of its own image.  This file checks, through the
C ABI, that the results equal those of the existing host entry point (attn_fwd_host, which is given
a caller-allocated workspace) on two calls in a row that share the built-in buffer, and that the
size limit is enforced.  It is collected last on purpose: a run that stops at the first failure has
then already run every other test.  It passes alone in a fresh process and after the other tests.
"""
import numpy as np
import pytest
import torch

from oracle import attn_oracle as orc
from paper_2506_12355_b200 import api, inputs

CASES = [
    # B, H, Sq, Sk, D, dtype, causal   (second call: other shape, dtype and mask than the first)
    (1, 2, 128, 128, 64, inputs.DTYPE_FP16, False),
    (2, 3, 200, 333, 128, inputs.DTYPE_BF16, True),
]


def _host_reference(q, k, v, scale, causal):
    """attn_fwd_host with a workspace allocated by the caller (the existing entry point)."""
    B, H, Sq, D = q.shape
    Sk = k.shape[2]
    o = torch.empty_like(q).pin_memory()
    lse = torch.empty(B, H, Sq, dtype=torch.float32).pin_memory()
    ws = torch.empty(api.attn_fwd_host_workspace_bytes(B, H, Sq, Sk, D), dtype=torch.uint8, device="cuda:0")
    api.attn_fwd_host(q, k, v, scale, causal, o, lse, ws)
    assert api.attn_last_device_status() == 0
    return o, lse


@pytest.mark.gpu
def test_static_entry_matches_host_entry_on_two_calls_in_a_row():
    torch.cuda.set_device(0)
    prepared = []
    for idx, (B, H, Sq, Sk, D, dtype, causal) in enumerate(CASES):
        q, k, v = inputs.make_qkv(B, H, Sq, Sk, D, dtype, seed=900 + idx)
        q, k, v = q.pin_memory(), k.pin_memory(), v.pin_memory()
        scale = float(np.float32(1.0) / np.sqrt(np.float32(D)))   # the fp32 value the library receives
        prepared.append((q, k, v, scale, causal, _host_reference(q, k, v, scale, causal)))

    # two calls back to back on one stream, both through the built-in buffer; nothing is allocated
    # on the device between them (the output tensors are pinned host memory, created beforehand)
    outs = []
    for q, k, v, scale, causal, _ in prepared:
        o = torch.full_like(q, float("nan")).pin_memory()
        lse = torch.full((q.shape[0], q.shape[1], q.shape[2]), float("nan"), dtype=torch.float32).pin_memory()
        outs.append((o, lse))
    torch.cuda.synchronize()
    free_before, _ = torch.cuda.mem_get_info()
    for (q, k, v, scale, causal, _), (o, lse) in zip(prepared, outs):
        api.attn_fwd_host_static(q, k, v, scale, causal, o, lse)
    assert api.attn_last_device_status() == 0     # synchronises the stream
    free_after, _ = torch.cuda.mem_get_info()
    # the driver's own count of free device memory: the two calls took none (this process is the GPU's only user)
    assert free_after == free_before

    for (q, k, v, scale, causal, (o_ref, lse_ref)), (o, lse) in zip(prepared, outs):
        tol = 1e-2 if q.dtype == torch.float16 else 2e-2
        assert not torch.isnan(o.float()).any() and not torch.isnan(lse).any()
        assert float((o.float() - o_ref.float()).abs().max()) <= tol
        assert float((lse - lse_ref).abs().max()) <= 1e-3
        # same kernel, same inputs: in fact the bytes are identical
        assert torch.equal(o.view(torch.int16), o_ref.view(torch.int16)) and torch.equal(lse, lse_ref)
        # and, like every other entry point, against the fp64 oracle itself
        dtype = inputs.DTYPE_FP16 if q.dtype == torch.float16 else inputs.DTYPE_BF16
        want_o, want_l = orc.attention(*(orc.widen(inputs.bits(t), dtype) for t in (q, k, v)), scale, causal)
        assert np.abs(o.double().numpy() - want_o).max() <= tol
        assert np.abs(lse.double().numpy() - want_l).max() <= 1e-3


@pytest.mark.gpu
def test_static_entry_refuses_problems_beyond_its_capacity():
    cap = api.attn_fwd_host_static_capacity()
    assert cap == 16 << 20
    B, H, S, D = 1, 8, 4096, 128      # 4 x 8 MiB of staging: does not fit
    assert api.attn_fwd_host_workspace_bytes(B, H, S, S, D) > cap
    q = torch.zeros(B, H, S, D, dtype=torch.float16)
    o = torch.zeros_like(q)
    lse = torch.zeros(B, H, S, dtype=torch.float32)
    with pytest.raises(api.AttnError) as err:
        api.attn_fwd_host_static(q, q, q, 0.1, False, o, lse)
    assert err.value.status == 11 and api.attn_status_string(11) == "ATTN_ERR_STATIC_CAPACITY"


def test_static_entry_validates_before_touching_a_device():
    # CPU-only part: argument checks and the capacity check come before any device call
    lib = api.load()
    args = [0x1000, 0x2000, 0x3000, 0x4000, 0x5000, 1, 8, 4096, 4096, 128, 0.1, 0, 0, None]
    assert lib.attn_fwd_host_static(*args) == 11
    bad = list(args)
    bad[9] = 96
    assert lib.attn_fwd_host_static(*bad) == 3
    bad = list(args)
    bad[0] = None
    assert lib.attn_fwd_host_static(*bad) == 1
    assert lib.attn_fwd_host_static_capacity() == 16 << 20
