"""The bounded-wait path of the kernels, made to run out once in the permitted, non-faulting form.

Every on-chip wait of the kernels has a time limit; when one expires the CTA raises an abort flag, all its
warps fall through to the normal end of the kernel (tensor memory is freed, the work counter handed back) and
a status word reports ATTN_ERR_DEVICE_TIMEOUT.  Nothing traps, spins without bound or touches a bad address.
To reach that path this test uses a SEPARATE build of the same sources (libattn_fwd_waittest.so: waits limited
to 1 ms, plus one extra entry that makes the producer warp leave out a single K/V tile load of the next
launch), on a problem of one CTA.  The consumer of that tile waits 1 ms, gives up, and the kernel returns.
Checked: the status is reported exactly once, and a normal call right afterwards is bit-equal to the same call
before (no state of the aborted launch leaks into the next one).
"""
import ctypes

import pytest
import torch

from paper_2506_12355_b200 import build, inputs

pytestmark = pytest.mark.gpu

ATTN_ERR_DEVICE_TIMEOUT = 9


def _load():
    lib = ctypes.CDLL(build.build_wait_test())
    vp, i, f = ctypes.c_void_p, ctypes.c_int, ctypes.c_float
    lib.attn_fwd.restype = i
    lib.attn_fwd.argtypes = [vp, vp, vp, vp, vp, i, i, i, i, i, f, i, i, vp]
    lib.attn_last_device_status.restype = i
    lib.attn_last_device_status.argtypes = [vp]
    lib.attn_test_skip_kv_load.restype = None
    lib.attn_test_skip_kv_load.argtypes = [i]
    return lib


@pytest.mark.parametrize("D,Sq,Sk,causal,skip", [(128, 256, 512, False, 3), (64, 200, 640, False, 4)])
def test_a_wait_that_runs_out_returns_a_status_and_leaves_no_trace(D, Sq, Sk, causal, skip):
    lib = _load()
    dev = torch.device("cuda:0")
    torch.cuda.set_device(0)
    q, k, v = (t.to(dev) for t in inputs.make_qkv(1, 1, Sq, Sk, D, inputs.DTYPE_BF16, seed=4100 + D))
    stream = torch.cuda.current_stream().cuda_stream

    def call(o, lse):
        return lib.attn_fwd(q.data_ptr(), k.data_ptr(), v.data_ptr(), o.data_ptr(), lse.data_ptr(), 1, 1, Sq, Sk, D,
                            D ** -0.5, int(causal), inputs.DTYPE_BF16, stream)

    o_before, l_before = torch.empty_like(q), torch.empty(1, 1, Sq, dtype=torch.float32, device=dev)
    assert call(o_before, l_before) == 0
    assert lib.attn_last_device_status(stream) == 0

    # the producer leaves out ring group `skip` (group 0 is K_0, group i is V_{i-1} with K_i): its consumer gives up after 1 ms
    o_bad, l_bad = torch.empty_like(q), torch.empty_like(l_before)
    lib.attn_test_skip_kv_load(skip)
    assert call(o_bad, l_bad) == 0                                    # the launch itself succeeds
    assert lib.attn_last_device_status(stream) == ATTN_ERR_DEVICE_TIMEOUT   # synchronises; the kernel has returned
    assert lib.attn_last_device_status(stream) == 0                   # reported once, then cleared

    o_after, l_after = torch.empty_like(q), torch.empty_like(l_before)
    assert call(o_after, l_after) == 0
    assert lib.attn_last_device_status(stream) == 0
    assert torch.equal(o_after.view(torch.int16), o_before.view(torch.int16)) and torch.equal(l_after, l_before)
