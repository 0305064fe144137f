"""Host-side checks of the C ABI: the library loads, exports what the header declares, and
rejects bad arguments before touching a device (CPU only; nothing is launched)."""
import ctypes
import os
import re

import pytest

from paper_2506_12355_b200 import api, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "attn_fwd.h")


def no_device():
    """True on a box without a CUDA device.  Calls whose arguments pass validation carry FAKE pointers here, so
    they may only be made where the library stops at its device check; with a GPU present they would launch."""
    import torch
    return not torch.cuda.is_available()


@pytest.fixture(scope="module")
def lib():
    build.build()
    return api.load()


def declared_functions():
    text = open(HEADER).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(attn_[a-z_0-9]+)\s*\(", text)))


def test_header_declares_the_documented_entry_points():
    names = declared_functions()
    assert "attn_fwd" in names and "attn_status_string" in names
    assert sorted(api.EXPORTS) == names


def test_library_exports_every_declared_symbol(lib):
    for name in declared_functions():
        assert hasattr(lib, name), name


def test_status_strings(lib):
    for code, name in api.STATUS_NAMES.items():
        assert api.attn_status_string(code) == name
    assert api.attn_status_string(12345) == "ATTN_ERR_UNKNOWN"


GOOD = dict(q=0x1000, k=0x2000, v=0x3000, o=0x4000, lse=0x5000, B=1, H=1, Sq=128, Sk=128, D=64,
            scale=0.125, causal=0, dtype=0, stream=None)


def call(lib, fn="attn_fwd", **over):
    a = dict(GOOD)
    a.update(over)
    return getattr(lib, fn)(a["q"], a["k"], a["v"], a["o"], a["lse"], a["B"], a["H"], a["Sq"], a["Sk"],
                            a["D"], a["scale"], a["causal"], a["dtype"], a["stream"])


@pytest.mark.parametrize("fn", ["attn_fwd", "attn_fwd_simt"])
def test_argument_validation_happens_before_any_launch(lib, fn):
    # the pointers are fake: every call below must be refused by host-side validation
    for name in ("q", "k", "v", "o", "lse"):
        assert call(lib, fn, **{name: None}) == 1
    for name in ("B", "H", "Sq", "Sk"):
        assert call(lib, fn, **{name: -1}) == 2
    assert call(lib, fn, B=70000, H=70000) == 2
    for d in (0, 32, 96, 192, 512):
        assert call(lib, fn, D=d) == 3
    assert call(lib, fn, dtype=2) == 4
    assert call(lib, fn, dtype=-1) == 4
    for name in ("q", "k", "v", "o"):
        assert call(lib, fn, **{name: GOOD[name] + 8}) == 5
    assert call(lib, fn, lse=GOOD["lse"] + 2) == 5
    assert call(lib, fn, scale=float("nan")) == 6
    assert call(lib, fn, scale=float("inf")) == 6
    assert call(lib, fn, scale=-0.5) == 6
    # empty problems are a successful no-op, decided before the device is looked at
    assert call(lib, fn, B=0) == 0
    assert call(lib, fn, Sq=0) == 0
    assert call(lib, fn, Sq=0, q=None, o=None, lse=None) == 0
    # k, v may be NULL only when there are no keys (that case reaches the device check)
    if no_device():
        assert call(lib, fn, Sk=0, k=None, v=None) in (7, 8)


def test_fp8_entry_validation(lib):
    def f8(q=0x1000, k=0x2000, v=0x3000, o=0x4000, lse=0x5000, B=1, H=4, Hkv=2, Sq=128, Sk=128, D=128, scale=0.1,
           fq=1.0, fk=1.0, fv=1.0, causal=1, impl=0):
        return lib.attn_fwd_fp8(q, k, v, o, lse, B, H, Hkv, Sq, Sk, D, scale, fq, fk, fv, causal, impl, None)
    for name in ("q", "k", "v", "o", "lse"):
        assert f8(**{name: None}) == 1
    assert f8(B=-1) == 2 and f8(Sk=-3) == 2
    assert f8(H=4, Hkv=3) == 2
    for d in (64, 256, 96):
        assert f8(D=d) == 3                     # 8-bit inputs: head dim 128 only
    assert f8(q=0x1008) == 5
    for bad in (0.0, -1.0, float("nan"), float("inf")):
        assert f8(fq=bad) == 6 and f8(fk=bad) == 6 and f8(fv=bad) == 6
    assert f8(scale=float("nan")) == 6
    assert f8(scale=3e38, fq=10.0) == 6         # the effective scale must stay finite
    assert f8(impl=2) == 4
    assert f8(Sq=0) == 0
    if no_device():
        assert f8() in (7, 8)                   # valid arguments reach the device check


def test_bwd_entry_validation(lib):
    ws_bytes = lib.attn_bwd_workspace_bytes
    ws_bytes.restype = ctypes.c_size_t
    # two fp32 row vectors, rows padded to a multiple of 64 per head, each 256-byte aligned
    assert ws_bytes(2, 3, 100) == 2 * ((2 * 3 * 128 * 4 + 255) // 256 * 256)
    assert ws_bytes(1, 1, 64) == 2 * 256 and ws_bytes(-1, 1, 1) == 0

    def bwd(q=0x1000, k=0x2000, v=0x3000, o=0x4000, lse=0x5000, dout=0x6000, dq=0x7000, dk=0x8000, dv=0x9000, B=1, H=4,
            Hkv=2, Sq=128, Sk=256, D=128, scale=0.1, causal=1, dtype=1, ws=0x10000, ws_n=1 << 20):
        return lib.attn_bwd(q, k, v, o, lse, dout, dq, dk, dv, B, H, Hkv, Sq, Sk, D, scale, causal, dtype, ws, ws_n, None)
    for name in ("q", "k", "v", "o", "lse", "dout", "dq", "dk", "dv"):
        assert bwd(**{name: None}) == 1, name
    assert bwd(B=-1) == 2 and bwd(H=4, Hkv=3) == 2
    for d in (256, 96, 0):
        assert bwd(D=d) == 3                    # backward kernels: head dims 64 and 128
    assert bwd(dtype=2) == 4
    assert bwd(dout=0x6008) == 5 and bwd(dk=0x8004) == 5
    assert bwd(scale=float("nan")) == 6 and bwd(scale=-1.0) == 6
    assert bwd(ws=None) == 10 and bwd(ws=0x10010) == 10 and bwd(ws_n=100) == 10
    assert bwd(Sq=0, Sk=0) == 0                 # nothing to do
    if no_device():
        assert bwd() in (7, 8)                  # valid arguments reach the device check


def test_splitkv_entry_validation(lib):
    lib.attn_fwd_splitkv_workspace_bytes.restype = __import__("ctypes").c_size_t
    assert lib.attn_fwd_splitkv_workspace_bytes(1, 4, 3, 128, 6) == (6 * 12 * 128 * 2 + 255) // 256 * 256 + (6 * 12 * 4 + 255) // 256 * 256
    assert lib.attn_fwd_splitkv_workspace_bytes(1, 4, 3, 128, 0) == 0
    args = [0x1000, 0x2000, 0x3000, 0x4000, 0x5000, 1, 4, 2, 3, 4096, 128, 0.1, 0, 1]
    assert lib.attn_fwd_splitkv(*args, 0, 0x10000, 1 << 30, None) == 2      # n_splits out of range
    assert lib.attn_fwd_splitkv(*args, 65, 0x10000, 1 << 30, None) == 2
    assert lib.attn_fwd_splitkv(*args, 4, None, 0, None) == 10              # no workspace
    assert lib.attn_fwd_splitkv(*args, 4, 0x10010, 1 << 30, None) == 10     # misaligned
    bad = list(args)
    bad[7] = 3                                                              # H % Hkv != 0
    assert lib.attn_fwd_splitkv(*bad, 4, 0x10000, 1 << 30, None) == 2
    bad = list(args)
    bad[8] = 0                                                              # no query rows: nothing to do
    assert lib.attn_fwd_splitkv(*bad, 4, None, 0, None) == 0


def test_combine_gather_validation(lib):
    import ctypes
    def cg(o_ptrs, l_ptrs, n, o=0x4000, lse=0x5000, B=1, H=2, Sq=8, D=64, dtype=0, rb=0, rc=16):
        oa = (ctypes.c_void_p * max(len(o_ptrs), 1))(*o_ptrs)
        la = (ctypes.c_void_p * max(len(l_ptrs), 1))(*l_ptrs)
        return lib.attn_combine_gather(oa, la, n, o, lse, B, H, Sq, D, dtype, rb, rc, None)
    good_o, good_l = [0x1000, 0x2000], [0x3000, 0x3100]
    assert cg(good_o, good_l, 0) == 2 and cg(good_o, good_l, 33) == 2
    assert cg(good_o, good_l, 2, rb=10, rc=7) == 2 and cg(good_o, good_l, 2, rb=-1) == 2
    assert cg(good_o, good_l, 2, D=60) == 3 and cg(good_o, good_l, 2, dtype=2) == 4
    assert cg([0x1000, None], good_l, 2) == 1 and cg(good_o, good_l, 2, o=None) == 1
    assert cg([0x1000, 0x2008], good_l, 2) == 5 and cg(good_o, [0x3000, 0x3102], 2) == 5
    assert cg(good_o, good_l, 2, rc=0) == 0                     # an empty row range is a successful no-op
    if no_device():
        assert cg(good_o, good_l, 2) in (7, 8)                  # valid arguments reach the device check


def test_host_entry_validation(lib):
    n = lib.attn_fwd_host_workspace_bytes(2, 3, 100, 50, 64)
    qo = (2 * 3 * 100 * 64 * 2 + 255) // 256 * 256
    kv = (2 * 3 * 50 * 64 * 2 + 255) // 256 * 256
    ls = (2 * 3 * 100 * 4 + 255) // 256 * 256
    assert n == 2 * qo + 2 * kv + ls
    assert lib.attn_fwd_host_workspace_bytes(-1, 1, 1, 1, 64) == 0
    args = [0x1000, 0x2000, 0x3000, 0x4000, 0x5000, 2, 3, 100, 50, 64, 0.125, 0, 0]
    assert lib.attn_fwd_host(*args, None, 0, None) == 10            # no workspace
    assert lib.attn_fwd_host(*args, 0x10000, n - 1, None) == 10     # too small
    assert lib.attn_fwd_host(*args, 0x10010, n, None) == 10         # misaligned
    bad = list(args)
    bad[9] = 100
    assert lib.attn_fwd_host(*bad, 0x10000, n, None) == 3


def test_no_fallback_without_a_device(lib):
    if not no_device():
        pytest.skip("a device is present")
    # valid arguments but no B200: the library must report an error, not compute on the CPU
    assert call(lib) in (7, 8)
    assert api.attn_query_support(64, 0, False) in (7, 8)
    assert api.attn_query_support(96, 0, False) == 3
    assert api.attn_query_support(64, 5, False) == 4
