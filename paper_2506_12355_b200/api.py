"""Python binding of the C ABI in include/attn_fwd.h.

Argument marshalling only: every step of the attention forward pass runs in the
CUDA kernels of libattn_fwd.so.  PyTorch supplies device memory and streams.
There is no fallback: if the library is missing the import of a symbol fails.
"""
from __future__ import annotations

import ctypes
import os

import torch

from . import build as _build

DTYPE_FP16 = 0
DTYPE_BF16 = 1

STATUS_NAMES = {
    0: "ATTN_OK", 1: "ATTN_ERR_NULL_POINTER", 2: "ATTN_ERR_BAD_SHAPE",
    3: "ATTN_ERR_UNSUPPORTED_HEAD_DIM", 4: "ATTN_ERR_UNSUPPORTED_DTYPE", 5: "ATTN_ERR_MISALIGNED",
    6: "ATTN_ERR_BAD_SCALE", 7: "ATTN_ERR_UNSUPPORTED_ARCH", 8: "ATTN_ERR_CUDA",
    9: "ATTN_ERR_DEVICE_TIMEOUT", 10: "ATTN_ERR_WORKSPACE", 11: "ATTN_ERR_STATIC_CAPACITY",
    12: "ATTN_ERR_COUNTER_SLOTS",
}

# every symbol include/attn_fwd.h declares
EXPORTS = ["attn_bwd", "attn_bwd_workspace_bytes", "attn_fwd", "attn_fwd_gqa", "attn_fwd_partial", "attn_combine", "attn_combine_gather", "attn_fwd_qkv_dims", "attn_fwd_splitkv", "attn_fwd_splitkv_workspace_bytes", "attn_fwd_fp8", "attn_fwd_simt", "attn_fwd_host", "attn_fwd_host_workspace_bytes",
           "attn_fwd_host_static", "attn_fwd_host_static_capacity",
           "attn_query_support", "attn_last_device_status", "attn_status_string"]

_lib = None


class AttnError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__("%s failed: %s (%d)" % (where, STATUS_NAMES.get(status, "?"), status))


def lib_path() -> str:
    return _build.LIB_PATH


def load() -> ctypes.CDLL:
    """Loads libattn_fwd.so (built in-tree).  Raises if it does not exist: there is no fallback."""
    global _lib
    if _lib is not None:
        return _lib
    path = lib_path()
    if not os.path.exists(path):
        raise ImportError("libattn_fwd.so is not built; run `python -m paper_2506_12355_b200.build` "
                          "or __graft_entry__.build()")
    lib = ctypes.CDLL(path)
    vp, i, f = ctypes.c_void_p, ctypes.c_int, ctypes.c_float
    sig = [vp, vp, vp, vp, vp, i, i, i, i, i, f, i, i, vp]
    lib.attn_fwd.restype = i
    lib.attn_fwd.argtypes = sig
    lib.attn_fwd_gqa.restype = i
    lib.attn_fwd_gqa.argtypes = [vp, vp, vp, vp, vp, i, i, i, i, i, i, f, i, i, vp]
    lib.attn_fwd_partial.restype = i
    lib.attn_fwd_partial.argtypes = [vp, vp, vp, vp, vp, i, i, i, i, i, i, f, i, i, i, vp]
    lib.attn_combine.restype = i
    lib.attn_combine.argtypes = [vp, vp, i, vp, vp, i, i, i, i, i, vp]
    lib.attn_combine_gather.restype = i
    lib.attn_combine_gather.argtypes = [vp, vp, i, vp, vp, i, i, i, i, i, ctypes.c_longlong, ctypes.c_longlong, vp]
    lib.attn_fwd_qkv_dims.restype = i
    lib.attn_fwd_qkv_dims.argtypes = [vp, vp, vp, vp, vp, i, i, i, i, i, i, i, f, i, i, vp]
    lib.attn_fwd_splitkv.restype = i
    lib.attn_fwd_splitkv.argtypes = [vp, vp, vp, vp, vp, i, i, i, i, i, i, f, i, i, i, vp, ctypes.c_size_t, vp]
    lib.attn_fwd_splitkv_workspace_bytes.restype = ctypes.c_size_t
    lib.attn_fwd_splitkv_workspace_bytes.argtypes = [i] * 5
    lib.attn_fwd_fp8.restype = i
    lib.attn_fwd_fp8.argtypes = [vp, vp, vp, vp, vp, i, i, i, i, i, i, f, f, f, f, i, i, vp]
    lib.attn_bwd.restype = i
    lib.attn_bwd.argtypes = [vp] * 9 + [i] * 6 + [f, i, i, vp, ctypes.c_size_t, vp]
    lib.attn_bwd_workspace_bytes.restype = ctypes.c_size_t
    lib.attn_bwd_workspace_bytes.argtypes = [i] * 3
    lib.attn_fwd_simt.restype = i
    lib.attn_fwd_simt.argtypes = sig
    lib.attn_fwd_host.restype = i
    lib.attn_fwd_host.argtypes = sig[:-1] + [vp, ctypes.c_size_t, vp]
    lib.attn_fwd_host_workspace_bytes.restype = ctypes.c_size_t
    lib.attn_fwd_host_workspace_bytes.argtypes = [i] * 5
    lib.attn_fwd_host_static.restype = i
    lib.attn_fwd_host_static.argtypes = sig
    lib.attn_fwd_host_static_capacity.restype = ctypes.c_size_t
    lib.attn_fwd_host_static_capacity.argtypes = []
    lib.attn_query_support.restype = i
    lib.attn_query_support.argtypes = [i, i, i]
    lib.attn_last_device_status.restype = i
    lib.attn_last_device_status.argtypes = [vp]
    lib.attn_status_string.restype = ctypes.c_char_p
    lib.attn_status_string.argtypes = [i]
    _lib = lib
    return lib


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float16:
        return DTYPE_FP16
    if t.dtype == torch.bfloat16:
        return DTYPE_BF16
    raise TypeError("q/k/v must be float16 or bfloat16, got %s" % t.dtype)


def _stream_ptr(stream) -> int:
    if stream is None:
        stream = torch.cuda.current_stream()
    return int(stream.cuda_stream)


def _check_qkv(q, k, v):
    if q.dim() != 4 or k.dim() != 4 or v.dim() != 4:
        raise ValueError("q, k, v must be [B,H,S,D]")
    B, H, Sq, D = q.shape
    Sk = k.shape[2]
    if tuple(k.shape) != (B, H, Sk, D) or tuple(v.shape) != (B, H, Sk, D):
        raise ValueError("k, v must be [B,H,Sk,D] matching q's B, H, D")
    if not (q.is_contiguous() and k.is_contiguous() and v.is_contiguous()):
        raise ValueError("q, k, v must be contiguous")
    if not (q.dtype == k.dtype == v.dtype):
        raise TypeError("q, k, v must share one dtype")
    return B, H, Sq, Sk, D


def _check_grouped(q, k, v, same_v_dim=True):
    """The shared checks of the device entry points with grouped K/V heads: q [B,H,Sq,D], k [B,Hkv,Sk,D],
    v [B,Hkv,Sk,Dv] (Dv == D unless same_v_dim is False), contiguous CUDA tensors of one dtype.
    Returns (B, H, Hkv, Sq, Sk, D, Dv)."""
    if q.dim() != 4 or k.dim() != 4 or v.dim() != 4:
        raise ValueError("q must be [B,H,Sq,D]; k, v must be [B,Hkv,Sk,D]")
    B, H, Sq, D = q.shape
    Hkv, Sk, Dv = k.shape[1], k.shape[2], v.shape[3]
    if tuple(k.shape) != (B, Hkv, Sk, D) or tuple(v.shape) != (B, Hkv, Sk, Dv) or (same_v_dim and Dv != D):
        raise ValueError("k must be [B,Hkv,Sk,D] and v [B,Hkv,Sk,%s] matching q's B and D" % ("D" if same_v_dim else "Dv"))
    if not (q.is_contiguous() and k.is_contiguous() and v.is_contiguous()):
        raise ValueError("q, k, v must be contiguous")
    if not (q.is_cuda and k.is_cuda and v.is_cuda) or not (q.dtype == k.dtype == v.dtype):
        raise ValueError("q, k, v must be CUDA tensors of one dtype")
    return B, H, Hkv, Sq, Sk, D, Dv


def _outputs(q, B, H, Sq, Dv, out, lse, dtype=None):
    """O [B,H,Sq,Dv] and LSE [B,H,Sq] (fp32), allocated on q's device when not given."""
    if out is None:
        out = torch.empty((B, H, Sq, Dv), dtype=q.dtype if dtype is None else dtype, device=q.device)
    if lse is None:
        lse = torch.empty((B, H, Sq), dtype=torch.float32, device=q.device)
    return out, lse


def _call_device(fn_name, q, k, v, scale, causal, out, lse, stream):
    B, H, Sq, Sk, D = _check_qkv(q, k, v)
    if not (q.is_cuda and k.is_cuda and v.is_cuda):
        raise ValueError("q, k, v must be CUDA tensors")
    dt = _dtype_code(q)
    out, lse = _outputs(q, B, H, Sq, D, out, lse)
    with torch.cuda.device(q.device):
        rc = getattr(load(), fn_name)(q.data_ptr(), k.data_ptr(), v.data_ptr(), out.data_ptr(),
                                      lse.data_ptr(), B, H, Sq, Sk, D, float(scale),
                                      int(bool(causal)), dt, _stream_ptr(stream))
    if rc != 0:
        raise AttnError(rc, fn_name)
    return out, lse


def attn_fwd(q, k, v, scale: float, causal: bool = False, out=None, lse=None, stream=None):
    """O [B,H,Sq,D] (dtype of q) and LSE [B,H,Sq] (fp32) on the tensor-core kernel.

    Enqueues on `stream` (default: torch's current stream) and returns without synchronising.
    """
    return _call_device("attn_fwd", q, k, v, scale, causal, out, lse, stream)


def attn_fwd_gqa(q, k, v, scale: float, causal: bool = False, out=None, lse=None, stream=None):
    """Grouped-query / multi-query attention: q [B,H,Sq,D], k, v [B,Hkv,Sk,D] with H % Hkv == 0."""
    B, H, Hkv, Sq, Sk, D, _ = _check_grouped(q, k, v)
    dt = _dtype_code(q)
    out, lse = _outputs(q, B, H, Sq, D, out, lse)
    with torch.cuda.device(q.device):
        rc = load().attn_fwd_gqa(q.data_ptr(), k.data_ptr(), v.data_ptr(), out.data_ptr(), lse.data_ptr(),
                                 B, H, Hkv, Sq, Sk, D, float(scale), int(bool(causal)), dt, _stream_ptr(stream))
    if rc != 0:
        raise AttnError(rc, "attn_fwd_gqa")
    return out, lse


def attn_fwd_partial(q, k, v, scale: float, causal: bool, k_offset: int, out=None, lse=None, stream=None):
    """Attention over one K/V shard whose first key has global index k_offset: q [B,H,Sq,D],
    k, v [B,Hkv,Sk_shard,D].  Returns the shard's normalised O_r and LSE_r (merge with attn_combine)."""
    B, H, Hkv, Sq, Sk, D, _ = _check_grouped(q, k, v)
    dt = _dtype_code(q)
    out, lse = _outputs(q, B, H, Sq, D, out, lse)
    with torch.cuda.device(q.device):
        rc = load().attn_fwd_partial(q.data_ptr(), k.data_ptr(), v.data_ptr(), out.data_ptr(), lse.data_ptr(),
                                     B, H, Hkv, Sq, Sk, D, float(scale), int(bool(causal)), int(k_offset), dt,
                                     _stream_ptr(stream))
    if rc != 0:
        raise AttnError(rc, "attn_fwd_partial")
    return out, lse


def attn_combine(o_parts, lse_parts, out=None, lse=None, stream=None):
    """Merges partial results: o_parts [n,B,H,Sq,D] (16-bit), lse_parts [n,B,H,Sq] (fp32)."""
    n, B, H, Sq, D = o_parts.shape
    if tuple(lse_parts.shape) != (n, B, H, Sq) or lse_parts.dtype != torch.float32:
        raise ValueError("lse_parts must be fp32 [n,B,H,Sq]")
    if not (o_parts.is_contiguous() and lse_parts.is_contiguous() and o_parts.is_cuda and lse_parts.is_cuda):
        raise ValueError("o_parts, lse_parts must be contiguous CUDA tensors")
    dt = _dtype_code(o_parts)
    if out is None:
        out = torch.empty((B, H, Sq, D), dtype=o_parts.dtype, device=o_parts.device)
    if lse is None:
        lse = torch.empty((B, H, Sq), dtype=torch.float32, device=o_parts.device)
    with torch.cuda.device(o_parts.device):
        rc = load().attn_combine(o_parts.data_ptr(), lse_parts.data_ptr(), n, out.data_ptr(), lse.data_ptr(),
                                 B, H, Sq, D, dt, _stream_ptr(stream))
    if rc != 0:
        raise AttnError(rc, "attn_combine")
    return out, lse


def attn_combine_gather(o_part_ptrs, lse_part_ptrs, shape, dtype, out, lse, row_begin=0, row_count=None, stream=None):
    """Merge of partial results that lie behind separate device pointers (possibly peer GPUs' memory), for the
    rows [row_begin, row_begin + row_count) of the flattened (batch, head, query) axis.  o_part_ptrs, lse_part_ptrs:
    lists of integer device addresses; shape: (B, H, Sq, D); dtype: torch.float16 / torch.bfloat16; out, lse: full-size
    CUDA tensors of which only those rows are written."""
    B, H, Sq, D = shape
    n = len(o_part_ptrs)
    if n != len(lse_part_ptrs):
        raise ValueError("as many O pointers as LSE pointers")
    rows = B * H * Sq
    if row_count is None:
        row_count = rows - row_begin
    o_arr = (ctypes.c_void_p * max(n, 1))(*[int(p) for p in o_part_ptrs])
    l_arr = (ctypes.c_void_p * max(n, 1))(*[int(p) for p in lse_part_ptrs])
    dt = DTYPE_FP16 if dtype == torch.float16 else DTYPE_BF16
    with torch.cuda.device(out.device):
        rc = load().attn_combine_gather(o_arr, l_arr, n, out.data_ptr(), lse.data_ptr(), B, H, Sq, D, dt,
                                        int(row_begin), int(row_count), _stream_ptr(stream))
    if rc != 0:
        raise AttnError(rc, "attn_combine_gather")
    return out, lse


def attn_fwd_qkv_dims(q, k, v, scale: float, causal: bool = False, out=None, lse=None, stream=None):
    """Attention with separate Q/K and V head dims (the 192/128 MLA head shape): q [B,H,Sq,Dqk],
    k [B,Hkv,Sk,Dqk], v [B,Hkv,Sk,Dv]; returns o [B,H,Sq,Dv] and lse [B,H,Sq]."""
    B, H, Hkv, Sq, Sk, Dqk, Dv = _check_grouped(q, k, v, same_v_dim=False)
    dt = _dtype_code(q)
    out, lse = _outputs(q, B, H, Sq, Dv, out, lse)
    with torch.cuda.device(q.device):
        rc = load().attn_fwd_qkv_dims(q.data_ptr(), k.data_ptr(), v.data_ptr(), out.data_ptr(), lse.data_ptr(),
                                      B, H, Hkv, Sq, Sk, Dqk, Dv, float(scale), int(bool(causal)), dt,
                                      _stream_ptr(stream))
    if rc != 0:
        raise AttnError(rc, "attn_fwd_qkv_dims")
    return out, lse


def attn_fwd_splitkv_workspace_bytes(B, H, Sq, D, n_splits) -> int:
    return int(load().attn_fwd_splitkv_workspace_bytes(B, H, Sq, D, n_splits))


def attn_fwd_splitkv(q, k, v, scale: float, causal: bool, n_splits: int, workspace=None, out=None, lse=None, stream=None):
    """attn_fwd_gqa with the keys split into n_splits ranges that run concurrently, then merged (split-KV
    decoding).  `workspace`: CUDA uint8 tensor of at least attn_fwd_splitkv_workspace_bytes(...) bytes
    (allocated here when None)."""
    B, H, Hkv, Sq, Sk, D, _ = _check_grouped(q, k, v)
    dt = _dtype_code(q)
    if workspace is None:
        workspace = torch.empty(attn_fwd_splitkv_workspace_bytes(B, H, Sq, D, n_splits), dtype=torch.uint8, device=q.device)
    out, lse = _outputs(q, B, H, Sq, D, out, lse)
    with torch.cuda.device(q.device):
        rc = load().attn_fwd_splitkv(q.data_ptr(), k.data_ptr(), v.data_ptr(), out.data_ptr(), lse.data_ptr(),
                                     B, H, Hkv, Sq, Sk, D, float(scale), int(bool(causal)), dt, int(n_splits),
                                     workspace.data_ptr(), workspace.numel(), _stream_ptr(stream))
    if rc != 0:
        raise AttnError(rc, "attn_fwd_splitkv")
    return out, lse


def attn_fwd_fp8(q, k, v, scale: float, q_factor: float = 1.0, k_factor: float = 1.0, v_factor: float = 1.0,
                 causal: bool = False, out=None, lse=None, stream=None, impl: int = 0):
    """Attention on E4M3 inputs with one dequantisation factor per tensor: q [B,H,Sq,128],
    k, v [B,Hkv,Sk,128] as CUDA uint8 (or torch.float8_e4m3fn) tensors; returns o (bf16) and lse (fp32).
    impl 0: tensor-core kernel; impl 1: CUDA-core cross-check kernel."""
    if q.dim() != 4 or k.dim() != 4 or v.dim() != 4:
        raise ValueError("q, k, v must be [B,H,S,D]")
    for t in (q, k, v):
        if t.dtype not in (torch.uint8, torch.float8_e4m3fn) or not t.is_cuda or not t.is_contiguous():
            raise ValueError("q, k, v must be contiguous CUDA tensors of E4M3 bytes")
    B, H, Sq, D = q.shape
    Hkv, Sk = k.shape[1], k.shape[2]
    if tuple(k.shape) != (B, Hkv, Sk, D) or tuple(v.shape) != (B, Hkv, Sk, D):
        raise ValueError("k, v must be [B,Hkv,Sk,D] matching q's B and D")
    if out is None:
        out = torch.empty((B, H, Sq, D), dtype=torch.bfloat16, device=q.device)
    if lse is None:
        lse = torch.empty((B, H, Sq), dtype=torch.float32, device=q.device)
    with torch.cuda.device(q.device):
        rc = load().attn_fwd_fp8(q.data_ptr(), k.data_ptr(), v.data_ptr(), out.data_ptr(), lse.data_ptr(),
                                 B, H, Hkv, Sq, Sk, D, float(scale), float(q_factor), float(k_factor),
                                 float(v_factor), int(bool(causal)), int(impl), _stream_ptr(stream))
    if rc != 0:
        raise AttnError(rc, "attn_fwd_fp8")
    return out, lse


def attn_bwd_workspace_bytes(B, H, Sq) -> int:
    return int(load().attn_bwd_workspace_bytes(B, H, Sq))


def attn_bwd(q, k, v, o, lse, dout, scale: float, causal: bool = False, dq=None, dk=None, dv=None, workspace=None,
             stream=None):
    """Gradients (dq, dk, dv) of the attention output for the upstream gradient dout: q, o, dout [B,H,Sq,D];
    k, v [B,Hkv,Sk,D]; lse [B,H,Sq] fp32; o and lse from the forward call on the same inputs.  D in {64, 128}.
    `workspace`: CUDA uint8 tensor of at least attn_bwd_workspace_bytes(B, H, Sq) bytes (allocated here when None)."""
    B, H, Hkv, Sq, Sk, D, _ = _check_grouped(q, k, v)
    if tuple(o.shape) != tuple(q.shape) or tuple(dout.shape) != tuple(q.shape):
        raise ValueError("o and dout must have q's shape")
    if tuple(lse.shape) != (B, H, Sq) or lse.dtype != torch.float32:
        raise ValueError("lse must be fp32 [B,H,Sq]")
    for t in (o, dout, lse):
        if not (t.is_cuda and t.is_contiguous()):
            raise ValueError("o, dout, lse must be contiguous CUDA tensors")
    if not (q.dtype == o.dtype == dout.dtype):
        raise TypeError("q, k, v, o, dout must share one dtype")
    dt = _dtype_code(q)
    dq = torch.empty_like(q) if dq is None else dq
    dk = torch.empty_like(k) if dk is None else dk
    dv = torch.empty_like(v) if dv is None else dv
    if workspace is None:
        workspace = torch.empty(max(attn_bwd_workspace_bytes(B, H, Sq), 256), dtype=torch.uint8, device=q.device)
    with torch.cuda.device(q.device):
        rc = load().attn_bwd(q.data_ptr(), k.data_ptr(), v.data_ptr(), o.data_ptr(), lse.data_ptr(), dout.data_ptr(),
                             dq.data_ptr(), dk.data_ptr(), dv.data_ptr(), B, H, Hkv, Sq, Sk, D, float(scale),
                             int(bool(causal)), dt, workspace.data_ptr(), workspace.numel(), _stream_ptr(stream))
    if rc != 0:
        raise AttnError(rc, "attn_bwd")
    return dq, dk, dv


def attn_fwd_simt(q, k, v, scale: float, causal: bool = False, out=None, lse=None, stream=None):
    """Same operator on the slow CUDA-core cross-check kernel."""
    return _call_device("attn_fwd_simt", q, k, v, scale, causal, out, lse, stream)


def attn_fwd_host_workspace_bytes(B, H, Sq, Sk, D) -> int:
    return int(load().attn_fwd_host_workspace_bytes(B, H, Sq, Sk, D))


def attn_fwd_host(q, k, v, scale: float, causal: bool, out, lse, workspace, stream=None):
    """attn_fwd for HOST tensors (pinned for asynchronous copies); `workspace` is a CUDA uint8
    tensor of at least attn_fwd_host_workspace_bytes(...) bytes.  Results are valid after the
    stream has been synchronised."""
    B, H, Sq, Sk, D = _check_qkv(q, k, v)
    dt = _dtype_code(q)
    with torch.cuda.device(workspace.device):
        rc = load().attn_fwd_host(q.data_ptr(), k.data_ptr(), v.data_ptr(), out.data_ptr(),
                                  lse.data_ptr(), B, H, Sq, Sk, D, float(scale), int(bool(causal)),
                                  dt, workspace.data_ptr(), workspace.numel() * workspace.element_size(),
                                  _stream_ptr(stream))
    if rc != 0:
        raise AttnError(rc, "attn_fwd_host")
    return out, lse


def attn_fwd_host_static_capacity() -> int:
    return int(load().attn_fwd_host_static_capacity())


def attn_fwd_host_static(q, k, v, scale: float, causal: bool, out, lse, stream=None, device=None):
    """attn_fwd_host for callers that cannot allocate device memory: Q, K, V, O and LSE are staged in
    the 16 MiB buffer built into the library image, so no workspace is passed and nothing is
    allocated.  Host tensors in, host tensors out; valid after the stream has been synchronised.
    Problems that need more staging than attn_fwd_host_static_capacity() raise
    AttnError(ATTN_ERR_STATIC_CAPACITY).  All calls on a device share the one buffer: keep them on
    one stream (overlapping calls race).  The first call on a device resolves the buffer's address
    and should come before any stream capture."""
    B, H, Sq, Sk, D = _check_qkv(q, k, v)
    dt = _dtype_code(q)
    dev = torch.device("cuda", torch.cuda.current_device()) if device is None else torch.device(device)
    with torch.cuda.device(dev):
        rc = load().attn_fwd_host_static(q.data_ptr(), k.data_ptr(), v.data_ptr(), out.data_ptr(),
                                         lse.data_ptr(), B, H, Sq, Sk, D, float(scale),
                                         int(bool(causal)), dt, _stream_ptr(stream))
    if rc != 0:
        raise AttnError(rc, "attn_fwd_host_static")
    return out, lse


def attn_query_support(D: int, dtype: int, causal: bool) -> int:
    return int(load().attn_query_support(int(D), int(dtype), int(bool(causal))))


def attn_last_device_status(stream=None) -> int:
    return int(load().attn_last_device_status(_stream_ptr(stream)))


def attn_status_string(status: int) -> str:
    return load().attn_status_string(int(status)).decode()
