"""ctypes front end of the fp64 CPU oracle (oracle/attn_oracle.c).

TEST INFRASTRUCTURE, not product code: only tests, the smoke check and the
benchmark's cpu_baseline / reference legs may import this module.  It imports
nothing from the CUDA package.

The arithmetic lives in the C file (Section 2.2 of the paper, written out as
the definition); this module only compiles it with gcc, loads it and passes
numpy arrays through.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "attn_oracle.c")
_LIB = os.path.join(_HERE, "liboracle.so")

DTYPE_FP16 = 0
DTYPE_BF16 = 1

_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (OpenMP) if the shared object is missing or stale."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp.%d" % os.getpid()
        subprocess.check_call(
            ["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-o", tmp, _SRC, "-lm"]
        )
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        dp = ctypes.POINTER(ctypes.c_double)
        u16p = ctypes.POINTER(ctypes.c_uint16)
        i64p = ctypes.POINTER(ctypes.c_int64)
        lib.attn_oracle_f64.restype = ctypes.c_int
        lib.attn_oracle_f64.argtypes = [dp, dp, dp, dp, dp, dp] + [ctypes.c_int] * 5 + [
            ctypes.c_double, ctypes.c_int]
        lib.attn_oracle_rows_16.restype = ctypes.c_int
        lib.attn_oracle_rows_16.argtypes = [u16p, u16p, u16p, ctypes.c_int, i64p, ctypes.c_int64,
                                            dp, dp] + [ctypes.c_int] * 5 + [ctypes.c_double,
                                                                            ctypes.c_int]
        lib.attn_oracle_gqa_f64.restype = ctypes.c_int
        lib.attn_oracle_gqa_f64.argtypes = [dp, dp, dp, dp, dp] + [ctypes.c_int] * 6 + [ctypes.c_double, ctypes.c_int]
        lib.attn_oracle_gqa_dv_f64.restype = ctypes.c_int
        lib.attn_oracle_gqa_dv_f64.argtypes = [dp, dp, dp, dp, dp] + [ctypes.c_int] * 7 + [ctypes.c_double, ctypes.c_int]
        lib.attn_oracle_shard_f64.restype = ctypes.c_int
        lib.attn_oracle_shard_f64.argtypes = [dp, dp, dp, dp, dp] + [ctypes.c_int] * 6 + [ctypes.c_double, ctypes.c_int, ctypes.c_int]
        lib.attn_oracle_combine_f64.restype = None
        lib.attn_oracle_combine_f64.argtypes = [dp, dp, ctypes.c_int, dp, dp, ctypes.c_int64, ctypes.c_int]
        lib.oracle_widen.restype = None
        lib.oracle_widen.argtypes = [u16p, dp, ctypes.c_int64, ctypes.c_int]
        u8p = ctypes.POINTER(ctypes.c_uint8)
        lib.oracle_widen_e4m3.argtypes = [u8p, dp, ctypes.c_int64, ctypes.c_double]
        lib.oracle_widen_e4m3.restype = None
        lib.oracle_e4m3_bits_to_f64.argtypes = [ctypes.c_uint8]
        lib.oracle_e4m3_bits_to_f64.restype = ctypes.c_double
        lib.attn_oracle_rows_e4m3.argtypes = [u8p, u8p, u8p, ctypes.c_double, ctypes.c_double, ctypes.c_double,
                                              i64p, ctypes.c_int64, dp, dp] + [ctypes.c_int] * 6 + [
                                                  ctypes.c_double, ctypes.c_int]
        lib.attn_oracle_rows_e4m3.restype = ctypes.c_int
        lib.attn_oracle_bwd_f64.restype = ctypes.c_int
        lib.attn_oracle_bwd_f64.argtypes = [dp] * 7 + [ctypes.c_int] * 6 + [ctypes.c_double, ctypes.c_int]
        lib.oracle_num_threads.restype = ctypes.c_int
        _lib = lib
    return _lib


def _dptr(a):
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_double))


def _u16ptr(a):
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_uint16))


def num_threads() -> int:
    return int(_load().oracle_num_threads())


def widen(bits: np.ndarray, dtype: int) -> np.ndarray:
    """Exact widening of fp16 (dtype 0) / bf16 (dtype 1) bit patterns (uint16) to float64."""
    bits = np.ascontiguousarray(bits, dtype=np.uint16)
    out = np.empty(bits.shape, dtype=np.float64)
    _load().oracle_widen(_u16ptr(bits), _dptr(out), bits.size, int(dtype))
    return out


def attention(q, k, v, scale: float, causal: bool, return_rowsum: bool = False):
    """O, LSE (and optionally the row sums of the probabilities) for float64 arrays.

    q: [B,H,Sq,D]; k, v: [B,H,Sk,D].  Returns o [B,H,Sq,D], lse [B,H,Sq].
    """
    q = np.ascontiguousarray(q, dtype=np.float64)
    k = np.ascontiguousarray(k, dtype=np.float64)
    v = np.ascontiguousarray(v, dtype=np.float64)
    B, H, Sq, D = q.shape
    Sk = k.shape[2]
    assert k.shape == (B, H, Sk, D) and v.shape == (B, H, Sk, D)
    o = np.empty((B, H, Sq, D), dtype=np.float64)
    lse = np.empty((B, H, Sq), dtype=np.float64)
    rs = np.empty((B, H, Sq), dtype=np.float64) if return_rowsum else None
    rc = _load().attn_oracle_f64(_dptr(q), _dptr(k), _dptr(v), _dptr(o), _dptr(lse),
                                 _dptr(rs) if rs is not None else None,
                                 B, H, Sq, Sk, D, float(scale), int(bool(causal)))
    if rc != 0:
        raise MemoryError("oracle scratch allocation failed")
    return (o, lse, rs) if return_rowsum else (o, lse)


def attention_gqa(q, k, v, scale: float, causal: bool):
    """Grouped-query attention for float64 arrays: q [B,H,Sq,D]; k, v [B,Hkv,Sk,D], H % Hkv == 0."""
    q = np.ascontiguousarray(q, dtype=np.float64)
    k = np.ascontiguousarray(k, dtype=np.float64)
    v = np.ascontiguousarray(v, dtype=np.float64)
    B, H, Sq, D = q.shape
    Hkv, Sk = k.shape[1], k.shape[2]
    assert k.shape == (B, Hkv, Sk, D) and v.shape == (B, Hkv, Sk, D)
    o = np.empty((B, H, Sq, D), dtype=np.float64)
    lse = np.empty((B, H, Sq), dtype=np.float64)
    rc = _load().attn_oracle_gqa_f64(_dptr(q), _dptr(k), _dptr(v), _dptr(o), _dptr(lse), B, H, Hkv, Sq, Sk, D,
                                     float(scale), int(bool(causal)))
    if rc == -2:
        raise ValueError("H must be a multiple of Hkv")
    if rc != 0:
        raise MemoryError("oracle scratch allocation failed")
    return o, lse


def attention_gqa_dv(q, k, v, scale: float, causal: bool):
    """Attention whose V (and O) head dim differs from the Q/K head dim: q [B,H,Sq,D]; k [B,Hkv,Sk,D];
    v [B,Hkv,Sk,Dv]; returns o [B,H,Sq,Dv], lse [B,H,Sq]."""
    q = np.ascontiguousarray(q, dtype=np.float64)
    k = np.ascontiguousarray(k, dtype=np.float64)
    v = np.ascontiguousarray(v, dtype=np.float64)
    B, H, Sq, D = q.shape
    Hkv, Sk, Dv = k.shape[1], k.shape[2], v.shape[3]
    assert k.shape == (B, Hkv, Sk, D) and v.shape == (B, Hkv, Sk, Dv)
    o = np.empty((B, H, Sq, Dv), dtype=np.float64)
    lse = np.empty((B, H, Sq), dtype=np.float64)
    rc = _load().attn_oracle_gqa_dv_f64(_dptr(q), _dptr(k), _dptr(v), _dptr(o), _dptr(lse), B, H, Hkv, Sq, Sk, D, Dv,
                                        float(scale), int(bool(causal)))
    if rc == -2:
        raise ValueError("H must be a multiple of Hkv")
    if rc != 0:
        raise MemoryError("oracle scratch allocation failed")
    return o, lse


def attention_shard(q, k, v, scale: float, causal: bool, k_offset: int):
    """One K/V shard whose first key has global index k_offset: q [B,H,Sq,D]; k, v [B,Hkv,Sk,D]."""
    q = np.ascontiguousarray(q, dtype=np.float64)
    k = np.ascontiguousarray(k, dtype=np.float64)
    v = np.ascontiguousarray(v, dtype=np.float64)
    B, H, Sq, D = q.shape
    Hkv, Sk = k.shape[1], k.shape[2]
    assert k.shape == (B, Hkv, Sk, D) and v.shape == (B, Hkv, Sk, D)
    o = np.empty((B, H, Sq, D), dtype=np.float64)
    lse = np.empty((B, H, Sq), dtype=np.float64)
    rc = _load().attn_oracle_shard_f64(_dptr(q), _dptr(k), _dptr(v), _dptr(o), _dptr(lse), B, H, Hkv, Sq, Sk, D,
                                       float(scale), int(bool(causal)), int(k_offset))
    if rc != 0:
        raise ValueError("bad head counts" if rc == -2 else "oracle scratch allocation failed")
    return o, lse


def combine(o_parts, lse_parts):
    """Merge of shard results: o_parts [n, ..., D], lse_parts [n, ...] -> o [..., D], lse [...]."""
    o_parts = np.ascontiguousarray(o_parts, dtype=np.float64)
    lse_parts = np.ascontiguousarray(lse_parts, dtype=np.float64)
    n, D = o_parts.shape[0], o_parts.shape[-1]
    rows = int(np.prod(lse_parts.shape[1:]))
    o = np.empty(o_parts.shape[1:], dtype=np.float64)
    lse = np.empty(lse_parts.shape[1:], dtype=np.float64)
    _load().attn_oracle_combine_f64(_dptr(o_parts), _dptr(lse_parts), n, _dptr(o), _dptr(lse), rows, D)
    return o, lse


def attention_bwd(q, k, v, dout, scale: float, causal: bool):
    """Gradients (dq, dk, dv) of the attention output with respect to q, k, v for the upstream gradient
    dout = dL/dO, by the chain rule on the definition.  q, dout: [B,H,Sq,D]; k, v: [B,Hkv,Sk,D] (float64)."""
    q = np.ascontiguousarray(q, dtype=np.float64)
    k = np.ascontiguousarray(k, dtype=np.float64)
    v = np.ascontiguousarray(v, dtype=np.float64)
    dout = np.ascontiguousarray(dout, dtype=np.float64)
    B, H, Sq, D = q.shape
    Hkv, Sk = k.shape[1], k.shape[2]
    assert k.shape == (B, Hkv, Sk, D) and v.shape == (B, Hkv, Sk, D) and dout.shape == q.shape
    dq, dk, dv = np.empty_like(q), np.empty_like(k), np.empty_like(v)
    rc = _load().attn_oracle_bwd_f64(_dptr(q), _dptr(k), _dptr(v), _dptr(dout), _dptr(dq), _dptr(dk), _dptr(dv),
                                     B, H, Hkv, Sq, Sk, D, float(scale), int(bool(causal)))
    if rc == -2:
        raise ValueError("H must be a multiple of Hkv")
    if rc != 0:
        raise MemoryError("oracle scratch allocation failed")
    return dq, dk, dv


def attention_rows_16(q_bits, k_bits, v_bits, dtype: int, rows, scale: float, causal: bool):
    """Oracle for a chosen subset of rows, straight from 16-bit inputs.

    q_bits: uint16 [B,H,Sq,D]; k_bits, v_bits: uint16 [B,H,Sk,D]; rows: flat
    row indices (b*H + h)*Sq + i.  Returns o [n,D] and lse [n] in float64.
    """
    q_bits = np.ascontiguousarray(q_bits, dtype=np.uint16)
    k_bits = np.ascontiguousarray(k_bits, dtype=np.uint16)
    v_bits = np.ascontiguousarray(v_bits, dtype=np.uint16)
    rows = np.ascontiguousarray(rows, dtype=np.int64)
    B, H, Sq, D = q_bits.shape
    Sk = k_bits.shape[2]
    assert k_bits.shape == (B, H, Sk, D) and v_bits.shape == (B, H, Sk, D)
    assert rows.size == 0 or (rows.min() >= 0 and rows.max() < B * H * Sq)
    assert np.all(np.diff(rows) >= 0), "rows must be in ascending order"
    o = np.empty((rows.size, D), dtype=np.float64)
    lse = np.empty((rows.size,), dtype=np.float64)
    rc = _load().attn_oracle_rows_16(
        _u16ptr(q_bits), _u16ptr(k_bits), _u16ptr(v_bits), int(dtype),
        rows.ctypes.data_as(ctypes.POINTER(ctypes.c_int64)), rows.size, _dptr(o), _dptr(lse),
        B, H, Sq, Sk, D, float(scale), int(bool(causal)))
    if rc != 0:
        raise MemoryError("oracle scratch allocation failed")
    return o, lse


def _u8ptr(a):
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_uint8))


def widen_e4m3(bits: np.ndarray, factor: float = 1.0) -> np.ndarray:
    """factor * value of E4M3 bit patterns (uint8), exactly, as float64: the dequantised tensor."""
    bits = np.ascontiguousarray(bits, dtype=np.uint8)
    out = np.empty(bits.shape, dtype=np.float64)
    _load().oracle_widen_e4m3(_u8ptr(bits), _dptr(out), bits.size, float(factor))
    return out


def attention_fp8(q_bits, k_bits, v_bits, q_f: float, k_f: float, v_f: float, scale: float, causal: bool):
    """FP8 attention by the definition on the dequantised tensors: q_bits uint8 [B,H,Sq,D];
    k_bits, v_bits uint8 [B,Hkv,Sk,D]; one dequantisation factor per tensor.  Returns o, lse (float64)."""
    return attention_gqa(widen_e4m3(q_bits, q_f), widen_e4m3(k_bits, k_f), widen_e4m3(v_bits, v_f), scale, causal)


def attention_rows_fp8(q_bits, k_bits, v_bits, q_f: float, k_f: float, v_f: float, rows, scale: float, causal: bool):
    """Row subset of `attention_fp8` straight from the 8-bit inputs (rows: ascending flat indices
    (b*H + h)*Sq + i).  Returns o [n,D] and lse [n] in float64."""
    q_bits = np.ascontiguousarray(q_bits, dtype=np.uint8)
    k_bits = np.ascontiguousarray(k_bits, dtype=np.uint8)
    v_bits = np.ascontiguousarray(v_bits, dtype=np.uint8)
    rows = np.ascontiguousarray(rows, dtype=np.int64)
    B, H, Sq, D = q_bits.shape
    Hkv, Sk = k_bits.shape[1], k_bits.shape[2]
    assert k_bits.shape == (B, Hkv, Sk, D) and v_bits.shape == (B, Hkv, Sk, D)
    assert rows.size == 0 or (rows.min() >= 0 and rows.max() < B * H * Sq)
    assert np.all(np.diff(rows) >= 0), "rows must be in ascending order"
    o = np.empty((rows.size, D), dtype=np.float64)
    lse = np.empty((rows.size,), dtype=np.float64)
    rc = _load().attn_oracle_rows_e4m3(
        _u8ptr(q_bits), _u8ptr(k_bits), _u8ptr(v_bits), float(q_f), float(k_f), float(v_f),
        rows.ctypes.data_as(ctypes.POINTER(ctypes.c_int64)), rows.size, _dptr(o), _dptr(lse),
        B, H, Hkv, Sq, Sk, D, float(scale), int(bool(causal)))
    if rc == -2:
        raise ValueError("H must be a multiple of Hkv")
    if rc != 0:
        raise MemoryError("oracle scratch allocation failed")
    return o, lse
