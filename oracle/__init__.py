"""Test infrastructure: loader for the fp64 CPU oracle of paged GQA decode attention.

The oracle is the plain definition of softmax attention (two passes, fp64, no
tiling, no splits) read through a block table; see ``decode_attn_oracle.c`` for
the statement it follows.  Only the tests, the smoke check and the benchmark's
CPU-baseline leg may import this package.  It imports nothing from the CUDA
package and the CUDA package imports nothing from here.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "decode_attn_oracle.c")
_LIB = os.path.join(_HERE, "libdecode_attn_oracle.so")
_lock = threading.Lock()
_lib = None


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (OpenMP) into a shared library beside its source."""
    if (not force and os.path.exists(_LIB)
            and os.path.getmtime(_LIB) >= os.path.getmtime(_SRC)):
        return _LIB
    tmp = _LIB + f".tmp{os.getpid()}"
    cmd = ["gcc", "-O2", "-std=c11", "-fopenmp", "-fPIC", "-shared", "-Wall", "-Wextra",
           "-o", tmp, _SRC, "-lm"]
    subprocess.run(cmd, check=True)
    os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    with _lock:
        if _lib is None:
            lib = ctypes.CDLL(build())
            i64, i32, p = ctypes.c_int64, ctypes.c_int32, ctypes.c_void_p
            lib.decode_attn_oracle.restype = ctypes.c_int
            lib.decode_attn_oracle.argtypes = [
                p, i64, i64, i64,            # q, B, Hq, D
                p, p, i64, i64, i64,         # k_pages, v_pages, num_pages, Hkv, P
                i64, i64, i64,               # strides (elements): page, head, token
                p, i64, p,                   # block_table, max_pages, seq_lens
                i32, ctypes.c_double,        # window, scale
                p, p, i32,                   # out, lse, num_threads
            ]
            lib.kv_append_oracle.restype = ctypes.c_int
            lib.kv_append_oracle.argtypes = [p, p, i64, i64, i64, p, p, i64, i64, i64, i64, i64, p, i64, p]
            lib.decode_attn_oracle_max_threads.restype = ctypes.c_int
            lib.e4m3_bits_to_double.restype = ctypes.c_double
            lib.e4m3_bits_to_double.argtypes = [ctypes.c_uint8]
            lib.e4m3_nearest_code.restype = ctypes.c_uint8
            lib.e4m3_nearest_code.argtypes = [ctypes.c_double]
            lib.e4m3_quantize_oracle.restype = None
            lib.e4m3_quantize_oracle.argtypes = [p, i64, ctypes.c_float, p]
            lib.decode_attn_fp8kv_oracle.restype = ctypes.c_int
            lib.decode_attn_fp8kv_oracle.argtypes = [
                p, i64, i64, i64,            # q, B, Hq, D
                p, p, i64, i64, i64,         # k codes, v codes, num_pages, Hkv, P
                i64, i64, i64,               # strides (bytes): page, head, token
                p, p,                        # k_scale, v_scale (float [Hkv] or NULL)
                p, i64, p,                   # block_table, max_pages, seq_lens
                i32, ctypes.c_double,        # window, scale
                p, p, i32,                   # out, lse, num_threads
            ]
            lib.kv_append_fp8_oracle.restype = ctypes.c_int
            lib.kv_append_fp8_oracle.argtypes = [p, p, i64, i64, i64, p, p, i64, i64, i64, i64, i64, p, p, p, i64, p]
            _lib = lib
    return _lib


def _bf16_bits(x) -> np.ndarray:
    """View a bf16 tensor (torch CPU bfloat16, or numpy uint16 bit patterns) as uint16 bits."""
    if isinstance(x, np.ndarray):
        if x.dtype != np.uint16:
            raise TypeError("numpy inputs must hold bf16 bit patterns as uint16")
        return x
    import torch  # only to reinterpret a CPU bf16 tensor's storage

    if x.dtype != torch.bfloat16 or x.device.type != "cpu":
        raise TypeError("expected a CPU torch.bfloat16 tensor")
    return x.view(torch.int16).numpy().view(np.uint16)


def max_threads() -> int:
    return int(_load().decode_attn_oracle_max_threads())


def decode_attn_oracle(q, k_pages, v_pages, block_table, seq_lens, window: int, scale: float,
                       num_threads: int = 0):
    """fp64 decode attention over a paged KV cache.

    q            bf16 [B, Hq, D]
    k_pages      bf16 [num_pages, Hkv, P, D] in any strides with a contiguous last dim
    v_pages      same shape and strides as k_pages
    block_table  int32 [B, max_pages]
    seq_lens     int32 [B]
    window       <= 0 for full attention, else the number of most recent tokens attended
    scale        the float that multiplies q.k (taken at fp32 precision, as the C-ABI takes it)

    Returns (out float64 [B, Hq, D], lse float64 [B, Hq]).
    """
    lib = _load()
    qb = np.ascontiguousarray(_bf16_bits(q))
    kb, vb = _bf16_bits(k_pages), _bf16_bits(v_pages)
    if kb.shape != vb.shape or kb.strides != vb.strides:
        raise ValueError("k_pages and v_pages must share shape and strides")
    if kb.ndim != 4 or qb.ndim != 3:
        raise ValueError("q must be [B,Hq,D] and k_pages [num_pages,Hkv,P,D]")
    B, Hq, D = qb.shape
    num_pages, Hkv, P, Dk = kb.shape
    if Dk != D or kb.strides[3] != 2:
        raise ValueError("head_dim mismatch or non-contiguous last dim")
    bt = np.ascontiguousarray(np.asarray(block_table, dtype=np.int32))
    sl = np.ascontiguousarray(np.asarray(seq_lens, dtype=np.int32))
    if bt.ndim != 2 or bt.shape[0] != B or sl.shape != (B,):
        raise ValueError("block_table must be [B,max_pages] and seq_lens [B]")
    out = np.empty((B, Hq, D), dtype=np.float64)
    lse = np.empty((B, Hq), dtype=np.float64)
    st = [s // 2 for s in kb.strides]
    rc = lib.decode_attn_oracle(
        qb.ctypes.data, B, Hq, D,
        kb.ctypes.data, vb.ctypes.data, num_pages, Hkv, P,
        st[0], st[1], st[2],
        bt.ctypes.data, bt.shape[1], sl.ctypes.data,
        int(window), float(np.float32(scale)),
        out.ctypes.data, lse.ctypes.data, int(num_threads))
    if rc != 0:
        raise RuntimeError(f"decode_attn_oracle failed with code {rc}")
    return out, lse


def kv_append_oracle(k_new, v_new, k_pages, v_pages, block_table, seq_lens) -> None:
    """Write each sequence's new K/V rows (bf16 [B, Hkv, D]) into position seq_lens[b]-1 of the paged
    cache, IN PLACE in ``k_pages`` / ``v_pages`` (CPU torch bf16 tensors or uint16 arrays)."""
    lib = _load()
    kn = np.ascontiguousarray(_bf16_bits(k_new))
    vn = np.ascontiguousarray(_bf16_bits(v_new))
    kb, vb = _bf16_bits(k_pages), _bf16_bits(v_pages)
    if kb.shape != vb.shape or kb.strides != vb.strides or kb.ndim != 4 or kb.strides[3] != 2:
        raise ValueError("k_pages and v_pages must share shape and strides, contiguous last dim")
    B, Hkv, D = kn.shape
    num_pages, Hk, P, Dk = kb.shape
    if Hk != Hkv or Dk != D or vn.shape != kn.shape:
        raise ValueError("shape mismatch")
    bt = np.ascontiguousarray(np.asarray(block_table, dtype=np.int32))
    sl = np.ascontiguousarray(np.asarray(seq_lens, dtype=np.int32))
    st = [x // 2 for x in kb.strides]
    rc = lib.kv_append_oracle(kn.ctypes.data, vn.ctypes.data, B, Hkv, D, kb.ctypes.data, vb.ctypes.data,
                              num_pages, P, st[0], st[1], st[2], bt.ctypes.data, bt.shape[1], sl.ctypes.data)
    if rc != 0:
        raise RuntimeError(f"kv_append_oracle failed with code {rc}")


def extend_attn_oracle(q, k_pages, v_pages, block_table, seq_lens, scale: float, num_threads: int = 0):
    """Causal attention of Lq new tokens per sequence, by its definition in terms of the single-token
    oracle: query qi of sequence b sits at position L_b - Lq + qi, so it is decode attention over a
    cache cut to L_b - Lq + qi + 1 tokens.  q: bf16 [B, Lq, Hq, D]; ``seq_lens`` counts the new
    tokens.  Returns (out float64 [B, Lq, Hq, D], lse float64 [B, Lq, Hq])."""
    import torch
    B, Lq, Hq, D = q.shape
    sl = np.asarray(seq_lens, dtype=np.int64)
    out = np.zeros((B, Lq, Hq, D))
    lse = np.full((B, Lq, Hq), -np.inf)
    for qi in range(Lq):
        cut = np.where(sl > 0, sl - Lq + qi + 1, 0).astype(np.int32)
        o, l = decode_attn_oracle(q[:, qi].contiguous(), k_pages, v_pages, block_table, cut, 0, scale, num_threads)
        out[:, qi], lse[:, qi] = o, l
    return out, lse


# ----------------------------------------------------------------------------- 8-bit (E4M3) cache

def _u8_codes(x) -> np.ndarray:
    """View a cache of E4M3 codes (torch CPU uint8 / float8_e4m3fn, or numpy uint8) as uint8."""
    if isinstance(x, np.ndarray):
        if x.dtype != np.uint8:
            raise TypeError("numpy inputs must hold E4M3 codes as uint8")
        return x
    import torch  # only to reinterpret a CPU tensor's storage

    if x.device.type != "cpu":
        raise TypeError("expected a CPU tensor")
    if x.dtype == torch.float8_e4m3fn:
        x = x.view(torch.uint8)
    if x.dtype != torch.uint8:
        raise TypeError("expected uint8 or float8_e4m3fn codes")
    return x.numpy()


def _scales(x, Hkv):
    if x is None:
        return None
    a = np.ascontiguousarray(np.asarray(x, dtype=np.float32))
    if a.shape != (Hkv,):
        raise ValueError("a scale array must be [Hkv]")
    return a


def e4m3_value(code: int) -> float:
    """Value of one E4M3 code (NaN for 0x7F / 0xFF)."""
    return float(_load().e4m3_bits_to_double(int(code) & 0xFF))


def e4m3_nearest_code(x: float) -> int:
    """The E4M3 code nearest to x: ties to even, saturating at +-448, NaN -> 0x7F."""
    return int(_load().e4m3_nearest_code(float(x)))


def e4m3_quantize(x_bf16, scale: float) -> np.ndarray:
    """Codes of nearest_e4m3(x / scale) with the quotient taken in fp32; x: bf16 (any shape)."""
    xb = np.ascontiguousarray(_bf16_bits(x_bf16))
    out = np.empty(xb.shape, dtype=np.uint8)
    _load().e4m3_quantize_oracle(xb.ctypes.data, xb.size, float(np.float32(scale)), out.ctypes.data)
    return out


def decode_attn_fp8kv_oracle(q, k_pages, v_pages, k_scale, v_scale, block_table, seq_lens, window: int,
                             scale: float, num_threads: int = 0):
    """fp64 decode attention over a paged cache of E4M3 codes with per-KV-head fp32 factors.

    q                 bf16 [B, Hq, D]
    k_pages, v_pages  E4M3 codes [num_pages, Hkv, P, D], any strides with a contiguous last dim
    k_scale, v_scale  float32 [Hkv] or None (all 1): K = k_scale[g] * e4m3(code)
    other arguments and the result as decode_attn_oracle
    """
    lib = _load()
    qb = np.ascontiguousarray(_bf16_bits(q))
    kb, vb = _u8_codes(k_pages), _u8_codes(v_pages)
    if kb.shape != vb.shape or kb.strides != vb.strides or kb.ndim != 4 or qb.ndim != 3:
        raise ValueError("pools must share shape and strides; q must be [B,Hq,D]")
    B, Hq, D = qb.shape
    num_pages, Hkv, P, Dk = kb.shape
    if Dk != D or kb.strides[3] != 1:
        raise ValueError("head_dim mismatch or non-contiguous last dim")
    ks, vs = _scales(k_scale, Hkv), _scales(v_scale, Hkv)
    bt = np.ascontiguousarray(np.asarray(block_table, dtype=np.int32))
    sl = np.ascontiguousarray(np.asarray(seq_lens, dtype=np.int32))
    if bt.ndim != 2 or bt.shape[0] != B or sl.shape != (B,):
        raise ValueError("block_table must be [B,max_pages] and seq_lens [B]")
    out = np.empty((B, Hq, D), dtype=np.float64)
    lse = np.empty((B, Hq), dtype=np.float64)
    rc = lib.decode_attn_fp8kv_oracle(
        qb.ctypes.data, B, Hq, D, kb.ctypes.data, vb.ctypes.data, num_pages, Hkv, P,
        kb.strides[0], kb.strides[1], kb.strides[2],
        ks.ctypes.data if ks is not None else None, vs.ctypes.data if vs is not None else None,
        bt.ctypes.data, bt.shape[1], sl.ctypes.data, int(window), float(np.float32(scale)),
        out.ctypes.data, lse.ctypes.data, int(num_threads))
    if rc != 0:
        raise RuntimeError(f"decode_attn_fp8kv_oracle failed with code {rc}")
    return out, lse


def kv_append_fp8_oracle(k_new, v_new, k_pages, v_pages, k_scale, v_scale, block_table, seq_lens) -> None:
    """Quantise each sequence's new bf16 K/V rows [B, Hkv, D] per KV head and write the codes into
    position seq_lens[b]-1 of the 8-bit cache, IN PLACE."""
    lib = _load()
    kn = np.ascontiguousarray(_bf16_bits(k_new))
    vn = np.ascontiguousarray(_bf16_bits(v_new))
    kb, vb = _u8_codes(k_pages), _u8_codes(v_pages)
    if kb.shape != vb.shape or kb.strides != vb.strides or kb.ndim != 4 or kb.strides[3] != 1:
        raise ValueError("k_pages and v_pages must share shape and strides, contiguous last dim")
    B, Hkv, D = kn.shape
    num_pages, Hk, P, Dk = kb.shape
    if Hk != Hkv or Dk != D or vn.shape != kn.shape:
        raise ValueError("shape mismatch")
    ks, vs = _scales(k_scale, Hkv), _scales(v_scale, Hkv)
    bt = np.ascontiguousarray(np.asarray(block_table, dtype=np.int32))
    sl = np.ascontiguousarray(np.asarray(seq_lens, dtype=np.int32))
    rc = lib.kv_append_fp8_oracle(kn.ctypes.data, vn.ctypes.data, B, Hkv, D, kb.ctypes.data, vb.ctypes.data,
                                  num_pages, P, kb.strides[0], kb.strides[1], kb.strides[2],
                                  ks.ctypes.data if ks is not None else None,
                                  vs.ctypes.data if vs is not None else None,
                                  bt.ctypes.data, bt.shape[1], sl.ctypes.data)
    if rc != 0:
        raise RuntimeError(f"kv_append_fp8_oracle failed with code {rc}")


def extend_attn_fp8kv_oracle(q, k_pages, v_pages, k_scale, v_scale, block_table, seq_lens, scale: float,
                             num_threads: int = 0):
    """``extend_attn_oracle`` over the 8-bit cache: query qi of sequence b is single-token attention over a
    cache cut to L_b - Lq + qi + 1 tokens.  q: bf16 [B, Lq, Hq, D]."""
    B, Lq, Hq, D = q.shape
    sl = np.asarray(seq_lens, dtype=np.int64)
    out = np.zeros((B, Lq, Hq, D))
    lse = np.full((B, Lq, Hq), -np.inf)
    for qi in range(Lq):
        cut = np.where(sl > 0, sl - Lq + qi + 1, 0).astype(np.int32)
        o, l = decode_attn_fp8kv_oracle(q[:, qi].contiguous(), k_pages, v_pages, k_scale, v_scale, block_table, cut,
                                        0, scale, num_threads)
        out[:, qi], lse[:, qi] = o, l
    return out, lse
