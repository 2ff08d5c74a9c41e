"""ctypes binding of include/decode_attn.h.  Argument marshalling only.

torch is used for device buffers and streams; nothing here computes.  The shared library is
loaded from this directory (built in-tree by ``build.py``); if it is missing, or a call is made
without a CUDA device, an exception is raised -- there is no fallback path.
"""
from __future__ import annotations

import ctypes
import os
import threading
from typing import Optional

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
# DECODE_ATTN_LIBRARY names another build of the same library (the timeline build); default: the in-tree one
_LIB_PATH = os.environ.get("DECODE_ATTN_LIBRARY") or os.path.join(_HERE, "libdecode_attn.so")
_lock = threading.Lock()
_lib = None
_workspaces = {}   # device index -> torch uint8 tensor kept alive while registered

DA_BF16, DA_F32, DA_I32, DA_FP8_E4M3 = 1, 2, 3, 4
# E4M3 codes may be handed over as torch.uint8 or torch.float8_e4m3fn storage
_DTYPES = {torch.bfloat16: DA_BF16, torch.float32: DA_F32, torch.int32: DA_I32,
           torch.uint8: DA_FP8_E4M3, torch.float8_e4m3fn: DA_FP8_E4M3}


class DecodeAttnError(RuntimeError):
    def __init__(self, status: int, what: str):
        super().__init__(f"decode_attn status {status}: {what}")
        self.status = status


class DaTensor(ctypes.Structure):
    _fields_ = [("data", ctypes.c_void_p), ("dtype", ctypes.c_int32), ("ndim", ctypes.c_int32),
                ("shape", ctypes.c_int64 * 4), ("stride", ctypes.c_int64 * 4)]


def use_library(path: str) -> None:
    """Load another build of the library (the timeline build) instead of the in-tree default.  Must be
    called before the first library call of the process."""
    global _LIB_PATH
    with _lock:
        if _lib is not None:
            raise RuntimeError("the library is already loaded")
        _LIB_PATH = os.path.abspath(path)


def lib() -> ctypes.CDLL:
    """The loaded C-ABI library (raises if it has not been built)."""
    global _lib
    with _lock:
        if _lib is None:
            if not os.path.exists(_LIB_PATH):
                raise FileNotFoundError(
                    f"{_LIB_PATH} is missing: build it with `python -m paper_2512_10977_b200.build`")
            L = ctypes.CDLL(_LIB_PATH)
            T = ctypes.POINTER(DaTensor)
            vp, i32, i64 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64
            L.decode_attn.restype = ctypes.c_int
            L.decode_attn.argtypes = [T, T, T, T, T, i32, ctypes.c_float, T, T, vp]
            L.decode_attn_fp8kv.restype = ctypes.c_int
            L.decode_attn_fp8kv.argtypes = [T, T, T, vp, vp, T, T, i32, ctypes.c_float, T, T, vp]
            L.decode_attn_append_fp8kv.restype = ctypes.c_int
            L.decode_attn_append_fp8kv.argtypes = [T, T, T, T, vp, vp, T, T, vp]
            L.decode_attn_cascade.restype = ctypes.c_int
            L.decode_attn_cascade.argtypes = [T, T, T, T, T, i32, ctypes.c_float, T, T, vp]
            L.decode_attn_fp8kv_cascade.restype = ctypes.c_int
            L.decode_attn_fp8kv_cascade.argtypes = [T, T, T, vp, vp, T, T, i32, ctypes.c_float, T, T, vp, ctypes.c_size_t, vp]
            L.decode_attn_fp8kv_cascade_scratch_bytes.restype = ctypes.c_size_t
            L.decode_attn_fp8kv_cascade_scratch_bytes.argtypes = [i32, i32, i32]
            L.decode_attn_append.restype = ctypes.c_int
            L.decode_attn_append.argtypes = [T, T, T, T, T, T, vp]
            L.decode_attn_extend.restype = ctypes.c_int
            L.decode_attn_extend.argtypes = [T, T, T, T, T, ctypes.c_float, T, T, vp]
            L.decode_attn_fp8kv_extend.restype = ctypes.c_int
            L.decode_attn_fp8kv_extend.argtypes = [T, T, T, vp, vp, T, T, ctypes.c_float, T, T, vp]
            L.decode_attn_fp8kv_extend_wide.restype = ctypes.c_int
            L.decode_attn_fp8kv_extend_wide.argtypes = [T, T, T, vp, vp, T, T, ctypes.c_float, T, T, vp, ctypes.c_size_t, vp]
            L.decode_attn_fp8kv_extend_wide_scratch_bytes.restype = ctypes.c_size_t
            L.decode_attn_fp8kv_extend_wide_scratch_bytes.argtypes = [i32, i64, i32, i32]
            L.decode_attn_host_io.restype = ctypes.c_int
            L.decode_attn_host_io.argtypes = [T, T, T, T, T, i32, ctypes.c_float, T, T, vp]
            L.decode_attn_fp8kv_host_io.restype = ctypes.c_int
            L.decode_attn_fp8kv_host_io.argtypes = [T, T, T, vp, vp, T, T, i32, ctypes.c_float, T, T, vp]
            L.decode_attn_static_scratch.restype = ctypes.c_int
            L.decode_attn_static_scratch.argtypes = [T, T, T, T, T, i32, ctypes.c_float, T, T, vp, vp]
            L.decode_attn_workspace_bytes.restype = ctypes.c_size_t
            L.decode_attn_workspace_bytes.argtypes = [i32, i32, i32, i32, i32, i64]
            L.decode_attn_set_workspace.restype = ctypes.c_int
            L.decode_attn_set_workspace.argtypes = [vp, ctypes.c_size_t]
            L.decode_attn_read_device_status.restype = ctypes.c_int
            L.decode_attn_read_device_status.argtypes = [vp, ctypes.POINTER(i32)]
            L.decode_attn_plan.restype = ctypes.c_int
            L.decode_attn_plan.argtypes = [T, i32, i32, i32, i64, ctypes.POINTER(i32), ctypes.POINTER(i32),
                                           ctypes.POINTER(i32), ctypes.POINTER(i32), ctypes.POINTER(i32), vp]
            L.decode_attn_set_option.restype = ctypes.c_int
            L.decode_attn_set_option.argtypes = [ctypes.c_char_p, i64]
            L.decode_attn_get_option.restype = i64
            L.decode_attn_get_option.argtypes = [ctypes.c_char_p]
            L.decode_attn_strerror.restype = ctypes.c_char_p
            L.decode_attn_strerror.argtypes = [ctypes.c_int]
            L.decode_attn_last_cuda_error.restype = ctypes.c_int
            L.decode_attn_version.restype = ctypes.c_int
            L.decode_attn_launch_count.restype = i64
            L.decode_attn_timeline.restype = ctypes.c_int
            L.decode_attn_timeline.argtypes = [ctypes.POINTER(ctypes.c_ulonglong), i64, i32]
            _lib = L
    return _lib


def _check(rc: int) -> None:
    if rc != 0:
        L = lib()
        msg = L.decode_attn_strerror(rc).decode()
        if rc == 7:
            msg += f" [cudaError {L.decode_attn_last_cuda_error()}]"
        raise DecodeAttnError(rc, msg)


def _view(t: Optional[torch.Tensor]) -> Optional[DaTensor]:
    if t is None:
        return None
    if t.dtype not in _DTYPES:
        raise TypeError(f"unsupported dtype {t.dtype}")
    if t.dim() > 4:
        raise ValueError("at most 4 dimensions")
    d = DaTensor()
    d.data = t.data_ptr()
    d.dtype = _DTYPES[t.dtype]
    n = d.ndim = t.dim()
    d.shape[0:n] = tuple(t.shape)
    d.stride[0:n] = t.stride()
    return d


def _ref(d: Optional[DaTensor]):
    return ctypes.byref(d) if d is not None else None


_have_cuda = None


def _stream_ptr(stream: Optional[torch.cuda.Stream]) -> int:
    global _have_cuda
    if _have_cuda is None:
        _have_cuda = torch.cuda.is_available()
    if not _have_cuda:
        raise RuntimeError("decode_attn needs a CUDA device; there is no CPU path")
    s = stream if stream is not None else torch.cuda.current_stream()
    return s.cuda_stream


TIMELINE_ROWS, TIMELINE_COLS = 1064, 8


def timeline(clear: bool = True):
    """The kernels' global-timer stamps of their last launch as a [TIMELINE_ROWS, TIMELINE_COLS] int64
    array (timeline build of the library only; see include/decode_attn.h for the rows)."""
    import numpy as np
    buf = (ctypes.c_ulonglong * (TIMELINE_ROWS * TIMELINE_COLS))()
    _check(lib().decode_attn_timeline(buf, TIMELINE_ROWS * TIMELINE_COLS, 1 if clear else 0))
    return np.frombuffer(buf, dtype=np.uint64).astype(np.int64).reshape(TIMELINE_ROWS, TIMELINE_COLS)


def version() -> int:
    return lib().decode_attn_version()


def launch_count() -> int:
    return int(lib().decode_attn_launch_count())


_ws_seen = {}   # (device, extents) -> bytes needed, for the current launch options


def set_option(name: str, value: int) -> None:
    _check(lib().decode_attn_set_option(name.encode(), int(value)))
    _ws_seen.clear()   # the workspace size depends on the launch options


def get_option(name: str) -> int:
    return int(lib().decode_attn_get_option(name.encode()))


def workspace_bytes(B: int, Hq: int, Hkv: int, D: int, P: int, max_pages: int) -> int:
    return int(lib().decode_attn_workspace_bytes(B, Hq, Hkv, D, P, max_pages))


def ensure_workspace(B: int, Hq: int, Hkv: int, D: int, P: int, max_pages: int,
                     device: Optional[torch.device] = None) -> torch.Tensor:
    """Make sure the current device has a registered workspace large enough for these extents.
    The buffer is a torch allocation owned here; the library only borrows the pointer."""
    dev = torch.device("cuda", torch.cuda.current_device()) if device is None else torch.device(device)
    key = (dev.index, B, Hq, Hkv, D, P, max_pages)
    need = _ws_seen.get(key)
    cur = _workspaces.get(dev.index)
    if need is not None and cur is not None and cur.numel() >= need:
        return cur    # seen before with these options, and the registered buffer is large enough
    with torch.cuda.device(dev):
        need = workspace_bytes(B, Hq, Hkv, D, P, max_pages)
        _ws_seen[key] = need
        cur = _workspaces.get(dev.index)
        if cur is None or cur.numel() < need:
            torch.cuda.synchronize()
            buf = torch.empty(max(need, 256), dtype=torch.uint8, device=dev)
            _check(lib().decode_attn_set_workspace(buf.data_ptr(), buf.numel()))
            _workspaces[dev.index] = buf
        return _workspaces[dev.index]


def _auto_workspace(q, k_pages, block_table):
    ensure_workspace(q.shape[0], q.shape[1], k_pages.shape[1], q.shape[2], k_pages.shape[2],
                     block_table.shape[1], k_pages.device)


def decode_attn(q, k_pages, v_pages, block_table, seq_lens, window: int, scale: float,
                out: Optional[torch.Tensor] = None, lse: Optional[torch.Tensor] = None,
                stream: Optional[torch.cuda.Stream] = None, out_dtype=torch.float32, want_lse: bool = True):
    """GQA decode attention over a paged bf16 KV cache (see include/decode_attn.h for the contract).

    Allocates ``out`` / ``lse`` with torch when not given, registers a workspace on first use and
    enqueues the library call on ``stream`` (default: torch's current stream).  Returns (out, lse).
    """
    if out is None:
        out = torch.empty(q.shape, dtype=out_dtype, device=q.device)
    if lse is None and want_lse:
        lse = torch.empty(q.shape[:2], dtype=torch.float32, device=q.device)
    with torch.cuda.device(k_pages.device):
        _auto_workspace(q, k_pages, block_table)
        tv = [_view(t) for t in (q, k_pages, v_pages, block_table, seq_lens, out, lse)]
        _check(lib().decode_attn(_ref(tv[0]), _ref(tv[1]), _ref(tv[2]), _ref(tv[3]), _ref(tv[4]),
                                 int(window), float(scale), _ref(tv[5]), _ref(tv[6]), _stream_ptr(stream)))
    return out, lse


def decode_attn_fp8kv(q, k_pages, v_pages, k_scale, v_scale, block_table, seq_lens, window: int, scale: float,
                      out: Optional[torch.Tensor] = None, lse: Optional[torch.Tensor] = None,
                      stream: Optional[torch.cuda.Stream] = None, out_dtype=torch.float32, want_lse: bool = True):
    """``decode_attn`` over a cache of FP8 E4M3 codes (torch.uint8 or float8_e4m3fn pools) with fp32
    per-KV-head factors ``k_scale`` / ``v_scale`` (device tensors [Hkv], or None for 1).  Returns (out, lse)."""
    if out is None:
        out = torch.empty(q.shape, dtype=out_dtype, device=q.device)
    if lse is None and want_lse:
        lse = torch.empty(q.shape[:2], dtype=torch.float32, device=q.device)
    for sc in (k_scale, v_scale):
        if sc is not None and (sc.dtype != torch.float32 or not sc.is_contiguous() or sc.device != k_pages.device
                               or sc.numel() != k_pages.shape[1]):
            raise ValueError("scales must be contiguous float32 [Hkv] tensors on the cache's device")
    with torch.cuda.device(k_pages.device):
        _auto_workspace(q, k_pages, block_table)
        tv = [_view(t) for t in (q, k_pages, v_pages, block_table, seq_lens, out, lse)]
        _check(lib().decode_attn_fp8kv(_ref(tv[0]), _ref(tv[1]), _ref(tv[2]),
                                       k_scale.data_ptr() if k_scale is not None else None,
                                       v_scale.data_ptr() if v_scale is not None else None,
                                       _ref(tv[3]), _ref(tv[4]), int(window), float(scale), _ref(tv[5]), _ref(tv[6]),
                                       _stream_ptr(stream)))
    return out, lse


def decode_attn_cascade(q, k_pages, v_pages, block_table, seq_lens, shared_prefix_tokens: int, scale: float,
                        out: Optional[torch.Tensor] = None, lse: Optional[torch.Tensor] = None,
                        stream: Optional[torch.cuda.Stream] = None, out_dtype=torch.float32):
    """decode_attn (no window) for sequences whose first ``shared_prefix_tokens`` tokens are the same
    physical pages in every block-table row; the prefix is attended once for the whole batch on the
    tensor cores.  Same result as ``decode_attn``.  Returns (out, lse)."""
    if out is None:
        out = torch.empty(q.shape, dtype=out_dtype, device=q.device)
    if lse is None:
        lse = torch.empty(q.shape[:2], dtype=torch.float32, device=q.device)
    with torch.cuda.device(k_pages.device):
        _auto_workspace(q, k_pages, block_table)
        tv = [_view(t) for t in (q, k_pages, v_pages, block_table, seq_lens, out, lse)]
        _check(lib().decode_attn_cascade(_ref(tv[0]), _ref(tv[1]), _ref(tv[2]), _ref(tv[3]), _ref(tv[4]),
                                         int(shared_prefix_tokens), float(scale), _ref(tv[5]), _ref(tv[6]),
                                         _stream_ptr(stream)))
    return out, lse


_prefix_scratch = {}   # device index -> torch uint8 tensor for the widened prefix of the 8-bit cascade


def decode_attn_fp8kv_cascade(q, k_pages, v_pages, k_scale, v_scale, block_table, seq_lens, shared_prefix_tokens: int,
                              scale: float, out: Optional[torch.Tensor] = None, lse: Optional[torch.Tensor] = None,
                              stream: Optional[torch.cuda.Stream] = None, out_dtype=torch.float32,
                              prefix_scratch: Optional[torch.Tensor] = None):
    """``decode_attn_cascade`` over the 8-bit cache (pools of E4M3 codes, per-KV-head factors).  The bf16 copy
    of the shared prefix goes to ``prefix_scratch`` (a uint8 device tensor; one is kept per device when not
    given).  Returns (out, lse)."""
    if out is None:
        out = torch.empty(q.shape, dtype=out_dtype, device=q.device)
    if lse is None:
        lse = torch.empty(q.shape[:2], dtype=torch.float32, device=q.device)
    with torch.cuda.device(k_pages.device):
        _auto_workspace(q, k_pages, block_table)
        need = int(lib().decode_attn_fp8kv_cascade_scratch_bytes(int(shared_prefix_tokens), k_pages.shape[1], k_pages.shape[2]))
        if prefix_scratch is None:
            prefix_scratch = _prefix_scratch.get(k_pages.device.index)
            if prefix_scratch is None or prefix_scratch.numel() < need:
                prefix_scratch = torch.empty(max(need, 256), dtype=torch.uint8, device=k_pages.device)
                _prefix_scratch[k_pages.device.index] = prefix_scratch
        tv = [_view(t) for t in (q, k_pages, v_pages, block_table, seq_lens, out, lse)]
        _check(lib().decode_attn_fp8kv_cascade(_ref(tv[0]), _ref(tv[1]), _ref(tv[2]),
                                               k_scale.data_ptr() if k_scale is not None else None,
                                               v_scale.data_ptr() if v_scale is not None else None,
                                               _ref(tv[3]), _ref(tv[4]), int(shared_prefix_tokens), float(scale),
                                               _ref(tv[5]), _ref(tv[6]), prefix_scratch.data_ptr(), prefix_scratch.numel(),
                                               _stream_ptr(stream)))
    return out, lse


def decode_attn_append(k_new, v_new, k_pages, v_pages, block_table, seq_lens,
                       stream: Optional[torch.cuda.Stream] = None) -> None:
    """Write the new token's K/V rows (bf16 [B, Hkv, 128]) into position seq_lens[b]-1 of the paged
    cache, in place (the step before ``decode_attn`` in a decoding loop)."""
    with torch.cuda.device(k_pages.device):
        ensure_workspace(k_new.shape[0], k_new.shape[1], k_pages.shape[1], 128, k_pages.shape[2],
                         block_table.shape[1], k_pages.device)
        tv = [_view(t) for t in (k_new, v_new, k_pages, v_pages, block_table, seq_lens)]
        _check(lib().decode_attn_append(*[_ref(t) for t in tv], _stream_ptr(stream)))


def decode_attn_append_fp8kv(k_new, v_new, k_pages, v_pages, k_scale, v_scale, block_table, seq_lens,
                             stream: Optional[torch.cuda.Stream] = None) -> None:
    """Quantise the new token's bf16 K/V rows [B, Hkv, 128] per KV head (code = nearest E4M3 of
    x / scale[g]) and write the codes into position seq_lens[b]-1 of the 8-bit cache, in place."""
    with torch.cuda.device(k_pages.device):
        ensure_workspace(k_new.shape[0], k_new.shape[1], k_pages.shape[1], 128, k_pages.shape[2],
                         block_table.shape[1], k_pages.device)
        tv = [_view(t) for t in (k_new, v_new, k_pages, v_pages, block_table, seq_lens)]
        _check(lib().decode_attn_append_fp8kv(_ref(tv[0]), _ref(tv[1]), _ref(tv[2]), _ref(tv[3]),
                                              k_scale.data_ptr() if k_scale is not None else None,
                                              v_scale.data_ptr() if v_scale is not None else None,
                                              _ref(tv[4]), _ref(tv[5]), _stream_ptr(stream)))


def decode_attn_extend(q, k_pages, v_pages, block_table, seq_lens, scale: float,
                       out: Optional[torch.Tensor] = None, lse: Optional[torch.Tensor] = None,
                       stream: Optional[torch.cuda.Stream] = None, out_dtype=torch.float32):
    """Causal attention of Lq new tokens per sequence (q: bf16 [B, Lq, Hq, 128]) over the paged cache,
    which already holds their K/V (``seq_lens`` counts them).  Returns (out [B,Lq,Hq,128], lse [B,Lq,Hq])."""
    if out is None:
        out = torch.empty(q.shape, dtype=out_dtype, device=q.device)
    if lse is None:
        lse = torch.empty(q.shape[:3], dtype=torch.float32, device=q.device)
    with torch.cuda.device(k_pages.device):
        ensure_workspace(q.shape[0], q.shape[2], k_pages.shape[1], q.shape[3], k_pages.shape[2],
                         block_table.shape[1], k_pages.device)
        tv = [_view(t) for t in (q, k_pages, v_pages, block_table, seq_lens, out, lse)]
        _check(lib().decode_attn_extend(_ref(tv[0]), _ref(tv[1]), _ref(tv[2]), _ref(tv[3]), _ref(tv[4]),
                                        float(scale), _ref(tv[5]), _ref(tv[6]), _stream_ptr(stream)))
    return out, lse


def decode_attn_fp8kv_extend(q, k_pages, v_pages, k_scale, v_scale, block_table, seq_lens, scale: float,
                             out: Optional[torch.Tensor] = None, lse: Optional[torch.Tensor] = None,
                             stream: Optional[torch.cuda.Stream] = None, out_dtype=torch.float32):
    """``decode_attn_extend`` over the 8-bit cache, for a few new tokens (Lq * Hq / Hkv <= 16)."""
    if out is None:
        out = torch.empty(q.shape, dtype=out_dtype, device=q.device)
    if lse is None:
        lse = torch.empty(q.shape[:3], dtype=torch.float32, device=q.device)
    with torch.cuda.device(k_pages.device):
        ensure_workspace(q.shape[0], q.shape[2], k_pages.shape[1], q.shape[3], k_pages.shape[2],
                         block_table.shape[1], k_pages.device)
        tv = [_view(t) for t in (q, k_pages, v_pages, block_table, seq_lens, out, lse)]
        _check(lib().decode_attn_fp8kv_extend(_ref(tv[0]), _ref(tv[1]), _ref(tv[2]),
                                              k_scale.data_ptr() if k_scale is not None else None,
                                              v_scale.data_ptr() if v_scale is not None else None,
                                              _ref(tv[3]), _ref(tv[4]), float(scale), _ref(tv[5]), _ref(tv[6]),
                                              _stream_ptr(stream)))
    return out, lse


_wide_scratch = {}   # device index -> torch uint8 tensor for the widened cache of decode_attn_fp8kv_extend_wide


def decode_attn_fp8kv_extend_wide(q, k_pages, v_pages, k_scale, v_scale, block_table, seq_lens, scale: float,
                                  out: Optional[torch.Tensor] = None, lse: Optional[torch.Tensor] = None,
                                  stream: Optional[torch.cuda.Stream] = None, out_dtype=torch.float32,
                                  scratch: Optional[torch.Tensor] = None):
    """``decode_attn_extend`` over the 8-bit cache for query blocks of any length: beyond 48 query rows per KV
    head the attended pages are widened to bf16 in ``scratch`` (a uint8 device tensor; one is kept per device
    when not given) and the tensor-core kernel runs over that copy.  Returns (out, lse)."""
    if out is None:
        out = torch.empty(q.shape, dtype=out_dtype, device=q.device)
    if lse is None:
        lse = torch.empty(q.shape[:3], dtype=torch.float32, device=q.device)
    with torch.cuda.device(k_pages.device):
        ensure_workspace(q.shape[0], q.shape[2], k_pages.shape[1], q.shape[3], k_pages.shape[2],
                         block_table.shape[1], k_pages.device)
        need = int(lib().decode_attn_fp8kv_extend_wide_scratch_bytes(q.shape[0], block_table.shape[1], k_pages.shape[1],
                                                                     k_pages.shape[2]))
        if scratch is None:
            scratch = _wide_scratch.get(k_pages.device.index)
            if scratch is None or scratch.numel() < need:
                scratch = torch.empty(max(need, 256), dtype=torch.uint8, device=k_pages.device)
                _wide_scratch[k_pages.device.index] = scratch
        tv = [_view(t) for t in (q, k_pages, v_pages, block_table, seq_lens, out, lse)]
        _check(lib().decode_attn_fp8kv_extend_wide(_ref(tv[0]), _ref(tv[1]), _ref(tv[2]),
                                                   k_scale.data_ptr() if k_scale is not None else None,
                                                   v_scale.data_ptr() if v_scale is not None else None,
                                                   _ref(tv[3]), _ref(tv[4]), float(scale), _ref(tv[5]), _ref(tv[6]),
                                                   scratch.data_ptr(), scratch.numel(), _stream_ptr(stream)))
    return out, lse


def decode_attn_host_io(q_host, k_pages, v_pages, block_table_host, seq_lens_host, window: int, scale: float,
                        out_host, lse_host=None, stream: Optional[torch.cuda.Stream] = None):
    """Same call with q / block_table / seq_lens / out / lse in (pinned) HOST memory; the KV pools
    stay on the device.  Copies and kernels are enqueued on ``stream``; nothing synchronises."""
    with torch.cuda.device(k_pages.device):
        _auto_workspace(q_host, k_pages, block_table_host)
        tv = [_view(t) for t in (q_host, k_pages, v_pages, block_table_host, seq_lens_host, out_host, lse_host)]
        _check(lib().decode_attn_host_io(_ref(tv[0]), _ref(tv[1]), _ref(tv[2]), _ref(tv[3]), _ref(tv[4]),
                                         int(window), float(scale), _ref(tv[5]), _ref(tv[6]),
                                         _stream_ptr(stream)))
    return out_host, lse_host


def decode_attn_fp8kv_host_io(q_host, k_pages, v_pages, k_scale, v_scale, block_table_host, seq_lens_host, window: int,
                              scale: float, out_host, lse_host=None, stream: Optional[torch.cuda.Stream] = None):
    """``decode_attn_host_io`` for the 8-bit cache (pools and factors on the device, per-step tensors on the host)."""
    with torch.cuda.device(k_pages.device):
        _auto_workspace(q_host, k_pages, block_table_host)
        tv = [_view(t) for t in (q_host, k_pages, v_pages, block_table_host, seq_lens_host, out_host, lse_host)]
        _check(lib().decode_attn_fp8kv_host_io(_ref(tv[0]), _ref(tv[1]), _ref(tv[2]),
                                               k_scale.data_ptr() if k_scale is not None else None,
                                               v_scale.data_ptr() if v_scale is not None else None,
                                               _ref(tv[3]), _ref(tv[4]), int(window), float(scale), _ref(tv[5]), _ref(tv[6]),
                                               _stream_ptr(stream)))
    return out_host, lse_host


def decode_attn_static_scratch(q, k_pages, v_pages, block_table, seq_lens, window: int, scale: float,
                               out: torch.Tensor, lse: Optional[torch.Tensor] = None,
                               dev_status: Optional[torch.Tensor] = None,
                               stream: Optional[torch.cuda.Stream] = None):
    """decode_attn for callers that cannot allocate: scratch is the library's fixed 6 MiB device array.

    Unlike ``decode_attn`` this wrapper allocates nothing either: ``out`` (and ``lse`` and the
    optional int32[4] device tensor ``dev_status``) must be passed in, and no workspace is
    registered.  Raises DecodeAttnError(6) beyond 4096 sequences or 320 partition blocks.
    """
    with torch.cuda.device(k_pages.device):
        tv = [_view(t) for t in (q, k_pages, v_pages, block_table, seq_lens, out, lse)]
        _check(lib().decode_attn_static_scratch(
            _ref(tv[0]), _ref(tv[1]), _ref(tv[2]), _ref(tv[3]), _ref(tv[4]), int(window), float(scale),
            _ref(tv[5]), _ref(tv[6]), dev_status.data_ptr() if dev_status is not None else None,
            _stream_ptr(stream)))
    return out, lse


def read_device_status(stream: Optional[torch.cuda.Stream] = None):
    """Synchronise and return the device status record as a 4-tuple; (0, 0, 0, 0) is clean."""
    buf = (ctypes.c_int32 * 4)()
    _check(lib().decode_attn_read_device_status(_stream_ptr(stream), buf))
    return tuple(int(x) for x in buf)


def plan(seq_lens: torch.Tensor, window: int, Hkv: int, P: int, max_pages: int,
         stream: Optional[torch.cuda.Stream] = None):
    """Run only the plan kernel; returns (seq_info [B,4], unit_work [units,4], num_static, tile_tokens)
    as host values: per sequence {lo, L, first_tile, num_tiles}; per work unit
    {b, kv_head, first tile relative to the pair's first_tile, tiles}.  Units below num_static are
    the thread blocks' own ranges, the rest are handed out by ticket."""
    B = seq_lens.shape[0]
    with torch.cuda.device(seq_lens.device):
        ensure_workspace(B, 1, Hkv, 128, P, max_pages, seq_lens.device)
        cap = 8192
        seq_info = torch.zeros((max(B, 1), 4), dtype=torch.int32)
        unit_work = torch.zeros((cap, 4), dtype=torch.int32)
        nu, ns, tt = ctypes.c_int32(cap), ctypes.c_int32(0), ctypes.c_int32(0)
        sv = _view(seq_lens)
        i32p = ctypes.POINTER(ctypes.c_int32)
        _check(lib().decode_attn_plan(_ref(sv), int(window), int(Hkv), int(P), int(max_pages),
                                      ctypes.cast(seq_info.data_ptr(), i32p),
                                      ctypes.cast(unit_work.data_ptr(), i32p),
                                      ctypes.byref(nu), ctypes.byref(ns), ctypes.byref(tt), _stream_ptr(stream)))
    return seq_info[:B], unit_work[:nu.value], ns.value, tt.value
