"""ctypes binding of the C-ABI library ``libarb.so`` (``include/arb.h``).

Argument marshalling only: every step of the path runs in the CUDA kernels.  torch supplies device
memory and streams; raw pointers cross the boundary.  Importing this module fails loudly when the
library has not been built (``python -m paper_2512_05033_b200.build``): there is no fallback.
"""
from __future__ import annotations

import ctypes
from pathlib import Path

import torch

import os

# ARB_LIB_VARIANT=checks selects the bounds-check build (python -m paper_2512_05033_b200.build --checks)
_LIB_PATH = Path(__file__).resolve().parent / ("libarb_checks.so" if os.environ.get("ARB_LIB_VARIANT") == "checks"
                                               else "libarb.so")
if not _LIB_PATH.exists():
    raise ImportError(
        f"{_LIB_PATH} is missing: build the CUDA library first "
        "(python -m paper_2512_05033_b200.build); there is no CPU fallback")

lib = ctypes.CDLL(str(_LIB_PATH))

ARB_OK = 0
ARB_ERR_INVALID_ARG, ARB_ERR_UNSUPPORTED, ARB_ERR_WORKSPACE, ARB_ERR_CUDA, ARB_ERR_DEVICE_STATUS = 1, 2, 3, 4, 5
ARB_ERR_STATIC_LIMIT = 6
ARB_F32, ARB_BF16 = 0, 1
DEV_BAD_SEQ_LEN, DEV_BAD_PAGE, DEV_ROLLBACK_UNDERFLOW, DEV_WAIT_TIMEOUT, DEV_CHECK_FAILED = 1, 2, 4, 8, 16
ATTN_OVERLAP_PREVIOUS = 1
ATTN_NO_TENSOR_CORES = 2
POLICY_RSD, POLICY_ORACLE_THRESHOLD, POLICY_ORACLE_ARGMAX, POLICY_ORACLE_BUDGET = 0, 1, 2, 3
HEAD_SOFTMAX, HEAD_ORDINAL = 0, 1
MAX_CLASSES = 16

# every symbol include/arb.h declares
EXPORTS = ("arb_create", "arb_destroy", "arb_attn_workspace_bytes", "arb_attn", "arb_attn_host",
           "arb_attn_host_begin", "arb_attn_host_wait",
           "arb_attn_decode_static", "arb_decode_step", "arb_decode_step_e4m3", "arb_decode_step_i4", "arb_kv_append_i4",
           "arb_route", "arb_rollback", "arb_policy", "arb_route_classes", "arb_kv_append", "arb_kv_append_e4m3", "arb_attn_decode_e4m3", "arb_attn_e4m3", "arb_phase_lens", "arb_phase_lens_tokens", "arb_spearman",
           "arb_selftest_wait_timeout", "arb_selftest_guard_zones", "arb_poll_status", "arb_launch_count", "arb_status_string")


class AttnParams(ctypes.Structure):
    _fields_ = [("dtype", ctypes.c_int32), ("batch", ctypes.c_int32), ("num_q_heads", ctypes.c_int32),
                ("num_kv_heads", ctypes.c_int32), ("head_dim", ctypes.c_int32), ("page_size", ctypes.c_int32),
                ("num_pages", ctypes.c_int32), ("max_pages_per_seq", ctypes.c_int32),
                ("total_q", ctypes.c_int32), ("max_q_len", ctypes.c_int32), ("softmax_scale", ctypes.c_float),
                ("flags", ctypes.c_uint32)]


_vp, _i32, _f = ctypes.c_void_p, ctypes.c_int32, ctypes.c_float
lib.arb_create.restype = ctypes.c_int
lib.arb_create.argtypes = [ctypes.POINTER(_vp), ctypes.c_int, ctypes.c_size_t]
lib.arb_destroy.restype = ctypes.c_int
lib.arb_destroy.argtypes = [_vp]
lib.arb_attn_workspace_bytes.restype = ctypes.c_size_t
lib.arb_attn_workspace_bytes.argtypes = [ctypes.POINTER(AttnParams)]
lib.arb_attn.restype = ctypes.c_int
lib.arb_attn.argtypes = [_vp, ctypes.POINTER(AttnParams), _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp]
lib.arb_attn_host.restype = ctypes.c_int
lib.arb_attn_host.argtypes = [_vp, ctypes.POINTER(AttnParams), _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp]
lib.arb_attn_host_begin.restype = ctypes.c_int
lib.arb_attn_host_begin.argtypes = [_vp, ctypes.POINTER(AttnParams), _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp]
lib.arb_attn_host_wait.restype = ctypes.c_int
lib.arb_attn_host_wait.argtypes = [_vp]
lib.arb_attn_decode_static.restype = ctypes.c_int
lib.arb_attn_decode_static.argtypes = [ctypes.POINTER(AttnParams), _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp]
lib.arb_decode_step.restype = ctypes.c_int
lib.arb_decode_step.argtypes = [_vp, ctypes.POINTER(AttnParams), _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp]
lib.arb_kv_append_i4.restype = ctypes.c_int
lib.arb_kv_append_i4.argtypes = [_vp, ctypes.POINTER(AttnParams), ctypes.c_int32, _vp, _vp, _vp, _vp, _vp, ctypes.c_int32,
                                 _vp, _vp, _vp, _vp, _vp]
lib.arb_decode_step_i4.restype = ctypes.c_int
lib.arb_decode_step_i4.argtypes = [_vp, ctypes.POINTER(AttnParams)] + [_vp] * 12
lib.arb_decode_step_e4m3.restype = ctypes.c_int
lib.arb_decode_step_e4m3.argtypes = [_vp, ctypes.POINTER(AttnParams), _vp, _vp, _vp, _vp, _vp, ctypes.c_float, ctypes.c_float,
                                     ctypes.c_float, ctypes.c_float, _vp, _vp, _vp, _vp, _vp]
lib.arb_route.restype = ctypes.c_int
lib.arb_route.argtypes = [_vp, _i32, _i32, _i32, _vp, _vp, _f, _f, _vp, _vp, _vp]
lib.arb_rollback.restype = ctypes.c_int
lib.arb_rollback.argtypes = [_vp, _i32, _vp, _vp, _vp, _vp]
lib.arb_attn_decode_e4m3.restype = ctypes.c_int
lib.arb_attn_decode_e4m3.argtypes = [_vp, ctypes.POINTER(AttnParams), _vp, _vp, _vp, _f, _f, _vp, _vp, _vp, _vp, _vp]
lib.arb_attn_e4m3.restype = ctypes.c_int
lib.arb_attn_e4m3.argtypes = [_vp, ctypes.POINTER(AttnParams), _vp, _vp, _vp, _f, _f, _vp, _vp, _vp, _vp, _vp]
lib.arb_kv_append_e4m3.restype = ctypes.c_int
lib.arb_kv_append_e4m3.argtypes = [_vp, ctypes.POINTER(AttnParams), _i32, _vp, _vp, _f, _f, _vp, _vp, _vp, _i32, _vp, _vp, _vp]
lib.arb_spearman.restype = ctypes.c_int
lib.arb_spearman.argtypes = [_vp, _i32, _vp, _vp, _vp, _vp]
lib.arb_phase_lens.restype = ctypes.c_int
lib.arb_phase_lens.argtypes = [_vp, _i32, _vp, _vp, _i32, _i32, _vp, _vp]
lib.arb_phase_lens_tokens.restype = ctypes.c_int
lib.arb_phase_lens_tokens.argtypes = [_vp, _i32, _vp, _vp, _i32, _i32, _vp, _vp]
lib.arb_policy.restype = ctypes.c_int
lib.arb_policy.argtypes = [_vp, _i32, _i32, _vp, _vp, _f, _i32, _vp, _vp, _vp]
lib.arb_route_classes.restype = ctypes.c_int
lib.arb_route_classes.argtypes = [_vp, _i32, _i32, _i32, _i32, _i32, _vp, _vp, ctypes.POINTER(ctypes.c_float), _f,
                                  _vp, _vp, _vp, _vp]
lib.arb_kv_append.restype = ctypes.c_int
lib.arb_kv_append.argtypes = [_vp, ctypes.POINTER(AttnParams), _i32, _vp, _vp, _vp, _vp, _vp, _i32, _vp, _vp, _vp]
lib.arb_selftest_wait_timeout.restype = ctypes.c_int
lib.arb_selftest_wait_timeout.argtypes = [_vp, ctypes.c_int64, _vp, _vp]
lib.arb_selftest_guard_zones.restype = ctypes.c_int
lib.arb_selftest_guard_zones.argtypes = [_vp, _vp, ctypes.POINTER(ctypes.c_int64), ctypes.POINTER(ctypes.c_int64)]
lib.arb_poll_status.restype = ctypes.c_int
lib.arb_poll_status.argtypes = [_vp, _vp, ctypes.POINTER(ctypes.c_uint32)]
lib.arb_launch_count.restype = ctypes.c_uint64
lib.arb_launch_count.argtypes = [_vp]
lib.arb_status_string.restype = ctypes.c_char_p
lib.arb_status_string.argtypes = [ctypes.c_int]


class ArbError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {lib.arb_status_string(status).decode()} (arb_status {status})")


def _check(status: int, where: str):
    if status != ARB_OK:
        raise ArbError(status, where)


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return ARB_F32
    if t.dtype == torch.bfloat16:
        return ARB_BF16
    raise TypeError(f"arb takes fp32 or bf16 tensors, got {t.dtype}")


def _stream_ptr(stream) -> int:
    if stream is None:
        stream = torch.cuda.current_stream()
    return int(stream.cuda_stream)


def _dev(t: torch.Tensor, name: str, dtype=None) -> int:
    if not t.is_cuda or not t.is_contiguous():
        raise ValueError(f"{name} must be a contiguous CUDA tensor")
    if dtype is not None and t.dtype != dtype:
        raise TypeError(f"{name} must be {dtype}, got {t.dtype}")
    return t.data_ptr()


def attn_params(q_dtype_code, batch, num_q_heads, num_kv_heads, head_dim, num_pages, max_pages_per_seq, total_q,
                max_q_len, softmax_scale=0.0, page_size=16, flags=0) -> AttnParams:
    return AttnParams(q_dtype_code, batch, num_q_heads, num_kv_heads, head_dim, page_size, num_pages,
                      max_pages_per_seq, total_q, max_q_len, softmax_scale, flags)


def attn_decode_static(q, k_pages, v_pages, block_table, seq_lens, q_lens, out=None, device_status=None,
                       softmax_scale: float = 0.0, stream=None):
    """Decode attention (every q_len 1 or 0) through arb_attn_decode_static: no arb_ctx, and no
    allocation inside the library -- its scratch is a fixed array in the library image.  For hosts
    that must not allocate after start-up (a server whose free memory all went to the KV pool, a
    plug-in inside another framework's operator).  `out` should be passed in for the same reason;
    it is created here only as a convenience.  Calls that overlap on the GPU race on the shared
    scratch.  Returns out."""
    if out is None:
        out = torch.empty_like(q)
    total_q, Hq, D = q.shape
    num_pages, Hkv, P, _ = k_pages.shape
    B, max_pages = block_table.shape
    p = attn_params(_dtype_code(q), B, Hq, Hkv, D, num_pages, max_pages, total_q, 1, softmax_scale, P)
    sp = None if device_status is None else _dev(device_status, "device_status", torch.int32)
    st = lib.arb_attn_decode_static(ctypes.byref(p), _dev(q, "q"), _dev(k_pages, "k_pages", q.dtype),
                                    _dev(v_pages, "v_pages", q.dtype), _dev(block_table, "block_table", torch.int32),
                                    _dev(seq_lens, "seq_lens", torch.int32), _dev(q_lens, "q_lens", torch.int32),
                                    _dev(out, "out", q.dtype), sp, _stream_ptr(stream))
    _check(st, "arb_attn_decode_static")
    return out


class Context:
    """Owns one arb_ctx on a CUDA device (split-KV workspace, status word, staging buffers)."""

    def __init__(self, device=0, workspace_bytes: int = 0):
        self.device = torch.device("cuda", device) if isinstance(device, int) else torch.device(device)
        torch.cuda.init()
        h = _vp()
        with torch.cuda.device(self.device):
            _check(lib.arb_create(ctypes.byref(h), self.device.index or 0, workspace_bytes), "arb_create")
        self._h = h

    def close(self):
        if getattr(self, "_h", None):
            lib.arb_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- arb_attn -----------------------------------------------------------------------------
    def params_for(self, q, k_pages, block_table, max_q_len: int, softmax_scale: float = 0.0,
                   flags: int = 0) -> AttnParams:
        total_q, Hq, D = q.shape
        num_pages, Hkv, P, _ = k_pages.shape
        B, max_pages = block_table.shape
        return attn_params(_dtype_code(q), B, Hq, Hkv, D, num_pages, max_pages, total_q, max_q_len, softmax_scale, P,
                           flags)

    def attn(self, q, k_pages, v_pages, block_table, seq_lens, q_lens, max_q_len: int, out=None,
             softmax_scale: float = 0.0, stream=None, params: AttnParams | None = None):
        """out[total_q, Hq, D] = paged GQA attention; all tensors on the device.  Asynchronous."""
        if out is None:
            out = torch.empty_like(q)
        p = params or self.params_for(q, k_pages, block_table, max_q_len, softmax_scale)
        st = lib.arb_attn(self._h, ctypes.byref(p), _dev(q, "q"), _dev(k_pages, "k_pages", q.dtype),
                          _dev(v_pages, "v_pages", q.dtype), _dev(block_table, "block_table", torch.int32),
                          _dev(seq_lens, "seq_lens", torch.int32), _dev(q_lens, "q_lens", torch.int32),
                          _dev(out, "out", q.dtype), _stream_ptr(stream))
        _check(st, "arb_attn")
        return out

    def attn_raw(self, p: AttnParams, q_ptr, k_ptr, v_ptr, bt_ptr, sl_ptr, ql_ptr, out_ptr, stream_ptr) -> int:
        """Pointer-level call (no tensor checks) for timing loops; returns the arb_status."""
        return lib.arb_attn(self._h, ctypes.byref(p), q_ptr, k_ptr, v_ptr, bt_ptr, sl_ptr, ql_ptr, out_ptr, stream_ptr)

    def attn_host(self, q_host, k_pages, v_pages, block_table_host, seq_lens_host, q_lens_host, max_q_len: int,
                  out_host=None, softmax_scale: float = 0.0, stream=None):
        """Same with q / block_table / lengths / out in host memory (pinned for async copies).
        Synchronises the stream before returning."""
        if out_host is None:
            out_host = torch.empty_like(q_host, pin_memory=True)
        for t in (q_host, block_table_host, seq_lens_host, q_lens_host, out_host):
            if t.is_cuda or not t.is_contiguous():
                raise ValueError("host tensors must be contiguous CPU tensors")
        p = self.params_for(q_host, k_pages, block_table_host, max_q_len, softmax_scale)
        st = lib.arb_attn_host(self._h, ctypes.byref(p), q_host.data_ptr(), _dev(k_pages, "k_pages"),
                               _dev(v_pages, "v_pages"), block_table_host.data_ptr(), seq_lens_host.data_ptr(),
                               q_lens_host.data_ptr(), out_host.data_ptr(), _stream_ptr(stream))
        _check(st, "arb_attn_host")
        return out_host

    def attn_host_raw(self, p: AttnParams, q_ptr, k_ptr, v_ptr, bt_ptr, sl_ptr, ql_ptr, out_ptr, stream_ptr) -> int:
        """Pointer-level form of attn_host (host pointers for q, block table, lengths and out); returns the arb_status."""
        return lib.arb_attn_host(self._h, ctypes.byref(p), q_ptr, k_ptr, v_ptr, bt_ptr, sl_ptr, ql_ptr, out_ptr, stream_ptr)

    def attn_host_begin(self, q_host, k_pages, v_pages, block_table_host, seq_lens_host, q_lens_host, max_q_len: int,
                        out_host, softmax_scale: float = 0.0, flags: int = 0, stream=None):
        """First half of the pipelined host call: enqueues copies and kernels and returns; out_host (pinned) holds
        the result once attn_host_wait() has returned."""
        for t in (q_host, block_table_host, seq_lens_host, q_lens_host, out_host):
            if t.is_cuda or not t.is_contiguous():
                raise ValueError("host tensors must be contiguous CPU tensors")
        p = self.params_for(q_host, k_pages, block_table_host, max_q_len, softmax_scale)
        p.flags = flags
        st = lib.arb_attn_host_begin(self._h, ctypes.byref(p), q_host.data_ptr(), _dev(k_pages, "k_pages"),
                                     _dev(v_pages, "v_pages"), block_table_host.data_ptr(), seq_lens_host.data_ptr(),
                                     q_lens_host.data_ptr(), out_host.data_ptr(), _stream_ptr(stream))
        _check(st, "arb_attn_host_begin")
        return out_host

    def attn_host_begin_raw(self, p: AttnParams, q_ptr, k_ptr, v_ptr, bt_ptr, sl_ptr, ql_ptr, out_ptr, stream_ptr) -> int:
        """Pointer-level form of attn_host_begin; returns the arb_status."""
        return lib.arb_attn_host_begin(self._h, ctypes.byref(p), q_ptr, k_ptr, v_ptr, bt_ptr, sl_ptr, ql_ptr, out_ptr,
                                       stream_ptr)

    def attn_host_wait(self):
        """Blocks until every attn_host_begin of this context has delivered its result."""
        _check(lib.arb_attn_host_wait(self._h), "arb_attn_host_wait")

    # -- arb_decode_step ----------------------------------------------------------------------
    def decode_step(self, q, k_new, v_new, k_pages, v_pages, block_table, seq_lens, q_lens, out=None,
                    softmax_scale: float = 0.0, stream=None, params: AttnParams | None = None):
        """One decode token in one launch: the new K/V rows go into the cache, out = attention over the cache
        including them, seq_lens += q_lens (in place).  Asynchronous."""
        if out is None:
            out = torch.empty_like(q)
        p = params or self.params_for(q, k_pages, block_table, 1, softmax_scale)
        st = lib.arb_decode_step(self._h, ctypes.byref(p), _dev(q, "q"), _dev(k_new, "k_new", q.dtype),
                                 _dev(v_new, "v_new", q.dtype), _dev(k_pages, "k_pages", q.dtype),
                                 _dev(v_pages, "v_pages", q.dtype), _dev(block_table, "block_table", torch.int32),
                                 _dev(seq_lens, "seq_lens", torch.int32), _dev(q_lens, "q_lens", torch.int32),
                                 _dev(out, "out", q.dtype), _stream_ptr(stream))
        _check(st, "arb_decode_step")
        return out

    # -- arb_decode_step_e4m3 -----------------------------------------------------------------
    def decode_step_e4m3(self, q, k_new, v_new, k_codes, v_codes, k_scale: float, v_scale: float, k_inv_scale: float,
                         v_inv_scale: float, block_table, seq_lens, q_lens, out=None, softmax_scale: float = 0.0,
                         stream=None, params: AttnParams | None = None):
        """decode_step over an E4M3 cache: the new rows are quantised into the code pools, out = attention over
        the codes including them, seq_lens += q_lens (in place).  Asynchronous."""
        if out is None:
            out = torch.empty_like(q)
        p = params or self.params_for(q, k_codes, block_table, 1, softmax_scale)
        st = lib.arb_decode_step_e4m3(self._h, ctypes.byref(p), _dev(q, "q", torch.bfloat16),
                                      _dev(k_new, "k_new", torch.bfloat16), _dev(v_new, "v_new", torch.bfloat16),
                                      _dev(k_codes, "k_codes", torch.uint8), _dev(v_codes, "v_codes", torch.uint8),
                                      float(k_scale), float(v_scale), float(k_inv_scale), float(v_inv_scale),
                                      _dev(block_table, "block_table", torch.int32),
                                      _dev(seq_lens, "seq_lens", torch.int32), _dev(q_lens, "q_lens", torch.int32),
                                      _dev(out, "out", torch.bfloat16), _stream_ptr(stream))
        _check(st, "arb_decode_step_e4m3")
        return out

    # -- arb_decode_step_i4 -------------------------------------------------------------------
    def decode_step_i4(self, q, k_new, v_new, k_codes, v_codes, k_scales, v_scales, block_table, seq_lens, q_lens,
                       out=None, softmax_scale: float = 0.0, stream=None, params: AttnParams | None = None):
        """decode_step over a 4-bit cache (codes uint8 [pages, Hkv, P, D / 2], scales fp32 [pages, Hkv, P]): the new
        rows are quantised into the pools, out = attention over scale * code including them, seq_lens += q_lens."""
        if out is None:
            out = torch.empty_like(q)
        if params is None:
            num_pages, Hkv, P, _ = k_codes.shape
            B, max_pages = block_table.shape
            params = attn_params(_dtype_code(q), B, q.shape[1], Hkv, q.shape[2], num_pages, max_pages, q.shape[0], 1,
                                 softmax_scale, P, 0)
        st = lib.arb_decode_step_i4(self._h, ctypes.byref(params), _dev(q, "q", torch.bfloat16),
                                    _dev(k_new, "k_new", torch.bfloat16), _dev(v_new, "v_new", torch.bfloat16),
                                    _dev(k_codes, "k_codes", torch.uint8), _dev(v_codes, "v_codes", torch.uint8),
                                    _dev(k_scales, "k_scales", torch.float32), _dev(v_scales, "v_scales", torch.float32),
                                    _dev(block_table, "block_table", torch.int32),
                                    _dev(seq_lens, "seq_lens", torch.int32), _dev(q_lens, "q_lens", torch.int32),
                                    _dev(out, "out", torch.bfloat16), _stream_ptr(stream))
        _check(st, "arb_decode_step_i4")
        return out

    # -- arb_kv_append_i4 ---------------------------------------------------------------------
    def kv_append_i4(self, k_new, v_new, block_table, seq_lens, new_lens, k_codes, v_codes, k_scales, v_scales,
                     update_lens: bool = True, stream=None):
        """In place: the new rows are quantised to the 4-bit format and written behind each sequence's tokens."""
        num_pages, Hkv, P, half = k_codes.shape
        B, max_pages = block_table.shape
        p = attn_params(_dtype_code(k_new), B, Hkv, Hkv, 2 * half, num_pages, max_pages, 0, 0, 0.0, P, 0)
        st = lib.arb_kv_append_i4(self._h, ctypes.byref(p), k_new.shape[0], _dev(k_new, "k_new", torch.bfloat16),
                                  _dev(v_new, "v_new", torch.bfloat16), _dev(block_table, "block_table", torch.int32),
                                  _dev(seq_lens, "seq_lens", torch.int32), _dev(new_lens, "new_lens", torch.int32),
                                  1 if update_lens else 0, _dev(k_codes, "k_codes", torch.uint8),
                                  _dev(v_codes, "v_codes", torch.uint8), _dev(k_scales, "k_scales", torch.float32),
                                  _dev(v_scales, "v_scales", torch.float32), _stream_ptr(stream))
        _check(st, "arb_kv_append_i4")

    # -- arb_route ----------------------------------------------------------------------------
    def route(self, hidden, w, b: float, tau: float, scores=None, decisions=None, stream=None):
        """scores fp32 [S] = sigmoid(hidden . w + b); decisions uint8 [S] = (score > tau)."""
        S, H = hidden.shape
        if scores is None:
            scores = torch.empty(S, dtype=torch.float32, device=hidden.device)
        if decisions is None:
            decisions = torch.empty(S, dtype=torch.uint8, device=hidden.device)
        st = lib.arb_route(self._h, _dtype_code(hidden), S, H, _dev(hidden, "hidden"), _dev(w, "w", hidden.dtype),
                           float(b), float(tau), _dev(scores, "scores", torch.float32),
                           _dev(decisions, "decisions", torch.uint8), _stream_ptr(stream))
        _check(st, "arb_route")
        return scores, decisions

    # -- arb_rollback -------------------------------------------------------------------------
    def rollback(self, seq_lens, step_lens, decisions=None, stream=None):
        """In place: seq_lens[i] -= step_lens[i] where decisions is None or decisions[i] != 0."""
        dp = None if decisions is None else _dev(decisions, "decisions", torch.uint8)
        st = lib.arb_rollback(self._h, seq_lens.shape[0], _dev(seq_lens, "seq_lens", torch.int32),
                              _dev(step_lens, "step_lens", torch.int32), dp, _stream_ptr(stream))
        _check(st, "arb_rollback")
        return seq_lens

    # -- arb_attn_decode_e4m3 -----------------------------------------------------------------
    def attn_decode_e4m3(self, q, k_codes, v_codes, k_scale: float, v_scale: float, block_table, seq_lens, q_lens,
                         out=None, softmax_scale: float = 0.0, flags: int = 0, stream=None, params=None):
        """Decode attention (q_len 1 or 0) over an E4M3 cache; q and out bf16.  Asynchronous."""
        if out is None:
            out = torch.empty_like(q)
        p = params or self.params_for(q, k_codes, block_table, 1, softmax_scale, flags=flags)
        st = lib.arb_attn_decode_e4m3(self._h, ctypes.byref(p), _dev(q, "q", torch.bfloat16),
                                      _dev(k_codes, "k_codes", torch.uint8), _dev(v_codes, "v_codes", torch.uint8),
                                      float(k_scale), float(v_scale), _dev(block_table, "block_table", torch.int32),
                                      _dev(seq_lens, "seq_lens", torch.int32), _dev(q_lens, "q_lens", torch.int32),
                                      _dev(out, "out", torch.bfloat16), _stream_ptr(stream))
        _check(st, "arb_attn_decode_e4m3")
        return out

    # -- arb_attn_e4m3 ------------------------------------------------------------------------
    def attn_e4m3(self, q, k_codes, v_codes, k_scale: float, v_scale: float, block_table, seq_lens, q_lens,
                  max_q_len: int, out=None, softmax_scale: float = 0.0, stream=None, params=None):
        """Attention (decode rows and step chunks) over an E4M3 cache; q and out bf16.  Asynchronous."""
        if out is None:
            out = torch.empty_like(q)
        p = params or self.params_for(q, k_codes, block_table, max_q_len, softmax_scale)
        st = lib.arb_attn_e4m3(self._h, ctypes.byref(p), _dev(q, "q", torch.bfloat16),
                               _dev(k_codes, "k_codes", torch.uint8), _dev(v_codes, "v_codes", torch.uint8),
                               float(k_scale), float(v_scale), _dev(block_table, "block_table", torch.int32),
                               _dev(seq_lens, "seq_lens", torch.int32), _dev(q_lens, "q_lens", torch.int32),
                               _dev(out, "out", torch.bfloat16), _stream_ptr(stream))
        _check(st, "arb_attn_e4m3")
        return out

    # -- arb_kv_append_e4m3 -------------------------------------------------------------------
    def kv_append_e4m3(self, k_new, v_new, k_inv_scale: float, v_inv_scale: float, block_table, seq_lens, new_lens,
                       k_codes, v_codes, update_lens: bool = True, stream=None):
        """In place: the new rows are quantised to E4M3 (x * inv_scale) and written behind each sequence's tokens."""
        num_pages, Hkv, P, D = k_codes.shape
        B, max_pages = block_table.shape
        p = attn_params(_dtype_code(k_new), B, Hkv, Hkv, D, num_pages, max_pages, 0, 0, 0.0, P, 0)
        st = lib.arb_kv_append_e4m3(self._h, ctypes.byref(p), k_new.shape[0], _dev(k_new, "k_new"),
                                    _dev(v_new, "v_new", k_new.dtype), float(k_inv_scale), float(v_inv_scale),
                                    _dev(block_table, "block_table", torch.int32), _dev(seq_lens, "seq_lens", torch.int32),
                                    _dev(new_lens, "new_lens", torch.int32), 1 if update_lens else 0,
                                    _dev(k_codes, "k_codes", torch.uint8), _dev(v_codes, "v_codes", torch.uint8),
                                    _stream_ptr(stream))
        _check(st, "arb_kv_append_e4m3")
        return seq_lens

    # -- arb_spearman -------------------------------------------------------------------------
    def spearman(self, x, y, rho=None, stream=None):
        """rho (device float64 [1]) = Spearman's rank correlation of two fp32 device vectors."""
        if rho is None:
            rho = torch.empty(1, dtype=torch.float64, device=x.device)
        st = lib.arb_spearman(self._h, x.shape[0], _dev(x, "x", torch.float32), _dev(y, "y", torch.float32),
                              _dev(rho, "rho", torch.float64), _stream_ptr(stream))
        _check(st, "arb_spearman")
        return rho

    # -- arb_phase_lens -----------------------------------------------------------------------
    def phase_lens(self, step_lens, decisions=None, want: int = 1, t: int = -1, out=None, stream=None):
        """out int32 [B]: lengths of the next call of a phase of the step loop (see arb_phase_lens)."""
        if out is None:
            out = torch.empty_like(step_lens)
        dp = None if decisions is None else _dev(decisions, "decisions", torch.uint8)
        st = lib.arb_phase_lens(self._h, step_lens.shape[0], _dev(step_lens, "step_lens", torch.int32), dp, int(want),
                                int(t), _dev(out, "out", torch.int32), _stream_ptr(stream))
        _check(st, "arb_phase_lens")
        return out

    def phase_lens_tokens(self, step_lens, n_tokens: int, decisions=None, want: int = 1, out=None, stream=None):
        """out int32 [n_tokens, B]: row t = phase_lens(..., t=t), all rows in one launch."""
        B = step_lens.shape[0]
        if out is None:
            out = torch.empty(n_tokens, B, dtype=torch.int32, device=step_lens.device)
        dp = None if decisions is None else _dev(decisions, "decisions", torch.uint8)
        st = lib.arb_phase_lens_tokens(self._h, B, _dev(step_lens, "step_lens", torch.int32), dp, int(want), int(n_tokens),
                                       _dev(out, "out", torch.int32), _stream_ptr(stream))
        _check(st, "arb_phase_lens_tokens")
        return out

    # -- arb_policy ---------------------------------------------------------------------------
    def policy(self, kind: int, s_d, s_t=None, tau: float = 0.0, budget: int = 0, decisions=None, stats=None,
               stream=None):
        """Escalation decisions uint8 [N] from PRM scores (fp32 device tensors).  `stats`, if given, is a
        device tensor of 3 float64 that receives the arb_policy_stats record (two uint32 counters, then the
        realised score and the gain); read it with policy_stats()."""
        n = s_d.shape[0]
        if decisions is None:
            decisions = torch.empty(n, dtype=torch.uint8, device=s_d.device)
        sp = None if stats is None else _dev(stats, "stats", torch.float64)
        tp = None if s_t is None else _dev(s_t, "s_t", torch.float32)
        st = lib.arb_policy(self._h, kind, n, _dev(s_d, "s_d", torch.float32), tp, float(tau), int(budget),
                            _dev(decisions, "decisions", torch.uint8), sp, _stream_ptr(stream))
        _check(st, "arb_policy")
        return decisions

    @staticmethod
    def new_policy_stats(device):
        return torch.zeros(3, dtype=torch.float64, device=device)

    @staticmethod
    def policy_stats(stats) -> dict:
        """Decodes the 24-byte arb_policy_stats record held in a float64[3] tensor (synchronises)."""
        raw = stats.cpu().numpy().tobytes()
        import struct
        esc, wasted, realised, gain = struct.unpack("<IIdd", raw)
        return {"escalated": esc, "wasted": wasted, "realised": realised, "gain": gain}

    # -- arb_route_classes --------------------------------------------------------------------
    def route_classes(self, mode: int, hidden, w, b, tau: float, probs=None, scores=None, decisions=None,
                      stream=None):
        """C-way head: returns (probs fp32 [S, C], scores fp32 [S], decisions uint8 [S]).  b: C host floats."""
        S, H = hidden.shape
        C = len(b)
        if probs is None:
            probs = torch.empty(S, C, dtype=torch.float32, device=hidden.device)
        if scores is None:
            scores = torch.empty(S, dtype=torch.float32, device=hidden.device)
        if decisions is None:
            decisions = torch.empty(S, dtype=torch.uint8, device=hidden.device)
        bh = (ctypes.c_float * C)(*[float(x) for x in b])
        st = lib.arb_route_classes(self._h, _dtype_code(hidden), mode, S, H, C, _dev(hidden, "hidden"),
                                   _dev(w, "w", hidden.dtype), bh, float(tau), _dev(probs, "probs", torch.float32),
                                   _dev(scores, "scores", torch.float32), _dev(decisions, "decisions", torch.uint8),
                                   _stream_ptr(stream))
        _check(st, "arb_route_classes")
        return probs, scores, decisions

    # -- arb_kv_append ------------------------------------------------------------------------
    def kv_append(self, k_new, v_new, block_table, seq_lens, new_lens, k_pages, v_pages, update_lens: bool = True,
                  stream=None):
        """In place: the new tokens' K/V go behind each sequence's cached tokens; seq_lens += new_lens."""
        num_pages, Hkv, P, D = k_pages.shape
        B, max_pages = block_table.shape
        p = attn_params(_dtype_code(k_pages), B, Hkv, Hkv, D, num_pages, max_pages, 0, 0, 0.0, P, 0)
        total_new = k_new.shape[0]
        st = lib.arb_kv_append(self._h, ctypes.byref(p), total_new, _dev(k_new, "k_new", k_pages.dtype),
                               _dev(v_new, "v_new", k_pages.dtype), _dev(block_table, "block_table", torch.int32),
                               _dev(seq_lens, "seq_lens", torch.int32), _dev(new_lens, "new_lens", torch.int32),
                               1 if update_lens else 0, _dev(k_pages, "k_pages"), _dev(v_pages, "v_pages", k_pages.dtype),
                               _stream_ptr(stream))
        _check(st, "arb_kv_append")
        return seq_lens

    # -- self-test ----------------------------------------------------------------------------
    def selftest_wait_timeout(self, limit_cycles: int, report=None, stream=None):
        """Launches the kernel whose wait can only run out (see arb_selftest_wait_timeout); returns the int32[3]
        device report.  The status word carries DEV_WAIT_TIMEOUT afterwards."""
        if report is None:
            report = torch.zeros(3, dtype=torch.int32, device=self.device)
        _check(lib.arb_selftest_wait_timeout(self._h, int(limit_cycles), _dev(report, "report", torch.int32),
                                             _stream_ptr(stream)), "arb_selftest_wait_timeout")
        return report

    def guard_zones(self, stream=None):
        """(bytes of the guard zones that were overwritten, guard bytes checked); (0, 0) in the ordinary build."""
        bad, checked = ctypes.c_int64(0), ctypes.c_int64(0)
        _check(lib.arb_selftest_guard_zones(self._h, _stream_ptr(stream), ctypes.byref(bad), ctypes.byref(checked)),
               "arb_selftest_guard_zones")
        return int(bad.value), int(checked.value)

    # -- status -------------------------------------------------------------------------------
    def poll_status(self, stream=None) -> int:
        """Synchronises; returns the device status bits (and clears them)."""
        bits = ctypes.c_uint32(0)
        st = lib.arb_poll_status(self._h, _stream_ptr(stream), ctypes.byref(bits))
        if st not in (ARB_OK, ARB_ERR_DEVICE_STATUS):
            _check(st, "arb_poll_status")
        return int(bits.value)

    def launch_count(self) -> int:
        return int(lib.arb_launch_count(self._h))
