"""ctypes front end of the fp64 CPU oracle (``arb_oracle.c``).

TEST INFRASTRUCTURE ONLY.  Imported by the tests, the smoke check and the CPU-baseline leg of the
benchmark; never by the product package.  It shares no code with the CUDA path: the only thing
both sides consume is the seeded input tensors.

Tensors are passed as torch CPU tensors (fp32 or bf16) or numpy arrays; results come back as
numpy fp64 / uint8 / int32 arrays.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "arb_oracle.c"
_LIB = _HERE / "liboracle.so"

F32, BF16 = 0, 1
BAD_SEQ_LEN, BAD_PAGE, ROLLBACK_UNDERFLOW = 1, 2, 4

_lib = None


def build(force: bool = False) -> Path:
    """Compile arb_oracle.c into liboracle.so with gcc (OpenMP over independent rows)."""
    if force or not _LIB.exists() or _LIB.stat().st_mtime < _SRC.stat().st_mtime:
        tmp = _LIB.with_suffix(f".tmp{os.getpid()}.so")
        subprocess.check_call(
            ["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11", "-o", str(tmp), str(_SRC), "-lm"]
        )
        os.replace(tmp, _LIB)
    return _LIB


def bind(lib):
    """Declare the C signatures on a loaded library (the built one, or a variant a test compiled)."""
    c_int, c_long, c_dbl, vp = ctypes.c_int, ctypes.c_long, ctypes.c_double, ctypes.c_void_p
    lib.oracle_num_threads.restype = c_int
    lib.oracle_attn.restype = ctypes.c_uint
    lib.oracle_attn.argtypes = [c_int, c_int, c_int, c_int, c_int, c_int, c_long, c_int,
                            vp, vp, vp, vp, vp, vp, c_dbl, vp]
    lib.oracle_attn_row_probs.restype = ctypes.c_uint
    lib.oracle_attn_row_probs.argtypes = [c_int, c_int, c_int, c_int, c_int, c_long, c_int,
                                      vp, vp, vp, vp, c_long, c_int, c_long, c_dbl, vp, vp]
    lib.oracle_route.restype = None
    lib.oracle_route.argtypes = [c_int, c_int, c_int, vp, vp, c_dbl, ctypes.c_float, vp, vp]
    lib.oracle_rollback.restype = ctypes.c_uint
    lib.oracle_rollback.argtypes = [c_int, vp, vp, vp]
    return lib


def _load():
    global _lib
    if _lib is None:
        build()
        _lib = bind(ctypes.CDLL(str(_LIB)))
    return _lib


def num_threads() -> int:
    return int(_load().oracle_num_threads())


def _raw(t):
    """(dtype code, pointer, keep-alive) of a contiguous fp32/bf16 torch tensor or fp32 numpy array."""
    if isinstance(t, np.ndarray):
        a = np.ascontiguousarray(t, dtype=np.float32)
        return F32, a.ctypes.data, a
    import torch

    t = t.detach().cpu().contiguous()
    if t.dtype == torch.float32:
        return F32, t.data_ptr(), t
    if t.dtype == torch.bfloat16:
        return BF16, t.data_ptr(), t
    raise TypeError(f"oracle takes fp32 or bf16 inputs, got {t.dtype}")


def _i32(t):
    if isinstance(t, np.ndarray):
        return np.ascontiguousarray(t, dtype=np.int32)
    return np.ascontiguousarray(t.detach().cpu().numpy().astype(np.int32))


def attn(q, k_pages, v_pages, block_table, seq_lens, q_lens, scale: float = 0.0):
    """Paged GQA attention in fp64.  Returns (out[total_q, Hq, D] fp64, status bits)."""
    dt, qp, qk = _raw(q)
    dk, kp, kk = _raw(k_pages)
    dv, vp_, vk = _raw(v_pages)
    assert dt == dk == dv, "q, k_pages, v_pages share one dtype"
    total_q, Hq, D = q.shape
    num_pages, Hkv, P, D2 = k_pages.shape
    assert D2 == D and tuple(v_pages.shape) == tuple(k_pages.shape)
    bt = _i32(block_table)
    sl = _i32(seq_lens)
    ql = _i32(q_lens)
    B, max_pages = bt.shape
    assert int(np.clip(ql, 0, None).sum()) == total_q, "q rows must equal sum of q_lens"
    out = np.zeros((total_q, Hq, D), dtype=np.float64)
    st = _load().oracle_attn(dt, B, Hq, Hkv, D, P, num_pages, max_pages, qp, kp, vp_,
                             bt.ctypes.data, sl.ctypes.data, ql.ctypes.data, float(scale),
                             out.ctypes.data)
    return out, int(st)


def attn_row_probs(q, k_pages, v_pages, block_row, q_row: int, h: int, pos: int, scale: float = 0.0):
    """One output row (query row q_row, head h, attending keys 0..pos) and its softmax weights."""
    dt, qp, qk = _raw(q)
    dk, kp, kk = _raw(k_pages)
    dv, vp_, vk = _raw(v_pages)
    assert dt == dk == dv
    _, Hq, D = q.shape
    num_pages, Hkv, P, _ = k_pages.shape
    br = _i32(block_row)
    out = np.zeros(D, dtype=np.float64)
    probs = np.zeros(pos + 1, dtype=np.float64)
    st = _load().oracle_attn_row_probs(dt, Hq, Hkv, D, P, num_pages, br.shape[0], qp, kp, vp_,
                                       br.ctypes.data, q_row, h, pos, float(scale),
                                       out.ctypes.data, probs.ctypes.data)
    return out, probs, int(st)


def route(hidden, w, b: float, tau: float):
    """Router head.  Returns (scores fp64 [S], decisions uint8 [S]); 1 = escalate (score > tau)."""
    dh, hp, hk = _raw(hidden)
    dw, wp, wk = _raw(w)
    assert dh == dw
    S, H = hidden.shape
    scores = np.zeros(S, dtype=np.float64)
    dec = np.zeros(S, dtype=np.uint8)
    _load().oracle_route(dh, S, H, hp, wp, float(b), float(tau), scores.ctypes.data, dec.ctypes.data)
    return scores, dec


def rollback(seq_lens, step_lens, decisions=None):
    """Returns (new seq_lens int32 [B], status bits); the input array is not modified."""
    sl = _i32(seq_lens).copy()
    st = _i32(step_lens)
    if decisions is None:
        dp, dk = None, None
    else:
        dk = np.ascontiguousarray(
            decisions if isinstance(decisions, np.ndarray) else decisions.detach().cpu().numpy(),
            dtype=np.uint8)
        dp = dk.ctypes.data
    status = _load().oracle_rollback(sl.shape[0], sl.ctypes.data, st.ctypes.data, dp)
    return sl, int(status)
