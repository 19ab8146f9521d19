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
    lib.oracle_policy.restype = c_int
    lib.oracle_policy.argtypes = [c_int, c_int, vp, vp, ctypes.c_float, c_int, vp, vp]
    lib.oracle_route_classes.restype = c_int
    lib.oracle_route_classes.argtypes = [c_int, c_int, c_int, c_int, c_int, vp, vp, vp, ctypes.c_float, vp, vp, vp]
    lib.oracle_e4m3_decode.restype = c_dbl
    lib.oracle_e4m3_decode.argtypes = [ctypes.c_uint8]
    lib.oracle_e4m3_encode.restype = ctypes.c_uint8
    lib.oracle_e4m3_encode.argtypes = [ctypes.c_float]
    lib.oracle_e4m3_encode_array.restype = None
    lib.oracle_e4m3_encode_array.argtypes = [c_long, vp, ctypes.c_float, vp]
    lib.oracle_e4m3_decode_array.restype = None
    lib.oracle_e4m3_decode_array.argtypes = [c_long, vp, vp]
    lib.oracle_spearman.restype = c_dbl
    lib.oracle_spearman.argtypes = [c_int, vp, vp, vp, vp]
    lib.oracle_phase_lens.restype = None
    lib.oracle_phase_lens.argtypes = [c_int, vp, vp, c_int, c_int, vp]
    lib.oracle_kv_append.restype = ctypes.c_uint
    lib.oracle_kv_append.argtypes = [c_int, c_int, c_int, c_int, c_int, c_long, c_int, vp, vp, vp, vp, vp, c_int, vp, vp]
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
    if hasattr(t, "detach"):
        return np.ascontiguousarray(t.detach().cpu().numpy().astype(np.int32))
    return np.ascontiguousarray(np.asarray(t), dtype=np.int32)


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


POLICY_RSD, POLICY_ORACLE_THRESHOLD, POLICY_ORACLE_ARGMAX, POLICY_ORACLE_BUDGET = 0, 1, 2, 3
HEAD_SOFTMAX, HEAD_ORDINAL = 0, 1


def _f32(t):
    if hasattr(t, "detach"):
        return np.ascontiguousarray(t.detach().cpu().float().numpy())
    return np.ascontiguousarray(np.asarray(t, dtype=np.float32))


def policy(kind: int, s_d, s_t=None, tau: float = 0.0, budget: int = 0):
    """Escalation policy on PRM scores.  Returns (decisions uint8 [N], stats dict)."""
    sd = _f32(s_d)
    st = _f32(s_t) if s_t is not None else None
    n = sd.shape[0]
    dec = np.zeros(n, dtype=np.uint8)
    stats = np.zeros(4, dtype=np.float64)
    rc = _load().oracle_policy(kind, n, sd.ctypes.data, st.ctypes.data if st is not None else None,
                               float(tau), int(budget), dec.ctypes.data, stats.ctypes.data)
    assert rc == 0, rc
    return dec, {"escalated": int(stats[0]), "wasted": int(stats[1]), "realised": float(stats[2]),
                 "gain": float(stats[3])}


def route_classes(mode: int, hidden, w, b, tau: float):
    """C-way router head.  w: [C, H] (softmax) or [1, H] / [H] (ordinal); b: C numbers (softmax biases, or the
    ordinal head's bias followed by its C - 1 cut points).  Returns (probs [S, C], scores [S], decisions [S])."""
    dh, hp, hk = _raw(hidden)
    dw, wp, wk = _raw(w)
    assert dh == dw
    S, H = hidden.shape
    bb = np.ascontiguousarray(np.asarray(b, dtype=np.float64))
    C = bb.shape[0]
    probs = np.zeros((S, C), dtype=np.float64)
    scores = np.zeros(S, dtype=np.float64)
    dec = np.zeros(S, dtype=np.uint8)
    rc = _load().oracle_route_classes(dh, mode, S, H, C, hp, wp, bb.ctypes.data, float(tau), probs.ctypes.data,
                                      scores.ctypes.data, dec.ctypes.data)
    assert rc == 0, rc
    return probs, scores, dec


def kv_append(k_new, v_new, block_table, seq_lens, new_lens, k_pages, v_pages, update_lens: bool = True):
    """Writes the new tokens into copies of the pools.  Returns (k_pages, v_pages, seq_lens, status bits)."""
    import torch

    kp = k_pages.detach().cpu().contiguous().clone()
    vp_ = v_pages.detach().cpu().contiguous().clone()
    kn = k_new.detach().cpu().contiguous()
    vn = v_new.detach().cpu().contiguous()
    assert kn.dtype == kp.dtype == vn.dtype == vp_.dtype
    num_pages, Hkv, P, D = kp.shape
    bt = _i32(block_table)
    sl = _i32(seq_lens).copy()
    nl = _i32(new_lens)
    st = _load().oracle_kv_append(kp.element_size(), bt.shape[0], Hkv, D, P, num_pages, bt.shape[1],
                                  kn.data_ptr(), vn.data_ptr(), bt.ctypes.data, sl.ctypes.data, nl.ctypes.data,
                                  1 if update_lens else 0, kp.data_ptr(), vp_.data_ptr())
    return kp, vp_, sl, int(st)


def phase_lens(step_lens, decisions=None, want: int = 1, t: int = -1):
    """Per-sequence lengths of the next call of a phase of the step loop (int32 [B])."""
    sl = _i32(step_lens)
    if decisions is None:
        dp, dk = None, None
    else:
        dk = np.ascontiguousarray(decisions.detach().cpu().numpy() if hasattr(decisions, "detach") else np.asarray(decisions),
                                  dtype=np.uint8)
        dp = dk.ctypes.data
    out = np.zeros(sl.shape[0], dtype=np.int32)
    _load().oracle_phase_lens(sl.shape[0], sl.ctypes.data, dp, int(want), int(t), out.ctypes.data)
    return out


def spearman(x, y, return_ranks: bool = False):
    """Spearman's rho of two fp32 samples (average ranks for ties); NaN if undefined."""
    xa, ya = _f32(x), _f32(y)
    assert xa.shape == ya.shape and xa.ndim == 1
    n = xa.shape[0]
    rx = np.zeros(n, dtype=np.float64)
    ry = np.zeros(n, dtype=np.float64)
    rho = float(_load().oracle_spearman(n, xa.ctypes.data, ya.ctypes.data, rx.ctypes.data, ry.ctypes.data))
    return (rho, rx, ry) if return_ranks else rho


# ---- E4M3 (8-bit floating point) KV cache ---------------------------------------------------------------

def e4m3_decode(codes):
    """uint8 codes (numpy or torch) -> fp32 numpy array of the same shape (exact)."""
    c = np.ascontiguousarray(codes.detach().cpu().numpy() if hasattr(codes, "detach") else np.asarray(codes), dtype=np.uint8)
    out = np.zeros(c.shape, dtype=np.float32)
    _load().oracle_e4m3_decode_array(c.size, c.ctypes.data, out.ctypes.data)
    return out


def e4m3_encode(x, inv_scale: float = 1.0):
    """values -> uint8 codes of x * inv_scale (fp32 product; nearest, ties to even, saturating at 448)."""
    a = _f32(x)
    out = np.zeros(a.shape, dtype=np.uint8)
    _load().oracle_e4m3_encode_array(a.size, a.ctypes.data, float(inv_scale), out.ctypes.data)
    return out


def kv_append_e4m3(k_new, v_new, block_table, seq_lens, new_lens, k_codes, v_codes, k_inv_scale: float,
                   v_inv_scale: float, update_lens: bool = True):
    """Quantising append: the new rows are encoded (x * inv_scale) and written into copies of the uint8 pools."""
    import torch

    kc = torch.from_numpy(e4m3_encode(k_new, k_inv_scale))
    vc = torch.from_numpy(e4m3_encode(v_new, v_inv_scale))
    return kv_append(kc, vc, block_table, seq_lens, new_lens, k_codes, v_codes, update_lens)


def attn_e4m3(q, k_codes, v_codes, k_scale: float, v_scale: float, block_table, seq_lens, q_lens, scale: float = 0.0):
    """Attention over an E4M3 cache: keys are k_scale * decode(code), values v_scale * decode(code)."""
    import math
    import torch

    D = q.shape[-1]
    sm = scale if scale > 0 else 1.0 / math.sqrt(D)
    kf = torch.from_numpy(e4m3_decode(k_codes))
    vf = torch.from_numpy(e4m3_decode(v_codes))
    out, st = attn(q.float(), kf, vf, block_table, seq_lens, q_lens, sm * float(k_scale))
    return out * float(v_scale), st


# ---- 4-bit KV cache (this library's format, stated here in full) ------------------------------------------
#
# Every (token, kv head) row of D values has one fp32 scale s = max|x| / 7 (IEEE division in fp32; s = 0 for a row
# of zeros) and D codes c = clamp(rint(x * (7 / max|x|)), -7, 7): the reciprocal 7 / max|x| by IEEE division in fp32,
# the product in fp32, rint to nearest with ties to even; c = 0 for a row of zeros.  The value read back is s * c.
# A nibble holds c + 8 (1 .. 15).  The D / 2 bytes of a row are packed per group of 8 dimensions d0 .. d7 into one
# little-endian 32-bit word whose nibbles 0 .. 7 (from the least significant) hold d0, d2, d4, d6, d1, d3, d5, d7:
# the pair (nibble i, nibble i + 4) is the pair of neighbouring dimensions (2i, 2i + 1).
# A quantised draft (Section 5.1 runs 4-bit and 3-bit drafts) is the reason for the cache; the format itself is not
# the paper's.  NaN or infinite inputs are outside the format (the row's scale would not be finite).

_I4_NIBBLE_OF_DIM = (0, 4, 1, 5, 2, 6, 3, 7)   # dimension d of a group of 8 sits in nibble _I4_NIBBLE_OF_DIM[d]


def i4_encode(x):
    """values [..., D] -> (codes uint8 [..., D / 2], scales fp32 [...])."""
    a = _f32(x)
    D = a.shape[-1]
    assert D % 8 == 0
    m = np.max(np.abs(a), axis=-1).astype(np.float32)
    with np.errstate(divide="ignore", invalid="ignore"):
        scale = np.where(m > 0, m / np.float32(7), np.float32(0)).astype(np.float32)
        inv = np.where(m > 0, np.float32(7) / m, np.float32(0)).astype(np.float32)
    c = np.rint((a * inv[..., None]).astype(np.float32))          # fp32 product, ties to even
    c = np.clip(c, -7, 7).astype(np.int64) + 8                      # nibble values 1 .. 15
    g = c.reshape(a.shape[:-1] + (D // 8, 8))
    word = np.zeros(g.shape[:-1], dtype=np.uint64)
    for d in range(8):
        word |= g[..., d].astype(np.uint64) << np.uint64(4 * _I4_NIBBLE_OF_DIM[d])
    word = word.astype(np.uint32)
    codes = np.stack([(word >> np.uint32(8 * b)) & np.uint32(0xff) for b in range(4)], axis=-1).astype(np.uint8)
    return codes.reshape(a.shape[:-1] + (D // 2,)), scale


def i4_decode(codes, scales):
    """(codes uint8 [..., D / 2], scales fp32 [...]) -> float64 values [..., D] = scale * code (exact)."""
    c = np.ascontiguousarray(codes.detach().cpu().numpy() if hasattr(codes, "detach") else np.asarray(codes), dtype=np.uint8)
    s = _f32(scales).astype(np.float64)
    half = c.shape[-1]
    b = c.reshape(c.shape[:-1] + (half // 4, 4)).astype(np.uint32)
    word = b[..., 0] | (b[..., 1] << np.uint32(8)) | (b[..., 2] << np.uint32(16)) | (b[..., 3] << np.uint32(24))
    out = np.zeros(word.shape + (8,), dtype=np.float64)
    for d in range(8):
        out[..., d] = ((word >> np.uint32(4 * _I4_NIBBLE_OF_DIM[d])) & np.uint32(0xf)).astype(np.float64) - 8.0
    return out.reshape(c.shape[:-1] + (2 * half,)) * s[..., None]


def kv_append_i4(k_new, v_new, block_table, seq_lens, new_lens, k_codes, v_codes, k_scales, v_scales,
                 update_lens: bool = True):
    """Quantising append into copies of the code pools [num_pages, Hkv, P, D / 2] and scale pools [num_pages, Hkv, P]:
    the placement rule and the refusals are kv_append's (a scale is a one-element row of the same slot)."""
    import torch

    kc, ks = i4_encode(k_new)
    vc, vs = i4_encode(v_new)
    ok, ov, sl, st = kv_append(torch.from_numpy(kc), torch.from_numpy(vc), block_table, seq_lens, new_lens, k_codes, v_codes,
                               update_lens)
    ks_p = torch.as_tensor(np.asarray(_f32(k_scales)))[..., None]
    vs_p = torch.as_tensor(np.asarray(_f32(v_scales)))[..., None]
    oks, ovs, _, _ = kv_append(torch.from_numpy(ks)[..., None], torch.from_numpy(vs)[..., None], block_table, seq_lens,
                               new_lens, ks_p, vs_p, update_lens)
    return ok, ov, oks[..., 0], ovs[..., 0], sl, st


def attn_i4(q, k_codes, v_codes, k_scales, v_scales, block_table, seq_lens, q_lens, scale: float = 0.0):
    """Attention over a 4-bit cache: keys and values are i4_decode of the pools, handed to `attn` as fp32 (its input
    type: the product scale * code is rounded once, 2^-24 relative; fp64 from there on)."""
    import torch

    kf = torch.from_numpy(i4_decode(k_codes, k_scales).astype(np.float32))
    vf = torch.from_numpy(i4_decode(v_codes, v_scales).astype(np.float32))
    return attn(q.float(), kf, vf, block_table, seq_lens, q_lens, scale)
