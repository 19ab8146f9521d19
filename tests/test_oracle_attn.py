"""Pins of the attention oracle against things other than itself (no GPU).

Each test is chosen so that a plausible mistake in the oracle (a dropped scale, a wrong causal
bound, a transposed operand, a wrong GQA mapping, a wrong page index, a bad bf16 widening) fails
at least one of them.
"""
import math

import numpy as np
import pytest
import torch

from oracle import oracle
from paper_2512_05033_b200 import workloads as wl

P = wl.PAGE


def dense_kv(inp, b):
    """Gather sequence b's K and V into dense fp64 [L, Hkv, D] arrays (independent code path)."""
    L = int(inp.seq_lens[b])
    K = inp.k_pages.to(torch.float64).numpy()
    V = inp.v_pages.to(torch.float64).numpy()
    bt = inp.block_table[b].numpy()
    Kd = np.stack([K[bt[j // P], :, j % P, :] for j in range(L)])
    Vd = np.stack([V[bt[j // P], :, j % P, :] for j in range(L)])
    return Kd, Vd


def brute_force(inp, scale=None):
    """Masked dense softmax(QK^T)V with numpy matmuls in fp64."""
    q = inp.q.to(torch.float64).numpy()
    T, Hq, D = q.shape
    Hkv = inp.k_pages.shape[1]
    g = Hq // Hkv
    scale = 1.0 / math.sqrt(D) if scale is None else scale
    out = np.zeros_like(q)
    row = 0
    for b in range(inp.seq_lens.shape[0]):
        n, L = int(inp.q_lens[b]), int(inp.seq_lens[b])
        if n <= 0:
            continue
        Kd, Vd = dense_kv(inp, b)
        for h in range(Hq):
            Kh, Vh = Kd[:, h // g, :], Vd[:, h // g, :]
            S = scale * (q[row:row + n, h, :] @ Kh.T)                  # [n, L]
            pos = (L - n) + np.arange(n)[:, None]
            S = np.where(np.arange(L)[None, :] <= pos, S, -np.inf)
            S = S - S.max(axis=1, keepdims=True)
            W = np.exp(S)
            W /= W.sum(axis=1, keepdims=True)
            out[row:row + n, h, :] = W @ Vh
        row += n
    return out


CASES = [
    # (B, Hq, Hkv, D, dtype, seq_lens, q_lens)
    (1, 8, 2, 64, torch.float32, [40], [1]),
    (2, 6, 2, 64, torch.float32, [17, 64], [5, 16]),
    (3, 12, 2, 128, torch.bfloat16, [33, 1, 50], [1, 1, 7]),
    (2, 7, 1, 128, torch.bfloat16, [31, 48], [31, 3]),
    (2, 4, 4, 64, torch.bfloat16, [16, 19], [0, 2]),
]


@pytest.mark.parametrize("case", CASES)
def test_matches_bruteforce_dense(case):
    B, Hq, Hkv, D, dt, sl, ql = case
    inp = wl.small_attn_case(B, Hq, Hkv, D, dt, sl, ql, seed=11)
    out, st = oracle.attn(inp.q, inp.k_pages, inp.v_pages, inp.block_table, inp.seq_lens, inp.q_lens)
    assert st == 0
    np.testing.assert_allclose(out, brute_force(inp), rtol=0, atol=1e-12)


def test_matches_library_sdpa_fp64():
    """A library routine (torch SDPA on CPU in fp64) on a dense, single-sequence multi-head case."""
    Hq, D, L, n = 4, 64, 37, 6
    inp = wl.small_attn_case(1, Hq, Hq, D, torch.float32, [L], [n], seed=5)
    out, _ = oracle.attn(inp.q, inp.k_pages, inp.v_pages, inp.block_table, inp.seq_lens, inp.q_lens)
    Kd, Vd = dense_kv(inp, 0)
    q = inp.q.to(torch.float64).permute(1, 0, 2)[None]                 # [1, H, n, D]
    k = torch.from_numpy(Kd).permute(1, 0, 2)[None]
    v = torch.from_numpy(Vd).permute(1, 0, 2)[None]
    mask = (torch.arange(L)[None, :] <= (L - n + torch.arange(n))[:, None])
    ref = torch.nn.functional.scaled_dot_product_attention(q, k, v, attn_mask=mask)
    np.testing.assert_allclose(out, ref[0].permute(1, 0, 2).numpy(), rtol=0, atol=1e-12)


def test_scale_argument():
    inp = wl.small_attn_case(1, 2, 1, 64, torch.float32, [23], [2], seed=6)
    out, _ = oracle.attn(inp.q, inp.k_pages, inp.v_pages, inp.block_table, inp.seq_lens, inp.q_lens, scale=0.3)
    np.testing.assert_allclose(out, brute_force(inp, scale=0.3), atol=1e-12)
    out0, _ = oracle.attn(inp.q, inp.k_pages, inp.v_pages, inp.block_table, inp.seq_lens, inp.q_lens, scale=0.0)
    np.testing.assert_allclose(out0, brute_force(inp), atol=1e-12)
    assert np.abs(out - out0).max() > 1e-3


def test_softmax_rows_sum_to_one():
    inp = wl.small_attn_case(1, 8, 2, 64, torch.float32, [100], [4], seed=7)
    for h in (0, 5):
        for i in range(4):
            pos = 100 - 4 + i
            _, p, st = oracle.attn_row_probs(inp.q, inp.k_pages, inp.v_pages, inp.block_table[0], i, h, pos)
            assert st == 0 and p.shape == (pos + 1,)
            assert abs(p.sum() - 1.0) < 1e-14
            assert (p > 0).all() and (p <= 1).all()


def test_two_key_closed_form():
    """q.k = [0, ln 3 / scale]  =>  weights (1/4, 3/4): out = v0/4 + 3 v1/4."""
    D = 64
    inp = wl.small_attn_case(1, 1, 1, D, torch.float32, [2], [1], seed=8)
    scale = 1.0 / math.sqrt(D)
    inp.q.zero_()
    inp.q[0, 0, 3] = math.log(3.0) / scale
    pg = int(inp.block_table[0, 0])
    inp.k_pages[pg, 0, 0].zero_()
    inp.k_pages[pg, 0, 1].zero_()
    inp.k_pages[pg, 0, 1, 3] = 1.0
    out, _ = oracle.attn(inp.q, inp.k_pages, inp.v_pages, inp.block_table, inp.seq_lens, inp.q_lens)
    v = inp.v_pages[pg, 0].to(torch.float64).numpy()
    # q holds ln3/scale rounded to fp32, so the weights are 3/4, 1/4 to fp32 rounding
    np.testing.assert_allclose(out[0, 0], 0.25 * v[0] + 0.75 * v[1], atol=2e-7)
    _, p, _ = oracle.attn_row_probs(inp.q, inp.k_pages, inp.v_pages, inp.block_table[0], 0, 0, 1)
    np.testing.assert_allclose(p, [0.25, 0.75], atol=1e-7)


def test_uniform_keys_give_mean_of_v():
    inp = wl.small_attn_case(2, 4, 2, 64, torch.float32, [45, 20], [3, 1], seed=9)
    inp.k_pages[:] = inp.k_pages[0, 0, 0]            # every key identical
    out, _ = oracle.attn(inp.q, inp.k_pages, inp.v_pages, inp.block_table, inp.seq_lens, inp.q_lens)
    Kd, Vd = dense_kv(inp, 0)
    for i in range(3):
        pos = 45 - 3 + i
        for h in range(4):
            np.testing.assert_allclose(out[i, h], Vd[:pos + 1, h // 2].mean(axis=0), atol=1e-14)
    # q = 0 has the same effect whatever the keys are
    inp2 = wl.small_attn_case(1, 4, 2, 64, torch.float32, [30], [1], seed=10)
    inp2.q.zero_()
    out2, _ = oracle.attn(inp2.q, inp2.k_pages, inp2.v_pages, inp2.block_table, inp2.seq_lens, inp2.q_lens)
    _, Vd2 = dense_kv(inp2, 0)
    np.testing.assert_allclose(out2[0, 3], Vd2[:, 1].mean(axis=0), atol=1e-14)


def test_single_key_returns_its_value():
    inp = wl.small_attn_case(1, 4, 2, 64, torch.bfloat16, [1], [1], seed=12)
    out, _ = oracle.attn(inp.q, inp.k_pages, inp.v_pages, inp.block_table, inp.seq_lens, inp.q_lens)
    pg = int(inp.block_table[0, 0])
    for h in range(4):
        np.testing.assert_array_equal(out[0, h], inp.v_pages[pg, h // 2, 0].to(torch.float64).numpy())


def test_dominant_key_returns_its_value():
    D = 64
    inp = wl.small_attn_case(1, 2, 1, D, torch.float32, [50], [1], seed=13)
    j = 37
    pg, slot = int(inp.block_table[0, j // P]), j % P
    inp.k_pages.mul_(0.01)
    inp.k_pages[pg, 0, slot] = inp.q[0, 0] * 100.0    # score gap far above 50
    out, _ = oracle.attn(inp.q, inp.k_pages, inp.v_pages, inp.block_table, inp.seq_lens, inp.q_lens)
    np.testing.assert_allclose(out[0, 0], inp.v_pages[pg, 0, slot].to(torch.float64).numpy(), atol=1e-15)


def test_score_shift_invariance():
    """Adding to every key a vector a with q.a = c shifts every score by scale*c: same output."""
    inp = wl.small_attn_case(1, 1, 1, 64, torch.float32, [29], [1], seed=14)
    out, _ = oracle.attn(inp.q, inp.k_pages, inp.v_pages, inp.block_table, inp.seq_lens, inp.q_lens)
    q = inp.q[0, 0]
    a = q * (40.0 / float(q @ q))
    inp.k_pages += a
    out2, _ = oracle.attn(inp.q, inp.k_pages, inp.v_pages, inp.block_table, inp.seq_lens, inp.q_lens)
    np.testing.assert_allclose(out2, out, atol=1e-5)   # fp32 rounding of the shifted keys


def test_page_permutation_invariance_bit_identical():
    inp = wl.small_attn_case(2, 4, 2, 64, torch.bfloat16, [70, 33], [4, 1], seed=15)
    out, _ = oracle.attn(inp.q, inp.k_pages, inp.v_pages, inp.block_table, inp.seq_lens, inp.q_lens)
    n = inp.num_pages
    perm = torch.randperm(n, generator=torch.Generator().manual_seed(3))
    k2 = torch.empty_like(inp.k_pages)
    v2 = torch.empty_like(inp.v_pages)
    k2[perm] = inp.k_pages
    v2[perm] = inp.v_pages
    bt2 = inp.block_table.clone()
    valid = bt2 >= 0
    bt2[valid] = perm[bt2[valid].long()].to(torch.int32)
    out2, _ = oracle.attn(inp.q, k2, v2, bt2, inp.seq_lens, inp.q_lens)
    np.testing.assert_array_equal(out, out2)


def test_sequences_do_not_see_each_others_pages():
    inp = wl.small_attn_case(2, 2, 1, 64, torch.float32, [20, 24], [1, 1], seed=16)
    out, _ = oracle.attn(inp.q, inp.k_pages, inp.v_pages, inp.block_table, inp.seq_lens, inp.q_lens)
    for pgi in inp.block_table[1][:2]:
        inp.v_pages[int(pgi)] = 1e6                      # sentinel in sequence 1's pages
    out2, _ = oracle.attn(inp.q, inp.k_pages, inp.v_pages, inp.block_table, inp.seq_lens, inp.q_lens)
    np.testing.assert_array_equal(out[0], out2[0])
    assert np.abs(out2[1]).max() > 1e5


def test_chunk_equals_sequence_of_decodes_and_is_causal():
    n, L = 9, 41
    inp = wl.small_attn_case(1, 6, 2, 64, torch.bfloat16, [L], [n], seed=17)
    out, _ = oracle.attn(inp.q, inp.k_pages, inp.v_pages, inp.block_table, inp.seq_lens, inp.q_lens)
    for i in range(n):
        one = torch.tensor([L - n + i + 1], dtype=torch.int32)
        oi, _ = oracle.attn(inp.q[i:i + 1], inp.k_pages, inp.v_pages, inp.block_table, one,
                            torch.tensor([1], dtype=torch.int32))
        np.testing.assert_array_equal(out[i], oi[0])
    # poisoning K/V at positions after a row's own position leaves that row bit-identical
    i = 4
    pos = L - n + i
    k2, v2 = inp.k_pages.clone(), inp.v_pages.clone()
    for j in range(pos + 1, L):
        pg = int(inp.block_table[0, j // P])
        k2[pg, :, j % P] = float("nan")
        v2[pg, :, j % P] = float("nan")
    out2, _ = oracle.attn(inp.q, k2, v2, inp.block_table, inp.seq_lens, inp.q_lens)
    np.testing.assert_array_equal(out[:i + 1], out2[:i + 1])
    assert np.isnan(out2[i + 1:]).all()


def test_gqa_head_sharing():
    inp = wl.small_attn_case(1, 6, 2, 64, torch.float32, [27], [1], seed=18)
    inp.q[:] = inp.q[:, :1]                              # every head gets the same query row
    out, _ = oracle.attn(inp.q, inp.k_pages, inp.v_pages, inp.block_table, inp.seq_lens, inp.q_lens)
    for h in (1, 2):
        np.testing.assert_array_equal(out[0, 0], out[0, h])    # heads 0..2 -> kv head 0
    for h in (4, 5):
        np.testing.assert_array_equal(out[0, 3], out[0, h])    # heads 3..5 -> kv head 1
    assert np.abs(out[0, 0] - out[0, 3]).max() > 1e-3


def test_bf16_inputs_are_widened_exactly():
    inp = wl.small_attn_case(1, 2, 2, 64, torch.bfloat16, [18], [1], seed=19)
    out, _ = oracle.attn(inp.q, inp.k_pages, inp.v_pages, inp.block_table, inp.seq_lens, inp.q_lens)
    f32 = wl.AttnInputs(inp.shape, inp.q.float(), inp.k_pages.float(), inp.v_pages.float(),
                        inp.block_table, inp.seq_lens, inp.q_lens)
    out32, _ = oracle.attn(f32.q, f32.k_pages, f32.v_pages, f32.block_table, f32.seq_lens, f32.q_lens)
    np.testing.assert_array_equal(out, out32)


def test_split_merge_identity():
    """Merging (m, l, o~) partials over any partition of the keys gives the unsplit result."""
    L = 53
    inp = wl.small_attn_case(1, 2, 1, 64, torch.float32, [L], [1], seed=20)
    out, _ = oracle.attn(inp.q, inp.k_pages, inp.v_pages, inp.block_table, inp.seq_lens, inp.q_lens)
    Kd, Vd = dense_kv(inp, 0)
    q = inp.q.to(torch.float64).numpy()[0, 1]
    s = (Kd[:, 0] @ q) / math.sqrt(64)
    parts = [(0, 16), (16, 17), (17, 48), (48, 53)]
    ms = [s[a:b].max() for a, b in parts]
    ls = [np.exp(s[a:b] - m).sum() for (a, b), m in zip(parts, ms)]
    os_ = [np.exp(s[a:b] - m) @ Vd[a:b, 0] for (a, b), m in zip(parts, ms)]
    m = max(ms)
    l = sum(li * math.exp(mi - m) for li, mi in zip(ls, ms))
    o = sum(oi * math.exp(mi - m) for oi, mi in zip(os_, ms)) / l
    np.testing.assert_allclose(out[0, 1], o, atol=1e-14)


def test_bad_lengths_and_pages_are_reported_not_computed():
    inp = wl.small_attn_case(2, 2, 1, 64, torch.float32, [5, 20], [8, 1], seed=21)   # seq_len < q_len
    out, st = oracle.attn(inp.q, inp.k_pages, inp.v_pages, inp.block_table, inp.seq_lens, inp.q_lens)
    assert st & oracle.BAD_SEQ_LEN
    assert (out[:8] == 0).all() and np.abs(out[8]).max() > 0
    inp = wl.small_attn_case(1, 2, 1, 64, torch.float32, [20], [1], seed=22)
    inp.block_table[0, 1] = inp.num_pages + 5
    _, st = oracle.attn(inp.q, inp.k_pages, inp.v_pages, inp.block_table, inp.seq_lens, inp.q_lens)
    assert st & oracle.BAD_PAGE
