"""arb_decode_step -- one decode token in one launch (cache write, attention, combine, length update) -- against
the oracle's kv_append followed by its attention: pools bit for bit, lengths exact, rows within tolerance."""
import numpy as np
import pytest
import torch

from oracle import oracle
from paper_2512_05033_b200 import workloads as wl
from tests import helpers as H

pytestmark = pytest.mark.gpu
BF, F32 = torch.bfloat16, torch.float32


def _new_rows(inp, n, seed):
    Hkv, D = inp.k_pages.shape[1], inp.k_pages.shape[3]
    return (wl.normal((n, Hkv, D), 1.0, inp.q.dtype, "cpu", seed), wl.normal((n, Hkv, D), 1.0, inp.q.dtype, "cpu", seed + 1))


def _run(c, inp, k_new, v_new, dev=None):
    """One step on the device and through the oracle.  `inp.seq_lens` are the lengths BEFORE the token.
    Returns (out, pools, lens, bits) of the device and (out, pools, lens, status) of the oracle."""
    d = dev or inp.to("cuda")
    out = torch.full_like(d.q, float("nan"))
    c.decode_step(d.q, k_new.cuda(), v_new.cuda(), d.k_pages, d.v_pages, d.block_table, d.seq_lens, d.q_lens, out=out)
    bits = c.poll_status()
    ok, ov, osl, st = oracle.kv_append(k_new, v_new, inp.block_table, inp.seq_lens, inp.q_lens, inp.k_pages, inp.v_pages)
    ref, st2 = oracle.attn(inp.q, ok, ov, inp.block_table, osl, inp.q_lens)
    return (out, d, bits), (ref, ok, ov, osl, st | st2)


def _same_bits(a, b):
    """Bit-for-bit equality (pools may hold NaN on purpose)."""
    it = torch.int16 if a.element_size() == 2 else torch.int32
    return torch.equal(a.cpu().contiguous().view(it), b.cpu().contiguous().view(it))


def _check(got, exp, dt, tight):
    (out, d, bits), (ref, ok, ov, osl, st) = got, exp
    assert bits == 0 and st == 0
    assert np.array_equal(d.seq_lens.cpu().numpy(), osl)
    assert _same_bits(d.k_pages, ok) and _same_bits(d.v_pages, ov)
    H.assert_close(out.double().cpu().numpy(), ref, dt, tight=tight if dt == BF else None)


STEP_CASES = [
    # (B, Hq, Hkv, D, dtype, lengths before the token, q_lens)
    (3, 12, 2, 128, BF, [15, 16, 17], [1, 1, 1]),                       # last slot of a page, first slot of a new page
    (4, 12, 2, 128, BF, [0, 1, 31, 32], [1, 1, 1, 1]),                  # an empty sequence: the token is its only key
    (8, 12, 2, 128, BF, [1025, 2000, 3001, 777, 4096, 1, 640, 5555], [1] * 8),   # draft-shaped, ragged
    (4, 32, 8, 128, BF, [4100, 9000, 33, 12000], [1, 1, 1, 1]),         # target-shaped heads
    (2, 28, 4, 128, BF, [3000, 150], [1, 1]),                           # g = 7
    (5, 16, 2, 128, BF, [2100, 5, 900, 77, 4000], [1, 0, 1, 0, 1]),     # g = 8, idle slots
    (1, 5, 1, 128, BF, [40000], [1]),                                   # one long sequence over every CTA
    (2, 8, 8, 128, BF, [260, 100], [1, 1]),                             # g = 1
    (16, 32, 8, 128, BF, [100 * i + 7 for i in range(16)], [1] * 16),   # many short segments per CTA
    (1, 8, 2, 64, F32, [512], [1]),                                     # the tiny config's shape: two launches inside
    (2, 6, 2, 64, BF, [700, 70], [1, 1]),                               # bf16, head_dim 64: two launches inside
]


@pytest.mark.parametrize("case", STEP_CASES)
def test_decode_step_matches_append_then_attention(case):
    B, Hq, Hkv, D, dt, sl, ql = case
    inp = wl.small_attn_case(B, Hq, Hkv, D, dt, sl, ql, seed=800 + len(sl) + Hq, extra_tokens=4)
    k_new, v_new = _new_rows(inp, sum(ql), 8100 + Hq)
    single = dt == BF and D == 128
    _check(*_run(H.ctx(), inp, k_new, v_new), dt, 3e-3 if single else 1e-3)


def test_decode_step_over_stale_slots_after_a_rollback():
    """A rejected step leaves its slots behind: beyond the length they hold anything (NaN here).  The next token
    overwrites the first of them and must see none of the others."""
    c = H.ctx()
    sl = [3000, 45, 640, 16]
    inp = wl.small_attn_case(4, 12, 2, 128, BF, sl, [1] * 4, seed=77, extra_tokens=40)
    for b, L in enumerate(sl):                       # poison everything from position L on, 30 tokens deep
        for pos in range(L, L + 30):
            page = int(inp.block_table[b, pos // 16])
            inp.k_pages[page, :, pos % 16, :] = float("nan")
            inp.v_pages[page, :, pos % 16, :] = float("nan")
    k_new, v_new = _new_rows(inp, 4, 91)
    _check(*_run(c, inp, k_new, v_new), BF, 3e-3)


def test_decode_step_chain_in_place():
    """Twenty tokens in a row on the same cache: every call finds the lengths the previous one left, in place, with
    the set of active sequences changing from token to token; then the same chain replayed as one CUDA graph."""
    c = H.ctx()
    B, T = 6, 20
    inp = wl.small_attn_case(B, 12, 2, 128, BF, [500, 33, 2100, 0, 1500, 64], [1] * B, seed=78, extra_tokens=T + 2)
    g = torch.Generator().manual_seed(5)
    active = (torch.rand(T, B, generator=g) < 0.7).to(torch.int32)
    active[:, 0] = 1
    q = wl.normal((T, B, 12, 128), 1.0, BF, "cpu", 79)
    kn = wl.normal((T, B, 2, 128), 1.0, BF, "cpu", 80)
    vn = wl.normal((T, B, 2, 128), 1.0, BF, "cpu", 81)
    d = inp.to("cuda")
    start = (d.k_pages.clone(), d.v_pages.clone(), d.seq_lens.clone())
    dq, dk, dv, dact = q.cuda(), kn.cuda(), vn.cuda(), active.cuda()
    outs = [torch.full((B, 12, 128), float("nan"), dtype=BF, device="cuda") for _ in range(T)]

    def chain():
        for t in range(T):
            n = int(active[t].sum())
            p = c.params_for(dq[t][:n], d.k_pages, d.block_table, 1)
            c.decode_step(dq[t][:n], dk[t][:n], dv[t][:n], d.k_pages, d.v_pages, d.block_table, d.seq_lens, dact[t],
                          out=outs[t][:n], params=p)

    chain()
    assert c.poll_status() == 0
    k, v, sl = inp.k_pages, inp.v_pages, inp.seq_lens.numpy()
    refs = []
    for t in range(T):
        n = int(active[t].sum())
        k, v, sl, st = oracle.kv_append(kn[t][:n], vn[t][:n], inp.block_table, sl, active[t], k, v)
        ref, st2 = oracle.attn(q[t][:n], k, v, inp.block_table, sl, active[t])
        assert st == 0 and st2 == 0
        refs.append(ref)
        H.assert_close(outs[t][:n].double().cpu().numpy(), ref, BF, tight=3e-3)
    assert np.array_equal(d.seq_lens.cpu().numpy(), sl)
    assert torch.equal(d.k_pages.cpu(), k) and torch.equal(d.v_pages.cpu(), v)
    # the same chain as a graph, replayed twice from the starting state
    eager = [o.clone() for o in outs]
    gr = torch.cuda.CUDAGraph()
    for t_, s_ in zip((d.k_pages, d.v_pages, d.seq_lens), start):
        t_.copy_(s_)
    with torch.cuda.graph(gr):
        chain()
    for rep in range(2):
        for t_, s_ in zip((d.k_pages, d.v_pages, d.seq_lens), start):
            t_.copy_(s_)
        for o in outs:
            o.fill_(float("nan"))
        gr.replay()
        torch.cuda.synchronize()
        for t in range(T):
            n = int(active[t].sum())
            assert torch.equal(outs[t][:n], eager[t][:n]), (rep, t)
        assert np.array_equal(d.seq_lens.cpu().numpy(), sl)
    assert c.poll_status() == 0


def test_decode_step_refuses_what_does_not_fit():
    """A token that does not fit under the block-table row: the sequence is left untouched, its row is zero, the bit
    is raised; a new row whose page lies outside the pool is not written and the length stays."""
    from paper_2512_05033_b200 import binding
    c = H.ctx()
    inp = wl.small_attn_case(3, 12, 2, 128, BF, [100, 64, 300], [1, 1, 1], seed=83)
    inp.seq_lens[1] = inp.block_table.shape[1] * 16          # full: one more token does not fit
    k_new, v_new = _new_rows(inp, 3, 84)
    d = inp.to("cuda")
    k0, v0 = d.k_pages.clone(), d.v_pages.clone()
    out = torch.full_like(d.q, float("nan"))
    c.decode_step(d.q, k_new.cuda(), v_new.cuda(), d.k_pages, d.v_pages, d.block_table, d.seq_lens, d.q_lens, out=out)
    assert c.poll_status() == binding.DEV_BAD_SEQ_LEN
    ok, ov, osl, st = oracle.kv_append(k_new, v_new, inp.block_table, inp.seq_lens, inp.q_lens, inp.k_pages, inp.v_pages)
    assert st == oracle.BAD_SEQ_LEN
    assert np.array_equal(d.seq_lens.cpu().numpy(), osl)
    assert torch.equal(d.k_pages.cpu(), ok) and torch.equal(d.v_pages.cpu(), ov)
    assert float(out[1].abs().max()) == 0.0
    keep = torch.tensor([1, 0, 1], dtype=torch.int32)
    ref, _ = oracle.attn(inp.q[[0, 2]], ok, ov, inp.block_table, osl, keep)
    H.assert_close(out[[0, 2]].double().cpu().numpy(), ref, BF, tight=3e-3)
    # a page id outside the pool at the new row's place
    inp2 = wl.small_attn_case(2, 12, 2, 128, BF, [100, 47], [1, 1], seed=85)
    inp2.block_table[1, 47 // 16] = inp2.k_pages.shape[0] + 5
    d2 = inp2.to("cuda")
    k2 = d2.k_pages.clone()
    kn2, vn2 = _new_rows(inp2, 2, 86)
    out2 = c.decode_step(d2.q, kn2.cuda(), vn2.cuda(), d2.k_pages, d2.v_pages, d2.block_table, d2.seq_lens, d2.q_lens)
    assert c.poll_status() == binding.DEV_BAD_PAGE
    assert d2.seq_lens.cpu().tolist() == [101, 47]
    assert torch.isfinite(out2.float()).all()
    changed = (d2.k_pages != k2).flatten(1).any(1).nonzero().flatten().cpu().tolist()
    assert changed == [int(inp2.block_table[0, 100 // 16])]   # only sequence 0's page was written
    # host-side refusals
    p = c.params_for(d2.q, d2.k_pages, d2.block_table, 1, flags=binding.ATTN_OVERLAP_PREVIOUS)
    with pytest.raises(binding.ArbError):
        c.decode_step(d2.q, kn2.cuda(), vn2.cuda(), d2.k_pages, d2.v_pages, d2.block_table, d2.seq_lens, d2.q_lens, params=p)


# ---- arb_decode_step_e4m3: the same token over an E4M3 cache -------------------------------------------------------

E4M3_STEP_CASES = [
    # (B, Hq, Hkv, lengths before the token, q_lens)
    (3, 12, 2, [15, 16, 17], [1, 1, 1]),
    (4, 12, 2, [0, 1, 31, 32], [1, 1, 1, 1]),
    (8, 12, 2, [1025, 2000, 3001, 777, 4096, 1, 640, 5555], [1] * 8),
    (4, 32, 8, [4100, 9000, 33, 12000], [1, 1, 1, 1]),
    (2, 28, 4, [3000, 150], [1, 1]),
    (5, 16, 2, [2100, 5, 900, 77, 4000], [1, 0, 1, 0, 1]),
    (1, 5, 1, [40000], [1]),
    (2, 8, 8, [260, 100], [1, 1]),
]
KS, VS = 0.011, 0.017     # N(0,1) values / scale reach about 400: the whole range of the format is used


def _e4m3_case(B, Hq, Hkv, sl, ql, seed, extra=4):
    inp = wl.small_attn_case(B, Hq, Hkv, 128, BF, sl, ql, seed=seed, extra_tokens=extra)
    kc = torch.from_numpy(oracle.e4m3_encode(inp.k_pages, 1 / KS))
    vc = torch.from_numpy(oracle.e4m3_encode(inp.v_pages, 1 / VS))
    for b in range(B):              # stale slots past the ends hold NaN codes: they must never reach the arithmetic
        for pos in range(sl[b], sl[b] + extra):
            page = int(inp.block_table[b, pos // 16])
            kc[page, :, pos % 16, :] = 0x7f
            vc[page, :, pos % 16, :] = 0xff
    return inp, kc, vc


@pytest.mark.parametrize("case", E4M3_STEP_CASES)
def test_decode_step_e4m3_matches_quantising_append_then_attention(case):
    B, Hq, Hkv, sl, ql = case
    inp, kc, vc = _e4m3_case(B, Hq, Hkv, sl, ql, 900 + len(sl) + Hq)
    k_new, v_new = _new_rows(inp, sum(ql), 9100 + Hq)
    k_new[0, 0, :4] = torch.tensor([1e4, -1e4, 0.0, 448 * KS])          # saturation on both sides, zero, the edge
    c = H.ctx()
    d = inp.to("cuda")
    dk, dv = kc.cuda(), vc.cuda()
    out = torch.full_like(d.q, float("nan"))
    c.decode_step_e4m3(d.q, k_new.cuda(), v_new.cuda(), dk, dv, KS, VS, 1 / KS, 1 / VS, d.block_table, d.seq_lens,
                       d.q_lens, out=out)
    assert c.poll_status() == 0
    ok, ov, osl, st = oracle.kv_append_e4m3(k_new, v_new, inp.block_table, inp.seq_lens, inp.q_lens, kc, vc, 1 / KS, 1 / VS)
    ref, st2 = oracle.attn_e4m3(inp.q, ok, ov, KS, VS, inp.block_table, osl, inp.q_lens)
    assert st == 0 and st2 == 0
    assert np.array_equal(d.seq_lens.cpu().numpy(), osl)
    assert torch.equal(dk.cpu(), ok) and torch.equal(dv.cpu(), ov)       # codes: bit for bit
    H.assert_close(out.double().cpu().numpy(), ref, BF, tight=3e-3)


def test_decode_step_e4m3_chain_equals_the_two_calls():
    """Twelve tokens in a row, in place, then as one CUDA graph: codes and lengths equal those the two separate
    calls (arb_kv_append_e4m3, arb_attn_decode_e4m3) leave on a copy of the cache, rows equal the oracle's."""
    c = H.ctx()
    B, T = 5, 12
    inp, kc, vc = _e4m3_case(B, 12, 2, [500, 33, 2100, 0, 1500], [1] * B, 93, extra=T + 2)
    q = wl.normal((T, B, 12, 128), 1.0, BF, "cpu", 94)
    kn = wl.normal((T, B, 2, 128), 1.0, BF, "cpu", 95)
    vn = wl.normal((T, B, 2, 128), 1.0, BF, "cpu", 96)
    d = inp.to("cuda")
    dk, dv = kc.cuda(), vc.cuda()
    start = (dk.clone(), dv.clone(), d.seq_lens.clone())
    dq, dkn, dvn = q.cuda(), kn.cuda(), vn.cuda()
    outs = [torch.full((B, 12, 128), float("nan"), dtype=BF, device="cuda") for _ in range(T)]
    p = c.params_for(dq[0], dk, d.block_table, 1)

    def chain():
        for t in range(T):
            c.decode_step_e4m3(dq[t], dkn[t], dvn[t], dk, dv, KS, VS, 1 / KS, 1 / VS, d.block_table, d.seq_lens,
                               d.q_lens, out=outs[t], params=p)

    chain()
    assert c.poll_status() == 0
    k, v, sl = kc, vc, inp.seq_lens.numpy()
    for t in range(T):
        k, v, sl, st = oracle.kv_append_e4m3(kn[t], vn[t], inp.block_table, sl, inp.q_lens, k, v, 1 / KS, 1 / VS)
        ref, st2 = oracle.attn_e4m3(q[t], k, v, KS, VS, inp.block_table, sl, inp.q_lens)
        assert st == 0 and st2 == 0
        H.assert_close(outs[t].double().cpu().numpy(), ref, BF, tight=3e-3)
    assert np.array_equal(d.seq_lens.cpu().numpy(), sl)
    assert torch.equal(dk.cpu(), k) and torch.equal(dv.cpu(), v)
    # the two separate calls on a copy of the starting cache
    k2, v2, sl2 = (t_.clone() for t_ in start)
    for t in range(T):
        c.kv_append_e4m3(dkn[t], dvn[t], 1 / KS, 1 / VS, d.block_table, sl2, d.q_lens, k2, v2)
        two = c.attn_decode_e4m3(dq[t], k2, v2, KS, VS, d.block_table, sl2, d.q_lens)
        assert float((two.float() - outs[t].float()).abs().max()) <= 2e-2
    assert torch.equal(k2, dk) and torch.equal(v2, dv) and torch.equal(sl2, d.seq_lens)
    eager = [o.clone() for o in outs]
    gr = torch.cuda.CUDAGraph()
    for t_, s_ in zip((dk, dv, d.seq_lens), start):
        t_.copy_(s_)
    with torch.cuda.graph(gr):
        chain()
    for rep in range(2):
        for t_, s_ in zip((dk, dv, d.seq_lens), start):
            t_.copy_(s_)
        for o in outs:
            o.fill_(float("nan"))
        gr.replay()
        torch.cuda.synchronize()
        for t in range(T):
            assert torch.equal(outs[t], eager[t]), (rep, t)
        assert np.array_equal(d.seq_lens.cpu().numpy(), sl)


def test_decode_step_e4m3_refusals():
    """Host-side refusals, and a token that does not fit: sequence untouched, zero row, status bit."""
    from paper_2512_05033_b200 import binding
    c = H.ctx()
    inp, kc, vc = _e4m3_case(3, 12, 2, [100, 64, 300], [1, 1, 1], 97, extra=0)
    k_new, v_new = _new_rows(inp, 3, 98)
    d = inp.to("cuda")
    with pytest.raises(binding.ArbError):      # a scale that is not positive
        c.decode_step_e4m3(d.q, k_new.cuda(), v_new.cuda(), kc.cuda(), vc.cuda(), 0.0, VS, 1 / KS, 1 / VS, d.block_table,
                           d.seq_lens, d.q_lens)
    with pytest.raises(binding.ArbError):      # a series flag: the call writes the cache it reads
        p = c.params_for(d.q, kc.cuda(), d.block_table, 1, flags=binding.ATTN_OVERLAP_PREVIOUS)
        c.decode_step_e4m3(d.q, k_new.cuda(), v_new.cuda(), kc.cuda(), vc.cuda(), KS, VS, 1 / KS, 1 / VS, d.block_table,
                           d.seq_lens, d.q_lens, params=p)
    inp.seq_lens[1] = inp.block_table.shape[1] * 16          # full: one more token does not fit
    d = inp.to("cuda")
    dk, dv = kc.cuda(), vc.cuda()
    out = torch.full_like(d.q, float("nan"))
    c.decode_step_e4m3(d.q, k_new.cuda(), v_new.cuda(), dk, dv, KS, VS, 1 / KS, 1 / VS, d.block_table, d.seq_lens,
                       d.q_lens, out=out)
    assert c.poll_status() == binding.DEV_BAD_SEQ_LEN
    ok, ov, osl, st = oracle.kv_append_e4m3(k_new, v_new, inp.block_table, inp.seq_lens, inp.q_lens, kc, vc, 1 / KS, 1 / VS)
    assert st == oracle.BAD_SEQ_LEN
    assert np.array_equal(d.seq_lens.cpu().numpy(), osl)
    assert torch.equal(dk.cpu(), ok) and torch.equal(dv.cpu(), ov)
    assert float(out[1].abs().max()) == 0.0
    keep = torch.tensor([1, 0, 1], dtype=torch.int32)
    ref, _ = oracle.attn_e4m3(inp.q[[0, 2]], ok, ov, KS, VS, inp.block_table, osl, keep)
    H.assert_close(out[[0, 2]].double().cpu().numpy(), ref, BF, tight=3e-3)


# ---- arb_decode_step_i4: the same token over a 4-bit cache (per-row scales) ----------------------------------------

def _i4_case(B, Hq, Hkv, sl, ql, seed, extra=4, row_std=None):
    """Pools quantised by the oracle; slots past the ends hold nibble 0 (a code the format never writes) and NaN scales."""
    inp = wl.small_attn_case(B, Hq, Hkv, 128, BF, sl, ql, seed=seed, extra_tokens=extra)
    if row_std is not None:     # rows of very different magnitude: the per-row scales matter
        g = torch.Generator().manual_seed(seed + 1)
        for pool in (inp.k_pages, inp.v_pages):
            f = torch.exp(torch.randn(pool.shape[:3], generator=g) * row_std)[..., None]
            pool.copy_((pool.float() * f).to(pool.dtype))
    kc, ks = oracle.i4_encode(inp.k_pages)
    vc, vs = oracle.i4_encode(inp.v_pages)
    kc, vc, ks, vs = torch.from_numpy(kc), torch.from_numpy(vc), torch.from_numpy(ks), torch.from_numpy(vs)
    for b in range(B):
        for pos in range(sl[b], sl[b] + extra):
            page = int(inp.block_table[b, pos // 16])
            kc[page, :, pos % 16, :] = 0
            vc[page, :, pos % 16, :] = 0
            ks[page, :, pos % 16] = float("nan")
            vs[page, :, pos % 16] = float("nan")
    return inp, kc, vc, ks, vs


def _i4_close(out, ref, v_scales):
    """The bar of the other decode tests (bf16 rounding of the output, 2^-8 |ref|, plus 3e-3 for N(0,1) values), its
    absolute part scaled with the size of the values: the weights reach the tensor core rounded to bf16, an error of
    2^-9 of weight x value per key, and the largest value of a pool of N(0,1) rows is about 4.5."""
    s = np.asarray(v_scales, dtype=np.float64)
    vmax = float(np.nanmax(s)) * 7.0
    err = np.abs(out.double().cpu().numpy() - ref)
    assert np.isfinite(out.float().cpu().numpy()).all()
    bar = 2.0 ** -8 * np.abs(ref) + 3e-3 * max(1.0, vmax / 4.5)
    assert (err <= bar).all(), f"error {err.max():.3e} above the bar (largest value {vmax:.1f})"


def _same_f32_bits(a, b):
    return torch.equal(a.cpu().contiguous().view(torch.int32), torch.as_tensor(np.asarray(b)).contiguous().view(torch.int32))


@pytest.mark.parametrize("case", E4M3_STEP_CASES)
def test_decode_step_i4_matches_quantising_append_then_attention(case):
    B, Hq, Hkv, sl, ql = case
    inp, kc, vc, ks, vs = _i4_case(B, Hq, Hkv, sl, ql, 950 + len(sl) + Hq, row_std=1.0 if B % 2 else None)
    k_new, v_new = _new_rows(inp, sum(ql), 9700 + Hq)
    k_new[0, 0, :] = 0.0                                             # a row of zeros: scale 0, codes 0
    v_new[0, 0, :8] = torch.tensor([7, -7, 3.5, 2.5, -0.5, 0.49, 6.5, -6.5])   # ties (when the row's max is 7)
    v_new[0, 0, 8:] = 0.0
    c = H.ctx()
    d = inp.to("cuda")
    dk, dv, dks, dvs = kc.cuda(), vc.cuda(), ks.cuda(), vs.cuda()
    out = torch.full_like(d.q, float("nan"))
    c.decode_step_i4(d.q, k_new.cuda(), v_new.cuda(), dk, dv, dks, dvs, d.block_table, d.seq_lens, d.q_lens, out=out)
    assert c.poll_status() == 0
    ok, ov, oks, ovs, osl, st = oracle.kv_append_i4(k_new, v_new, inp.block_table, inp.seq_lens, inp.q_lens, kc, vc, ks, vs)
    ref, st2 = oracle.attn_i4(inp.q, _live(ok, oks, inp, osl)[0], _live(ov, ovs, inp, osl)[0], _live(ok, oks, inp, osl)[1],
                              _live(ov, ovs, inp, osl)[1], inp.block_table, osl, inp.q_lens)
    assert st == 0 and st2 == 0
    assert np.array_equal(d.seq_lens.cpu().numpy(), osl)
    assert torch.equal(dk.cpu(), ok) and torch.equal(dv.cpu(), ov)                    # codes: bit for bit
    assert _same_f32_bits(dks, oks) and _same_f32_bits(dvs, ovs)                      # scales: bit for bit (NaN included)
    _i4_close(out, ref, ovs)


def _live(codes, scales, inp, lens):
    """The pools with every slot past a sequence's end given a finite scale (the oracle's attention decodes whole pools
    before it looks at the lengths; what those slots hold must not matter to the result)."""
    s = torch.as_tensor(np.asarray(scales)).clone()
    s[torch.isnan(s)] = 0.0
    return codes, s


def test_decode_step_i4_chain_in_place_and_as_a_graph():
    c = H.ctx()
    B, T = 5, 10
    inp, kc, vc, ks, vs = _i4_case(B, 12, 2, [500, 33, 2100, 0, 1500], [1] * B, 961, extra=T + 2, row_std=0.7)
    q = wl.normal((T, B, 12, 128), 1.0, BF, "cpu", 962)
    kn = wl.normal((T, B, 2, 128), 1.0, BF, "cpu", 963)
    vn = wl.normal((T, B, 2, 128), 3.0, BF, "cpu", 964)
    d = inp.to("cuda")
    pools = [kc.cuda(), vc.cuda(), ks.cuda(), vs.cuda()]
    start = [t.clone() for t in pools] + [d.seq_lens.clone()]
    dq, dkn, dvn = q.cuda(), kn.cuda(), vn.cuda()
    outs = [torch.full((B, 12, 128), float("nan"), dtype=BF, device="cuda") for _ in range(T)]

    def chain():
        for t in range(T):
            c.decode_step_i4(dq[t], dkn[t], dvn[t], *pools, d.block_table, d.seq_lens, d.q_lens, out=outs[t])

    chain()
    assert c.poll_status() == 0
    k, v, sk, sv, sl = kc, vc, ks, vs, inp.seq_lens.numpy()
    for t in range(T):
        k, v, sk, sv, sl, st = oracle.kv_append_i4(kn[t], vn[t], inp.block_table, sl, inp.q_lens, k, v, sk, sv)
        ref, st2 = oracle.attn_i4(q[t], k, v, _live(k, sk, inp, sl)[1], _live(v, sv, inp, sl)[1], inp.block_table, sl, inp.q_lens)
        assert st == 0 and st2 == 0
        _i4_close(outs[t], ref, sv)
    assert np.array_equal(d.seq_lens.cpu().numpy(), sl)
    assert torch.equal(pools[0].cpu(), k) and torch.equal(pools[1].cpu(), v)
    assert _same_f32_bits(pools[2], sk) and _same_f32_bits(pools[3], sv)
    eager = [o.clone() for o in outs]
    gr = torch.cuda.CUDAGraph()
    for t_, s_ in zip(pools + [d.seq_lens], start):
        t_.copy_(s_)
    with torch.cuda.graph(gr):
        chain()
    for t_, s_ in zip(pools + [d.seq_lens], start):
        t_.copy_(s_)
    gr.replay()
    torch.cuda.synchronize()
    for t in range(T):
        assert torch.equal(outs[t], eager[t]), t


def test_decode_step_i4_refusals():
    from paper_2512_05033_b200 import binding
    c = H.ctx()
    inp, kc, vc, ks, vs = _i4_case(3, 12, 2, [100, 64, 300], [1, 1, 1], 971, extra=0)
    k_new, v_new = _new_rows(inp, 3, 972)
    inp.seq_lens[1] = inp.block_table.shape[1] * 16          # full: one more token does not fit
    d = inp.to("cuda")
    pools = [kc.cuda(), vc.cuda(), ks.cuda(), vs.cuda()]
    out = torch.full_like(d.q, float("nan"))
    c.decode_step_i4(d.q, k_new.cuda(), v_new.cuda(), *pools, d.block_table, d.seq_lens, d.q_lens, out=out)
    assert c.poll_status() == binding.DEV_BAD_SEQ_LEN
    ok, ov, oks, ovs, osl, st = oracle.kv_append_i4(k_new, v_new, inp.block_table, inp.seq_lens, inp.q_lens, kc, vc, ks, vs)
    assert st == oracle.BAD_SEQ_LEN
    assert np.array_equal(d.seq_lens.cpu().numpy(), osl)
    assert torch.equal(pools[0].cpu(), ok) and torch.equal(pools[1].cpu(), ov)
    assert _same_f32_bits(pools[2], oks) and _same_f32_bits(pools[3], ovs)
    assert float(out[1].abs().max()) == 0.0
    keep = torch.tensor([1, 0, 1], dtype=torch.int32)
    ref, _ = oracle.attn_i4(inp.q[[0, 2]], ok, ov, oks, ovs, inp.block_table, osl, keep)
    H.assert_close(out[[0, 2]].double().cpu().numpy(), ref, BF, tight=3e-3)
    with pytest.raises(binding.ArbError):      # scale pools are required: a null pool is refused by the library
        p = c.params_for(d.q, inp.k_pages, d.block_table, 1)
        st = binding.lib.arb_decode_step_i4(c._h, __import__("ctypes").byref(p), d.q.data_ptr(), k_new.cuda().data_ptr(),
                                            v_new.cuda().data_ptr(), pools[0].data_ptr(), pools[1].data_ptr(), None, None,
                                            d.block_table.data_ptr(), d.seq_lens.data_ptr(), d.q_lens.data_ptr(),
                                            out.data_ptr(), None)
        binding._check(st, "arb_decode_step_i4")


def test_kv_append_i4_prefill_then_tokens():
    """arb_kv_append_i4 writes a ragged batch of new rows (a prefix for an empty sequence, a step for others, none for
    one, one that does not fit), bit for bit like the oracle's encoder; arb_decode_step_i4 then runs on that cache."""
    from paper_2512_05033_b200 import binding
    c = H.ctx()
    sl = [0, 40, 1000, 31, 200]
    inp, kc, vc, ks, vs = _i4_case(5, 12, 2, sl, [1] * 5, 981, extra=70, row_std=0.5)
    new = torch.tensor([64, 17, 0, 1, 33], dtype=torch.int32)
    n = int(new.sum())
    kn = wl.normal((n, 2, 128), 1.0, BF, "cpu", 982)
    vn = wl.normal((n, 2, 128), 2.0, BF, "cpu", 983)
    kn[3] = 0.0                                   # rows of zeros
    d = inp.to("cuda")
    pools = [kc.cuda(), vc.cuda(), ks.cuda(), vs.cuda()]
    c.kv_append_i4(kn.cuda(), vn.cuda(), d.block_table, d.seq_lens, new.cuda(), *pools)
    assert c.poll_status() == 0
    ok, ov, oks, ovs, osl, st = oracle.kv_append_i4(kn, vn, inp.block_table, inp.seq_lens, new, kc, vc, ks, vs)
    assert st == 0 and np.array_equal(d.seq_lens.cpu().numpy(), osl)
    assert torch.equal(pools[0].cpu(), ok) and torch.equal(pools[1].cpu(), ov)
    assert _same_f32_bits(pools[2], oks) and _same_f32_bits(pools[3], ovs)
    # a token on top of it
    k1, v1 = _new_rows(inp, 5, 984)
    out = c.decode_step_i4(d.q, k1.cuda(), v1.cuda(), *pools, d.block_table, d.seq_lens, d.q_lens)
    assert c.poll_status() == 0
    ok, ov, oks, ovs, osl2, st = oracle.kv_append_i4(k1, v1, inp.block_table, osl, inp.q_lens, ok, ov, oks, ovs)
    ref, st2 = oracle.attn_i4(inp.q, ok, ov, _live(ok, oks, inp, osl2)[1], _live(ov, ovs, inp, osl2)[1], inp.block_table, osl2,
                              inp.q_lens)
    assert st == 0 and st2 == 0
    _i4_close(out, ref, ovs)
    assert torch.equal(pools[0].cpu(), ok) and _same_f32_bits(pools[3], ovs)
    # a sequence whose rows do not fit is left untouched, with the status bit
    too_many = torch.tensor([0, 0, 0, 0, inp.block_table.shape[1] * 16], dtype=torch.int32)
    before = [t.clone() for t in pools] + [d.seq_lens.clone()]
    big = wl.normal((int(too_many.sum()), 2, 128), 1.0, BF, "cuda", 985)
    c.kv_append_i4(big, big, d.block_table, d.seq_lens, too_many.cuda(), *pools)
    assert c.poll_status() == binding.DEV_BAD_SEQ_LEN
    for t_, b_ in zip(pools + [d.seq_lens], before):
        assert torch.equal(t_.view(torch.uint8) if t_.dtype == torch.float32 else t_, b_.view(torch.uint8) if b_.dtype == torch.float32 else b_)
