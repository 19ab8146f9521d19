"""GPU parity of arb_policy, arb_route_classes and arb_kv_append against the oracle (through the C ABI)."""
import numpy as np
import pytest
import torch

from oracle import oracle
from paper_2512_05033_b200 import workloads as wl
from tests import helpers as H

pytestmark = pytest.mark.gpu
BF, F32 = torch.bfloat16, torch.float32


def _scores(n, seed, quantised=False):
    g = torch.Generator().manual_seed(seed)
    sd, st = torch.rand(n, generator=g), torch.rand(n, generator=g)
    if quantised:   # many exact ties, for the tie rules
        sd, st = torch.round(sd * 16) / 16, torch.round(st * 16) / 16
    return sd, st


@pytest.mark.parametrize("n", [1, 31, 256, 257, 1000, 5000])
@pytest.mark.parametrize("quantised", [False, True])
def test_policies_match_oracle(n, quantised):
    from paper_2512_05033_b200 import binding
    c = H.ctx()
    sd, st = _scores(n, 40 + n, quantised)
    dsd, dst = sd.cuda(), st.cuda()
    stats = c.new_policy_stats("cuda")
    cases = [(binding.POLICY_RSD, 0.3, 0), (binding.POLICY_RSD, 0.5, 0), (binding.POLICY_RSD, 0.7, 0),
             (binding.POLICY_ORACLE_THRESHOLD, 0.0, 0), (binding.POLICY_ORACLE_THRESHOLD, 0.25, 0),
             (binding.POLICY_ORACLE_THRESHOLD, -0.125, 0), (binding.POLICY_ORACLE_ARGMAX, 0.0, 0),
             (binding.POLICY_ORACLE_BUDGET, 0.0, 0), (binding.POLICY_ORACLE_BUDGET, 0.0, max(1, n // 7)),
             (binding.POLICY_ORACLE_BUDGET, 0.0, n // 2 + 1), (binding.POLICY_ORACLE_BUDGET, 0.0, 2 * n)]
    for kind, tau, budget in cases:
        dec = c.policy(kind, dsd, dst, tau=tau, budget=budget, stats=stats)
        got = c.policy_stats(stats)
        ref, rs = oracle.policy(kind, sd, st, tau=tau, budget=budget)
        assert np.array_equal(dec.cpu().numpy(), ref), (kind, tau, budget)      # integer work: bit-exact
        assert (got["escalated"], got["wasted"]) == (rs["escalated"], rs["wasted"])
        assert abs(got["realised"] - rs["realised"]) <= 1e-9 * max(1.0, abs(rs["realised"]))
        assert abs(got["gain"] - rs["gain"]) <= 1e-9 * max(1.0, abs(rs["gain"]))
    assert c.poll_status() == 0


def test_policy_without_target_scores_and_argument_checks():
    from paper_2512_05033_b200 import binding
    c = H.ctx()
    sd, st = _scores(100, 3)
    dec = c.policy(binding.POLICY_RSD, sd.cuda(), None, tau=0.5)
    ref, _ = oracle.policy(oracle.POLICY_RSD, sd, None, tau=0.5)
    assert np.array_equal(dec.cpu().numpy(), ref)
    with pytest.raises(binding.ArbError):
        c.policy(binding.POLICY_ORACLE_THRESHOLD, sd.cuda(), None)
    with pytest.raises(binding.ArbError):
        c.policy(binding.POLICY_RSD, sd.cuda(), None, stats=c.new_policy_stats("cuda"))
    with pytest.raises(binding.ArbError):
        c.policy(7, sd.cuda(), st.cuda())


@pytest.mark.parametrize("dtype", [F32, BF])
@pytest.mark.parametrize("C,H_", [(2, 256), (4, 3584), (10, 3584), (16, 264)])
def test_class_heads_match_oracle(dtype, C, H_):
    from paper_2512_05033_b200 import binding
    c = H.ctx()
    g = torch.Generator().manual_seed(C * 1000 + H_)
    S = 37
    hidden = torch.randn(S, H_, generator=g).to(dtype)
    w = (torch.randn(C, H_, generator=g) / H_ ** 0.5).to(dtype)
    b = (torch.randn(C, generator=g) * 0.3).tolist()
    for tau in (0.3, 0.5, 0.7):
        probs, scores, dec = c.route_classes(binding.HEAD_SOFTMAX, hidden.cuda(), w.cuda(), b, tau)
        p_ref, s_ref, d_ref = oracle.route_classes(oracle.HEAD_SOFTMAX, hidden, w, np.float32(b), tau)
        assert np.abs(probs.cpu().numpy() - p_ref).max() <= 1e-5
        assert np.abs(scores.cpu().numpy() - s_ref).max() <= 1e-5
        clear = np.abs(s_ref - tau) > 1e-3
        assert np.array_equal(dec.cpu().numpy()[clear], d_ref[clear])
    cuts = sorted((torch.randn(C - 1, generator=g)).tolist())
    bo = [0.1] + cuts
    probs, scores, dec = c.route_classes(binding.HEAD_ORDINAL, hidden.cuda(), w[0].contiguous().cuda(), bo, 0.5)
    p_ref, s_ref, d_ref = oracle.route_classes(oracle.HEAD_ORDINAL, hidden, w[:1], np.float32(bo), 0.5)
    assert np.abs(probs.cpu().numpy() - p_ref).max() <= 1e-5 and np.abs(scores.cpu().numpy() - s_ref).max() <= 1e-5
    clear = np.abs(s_ref - 0.5) > 1e-3
    assert np.array_equal(dec.cpu().numpy()[clear], d_ref[clear])
    assert c.poll_status() == 0


def test_two_class_head_equals_the_default_router():
    from paper_2512_05033_b200 import binding
    c = H.ctx()
    r = wl.make_router_inputs(32, 3584, BF, seed=3, b_std=0.1 ** 0.5)
    w2 = torch.stack([torch.zeros_like(r.w), r.w]).contiguous()
    _, s2, d2 = c.route_classes(binding.HEAD_SOFTMAX, r.hidden.cuda(), w2.cuda(), [0.0, r.b], 0.5)
    s1, d1 = c.route(r.hidden.cuda(), r.w.cuda(), r.b, 0.5)
    assert (s1 - s2).abs().max().item() <= 1e-6
    clear = (s1 - 0.5).abs() > 1e-3
    assert torch.equal(d1[clear], d2[clear])


APPEND_CASES = [
    # (B, Hkv, D, dtype, seq_lens, new_lens)
    (3, 2, 64, F32, [40, 17, 96], [5, 0, 33]),
    (4, 2, 128, BF, [1000, 15, 16, 1], [1, 1, 1, 1]),              # one decode token each, page boundaries
    (5, 4, 128, BF, [2048, 700, 33, 5000, 64], [128, 16, 0, 77, 100]),   # step chunks
    (2, 8, 128, F32, [300, 31], [17, 2]),
    (1, 1, 64, BF, [0], [50]),                                       # an empty cache
]


@pytest.mark.parametrize("case", APPEND_CASES)
def test_kv_append_matches_oracle(case):
    B, Hkv, D, dt, sl, nl = case
    c = H.ctx()
    inp = wl.small_attn_case(B, Hkv, Hkv, D, dt, sl, [1] * B, seed=300 + B + D, extra_tokens=max(nl) + 16)
    seq = torch.tensor(sl, dtype=torch.int32)
    new = torch.tensor(nl, dtype=torch.int32)
    g = torch.Generator().manual_seed(17)
    k_new = torch.randn(sum(nl), Hkv, D, generator=g).to(dt)
    v_new = torch.randn(sum(nl), Hkv, D, generator=g).to(dt)
    kp, vp, dseq = inp.k_pages.cuda(), inp.v_pages.cuda(), seq.cuda()
    c.kv_append(k_new.cuda(), v_new.cuda(), inp.block_table.cuda(), dseq, new.cuda(), kp, vp)
    k_ref, v_ref, sl_ref, st = oracle.kv_append(k_new, v_new, inp.block_table, seq, new, inp.k_pages, inp.v_pages)
    assert st == 0 and c.poll_status() == 0
    assert torch.equal(kp.cpu(), k_ref) and torch.equal(vp.cpu(), v_ref)            # byte work: bit-exact
    assert np.array_equal(dseq.cpu().numpy(), sl_ref)


def test_kv_append_leaves_bad_sequences_alone():
    from paper_2512_05033_b200 import binding
    c = H.ctx()
    inp = wl.small_attn_case(3, 2, 2, 128, BF, [40, 17, 96], [1, 1, 1], seed=77, extra_tokens=32)
    cap = inp.block_table.shape[1] * 16
    new = torch.tensor([5, cap, 3], dtype=torch.int32)
    bt = inp.block_table.clone()
    bt[2, 96 // 16] = inp.k_pages.shape[0] + 9                        # sequence 2 points outside the pool
    k_new = torch.ones(int(new.sum()), 2, 128, dtype=BF)
    seq = inp.seq_lens.clone()
    kp, vp, dseq = inp.k_pages.cuda(), inp.v_pages.cuda(), seq.cuda()
    c.kv_append(k_new.cuda(), k_new.cuda(), bt.cuda(), dseq, new.cuda(), kp, vp)
    k_ref, v_ref, sl_ref, st = oracle.kv_append(k_new, k_new, bt, seq, new, inp.k_pages, inp.v_pages)
    bits = c.poll_status()
    assert bits == (binding.DEV_BAD_SEQ_LEN | binding.DEV_BAD_PAGE) == st
    assert torch.equal(kp.cpu(), k_ref) and torch.equal(vp.cpu(), v_ref)
    assert list(dseq.cpu().numpy()) == list(sl_ref) == [45, 17, 96]


def test_one_round_of_the_step_loop_matches_oracle():
    """Algorithm 1, one round for a small batch: the draft step's K/V are appended, the router scores the
    step (chunk attention over the grown cache, then the head on hidden rows), escalated steps are rolled
    back, and the target's step overwrites the same slots before the next attention call."""
    c = H.ctx()
    B, Hq, Hkv, D = 4, 8, 2, 128
    prefix, step = [700, 64, 2500, 33], [40, 16, 128, 9]
    inp = wl.small_attn_case(B, Hq, Hkv, D, BF, prefix, step, seed=91, extra_tokens=160)
    g = torch.Generator().manual_seed(5)
    new = torch.tensor(step, dtype=torch.int32)
    kd, vd = torch.randn(sum(step), Hkv, D, generator=g).to(BF), torch.randn(sum(step), Hkv, D, generator=g).to(BF)
    kt, vt = torch.randn(sum(step), Hkv, D, generator=g).to(BF), torch.randn(sum(step), Hkv, D, generator=g).to(BF)
    r = wl.make_router_inputs(B, 256, BF, seed=9)
    # ---- oracle
    k1, v1, sl1, _ = oracle.kv_append(kd, vd, inp.block_table, inp.seq_lens, new, inp.k_pages, inp.v_pages)
    o1, _ = oracle.attn(inp.q, k1, v1, inp.block_table, sl1, new)
    s_ref, d_ref = oracle.route(r.hidden, r.w, 0.0, 0.5)
    sl2, _ = oracle.rollback(sl1, new.numpy(), d_ref)
    new_t = new * torch.from_numpy(d_ref.astype(np.int32))              # only escalated sequences regenerate
    rows = torch.repeat_interleave(torch.from_numpy(d_ref.astype(bool)), new.long())
    k2, v2, sl3, _ = oracle.kv_append(kt[rows], vt[rows], inp.block_table, sl2, new_t, k1, v1)
    o2, _ = oracle.attn(inp.q[rows], k2, v2, inp.block_table, sl3, new_t)
    # ---- device, lengths never leave it
    kp, vp, seq = inp.k_pages.cuda(), inp.v_pages.cuda(), inp.seq_lens.cuda()
    bt, dnew = inp.block_table.cuda(), new.cuda()
    c.kv_append(kd.cuda(), vd.cuda(), bt, seq, dnew, kp, vp)
    out1 = c.attn(inp.q.cuda(), kp, vp, bt, seq, dnew, max(step))
    scores, dec = c.route(r.hidden.cuda(), r.w.cuda(), 0.0, 0.5)
    assert np.array_equal(dec.cpu().numpy(), d_ref)                      # scores here are far from tau
    c.rollback(seq, dnew, dec)
    dnew_t = dnew * dec.to(torch.int32)
    c.kv_append(kt[rows].cuda(), vt[rows].cuda(), bt, seq, dnew_t, kp, vp)
    out2 = c.attn(inp.q[rows].cuda(), kp, vp, bt, seq, dnew_t, max(step))
    assert c.poll_status() == 0
    assert np.array_equal(seq.cpu().numpy(), sl3)
    assert torch.equal(kp.cpu(), k2) and torch.equal(vp.cpu(), v2)
    H.assert_close(out1.double().cpu().numpy(), o1, BF, tight=3e-3)
    H.assert_close(out2.double().cpu().numpy(), o2, BF, tight=3e-3)


@pytest.mark.parametrize("n,ties", [(2, False), (255, False), (256, True), (1000, True), (5000, False), (20000, True)])
def test_spearman_matches_oracle(n, ties):
    import math
    c = H.ctx()
    g = torch.Generator().manual_seed(n)
    x = torch.randn(n, generator=g)
    y = 0.2 * x + torch.randn(n, generator=g)
    if ties:
        x, y = torch.round(x * 4) / 4, torch.round(y * 3) / 3
    ref = oracle.spearman(x, y)
    got = float(c.spearman(x.cuda(), y.cuda()).item())
    assert abs(got - ref) <= 1e-12, (got, ref)        # same ranks; fp64 sums in another order
    const = float(c.spearman(torch.ones(n).cuda(), y.cuda()).item())
    assert math.isnan(const) and math.isnan(oracle.spearman(torch.ones(n), y))
    assert c.poll_status() == 0


@pytest.mark.parametrize("dtype,D", [(BF, 128), (F32, 128), (BF, 64), (F32, 64)])
def test_quantising_append_matches_oracle(dtype, D):
    c = H.ctx()
    B, Hkv = 4, 2
    sl, nl = [100, 15, 16, 0], [33, 1, 17, 40]
    inp = wl.small_attn_case(B, Hkv, Hkv, D, dtype, sl, [1] * B, seed=640 + D, extra_tokens=64)
    g = torch.Generator().manual_seed(19)
    # values across the whole range of the format: subnormal codes, ties, saturation
    k_new = (torch.randn(sum(nl), Hkv, D, generator=g) * torch.logspace(-4, 2.5, sum(nl)).view(-1, 1, 1)).to(dtype)
    v_new = torch.randn(sum(nl), Hkv, D, generator=g).to(dtype)
    k_new[0, 0, :8] = torch.tensor([1.0625, 1.1875, 500.0, -1e6, 2.0 ** -10, 3 * 2.0 ** -10, 0.0, -0.0]).to(dtype)
    kc = torch.randint(0, 127, inp.k_pages.shape, generator=g, dtype=torch.uint8)
    vc = torch.randint(0, 127, inp.k_pages.shape, generator=g, dtype=torch.uint8)
    seq, new = torch.tensor(sl, dtype=torch.int32), torch.tensor(nl, dtype=torch.int32)
    dk, dv, dseq = kc.cuda(), vc.cuda(), seq.cuda()
    c.kv_append_e4m3(k_new.cuda(), v_new.cuda(), 1.0, 1 / 0.03, inp.block_table.cuda(), dseq, new.cuda(), dk, dv)
    k_ref, v_ref, sl_ref, st = oracle.kv_append_e4m3(k_new, v_new, inp.block_table, seq, new, kc, vc, 1.0, 1 / 0.03)
    assert st == 0 and c.poll_status() == 0
    assert torch.equal(dk.cpu(), k_ref) and torch.equal(dv.cpu(), v_ref)          # codes: bit-exact
    assert np.array_equal(dseq.cpu().numpy(), sl_ref)
