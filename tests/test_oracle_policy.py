"""Pins of the oracle's policy rules, C-way router heads and KV append (CPU only).

Nothing here restates the oracle's own code: decisions are checked against a hand-written table, against
brute force over every subset (the budgeted rule, Appendix B), against closed forms, against library
routines (scipy's softmax and expit) and against structural properties the paper states."""
import itertools
import math
from pathlib import Path

import numpy as np
import pytest
import torch
from scipy.special import expit, softmax

from oracle import oracle
from paper_2512_05033_b200 import workloads as wl

GOLDEN = Path(__file__).parent / "golden" / "policy_truth_table.txt"


def _table():
    rows = []
    for line in GOLDEN.read_text().splitlines():
        if line.strip() and not line.startswith("#"):
            f = line.split()
            rows.append((float(f[0]), float(f[1]), float(f[2]), int(f[3]), int(f[4]), int(f[5]), int(f[6])))
    return rows


def test_policy_truth_table():
    for sd, st, tau, rsd, rsd_wasted, thr, amax in _table():
        d, s = oracle.policy(oracle.POLICY_RSD, [sd], [st], tau=tau)
        assert (int(d[0]), s["wasted"]) == (rsd, rsd_wasted), (sd, st, tau)
        d, s = oracle.policy(oracle.POLICY_ORACLE_THRESHOLD, [sd], [st], tau=tau)
        assert int(d[0]) == thr, (sd, st, tau)
        d, s = oracle.policy(oracle.POLICY_ORACLE_ARGMAX, [sd], [st])
        assert int(d[0]) == amax and s["wasted"] == 0, (sd, st)
        assert s["realised"] == max(sd, st)


def test_rsd_polarity_and_monotonicity():
    """Section 3.1: acceptance is inversely related to tau; a tie s_d == tau is not accepted."""
    rng = np.random.default_rng(0)
    sd = rng.random(500).astype(np.float32)
    st = rng.random(500).astype(np.float32)
    prev = None
    for tau in (0.1, 0.3, 0.5, 0.7, 0.9):
        d, s = oracle.policy(oracle.POLICY_RSD, sd, st, tau=tau)
        assert (d == (sd <= np.float32(tau))).all()
        assert s["wasted"] == int(((sd <= np.float32(tau)) & (st <= sd)).sum())
        if prev is not None:
            assert (d >= prev).all()          # the escalated set only grows with tau
        prev = d
    d, _ = oracle.policy(oracle.POLICY_RSD, [0.5], [0.9], tau=0.5)
    assert d[0] == 1


def test_oracle_threshold_nesting_zero_waste_and_argmax():
    rng = np.random.default_rng(1)
    sd = rng.random(400).astype(np.float32)
    st = rng.random(400).astype(np.float32)
    prev = None
    for tau in (-0.5, -0.1, 0.0, 0.2, 0.6):
        d, s = oracle.policy(oracle.POLICY_ORACLE_THRESHOLD, sd, st, tau=tau)
        assert (d == ((st - sd) > np.float32(tau))).all()
        if prev is not None:
            assert (d <= prev).all()          # a higher threshold escalates a subset
        prev = d
        if tau >= 0:
            assert s["wasted"] == 0           # Corollary (zero wasted computation)
        assert abs(s["realised"] - (sd.astype(np.float64).sum() + s["gain"])) < 1e-9   # S(a) = s_d + a Delta
    d0, _ = oracle.policy(oracle.POLICY_ORACLE_THRESHOLD, sd, st, tau=0.0)
    da, sa = oracle.policy(oracle.POLICY_ORACLE_ARGMAX, sd, st)
    assert (d0 == da).all()
    assert abs(sa["realised"] - np.maximum(sd, st).astype(np.float64).sum()) < 1e-9


@pytest.mark.parametrize("seed", range(6))
def test_budgeted_rule_is_optimal_by_brute_force(seed):
    """Appendix B, Theorem: among all a with sum(a) <= B the rule maximises sum(a Delta); it uses
    k = min(B, #{Delta > 0}) escalations and equals a threshold policy."""
    rng = np.random.default_rng(100 + seed)
    n = int(rng.integers(1, 11))
    sd = (rng.integers(0, 64, n) / 64.0).astype(np.float32)     # exact values, ties included
    st = (rng.integers(0, 64, n) / 64.0).astype(np.float32)
    delta = st.astype(np.float64) - sd.astype(np.float64)
    for budget in range(0, n + 2):
        d, s = oracle.policy(oracle.POLICY_ORACLE_BUDGET, sd, st, budget=budget)
        best = max(sum(delta[i] for i in sub)
                   for k in range(0, min(budget, n) + 1) for sub in itertools.combinations(range(n), k))
        assert abs(s["gain"] - best) < 1e-12
        assert s["escalated"] == min(budget, int((delta > 0).sum()))
        assert s["wasted"] == 0
        chosen, rest = delta[d == 1], delta[(d == 0) & (delta > 0)]
        if len(chosen) and len(rest):
            assert chosen.min() >= rest.max()
        # the same set as a threshold policy, whenever a threshold can separate it (no tie at the cut)
        if len(chosen) and (not len(rest) or chosen.min() > rest.max()):
            lo = max(rest.max() if len(rest) else 0.0, 0.0)
            tau = (chosen.min() + lo) / 2
            dt, _ = oracle.policy(oracle.POLICY_ORACLE_THRESHOLD, sd, st, tau=tau)
            assert (dt == d).all()


def test_budgeted_rule_ties_go_to_the_lower_index_and_majorise_rsd():
    d, _ = oracle.policy(oracle.POLICY_ORACLE_BUDGET, [0.25, 0.25, 0.25], [0.5, 0.5, 0.5], budget=2)
    assert list(d) == [1, 1, 0]
    rng = np.random.default_rng(7)
    sd = rng.random(60).astype(np.float32)
    st = rng.random(60).astype(np.float32)
    for tau in (0.2, 0.5, 0.8):        # Corollary (Pareto frontier): no policy of the same cost scores higher
        dr, sr = oracle.policy(oracle.POLICY_RSD, sd, st, tau=tau)
        _, sb = oracle.policy(oracle.POLICY_ORACLE_BUDGET, sd, st, budget=sr["escalated"])
        assert sb["realised"] >= sr["realised"] - 1e-12


# ---- C-way heads -------------------------------------------------------------------------------------

def test_two_class_softmax_head_is_the_default_head():
    r = wl.make_router_inputs(16, 256, torch.float32, seed=5)
    rng = np.random.default_rng(5)
    w0 = rng.normal(0, 1 / 16, 256).astype(np.float32)
    w = np.stack([w0, w0 + r.w.numpy()])                      # w1 - w0 = the default head's w
    p, s, d = oracle.route_classes(oracle.HEAD_SOFTMAX, r.hidden, w, [0.125, 0.375], 0.5)
    w_diff = torch.from_numpy(w[1] - w[0])
    s_ref, d_ref = oracle.route(r.hidden, w_diff, 0.25, 0.5)
    assert np.allclose(s, s_ref, atol=1e-12) and (d == d_ref).all()
    assert np.allclose(p.sum(axis=1), 1.0, atol=1e-15) and np.allclose(p[:, 1], s, atol=1e-15)


@pytest.mark.parametrize("C", [2, 4, 10])
def test_softmax_head_against_library_softmax(C):
    rng = np.random.default_rng(C)
    hidden = rng.normal(size=(9, 64)).astype(np.float32)
    w = rng.normal(0, 0.2, size=(C, 64)).astype(np.float32)
    b = rng.normal(0, 0.3, size=C)
    p, s, d = oracle.route_classes(oracle.HEAD_SOFTMAX, hidden, w, b, 0.5)
    logits = hidden.astype(np.float64) @ w.astype(np.float64).T + b
    p_ref = softmax(logits, axis=1)
    assert np.allclose(p, p_ref, atol=1e-13)
    assert np.allclose(s, p_ref @ (np.arange(C) / (C - 1)), atol=1e-13)
    assert (d == (s.astype(np.float32) > np.float32(0.5))).all()


def test_softmax_head_closed_forms():
    hidden = np.zeros((3, 8), dtype=np.float32)
    hidden[1, 0] = 1.0
    hidden[2, 0] = 1.0
    w = np.zeros((4, 8), dtype=np.float32)
    w[2, 0] = 60.0                                            # row 1, 2: class 2 dominates by 60 nats
    p, s, d = oracle.route_classes(oracle.HEAD_SOFTMAX, hidden, w, [0.0] * 4, 0.5)
    assert np.allclose(p[0], 0.25) and s[0] == 0.5 and d[0] == 0       # equal logits; a tie accepts
    assert abs(s[1] - 2 / 3) < 1e-12 and d[1] == 1


def test_ordinal_head_closed_forms_and_two_class_case():
    hidden = np.zeros((2, 8), dtype=np.float32)
    hidden[1, 0] = 1.0
    w = np.zeros((1, 8), dtype=np.float32)
    w[0, 0] = math.log(3.0)
    cuts = [-math.log(3.0), 0.0, math.log(3.0)]
    p, s, d = oracle.route_classes(oracle.HEAD_ORDINAL, hidden, w, [0.0] + cuts, 0.5)
    # z = 0: P(y >= k) = 3/4, 1/2, 1/4 -> four equal classes, expected level 1/2
    assert np.allclose(p[0], 0.25, atol=1e-15) and abs(s[0] - 0.5) < 1e-15 and d[0] == 0
    # z = ln 3 (as rounded to fp32, hence 1e-7): P(y >= k) = sigmoid(ln 9), sigmoid(ln 3), 1/2 = 0.9, 0.75, 0.5
    assert np.allclose(p[1], [0.1, 0.15, 0.25, 0.5], rtol=0, atol=1e-7) and abs(s[1] - (0.9 + 0.75 + 0.5) / 3) < 1e-7
    r = wl.make_router_inputs(12, 128, torch.float32, seed=9)
    p2, s2, d2 = oracle.route_classes(oracle.HEAD_ORDINAL, r.hidden, r.w.reshape(1, -1), [0.3, 0.0], 0.4)
    s_ref, d_ref = oracle.route(r.hidden, r.w, 0.3, 0.4)     # one cut at 0: the default head again
    assert np.allclose(s2, s_ref, atol=1e-12) and (d2 == d_ref).all()
    z = r.hidden.double().numpy() @ r.w.double().numpy() + 0.3
    assert np.allclose(p2[:, 1], expit(z), atol=1e-12)


# ---- KV append ---------------------------------------------------------------------------------------

def _append_case(dtype, seed):
    inp = wl.small_attn_case(3, 8, 2, 64, dtype, [40, 17, 96], [1, 1, 1], seed=seed, extra_tokens=40)
    gen = torch.Generator().manual_seed(seed + 1)
    new_lens = torch.tensor([5, 0, 33], dtype=torch.int32)
    k_new = torch.randn(int(new_lens.sum()), 2, 64, generator=gen).to(dtype)
    v_new = torch.randn(int(new_lens.sum()), 2, 64, generator=gen).to(dtype)
    return inp, new_lens, k_new, v_new


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_kv_append_puts_every_token_where_attention_reads_it(dtype):
    inp, new_lens, k_new, v_new = _append_case(dtype, 21)
    kp, vp, sl, st = oracle.kv_append(k_new, v_new, inp.block_table, inp.seq_lens, new_lens, inp.k_pages, inp.v_pages)
    assert st == 0 and list(sl) == [45, 17, 129]
    # independent placement by plain indexing
    k_ref, v_ref = inp.k_pages.clone(), inp.v_pages.clone()
    row = 0
    for b in range(3):
        for j in range(int(new_lens[b])):
            pos = int(inp.seq_lens[b]) + j
            page = int(inp.block_table[b, pos // 16])
            k_ref[page, :, pos % 16, :] = k_new[row]
            v_ref[page, :, pos % 16, :] = v_new[row]
            row += 1
    assert torch.equal(kp, k_ref) and torch.equal(vp, v_ref)
    # and attention over the grown cache sees the new tokens: the last query of sequence 2 at its new length
    q = inp.q
    out, st2 = oracle.attn(q, kp, vp, inp.block_table, torch.from_numpy(sl), inp.q_lens)
    out_old, _ = oracle.attn(q, inp.k_pages, inp.v_pages, inp.block_table, inp.seq_lens, inp.q_lens)
    assert st2 == 0 and not np.allclose(out[2], out_old[2]) and np.array_equal(out[1], out_old[1])


def test_kv_append_refuses_what_does_not_fit():
    inp, new_lens, k_new, v_new = _append_case(torch.float32, 22)
    cap = inp.block_table.shape[1] * 16
    too_long = torch.tensor([5, 0, cap], dtype=torch.int32)
    big_k = torch.zeros(int(too_long.sum()), 2, 64)
    kp, vp, sl, st = oracle.kv_append(big_k, big_k, inp.block_table, inp.seq_lens, too_long, inp.k_pages, inp.v_pages)
    assert st & oracle.BAD_SEQ_LEN and list(sl) == [45, 17, 96]
    bad_bt = inp.block_table.clone()
    bad_bt[0, 40 // 16] = inp.k_pages.shape[0] + 3
    kp, vp, sl, st = oracle.kv_append(k_new, v_new, bad_bt, inp.seq_lens, new_lens, inp.k_pages, inp.v_pages)
    assert st & oracle.BAD_PAGE and list(sl) == [40, 17, 129]
    neg = torch.tensor([-1, 0, 0], dtype=torch.int32)
    kp, vp, sl, st = oracle.kv_append(k_new[:0], v_new[:0], inp.block_table, inp.seq_lens, neg, inp.k_pages, inp.v_pages)
    assert st & oracle.BAD_SEQ_LEN and torch.equal(kp, inp.k_pages)


def test_rollback_then_append_overwrites_the_rejected_step():
    """Algorithm 1, escalation branch: the rejected draft step's slots are reused by the target's step."""
    inp, new_lens, k_new, v_new = _append_case(torch.float32, 23)
    kp, vp, sl, _ = oracle.kv_append(k_new, v_new, inp.block_table, inp.seq_lens, new_lens, inp.k_pages, inp.v_pages)
    rolled, _ = oracle.rollback(sl, new_lens.numpy(), np.array([1, 1, 1], dtype=np.uint8))
    assert list(rolled) == [40, 17, 96]
    k2, v2 = -k_new, -v_new
    kp2, vp2, sl2, _ = oracle.kv_append(k2, v2, inp.block_table, torch.from_numpy(rolled), new_lens, kp, vp)
    kp_direct, vp_direct, _, _ = oracle.kv_append(k2, v2, inp.block_table, inp.seq_lens, new_lens, inp.k_pages, inp.v_pages)
    assert torch.equal(kp2, kp_direct) and torch.equal(vp2, vp_direct) and list(sl2) == list(sl)


def test_phase_lens_partitions_the_batch():
    """Every sequence is in exactly one of the two branches after the decision, and a step decoded token by
    token adds up to the step absorbed at once."""
    rng = np.random.default_rng(3)
    step = rng.integers(0, 9, 50).astype(np.int32)
    dec = rng.integers(0, 2, 50).astype(np.uint8)
    acc = oracle.phase_lens(step, dec, want=0, t=-1)
    esc = oracle.phase_lens(step, dec, want=1, t=-1)
    assert np.array_equal(acc + esc, step) and np.array_equal(acc[dec == 1], 0 * acc[dec == 1])
    assert np.array_equal(esc, step * dec)
    by_token = sum(oracle.phase_lens(step, dec, want=1, t=t) for t in range(9))
    assert np.array_equal(by_token, esc)
    assert list(oracle.phase_lens([3, -4, 0], None, t=-1)) == [3, 0, 0]
    assert list(oracle.phase_lens([3, 1, 2], None, t=1)) == [1, 0, 1]


# ---- Spearman ----------------------------------------------------------------------------------------

def test_spearman_against_library_and_closed_forms():
    from scipy.stats import rankdata, spearmanr
    rng = np.random.default_rng(11)
    for n, ties in ((2, False), (17, False), (200, False), (200, True), (1000, True)):
        x = rng.normal(size=n).astype(np.float32)
        y = (0.3 * x + rng.normal(size=n)).astype(np.float32)
        if ties:
            x, y = np.round(x * 2) / 2, np.round(y * 3) / 3
        rho, rx, ry = oracle.spearman(x, y, return_ranks=True)
        assert np.array_equal(rx, rankdata(x)) and np.array_equal(ry, rankdata(y))     # average ranks
        assert abs(rho - spearmanr(x, y).statistic) < 1e-12
        if not ties:      # the textbook form for distinct values: 1 - 6 sum d^2 / (n (n^2 - 1))
            d = rankdata(x) - rankdata(y)
            assert abs(rho - (1 - 6 * float((d * d).sum()) / (n * (n * n - 1)))) < 1e-12
    # by hand: x = 1 2 2 3 -> ranks 1 2.5 2.5 4; y = 1 2 3 4: sums 4.5, 4.5, 5 -> rho = 3 / sqrt(10)
    assert abs(oracle.spearman([1, 2, 2, 3], [1, 2, 3, 4]) - 3 / math.sqrt(10)) < 1e-15
    x = rng.normal(size=50).astype(np.float32)
    assert oracle.spearman(x, np.exp(x)) == 1.0 and oracle.spearman(x, -x ** 3) == -1.0    # monotone maps
    assert abs(oracle.spearman(x, x[::-1].copy()) - oracle.spearman(x[::-1].copy(), x)) < 1e-15   # symmetric
    assert math.isnan(oracle.spearman([1, 1, 1], [1, 2, 3])) and math.isnan(oracle.spearman([1], [2]))


# ---- E4M3 ----------------------------------------------------------------------------------------------

def test_e4m3_against_the_library_type_and_the_format():
    codes = np.arange(256, dtype=np.uint8)
    ours = oracle.e4m3_decode(codes)
    lib = torch.from_numpy(codes).view(torch.float8_e4m3fn).float().numpy()
    assert np.array_equal(np.isnan(ours), np.isnan(lib)) and np.array_equal(ours[~np.isnan(ours)], lib[~np.isnan(lib)])
    # format facts: largest finite 448, smallest subnormal 2^-9, smallest normal 2^-6, no infinities
    assert ours[0x7e] == 448.0 and ours[0x01] == 2.0 ** -9 and ours[0x08] == 2.0 ** -6 and np.isnan(ours[0x7f])
    assert not np.isinf(ours).any() and ours[0x80] == 0.0 and np.signbit(ours[0x80])
    finite = codes[~np.isnan(ours)]
    assert np.array_equal(oracle.e4m3_encode(ours[finite]), finite)                 # round trip, -0 included
    # nearest with ties to even, against the library's conversion inside the finite range
    rng = np.random.default_rng(8)
    x = np.concatenate([rng.normal(0, 1, 4000), rng.normal(0, 60, 2000), rng.uniform(-2.0 ** -6, 2.0 ** -6, 1000),
                        [1.0625, 1.1875, 2.0 ** -10, 3 * 2.0 ** -10, 464.0 - 1e-3, -447.9]]).astype(np.float32)
    x = x[np.abs(x) < 464.0]
    lib_codes = torch.from_numpy(x).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    assert np.array_equal(oracle.e4m3_encode(x), lib_codes)
    # saturation (this library's choice; the library type gives NaN there): by definition
    assert list(oracle.e4m3_encode(np.float32([464.0, 1e9, -500.0, np.inf]))) == [0x7e, 0x7e, 0xfe, 0x7e]
    assert oracle.e4m3_encode(np.float32([3.0]), inv_scale=0.5)[0] == 0x3c           # 1.5 = (1 + 4/8) * 2^0


def test_e4m3_cache_attention_and_quantising_append():
    inp = wl.small_attn_case(2, 8, 2, 64, torch.bfloat16, [70, 33], [1, 1], seed=61, extra_tokens=32)
    ks, vs = 0.02, 0.03
    kc = torch.from_numpy(oracle.e4m3_encode(inp.k_pages, 1 / ks))
    vc = torch.from_numpy(oracle.e4m3_encode(inp.v_pages, 1 / vs))
    out, st = oracle.attn_e4m3(inp.q, kc, vc, ks, vs, inp.block_table, inp.seq_lens, inp.q_lens)
    # the same thing spelled out with the library type: dequantise, then the bf16-cache oracle path on fp32 pools
    kf = kc.view(torch.float8_e4m3fn).float() * ks
    vf = vc.view(torch.float8_e4m3fn).float() * vs
    ref, _ = oracle.attn(inp.q.float(), kf, vf, inp.block_table, inp.seq_lens, inp.q_lens)
    assert st == 0 and np.allclose(out, ref, rtol=0, atol=1e-6)
    full, _ = oracle.attn(inp.q, inp.k_pages, inp.v_pages, inp.block_table, inp.seq_lens, inp.q_lens)
    assert np.abs(out - full).max() < 0.15                                           # and it is a fair copy of the cache
    new = torch.tensor([3, 20], dtype=torch.int32)
    g = torch.Generator().manual_seed(3)
    kn, vn = torch.randn(23, 2, 64, generator=g).bfloat16(), torch.randn(23, 2, 64, generator=g).bfloat16()
    kc2, vc2, sl, st = oracle.kv_append_e4m3(kn, vn, inp.block_table, inp.seq_lens, new, kc, vc, 1 / ks, 1 / vs)
    page, slot = int(inp.block_table[1, 33 // 16]), 33 % 16
    want = torch.from_numpy((kn[3].float() / 1).numpy() * np.float32(1 / ks)).to(torch.float8_e4m3fn).view(torch.uint8)
    assert st == 0 and list(sl) == [73, 53] and torch.equal(kc2[page, :, slot, :], want)
