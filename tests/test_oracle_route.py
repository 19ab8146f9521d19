"""Pins of the router and rollback oracles (no GPU): hand-built scores, the tie rule, closed forms,
nesting over tau, the softmax-of-two identity, and rollback as 'the cache never saw the step'."""
import math
from pathlib import Path

import numpy as np
import torch

from oracle import oracle
from paper_2512_05033_b200 import workloads as wl

GOLDEN = Path(__file__).parent / "golden" / "router_truth_table.txt"


def _z(expr):
    return {"0": 0.0, "ln3": math.log(3), "-ln3": -math.log(3), "ln9": math.log(9),
            "-ln9": -math.log(9), "ln(7/3)": math.log(7 / 3)}[expr]


def test_truth_table_from_the_rule():
    H = 16
    rows = [l.split() for l in GOLDEN.read_text().splitlines() if l.strip() and not l.startswith("#")]
    assert len(rows) >= 10
    for expr, score, tau, dec in rows:
        z = _z(expr)
        # hidden = c * e_k, w = e_k  =>  z = c + b; split z between the dot product and the bias
        hidden = np.zeros((1, H), dtype=np.float32)
        w = np.zeros(H, dtype=np.float32)
        hidden[0, 5] = 2.0
        w[5] = 0.25                      # dot = 0.5 exactly
        s, d = oracle.route(hidden, w, z - 0.5, float(tau))
        assert abs(s[0] - float(score)) < 1e-12, (expr, s)
        # closed-form scores sit exactly on tau only in the tie rows, where fp32(score) == fp32(tau)
        assert int(d[0]) == int(dec), (expr, tau, s)


def test_tie_accepts_and_polarity():
    hidden = np.zeros((3, 8), dtype=np.float32)
    w = np.ones(8, dtype=np.float32)
    hidden[1, 0] = 1e-3
    hidden[2, 0] = -1e-3
    s, d = oracle.route(hidden, w, 0.0, 0.5)
    assert s[0] == 0.5 and list(d) == [0, 1, 0]        # tie -> accept; above -> escalate


def test_sigmoid_symmetry_and_range():
    r = wl.make_router_inputs(64, 256, torch.float32, seed=3)
    s, _ = oracle.route(r.hidden, r.w, 0.3, 0.5)
    s2, _ = oracle.route(-r.hidden, r.w, -0.3, 0.5)
    np.testing.assert_allclose(s + s2, 1.0, atol=1e-15)
    assert ((s > 0) & (s < 1)).all()
    # independent recomputation of z with numpy in fp64
    z = r.hidden.double().numpy() @ r.w.double().numpy() + 0.3
    np.testing.assert_allclose(s, 1 / (1 + np.exp(-z)), atol=1e-15)


def test_decision_flips_at_logit_of_tau():
    for tau in (0.3, 0.5, 0.7):
        zc = math.log(tau / (1 - tau))
        hidden = np.array([[zc - 1e-3], [zc + 1e-3]], dtype=np.float32).repeat(8, axis=1) / 8
        w = np.ones(8, dtype=np.float32)
        _, d = oracle.route(hidden, w, 0.0, tau)
        assert list(d) == [0, 1]
    assert abs(math.log(0.7 / 0.3) - 0.8473) < 1e-4


def test_escalation_sets_nest_over_tau():
    """Raising tau can only shrink the escalated set (Section 4.1: tau regulates how often we escalate)."""
    r = wl.make_router_inputs(512, 3584, torch.bfloat16, seed=4, b_std=math.sqrt(0.1))
    d = {tau: oracle.route(r.hidden, r.w, r.b, tau)[1].astype(bool) for tau in (0.3, 0.5, 0.7)}
    assert (d[0.7] <= d[0.5]).all() and (d[0.5] <= d[0.3]).all()
    assert d[0.3].sum() > d[0.5].sum() > d[0.7].sum() > 0


def test_two_class_softmax_head_is_sigmoid_of_logit_difference():
    g = torch.Generator().manual_seed(5)
    hidden = torch.randn(32, 64, generator=g)
    W = torch.randn(2, 64, generator=g) / 8
    bias = torch.randn(2, generator=g)
    logits = hidden.double() @ W.double().T + bias.double()
    p1 = torch.softmax(logits, dim=1)[:, 1].numpy()
    # (w1 - w0) in fp64 is not representable in fp32 in general, so widen by hand
    wd = (W[1].double() - W[0].double())
    z = hidden.double() @ wd + float(bias[1].double() - bias[0].double())
    np.testing.assert_allclose(p1, 1 / (1 + np.exp(-z.numpy())), atol=1e-15)
    w32 = (W[1] - W[0])
    s, _ = oracle.route(hidden, w32, float(bias[1] - bias[0]), 0.5)
    np.testing.assert_allclose(s, p1, atol=1e-6)


def test_rollback_integer_identity():
    sl = np.array([100, 50, 7, 0, 9], dtype=np.int32)
    st = np.array([10, 50, 8, 0, -1], dtype=np.int32)
    new, status = oracle.rollback(sl, st)
    assert list(new) == [90, 0, 0, 0, 9] and status == oracle.ROLLBACK_UNDERFLOW
    dec = np.array([1, 0, 0, 1, 0], dtype=np.uint8)
    new, status = oracle.rollback(sl, st, dec)
    assert list(new) == [90, 50, 7, 0, 9] and status == 0
    assert list(sl) == [100, 50, 7, 0, 9]


def test_attention_after_rollback_equals_cache_that_never_saw_the_step():
    """Escalation regenerates from the same prefix x (Algorithm 1): poison the dropped slots."""
    L0, step = 37, 11
    inp = wl.small_attn_case(1, 4, 2, 64, torch.bfloat16, [L0 + step + 1], [1], seed=23)
    fresh_len = torch.tensor([L0 + 1], dtype=torch.int32)
    # decode one token at position L0 on a cache holding only the prefix (+ that token)
    out_fresh, _ = oracle.attn(inp.q, inp.k_pages, inp.v_pages, inp.block_table, fresh_len, inp.q_lens)
    # the cache absorbed a draft step of `step` tokens, then rolled it back; its slots hold poison
    new_len, _ = oracle.rollback(np.array([L0 + step]), np.array([step]))
    assert int(new_len[0]) == L0
    k2, v2 = inp.k_pages.clone(), inp.v_pages.clone()
    for j in range(L0 + 1, L0 + step + 1):
        pg = int(inp.block_table[0, j // wl.PAGE])
        k2[pg, :, j % wl.PAGE] = float("nan")
        v2[pg, :, j % wl.PAGE] = 1e30
    out_rb, _ = oracle.attn(inp.q, k2, v2, inp.block_table, torch.tensor([int(new_len[0]) + 1]), inp.q_lens)
    np.testing.assert_array_equal(out_fresh, out_rb)
