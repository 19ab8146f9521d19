"""Parity of arb_route and arb_rollback with the oracle; the rollback-then-attend identity on the GPU."""
import math

import numpy as np
import pytest
import torch

from oracle import oracle
from paper_2512_05033_b200 import workloads as wl
from tests import helpers as H

pytestmark = pytest.mark.gpu


def _route_both(r, tau):
    c = H.ctx()
    s, d = c.route(r.hidden.cuda(), r.w.cuda(), r.b, tau)
    torch.cuda.synchronize()
    so, do = oracle.route(r.hidden, r.w, r.b, tau)
    return s.cpu().numpy(), d.cpu().numpy(), so, do


@pytest.mark.parametrize("n,H_,dt,b_std", [(1, 256, torch.float32, 0.0), (32, 3584, torch.bfloat16, math.sqrt(0.1)),
                                           (67, 1024, torch.bfloat16, 0.3), (5, 8, torch.float32, 0.0),
                                           (130, 4096, torch.float32, 0.2)])
def test_route_matches_oracle(n, H_, dt, b_std):
    r = wl.make_router_inputs(n, H_, dt, seed=n + H_, b_std=b_std)
    for tau in (0.3, 0.5, 0.7):
        s, d, so, do = _route_both(r, tau)
        assert np.abs(s - so).max() <= 1e-5
        clear = np.abs(so - tau) > 1e-3          # decisions are bit-exact outside the band
        np.testing.assert_array_equal(d[clear], do[clear])
        assert set(np.unique(d)) <= {0, 1}


def test_route_tie_and_hand_built_scores():
    hidden = torch.zeros(4, 16)
    w = torch.zeros(16)
    w[3] = 1.0
    hidden[1, 3] = math.log(3.0)
    hidden[2, 3] = -math.log(3.0)
    hidden[3, 3] = 1e-2
    c = H.ctx()
    s, d = c.route(hidden.cuda(), w.cuda(), 0.0, 0.5)
    s, d = s.cpu().numpy(), d.cpu().numpy()
    assert s[0] == 0.5 and d[0] == 0                 # tie accepts
    np.testing.assert_allclose(s[1:3], [0.75, 0.25], atol=1e-6)
    assert list(d) == [0, 1, 0, 1]


def test_rollback_matches_oracle_and_flags_underflow():
    from paper_2512_05033_b200 import binding
    c = H.ctx()
    sl = torch.tensor([100, 50, 7, 0, 9, 4000], dtype=torch.int32)
    st = torch.tensor([10, 50, 8, 0, -1, 128], dtype=torch.int32)
    dec = torch.tensor([1, 0, 0, 1, 0, 1], dtype=torch.uint8)
    g = c.rollback(sl.cuda(), st.cuda(), dec.cuda()).cpu().numpy()
    exp, status = oracle.rollback(sl, st, dec)
    np.testing.assert_array_equal(g, exp)
    assert c.poll_status() == 0 and status == 0
    g = c.rollback(sl.cuda(), st.cuda(), None).cpu().numpy()
    exp, status = oracle.rollback(sl, st, None)
    np.testing.assert_array_equal(g, exp)
    assert c.poll_status() == binding.DEV_ROLLBACK_UNDERFLOW and status == oracle.ROLLBACK_UNDERFLOW


def test_route_then_rollback_then_attend_on_device():
    """Algorithm 1's escalation branch end to end on the device: scores -> decisions -> seq_len reset ->
    the next decode sees the prefix only, although the rejected step's slots still hold its K/V."""
    B, step = 6, 9
    prefix = [300, 45, 1000, 16, 77, 512]
    inp = wl.small_attn_case(B, 12, 2, 128, torch.bfloat16, [p + step for p in prefix], [1] * B, seed=61,
                             extra_tokens=4)
    r = wl.make_router_inputs(B, 256, torch.bfloat16, seed=62)
    c = H.ctx()
    d = inp.to("cuda")
    scores, dec = c.route(r.hidden.cuda(), r.w.cuda(), 0.0, 0.5)
    seq = d.seq_lens.clone()
    c.rollback(seq, torch.full((B,), step, dtype=torch.int32, device="cuda"), dec)
    seq += 1                                   # the regenerated step's first token
    out = torch.empty_like(d.q)
    c.attn(d.q, d.k_pages, d.v_pages, d.block_table, seq, d.q_lens, 1, out=out)
    assert c.poll_status() == 0
    _, do = oracle.route(r.hidden, r.w, 0.0, 0.5)
    exp_len, _ = oracle.rollback(inp.seq_lens, np.full(B, step), do)
    np.testing.assert_array_equal(seq.cpu().numpy(), exp_len + 1)
    assert 0 < do.sum() < B
    ref, _ = oracle.attn(inp.q, inp.k_pages, inp.v_pages, inp.block_table, exp_len + 1, inp.q_lens)
    H.assert_close(out.double().cpu().numpy(), ref, torch.bfloat16)
