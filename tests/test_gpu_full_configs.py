"""The five workloads at their full sizes, through the same calls bench.py times, against the oracle: every
element of every output for tiny, draft-shaped, target-shaped and step scoring, and for the first and the last
iteration of the mixed loop (the oracle needs some tens of seconds for each of the two large ones); sampled rows
for the loop's other iterations."""
import numpy as np
import pytest
import torch

from oracle import oracle
from paper_2512_05033_b200 import workloads as wl
from tests import helpers as H

pytestmark = pytest.mark.gpu
BF = torch.bfloat16


def _sample_rows(inp_cpu, out_gpu, n_samples, seed, tol=1e-2):
    """Compare sampled (row, head) outputs with the oracle's single-row routine."""
    rng = np.random.default_rng(seed)
    ql = inp_cpu.q_lens.numpy().astype(np.int64)
    sl = inp_cpu.seq_lens.numpy().astype(np.int64)
    rows0 = np.concatenate([[0], np.cumsum(ql)])
    Hq = inp_cpu.q.shape[1]
    worst = 0.0
    for _ in range(n_samples):
        b = int(rng.integers(0, len(ql)))
        if ql[b] == 0:
            continue
        i = int(rng.integers(0, ql[b])) if rng.random() < 0.7 else int(ql[b] - 1)
        h = int(rng.integers(0, Hq))
        row, pos = int(rows0[b] + i), int(sl[b] - ql[b] + i)
        o, _, st = oracle.attn_row_probs(inp_cpu.q, inp_cpu.k_pages, inp_cpu.v_pages, inp_cpu.block_table[b], row, h, pos)
        assert st == 0
        err = float(np.abs(out_gpu[row, h].double().cpu().numpy() - o).max())
        worst = max(worst, err)
        assert err <= tol, (b, i, h, err)
    return worst


def test_tiny_config():
    c = H.ctx()
    for shape in (wl.TINY_DECODE, wl.TINY_CHUNK):
        inp = wl.make_attn_inputs(shape)
        out, bits = H.gpu_attn(inp)
        ref, _ = H.oracle_attn(inp)
        assert bits == 0
        H.assert_close(out, ref, torch.float32)
    r = wl.make_router_inputs(1, 256, torch.float32, seed=0)
    s, d = c.route(r.hidden.cuda(), r.w.cuda(), 0.0, 0.5)
    so, do = oracle.route(r.hidden, r.w, 0.0, 0.5)
    assert abs(float(s[0]) - so[0]) <= 1e-5 and (abs(so[0] - 0.5) <= 1e-3 or int(d[0]) == int(do[0]))


def test_draft_shaped_decode_full():
    from paper_2512_05033_b200 import binding
    inp = wl.make_attn_inputs(wl.DRAFT_DECODE)
    d = inp.to("cuda")
    c = H.ctx()
    # the launch configuration of the benchmark: programmatic dependents, back to back
    p = c.params_for(d.q, d.k_pages, d.block_table, 1, flags=binding.ATTN_OVERLAP_PREVIOUS)
    outs = [torch.empty_like(d.q) for _ in range(3)]
    for o in outs:
        c.attn(d.q, d.k_pages, d.v_pages, d.block_table, d.seq_lens, d.q_lens, 1, out=o, params=p)
    assert c.poll_status() == 0
    ref, _ = H.oracle_attn(inp)
    for o in outs:
        H.assert_close(o.double().cpu().numpy(), ref, BF, tight=1e-3)


def test_target_shaped_decode_full():
    inp = wl.make_attn_inputs(wl.TARGET_DECODE, device="cuda")
    c = H.ctx()
    out = c.attn(inp.q, inp.k_pages, inp.v_pages, inp.block_table, inp.seq_lens, inp.q_lens, 1)
    assert c.poll_status() == 0
    cpu = inp.to("cpu")
    ref, st = H.oracle_attn(cpu)
    assert st == 0
    H.assert_close(out.double().cpu().numpy(), ref, BF, tight=1e-3)


def test_step_scoring_full():
    shape = wl.STEP_SCORING
    inp = wl.make_attn_inputs(shape, device="cuda")
    c = H.ctx()
    out = c.attn(inp.q, inp.k_pages, inp.v_pages, inp.block_table, inp.seq_lens, inp.q_lens, int(inp.q_lens.max()))
    assert c.poll_status() == 0
    ref, st = H.oracle_attn(inp.to("cpu"))          # all 2490 rows x 28 heads
    assert st == 0
    H.assert_close(out.double().cpu().numpy(), ref, BF, tight=3e-3)
    # router over hidden 3584 with the three thresholds, then the rollback of the escalated steps
    r = wl.make_router_inputs(shape.batch, shape.hidden, shape.dtype, seed=shape.seed, b_std=0.1 ** 0.5)
    prev = None
    for tau in (0.3, 0.5, 0.7):
        s, d = c.route(r.hidden.cuda(), r.w.cuda(), r.b, tau)
        so, do = oracle.route(r.hidden, r.w, r.b, tau)
        assert np.abs(s.cpu().numpy() - so).max() <= 1e-5
        clear = np.abs(so - tau) > 1e-3
        np.testing.assert_array_equal(d.cpu().numpy()[clear], do[clear])
        seq = inp.seq_lens.clone()
        c.rollback(seq, inp.q_lens, d)
        exp, _ = oracle.rollback(inp.seq_lens.cpu(), inp.q_lens.cpu(), d.cpu().numpy())
        np.testing.assert_array_equal(seq.cpu().numpy(), exp)
        if prev is not None:
            assert (d.cpu().numpy() <= prev).all()      # a higher tau escalates a subset
        prev = d.cpu().numpy()


def test_mixed_serving_loop_full():
    m = wl.make_mixed_loop(device="cuda")
    c = H.ctx()
    B = m.shape.batch
    seq = m.seq_lens0.clone()
    seq_ref = m.seq_lens0.cpu().numpy().astype(np.int64)
    k_cpu, v_cpu, bt_cpu = m.k_pages.cpu(), m.v_pages.cpu(), m.block_table.cpu()
    escalated = 0
    for it in range(len(m.q_lens)):
        ql = m.q_lens[it]
        seq += ql                                           # the new tokens' K/V are in place: append
        out = c.attn(m.q[it], m.k_pages, m.v_pages, m.block_table, seq, ql, int(ql.max()))
        scores, dec = c.route(m.hidden[it], m.w, m.b, m.tau)
        step_lens = torch.where(ql > 1, ql, torch.zeros_like(ql))   # decode tokens are never rolled back
        seq_before = seq.clone()
        c.rollback(seq, step_lens, dec)
        assert c.poll_status() == 0
        # oracle side of the same iteration
        seq_ref = seq_ref + ql.cpu().numpy()
        np.testing.assert_array_equal(seq_before.cpu().numpy(), seq_ref)
        snap = wl.AttnInputs(m.shape, m.q[it].cpu(), k_cpu, v_cpu, bt_cpu, torch.from_numpy(seq_ref.astype(np.int32)),
                             ql.cpu())
        if it in (0, len(m.q_lens) - 1):            # every element of the iteration's output
            ref, st = H.oracle_attn(snap)
            assert st == 0
            H.assert_close(out.double().cpu().numpy(), ref, BF, tight=3e-3)
        else:
            _sample_rows(snap, out, 24, seed=100 + it)
        so, do = oracle.route(m.hidden[it].cpu(), m.w.cpu(), m.b, m.tau)
        assert np.abs(scores.cpu().numpy() - so).max() <= 1e-5
        clear = np.abs(so - m.tau) > 1e-3
        np.testing.assert_array_equal(dec.cpu().numpy()[clear], do[clear])
        seq_ref, st = oracle.rollback(seq_ref, step_lens.cpu().numpy(), dec.cpu().numpy())
        seq_ref = seq_ref.astype(np.int64)
        assert st == 0
        np.testing.assert_array_equal(seq.cpu().numpy(), seq_ref)
        escalated += int((dec.cpu().numpy() * (ql.cpu().numpy() > 1)).sum())
    assert 0 < escalated < B * len(m.q_lens) // 2


def test_draft_shaped_decode_step_full():
    """The single-launch token (arb_decode_step) on the draft-shaped batch, in the chain bench.py times: three tokens in a
    row on one cache, every call finding what the one before it left; pools bit for bit, lengths exact, every row."""
    shape = wl.DRAFT_DECODE
    inp = wl.make_attn_inputs(shape, extra_tokens=8)
    d = inp.to("cuda")
    c = H.ctx()
    sl = inp.seq_lens.numpy().copy()
    k_ref, v_ref = inp.k_pages, inp.v_pages
    ones = torch.ones(shape.batch, dtype=torch.int32)
    outs, news = [], []
    for t in range(3):
        q = wl.normal((shape.batch, shape.num_q_heads, shape.head_dim), 1.0, BF, "cpu", 9100 + t)
        kn = wl.normal((shape.batch, shape.num_kv_heads, shape.head_dim), 1.0, BF, "cpu", 9200 + t)
        vn = wl.normal((shape.batch, shape.num_kv_heads, shape.head_dim), 1.0, BF, "cpu", 9300 + t)
        news.append((q, kn, vn))
        outs.append(c.decode_step(q.cuda(), kn.cuda(), vn.cuda(), d.k_pages, d.v_pages, d.block_table, d.seq_lens, d.q_lens))
    assert c.poll_status() == 0
    for (q, kn, vn), out in zip(news, outs):
        k_ref, v_ref, sl, st = oracle.kv_append(kn, vn, inp.block_table, sl, ones, k_ref, v_ref)
        ref, st2 = oracle.attn(q, k_ref, v_ref, inp.block_table, sl, ones)
        assert st == 0 and st2 == 0
        H.assert_close(out.double().cpu().numpy(), ref, BF, tight=3e-3)
    assert np.array_equal(d.seq_lens.cpu().numpy(), sl)
    assert torch.equal(d.k_pages.cpu(), k_ref) and torch.equal(d.v_pages.cpu(), v_ref)


def test_draft_shaped_decode_step_e4m3_full():
    """arb_decode_step_e4m3 on the draft-shaped batch: two tokens in a row on one E4M3 cache; codes bit for bit,
    lengths exact, every row."""
    shape = wl.DRAFT_DECODE
    inp = wl.make_attn_inputs(shape, extra_tokens=8)
    ks, vs = 0.012, 0.015
    kc = torch.from_numpy(oracle.e4m3_encode(inp.k_pages, 1 / ks))
    vc = torch.from_numpy(oracle.e4m3_encode(inp.v_pages, 1 / vs))
    d = inp.to("cuda")
    dk, dv = kc.cuda(), vc.cuda()
    c = H.ctx()
    sl = inp.seq_lens.numpy().copy()
    ones = torch.ones(shape.batch, dtype=torch.int32)
    outs, news = [], []
    for t in range(2):
        q = wl.normal((shape.batch, shape.num_q_heads, shape.head_dim), 1.0, BF, "cpu", 9400 + t)
        kn = wl.normal((shape.batch, shape.num_kv_heads, shape.head_dim), 1.0, BF, "cpu", 9500 + t)
        vn = wl.normal((shape.batch, shape.num_kv_heads, shape.head_dim), 1.0, BF, "cpu", 9600 + t)
        news.append((q, kn, vn))
        outs.append(c.decode_step_e4m3(q.cuda(), kn.cuda(), vn.cuda(), dk, dv, ks, vs, 1 / ks, 1 / vs, d.block_table,
                                       d.seq_lens, d.q_lens))
    assert c.poll_status() == 0
    for (q, kn, vn), out in zip(news, outs):
        kc, vc, sl, st = oracle.kv_append_e4m3(kn, vn, inp.block_table, sl, ones, kc, vc, 1 / ks, 1 / vs)
        ref, st2 = oracle.attn_e4m3(q, kc, vc, ks, vs, inp.block_table, sl, ones)
        assert st == 0 and st2 == 0
        H.assert_close(out.double().cpu().numpy(), ref, BF, tight=3e-3)
    assert np.array_equal(d.seq_lens.cpu().numpy(), sl)
    assert torch.equal(dk.cpu(), kc) and torch.equal(dv.cpu(), vc)


def test_draft_shaped_decode_step_i4_full():
    """arb_decode_step_i4 on the draft-shaped batch: two tokens in a row on one 4-bit cache; codes and scales bit for
    bit, lengths exact, every row."""
    shape = wl.DRAFT_DECODE
    inp = wl.make_attn_inputs(shape, extra_tokens=8)
    kc, ks = (torch.from_numpy(x) for x in oracle.i4_encode(inp.k_pages))
    vc, vs = (torch.from_numpy(x) for x in oracle.i4_encode(inp.v_pages))
    d = inp.to("cuda")
    pools = [kc.cuda(), vc.cuda(), ks.cuda(), vs.cuda()]
    c = H.ctx()
    sl = inp.seq_lens.numpy().copy()
    ones = torch.ones(shape.batch, dtype=torch.int32)
    outs, news = [], []
    for t in range(2):
        q = wl.normal((shape.batch, shape.num_q_heads, shape.head_dim), 1.0, BF, "cpu", 9700 + t)
        kn = wl.normal((shape.batch, shape.num_kv_heads, shape.head_dim), 1.0, BF, "cpu", 9800 + t)
        vn = wl.normal((shape.batch, shape.num_kv_heads, shape.head_dim), 1.0, BF, "cpu", 9900 + t)
        news.append((q, kn, vn))
        outs.append(c.decode_step_i4(q.cuda(), kn.cuda(), vn.cuda(), *pools, d.block_table, d.seq_lens, d.q_lens))
    assert c.poll_status() == 0
    for (q, kn, vn), out in zip(news, outs):
        kc, vc, ks, vs, sl, st = oracle.kv_append_i4(kn, vn, inp.block_table, sl, ones, kc, vc, ks, vs)
        ref, st2 = oracle.attn_i4(q, kc, vc, ks, vs, inp.block_table, sl, ones)
        assert st == 0 and st2 == 0
        H.assert_close(out.double().cpu().numpy(), ref, BF, tight=3e-3)
    assert np.array_equal(d.seq_lens.cpu().numpy(), sl)
    assert torch.equal(pools[0].cpu(), kc) and torch.equal(pools[1].cpu(), vc)
    assert torch.equal(pools[2].cpu(), torch.as_tensor(np.asarray(ks))) and torch.equal(pools[3].cpu(), torch.as_tensor(np.asarray(vs)))


def test_step_scoring_full_over_the_e4m3_cache():
    """arb_attn_e4m3 on the step-scoring batch at full size (pools quantised by the oracle), every element."""
    shape = wl.STEP_SCORING
    inp = wl.make_attn_inputs(shape)
    ks, vs = 0.012, 0.015
    kc = torch.from_numpy(oracle.e4m3_encode(inp.k_pages, 1 / ks))
    vc = torch.from_numpy(oracle.e4m3_encode(inp.v_pages, 1 / vs))
    d = inp.to("cuda")
    c = H.ctx()
    out = c.attn_e4m3(d.q, kc.cuda(), vc.cuda(), ks, vs, d.block_table, d.seq_lens, d.q_lens, int(inp.q_lens.max()))
    assert c.poll_status() == 0
    ref, st = oracle.attn_e4m3(inp.q, kc, vc, ks, vs, inp.block_table, inp.seq_lens, inp.q_lens)
    assert st == 0
    H.assert_close(out.double().cpu().numpy(), ref, BF, tight=3e-3)
