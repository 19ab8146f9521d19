"""Two rounds of the step loop (Algorithm 1) through the library against the same rounds run with the oracle."""
import numpy as np
import pytest
import torch

from oracle import oracle
from paper_2512_05033_b200 import workloads as wl
from tests import helpers as H

pytestmark = pytest.mark.gpu
BF = torch.bfloat16


def _cache(B, Hq, Hkv, D, prefix, seed, room):
    inp = wl.small_attn_case(B, Hq, Hkv, D, BF, prefix, [1] * B, seed=seed, extra_tokens=room)
    return inp


def _acts(gen, B, nd, nt, geo):
    """Stand-in activations for one round, on the CPU."""
    def rows(n, heads, D):
        return torch.randn(n, heads, D, generator=gen).to(BF)
    (hq_d, hkv_d), (hq_r, hkv_r), (hq_t, hkv_t), D = geo
    def gen_rows(n, hq, hkv):
        return (torch.stack([rows(B, hq, D) for _ in range(n)]), torch.stack([rows(B, hkv, D) for _ in range(n)]),
                torch.stack([rows(B, hkv, D) for _ in range(n)]))
    def chunk_rows(n, hq, hkv):
        return rows(B * n, hq, D), rows(B * n, hkv, D), rows(B * n, hkv, D)
    return {"draft.gen": gen_rows(nd, hq_d, hkv_d), "target.gen": gen_rows(nt, hq_t, hkv_t),
            "router.zd": chunk_rows(nd, hq_r, hkv_r), "target.zd": chunk_rows(nd, hq_t, hkv_t),
            "router.zt": chunk_rows(nt, hq_r, hkv_r), "draft.zt": chunk_rows(nt, hq_d, hkv_d)}


class OracleCache:
    """The oracle's side of one cache.  e4m3 = (k_scale, v_scale): the pools hold E4M3 codes."""

    def __init__(self, inp, hq, e4m3=None):
        self.hq, self.bt, self.e4m3 = hq, inp.block_table, e4m3
        self.sl = inp.seq_lens.numpy().copy()
        if e4m3 is None:
            self.k, self.v = inp.k_pages.clone(), inp.v_pages.clone()
        else:
            self.k = torch.from_numpy(oracle.e4m3_encode(inp.k_pages, 1.0 / e4m3[0]))
            self.v = torch.from_numpy(oracle.e4m3_encode(inp.v_pages, 1.0 / e4m3[1]))

    def absorb(self, k_new, v_new, q, lens):
        n = int(lens.sum())
        if self.e4m3 is None:
            self.k, self.v, self.sl, st = oracle.kv_append(k_new[:n], v_new[:n], self.bt, self.sl, lens, self.k, self.v)
            assert st == 0
            out, st = oracle.attn(q[:n], self.k, self.v, self.bt, self.sl, lens)
        else:
            ks, vs = self.e4m3
            self.k, self.v, self.sl, st = oracle.kv_append_e4m3(k_new[:n], v_new[:n], self.bt, self.sl, lens, self.k,
                                                                self.v, 1.0 / ks, 1.0 / vs)
            assert st == 0
            out, st = oracle.attn_e4m3(q[:n], self.k, self.v, ks, vs, self.bt, self.sl, lens)
        assert st == 0
        return out


def _oracle_round(d, r, tg, step_d, step_t, hidden, w, b, tau, acts, nd, nt):
    outs = {}
    q, k, v = acts["draft.gen"]
    for t in range(nd):
        outs[f"draft.gen[{t}]"] = d.absorb(k[t], v[t], q[t], oracle.phase_lens(step_d, None, t=t))
    q, k, v = acts["router.zd"]
    outs["router.zd"] = r.absorb(k, v, q, oracle.phase_lens(step_d, None, t=-1))
    scores, dec = oracle.route(hidden, w, b, tau)
    q, k, v = acts["target.zd"]
    outs["target.zd"] = tg.absorb(k, v, q, oracle.phase_lens(step_d, dec, want=0, t=-1))
    d.sl, _ = oracle.rollback(d.sl, step_d, dec)
    r.sl, _ = oracle.rollback(r.sl, step_d, dec)
    q, k, v = acts["target.gen"]
    for t in range(nt):
        outs[f"target.gen[{t}]"] = tg.absorb(k[t], v[t], q[t], oracle.phase_lens(step_t, dec, want=1, t=t))
    lens = oracle.phase_lens(step_t, dec, want=1, t=-1)
    q, k, v = acts["router.zt"]
    outs["router.zt"] = r.absorb(k, v, q, lens)
    q, k, v = acts["draft.zt"]
    outs["draft.zt"] = d.absorb(k, v, q, lens)
    return scores, dec, outs


@pytest.mark.parametrize("draft_e4m3", [None, (0.02, 0.03)])
def test_two_rounds_of_the_step_loop_match_the_oracle(draft_e4m3):
    """draft_e4m3: the draft model's cache holds E4M3 codes (the quantised-draft regime): its tokens are appended
    quantised and decoded over the codes, and the target's step reaches it as a causal chunk over the codes."""
    from paper_2512_05033_b200 import binding
    from paper_2512_05033_b200.step_loop import Cache, StepLoop
    c = H.ctx()
    B, D, nd, nt, Hd = 4, 128, 5, 4, 256
    geo = ((12, 2), (28, 4), (32, 8), D)
    prefix = [300, 33, 1000, 64]
    room = 3 * (nd + nt) + 16
    inps = [_cache(B, hq, hkv, D, prefix, 400 + i, room) for i, (hq, hkv) in enumerate(geo[:3])]
    ora = [OracleCache(i, hq, draft_e4m3 if k == 0 else None) for k, (i, (hq, _)) in enumerate(zip(inps, geo[:3]))]
    dev_caches = [Cache(o.hq, o.k.cuda(), o.v.cuda(), i.block_table.cuda(), i.seq_lens.cuda(), e4m3=o.e4m3)
                  for i, o in zip(inps, ora)]
    g = torch.Generator().manual_seed(12)
    w = (torch.randn(Hd, generator=g) / Hd ** 0.5).to(BF)
    loop = StepLoop(c, *dev_caches, w.cuda(), 0.0, 0.5, nd, nt)
    for rnd in range(2):
        step_d = torch.randint(1, nd + 1, (B,), generator=g, dtype=torch.int32)
        step_t = torch.randint(1, nt + 1, (B,), generator=g, dtype=torch.int32)
        hidden = (torch.randn(B, Hd, generator=g) * 3).to(BF)          # scores well away from tau
        acts = _acts(g, B, nd, nt, geo)
        dacts = {k: tuple(t.cuda() for t in v) for k, v in acts.items()}
        dec = loop.round(step_d.cuda(), step_t.cuda(), hidden.cuda(), dacts)
        s_ref, d_ref, o_ref = _oracle_round(*ora, step_d.numpy(), step_t.numpy(), hidden, w, 0.0, 0.5, acts, nd, nt)
        assert c.poll_status() == 0
        assert np.abs(s_ref - 0.5).min() > 1e-3 and np.array_equal(dec.cpu().numpy(), d_ref)
        assert 0 < d_ref.sum() < B or rnd == 0                            # both branches are taken
        for dc, oc in zip(dev_caches, ora):                               # caches: bit-exact
            assert np.array_equal(dc.seq_lens.cpu().numpy(), oc.sl)
            assert torch.equal(dc.k_pages.cpu(), oc.k) and torch.equal(dc.v_pages.cpu(), oc.v)
        for name, ref in o_ref.items():                                    # attention of every phase
            n = ref.shape[0]
            if n:
                H.assert_close(loop.out[name][:n].double().cpu().numpy(), ref, BF, tight=3e-3)


def test_phase_lens_matches_oracle():
    c = H.ctx()
    g = torch.Generator().manual_seed(2)
    step = torch.randint(-2, 9, (70,), generator=g, dtype=torch.int32)
    dec = torch.randint(0, 2, (70,), generator=g, dtype=torch.uint8)
    for decisions in (None, dec):
        for want in (0, 1):
            for t in (-1, 0, 3, 8):
                got = c.phase_lens(step.cuda(), None if decisions is None else decisions.cuda(), want=want, t=t)
                assert np.array_equal(got.cpu().numpy(), oracle.phase_lens(step, decisions, want=want, t=t))
            table = c.phase_lens_tokens(step.cuda(), 9, None if decisions is None else decisions.cuda(), want=want)
            for t in range(9):   # one launch for all tokens of a step: row t is the call for token t
                assert np.array_equal(table[t].cpu().numpy(), oracle.phase_lens(step, decisions, want=want, t=t))
