"""One round of the step-level generation loop (Algorithm 1 of the paper) as a fixed sequence of library
calls: no arithmetic of the method happens here, and no length or routing decision is read on the host.

There are no models in this repository, so the "models" are stand-ins that hand out seeded random query,
key and value rows; what is real is everything the loop does to the three paged caches and the attention
work it causes:

  draft cache    the draft model writes its step z_d token by token (one arb_decode_step per token: cache
                 write, decode attention and length update in one launch); if the step is escalated it drops z_d (arb_rollback) and later absorbs the target's
                 step z_t as one chunk (arb_kv_append + chunk arb_attn)
  router cache   absorbs z_d as one chunk -- the router's single forward over (x, z_d), Section 4.2 -- and
                 the head turns the last token's hidden row into the decision (arb_route); on escalation it
                 drops z_d and absorbs z_t
  target cache   absorbs accepted draft steps as one chunk; generates z_t token by token for the escalated

A cache may be an E4M3 cache (Cache.e4m3 = its two scales): the reduced-precision cache of a quantised draft
(Section 5.1).  Its tokens go through arb_decode_step_e4m3, the chunks it absorbs through arb_kv_append_e4m3 and
arb_attn_e4m3.

Which sequences take part in a phase comes from arb_phase_lens / arb_phase_lens_tokens on the device.  A round is therefore a fixed
list of kernel launches for given maximum step lengths and can be captured in a CUDA graph.
"""
from __future__ import annotations

import dataclasses

import torch

from . import binding


@dataclasses.dataclass
class Cache:
    """One model's paged KV cache and head geometry (all tensors on the device)."""
    num_q_heads: int
    k_pages: torch.Tensor      # [num_pages, Hkv, 16, D]
    v_pages: torch.Tensor
    block_table: torch.Tensor  # int32 [B, max_pages]
    seq_lens: torch.Tensor     # int32 [B], advanced and rolled back in place
    e4m3: tuple | None = None  # (k_scale, v_scale): the pools hold E4M3 codes (uint8), keys = k_scale * code


class StepLoop:
    """Runs rounds of Algorithm 1 over a batch.  `rows` supplies the stand-in activations:
    rows(name, n_rows, heads, dim) -> tensor [n_rows, heads, dim] of the cache's dtype (seeded by the caller)."""

    def __init__(self, ctx: binding.Context, draft: Cache, router: Cache, target: Cache, w: torch.Tensor, b: float,
                 tau: float, max_draft_step: int, max_target_step: int):
        self.ctx, self.draft, self.router, self.target = ctx, draft, router, target
        self.w, self.b, self.tau = w, float(b), float(tau)
        self.nd, self.nt = int(max_draft_step), int(max_target_step)
        B = draft.seq_lens.shape[0]
        dev = draft.seq_lens.device
        self.B = B
        self.lens = torch.zeros(B, dtype=torch.int32, device=dev)       # lengths of the call in flight
        # ... of every token of a step that is generated token by token (one row per token)
        self.token_lens = {"draft.gen": torch.zeros(self.nd, B, dtype=torch.int32, device=dev),
                           "target.gen": torch.zeros(self.nt, B, dtype=torch.int32, device=dev)}
        self.scores = torch.empty(B, dtype=torch.float32, device=dev)
        self.decisions = torch.empty(B, dtype=torch.uint8, device=dev)
        self.out = {}                                                    # last outputs of every phase, by name

    # -- building blocks ---------------------------------------------------------------------------
    def _absorb(self, name: str, c: Cache, k_new, v_new, q, lens, max_len: int):
        """The cache takes `lens[b]` new tokens per sequence and attends from them (causal chunk)."""
        out = self.out.get(name)
        if out is None or out.shape != q.shape:
            out = self.out[name] = torch.zeros_like(q)
        if c.e4m3 is not None:   # a quantised cache: quantising append, attention over the codes
            ks, vs = c.e4m3
            self.ctx.kv_append_e4m3(k_new, v_new, 1.0 / ks, 1.0 / vs, c.block_table, c.seq_lens, lens, c.k_pages, c.v_pages)
            self.ctx.attn_e4m3(q, c.k_pages, c.v_pages, ks, vs, c.block_table, c.seq_lens, lens, max_len, out=out)
            return
        self.ctx.kv_append(k_new, v_new, c.block_table, c.seq_lens, lens, c.k_pages, c.v_pages)
        self.ctx.attn(q, c.k_pages, c.v_pages, c.block_table, c.seq_lens, lens, max_len, out=out)

    def _generate(self, name: str, c: Cache, step_lens, decisions, want: int, n_max: int, q, k_new, v_new):
        """Token-by-token generation of a step by the model that owns `c`: q, k_new, v_new are [n_max, B, ...];
        at token t only sequences that take part and have t < step_lens[b] are active."""
        lens = self.ctx.phase_lens_tokens(step_lens, n_max, decisions, want=want, out=self.token_lens[name])
        for t in range(n_max):   # one launch per token: cache write, attention and length update (arb_decode_step)
            key = f"{name}[{t}]"
            out = self.out.get(key)
            if out is None or out.shape != q[t].shape:
                out = self.out[key] = torch.zeros_like(q[t])
            if c.e4m3 is not None:   # a quantised cache: the same token over codes (arb_decode_step_e4m3)
                ks, vs = c.e4m3
                self.ctx.decode_step_e4m3(q[t], k_new[t], v_new[t], c.k_pages, c.v_pages, ks, vs, 1.0 / ks, 1.0 / vs,
                                          c.block_table, c.seq_lens, lens[t], out=out)
                continue
            self.ctx.decode_step(q[t], k_new[t], v_new[t], c.k_pages, c.v_pages, c.block_table, c.seq_lens, lens[t],
                                 out=out)

    # -- one round ---------------------------------------------------------------------------------
    def round(self, step_d, step_t, hidden, acts):
        """step_d, step_t: int32 [B] lengths of the draft's step and of the target's replacement;
        hidden: [B, H] rows the router head reads; acts: dict of stand-in activations:
          'draft.gen' -> (q [nd, B, Hq_d, D], k [nd, B, Hkv_d, D], v), 'target.gen' likewise with nt,
          'router.zd', 'target.zd', 'router.zt', 'draft.zt' -> (q [B * n, Hq, D], k [B * n, Hkv, D], v)."""
        d, r, tg, c = self.draft, self.router, self.target, self.ctx
        # 1. the draft model writes its step
        self._generate("draft.gen", d, step_d, None, 1, self.nd, *acts["draft.gen"])
        # 2. the router reads (x, z_d) in one forward and decides
        c.phase_lens(step_d, None, t=-1, out=self.lens)
        q, k, v = acts["router.zd"]
        self._absorb("router.zd", r, k, v, q, self.lens, self.nd)
        c.route(hidden, self.w, self.b, self.tau, scores=self.scores, decisions=self.decisions)
        # 3. accepted steps: the target's cache catches up with z_d
        c.phase_lens(step_d, self.decisions, want=0, t=-1, out=self.lens)
        q, k, v = acts["target.zd"]
        self._absorb("target.zd", tg, k, v, q, self.lens, self.nd)
        # 4. escalated steps: draft and router forget z_d, the target regenerates the step from the same prefix
        c.rollback(d.seq_lens, step_d, self.decisions)
        c.rollback(r.seq_lens, step_d, self.decisions)
        self._generate("target.gen", tg, step_t, self.decisions, 1, self.nt, *acts["target.gen"])
        # 5. ... and the caches that did not generate z_t catch up with it
        c.phase_lens(step_t, self.decisions, want=1, t=-1, out=self.lens)
        q, k, v = acts["router.zt"]
        self._absorb("router.zt", r, k, v, q, self.lens, self.nt)
        q, k, v = acts["draft.zt"]
        self._absorb("draft.zt", d, k, v, q, self.lens, self.nt)
        return self.decisions
