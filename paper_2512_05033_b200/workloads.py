"""Seeded synthetic inputs for the five workloads.

This module holds NO arithmetic of the method: it only draws lengths, page permutations and
N(0, sigma^2) tensors with a seeded generator and rounds them once to the storage dtype.  Both the
CUDA path and the CPU oracle consume exactly these tensors.

The workloads stand in for the paper's runs of LLaMA3 / Qwen2.5-Math draft, target and router
models on math-reasoning benchmarks (Section 5.1): only tensor shapes and length distributions
matter to this path.
"""
from __future__ import annotations

import dataclasses
import math
from typing import Optional

import torch

PAGE = 16


@dataclasses.dataclass(frozen=True)
class AttnShape:
    name: str
    batch: int
    num_q_heads: int
    num_kv_heads: int
    head_dim: int
    dtype: torch.dtype
    prefix_lo: int               # prefix (already cached context) length range, inclusive
    prefix_hi: int
    q_lo: int = 1                # new tokens per sequence, inclusive range
    q_hi: int = 1
    prefix_dist: str = "uniform"  # "uniform" | "lognormal" | "fixed"
    hidden: int = 0              # router hidden size (0 = no router in this workload)
    seed: int = 0


TINY_DECODE = AttnShape("tiny-decode", 1, 8, 2, 64, torch.float32, 512, 512, 1, 1, "fixed", 256, 0)
TINY_CHUNK = AttnShape("tiny-chunk", 1, 8, 2, 64, torch.float32, 512, 512, 16, 16, "fixed", 256, 0)
DRAFT_DECODE = AttnShape("draft-shaped decode", 8, 12, 2, 128, torch.bfloat16, 1024, 8192, seed=1)
TARGET_DECODE = AttnShape("target-shaped decode", 16, 32, 8, 128, torch.bfloat16, 4096, 32768, seed=2)
STEP_SCORING = AttnShape("step scoring + routing", 32, 28, 4, 128, torch.bfloat16, 2048, 16384,
                         16, 128, "uniform", 3584, 3)
MIXED_LOOP = AttnShape("mixed serving loop", 64, 32, 8, 128, torch.bfloat16, 256, 65536,
                       16, 128, "lognormal", 3584, 4)

CONFIGS = {c.name: c for c in (TINY_DECODE, TINY_CHUNK, DRAFT_DECODE, TARGET_DECODE, STEP_SCORING,
                               MIXED_LOOP)}


def _cpu_gen(seed: int) -> torch.Generator:
    g = torch.Generator(device="cpu")
    g.manual_seed(int(seed))
    return g


def draw_prefix_lens(shape: AttnShape, gen: torch.Generator) -> torch.Tensor:
    """Prefix lengths (tokens already in the cache before the new ones), int64 [batch]."""
    B = shape.batch
    if shape.prefix_dist == "fixed":
        return torch.full((B,), shape.prefix_lo, dtype=torch.int64)
    if shape.prefix_dist == "uniform":
        return torch.randint(shape.prefix_lo, shape.prefix_hi + 1, (B,), generator=gen)
    if shape.prefix_dist == "lognormal":  # median 8192, sigma 0.8 in log space, clipped
        z = torch.randn(B, generator=gen, dtype=torch.float64)
        L = torch.exp(math.log(8192.0) + 0.8 * z).round().to(torch.int64)
        return L.clamp(shape.prefix_lo, shape.prefix_hi)
    raise ValueError(shape.prefix_dist)


def draw_q_lens(shape: AttnShape, gen: torch.Generator) -> torch.Tensor:
    if shape.q_lo == shape.q_hi:
        return torch.full((shape.batch,), shape.q_lo, dtype=torch.int64)
    return torch.randint(shape.q_lo, shape.q_hi + 1, (shape.batch,), generator=gen)


def normal(shape, std: float, dtype: torch.dtype, device, seed: int) -> torch.Tensor:
    """N(0, std^2) drawn in fp32 on `device` with its own seeded generator, rounded once to dtype."""
    device = torch.device(device)
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    t = torch.randn(shape, generator=g, device=device, dtype=torch.float32)
    if std != 1.0:
        t.mul_(std)
    return t.to(dtype)


@dataclasses.dataclass
class AttnInputs:
    shape: AttnShape
    q: torch.Tensor            # [total_q, Hq, D]
    k_pages: torch.Tensor      # [num_pages, Hkv, PAGE, D]
    v_pages: torch.Tensor
    block_table: torch.Tensor  # int32 [B, max_pages]
    seq_lens: torch.Tensor     # int32 [B]  (prefix + q_len)
    q_lens: torch.Tensor       # int32 [B]

    @property
    def total_q(self) -> int:
        return int(self.q.shape[0])

    @property
    def num_pages(self) -> int:
        return int(self.k_pages.shape[0])

    @property
    def max_pages(self) -> int:
        return int(self.block_table.shape[1])

    def kv_tokens(self) -> int:
        return int(self.seq_lens.sum())

    def to(self, device) -> "AttnInputs":
        return dataclasses.replace(
            self, **{f: getattr(self, f).to(device) for f in
                     ("q", "k_pages", "v_pages", "block_table", "seq_lens", "q_lens")})


def make_block_table(seq_lens: torch.Tensor, gen: torch.Generator, extra_tokens: int = 0,
                     headroom_pages: int = 0, fill: int = -1):
    """Random permutation of a shared page pool cut into per-sequence page lists.

    Returns (block_table int32 [B, max_pages], num_pages).  Each sequence gets pages for
    seq_len + extra_tokens tokens; entries beyond that hold `fill` (never read by a correct kernel).
    """
    cap = (seq_lens + extra_tokens + PAGE - 1) // PAGE
    B = int(seq_lens.shape[0])
    max_pages = int(cap.max())
    used = int(cap.sum())
    num_pages = used + headroom_pages
    perm = torch.randperm(num_pages, generator=gen).to(torch.int32)
    bt = torch.full((B, max_pages), fill, dtype=torch.int32)
    at = 0
    for b in range(B):
        n = int(cap[b])
        bt[b, :n] = perm[at:at + n]
        at += n
    return bt, num_pages


def make_attn_inputs(shape: AttnShape, device="cpu", seed: Optional[int] = None,
                     q_std: float = 1.0, extra_tokens: int = 0,
                     prefix_lens: Optional[torch.Tensor] = None,
                     q_lens: Optional[torch.Tensor] = None) -> AttnInputs:
    """One layer-call worth of inputs for `shape`.

    Lengths and the page permutation are drawn on the CPU from `seed` (default shape.seed); the
    N(0,1) tensors are drawn on `device` (values differ between CPU and CUDA generators, each is
    reproducible).  q_std > 1 gives the "peaked" variant whose softmax concentrates on few keys.
    """
    seed = shape.seed if seed is None else seed
    gen = _cpu_gen(seed)
    prefix = draw_prefix_lens(shape, gen) if prefix_lens is None else prefix_lens.to(torch.int64)
    ql = draw_q_lens(shape, gen) if q_lens is None else q_lens.to(torch.int64)
    seq = prefix + ql
    bt, num_pages = make_block_table(seq, gen, extra_tokens=extra_tokens, headroom_pages=3)
    total_q = int(ql.sum())
    H, Hk, D = shape.num_q_heads, shape.num_kv_heads, shape.head_dim
    q = normal((total_q, H, D), q_std, shape.dtype, device, seed * 1000 + 1)
    k = normal((num_pages, Hk, PAGE, D), 1.0, shape.dtype, device, seed * 1000 + 2)
    v = normal((num_pages, Hk, PAGE, D), 1.0, shape.dtype, device, seed * 1000 + 3)
    return AttnInputs(shape, q, k, v, bt.to(device), seq.to(torch.int32).to(device),
                      ql.to(torch.int32).to(device))


def make_kv_pool(shape: AttnShape, num_pages: int, device, seed: int):
    """A further K/V pool of the same geometry (another layer's cache) for rotating over layers."""
    Hk, D = shape.num_kv_heads, shape.head_dim
    k = normal((num_pages, Hk, PAGE, D), 1.0, shape.dtype, device, seed * 1000 + 2)
    v = normal((num_pages, Hk, PAGE, D), 1.0, shape.dtype, device, seed * 1000 + 3)
    return k, v


@dataclasses.dataclass
class RouterInputs:
    hidden: torch.Tensor  # [n_steps, H]
    w: torch.Tensor       # [H]
    b: float
    taus: tuple


def make_router_inputs(n_steps: int, hidden_dim: int, dtype: torch.dtype, device="cpu", seed: int = 0,
                       b_std: float = 0.0, taus=(0.5,)) -> RouterInputs:
    """hidden ~ N(0,1); w ~ N(0, 1/H) (variance), so z = hidden.w + b is about N(0,1); b ~ N(0, b_std^2)."""
    hidden = normal((n_steps, hidden_dim), 1.0, dtype, device, seed * 1000 + 11)
    w = normal((hidden_dim,), 1.0 / math.sqrt(hidden_dim), dtype, device, seed * 1000 + 12)
    b = 0.0
    if b_std > 0.0:
        b = float(torch.randn(1, generator=_cpu_gen(seed * 1000 + 13)).item() * b_std)
    return RouterInputs(hidden, w, b, tuple(taus))


def small_attn_case(batch, num_q_heads, num_kv_heads, head_dim, dtype, seq_lens, q_lens, seed,
                    device="cpu", q_std: float = 1.0, extra_tokens: int = 0) -> AttnInputs:
    """Explicit lengths (lists) for parity and edge-case tests."""
    seq = torch.as_tensor(seq_lens, dtype=torch.int64)
    ql = torch.as_tensor(q_lens, dtype=torch.int64)
    shape = AttnShape(f"case-{seed}", batch, num_q_heads, num_kv_heads, head_dim, dtype, 0, 0, seed=seed)
    gen = _cpu_gen(seed)
    bt, num_pages = make_block_table(torch.clamp(seq, min=1), gen, extra_tokens=extra_tokens,
                                     headroom_pages=2)
    total_q = int(ql.clamp(min=0).sum())
    q = normal((total_q, num_q_heads, head_dim), q_std, dtype, device, seed * 1000 + 1)
    k = normal((num_pages, num_kv_heads, PAGE, head_dim), 1.0, dtype, device, seed * 1000 + 2)
    v = normal((num_pages, num_kv_heads, PAGE, head_dim), 1.0, dtype, device, seed * 1000 + 3)
    return AttnInputs(shape, q, k, v, bt.to(device), seq.to(torch.int32).to(device),
                      ql.to(torch.int32).to(device))


@dataclasses.dataclass
class MixedLoopInputs:
    """Everything the mixed serving loop draws: one KV pool whose slots already hold N(0,1) values
    (so appending a token is just a longer seq_len), the starting lengths, and per iteration the
    query lengths (even index + iteration: decode, q_len 1; odd: a step of 16..128 tokens), the query
    rows and the router's hidden rows."""
    shape: AttnShape
    k_pages: torch.Tensor
    v_pages: torch.Tensor
    block_table: torch.Tensor      # int32 [B, max_pages], capacity for every append of the loop
    seq_lens0: torch.Tensor        # int32 [B] lengths before the first iteration
    q_lens: list                   # per iteration int32 [B]
    q: list                        # per iteration [sum q_lens, Hq, D]
    hidden: list                   # per iteration [B, hidden]
    w: torch.Tensor
    b: float
    tau: float = 0.5


def make_mixed_loop(shape: AttnShape = MIXED_LOOP, iterations: int = 10, device="cpu",
                    seed: Optional[int] = None) -> MixedLoopInputs:
    seed = shape.seed if seed is None else seed
    gen = _cpu_gen(seed)
    B = shape.batch
    prefix = draw_prefix_lens(shape, gen)
    idx = torch.arange(B)
    q_lens, total_new = [], torch.zeros(B, dtype=torch.int64)
    for it in range(iterations):
        steps = torch.randint(shape.q_lo, shape.q_hi + 1, (B,), generator=gen)
        ql = torch.where((idx + it) % 2 == 0, torch.ones(B, dtype=torch.int64), steps)
        q_lens.append(ql)
        total_new += ql
    bt, num_pages = make_block_table(prefix, gen, extra_tokens=int(total_new.max()), headroom_pages=3)
    H, Hk, D = shape.num_q_heads, shape.num_kv_heads, shape.head_dim
    k = normal((num_pages, Hk, PAGE, D), 1.0, shape.dtype, device, seed * 1000 + 2)
    v = normal((num_pages, Hk, PAGE, D), 1.0, shape.dtype, device, seed * 1000 + 3)
    q = [normal((int(ql.sum()), H, D), 1.0, shape.dtype, device, seed * 1000 + 100 + it)
         for it, ql in enumerate(q_lens)]
    hidden = [normal((B, shape.hidden), 1.0, shape.dtype, device, seed * 1000 + 200 + it)
              for it in range(iterations)]
    w = normal((shape.hidden,), 1.0 / math.sqrt(shape.hidden), shape.dtype, device, seed * 1000 + 12)
    return MixedLoopInputs(shape, k, v, bt.to(device), prefix.to(torch.int32).to(device),
                           [x.to(torch.int32).to(device) for x in q_lens], q, hidden, w, 0.0, 0.5)
