"""Shared by the GPU parity tests: run the CUDA path through the C ABI and the oracle on the same inputs."""
import numpy as np
import torch

from oracle import oracle

_ctx = None


def ctx():
    global _ctx
    if _ctx is None:
        from paper_2512_05033_b200 import binding
        _ctx = binding.Context(0)
    return _ctx


def gpu_attn(inp, scale=0.0, flags=0):
    """inp: workloads.AttnInputs on the CPU.  Returns (out fp64 numpy, status bits)."""
    d = inp.to("cuda")
    max_q = int(inp.q_lens.max()) if inp.q_lens.numel() else 0
    # `out` lies between two guard rows: a store before its first or past its last row would show in them
    guard = 12345.0
    buf = torch.full((d.q.shape[0] + 2,) + tuple(d.q.shape[1:]), guard, dtype=d.q.dtype, device="cuda")
    out = buf[1:-1]
    out.fill_(float("nan"))
    c = ctx()
    p = c.params_for(d.q, d.k_pages, d.block_table, max_q, scale, flags=flags)
    c.attn(d.q, d.k_pages, d.v_pages, d.block_table, d.seq_lens, d.q_lens, max_q, out=out, params=p)
    bits = c.poll_status()
    assert bool((buf[0] == guard).all()) and bool((buf[-1] == guard).all()), "a row outside `out` was written"
    return out.double().cpu().numpy(), bits


def guard_zones():
    """(overwritten, checked) guard bytes of the shared context; (0, 0) unless the bounds-check build is loaded."""
    return _ctx.guard_zones() if _ctx is not None else (0, 0)


def oracle_attn(inp, scale=0.0):
    return oracle.attn(inp.q, inp.k_pages, inp.v_pages, inp.block_table, inp.seq_lens, inp.q_lens, scale)


def tol_for(dtype):
    # bf16 inputs, fp32 accumulation, bf16 output: 1e-2 max-abs; fp32: 1e-5
    return 1e-2 if dtype == torch.bfloat16 else 1e-5


def assert_close(gpu, ref, dtype, tight=None):
    err = np.abs(gpu - ref)
    assert np.isfinite(gpu).all(), "non-finite output"
    tol = tol_for(dtype)
    assert err.max() <= tol, f"max-abs error {err.max():.3e} > {tol}"
    if tight is not None:
        # internal bar: the bf16 rounding of the output (2^-9 relative) plus `tight` for the fp32 path
        bar = 2.0 ** -8 * np.abs(ref) + tight
        assert (err <= bar).all(), f"error {err.max():.3e} above the internal bar ({tight} + bf16 rounding)"
    return float(err.max())
