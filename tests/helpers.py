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
    out = torch.full_like(d.q, float("nan"))
    c = ctx()
    p = c.params_for(d.q, d.k_pages, d.block_table, max_q, scale, flags=flags)
    c.attn(d.q, d.k_pages, d.v_pages, d.block_table, d.seq_lens, d.q_lens, max_q, out=out, params=p)
    bits = c.poll_status()
    return out.double().cpu().numpy(), bits


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
