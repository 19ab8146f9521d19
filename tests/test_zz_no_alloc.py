"""arb_attn_decode_static: the entry point for hosts that must not allocate.

Some embedders cannot call cudaMalloc once they are running -- all free device memory already
belongs to their KV pool, or they sit inside another framework's operator where an allocation stalls
the device.  They cannot hold an arb_ctx (creating one allocates), so this call keeps its split-KV
scratch in a fixed array inside the library.  The test drives it through the C ABI and compares it
with arb_attn on the same inputs (bit for bit against the CUDA-core kernel it shares, within tolerance
against the default tensor-core kernel) and with the fp64 oracle, several times in a row with different
inputs, because the shared array keeps the previous call's contents.  This file is collected last on purpose.
"""
import ctypes

import numpy as np
import pytest
import torch

from oracle import oracle
from paper_2512_05033_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def _both(binding, ctx, inp):
    d = inp.to("cuda")
    ref = ctx.attn(d.q, d.k_pages, d.v_pages, d.block_table, d.seq_lens, d.q_lens, 1)
    same_kernel = ctx.attn(d.q, d.k_pages, d.v_pages, d.block_table, d.seq_lens, d.q_lens, 1,
                           params=ctx.params_for(d.q, d.k_pages, d.block_table, 1, flags=binding.ATTN_NO_TENSOR_CORES))
    out = torch.full_like(d.q, float("nan"))          # allocated by the test, not by the library
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    p = binding.attn_params(binding.ARB_BF16, d.block_table.shape[0], d.q.shape[1], d.k_pages.shape[1],
                            d.q.shape[2], d.k_pages.shape[0], d.block_table.shape[1], d.q.shape[0], 1)
    st = binding.lib.arb_attn_decode_static(ctypes.byref(p), d.q.data_ptr(), d.k_pages.data_ptr(),
                                            d.v_pages.data_ptr(), d.block_table.data_ptr(), d.seq_lens.data_ptr(),
                                            d.q_lens.data_ptr(), out.data_ptr(), status.data_ptr(),
                                            torch.cuda.current_stream().cuda_stream)
    assert st == binding.ARB_OK
    torch.cuda.synchronize()
    assert int(status.item()) == 0 and ctx.poll_status() == 0
    assert torch.equal(out, same_kernel)     # arb_attn on the CUDA-core decode kernel: the same kernel, the same plan
    return out.double().cpu().numpy(), ref.double().cpu().numpy()


def test_static_entry_point_matches_arb_attn_twice_in_a_row():
    from paper_2512_05033_b200 import binding
    ctx = binding.Context(0)
    first = wl.small_attn_case(6, 12, 2, 128, torch.bfloat16, [7000, 33, 1200, 1, 4096, 500], [1] * 6, seed=91)
    second = wl.small_attn_case(3, 32, 8, 128, torch.bfloat16, [9000, 2500, 64], [1, 1, 1], seed=92)
    for inp in (first, second, first):
        out, ref = _both(binding, ctx, inp)
        assert np.isfinite(out).all()
        # arb_attn may take the tensor-core decode kernel, the static call always the CUDA-core one
        assert np.abs(out - ref).max() <= 1e-2
        assert (np.abs(out - ref) <= 2.0 ** -7 * np.abs(ref) + 3e-3).all()
        # and the definition itself, at the bar of the CUDA-core kernels
        exact, st = oracle.attn(inp.q, inp.k_pages, inp.v_pages, inp.block_table, inp.seq_lens, inp.q_lens)
        assert st == 0
        assert (np.abs(out - exact) <= 2.0 ** -8 * np.abs(exact) + 1e-3).all(), np.abs(out - exact).max()
    ctx.close()


def test_static_entry_point_refuses_what_it_cannot_hold():
    from paper_2512_05033_b200 import binding
    inp = wl.small_attn_case(2, 8, 2, 64, torch.float32, [40, 50], [1, 1], seed=93).to("cuda")
    out = torch.empty_like(inp.q)
    args = [inp.q.data_ptr(), inp.k_pages.data_ptr(), inp.v_pages.data_ptr(), inp.block_table.data_ptr(),
            inp.seq_lens.data_ptr(), inp.q_lens.data_ptr(), out.data_ptr(), None, 0]
    big = binding.attn_params(binding.ARB_F32, 1024, 8, 2, 64, inp.k_pages.shape[0], inp.block_table.shape[1], 1024, 1)
    assert binding.lib.arb_attn_decode_static(ctypes.byref(big), *args) == binding.ARB_ERR_STATIC_LIMIT
    assert b"scratch" in binding.lib.arb_status_string(binding.ARB_ERR_STATIC_LIMIT)
    chunk = binding.attn_params(binding.ARB_F32, 2, 8, 2, 64, inp.k_pages.shape[0], inp.block_table.shape[1], 2, 2)
    assert binding.lib.arb_attn_decode_static(ctypes.byref(chunk), *args) == binding.ARB_ERR_INVALID_ARG
    ovl = binding.attn_params(binding.ARB_F32, 2, 8, 2, 64, inp.k_pages.shape[0], inp.block_table.shape[1], 2, 1,
                              flags=binding.ATTN_OVERLAP_PREVIOUS)
    assert binding.lib.arb_attn_decode_static(ctypes.byref(ovl), *args) == binding.ARB_ERR_INVALID_ARG
    ok = binding.attn_params(binding.ARB_F32, 2, 8, 2, 64, inp.k_pages.shape[0], inp.block_table.shape[1], 2, 1)
    assert binding.lib.arb_attn_decode_static(ctypes.byref(ok), *args) == binding.ARB_OK
    torch.cuda.synchronize()
