"""Parity of arb_attn (CUDA, through the C ABI) with the fp64 oracle, element by element."""
import numpy as np
import pytest
import torch

from oracle import oracle
from paper_2512_05033_b200 import workloads as wl
from tests import helpers as H

pytestmark = pytest.mark.gpu

BF, F32 = torch.bfloat16, torch.float32

DECODE_CASES = [
    # (B, Hq, Hkv, D, dtype, seq_lens)                       what it covers
    (1, 8, 2, 64, F32, [513]),                               # the tiny config: prefix 512 + 1
    (1, 8, 2, 64, F32, [1]),                                 # a single key
    (3, 12, 2, 128, BF, [16, 17, 15]),                       # page boundaries
    (8, 12, 2, 128, BF, [1025, 2000, 3001, 777, 4096, 1, 640, 5555]),   # draft-shaped, ragged
    (4, 32, 8, 128, BF, [4100, 9000, 33, 12000]),            # target-shaped heads
    (2, 28, 4, 128, BF, [3000, 150]),                        # g = 7 (odd group)
    (2, 6, 2, 64, BF, [700, 70]),                            # bf16, head_dim 64
    (2, 4, 2, 128, F32, [900, 31]),                          # fp32, head_dim 128
    (1, 5, 1, 128, BF, [40000]),                             # one long sequence over every CTA
    (2, 3, 3, 64, F32, [260, 100]),                          # g = 1
    (2, 16, 2, 128, BF, [2100, 900]),                        # g = 8
]


@pytest.mark.parametrize("cuda_cores", [False, True])
@pytest.mark.parametrize("case", DECODE_CASES)
def test_decode_matches_oracle(case, cuda_cores):
    """Both decode kernels: the default choice and, with ARB_ATTN_NO_TENSOR_CORES, the CUDA-core one."""
    from paper_2512_05033_b200 import binding
    B, Hq, Hkv, D, dt, sl = case
    inp = wl.small_attn_case(B, Hq, Hkv, D, dt, sl, [1] * B, seed=100 + len(sl) + Hq)
    out, bits = H.gpu_attn(inp, flags=binding.ATTN_NO_TENSOR_CORES if cuda_cores else 0)
    ref, st = H.oracle_attn(inp)
    assert bits == 0 and st == 0
    on_mma = (not cuda_cores) and dt == BF and D == 128 and Hq // Hkv <= 8
    H.assert_close(out, ref, dt, tight=(3e-3 if on_mma else 1e-3) if dt == BF else None)


def test_decode_peaked_softmax():
    """q scaled up so the softmax concentrates and outputs are O(1): the tolerance bites."""
    inp = wl.small_attn_case(4, 12, 2, 128, BF, [3000, 513, 64, 1500], [1] * 4, seed=7, q_std=6.0)
    out, bits = H.gpu_attn(inp)
    ref, _ = H.oracle_attn(inp)
    assert bits == 0
    err = np.abs(out - ref)
    # output is rounded to bf16 (2^-9 relative); the rest is the fp32 path
    assert (err <= 2.0 ** -8 * np.abs(ref) + 2e-3).all(), err.max()


def test_decode_idle_slots_and_scale():
    inp = wl.small_attn_case(5, 8, 2, 64, F32, [100, 1, 300, 1, 47], [1, 0, 1, 0, 1], seed=31)
    out, bits = H.gpu_attn(inp, scale=0.2)
    ref, _ = H.oracle_attn(inp, scale=0.2)
    assert bits == 0 and out.shape[0] == 3
    H.assert_close(out, ref, F32)


CHUNK_CASES = [
    # bf16 / head_dim 128 chunks run on the tensor cores, whatever their size
    (1, 32, 8, 128, BF, [300], [64]),                        # g = 4: 256 rows = two full row tiles
    (2, 28, 4, 128, BF, [600, 2100], [16, 100]),             # g = 7: 112 rows (one ragged tile), 700 rows
    (2, 12, 2, 128, BF, [131, 128], [128, 11]),              # chunk is almost the whole sequence; 66 rows
    (4, 32, 8, 128, BF, [5000, 77, 1300, 256], [1, 30, 128, 5]),   # decode rows beside large and small chunks
    (1, 16, 2, 128, BF, [4099], [19]),                       # g = 8: 152 rows, key count not a page multiple
    (3, 12, 2, 128, BF, [2, 17, 300], [2, 3, 2]),            # smallest chunks: 12 and 18 rows; the chunk is the whole sequence
    (2, 8, 8, 128, BF, [40, 300], [2, 9]),                   # g = 1: 2 and 9 rows in a 128-row tile
    (3, 16, 2, 128, BF, [33, 1000, 129], [3, 7, 1]),         # g = 8: 24 and 56 rows beside a decode row
    # few work items and sequences of 8 KV tiles and more: the call is cut over the keys to fill the SMs
    (3, 12, 2, 128, BF, [5000, 2500, 300], [24, 9, 1]),      # parts of two chunk sequences beside a decode row
    (2, 32, 8, 128, BF, [6000, 3000], [40, 64]),             # g = 4, one and two row tiles per sequence
    (1, 8, 2, 64, F32, [528], [16]),                         # the tiny config: 16-token chunk, prefix 512
    (2, 12, 2, 128, BF, [300, 40], [7, 40]),                 # chunk == whole sequence (no prefix)
    (3, 28, 4, 128, BF, [200, 90, 1000], [3, 1, 5]),         # decode and chunk rows in one call
    (2, 4, 4, 64, BF, [33, 64], [2, 17]),
    (2, 8, 1, 128, F32, [129, 50], [9, 2]),
]


SPLIT_CASES = [
    # sequences that see more than 160 KV tiles are cut into parts over their keys and merged afterwards
    (1, 32, 8, 128, BF, [26000], [100]),                     # g = 4: 400 rows = a full pair and a ragged one, 3 parts
    (3, 28, 4, 128, BF, [21000, 900, 40000], [40, 64, 17]),  # g = 7: split and unsplit sequences in one call, 4 parts
    (2, 16, 2, 128, BF, [20481, 65536], [16, 16]),           # g = 8: the first tile count that splits, and 64k keys
]


@pytest.mark.parametrize("case", SPLIT_CASES)
def test_split_chunk_matches_oracle(case):
    B, Hq, Hkv, D, dt, sl, ql = case
    inp = wl.small_attn_case(B, Hq, Hkv, D, dt, sl, ql, seed=500 + Hq)
    out, bits = H.gpu_attn(inp)
    ref, st = H.oracle_attn(inp)
    assert bits == 0 and st == 0
    H.assert_close(out, ref, dt, tight=3e-3)


def test_split_chunk_without_room_for_partials():
    """A context too small to hold every partial serves the sequences it has no room for unsplit: same
    results, only slower."""
    from paper_2512_05033_b200 import binding
    B, Hq, Hkv, D, dt, sl, ql = SPLIT_CASES[1]
    inp = wl.small_attn_case(B, Hq, Hkv, D, dt, sl, ql, seed=500 + Hq)
    ref, _ = H.oracle_attn(inp)
    d = inp.to("cuda")
    for ws in (2 << 20,):              # 4 MB for partials: room for the longest sequence's parts, not for the next one's
        c = binding.Context(0, workspace_bytes=ws)
        out = c.attn(d.q, d.k_pages, d.v_pages, d.block_table, d.seq_lens, d.q_lens, max(ql))
        assert c.poll_status() == 0
        H.assert_close(out.double().cpu().numpy(), ref, dt, tight=3e-3)
        c.close()


@pytest.mark.parametrize("case", CHUNK_CASES)
def test_chunk_matches_oracle(case):
    B, Hq, Hkv, D, dt, sl, ql = case
    inp = wl.small_attn_case(B, Hq, Hkv, D, dt, sl, ql, seed=200 + Hq)
    out, bits = H.gpu_attn(inp)
    ref, st = H.oracle_attn(inp)
    assert bits == 0 and st == 0
    # chunks on the tensor cores carry bf16 softmax weights into the second product
    on_mma = dt == BF and D == 128 and max(ql) >= 2
    H.assert_close(out, ref, dt, tight=(3e-3 if on_mma else 1e-3) if dt == BF else None)


def test_large_chunk_peaked_and_stale_slots():
    """Tensor-core chunk path: concentrated softmax, and NaN / 1e30 in the slots after the sequence end."""
    inp = wl.small_attn_case(2, 28, 4, 128, BF, [1000, 333], [40, 64], seed=43, q_std=4.0, extra_tokens=50)
    clean, bits = H.gpu_attn(inp)
    assert bits == 0
    ref, _ = H.oracle_attn(inp)
    err = np.abs(clean - ref)
    # The softmax weights enter the second product rounded to bf16 (relative 2^-9 each) while the denominator
    # sums them in fp32, and the output is rounded to bf16 once more.  Gross bound for every element, the bound
    # that follows from this arithmetic on sampled rows.
    vmax = float(inp.v_pages.abs().max())
    assert (err <= 2.0 ** -8 * np.abs(ref) + 2.0 ** -9 * 2 * vmax).all(), err.max()
    from oracle import oracle
    rng = np.random.default_rng(0)
    rows0 = np.cumsum([0] + [int(x) for x in inp.q_lens])
    Vd = inp.v_pages.double().numpy()
    for _ in range(48):
        b = int(rng.integers(0, 2)); n = int(inp.q_lens[b]); L = int(inp.seq_lens[b])
        i = int(rng.integers(0, n)); h = int(rng.integers(0, 28)); row = rows0[b] + i; pos = L - n + i
        o, p, _ = oracle.attn_row_probs(inp.q, inp.k_pages, inp.v_pages, inp.block_table[b], row, h, pos)
        bt = inp.block_table[b].numpy()
        v = np.stack([Vd[bt[j // wl.PAGE], h // 7, j % wl.PAGE] for j in range(pos + 1)])      # [keys, D]
        bound = 2.0 ** -9 * (p[:, None] * np.abs(v)).sum(axis=0) + 2.0 ** -8 * np.abs(o) + 1e-3
        assert (np.abs(clean[row, h] - o) <= bound).all(), (b, i, h)
    k2, v2 = inp.k_pages.clone(), inp.v_pages.clone()
    for b in range(2):
        L = int(inp.seq_lens[b])
        for j in range(L, L + 50):
            pg = int(inp.block_table[b, j // wl.PAGE])
            k2[pg, :, j % wl.PAGE] = float("nan")
            v2[pg, :, j % wl.PAGE] = 1e30
    out, bits = H.gpu_attn(wl.AttnInputs(inp.shape, inp.q, k2, v2, inp.block_table, inp.seq_lens, inp.q_lens))
    assert bits == 0
    np.testing.assert_array_equal(out, clean)


def test_stale_slots_never_reach_the_output():
    """Slots past each row's position hold NaN / 1e30 (a rolled-back step): the result must not change."""
    inp = wl.small_attn_case(3, 12, 2, 128, BF, [1000, 37, 300], [1, 1, 6], seed=41, extra_tokens=40)
    clean, bits = H.gpu_attn(inp)
    assert bits == 0
    k2, v2 = inp.k_pages.clone(), inp.v_pages.clone()
    for b in range(3):
        L = int(inp.seq_lens[b])
        for j in range(L, L + 40):
            pg = int(inp.block_table[b, j // wl.PAGE])
            k2[pg, :, j % wl.PAGE] = float("nan")
            v2[pg, :, j % wl.PAGE] = 1e30
    pois = wl.AttnInputs(inp.shape, inp.q, k2, v2, inp.block_table, inp.seq_lens, inp.q_lens)
    out, bits = H.gpu_attn(pois)
    assert bits == 0
    np.testing.assert_array_equal(out, clean)
    ref, _ = H.oracle_attn(pois)
    H.assert_close(out, ref, BF)


def test_bad_length_is_flagged_and_zero_filled():
    from paper_2512_05033_b200 import binding
    inp = wl.small_attn_case(3, 8, 2, 64, F32, [50, 3, 20], [1, 5, 1], seed=51)   # seq_len < q_len in slot 1
    out, bits = H.gpu_attn(inp)
    ref, st = H.oracle_attn(inp)
    assert bits & binding.DEV_BAD_SEQ_LEN and st & 1
    assert (out[1:6] == 0).all()
    H.assert_close(out, ref, F32)
    # decode row with seq_len 0
    inp = wl.small_attn_case(2, 8, 2, 64, F32, [0, 20], [1, 1], seed=52)
    out, bits = H.gpu_attn(inp)
    assert bits & binding.DEV_BAD_SEQ_LEN and (out[0] == 0).all()
    ref, _ = H.oracle_attn(inp)
    H.assert_close(out[1:], ref[1:], F32)
    assert H.ctx().poll_status() == 0       # the word was cleared


def test_bad_page_is_flagged_without_a_fault():
    from paper_2512_05033_b200 import binding
    inp = wl.small_attn_case(2, 8, 2, 64, F32, [100, 40], [1, 1], seed=53)
    inp.block_table[0, 2] = inp.num_pages + 7
    out, bits = H.gpu_attn(inp)
    assert bits & binding.DEV_BAD_PAGE
    good = wl.small_attn_case(2, 8, 2, 64, F32, [100, 40], [1, 1], seed=53)
    ref, _ = H.oracle_attn(good)
    H.assert_close(out[1:], ref[1:], F32)    # the other sequence is untouched
    assert np.isfinite(out).all()


def test_host_argument_errors():
    from paper_2512_05033_b200 import binding
    c = H.ctx()
    inp = wl.small_attn_case(1, 8, 2, 64, F32, [40], [1], seed=54).to("cuda")
    p = c.params_for(inp.q, inp.k_pages, inp.block_table, 1)
    args = [inp.q.data_ptr(), inp.k_pages.data_ptr(), inp.v_pages.data_ptr(), inp.block_table.data_ptr(),
            inp.seq_lens.data_ptr(), inp.q_lens.data_ptr(), torch.empty_like(inp.q).data_ptr(), 0]
    assert c.attn_raw(p, *args) == binding.ARB_OK
    bad = list(args); bad[1] = None
    assert c.attn_raw(p, *bad) == binding.ARB_ERR_INVALID_ARG
    bad = list(args); bad[0] = args[0] + 4
    assert c.attn_raw(p, *bad) == binding.ARB_ERR_INVALID_ARG          # misaligned q
    p2 = c.params_for(inp.q, inp.k_pages, inp.block_table, 1); p2.head_dim = 96
    assert c.attn_raw(p2, *args) == binding.ARB_ERR_UNSUPPORTED
    p3 = c.params_for(inp.q, inp.k_pages, inp.block_table, 1); p3.num_q_heads = 7
    assert c.attn_raw(p3, *args) == binding.ARB_ERR_INVALID_ARG         # not a multiple of kv heads
    small = binding.Context(0, workspace_bytes=1024)
    assert small.attn_raw(p, *args) == binding.ARB_ERR_WORKSPACE
    small.close()
    torch.cuda.synchronize()


def test_host_buffer_entry_point():
    inp = wl.small_attn_case(3, 12, 2, 128, BF, [500, 90, 2000], [1, 4, 1], seed=55)
    ref, _ = H.oracle_attn(inp)
    c = H.ctx()
    out = c.attn_host(inp.q.pin_memory(), inp.k_pages.cuda(), inp.v_pages.cuda(), inp.block_table.pin_memory(),
                      inp.seq_lens.pin_memory(), inp.q_lens.pin_memory(), 4)
    H.assert_close(out.double().numpy(), ref, BF)      # page-locked buffers: read and written in place over the bus
    pageable = torch.full_like(inp.q, float("nan"))
    out2 = c.attn_host(inp.q.clone(), inp.k_pages.cuda(), inp.v_pages.cuda(), inp.block_table.clone(),
                       inp.seq_lens.clone(), inp.q_lens.clone(), 4, out_host=pageable)
    H.assert_close(out2.double().numpy(), ref, BF)     # ordinary host memory: staged through device copies
    assert torch.equal(out, out2)


@pytest.mark.parametrize("pinned_out", [True, False])
@pytest.mark.parametrize("flagged", [False, True])
def test_pipelined_host_calls(flagged, pinned_out):
    """arb_attn_host_begin / arb_attn_host_wait: more calls in flight than the ring has slots, shapes that change from
    call to call (staging grows), inputs overwritten as soon as begin has returned; every result equals the one-shot
    host call bit for bit and the oracle within tolerance.  Flagged calls (operands moved in place over the bus,
    another split of the keys) are held to the oracle alone.  A page-locked result buffer is written by the kernels
    themselves, an ordinary one through a copy."""
    from paper_2512_05033_b200 import binding
    c = H.ctx()
    shapes = [([500, 90, 2000], [1, 4, 1]), ([33], [1]), ([4000, 4100, 777, 12, 640], [1, 1, 1, 1, 1]),
              ([300, 200], [16, 128])]
    cases, outs, expect = [], [], []
    for i in range(19):
        sl, ql = shapes[i % len(shapes)]
        inp = wl.small_attn_case(len(sl), 12, 2, 128, BF, sl, ql, seed=700 + i)
        kp, vp = inp.k_pages.cuda(), inp.v_pages.cuda()
        expect.append(c.attn_host(inp.q.pin_memory(), kp, vp, inp.block_table.pin_memory(), inp.seq_lens.pin_memory(),
                                  inp.q_lens.pin_memory(), max(ql)).clone())
        cases.append((inp, kp, vp, max(ql)))
    for inp, kp, vp, mq in cases:
        q, bt, sl, ql = inp.q.clone(), inp.block_table.clone(), inp.seq_lens.clone(), inp.q_lens.clone()
        out = torch.full_like(inp.q, float("nan"))
        if pinned_out:
            out = out.pin_memory()
        c.attn_host_begin(q, kp, vp, bt, sl, ql, mq, out, flags=binding.ATTN_OVERLAP_PREVIOUS if flagged else 0)
        q.fill_(float("nan")); bt.fill_(-1); sl.fill_(-1); ql.fill_(-1)   # the library has its own copy by now
        outs.append(out)
    c.attn_host_wait()
    c.attn_host_wait()                                                     # nothing in flight: returns at once
    assert c.poll_status() == 0
    if not flagged:
        for i, (out, exp) in enumerate(zip(outs, expect)):
            assert torch.equal(out, exp), i
    for i in ((0, 3, 18) if not flagged else range(19)):
        ref, _ = H.oracle_attn(cases[i][0])
        H.assert_close(outs[i].double().numpy(), ref, BF)


def test_pipelined_host_call_errors_leave_nothing_in_flight():
    """Bad arguments are refused by arb_attn_host_begin like by arb_attn; the context goes on working."""
    from paper_2512_05033_b200 import binding
    c = H.ctx()
    inp = wl.small_attn_case(2, 12, 2, 128, BF, [300, 45], [1, 1], seed=741)
    kp, vp = inp.k_pages.cuda(), inp.v_pages.cuda()
    host = [t.pin_memory() for t in (inp.q, inp.block_table, inp.seq_lens, inp.q_lens)]
    out = torch.empty_like(inp.q).pin_memory()
    p = c.params_for(host[0], kp, host[1], 1)
    args = [host[0].data_ptr(), kp.data_ptr(), vp.data_ptr(), host[1].data_ptr(), host[2].data_ptr(),
            host[3].data_ptr(), out.data_ptr(), 0]
    bad = list(args); bad[6] = None
    assert c.attn_host_begin_raw(p, *bad) == binding.ARB_ERR_INVALID_ARG          # no result buffer
    bad = list(args); bad[1] = None
    assert c.attn_host_begin_raw(p, *bad) == binding.ARB_ERR_INVALID_ARG          # no key pool
    p2 = c.params_for(host[0], kp, host[1], 1); p2.head_dim = 96
    assert c.attn_host_begin_raw(p2, *args) == binding.ARB_ERR_UNSUPPORTED
    small = binding.Context(0, workspace_bytes=1024)
    assert small.attn_host_begin_raw(p, *args) == binding.ARB_ERR_WORKSPACE
    small.attn_host_wait()
    small.close()
    for flags in (0, binding.ATTN_OVERLAP_PREVIOUS):
        p.flags = flags
        assert c.attn_host_begin_raw(p, *args) == binding.ARB_OK
        c.attn_host_wait()
        ref, _ = H.oracle_attn(inp)
        H.assert_close(out.double().numpy(), ref, BF)
        out.zero_()
    assert c.poll_status() == 0


def test_pipelined_host_calls_see_cache_updates_in_stream_order():
    """Kernels of begun calls run on the caller's stream in call order: an append enqueued between two calls is
    seen by the second and not by the first."""
    inp = wl.small_attn_case(2, 12, 2, 128, BF, [300, 45], [1, 1], seed=731).to("cuda")
    c = H.ctx()
    host = [t.cpu().pin_memory() for t in (inp.q, inp.block_table, inp.seq_lens, inp.q_lens)]
    out_a = torch.empty_like(host[0]).pin_memory()
    out_b = torch.empty_like(host[0]).pin_memory()
    g = torch.Generator().manual_seed(732)
    k_new = torch.randn(2, 2, 128, generator=g).to(BF).cuda()
    v_new = torch.randn(2, 2, 128, generator=g).to(BF).cuda()
    one = torch.ones(2, dtype=torch.int32, device="cuda")
    lens_dev = inp.seq_lens.clone()
    kp, vp = inp.k_pages.clone(), inp.v_pages.clone()
    c.attn_host_begin(*host[:1], kp, vp, *host[1:], 1, out_a)
    c.kv_append(k_new, v_new, inp.block_table, lens_dev, one, kp, vp)      # seq_lens += 1, new rows written
    longer = (inp.seq_lens + 1).cpu().pin_memory()
    c.attn_host_begin(host[0], kp, vp, host[1], longer, host[3], 1, out_b)
    c.attn_host_wait()
    before = c.attn(inp.q, inp.k_pages, inp.v_pages, inp.block_table, inp.seq_lens, inp.q_lens, 1)
    after = c.attn(inp.q, kp, vp, inp.block_table, inp.seq_lens + 1, inp.q_lens, 1)
    torch.cuda.synchronize()
    assert torch.equal(out_a, before.cpu()) and torch.equal(out_b, after.cpu())
    assert not torch.equal(out_a, out_b)


def test_pool_tensor_maps_are_cached_by_address_and_shape():
    """The tensor maps of the KV pools are kept per context.  The same device address with another pool shape must
    not get the earlier map (whose row bound would zero-fill the pages beyond it), and many pools in turn must
    each keep their own."""
    c = H.ctx()
    small = wl.small_attn_case(2, 12, 2, 128, BF, [100, 45], [1, 1], seed=801)
    large = wl.small_attn_case(2, 8, 1, 128, BF, [3000, 2100], [1, 1], seed=802)
    n_small, n_large = small.k_pages.numel(), large.k_pages.numel()
    assert n_large > 2 * n_small
    kbuf = torch.zeros(n_large, dtype=BF, device="cuda")
    vbuf = torch.zeros(n_large, dtype=BF, device="cuda")
    for inp, n in ((small, n_small), (large, n_large), (small, n_small)):
        k = kbuf[:n].view(inp.k_pages.shape); v = vbuf[:n].view(inp.v_pages.shape)
        k.copy_(inp.k_pages); v.copy_(inp.v_pages)
        d = inp.to("cuda")
        out = c.attn(d.q, k, v, d.block_table, d.seq_lens, d.q_lens, 1)
        ref, _ = H.oracle_attn(inp)
        H.assert_close(out.double().cpu().numpy(), ref, BF)
    # sixty pools of their own, visited twice
    d = small.to("cuda")
    pools = [(d.k_pages.clone(), d.v_pages.clone()) for _ in range(60)]
    first = [c.attn(d.q, k, v, d.block_table, d.seq_lens, d.q_lens, 1).clone() for k, v in pools]
    for k, v in pools[::7]:
        k.mul_(0.5)                      # same address, other contents: the map holds no data
    again = [c.attn(d.q, k, v, d.block_table, d.seq_lens, d.q_lens, 1).clone() for k, v in pools]
    torch.cuda.synchronize()
    for i, (x, y) in enumerate(zip(first, again)):
        assert torch.equal(x, y) == (i % 7 != 0), i
    assert c.poll_status() == 0


def test_repeated_calls_reuse_the_workspace():
    """Arrival counters return to zero after every call: same answer five times in a row."""
    inp = wl.small_attn_case(2, 12, 2, 128, BF, [9000, 5000], [1, 1], seed=56)
    first, _ = H.gpu_attn(inp)
    for _ in range(4):
        again, bits = H.gpu_attn(inp)
        assert bits == 0
        np.testing.assert_array_equal(first, again)


def _overlap_cases(n):
    return [wl.small_attn_case(4, 12, 2, 128, BF, [5000 + 100 * i, 700, 3000, 64], [1] * 4, seed=70 + i)
            for i in range(n)]


def test_overlap_flag_results():
    """Back-to-back calls launched as programmatic dependents (ARB_ATTN_OVERLAP_PREVIOUS): each call
    streams under the tail of the previous ones.  A flagged call may cut its sequences differently
    from an unflagged one, so it is compared with the oracle, and with itself: whatever else is in
    flight, the same call gives the same bits."""
    from paper_2512_05033_b200 import binding
    c = H.ctx()
    cpu_cases = _overlap_cases(6)
    cases = [d.to("cuda") for d in cpu_cases]
    params = [c.params_for(d.q, d.k_pages, d.block_table, 1, flags=binding.ATTN_OVERLAP_PREVIOUS) for d in cases]
    alone = []
    for d, p in zip(cases, params):     # one at a time, nothing else in flight
        alone.append(c.attn(d.q, d.k_pages, d.v_pages, d.block_table, d.seq_lens, d.q_lens, 1, params=p))
        torch.cuda.synchronize()
    outs = [torch.full_like(d.q, float("nan")) for d in cases]
    for rep in range(40):    # 240 calls in flight behind one another, workspace sets rotating
        for d, o, p in zip(cases, outs, params):
            c.attn(d.q, d.k_pages, d.v_pages, d.block_table, d.seq_lens, d.q_lens, 1, out=o, params=p)
    assert c.poll_status() == 0
    for a, b in zip(alone, outs):
        assert torch.equal(a, b)
    for d, o in zip(cpu_cases, outs):
        ref, _ = H.oracle_attn(d)
        H.assert_close(o.double().cpu().numpy(), ref, BF, tight=3e-3)


def test_overlap_flag_mixed_shapes():
    """A flagged series whose calls differ in shape and kernel: draft-like (12/2 heads) and target-like (32/8)
    tensor-core calls alternate, with a CUDA-core call (ARB_ATTN_NO_TENSOR_CORES) and an E4M3 call in every
    round.  The workspace sets of the rotation must lie at the same place whatever the call's shape, or a
    later call's early partials land on records an earlier call's combine is still reading.  Each call must
    give the bits it gives alone, and match the oracle."""
    from paper_2512_05033_b200 import binding
    c = H.ctx()
    F = binding.ATTN_OVERLAP_PREVIOUS
    geo = [(4, 12, 2, [5000, 700, 3000, 64], F), (4, 32, 8, [2100, 4000, 33, 900], F),
           (3, 28, 4, [3000, 150, 1024], F), (4, 12, 2, [1500, 2500, 17, 800], F | binding.ATTN_NO_TENSOR_CORES),
           (6, 16, 2, [6000, 100, 2000, 1, 4100, 333], F)]
    cpu_cases = [wl.small_attn_case(B, Hq, Hkv, 128, BF, sl, [1] * B, seed=170 + i)
                 for i, (B, Hq, Hkv, sl, _) in enumerate(geo)]
    cases = [d.to("cuda") for d in cpu_cases]
    params = [c.params_for(d.q, d.k_pages, d.block_table, 1, flags=g[4]) for d, g in zip(cases, geo)]
    # one E4M3 call in the series as well (same rotation, other kernel)
    e_cpu = wl.small_attn_case(4, 12, 2, 128, BF, [3100, 513, 64, 1500], [1] * 4, seed=177)
    kc = torch.from_numpy(oracle.e4m3_encode(e_cpu.k_pages, 1 / 0.012))
    vc = torch.from_numpy(oracle.e4m3_encode(e_cpu.v_pages, 1 / 0.012))
    e = e_cpu.to("cuda")
    ekc, evc = kc.cuda(), vc.cuda()

    def call(i, out=None):
        d, p = cases[i], params[i]
        return c.attn(d.q, d.k_pages, d.v_pages, d.block_table, d.seq_lens, d.q_lens, 1, out=out, params=p)

    def call_e(out=None):
        return c.attn_decode_e4m3(e.q, ekc, evc, 0.012, 0.012, e.block_table, e.seq_lens, e.q_lens, out=out, flags=F)

    alone = []
    for i in range(len(cases)):
        alone.append(call(i))
        torch.cuda.synchronize()
    alone_e = call_e()
    torch.cuda.synchronize()
    outs = [torch.full_like(d.q, float("nan")) for d in cases]
    out_e = torch.full_like(e.q, float("nan"))
    for rep in range(50):                      # 300 calls in flight behind one another
        for i in range(len(cases)):
            call(i, outs[i])
            if i == 2:
                call_e(out_e)
    assert c.poll_status() == 0
    for a, b in zip(alone, outs):
        assert torch.equal(a, b)
    assert torch.equal(alone_e, out_e)
    for d, o, g in zip(cpu_cases, outs, geo):
        ref, _ = H.oracle_attn(d)
        H.assert_close(o.double().cpu().numpy(), ref, BF, tight=1e-3 if g[4] & binding.ATTN_NO_TENSOR_CORES else 3e-3)
    ref, _ = oracle.attn_e4m3(e_cpu.q, kc, vc, 0.012, 0.012, e_cpu.block_table, e_cpu.seq_lens, e_cpu.q_lens)
    H.assert_close(out_e.double().cpu().numpy(), ref, BF, tight=3e-3)


def test_overlap_flag_in_a_replayed_graph():
    """Five flagged calls captured in one CUDA graph and replayed back to back.  The generation
    numbers of the workspace rotation are frozen into the graph and repeat with every replay, and
    five is not a multiple of the number of workspace sets: the first call of a replay lands on the
    set the last call of the previous replay is still using.  Results must not change."""
    from paper_2512_05033_b200 import binding
    c = H.ctx()
    cpu_cases = _overlap_cases(5)
    cases = [d.to("cuda") for d in cpu_cases]
    params = [c.params_for(d.q, d.k_pages, d.block_table, 1, flags=binding.ATTN_OVERLAP_PREVIOUS) for d in cases]
    outs = [torch.full_like(d.q, float("nan")) for d in cases]

    def run():
        for d, o, p in zip(cases, outs, params):
            c.attn(d.q, d.k_pages, d.v_pages, d.block_table, d.seq_lens, d.q_lens, 1, out=o, params=p)

    run()                                  # function attributes are set outside the capture
    torch.cuda.synchronize()
    expect = [o.clone() for o in outs]
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        run()
    for rep in range(30):
        for o in outs:
            o.fill_(float("nan"))
        g.replay()
        g.replay()
        g.replay()
        torch.cuda.synchronize()
        for a, b in zip(expect, outs):
            assert torch.equal(a, b), rep
    assert c.poll_status() == 0


E4M3_CASES = [
    # (B, Hq, Hkv, seq_lens)
    (3, 12, 2, [16, 17, 15]),                                  # page boundaries
    (8, 12, 2, [1025, 2000, 3001, 777, 4096, 1, 640, 5555]),   # draft-shaped, ragged
    (4, 32, 8, [4100, 9000, 33, 12000]),                       # g = 4
    (2, 28, 4, [3000, 150]),                                   # g = 7
    (1, 5, 1, [40000]),                                        # one long sequence over every CTA
    (2, 16, 2, [2100, 900]),                                   # g = 8
    (5, 8, 2, [100, 1, 300, 1, 47]),                           # with idle slots (below)
    # block tables wide enough for the launcher to treat the call as a large one (five consumer warps per CTA)
    (8, 12, 2, [12000, 9000, 700, 33, 5000, 11000, 1, 2500]),  # g = 6
    (4, 16, 2, [20000, 15000, 100, 9000]),                     # g = 8
]


@pytest.mark.parametrize("case", E4M3_CASES)
def test_e4m3_decode_matches_oracle(case):
    B, Hq, Hkv, sl = case
    ql = [1, 0, 1, 0, 1] if B == 5 else [1] * B
    inp = wl.small_attn_case(B, Hq, Hkv, 128, BF, sl, ql, seed=700 + Hq)
    ks, vs = 0.011, 0.017          # N(0,1) values / scale reach about 400: the whole range of the format is used
    kc = torch.from_numpy(oracle.e4m3_encode(inp.k_pages, 1 / ks))
    vc = torch.from_numpy(oracle.e4m3_encode(inp.v_pages, 1 / vs))
    # stale slots past the ends hold NaN codes: they must never reach the arithmetic
    for b in range(B):
        L = sl[b]
        if L % 16:
            page = int(inp.block_table[b, L // 16])
            kc[page, :, L % 16:, :] = 0x7f
            vc[page, :, L % 16:, :] = 0x7f
    c = H.ctx()
    d = inp.to("cuda")
    out = torch.full_like(d.q, float("nan"))
    c.attn_decode_e4m3(d.q, kc.cuda(), vc.cuda(), ks, vs, d.block_table, d.seq_lens, d.q_lens, out=out)
    assert c.poll_status() == 0
    ref, st = oracle.attn_e4m3(inp.q, kc, vc, ks, vs, inp.block_table, inp.seq_lens, inp.q_lens)
    assert st == 0
    H.assert_close(out.double().cpu().numpy(), ref, BF, tight=3e-3)


def test_e4m3_decode_peaked_and_back_to_back():
    """q scaled up so that few keys carry the weight, and flagged calls in flight behind one another."""
    from paper_2512_05033_b200 import binding
    inp = wl.small_attn_case(4, 12, 2, 128, BF, [3000, 513, 64, 1500], [1] * 4, seed=7, q_std=6.0)
    ks, vs = 0.012, 0.012
    kc = torch.from_numpy(oracle.e4m3_encode(inp.k_pages, 1 / ks))
    vc = torch.from_numpy(oracle.e4m3_encode(inp.v_pages, 1 / vs))
    ref, _ = oracle.attn_e4m3(inp.q, kc, vc, ks, vs, inp.block_table, inp.seq_lens, inp.q_lens)
    c = H.ctx()
    d = inp.to("cuda")
    dk, dv = kc.cuda(), vc.cuda()
    alone = c.attn_decode_e4m3(d.q, dk, dv, ks, vs, d.block_table, d.seq_lens, d.q_lens, flags=binding.ATTN_OVERLAP_PREVIOUS)
    torch.cuda.synchronize()
    outs = [torch.full_like(d.q, float("nan")) for _ in range(6)]
    for rep in range(20):
        for o in outs:
            c.attn_decode_e4m3(d.q, dk, dv, ks, vs, d.block_table, d.seq_lens, d.q_lens, out=o,
                               flags=binding.ATTN_OVERLAP_PREVIOUS)
    assert c.poll_status() == 0
    for o in outs:
        assert torch.equal(o, alone)
    err = np.abs(alone.double().cpu().numpy() - ref)
    assert (err <= 2.0 ** -8 * np.abs(ref) + 3e-3).all(), err.max()


E4M3_CHUNK_CASES = [
    # (B, Hq, Hkv, seq_lens, q_lens)
    (1, 32, 8, [300], [64]),                                   # g = 4: two full row tiles
    (2, 28, 4, [600, 2100], [16, 100]),                        # g = 7: a ragged tile and 700 rows
    (2, 12, 2, [131, 128], [128, 11]),                         # the chunk is almost the whole sequence
    (4, 32, 8, [5000, 77, 1300, 256], [1, 30, 128, 5]),        # decode rows beside large and small chunks
    (1, 16, 2, [4099], [19]),                                  # g = 8, key count not a page multiple
    (3, 12, 2, [2, 17, 300], [2, 3, 2]),                       # smallest chunks; the chunk is the whole sequence
    (2, 8, 8, [40, 300], [2, 9]),                              # g = 1
    (3, 12, 2, [5000, 2500, 300], [24, 9, 1]),                 # few work items: cut over the keys to fill the SMs
    (3, 28, 4, [21000, 900, 40000], [40, 64, 17]),             # long sequences split into parts and merged
    (5, 12, 2, [100, 1, 300, 1, 47], [3, 0, 1, 0, 20]),        # idle slots
]


@pytest.mark.parametrize("case", E4M3_CHUNK_CASES)
def test_e4m3_chunk_matches_oracle(case):
    """arb_attn_e4m3: step chunks (and the decode rows beside them) over an E4M3 cache against the oracle on the
    same codes; slots past each sequence's end hold NaN codes, which must never reach the arithmetic."""
    B, Hq, Hkv, sl, ql = case
    inp = wl.small_attn_case(B, Hq, Hkv, 128, BF, sl, ql, seed=900 + Hq + len(sl))
    ks, vs = 0.011, 0.017
    kc = torch.from_numpy(oracle.e4m3_encode(inp.k_pages, 1 / ks))
    vc = torch.from_numpy(oracle.e4m3_encode(inp.v_pages, 1 / vs))
    for b in range(B):
        L = sl[b]
        if L % 16:
            page = int(inp.block_table[b, L // 16])
            kc[page, :, L % 16:, :] = 0x7f
            vc[page, :, L % 16:, :] = 0x7f
    c = H.ctx()
    d = inp.to("cuda")
    out = torch.full_like(d.q, float("nan"))
    c.attn_e4m3(d.q, kc.cuda(), vc.cuda(), ks, vs, d.block_table, d.seq_lens, d.q_lens, max(ql), out=out)
    assert c.poll_status() == 0
    ref, st = oracle.attn_e4m3(inp.q, kc, vc, ks, vs, inp.block_table, inp.seq_lens, inp.q_lens)
    assert st == 0
    H.assert_close(out.double().cpu().numpy(), ref, BF, tight=3e-3)


def test_e4m3_chunk_peaked_and_bad_lengths():
    """Few keys carry the weight (outputs of order one), and a sequence whose lengths make no sense is zero-filled
    with the status bit while the others are served."""
    from paper_2512_05033_b200 import binding
    inp = wl.small_attn_case(3, 12, 2, 128, BF, [3000, 513, 700], [40, 7, 12], seed=907, q_std=6.0)
    ks, vs = 0.012, 0.012
    kc = torch.from_numpy(oracle.e4m3_encode(inp.k_pages, 1 / ks))
    vc = torch.from_numpy(oracle.e4m3_encode(inp.v_pages, 1 / vs))
    ref, _ = oracle.attn_e4m3(inp.q, kc, vc, ks, vs, inp.block_table, inp.seq_lens, inp.q_lens)
    c = H.ctx()
    d = inp.to("cuda")
    out = c.attn_e4m3(d.q, kc.cuda(), vc.cuda(), ks, vs, d.block_table, d.seq_lens, d.q_lens, 40)
    assert c.poll_status() == 0
    err = np.abs(out.double().cpu().numpy() - ref)
    assert (err <= 2.0 ** -8 * np.abs(ref) + 3e-3).all(), err.max()
    bad = d.seq_lens.clone()
    bad[1] = 3                                   # fewer keys than query tokens
    out2 = torch.full_like(d.q, float("nan"))
    c.attn_e4m3(d.q, kc.cuda(), vc.cuda(), ks, vs, d.block_table, bad, d.q_lens, 40, out=out2)
    assert c.poll_status() == binding.DEV_BAD_SEQ_LEN
    assert float(out2[40:47].abs().max()) == 0.0
    assert torch.equal(out2[:40], out[:40]) and torch.equal(out2[47:], out[47:])
