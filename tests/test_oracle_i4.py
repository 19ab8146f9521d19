"""Pins of the oracle's 4-bit KV functions: a row worked by hand (tests/golden/i4_format.txt), the error bound of the
format, the special rows, and attention / append over codes against the plain functions on data the format holds exactly."""
from pathlib import Path

import numpy as np
import torch

from oracle import oracle
from paper_2512_05033_b200 import workloads as wl

GOLD = Path(__file__).parent / "golden" / "i4_format.txt"


def _gold():
    rows = {}
    for line in GOLD.read_text().splitlines():
        if line and not line.startswith("#"):
            key, *vals = line.split()
            rows[key] = np.array([float(v) for v in vals])
    return rows


def test_worked_row_bytes_scale_and_values():
    g = _gold()
    codes, scale = oracle.i4_encode(g["values"].astype(np.float32)[None, :])
    assert scale.tolist() == [g["scale"][0]]
    assert codes[0].tolist() == [int(b) for b in g["bytes"]]
    assert oracle.i4_decode(codes, scale)[0].tolist() == g["decoded"].tolist()


def test_error_bound_range_and_extremes():
    rng = np.random.default_rng(5)
    x = (rng.standard_normal((200, 128)) * rng.uniform(1e-3, 50.0, (200, 1))).astype(np.float32)
    codes, scale = oracle.i4_encode(x)
    assert codes.shape == (200, 64) and scale.shape == (200,)
    lo, hi = codes & 0xf, codes >> 4
    assert lo.min() >= 1 and hi.min() >= 1          # nibble 0 (code -8) never occurs
    back = oracle.i4_decode(codes, scale)
    m = np.abs(x).max(axis=1)
    np.testing.assert_allclose(scale, m / np.float32(7), rtol=1e-7)
    assert (np.abs(back - x) <= 0.5 * scale[:, None] * (1 + 1e-5) + 1e-12).all()   # half a step
    arg = np.abs(x).argmax(axis=1)
    assert np.allclose(np.abs(back[np.arange(200), arg]), 7.0 * scale.astype(np.float64))   # the largest value is +-7 steps


def test_zero_row_and_exact_rows():
    z = np.zeros((2, 16), dtype=np.float32)
    codes, scale = oracle.i4_encode(z)
    assert (codes == 0x88).all() and (scale == 0).all() and (oracle.i4_decode(codes, scale) == 0).all()
    rng = np.random.default_rng(6)
    x = rng.integers(-7, 8, (50, 128)).astype(np.float32)
    x[:, 0] = 7.0                                   # max 7: scale 1, every value its own code
    x *= np.float32(0.25)                           # and a power-of-two scale keeps it exact
    codes, scale = oracle.i4_encode(x)
    assert (scale == np.float32(0.25)).all()
    assert (oracle.i4_decode(codes, scale) == x.astype(np.float64)).all()


def _exact_case(seed):
    """An attention case whose pools the format holds exactly (integers in -7..7 times 1/4, every row reaching 7)."""
    inp = wl.small_attn_case(3, 12, 2, 128, torch.bfloat16, [70, 33, 200], [1, 1, 1], seed=seed, extra_tokens=4)
    g = torch.Generator().manual_seed(seed)
    for pool in (inp.k_pages, inp.v_pages):
        vals = torch.randint(-7, 8, pool.shape, generator=g).float()
        vals[..., 0] = 7.0
        pool.copy_((vals * 0.25).to(pool.dtype))
    return inp


def test_attention_over_codes_equals_attention_over_the_values_they_hold():
    inp = _exact_case(11)
    kc, ks = oracle.i4_encode(inp.k_pages)
    vc, vs = oracle.i4_encode(inp.v_pages)
    got, st = oracle.attn_i4(inp.q, kc, vc, ks, vs, inp.block_table, inp.seq_lens, inp.q_lens)
    ref, st2 = oracle.attn(inp.q, inp.k_pages, inp.v_pages, inp.block_table, inp.seq_lens, inp.q_lens)
    assert st == 0 and st2 == 0
    np.testing.assert_allclose(got, ref, rtol=0, atol=1e-12)


def test_quantising_append_places_rows_like_the_plain_append():
    inp = _exact_case(12)
    kc, ks = oracle.i4_encode(inp.k_pages)
    vc, vs = oracle.i4_encode(inp.v_pages)
    new = torch.tensor([1, 0, 3], dtype=torch.int32)
    g = torch.Generator().manual_seed(3)
    kn = (torch.randint(-7, 8, (4, 2, 128), generator=g).float())
    vn = (torch.randint(-7, 8, (4, 2, 128), generator=g).float())
    kn[..., 5] = -7.0
    vn[..., 9] = 7.0
    kn, vn = (kn * 0.5).bfloat16(), (vn * 0.5).bfloat16()
    okc, ovc, oks, ovs, sl, st = oracle.kv_append_i4(kn, vn, inp.block_table, inp.seq_lens, new, torch.from_numpy(kc),
                                                      torch.from_numpy(vc), torch.from_numpy(ks), torch.from_numpy(vs))
    k_ref, v_ref, sl_ref, st_ref = oracle.kv_append(kn, vn, inp.block_table, inp.seq_lens, new, inp.k_pages, inp.v_pages)
    assert st == 0 and st_ref == 0 and (sl == sl_ref).all()
    # compare what the sequences hold (slots past the lengths are free to differ)
    dk, dv = oracle.i4_decode(okc, oks), oracle.i4_decode(ovc, ovs)
    for b in range(3):
        for pos in range(int(sl[b])):
            page, slot = int(inp.block_table[b, pos // 16]), pos % 16
            assert (dk[page, :, slot] == k_ref[page, :, slot].double().numpy()).all()
            assert (dv[page, :, slot] == v_ref[page, :, slot].double().numpy()).all()
