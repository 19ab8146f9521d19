"""The pins do bite: each plausible mistake, planted in a copy of the oracle's C source and compiled on
the CPU, is caught by at least one of the pin checks below (the same kinds of checks as in
test_oracle_attn.py / test_oracle_route.py / test_oracle_policy.py, run against the mutated build)."""
import ctypes
import math
import subprocess
from pathlib import Path

import numpy as np
import pytest
import torch

from oracle import oracle
from paper_2512_05033_b200 import workloads as wl
from tests.test_oracle_attn import brute_force

SRC = (Path(oracle.__file__).parent / "arb_oracle.c").read_text()

MUTATIONS = {
    "scale dropped": ("s[j] = scale * acc;", "s[j] = acc;"),
    "causal bound one short": ("long nkeys = pos + 1;", "long nkeys = pos > 0 ? pos : 1;"),
    "kv head by modulo": ("int kvh = h / g;", "int kvh = h % Hkv;"),
    "slot off by one": ("size_t koff = kv_offset(page, kvh, (int)(j % P), Hkv, P, D);",
                        "size_t koff = kv_offset(page, kvh, (int)((j + 1) % P), Hkv, P, D);"),
    "V read from the K offset of the next dim": ("out_row[d] += p * widen(v_pages, dtype, voff + d);",
                                                 "out_row[d] += p * widen(v_pages, dtype, voff + (d + 1) % D);"),
    "no max subtraction and no normalisation": ("double p = s[j] / Z;", "double p = s[j];"),
    "bf16 widened with the wrong shift": ("<< 16;", "<< 15;"),
    "sigmoid sign": ("1.0 / (1.0 + exp(-z))", "1.0 / (1.0 + exp(z))"),
    "bias dropped": ("double z = b;", "double z = 0.0;"),
    "tie escalates": ("((float)sc > tau)", "((float)sc >= tau)"),
    "rollback adds": ("long r = (long)seq_lens[i] - (long)step_lens[i];", "long r = (long)seq_lens[i] + (long)step_lens[i];"),
    "rollback ignores decisions": ("if (decisions && !decisions[i]) continue;", ""),
    "RSD polarity": ("if (kind == 0) a = !(s_d[i] > tau);", "if (kind == 0) a = (s_d[i] > tau);"),
    "oracle threshold on the draft score": ("float delta = s_t[i] - s_d[i]; a = delta > tau;", "float delta = s_t[i]; a = delta > tau;"),
    "budget spent on negative advantages": ("if (!(adv[r].delta > 0.0f)) break;", ""),
    "wasted counts improvements": ("if (!(st > sd)) wasted += 1;", "if (st > sd) wasted += 1;"),
    "class level not normalised": ("sc += p[c] * (double)c / (double)(C - 1);", "sc += p[c] * (double)c;"),
    "ordinal cut sign": ("ge[k] = 1.0 / (1.0 + exp(-(acc - b[k])));", "ge[k] = 1.0 / (1.0 + exp(-(acc + b[k])));"),
    "append one slot late": ("const int pos = L + j;", "const int pos = L + j + 1;"),
    "ties take the lowest rank": ("rx[i] = (double)lx + ((double)ex + 1.0) / 2.0;", "rx[i] = (double)lx + 1.0;"),
    "ranks not centred": ("const double m = ((double)n + 1.0) / 2.0;", "const double m = 0.0;"),
    "E4M3 bias off by one": ("ldexp(1.0, e - 7);", "ldexp(1.0, e - 8);"),
    "E4M3 ties away from even": ("(err == best_err && (c & 1) == 0)", "(err == best_err && (c & 1) == 1)"),
    "append swaps K and V": ("memcpy((char *)k_pages + dst, (const char *)k_new + src, tok_bytes);",
                             "memcpy((char *)k_pages + dst, (const char *)v_new + src, tok_bytes);"),
}


def _variant(tmp_path, name, old, new):
    assert SRC.count(old) >= 1, name
    c = tmp_path / "mut.c"
    so = tmp_path / f"mut_{abs(hash(name))}.so"
    c.write_text(SRC.replace(old, new))
    subprocess.check_call(["gcc", "-O1", "-fopenmp", "-fPIC", "-shared", "-std=c11", "-o", str(so), str(c), "-lm"])
    return oracle.bind(ctypes.CDLL(str(so)))


def _pins_pass() -> bool:
    """A compact set of pins; returns False as soon as one fails."""
    try:
        for case in [(2, 6, 2, 64, torch.float32, [17, 64], [5, 16]), (3, 12, 2, 128, torch.bfloat16, [33, 1, 50], [1, 1, 7])]:
            B, Hq, Hkv, D, dt, sl, ql = case
            inp = wl.small_attn_case(B, Hq, Hkv, D, dt, sl, ql, seed=11)
            out, st = oracle.attn(inp.q, inp.k_pages, inp.v_pages, inp.block_table, inp.seq_lens, inp.q_lens)
            if st or not np.allclose(out, brute_force(inp), rtol=0, atol=1e-12):
                return False
        hidden = np.zeros((3, 8), dtype=np.float32)
        w = np.ones(8, dtype=np.float32)
        hidden[1, 0] = math.log(3.0) - 0.25
        hidden[2, 0] = -0.25
        s, d = oracle.route(hidden, w, 0.25, 0.5)          # z = 0.25, ln 3, 0
        if not (abs(s[1] - 0.75) < 1e-7 and s[2] == 0.5 and list(d) == [1, 1, 0]):
            return False
        new, _ = oracle.rollback(np.array([100, 50]), np.array([10, 20]), np.array([1, 0], dtype=np.uint8))
        if list(new) != [90, 50]:
            return False
        # policies on exact scores: (s_d, s_t) = (1/4, 7/8), (5/8, 1/8), (1/2, 3/4)
        sd, st = [0.25, 0.625, 0.5], [0.875, 0.125, 0.75]
        d, s = oracle.policy(oracle.POLICY_RSD, sd, st, tau=0.5)
        if list(d) != [1, 0, 1] or s["wasted"] != 0:
            return False
        d, s = oracle.policy(oracle.POLICY_RSD, sd, st, tau=0.75)
        if list(d) != [1, 1, 1] or s["wasted"] != 1:
            return False
        d, _ = oracle.policy(oracle.POLICY_ORACLE_THRESHOLD, sd, st, tau=0.5)
        if list(d) != [1, 0, 0]:
            return False
        d, s = oracle.policy(oracle.POLICY_ORACLE_BUDGET, sd, st, budget=3)
        if list(d) != [1, 0, 1] or abs(s["gain"] - 0.875) > 1e-12:
            return False
        hid = np.zeros((1, 8), dtype=np.float32)
        hid[0, 0] = 1.0
        wc = np.zeros((4, 8), dtype=np.float32)
        wc[2, 0] = 60.0
        _, sc, _ = oracle.route_classes(oracle.HEAD_SOFTMAX, hid, wc, [0.0] * 4, 0.5)
        if abs(sc[0] - 2 / 3) > 1e-12:
            return False
        wo = np.zeros((1, 8), dtype=np.float32)
        p, _, _ = oracle.route_classes(oracle.HEAD_ORDINAL, hid, wo, [0.0, -math.log(3.0), 0.0, math.log(3.0)], 0.5)
        if not np.allclose(p[0], 0.25, atol=1e-12):
            return False
        p, _, _ = oracle.route_classes(oracle.HEAD_ORDINAL, hid, wo, [0.0, math.log(3.0), math.log(9.0)], 0.5)
        if not np.allclose(p[0], [0.75, 0.15, 0.1], atol=1e-12):
            return False
        if abs(oracle.spearman([1, 2, 2, 3], [1, 2, 3, 4]) - 3 / math.sqrt(10)) > 1e-12:
            return False
        if abs(oracle.spearman([1, 2, 3, 4, 5], [2, 1, 4, 3, 5]) - 0.8) > 1e-12:   # 1 - 6 * 4 / 120
            return False
        if list(oracle.e4m3_decode(np.uint8([0x38, 0x7e, 0x01]))) != [1.0, 448.0, 2.0 ** -9]:
            return False
        if list(oracle.e4m3_encode(np.float32([1.0625, 1.1875, 500.0]))) != [0x38, 0x3a, 0x7e]:
            return False
        inp = wl.small_attn_case(1, 2, 1, 64, torch.float32, [20], [1], seed=4, extra_tokens=16)
        kn = torch.full((3, 1, 64), 7.0)
        vn = torch.full((3, 1, 64), -7.0)
        kp, vp, sl, st_ = oracle.kv_append(kn, vn, inp.block_table, inp.seq_lens, torch.tensor([3], dtype=torch.int32),
                                           inp.k_pages, inp.v_pages)
        page = int(inp.block_table[0, 1])
        ok = (st_ == 0 and list(sl) == [23] and bool((kp[page, 0, 4:7] == 7.0).all()) and bool((vp[page, 0, 4:7] == -7.0).all())
              and torch.equal(kp[page, 0, 7:], inp.k_pages[page, 0, 7:]) and torch.equal(kp[page, 0, :4], inp.k_pages[page, 0, :4]))
        return ok
    except Exception:
        return False


def test_the_unmutated_oracle_passes_the_compact_pins():
    assert _pins_pass()


@pytest.mark.parametrize("name", sorted(MUTATIONS))
def test_mutation_is_caught(name, tmp_path, monkeypatch):
    old, new = MUTATIONS[name]
    oracle._load()
    monkeypatch.setattr(oracle, "_lib", _variant(tmp_path, name, old, new))
    assert not _pins_pass(), f"no pin noticed: {name}"
