"""delta-guided bit switching (Sec. 3.3): oracle pins, the host-side rule of the library against
the oracle (no GPU needed), and the L1 kernel against the oracle (GPU)."""
import math
import os

import numpy as np
import pytest
import torch

from oracle import dvdq_oracle as orc
from paper_2505_18663_b200 import binding as B

from helpers import to_bits

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "gbs_worked_example.txt")


def read_golden():
    out = {}
    for line in open(GOLDEN):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        key, *vals = line.split()
        out[key] = [float(v) for v in vals]
    return out


def library_schedule(l1_values, delta, b_low, b_high):
    g = B.dvdq_gbs_init(delta, b_low, b_high)
    bits = []
    for i in range(len(l1_values) + 1):
        bits.append(B.dvdq_gbs_next_bits(g))
        if i < len(l1_values):
            B.dvdq_gbs_observe(g, l1_values[i], 1.0)
    assert g.steps == len(bits) and g.high_steps == sum(b == b_high for b in bits) or b_low == b_high
    return bits


# ------------------------------------------------------------------ oracle pins

def test_oracle_schedule_matches_hand_worked_example():
    g = read_golden()
    bits = orc.gbs_schedule(g["l1"], g["delta"][0], int(g["b_low"][0]), int(g["b_high"][0]))
    assert bits == [int(b) for b in g["bits"]]


def test_oracle_l1_terms_match_hand_worked_example():
    g = read_golden()
    ft = torch.tensor(g["f_t"]).to(torch.bfloat16)
    fp = torch.tensor(g["f_prev"]).to(torch.bfloat16)
    num, den = orc.gbs_l1_terms(to_bits(ft), to_bits(fp))
    assert num == g["num"][0] and den == g["den"][0]


def test_oracle_schedule_limits():
    l1 = [0.3, 0.01, 0.7, 0.0, 0.2]
    assert orc.gbs_schedule(l1, 0.0, 4, 8) == [8] * 6           # delta -> 0: every step at b_high
    assert orc.gbs_schedule(l1, math.inf, 4, 8) == [4] * 6      # delta -> inf: every step at b_low
    # constant change c with delta = 2.5 c: the sum reaches delta after three observed steps
    assert orc.gbs_schedule([1.0] * 9, 2.5, 4, 8) == [4, 4, 4, 8, 4, 4, 8, 4, 4, 8]


def test_oracle_l1_properties():
    rng = np.random.default_rng(0)
    f = torch.from_numpy(rng.standard_normal(4099).astype(np.float32)).to(torch.bfloat16)
    num, den = orc.gbs_l1_terms(to_bits(f), to_bits(f))
    assert num == 0.0 and den == float(f.double().abs().sum())
    # F_t = 1.5 F_{t-1} is exact in bf16 for values with a short significand: relative change 0.5
    base = torch.tensor([1.0, -2.0, 0.5, 8.0, -0.25]).to(torch.bfloat16)
    num, den = orc.gbs_l1_terms(to_bits((base.float() * 1.5).to(torch.bfloat16)), to_bits(base))
    assert num / den == 0.5
    # torch's own norm agrees (a library routine, not this module's arithmetic)
    g = torch.from_numpy(rng.standard_normal(4099).astype(np.float32)).to(torch.bfloat16)
    num, den = orc.gbs_l1_terms(to_bits(g), to_bits(f))
    assert math.isclose(num, float(torch.linalg.vector_norm(g.double() - f.double(), ord=1)), rel_tol=1e-13)


# ------------------------------------------------------------------ host rule of the library (no GPU)

def test_library_rule_matches_oracle():
    g = read_golden()
    assert library_schedule(g["l1"], g["delta"][0], 4, 8) == [int(b) for b in g["bits"]]
    rng = np.random.default_rng(1)
    for delta in (0.0, 0.05, 0.2, 1.0, 50.0):
        l1 = rng.random(60) * 0.1
        for lo, hi in ((4, 8), (4, 6), (6, 8), (8, 8)):
            assert library_schedule(list(l1), delta, lo, hi) == orc.gbs_schedule(l1, delta, lo, hi)


def test_library_rule_rejects_bad_arguments():
    import ctypes as C
    lib = B.load()
    g = B.GbsState()
    assert lib.dvdq_gbs_init(None, 0.1, 4, 8) == B.ERR_NULL
    assert lib.dvdq_gbs_init(C.byref(g), -1.0, 4, 8) == B.ERR_SHAPE
    assert lib.dvdq_gbs_init(C.byref(g), float("nan"), 4, 8) == B.ERR_SHAPE
    assert lib.dvdq_gbs_init(C.byref(g), 0.1, 5, 8) == B.ERR_BITS
    assert lib.dvdq_gbs_init(C.byref(g), 0.1, 8, 4) == B.ERR_BITS
    assert lib.dvdq_gbs_next_bits(None) == 0
    assert lib.dvdq_gbs_observe(C.byref(g), -1.0, 1.0) == B.ERR_SHAPE
    assert lib.dvdq_gbs_l1_terms(None, None, -1, None, None) == B.ERR_SHAPE
    assert lib.dvdq_gbs_l1_terms(None, None, 8, None, None) == B.ERR_NULL


# ------------------------------------------------------------------ the L1 kernel (GPU)

@pytest.mark.gpu
@pytest.mark.parametrize("n", [0, 1, 7, 8, 4099, 1 << 20, (1 << 22) + 13])
def test_l1_terms_kernel_matches_oracle(n):
    g = torch.Generator().manual_seed(n)
    fp = (torch.randn(max(n, 1), generator=g) * 3.0).to(torch.bfloat16)[:n]
    ft = (fp.float() + 0.05 * torch.randn(max(n, 1), generator=g)[:n]).to(torch.bfloat16)
    terms = torch.full((2,), 123.0, dtype=torch.float64, device="cuda")
    B.dvdq_gbs_l1_terms(ft.cuda().contiguous(), fp.cuda().contiguous(), terms)
    num, den = terms.cpu().tolist()
    num_or, den_or = orc.gbs_l1_terms(to_bits(ft), to_bits(fp)) if n else (0.0, 0.0)
    # fp32 inside a 16-byte chunk (8 terms), fp64 across chunks: 8 * 2^-24 relative per chunk
    assert abs(num - num_or) <= 1e-6 * max(num_or, 1e-30) and abs(den - den_or) <= 1e-6 * max(den_or, 1e-30)


@pytest.mark.gpu
def test_bit_schedule_from_device_terms_matches_oracle():
    """A short synthetic denoising run: outputs drift slowly, then jump, then settle."""
    gen = torch.Generator().manual_seed(5)
    n = 200_003
    f = torch.randn(n, generator=gen).to(torch.bfloat16)
    steps = [0.01, 0.01, 0.02, 0.4, 0.01, 0.01, 0.3, 0.005, 0.005, 0.005]
    outs = [f]
    for s in steps:
        outs.append((outs[-1].float() + s * torch.randn(n, generator=gen)).to(torch.bfloat16))
    l1_or = []
    for t in range(1, len(outs)):
        num, den = orc.gbs_l1_terms(to_bits(outs[t]), to_bits(outs[t - 1]))
        l1_or.append(num / den)
    want = orc.gbs_schedule(l1_or, 0.25, 4, 8)
    assert 8 in want and 4 in want
    g = B.dvdq_gbs_init(0.25, 4, 8)
    terms = torch.zeros(2, dtype=torch.float64, device="cuda")
    dev = [o.cuda() for o in outs]
    got = [B.dvdq_gbs_next_bits(g)]
    for t in range(1, len(outs)):
        B.dvdq_gbs_l1_terms(dev[t], dev[t - 1], terms)
        num, den = terms.cpu().tolist()
        B.dvdq_gbs_observe(g, num, den)
        got.append(B.dvdq_gbs_next_bits(g))
    assert got == want
