"""Pins of the CPU oracle against what the paper and the mathematics fix.

None of these tests re-types the oracle's own formula: each compares it with a value
worked by hand (tests/golden), a closed form, an invariant, a library routine
(scipy's Hadamard matrix, numpy's integer matmul, torch's bf16 cast and GELU) or a
brute-force loop.  They run without a GPU.
"""
import math
import os

import numpy as np
import pytest
import scipy.linalg
import torch

from oracle import dvdq_oracle as orc

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def to_bits(t: torch.Tensor) -> np.ndarray:
    return t.to(torch.bfloat16).contiguous().view(torch.int16).numpy().view(np.uint16)


def bits_of(values) -> np.ndarray:
    return to_bits(torch.tensor(values, dtype=torch.float32))


def bf16_values(bits: np.ndarray) -> np.ndarray:
    return torch.from_numpy(bits.view(np.int16).copy()).view(torch.bfloat16).to(torch.float64).numpy()


def read_golden(name):
    rows = {}
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            parts = line.split()
            rows.setdefault(parts[0], []).append(parts[1:])
    return rows


# ------------------------------------------------------------------ rotation (Sec. 3.2)

@pytest.mark.parametrize("B", [1, 2, 4, 64, 256, 1024])
def test_hadamard_is_orthonormal_symmetric_and_matches_scipy(B):
    H = orc.hadamard(B)
    assert np.abs(H @ H.T - np.eye(B)).max() < 1e-12          # Q Q^T = I
    assert np.array_equal(H, H.T)                              # Sylvester H is symmetric
    assert np.abs(H @ H - np.eye(B)).max() < 1e-12             # hence an involution
    ref = scipy.linalg.hadamard(B).astype(np.float64) / math.sqrt(B)
    assert np.array_equal(H, ref)
    e0 = np.zeros(B); e0[0] = 1.0
    assert np.allclose(e0 @ H, np.full(B, 1 / math.sqrt(B)), atol=1e-15)
    assert np.allclose(np.ones(B) @ H, math.sqrt(B) * e0, atol=1e-12)
    assert abs(abs(np.linalg.det(H)) - 1.0) < 1e-9 if B <= 64 else True


@pytest.mark.parametrize("K,B", [(256, 256), (1536, 512), (384, 64), (1024, 1024), (512, 128)])
def test_rotate_equals_library_block_diagonal_product(K, B):
    g = torch.Generator().manual_seed(10 + K + B)
    x = torch.randn(7, K, generator=g)
    xb = to_bits(x)
    xt = orc.rotate(xb, B)
    Hs = scipy.linalg.hadamard(B).astype(np.float64) / math.sqrt(B)
    R = np.kron(np.eye(K // B), Hs)                           # I (x) H_B
    ref = bf16_values(xb) @ R
    assert np.abs(xt - ref).max() <= 1e-12 * max(1.0, np.abs(ref).max())
    # Parseval: an orthogonal rotation keeps every token's 2-norm.
    assert np.allclose(np.linalg.norm(xt, axis=1), np.linalg.norm(bf16_values(xb), axis=1), rtol=1e-12)


def test_rotate_block_zero_is_identity_and_bad_block_rejected():
    xb = bits_of([[1.0, -2.0, 3.5, 0.0]])
    assert np.array_equal(orc.rotate(xb, 0), [[1.0, -2.0, 3.5, 0.0]])
    with pytest.raises(ValueError):
        orc.rotate(xb, 3)
    with pytest.raises(ValueError):
        orc.rotate(bits_of([[1.0] * 6]), 4)


def test_rotation_respects_leading_block_structure():
    # A token that is non-zero only in block 1 must stay zero in every other block.
    K, B = 256, 64
    x = torch.zeros(1, K)
    x[0, 64:128] = torch.arange(64, dtype=torch.float32) - 31
    xt = orc.rotate(to_bits(x), B)
    assert np.all(xt[0, :64] == 0) and np.all(xt[0, 128:] == 0) and np.any(xt[0, 64:128] != 0)


def test_computational_invariance_of_the_rotation():
    # Y = X W^T = (X H)(W H)^T  (Sec. 3.2), fp64, relative 1e-10.
    g = torch.Generator().manual_seed(3)
    M, N, K, B = 9, 5, 512, 128
    xb = to_bits(torch.randn(M, K, generator=g))
    wb = to_bits(torch.randn(N, K, generator=g) * 0.02)
    y_plain = bf16_values(xb) @ bf16_values(wb).T
    y_rot = orc.exact_linear(orc.rotate(xb, B), orc.rotate(wb, B))
    assert np.abs(y_rot - y_plain).max() <= 1e-10 * np.abs(y_plain).max()
    # exact_linear itself against numpy on a non-square, non-symmetric case
    a = np.arange(12, dtype=np.float64).reshape(3, 4)
    b = np.arange(20, dtype=np.float64).reshape(5, 4) - 7
    assert np.array_equal(orc.exact_linear(a, b), a @ b.T)


# ------------------------------------------------------------------ activation quantizer (Eq. 10)

def test_worked_example_rotate_scale_quantize():
    rows = read_golden("arq_worked_example.txt")
    for case in "ABCD":
        d = {r[0]: [float(v) for v in r[1:]] for r in rows[case]}
        xb = bits_of([d["x"]])
        assert np.array_equal(bf16_values(xb)[0], d["x"]), "fixture inputs must be exact in bf16"
        codes, s64, s32, xt = orc.rotate_quantize(xb, 4, 4)
        assert np.array_equal(xt[0], d["xt"])
        assert s64[0] == d["s_num"][0] / d["s_den"][0]
        assert s32[0] == np.float32(d["s_num"][0] / d["s_den"][0])
        assert np.array_equal(codes[0], np.array(d["codes"], dtype=np.int32))


@pytest.mark.parametrize("bits", [4, 6])
@pytest.mark.parametrize("K,B", [(256, 256), (1536, 512)])
def test_quantizer_invariants(bits, K, B):
    g = torch.Generator().manual_seed(100 + bits + K)
    x = torch.randn(33, K, generator=g)
    x[:, 5] *= 20.0
    x[7] = 0.0                                                  # an all-zero token
    xb = to_bits(x)
    codes, s64, s32, xt = orc.rotate_quantize(xb, B, bits)
    qmax = 2 ** (bits - 1) - 1
    assert codes.min() >= -qmax and codes.max() <= qmax        # ranges [-8,7] / [-32,31], -2^(b-1) unused
    assert np.array_equal(s64 * qmax, np.abs(xt).max(axis=1)) or np.allclose(s64 * qmax, np.abs(xt).max(axis=1), rtol=1e-15)
    err = np.abs(xt - s64[:, None] * codes)
    assert np.all(err <= s64[:, None] / 2 * (1 + 1e-12))        # error <= scale / 2 per element
    nz = s64 > 0
    assert np.all(np.abs(codes[nz]).max(axis=1) == qmax)        # the absmax element sits on +-qmax
    assert s64[7] == 0 and s32[7] == 0 and np.all(codes[7] == 0)
    assert np.array_equal(s32, s64.astype(np.float32))


def test_scale_equivariance_under_powers_of_two():
    g = torch.Generator().manual_seed(5)
    x = torch.randn(8, 256, generator=g)
    c1, s1, _, _ = orc.rotate_quantize(to_bits(x), 256, 6)
    c2, s2, _, _ = orc.rotate_quantize(to_bits(x * 8.0), 256, 6)
    assert np.array_equal(c1, c2) and np.array_equal(s1 * 8.0, s2)


def test_rotation_lowers_quantization_error_on_outlier_channels():
    # Sec. 3.2: the rotation spreads massive outliers over the block.
    g = torch.Generator().manual_seed(0)
    x = torch.randn(64, 256, generator=g)
    x[:, [3, 77, 130, 201]] *= 20.0
    xb = to_bits(x)
    mse = {}
    for B in (0, 256):
        codes, s64, _, xt = orc.rotate_quantize(xb, B, 4)
        mse[B] = float(np.mean((xt - s64[:, None] * codes) ** 2))
    assert mse[256] < 0.5 * mse[0]


# ------------------------------------------------------------------ weight format (Sec. 3.1)

def test_minmax_weight_quantizer_matches_its_definition():
    g = torch.Generator().manual_seed(7)
    w = (torch.randn(16, 128, generator=g) * 0.02).to(torch.float64).numpy()
    w[3] += 0.03                                                 # shifted row -> zero point away from the middle
    u, d, z = orc.weight_quantize(w, "minmax")
    assert u.min() >= 0 and u.max() <= 15 and z.min() >= 0 and z.max() <= 15
    rng = w.max(axis=1) - w.min(axis=1)
    assert np.allclose(d, rng / 15.0, rtol=1e-7)                 # Delta = (max - min) / (2^b - 1)
    # extremes land on the end codes; reconstruction error <= Delta / 2 (+ the rounding of z)
    rec = d[:, None].astype(np.float64) * (u.astype(np.float64) - z[:, None])
    assert np.all(np.abs(rec - w) <= d[:, None] * (1.0 + 1e-6))
    rows = np.arange(16)
    assert np.all(u[rows, w.argmin(axis=1)] == 0) and np.all(u[rows, w.argmax(axis=1)] == 15)
    assert z[3] != z[0]
    # hand case: row (-1, 0, 2): Delta = 0.2, z = 5, codes (0, 5, 15)
    u2, d2, z2 = orc.weight_quantize(np.array([[-1.0, 0.0, 2.0]]), "minmax")
    assert abs(d2[0] - 0.2) < 1e-7 and z2[0] == 5 and list(u2[0]) == [0, 5, 15]


def test_symmetric_weight_quantizer():
    g = torch.Generator().manual_seed(8)
    w = (torch.randn(12, 256, generator=g) * 0.02).to(torch.float64).numpy()
    u, d, z = orc.weight_quantize(w, "symmetric")
    assert np.all(z == 8) and u.min() >= 1 and u.max() <= 15
    assert np.allclose(d, np.abs(w).max(axis=1) / 7.0, rtol=1e-7)
    rec = d[:, None].astype(np.float64) * (u.astype(np.float64) - 8.0)
    assert np.all(np.abs(rec - w) <= d[:, None] / 2 * (1 + 1e-6))
    # hand case, exact in binary: (0.875, -0.4375, 0.125) -> Delta 0.125, q = (7, -3.5 -> even -4, 1), u = q + 8
    u2, d2, z2 = orc.weight_quantize(np.array([[0.875, -0.4375, 0.125]]), "symmetric")
    assert list(u2[0]) == [15, 4, 9] and d2[0] == np.float32(0.125) and z2[0] == 8


# ------------------------------------------------------------------ integer GEMM (Eq. 10)

def test_int_gemm_against_brute_force_and_numpy():
    rng = np.random.default_rng(0)
    for (M, N, K) in [(1, 1, 1), (3, 5, 7), (17, 9, 64), (1, 33, 16), (40, 1, 24)]:
        c = rng.integers(-32, 32, size=(M, K), dtype=np.int32)
        u = rng.integers(0, 16, size=(N, K)).astype(np.uint8)
        z = rng.integers(0, 16, size=N).astype(np.int32)
        acc = orc.int_gemm(c, u, z)
        ref = c.astype(np.int64) @ (u.astype(np.int64) - z[:, None]).T
        assert np.array_equal(acc.astype(np.int64), ref)
        if M * N * K <= 3000:                                   # brute force, pure Python
            for i in range(M):
                for n in range(N):
                    s = 0
                    for k in range(K):
                        s += int(c[i, k]) * (int(u[n, k]) - int(z[n]))
                    assert s == int(acc[i, n])


def test_int_gemm_extremes_and_overflow_guard():
    K = 4096
    c = np.full((1, K), -32, dtype=np.int32)
    u = np.full((2, K), 15, dtype=np.uint8)
    u[1] = 0
    z = np.array([0, 15], dtype=np.int32)
    acc = orc.int_gemm(c, u, z)
    assert acc[0, 0] == -32 * 15 * K and acc[0, 1] == 32 * 15 * K
    big = np.full((1, 70000), 2 ** 15, dtype=np.int32)
    with pytest.raises(OverflowError):
        orc.int_gemm(big, np.full((1, 70000), 15, dtype=np.uint8), np.zeros(1, dtype=np.int32))


# ------------------------------------------------------------------ epilogue (Sec. 3.1 DeQuant, Eq. 10)

def test_worked_example_gemm_and_dequant():
    rows = read_golden("dequant_worked_example.txt")
    d = {k: [float(v) for v in vals[0]] for k, vals in rows.items()}
    codes = np.array([d["codes"]], dtype=np.int32)
    u = np.array([d["u0"], d["u1"]], dtype=np.uint8)
    z = np.array([d["z0"][0], d["z1"][0]], dtype=np.int32)
    acc = orc.int_gemm(codes, u, z)
    assert list(acc[0]) == [int(v) for v in d["acc"]]
    y = orc.epilogue(acc, np.array(d["scale"], dtype=np.float32), np.array(d["delta"], dtype=np.float32),
                     bits_of(d["bias"]), 0)
    assert list(bf16_values(y)[0]) == d["y"]
    y_nobias = orc.epilogue(acc, np.array(d["scale"], dtype=np.float32), np.array(d["delta"], dtype=np.float32), None, 0)
    assert list(bf16_values(y_nobias)[0]) == [-2.75, 9.0]


def test_bf16_rounding_matches_torch_and_breaks_ties_to_even():
    g = torch.Generator().manual_seed(11)
    v = torch.cat([torch.randn(4000, generator=g) * 3, torch.randn(2000, generator=g) * 1e-3,
                   torch.tensor([0.0, -0.0, 1.0, -1.0, 65504.0, 3.0e38, 1e-40, -1e-41])])
    want = to_bits(v)
    got = np.array([orc.double_to_bf16(float(x)) for x in v.to(torch.float64)], dtype=np.uint16)
    assert np.array_equal(got, want)
    # 1 + 2^-8 lies half-way between bf16 1.0 (even) and 1.0078125 (odd): goes to 1.0;
    # 1 + 3*2^-8 lies between 1.0078125 (odd) and 1.015625 (even): goes up.
    assert orc.double_to_bf16(1.0 + 2.0 ** -8) == orc.double_to_bf16(1.0)
    assert orc.double_to_bf16(1.0 + 3 * 2.0 ** -8) == orc.double_to_bf16(1.015625)
    # a double just above the half-way point must round up even though float32 would see a tie
    assert orc.double_to_bf16(1.0 + 2.0 ** -8 + 2.0 ** -40) == orc.double_to_bf16(1.0078125)
    for bits in (0x3F80, 0xC2F7, 0x0001, 0x7F7F):
        assert orc.double_to_bf16(orc.bf16_to_double(bits)) == bits


def test_gelu_tanh_against_torch_and_limits():
    xs = torch.linspace(-6, 6, 241, dtype=torch.float64)
    ref = torch.nn.functional.gelu(xs, approximate="tanh").numpy()
    got = np.array([orc.gelu_tanh(float(x)) for x in xs])
    assert np.abs(got - ref).max() < 1e-14
    assert orc.gelu_tanh(0.0) == 0.0 and abs(orc.gelu_tanh(30.0) - 30.0) < 1e-12 and abs(orc.gelu_tanh(-30.0)) < 1e-12


def test_epilogue_activation_rounds_twice():
    acc = np.array([[3, -5, 100]], dtype=np.int32)
    s = np.array([0.37], dtype=np.float32)
    dl = np.array([0.11, 0.23, 0.01], dtype=np.float32)
    y0 = bf16_values(orc.epilogue(acc, s, dl, None, 0))
    y1 = bf16_values(orc.epilogue(acc, s, dl, None, 1))
    ref = torch.nn.functional.gelu(torch.from_numpy(y0), approximate="tanh").to(torch.bfloat16).to(torch.float64).numpy()
    assert np.array_equal(y1, ref)


# ------------------------------------------------------------------ the method converges to the product it approximates

def test_error_halves_per_activation_bit_and_vanishes_without_weight_error():
    g = torch.Generator().manual_seed(21)
    M, N, K, B = 48, 40, 512, 512
    xb = to_bits(torch.randn(M, K, generator=g))
    wb = to_bits(torch.randn(N, K, generator=g) * 0.02)
    wt = orc.rotate(wb, B)
    exact = bf16_values(xb) @ bf16_values(wb).T
    xt = orc.rotate(xb, B)
    errs = {}
    for bits in (4, 6, 8, 10, 12, 16):
        codes, s64, _ = orc.act_quantize(xt, bits)
        y = (s64[:, None] * codes) @ wt.T                      # un-quantized weights
        errs[bits] = np.linalg.norm(y - exact) / np.linalg.norm(exact)
    for lo, hi in [(4, 6), (6, 8), (8, 10), (10, 12)]:
        ratio = errs[lo] / errs[hi]
        assert 3.0 < ratio < 5.5, (lo, hi, ratio)                # two bits = about 4x
    assert 10.0 < errs[12] / errs[16] < 24.0                     # four bits = about 16x
    assert errs[16] < 1e-4                                      # step / sqrt(12) relative to the token rms
    # full path at A4/W4 stays a sane approximation (weights dominate the error)
    u, d, z = orc.weight_quantize(wt, "symmetric")
    out = orc.qlinear(xb, u, d, z, B, 4)
    rel = np.linalg.norm(bf16_values(out["y"]) - exact) / np.linalg.norm(exact)
    assert 0.02 < rel < 0.35
    # and the dequantized integer result equals the same product in plain floating point
    ref = (out["scale32"].astype(np.float64)[:, None] * out["codes"]) @ (d.astype(np.float64)[:, None] * (u.astype(np.float64) - z[:, None])).T
    assert np.abs(bf16_values(out["y"]) - ref).max() <= np.abs(ref).max() * 2.0 ** -8


# ------------------------------------------------------------------ block-wise scales

def test_grouped_quantizer_reduces_to_the_per_token_one_and_keeps_its_invariants():
    g = torch.Generator().manual_seed(21)
    x = torch.randn(12, 2048, generator=g)
    x[:, 5] *= 30.0                                             # an outlier channel in the first block only
    xb = x.to(torch.bfloat16)
    w = (torch.randn(16, 2048, generator=g) * 0.02).to(torch.bfloat16)
    from helpers import to_bits, bf16_values
    u, d, z = orc.prepare_weights(to_bits(w), 1024, "minmax")
    # one block = the whole row: identical to the per-token path, bit for bit
    a = orc.qlinear_grouped(to_bits(xb), u, d, z, 1024, 4, 2048)
    b = orc.qlinear(to_bits(xb), u, d, z, 1024, 4)
    assert np.array_equal(a["codes"], b["codes"]) and np.array_equal(a["y"], b["y"])
    # two blocks: every block has its own scale = its own absmax / qmax, error <= scale / 2 per element
    c = orc.qlinear_grouped(to_bits(xb), u, d, z, 1024, 4, 1024)
    xt = c["xt"]
    for blk in range(2):
        sl = slice(blk * 1024, (blk + 1) * 1024)
        s = c["scale64"][:, blk]
        assert np.allclose(s * 7, np.abs(xt[:, sl]).max(axis=1), rtol=1e-15)
        assert (np.abs(xt[:, sl] - s[:, None] * c["codes"][:, sl]) <= s[:, None] / 2 * (1 + 1e-12)).all()
        assert (np.abs(c["codes"][:, sl]).max(axis=1) == 7).all()
    # the combination over blocks, retyped with numpy from the stage outputs
    acc0 = orc.int_gemm(c["codes"][:, :1024], np.ascontiguousarray(u[:, :1024]), z).astype(np.float64)
    acc1 = orc.int_gemm(c["codes"][:, 1024:], np.ascontiguousarray(u[:, 1024:]), z).astype(np.float64)
    v = (acc0 * c["scale32"][:, :1].astype(np.float64) + acc1 * c["scale32"][:, 1:].astype(np.float64)) * d.astype(np.float64)[None, :]
    ref = torch.from_numpy(v).to(torch.bfloat16).to(torch.float64).numpy()   # torch's cast: fp64 -> bf16, ties to even
    assert np.array_equal(bf16_values(c["y"]), ref)
    # the outlier only costs its own block its resolution: the block-wise result is closer to X W^T
    exact = xb.to(torch.float64).numpy() @ w.to(torch.float64).numpy().T
    err_tok = np.linalg.norm(bf16_values(b["y"]) - exact)
    err_blk = np.linalg.norm(bf16_values(c["y"]) - exact)
    assert err_blk < err_tok


def test_round_output_adds_the_bias_before_the_rounding_and_rounds_twice_around_the_gelu():
    # Hand-set fp64 values and bf16 biases; the expected bits come from torch alone: fp64 add, its
    # cast to bf16 (ties to even), its tanh-GELU in fp64 on the rounded value, its cast again.
    # 1.00390625 = 1 + 2^-8 is a bf16 tie (rounds down to 1.0 on its own); the bias 2^-9 lifts the
    # sum above the tie, so adding the bias AFTER the rounding gives a different bit pattern.
    v = np.array([[1.00390625, -2.7, 0.3333, 117.25, -0.0625, 3.0e-3],
                  [0.0, 5.5, -1.00390625, 0.49, 12.0, -40.0]], dtype=np.float64)
    bias = torch.tensor([2.0 ** -9, 0.5, -0.25, 3.0, 0.0625, -1.0e-3]).to(torch.bfloat16)
    bias_bits = to_bits(bias)
    summed = torch.from_numpy(v) + bias.to(torch.float64)[None, :]
    ref0 = summed.to(torch.bfloat16)
    ref1 = torch.nn.functional.gelu(ref0.to(torch.float64), approximate="tanh").to(torch.bfloat16)
    y0 = orc.round_output(v, bias_bits, 0)
    y1 = orc.round_output(v, bias_bits, 1)
    assert np.array_equal(y0, to_bits(ref0))
    assert np.array_equal(y1, to_bits(ref1))
    # the tie really is decided by the bias: without it the first element rounds to 1.0
    assert bf16_values(orc.round_output(v, None, 0))[0, 0] == 1.0 and bf16_values(y0)[0, 0] > 1.0
    # one rounding after the GELU is not the same thing: a fused fp64 GELU of the unrounded sum differs somewhere
    fused = torch.nn.functional.gelu(summed, approximate="tanh").to(torch.bfloat16)
    assert not np.array_equal(y1, to_bits(fused))
    # and it agrees with the per-token epilogue on the same numbers (acc * s * Delta formed here in fp64)
    acc = np.array([[3, -5, 100, 7, -9, 1]], dtype=np.int32)
    s = np.array([0.37], dtype=np.float32)
    dl = np.array([0.11, 0.23, 0.01, 0.5, 0.07, 0.9], dtype=np.float32)
    vv = acc.astype(np.float64) * s.astype(np.float64)[:, None] * dl.astype(np.float64)[None, :]
    for act in (0, 1):
        assert np.array_equal(orc.round_output(vv, bias_bits, act), orc.epilogue(acc, s, dl, bias_bits, act))
