"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle on the same
seeded inputs.  Bars (written here once):

  * packed formats, code sums, int32 accumulators: bit exact;
  * scales: 1e-6 relative;
  * codes: equal on >= 99.99 % of the elements, every mismatch +-1 on a rounding tie;
  * bf16 outputs: 4e-3 relative in max-norm (and <= 1 bf16 ulp elementwise when the GEMM is
    fed the oracle's own codes and scales).  Whole-layer comparisons validate the codes first
    and let the oracle take the GPU's side on rounding ties (oracle_y_for_validated_codes).
"""
import ctypes as C

import numpy as np
import pytest
import torch

from oracle import dvdq_oracle as orc
from paper_2505_18663_b200 import binding as B
from paper_2505_18663_b200 import workloads as W

from helpers import (act_quant, bf16_values, check_codes_against_oracle, from_bits, gpu_pack_codes,
                     gpu_pack_weights, gpu_rotate_quantize, oracle_y_for_validated_codes, to_bits)

pytestmark = pytest.mark.gpu
DEV = "cuda"

SCALE_RTOL = 1e-6
Y_MAXNORM_RTOL = 4e-3


def assert_device_ok():
    status, detail = B.dvdq_last_device_status()
    assert status == B.OK, f"device status {status} ({B.status_string(status)}), wait id {detail}"


def synth_x(M, K, seed, outliers=4, gain=20.0):
    g = torch.Generator().manual_seed(seed)
    x = torch.randn(M, K, generator=g)
    if outliers:
        x[:, torch.randperm(K, generator=g)[:outliers]] *= gain
    return x.to(torch.bfloat16)


def synth_w(N, K, seed):
    g = torch.Generator().manual_seed(seed)
    return (torch.randn(N, K, generator=g) * 0.02).to(torch.bfloat16)


# ------------------------------------------------------------------ formats

@pytest.mark.parametrize("bits", [4, 6, 8])
def test_activation_code_pack_unpack_roundtrip(bits):
    M, K = 37, 448
    lim = 2 ** (bits - 1)
    rng = np.random.default_rng(bits)
    codes = rng.integers(-lim, lim, size=(M, K)).astype(np.int8)
    codes[0, :] = lim - 1
    codes[1, :] = -lim
    packed, sums = gpu_pack_codes(codes, bits, 64)
    nat = torch.empty(M, K, dtype=torch.int8, device=DEV)
    B.dvdq_unpack_act_codes(packed, M, K, act_quant(bits, 64), nat)
    assert np.array_equal(nat.cpu().numpy(), codes)
    assert np.array_equal(sums.cpu().numpy(), codes.astype(np.int64).sum(axis=1))
    assert packed.numel() == M * K * bits // 8


def test_weight_blob_roundtrip():
    N, K = 264, 320
    rng = np.random.default_rng(1)
    u = rng.integers(0, 16, size=(N, K)).astype(np.uint8)
    d = rng.random(N).astype(np.float32) + 0.01
    z = rng.integers(0, 16, size=N).astype(np.int32)
    w, blob = gpu_pack_weights(u, d, z, 64)
    assert (w.N, w.K, w.rot_block) == (N, K, 64) and w.blob_bytes == blob.numel()
    u2 = torch.empty(N, K, dtype=torch.uint8, device=DEV)
    d2 = torch.empty(N, dtype=torch.float32, device=DEV)
    z2 = torch.empty(N, dtype=torch.int32, device=DEV)
    B.dvdq_unpack_weights(w, u2, d2, z2)
    assert np.array_equal(u2.cpu().numpy(), u) and np.array_equal(d2.cpu().numpy(), d) and np.array_equal(z2.cpu().numpy(), z)


# ------------------------------------------------------------------ rotate -> scale -> quantize -> pack

RQ_CASES = [
    # M, K, B  (several warps per token, ragged last span, every supported block size, no rotation)
    (256, 256, 256), (300, 1536, 512), (130, 3072, 1024), (67, 8960, 256), (33, 13824, 512),
    (129, 320, 64), (65, 640, 128), (40, 5120, 1024), (50, 1024, 0), (9, 12288, 1024),
    # rotation blocks that span two and four warps
    (37, 12288, 4096), (70, 4096, 2048), (19, 4096, 4096), (130, 2048, 2048), (11, 16384, 4096),
]


@pytest.mark.parametrize("bits", [4, 6, 8])
@pytest.mark.parametrize("M,K,Bk", RQ_CASES)
def test_rotate_quantize_matches_oracle(M, K, Bk, bits):
    x = synth_x(M, K, seed=M + K + bits)
    x[M // 2] = 0                                               # an all-zero token
    codes_or, s64, s32, xt = orc.rotate_quantize(to_bits(x), Bk, bits)
    _, scales, sums, nat = gpu_rotate_quantize(x.to(DEV), bits, Bk)
    s_gpu = scales.cpu().numpy().astype(np.float64)
    nz = s64 > 0
    assert np.all(s_gpu[~nz] == 0)
    assert np.abs(s_gpu[nz] / s64[nz] - 1.0).max() <= SCALE_RTOL
    nat_np = nat.cpu().numpy()
    qmax = 2 ** (bits - 1) - 1
    assert nat_np.min() >= -qmax and nat_np.max() <= qmax
    check_codes_against_oracle(nat_np, codes_or, xt, s64)
    assert np.all(nat_np[M // 2] == 0)
    assert np.array_equal(sums.cpu().numpy(), nat_np.astype(np.int64).sum(axis=1))   # sums describe the GPU's own codes
    assert np.all(np.abs(nat_np[nz]).max(axis=1) == qmax)       # absmax element sits on +-qmax
    assert_device_ok()


def test_rotate_quantize_strided_input_and_scale_equivariance():
    M, K, Bk = 77, 1536, 512
    big = torch.zeros(M, K + 64, dtype=torch.bfloat16)
    big[:, :K] = synth_x(M, K, 5)
    xd = big.to(DEV)[:, :K]                                      # row pitch K + 64
    _, s1, _, c1 = gpu_rotate_quantize(xd, 6, Bk)
    _, s0, _, c0 = gpu_rotate_quantize(xd.contiguous(), 6, Bk)
    assert torch.equal(c0, c1) and torch.equal(s0, s1)
    _, s2, _, c2 = gpu_rotate_quantize((xd.float() * 16.0).to(torch.bfloat16).contiguous(), 6, Bk)
    assert torch.equal(c0, c2) and torch.equal(s0 * 16.0, s2)   # exact in binary floating point


@pytest.mark.parametrize("bits,pattern", [(4, (60.0, 36.0, 16.0)), (4, (76.0, 36.0, 0.0)), (6, (284.0, 212.0, 0.0))])
def test_rotate_quantize_exact_ties_round_to_even(bits, pattern):
    # Tokens with two or three non-zero channels a, b, c: with B = 256 every rotated value is
    # (+-a +-b +-c) / 16.  The patterns make the absmax 7 (or 31), so the scale is exactly 1
    # (times a power of two per token), and put other values exactly half-way between two codes
    # (2.5, -0.5, 4.5 ...).  x~ / s is then exact in fp32 and fp64 alike, so both sides must take
    # the same round-half-to-even decision on every element.
    K = Bk = 256
    M = 32
    g = torch.Generator().manual_seed(9)
    x = torch.zeros(M, K)
    for i in range(M):
        pos = torch.randperm(K, generator=g)[:3]
        for p_, v in zip(pos.tolist(), pattern):
            x[i, p_] = v * (2.0 ** (i % 5 - 2))
    xb = x.to(torch.bfloat16)
    assert torch.equal(xb.float(), x)
    codes_or, s64, _, xt_or = orc.rotate_quantize(to_bits(xb), Bk, bits)
    ratio = xt_or / s64[:, None]
    assert np.any(np.abs(ratio * 2 % 2) == 1)                    # half-way cases are present
    assert np.all(np.log2(s64) == np.round(np.log2(s64)))        # scales are powers of two
    _, scales, _, nat = gpu_rotate_quantize(xb.to(DEV), bits, Bk)
    assert np.array_equal(scales.cpu().numpy().astype(np.float64), s64)
    assert np.array_equal(nat.cpu().numpy().astype(np.int32), codes_or)


def test_empty_and_single_token():
    q = act_quant(4, 256)
    e = torch.empty(1, dtype=torch.uint8, device=DEV)
    lib = B.load()
    assert lib.dvdq_rotate_quantize(None, 0, 256, 256, C.byref(q), None, None, None, None) == B.OK
    x = synth_x(1, 256, 3)
    codes_or, s64, _, xt = orc.rotate_quantize(to_bits(x), 256, 4)
    _, scales, _, nat = gpu_rotate_quantize(x.to(DEV), 4, 256)
    assert abs(float(scales[0]) / s64[0] - 1) <= SCALE_RTOL
    check_codes_against_oracle(nat.cpu().numpy(), codes_or, xt, s64, min_agree=0.99)
    del e


# ------------------------------------------------------------------ integer GEMM

GEMM_CASES = [
    # M, N, K, B, bits, weight mode  (M tail, N tail, one and many k-blocks, K not a multiple of 128, z != 8)
    (256, 256, 256, 256, 4, "symmetric"),
    (130, 264, 320, 64, 4, "minmax"),
    (1, 8, 64, 64, 6, "minmax"),
    (300, 512, 1536, 512, 6, "symmetric"),
    (257, 776, 3072, 1024, 4, "minmax"),
    (129, 256, 8960, 256, 6, "minmax"),
    # 8-bit activations (the b_high steps of the bit-width switching): M and N tails, K not a multiple of 256
    (300, 520, 1536, 512, 8, "minmax"),
    (257, 192, 3200, 128, 8, "symmetric"),
]


def oracle_layer(M, N, K, Bk, bits, mode, seed):
    x = synth_x(M, K, seed)
    wb = synth_w(N, K, seed + 1)
    if mode == "minmax":
        wb = (wb.float() + 0.004 * torch.randn(N, 1, generator=torch.Generator().manual_seed(seed))).to(torch.bfloat16)
    u, d, z = orc.prepare_weights(to_bits(wb), Bk, mode)
    codes, s64, s32, xt = orc.rotate_quantize(to_bits(x), Bk, bits)
    return x, u, d, z, codes, s64, s32, xt


@pytest.mark.parametrize("M,N,K,Bk,bits,mode", GEMM_CASES)
def test_int32_accumulators_are_bit_exact_on_oracle_codes(M, N, K, Bk, bits, mode):
    x, u, d, z, codes, s64, s32, xt = oracle_layer(M, N, K, Bk, bits, mode, seed=M + N)
    acc_or = orc.int_gemm(codes, u, z)
    w, blob = gpu_pack_weights(u, d, z, Bk)
    packed, sums = gpu_pack_codes(codes, bits, Bk)
    acc = torch.full((M, N), 12345, dtype=torch.int32, device=DEV)
    B.dvdq_qgemm_int32(packed, sums, M, act_quant(bits, Bk), w, acc)
    assert_device_ok()
    assert np.array_equal(acc.cpu().numpy(), acc_or)


@pytest.mark.parametrize("bits", [6, 8])
def test_int32_accumulators_at_code_extremes(bits):
    # every product at its largest magnitude: |acc| = K * 2^(bits-1) * 15
    M, N, K = 128, 256, 4096
    lim = 2 ** (bits - 1)
    codes = np.full((M, K), -lim, dtype=np.int32)
    codes[1::2] = lim - 1
    u = np.zeros((N, K), dtype=np.uint8)
    u[::2] = 15
    z = np.zeros(N, dtype=np.int32)
    z[1::2] = 15
    d = np.ones(N, dtype=np.float32)
    acc_or = orc.int_gemm(codes, u, z)
    assert np.abs(acc_or).max() == lim * 15 * K
    w, blob = gpu_pack_weights(u, d, z, 1024)
    packed, sums = gpu_pack_codes(codes, bits, 1024)
    acc = torch.zeros(M, N, dtype=torch.int32, device=DEV)
    B.dvdq_qgemm_int32(packed, sums, M, act_quant(bits, 1024), w, acc)
    assert_device_ok()
    assert np.array_equal(acc.cpu().numpy(), acc_or)


# ------------------------------------------------------------------ dequantizing epilogue

@pytest.mark.parametrize("act", [0, 1])
@pytest.mark.parametrize("M,N,K,Bk,bits,mode", [GEMM_CASES[1], GEMM_CASES[3], GEMM_CASES[4], GEMM_CASES[6]])
def test_bf16_output_on_oracle_codes_and_scales(M, N, K, Bk, bits, mode, act):
    x, u, d, z, codes, s64, s32, xt = oracle_layer(M, N, K, Bk, bits, mode, seed=3 * M + N)
    bias = (torch.randn(N, generator=torch.Generator().manual_seed(N)) * 0.05).to(torch.bfloat16)
    y_or = bf16_values(orc.epilogue(orc.int_gemm(codes, u, z), s32, d, to_bits(bias), act))
    w, blob = gpu_pack_weights(u, d, z, Bk)
    packed, sums = gpu_pack_codes(codes, bits, Bk)
    Y = torch.zeros(M, N + 8, dtype=torch.bfloat16, device=DEV)[:, :N]          # padded row pitch
    B.dvdq_qgemm(packed, torch.from_numpy(s32).to(DEV), sums, M, act_quant(bits, Bk), w, bias.to(DEV), act, Y)
    assert_device_ok()
    y = Y.to(torch.float64).cpu().numpy()
    assert np.abs(y - y_or).max() <= Y_MAXNORM_RTOL * np.abs(y_or).max()
    # identical integer inputs: only the fp32-vs-fp64 epilogue differs, i.e. at most one bf16 ulp
    # of the linear output; through GELU (slope <= 1.13) that ulp plus the second rounding.
    y0_or = bf16_values(orc.epilogue(orc.int_gemm(codes, u, z), s32, d, to_bits(bias), 0))
    ulp = np.maximum(np.abs(y0_or), 2.0 ** -100) * 2.0 ** -7
    assert np.all(np.abs(y - y_or) <= (ulp if act == 0 else 3 * ulp))
    assert np.mean(y != y_or) < 0.02


# ------------------------------------------------------------------ the whole layer

def run_qlinear(x_dev, w, bits, Bk, bias_dev, act, N):
    """dvdq_qlinear; returns (Y, natural-order codes read back from the head of the workspace)."""
    M, K = x_dev.shape
    q = act_quant(bits, Bk)
    ws = torch.empty(B.dvdq_qlinear_workspace_bytes(M, K, q), dtype=torch.uint8, device=DEV)
    Y = torch.empty(M, N, dtype=torch.bfloat16, device=DEV)
    B.dvdq_qlinear(x_dev, q, w, bias_dev, act, Y, ws)
    nat = torch.empty(M, K, dtype=torch.int8, device=DEV)
    B.dvdq_unpack_act_codes(ws, M, K, q, nat)
    return Y, nat.cpu().numpy()


@pytest.mark.parametrize("M,N,K,Bk,bits,mode", [GEMM_CASES[0], GEMM_CASES[3], GEMM_CASES[4], GEMM_CASES[6], GEMM_CASES[7]])
def test_qlinear_matches_oracle_end_to_end(M, N, K, Bk, bits, mode):
    x, u, d, z, codes, s64, s32, xt = oracle_layer(M, N, K, Bk, bits, mode, seed=7 * M + N)
    out = {"codes": codes, "xt": xt, "scale64": s64, "scale32": s32,
           "y": orc.epilogue(orc.int_gemm(codes, u, z), s32, d, None, 0)}
    w, blob = gpu_pack_weights(u, d, z, Bk)
    Y, nat = run_qlinear(x.to(DEV), w, bits, Bk, None, 0, N)
    assert_device_ok()
    y = Y.to(torch.float64).cpu().numpy()
    y_or = oracle_y_for_validated_codes(nat, out, u, d, z)
    assert np.abs(y - y_or).max() <= Y_MAXNORM_RTOL * np.abs(y_or).max()


def test_tiny_config_full_comparison():
    """The small single-layer case: 256 tokens x 256 -> 256, four outlier channels x20, W4A4, B = 256, seed 0."""
    wl = W.WORKLOADS["tiny"]
    layer = wl.layers[0]
    x = W.make_activations(wl, layer.K)
    wb = W.make_weights(wl, layer)
    u, d, z = orc.prepare_weights(to_bits(wb), layer.rot_block, "symmetric")
    out = orc.qlinear(to_bits(x), u, d, z, layer.rot_block, layer.bits)
    w, blob = gpu_pack_weights(u, d, z, layer.rot_block)
    _, scales, _, nat = gpu_rotate_quantize(x.to(DEV), layer.bits, layer.rot_block)
    assert np.abs(scales.cpu().numpy().astype(np.float64) / out["scale64"] - 1).max() <= SCALE_RTOL
    check_codes_against_oracle(nat.cpu().numpy(), out["codes"], out["xt"], out["scale64"])
    Y, nat_q = run_qlinear(x.to(DEV), w, layer.bits, layer.rot_block, None, 0, layer.N)
    assert_device_ok()
    y, y_or = Y.to(torch.float64).cpu().numpy(), oracle_y_for_validated_codes(nat_q, out, u, d, z)
    assert np.abs(y - y_or).max() <= Y_MAXNORM_RTOL * np.abs(y_or).max()
    exact = x.to(torch.float64).numpy() @ wb.to(torch.float64).numpy().T
    rel = np.linalg.norm(y - exact) / np.linalg.norm(exact)
    assert rel < 0.5                                             # W4A4 stays an approximation of X W^T


def test_ffn_chain_stage_by_stage():
    """Config-5 chain at a reduced token count: rq(A4) -> 3072->12288 -> GELU -> rq(A6) -> 12288->3072 + bias.
    Each stage is compared on identical inputs: the oracle's second stage is fed the GPU's
    first-stage output."""
    wl = W.WORKLOADS["ffn_chain"]
    up, down = wl.layers
    M = 200
    x = W.make_activations(wl, up.K, M=M)
    w1 = W.make_weights(wl, up)
    w2 = W.make_weights(wl, down)
    bias = W.make_bias(wl, down)
    u1, d1, z1 = orc.prepare_weights(to_bits(w1), up.rot_block)
    u2, d2, z2 = orc.prepare_weights(to_bits(w2), down.rot_block)
    h1, blob1 = gpu_pack_weights(u1, d1, z1, up.rot_block)
    h2, blob2 = gpu_pack_weights(u2, d2, z2, down.rot_block)
    Y1, nat1 = run_qlinear(x.to(DEV), h1, up.bits, up.rot_block, None, up.act, up.N)
    Y2, nat2 = run_qlinear(Y1, h2, down.bits, down.rot_block, bias.to(DEV), down.act, down.N)
    assert_device_ok()
    o1 = orc.qlinear(to_bits(x), u1, d1, z1, up.rot_block, up.bits, None, up.act)
    y1, y1_or = Y1.to(torch.float64).cpu().numpy(), oracle_y_for_validated_codes(nat1, o1, u1, d1, z1, None, up.act)
    assert np.abs(y1 - y1_or).max() <= Y_MAXNORM_RTOL * np.abs(y1_or).max()
    o2 = orc.qlinear(to_bits(Y1), u2, d2, z2, down.rot_block, down.bits, to_bits(bias), down.act)
    y2, y2_or = Y2.to(torch.float64).cpu().numpy(), oracle_y_for_validated_codes(nat2, o2, u2, d2, z2, to_bits(bias), down.act)
    assert np.abs(y2 - y2_or).max() <= Y_MAXNORM_RTOL * np.abs(y2_or).max()


# ------------------------------------------------------------------ full-size launch configuration, sampled rows

FULL_SIZE_CASES = [
    # workload, layer: the benchmark's own launch configurations plus the ragged ones of the other
    # configs (M = 32760 = 127 * 256 + 248 tokens, K = 1536 / 13824 with a partial last span, A6)
    ("hunyuan", 0), ("hunyuan", 3), ("wan1p3b", 2), ("wan14b", 3), ("ffn_chain", 1),
]


@pytest.mark.parametrize("container", [8, 0])
@pytest.mark.parametrize("workload,layer_idx", FULL_SIZE_CASES)
def test_full_size_layer_on_sampled_rows(workload, layer_idx, container):
    """Full token counts of the benchmark configurations, with the codes kept one int8 each (what
    the benchmark times by default) and packed: scales, codes and bf16 outputs on sampled rows
    (first tile, last full tile, ragged tail, seeded rows), computed one row at a time by the
    oracle; plus a property of the whole output."""
    wl = W.WORKLOADS[workload]
    layer = wl.layers[layer_idx]
    if workload == "hunyuan" and layer_idx == 3 and container == 8:
        import dataclasses
        layer = dataclasses.replace(layer, rot_block=4096)      # rotation blocks that span four warps, at full size
    M = wl.M
    x = W.make_activations(wl, layer.K, device=DEV)
    u, d, z = W.make_weight_codes(layer, seed=layer_idx, device=DEV, symmetric=(layer_idx != 3))
    blob = torch.empty(B.dvdq_weight_blob_bytes(layer.N, layer.K), dtype=torch.uint8, device=DEV)
    w = B.dvdq_pack_weights(u, d, z, layer.rot_block, blob)
    q = act_quant(layer.bits, layer.rot_block, container)
    codes = torch.empty(B.dvdq_act_codes_bytes_q(M, layer.K, q), dtype=torch.uint8, device=DEV)
    scales = torch.empty(M, dtype=torch.float32, device=DEV)
    sums = torch.empty(M, dtype=torch.int32, device=DEV)
    Y = torch.empty(M, layer.N, dtype=torch.bfloat16, device=DEV)
    bias = W.make_bias(wl, layer, device=DEV)
    # the three launches of a layer, as the benchmark issues them: the transform, the weight operand
    # written into a scratch area, the GEMM that reads it
    scratch = torch.empty(layer.N * layer.K, dtype=torch.uint8, device=DEV)
    B.dvdq_rotate_quantize(x, q, codes, scales, sums)
    B.dvdq_qgemm(codes, scales, sums, M, q, B.dvdq_widen_weights(w, scratch), bias, layer.act, Y)
    assert_device_ok()
    # the GEMM that widens the weights itself, tile by tile, gives the same bits
    Y_tile = torch.empty_like(Y)
    B.dvdq_qgemm(codes, scales, sums, M, q, w, bias, layer.act, Y_tile)
    assert_device_ok()
    assert torch.equal(Y, Y_tile)
    del Y_tile, scratch
    rows = W.sample_rows(M, 40, tile=256, seed=layer_idx)
    xs = x[rows.to(DEV)].cpu()
    un, dn, zn = u.cpu().numpy(), d.cpu().numpy(), z.cpu().numpy()
    bias_bits = None if bias is None else to_bits(bias)
    out = orc.qlinear(to_bits(xs), un, dn, zn, layer.rot_block, layer.bits, bias_bits, layer.act)
    s_gpu = scales[rows.to(DEV)].cpu().numpy().astype(np.float64)
    assert np.abs(s_gpu / out["scale64"] - 1.0).max() <= SCALE_RTOL
    nat = torch.empty(M, layer.K, dtype=torch.int8, device=DEV)
    B.dvdq_unpack_act_codes(codes, M, layer.K, q, nat)
    nat_s = nat[rows.to(DEV)].cpu().numpy()
    assert np.array_equal(sums[rows.to(DEV)].cpu().numpy(), nat_s.astype(np.int64).sum(axis=1))
    del nat
    y = Y[rows.to(DEV)].to(torch.float64).cpu().numpy()
    y_or = oracle_y_for_validated_codes(nat_s, out, un, dn, zn, bias_bits, layer.act)
    assert np.abs(y - y_or).max() <= Y_MAXNORM_RTOL * np.abs(y_or).max()
    # a property that holds at any size: no NaN/Inf anywhere in the full output
    assert bool(torch.isfinite(Y).all())
