"""One layer's GEMM fused with the next layer's activation transform (Eq. 10 applied layer after
layer: Y of one layer is X of the next): dvdq_qgemm_fused_rq against the unfused CUDA path and,
stage by stage on identical inputs, against the oracle (rotation by H_256, block-wise quantizer
with groups of 256, then the block-wise layer that consumes the codes)."""
import numpy as np
import pytest
import torch

from oracle import dvdq_oracle as orc
from paper_2505_18663_b200 import binding as B
from paper_2505_18663_b200 import workloads as W

from helpers import bf16_values, check_codes_against_oracle, gpu_pack_weights, to_bits

pytestmark = pytest.mark.gpu
DEV = "cuda"
SCALE_RTOL = 1e-6
Y_MAXNORM_RTOL = 4e-3
G = 256   # rotation block = scale group of the fused transform: the width of a GEMM tile


def assert_device_ok():
    status, detail = B.dvdq_last_device_status()
    assert status == B.OK, f"device status {status} ({B.status_string(status)}), wait id {detail}"


def first_stage(x_dev, bits, Bk, container=8):
    """The first layer's own transform: per-token scales, codes one int8 each or packed."""
    M, K = x_dev.shape
    q = B.ActQuant(bits, Bk, 0, container)
    codes = torch.empty(B.dvdq_act_codes_bytes_q(M, K, q), dtype=torch.uint8, device=DEV)
    scales = torch.empty(M, dtype=torch.float32, device=DEV)
    sums = torch.empty(M, dtype=torch.int32, device=DEV)
    B.dvdq_rotate_quantize(x_dev, q, codes, scales, sums)
    return q, codes, scales, sums


def run_fused(q, codes, scales, sums, M, w, bias, act, N, bits_next, with_y=True):
    qn = B.ActQuant(bits_next, G, G, 8)
    cn = torch.full((B.dvdq_act_codes_bytes_q(M, N, qn),), 0x55, dtype=torch.uint8, device=DEV)
    sn = torch.full((M * (N // G),), -1.0, dtype=torch.float32, device=DEV)
    Sn = torch.full((M * (N // G),), 123456, dtype=torch.int32, device=DEV)
    Y = torch.zeros(M, N, dtype=torch.bfloat16, device=DEV) if with_y else None
    B.dvdq_qgemm_fused_rq(codes, scales, sums, M, q, w, bias, act, qn, cn, sn, Sn, Y)
    assert_device_ok()
    # the weight operand written once (dvdq_widen_weights) instead of widened tile by tile: the same bits
    operand = torch.empty(w.N * w.K, dtype=torch.uint8, device=DEV)
    cn2, sn2, Sn2 = torch.zeros_like(cn), torch.zeros_like(sn), torch.zeros_like(Sn)
    B.dvdq_qgemm_fused_rq(codes, scales, sums, M, q, B.dvdq_widen_weights(w, operand), bias, act, qn, cn2, sn2, Sn2, None)
    assert_device_ok()
    assert torch.equal(cn, cn2) and torch.equal(sn, sn2) and torch.equal(Sn, Sn2)
    return qn, cn, sn.view(M, N // G), Sn.view(M, N // G), Y


def check_against_oracle(y_bits, nat, scales, sums, bits_next):
    """The fused outputs against the oracle's transform of the very bf16 values the kernel produced."""
    xt = orc.rotate(y_bits, G)
    codes_or, s64, _ = orc.act_quantize_grouped(xt, bits_next, G)
    s = scales.astype(np.float64)
    assert np.all(np.abs(s - s64) <= SCALE_RTOL * s64)
    assert (nat.astype(np.int32) == codes_or).mean() >= 0.9999
    for g in range(xt.shape[1] // G):
        sl = slice(g * G, (g + 1) * G)
        check_codes_against_oracle(nat[:, sl], codes_or[:, sl], xt[:, sl], s64[:, g], min_agree=0.0)
    M = nat.shape[0]
    assert np.array_equal(sums, nat.astype(np.int64).reshape(M, -1, G).sum(axis=2))
    qmax = 2 ** (bits_next - 1) - 1
    nz = s64 > 0
    assert np.all(np.abs(nat.reshape(M, -1, G)).max(axis=2)[nz] == qmax)


@pytest.mark.parametrize("container", [8, 0])
@pytest.mark.parametrize("M,K,N,Bk,bits,act,use_bias,bits_next", [
    (200, 512, 512, 256, 4, 1, True, 6),      # a row tail, two column tiles, GELU + bias
    (513, 1024, 256, 1024, 6, 0, False, 4),   # three row tiles (one with a single row), one column tile
    (64, 256, 768, 64, 8, 1, False, 8),
])
def test_fused_epilogue_matches_unfused_output_and_oracle_transform(M, K, N, Bk, bits, act, use_bias, bits_next, container):
    g = torch.Generator().manual_seed(M + K + N)
    x = torch.randn(M, K, generator=g)
    x[:, torch.randperm(K, generator=g)[:4]] *= 20.0
    x[M // 2] = 0                                              # an all-zero token: y = bias (or 0)
    x = x.to(torch.bfloat16)
    wb = (torch.randn(N, K, generator=g) * 0.02).to(torch.bfloat16)
    u, d, z = orc.prepare_weights(to_bits(wb), Bk, "minmax")
    w, blob = gpu_pack_weights(u, d, z, Bk)
    bias = (torch.randn(N, generator=g) * 0.1).to(torch.bfloat16).to(DEV) if use_bias else None
    q, codes, scales, sums = first_stage(x.to(DEV), bits, Bk, container)
    # the unfused layer on the same codes: its bf16 output is what the fused epilogue must reproduce, bit for bit
    Y_ref = torch.empty(M, N, dtype=torch.bfloat16, device=DEV)
    B.dvdq_qgemm(codes, scales, sums, M, q, w, bias, act, Y_ref)
    qn, cn, sn, Sn, Y = run_fused(q, codes, scales, sums, M, w, bias, act, N, bits_next)
    assert torch.equal(Y, Y_ref)
    nat = torch.empty(M, N, dtype=torch.int8, device=DEV)
    B.dvdq_unpack_act_codes(cn, M, N, qn, nat)
    check_against_oracle(to_bits(Y), nat.cpu().numpy(), sn.cpu().numpy(), Sn.cpu().numpy(), bits_next)
    if not use_bias:
        assert np.all(nat.cpu().numpy()[M // 2] == 0) and np.all(sn.cpu().numpy()[M // 2] == 0)
    # without the debug output the codes are the same
    _, cn2, sn2, Sn2, _ = run_fused(q, codes, scales, sums, M, w, bias, act, N, bits_next, with_y=False)
    assert torch.equal(cn, cn2) and torch.equal(sn, sn2) and torch.equal(Sn, Sn2)


def test_fused_chain_of_two_layers_matches_oracle_stage_by_stage():
    """rotate-quantize(A4) -> GEMM + GELU fused with rotate-quantize(A6, B = G = 256) -> block-wise GEMM + bias."""
    M, K1, N1, N2 = 300, 768, 1024, 264
    g = torch.Generator().manual_seed(17)
    x = torch.randn(M, K1, generator=g)
    x[:, 5] *= 30.0
    x = x.to(torch.bfloat16)
    w1 = (torch.randn(N1, K1, generator=g) * 0.02).to(torch.bfloat16)
    w2 = (torch.randn(N2, N1, generator=g) * 0.02).to(torch.bfloat16)
    bias2 = (torch.randn(N2, generator=g) * 0.1).to(torch.bfloat16)
    u1, d1, z1 = orc.prepare_weights(to_bits(w1), 256, "symmetric")
    u2, d2, z2 = orc.prepare_weights(to_bits(w2), G, "minmax")
    h1, blob1 = gpu_pack_weights(u1, d1, z1, 256)
    h2, blob2 = gpu_pack_weights(u2, d2, z2, G)
    q1, codes, scales, sums = first_stage(x.to(DEV), 4, 256)
    qn, cn, sn, Sn, Y1 = run_fused(q1, codes, scales, sums, M, h1, None, 1, N1, 6)
    # stage 1: the first layer (codes validated, then GEMM + epilogue on them by the oracle)
    out1 = orc.qlinear(to_bits(x), u1, d1, z1, 256, 4, None, 1)
    nat1 = torch.empty(M, K1, dtype=torch.int8, device=DEV)
    B.dvdq_unpack_act_codes(codes, M, K1, q1, nat1)
    from helpers import oracle_y_for_validated_codes
    y1_or = oracle_y_for_validated_codes(nat1.cpu().numpy(), out1, u1, d1, z1, None, 1)
    y1 = Y1.to(torch.float64).cpu().numpy()
    assert np.abs(y1 - y1_or).max() <= Y_MAXNORM_RTOL * np.abs(y1_or).max()
    # stage 2: the fused transform, on the kernel's own bf16 values
    nat2 = torch.empty(M, N1, dtype=torch.int8, device=DEV)
    B.dvdq_unpack_act_codes(cn, M, N1, qn, nat2)
    nat2 = nat2.cpu().numpy()
    check_against_oracle(to_bits(Y1), nat2, sn.cpu().numpy(), Sn.cpu().numpy(), 6)
    # stage 3: the block-wise layer that consumes them
    Y2 = torch.empty(M, N2, dtype=torch.bfloat16, device=DEV)
    B.dvdq_qgemm(cn, sn.reshape(-1), Sn.reshape(-1), M, qn, h2, bias2.to(DEV), 0, Y2)
    assert_device_ok()
    y2_or = bf16_values(orc.combine_grouped(nat2.astype(np.int32), u2, z2, sn.cpu().numpy(), d2, G, to_bits(bias2), 0))
    y2 = Y2.to(torch.float64).cpu().numpy()
    assert np.abs(y2 - y2_or).max() <= Y_MAXNORM_RTOL * np.abs(y2_or).max()
    # end to end against the oracle's own chain (reported, loosely gated: tie flips in either transform move whole rows)
    out2 = orc.qlinear_grouped(out1["y"], u2, d2, z2, G, 6, G, to_bits(bias2), 0)
    rel = np.linalg.norm(y2 - bf16_values(out2["y"])) / np.linalg.norm(bf16_values(out2["y"]))
    assert rel < 0.05, rel


def test_fused_options_are_validated():
    M, K, N = 64, 256, 256
    wl = W.WORKLOADS["tiny"]
    u, d, z = W.make_weight_codes(wl.layers[0], seed=0, device=DEV)
    blob = torch.empty(B.dvdq_weight_blob_bytes(N, K), dtype=torch.uint8, device=DEV)
    w = B.dvdq_pack_weights(u, d, z, 256, blob)
    x = W.make_activations(wl, K, M=M, device=DEV)
    q, codes, scales, sums = first_stage(x, 4, 256)
    cn = torch.empty(M * N, dtype=torch.uint8, device=DEV)
    sn = torch.empty(M, dtype=torch.float32, device=DEV)
    Sn = torch.empty(M, dtype=torch.int32, device=DEV)
    for bad in (B.ActQuant(6, 128, 256, 8), B.ActQuant(6, 256, 1024, 8), B.ActQuant(6, 256, 256, 0), B.ActQuant(6, 256, 0, 8)):
        with pytest.raises(B.DvdqError) as e:
            B.dvdq_qgemm_fused_rq(codes, scales, sums, M, q, w, None, 0, bad, cn, sn, Sn)
        assert e.value.status in (B.ERR_UNSUPPORTED, B.ERR_SHAPE)
    # the first layer must have per-token scales
    with pytest.raises(B.DvdqError) as e:
        B.dvdq_qgemm_fused_rq(codes, scales, sums, M, B.ActQuant(4, 256, 256, 8), w, None, 0, B.ActQuant(6, 256, 256, 8), cn, sn, Sn)
    assert e.value.status == B.ERR_UNSUPPORTED


def test_full_size_fused_chain_on_sampled_rows():
    """The FFN chain at its full token count, fused: sampled rows of every stage against the oracle."""
    wl = W.WORKLOADS["ffn_chain"]
    up, down = wl.layers
    M = wl.M
    x = W.make_activations(wl, up.K, device=DEV)
    u1, d1, z1 = W.make_weight_codes(up, seed=0, device=DEV)
    u2, d2, z2 = W.make_weight_codes(down, seed=1, device=DEV, symmetric=False)
    b1 = torch.empty(B.dvdq_weight_blob_bytes(up.N, up.K), dtype=torch.uint8, device=DEV)
    b2 = torch.empty(B.dvdq_weight_blob_bytes(down.N, down.K), dtype=torch.uint8, device=DEV)
    h1 = B.dvdq_pack_weights(u1, d1, z1, up.rot_block, b1)
    h2 = B.dvdq_pack_weights(u2, d2, z2, G, b2)
    bias2 = W.make_bias(wl, down, device=DEV)
    q1, codes, scales, sums = first_stage(x, up.bits, up.rot_block)
    qn, cn, sn, Sn, Y1 = run_fused(q1, codes, scales, sums, M, h1, None, up.act, up.N, down.bits)
    Y2 = torch.empty(M, down.N, dtype=torch.bfloat16, device=DEV)
    B.dvdq_qgemm(cn, sn.reshape(-1), Sn.reshape(-1), M, qn, h2, bias2, down.act, Y2)
    assert_device_ok()
    rows = W.sample_rows(M, 40, tile=256, seed=5).to(DEV)
    # the fused transform on the sampled rows' own bf16 values
    nat = torch.empty(M, up.N, dtype=torch.int8, device=DEV)
    B.dvdq_unpack_act_codes(cn, M, up.N, qn, nat)
    nat_s = nat[rows].cpu().numpy()
    del nat
    check_against_oracle(to_bits(Y1[rows]), nat_s, sn[rows].cpu().numpy(), Sn[rows].cpu().numpy(), down.bits)
    # the layer that consumes them
    y2_or = bf16_values(orc.combine_grouped(nat_s.astype(np.int32), u2.cpu().numpy(), z2.cpu().numpy(), sn[rows].cpu().numpy(),
                                            d2.cpu().numpy(), G, to_bits(bias2), down.act))
    y2 = Y2[rows].to(torch.float64).cpu().numpy()
    assert np.abs(y2 - y2_or).max() <= Y_MAXNORM_RTOL * np.abs(y2_or).max()
    assert bool(torch.isfinite(Y2).all())
    # and the first stage's bf16 values are the unfused kernel's, bit for bit, on a slice of rows
    Y_ref = torch.empty(4096, up.N, dtype=torch.bfloat16, device=DEV)
    B.dvdq_qgemm(codes[: 4096 * up.K], scales[:4096], sums[:4096], 4096, q1, h1, None, up.act, Y_ref)
    assert torch.equal(Y_ref, Y1[:4096])
