"""Activation codes kept one int8 per code (container_bits = 8) for 4- and 6-bit quantizers: the
same codes, scales and outputs as the packed layout, through the GEMM that takes the activation
operand from shared memory as TMA wrote it."""
import numpy as np
import pytest
import torch

from oracle import dvdq_oracle as orc
from paper_2505_18663_b200 import binding as B

from helpers import (act_quant, bf16_values, check_codes_against_oracle, gpu_pack_codes, gpu_pack_weights,
                     gpu_rotate_quantize, oracle_y_for_validated_codes, to_bits)

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
    x[:, torch.randperm(K, generator=g)[:outliers]] *= gain
    return x.to(torch.bfloat16)


def synth_w(N, K, seed, mode):
    g = torch.Generator().manual_seed(seed)
    w = torch.randn(N, K, generator=g) * 0.02
    if mode == "minmax":
        w += 0.004 * torch.randn(N, 1, generator=g)
    return w.to(torch.bfloat16)


def test_size_queries():
    assert B.dvdq_act_codes_bytes_q(1000, 3072, B.ActQuant(4, 1024, 0, 0)) == 1000 * 1536
    assert B.dvdq_act_codes_bytes_q(1000, 3072, B.ActQuant(4, 1024, 0, 8)) == 1000 * 3072
    assert B.dvdq_act_codes_bytes_q(1000, 3072, B.ActQuant(6, 1024, 0, 8)) == 1000 * 3072
    assert B.dvdq_act_codes_bytes_q(1000, 3072, B.ActQuant(4, 1024, 0, 6)) == 0  # no such container


@pytest.mark.parametrize("bits", [4, 6])
@pytest.mark.parametrize("M,K,Bk", [(300, 3072, 1024), (257, 1536, 512), (65, 320, 64), (130, 8960, 256)])
def test_rotate_quantize_into_bytes_matches_oracle_and_packed_layout(M, K, Bk, bits):
    x = synth_x(M, K, seed=M + K + bits)
    codes_or, s64, s32, xt = orc.rotate_quantize(to_bits(x), Bk, bits)
    _, scales, sums, nat = gpu_rotate_quantize(x.to(DEV), bits, Bk, container=8)
    _, scales_p, sums_p, nat_p = gpu_rotate_quantize(x.to(DEV), bits, Bk)
    assert_device_ok()
    s = scales.cpu().numpy().astype(np.float64)
    assert np.all(np.abs(s - s64) <= SCALE_RTOL * s64)
    nat = nat.cpu().numpy()
    lim = 2 ** (bits - 1)
    assert nat.min() >= -lim and nat.max() <= lim - 1
    check_codes_against_oracle(nat, codes_or, xt, s64)
    assert np.array_equal(sums.cpu().numpy(), nat.astype(np.int64).sum(axis=1))
    # the container changes where a code is stored, not the code
    assert torch.equal(nat_p.cpu(), torch.from_numpy(nat)) and torch.equal(scales, scales_p) and torch.equal(sums, sums_p)


CASES = [
    # M, N, K, B, bits, weight mode: M and N tails (N against the 256-wide tile), odd and even numbers of k-blocks, z != 8
    (1, 8, 64, 64, 6, "minmax"),
    (256, 256, 256, 256, 4, "symmetric"),
    (130, 264, 320, 64, 4, "minmax"),
    (300, 520, 1536, 512, 6, "symmetric"),
    (257, 776, 3072, 1024, 4, "minmax"),
    (129, 256, 8960, 256, 6, "minmax"),
]


@pytest.mark.parametrize("M,N,K,Bk,bits,mode", CASES)
def test_int32_accumulators_are_bit_exact(M, N, K, Bk, bits, mode):
    x = synth_x(M, K, seed=M + N)
    u, d, z = orc.prepare_weights(to_bits(synth_w(N, K, M + N + 1, mode)), Bk, mode)
    codes, s64, s32, xt = orc.rotate_quantize(to_bits(x), Bk, bits)
    w, blob = gpu_pack_weights(u, d, z, Bk)
    packed, sums = gpu_pack_codes(codes, bits, Bk, container=8)
    acc = torch.full((M, N), 12345, dtype=torch.int32, device=DEV)
    B.dvdq_qgemm_int32(packed, sums, M, act_quant(bits, Bk, 8), w, acc)
    assert_device_ok()
    assert np.array_equal(acc.cpu().numpy(), orc.int_gemm(codes, u, z))


@pytest.mark.parametrize("act", [0, 1])
@pytest.mark.parametrize("M,N,K,Bk,bits,mode", CASES[2:5])
def test_qlinear_matches_oracle_and_packed_layout(M, N, K, Bk, bits, mode, act):
    x = synth_x(M, K, seed=7 * M + N)
    u, d, z = orc.prepare_weights(to_bits(synth_w(N, K, M + N + 2, mode)), Bk, mode)
    bias = (torch.randn(N, generator=torch.Generator().manual_seed(N)) * 0.05).to(torch.bfloat16)
    out = orc.qlinear(to_bits(x), u, d, z, Bk, bits, to_bits(bias), act)
    w, blob = gpu_pack_weights(u, d, z, Bk)
    ys = []
    for container in (8, 0):
        q = act_quant(bits, Bk, container)
        ws = torch.empty(B.dvdq_qlinear_workspace_bytes(M, K, q), dtype=torch.uint8, device=DEV)
        Y = torch.zeros(M, N + 8, dtype=torch.bfloat16, device=DEV)[:, :N]
        B.dvdq_qlinear(x.to(DEV), q, w, bias.to(DEV), act, Y, ws)
        nat = torch.empty(M, K, dtype=torch.int8, device=DEV)
        B.dvdq_unpack_act_codes(ws, M, K, q, nat)
        assert_device_ok()
        ys.append(Y.clone())
        if container == 8:
            y_or = oracle_y_for_validated_codes(nat.cpu().numpy(), out, u, d, z, to_bits(bias), act)
            y = Y.to(torch.float64).cpu().numpy()
            assert np.abs(y - y_or).max() <= Y_MAXNORM_RTOL * np.abs(y_or).max()
    # same integers, and the epilogues differ only by exact powers of two: identical outputs
    assert torch.equal(ys[0], ys[1])


def test_empty_input_is_a_no_op():
    q = act_quant(4, 256, 8)
    x = torch.empty(0, 256, dtype=torch.bfloat16, device=DEV)
    one = torch.zeros(256, dtype=torch.uint8, device=DEV)
    B.dvdq_rotate_quantize(x, q, one, torch.zeros(1, device=DEV), torch.zeros(1, dtype=torch.int32, device=DEV))
    assert_device_ok()
    assert B.dvdq_act_codes_bytes_q(0, 256, q) == 0


@pytest.mark.parametrize("bits", [4, 6, 8])
def test_int32_accumulators_at_code_extremes_and_the_largest_k(bits):
    # every product at its largest magnitude, K at the library's limit: |acc| = K * 2^(bits-1) * 15,
    # and 16 x that inside the tensor core (the widened weights are 16 (u - 8)): still below 2^31
    M, N, K = 128, 264, 16384
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
    packed, sums = gpu_pack_codes(codes, bits, 1024, container=8)
    acc = torch.zeros(M, N, dtype=torch.int32, device=DEV)
    B.dvdq_qgemm_int32(packed, sums, M, act_quant(bits, 1024, 8), w, acc)
    assert_device_ok()
    assert np.array_equal(acc.cpu().numpy(), acc_or)


@pytest.mark.parametrize("workload,layer_idx", [("hunyuan", 3), ("hunyuan", 0), ("wan1p3b", 1), ("ffn_chain", 0)])
def test_full_size_outputs_repeat_and_agree_across_layouts(workload, layer_idx):
    """At the benchmark's token counts every launch must give the same bits, in both code layouts
    (long K, 6-bit codes, the eight-epilogue-warp variant with and without GELU): a stage handed
    back to its producer too early, or read too early, shows here as a few columns of one tile."""
    from paper_2505_18663_b200 import workloads as W
    wl = W.WORKLOADS[workload]
    layer = wl.layers[layer_idx]
    M = min(wl.M, 65536)
    x = W.make_activations(wl, layer.K, device=DEV)[:M]
    u, d, z = W.make_weight_codes(layer, seed=layer_idx, device=DEV, symmetric=False)
    blob = torch.empty(B.dvdq_weight_blob_bytes(layer.N, layer.K), dtype=torch.uint8, device=DEV)
    w = B.dvdq_pack_weights(u, d, z, layer.rot_block, blob)
    bias = W.make_bias(wl, layer, device=DEV)
    ref = None
    for container in (0, 8):
        q = act_quant(layer.bits, layer.rot_block, container)
        ws = torch.empty(B.dvdq_qlinear_workspace_bytes(M, layer.K, q), dtype=torch.uint8, device=DEV)
        for rep in range(6):
            Y = torch.empty(M, layer.N, dtype=torch.bfloat16, device=DEV)
            B.dvdq_qlinear(x, q, w, bias, layer.act, Y, ws)
            assert_device_ok()
            if ref is None:
                ref = Y
            else:
                bad = int((Y != ref).sum())
                assert bad == 0, f"container_bits={container}, launch {rep}: {bad} outputs differ"
