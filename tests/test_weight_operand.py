"""The GEMM's weight operand written once by dvdq_widen_weights (one int8 per 4-bit code, read by TMA)
instead of widened by every output tile for itself: the integer contraction of Eq. 10 sees the same
operand bytes either way, so outputs must be bit-identical to those of the plain handle, and they are
checked against the CPU oracle as well."""
import numpy as np
import pytest
import torch

from oracle import dvdq_oracle as orc
from paper_2505_18663_b200 import binding as B

from helpers import act_quant, to_bits, bf16_values, gpu_pack_weights, gpu_pack_codes

pytestmark = pytest.mark.gpu
DEV = "cuda"

CASES = [
    # M, N, K, B, bits, weight mode, GELU: tails in M and N, K not a multiple of 128 / 256, short and long K
    (130, 264, 320, 64, 4, "minmax", 0),
    (300, 512, 1536, 512, 6, "symmetric", 1),
    (257, 776, 3072, 1024, 4, "minmax", 0),
    (513, 520, 3072, 1024, 4, "symmetric", 1),
    (129, 256, 8960, 256, 6, "minmax", 0),
    (300, 520, 1536, 512, 8, "minmax", 1),
    (600, 1032, 12288, 1024, 4, "minmax", 0),
]


def synth(M, N, K, Bk, bits, mode, seed):
    g = torch.Generator().manual_seed(seed)
    x = torch.randn(M, K, generator=g).to(torch.bfloat16)
    x[:, 5] *= 20.0
    wb = (torch.randn(N, K, generator=g) * 0.02 + (0.004 * torch.randn(N, 1, generator=g) if mode == "minmax" else 0.0)).to(torch.bfloat16)
    u, d, z = orc.prepare_weights(to_bits(wb), Bk, mode)
    codes, s64, s32, xt = orc.rotate_quantize(to_bits(x), Bk, bits)
    return u, d, z, codes, s32


@pytest.mark.parametrize("container", [0, 8])
@pytest.mark.parametrize("M,N,K,Bk,bits,mode,act", CASES)
def test_gemm_with_widened_operand_is_bit_identical_and_matches_oracle(M, N, K, Bk, bits, mode, act, container):
    u, d, z, codes, s32 = synth(M, N, K, Bk, bits, mode, seed=M + N + K)
    bias = (torch.randn(N, generator=torch.Generator().manual_seed(N)) * 0.05).to(torch.bfloat16)
    y_or = bf16_values(orc.epilogue(orc.int_gemm(codes, u, z), s32, d, to_bits(bias), act))
    w, blob = gpu_pack_weights(u, d, z, Bk)
    assert w.operand is None and w.operand_bytes == 0
    assert B.dvdq_weight_operand_bytes(N, K) == N * K
    operand = torch.full((N * K + 256,), 0x5A, dtype=torch.uint8, device=DEV)
    ww = B.dvdq_widen_weights(w, operand[:N * K])
    assert ww.operand == operand.data_ptr() and ww.operand_bytes == N * K and ww.blob == w.blob
    assert bool((operand[N * K:] == 0x5A).all())                               # nothing past N * K bytes
    # each byte holds 16 x (u - 8), whatever the order along K: the multiset per row fixes it
    got = operand[:N * K].view(torch.int8).view(N, K).to(torch.int32).sort(dim=1).values.cpu().numpy()
    assert np.array_equal(got, np.sort(16 * (u.astype(np.int32) - 8), axis=1))
    q = act_quant(bits, Bk, container)
    packed, sums = gpu_pack_codes(codes, bits, Bk, container=container)
    s_dev = torch.from_numpy(s32).to(DEV)
    Y0 = torch.zeros(M, N, dtype=torch.bfloat16, device=DEV)
    Y1 = torch.zeros(M, N + 8, dtype=torch.bfloat16, device=DEV)[:, :N]
    B.dvdq_qgemm(packed, s_dev, sums, M, q, w, bias.to(DEV), act, Y0)
    B.dvdq_qgemm(packed, s_dev, sums, M, q, ww, bias.to(DEV), act, Y1)
    torch.cuda.synchronize()
    assert B.dvdq_last_device_status()[0] == 0
    assert torch.equal(Y0, Y1)
    y = Y1.to(torch.float64).cpu().numpy()
    y0_or = bf16_values(orc.epilogue(orc.int_gemm(codes, u, z), s32, d, to_bits(bias), 0))
    ulp = np.maximum(np.abs(y0_or), 2.0 ** -100) * 2.0 ** -7
    assert np.all(np.abs(y - y_or) <= (ulp if act == 0 else 3 * ulp))           # fp32 vs fp64 epilogue: one bf16 ulp
    assert np.mean(y != y_or) < 0.02


def test_widen_weights_argument_checks():
    N, K = 64, 256
    u = np.random.default_rng(0).integers(0, 16, (N, K)).astype(np.uint8)
    w, blob = gpu_pack_weights(u, np.ones(N, np.float32), np.full(N, 8, np.int32), 256)
    small = torch.empty(N * K - 1, dtype=torch.uint8, device=DEV)
    with pytest.raises(B.DvdqError):
        B.dvdq_widen_weights(w, small)
    odd = torch.empty(N * K + 16, dtype=torch.uint8, device=DEV)[16:]
    with pytest.raises(B.DvdqError):
        B.dvdq_widen_weights(w, odd)
    # a handle whose operand size does not fit its shape is refused by the GEMM
    ok = torch.empty(N * K, dtype=torch.uint8, device=DEV)
    ww = B.dvdq_widen_weights(w, ok)
    ww.operand_bytes = N * K - 64
    q = act_quant(4, 256, 8)
    codes = torch.zeros(8 * K, dtype=torch.uint8, device=DEV)
    with pytest.raises(B.DvdqError):
        B.dvdq_qgemm(codes, torch.ones(8, device=DEV), torch.zeros(8, dtype=torch.int32, device=DEV), 8, q, ww, None, 0,
                     torch.empty(8, N, dtype=torch.bfloat16, device=DEV))


def test_qlinear_with_room_for_the_operand_gives_the_same_bits():
    M, N, K, Bk, bits = 1300, 520, 3072, 1024, 4
    g = torch.Generator().manual_seed(11)
    x = torch.randn(M, K, generator=g).to(torch.bfloat16).to(DEV)
    u = np.random.default_rng(1).integers(0, 16, (N, K)).astype(np.uint8)
    w, blob = gpu_pack_weights(u, np.full(N, 0.01, np.float32), np.full(N, 7, np.int32), Bk)
    for container in (0, 8):
        q = act_quant(bits, Bk, container)
        base = B.dvdq_qlinear_workspace_bytes(M, K, q)
        ws_small = torch.empty(base, dtype=torch.uint8, device=DEV)
        ws_large = torch.full((base + B.dvdq_weight_operand_bytes(N, K) + 256,), 0xEE, dtype=torch.uint8, device=DEV)
        Y0 = torch.empty(M, N, dtype=torch.bfloat16, device=DEV)
        Y1 = torch.empty(M, N, dtype=torch.bfloat16, device=DEV)
        B.dvdq_qlinear(x, q, w, None, 1, Y0, ws_small)
        B.dvdq_qlinear(x, q, w, None, 1, Y1, ws_large)
        torch.cuda.synchronize()
        assert B.dvdq_last_device_status()[0] == 0
        assert torch.equal(Y0, Y1)
        # the operand was written behind the codes: 16 x (u - 8) in some order along K
        off = (base + 255) // 256 * 256
        got = ws_large[off:off + N * K].view(torch.int8).view(N, K).to(torch.int32).sort(dim=1).values.cpu().numpy()
        assert np.array_equal(got, np.sort(16 * (u.astype(np.int32) - 8), axis=1))


def test_widen_weights_beyond_one_pass_of_the_grid():
    # more 16-byte pieces than one pass of the widening kernel's grid covers, and the exact K order:
    # word by word, the four even-numbered codes of eight, then the four odd-numbered ones
    N, K = 5120, 8192
    u = torch.randint(0, 16, (N, K), dtype=torch.uint8, device=DEV, generator=torch.Generator(DEV).manual_seed(5))
    blob = torch.empty(B.dvdq_weight_blob_bytes(N, K), dtype=torch.uint8, device=DEV)
    w = B.dvdq_pack_weights(u, torch.ones(N, device=DEV), torch.full((N,), 8, dtype=torch.int32, device=DEV), 1024, blob)
    operand = torch.empty(N * K, dtype=torch.uint8, device=DEV)
    B.dvdq_widen_weights(w, operand)
    got = operand.view(torch.int8).view(N, K // 8, 8).to(torch.int32)
    want = 16 * (u.view(N, K // 8, 8).to(torch.int32) - 8)[:, :, [0, 2, 4, 6, 1, 3, 5, 7]]
    assert torch.equal(got, want)
