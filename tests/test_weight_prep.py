"""Offline weight preparation on the GPU (Eq. 10, W^ = Quant(W H)) against the CPU oracle:
the rotation W~ = W R along K and the symmetric 4-bit quantizer that writes a blob, so that
bf16 weights reach a quantized layer without any CPU step."""
import numpy as np
import pytest
import torch

from oracle import dvdq_oracle as orc
from paper_2505_18663_b200 import binding as B

from helpers import act_quant, to_bits, oracle_y_for_validated_codes

pytestmark = pytest.mark.gpu
DEV = "cuda"


def synth_w(N, K, seed):
    g = torch.Generator().manual_seed(seed)
    return (torch.randn(N, K, generator=g) * 0.02).to(torch.bfloat16)


ROT_CASES = [(24, 256, 256), (17, 1536, 512), (9, 3072, 1024), (5, 8960, 256), (8, 640, 128), (8, 320, 64),
             (3, 1024, 0), (6, 12288, 4096), (7, 4096, 2048), (4, 16384, 1024)]


@pytest.mark.parametrize("N,K,Bk", ROT_CASES)
def test_rotate_weights_matches_the_dense_fp64_rotation(N, K, Bk):
    w = synth_w(N, K, N + K)
    w[N // 2] = 0
    ref = orc.rotate(to_bits(w), Bk)
    out = torch.empty(N, K, dtype=torch.float32, device=DEV)
    B.dvdq_rotate_weights(w.to(DEV), Bk, out)
    got = out.cpu().numpy()
    ref32 = ref.astype(np.float32)
    log2b = Bk.bit_length() - 1 if Bk else 0
    if log2b % 2 == 0:
        # 1/sqrt(B) is a power of two: fp64 butterflies of bf16 values are exact, so is the oracle's sum
        assert np.array_equal(got, ref32)
    else:
        # one fp64 rounding of the irrational factor on either side: equal after the cast, or one fp32 ulp apart
        assert np.abs(got.astype(np.float64) - ref).max() <= 2.0 ** -23 * np.abs(ref).max()
        assert (got != ref32).mean() <= 1e-4


def test_rotate_weights_strided_rows_and_empty_input():
    N, K, Bk = 16, 512, 256
    big = torch.zeros(N, K + 64, dtype=torch.bfloat16)
    big[:, :K] = synth_w(N, K, 3)
    a = torch.empty(N, K, dtype=torch.float32, device=DEV)
    b = torch.empty(N, K, dtype=torch.float32, device=DEV)
    B.dvdq_rotate_weights(big.to(DEV)[:, :K], Bk, a)
    B.dvdq_rotate_weights(big[:, :K].contiguous().to(DEV), Bk, b)
    assert torch.equal(a, b)
    B.dvdq_rotate_weights(torch.empty(0, K, dtype=torch.bfloat16, device=DEV), Bk, torch.empty(0, K, dtype=torch.float32, device=DEV))


@pytest.mark.parametrize("N,K,Bk", [(264, 320, 64), (40, 1536, 512), (24, 3072, 1024), (16, 8960, 256), (8, 12288, 4096)])
def test_quantize_weights_symmetric_matches_oracle(N, K, Bk):
    w = synth_w(N, K, 7 * N + K)
    w[1] = 0                                                     # an all-zero output channel
    u_or, d_or, z_or = orc.prepare_weights(to_bits(w), Bk, "symmetric")
    blob = torch.zeros(B.dvdq_weight_blob_bytes(N, K), dtype=torch.uint8, device=DEV)   # zeros: the padding between sections is never written
    h = B.dvdq_quantize_weights_symmetric(w.to(DEV), Bk, blob)
    assert (h.N, h.K, h.rot_block, h.blob_bytes) == (N, K, Bk, blob.numel())
    u = torch.empty(N, K, dtype=torch.uint8, device=DEV)
    d = torch.empty(N, dtype=torch.float32, device=DEV)
    z = torch.empty(N, dtype=torch.int32, device=DEV)
    B.dvdq_unpack_weights(h, u, d, z)
    assert np.array_equal(z.cpu().numpy(), z_or) and np.all(z_or == 8)
    assert np.array_equal(d.cpu().numpy(), d_or)                 # fp64 absmax / 7, one rounding to fp32
    log2b = Bk.bit_length() - 1
    if log2b % 2 == 0:
        assert np.array_equal(u.cpu().numpy(), u_or)
    else:
        assert (u.cpu().numpy() != u_or).mean() <= 1e-5          # a quotient within one fp64 ulp of a tie
    # the blob is byte for byte what dvdq_pack_weights writes for the same codes
    blob2 = torch.zeros_like(blob)
    B.dvdq_pack_weights(u, d, z, Bk, blob2)
    assert torch.equal(blob, blob2)


def test_bf16_weights_to_quantized_layer_without_a_cpu_step():
    """dvdq_quantize_weights_symmetric -> dvdq_qlinear, against the oracle's whole path."""
    M, N, K, Bk, bits = 200, 264, 3072, 1024, 4
    g = torch.Generator().manual_seed(5)
    x = torch.randn(M, K, generator=g)
    x[:, 7] *= 25.0
    x = x.to(torch.bfloat16)
    w = synth_w(N, K, 9)
    blob = torch.empty(B.dvdq_weight_blob_bytes(N, K), dtype=torch.uint8, device=DEV)
    h = B.dvdq_quantize_weights_symmetric(w.to(DEV), Bk, blob)
    q = act_quant(bits, Bk)
    ws = torch.empty(B.dvdq_qlinear_workspace_bytes(M, K, q), dtype=torch.uint8, device=DEV)
    Y = torch.empty(M, N, dtype=torch.bfloat16, device=DEV)
    B.dvdq_qlinear(x.to(DEV), q, h, None, 0, Y, ws)
    nat = torch.empty(M, K, dtype=torch.int8, device=DEV)
    B.dvdq_unpack_act_codes(ws, M, K, q, nat)
    u, d, z = orc.prepare_weights(to_bits(w), Bk, "symmetric")
    out = orc.qlinear(to_bits(x), u, d, z, Bk, bits)
    y_or = oracle_y_for_validated_codes(nat.cpu().numpy(), out, u, d, z)
    y = Y.to(torch.float64).cpu().numpy()
    assert np.abs(y - y_or).max() <= 4e-3 * np.abs(y_or).max()
    exact = x.to(torch.float64).numpy() @ w.to(torch.float64).numpy().T
    assert np.linalg.norm(y - exact) / np.linalg.norm(exact) < 0.5
