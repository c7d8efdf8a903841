"""Block-wise activation scales (one scale per token and per group of 128, 256 or 1024 rotated
channels; the block-wise variant of Sec. 3.2's last paragraph): the CUDA path against the oracle's
block-wise quantizer and layer, for every group size the library builds."""
import numpy as np
import pytest
import torch

from oracle import dvdq_oracle as orc
from paper_2505_18663_b200 import binding as B

from helpers import bf16_values, check_codes_against_oracle, gpu_pack_weights, to_bits

pytestmark = pytest.mark.gpu
DEV = "cuda"
GROUPS = [1024, 256, 128]   # the groups the library builds: whole k-blocks of the GEMM
SCALE_RTOL = 1e-6
Y_MAXNORM_RTOL = 4e-3


def assert_device_ok():
    status, detail = B.dvdq_last_device_status()
    assert status == B.OK, f"device status {status} ({B.status_string(status)}), wait id {detail}"


def synth_x(M, K, seed, outliers=4, gain=20.0):
    g = torch.Generator().manual_seed(seed)
    x = torch.randn(M, K, generator=g)
    # tokens differ in size and the outlier channels sit in some blocks only: the case block-wise
    # scales are for
    x *= torch.exp(torch.randn(M, 1, generator=g))
    if outliers:
        x[:, torch.randperm(K, generator=g)[:outliers]] *= gain
    return x.to(torch.bfloat16)


def synth_w(N, K, seed, mode):
    g = torch.Generator().manual_seed(seed)
    w = torch.randn(N, K, generator=g) * 0.02
    if mode == "minmax":
        w += 0.004 * torch.randn(N, 1, generator=g)
    return w.to(torch.bfloat16)


def gpu_rotate_quantize_blockwise(x_dev, bits, Bk, G):
    M, K = x_dev.shape
    q = B.ActQuant(bits, Bk, G)
    n = B.dvdq_act_scales_count(M, K, q)
    assert n == M * (K // G)
    codes = torch.empty(B.dvdq_act_codes_bytes(M, K, bits), dtype=torch.uint8, device=DEV)
    scales = torch.full((n,), -1.0, dtype=torch.float32, device=DEV)
    sums = torch.full((n,), 123456, dtype=torch.int32, device=DEV)
    B.dvdq_rotate_quantize(x_dev, q, codes, scales, sums)
    nat = torch.empty(M, K, dtype=torch.int8, device=DEV)
    B.dvdq_unpack_act_codes(codes, M, K, q, nat)
    torch.cuda.synchronize()
    return codes, scales.view(M, K // G), sums.view(M, K // G), nat


def check_blockwise_codes(nat, codes_or, xt, s64, G, min_agree=0.9999):
    # the agreement bar is over the whole tensor (one legitimate tie flip in a 77 x 128 slice is
    # already 1e-4 of it); that every mismatch is +-1 on a tie is checked group by group, each
    # against its own scale
    assert (nat.astype(np.int32) == codes_or).mean() >= min_agree
    for g in range(codes_or.shape[1] // G):
        sl = slice(g * G, (g + 1) * G)
        check_codes_against_oracle(nat[:, sl], codes_or[:, sl], xt[:, sl], s64[:, g], min_agree=0.0)


@pytest.mark.parametrize("G", GROUPS)
@pytest.mark.parametrize("bits", [4, 6, 8])
@pytest.mark.parametrize("M,K,Bk", [(300, 3072, 256), (257, 2048, 1024), (65, 1024, 64), (130, 5120, 128),
                                    (77, 1536, 512), (41, 8960, 256), (36, 4096, 4096), (50, 1024, 0)])
def test_rotate_quantize_blockwise_matches_oracle(M, K, Bk, bits, G):
    if K % G:
        pytest.skip("K is not a multiple of the group")
    x = synth_x(M, K, seed=M + K + bits)
    x[M // 3] = 0                                               # an all-zero token: every group scale 0
    xt = orc.rotate(to_bits(x), Bk)
    codes_or, s64, s32 = orc.act_quantize_grouped(xt, bits, G)
    _, scales, sums, nat = gpu_rotate_quantize_blockwise(x.to(DEV), bits, Bk, G)
    assert_device_ok()
    s = scales.cpu().numpy().astype(np.float64)
    assert np.all(np.abs(s - s64) <= SCALE_RTOL * s64)
    nat = nat.cpu().numpy()
    assert np.all(nat[M // 3] == 0) and np.all(s[M // 3] == 0)
    # Without a rotation x~ is a bf16 value and the group's absmax another: quotients x~ qmax / absmax
    # that are EXACT half-integers are common (a few per ten thousand elements with short groups).
    # The GPU rounds the exact quotient half to even; the oracle's two fp64 roundings (s = a / qmax,
    # then x~ / s) land on either side of it.  Both codes are valid and the check below still
    # requires every mismatch to be +-1 on such a tie, so only the agreement bar is lower there.
    check_blockwise_codes(nat, codes_or, xt, s64, G, min_agree=0.9999 if Bk else 0.999)
    # the sums belong to the codes that were written, block by block, exactly
    assert np.array_equal(sums.cpu().numpy(), nat.astype(np.int64).reshape(M, K // G, G).sum(axis=2))


def test_blockwise_equals_per_token_when_there_is_one_block():
    M, K, bits, Bk = 200, 1024, 4, 256
    x = synth_x(M, K, seed=5).to(DEV)
    pc, ps, pS, pn = gpu_rotate_quantize_blockwise(x, bits, Bk, 1024)
    q = B.ActQuant(bits, Bk, 0)
    codes = torch.empty_like(pc)
    scales = torch.empty(M, dtype=torch.float32, device=DEV)
    sums = torch.empty(M, dtype=torch.int32, device=DEV)
    B.dvdq_rotate_quantize(x, q, codes, scales, sums)
    torch.cuda.synchronize()
    assert torch.equal(codes, pc) and torch.equal(scales, ps.view(-1)) and torch.equal(sums, pS.view(-1))


LAYER_CASES = [
    # M, N, K, B, bits, weight mode: M and N tails (N tail against the 128-wide tile), 1 to 40 groups, z != 8
    (257, 392, 3072, 256, 4, "minmax"),
    (300, 128, 1024, 1024, 4, "symmetric"),
    (130, 520, 2048, 128, 6, "minmax"),
    (513, 256, 5120, 512, 8, "minmax"),
]


def pack_blockwise(codes_np, bits, Bk, G):
    M, K = codes_np.shape
    q = B.ActQuant(bits, Bk, G)
    nat = torch.from_numpy(codes_np.astype(np.int8)).to(DEV)
    packed = torch.empty(B.dvdq_act_codes_bytes(M, K, bits), dtype=torch.uint8, device=DEV)
    sums = torch.empty(M * (K // G), dtype=torch.int32, device=DEV)
    B.dvdq_pack_act_codes(nat, q, packed, sums)
    return packed, sums, q


@pytest.mark.parametrize("G", GROUPS)
@pytest.mark.parametrize("act", [0, 1])
@pytest.mark.parametrize("M,N,K,Bk,bits,mode", LAYER_CASES)
def test_qgemm_blockwise_on_oracle_codes_and_scales(M, N, K, Bk, bits, mode, act, G):
    x = synth_x(M, K, seed=3 * M + N)
    u, d, z = orc.prepare_weights(to_bits(synth_w(N, K, M + N, mode)), Bk, mode)
    codes, s64, s32 = orc.act_quantize_grouped(orc.rotate(to_bits(x), Bk), bits, G)
    bias = (torch.randn(N, generator=torch.Generator().manual_seed(N)) * 0.05).to(torch.bfloat16)
    y_or = bf16_values(orc.combine_grouped(codes, u, z, s32, d, G, to_bits(bias), act))
    w, blob = gpu_pack_weights(u, d, z, Bk)
    packed, sums, q = pack_blockwise(codes, bits, Bk, G)
    assert np.array_equal(sums.cpu().numpy().reshape(M, K // G), codes.reshape(M, K // G, G).sum(axis=2))
    Y = torch.zeros(M, N + 8, dtype=torch.bfloat16, device=DEV)[:, :N]
    B.dvdq_qgemm(packed, torch.from_numpy(np.ascontiguousarray(s32)).to(DEV), sums, M, q, w, bias.to(DEV), act, Y)
    assert_device_ok()
    y = Y.to(torch.float64).cpu().numpy()
    assert np.abs(y - y_or).max() <= Y_MAXNORM_RTOL * np.abs(y_or).max()
    # same integer inputs: what differs is fp32 against fp64 in the combination of at most forty
    # group terms -- a few ulp of fp32, far below the bf16 rounding, so nearly every output is equal
    assert np.mean(y != y_or) < 0.02
    # the weight operand written once (dvdq_widen_weights) instead of widened tile by tile: the same bits
    operand = torch.empty(N * K, dtype=torch.uint8, device=DEV)
    Y2 = torch.zeros(M, N, dtype=torch.bfloat16, device=DEV)
    B.dvdq_qgemm(packed, torch.from_numpy(np.ascontiguousarray(s32)).to(DEV), sums, M, q, B.dvdq_widen_weights(w, operand),
                 bias.to(DEV), act, Y2)
    assert_device_ok()
    assert torch.equal(Y, Y2)
    # the int32 output does not depend on the scales: bit-exact against the whole-K integer GEMM
    acc = torch.zeros(M, N, dtype=torch.int32, device=DEV)
    B.dvdq_qgemm_int32(packed, sums, M, q, w, acc)
    assert_device_ok()
    assert np.array_equal(acc.cpu().numpy(), orc.int_gemm(codes, u, z))


@pytest.mark.parametrize("G", GROUPS)
@pytest.mark.parametrize("M,N,K,Bk,bits,mode", LAYER_CASES)
def test_qlinear_blockwise_matches_oracle_end_to_end(M, N, K, Bk, bits, mode, G):
    x = synth_x(M, K, seed=7 * M + N)
    u, d, z = orc.prepare_weights(to_bits(synth_w(N, K, M + N + 1, mode)), Bk, mode)
    out = orc.qlinear_grouped(to_bits(x), u, d, z, Bk, bits, G)
    w, blob = gpu_pack_weights(u, d, z, Bk)
    q = B.ActQuant(bits, Bk, G)
    ws = torch.empty(B.dvdq_qlinear_workspace_bytes(M, K, q), dtype=torch.uint8, device=DEV)
    Y = torch.empty(M, N, dtype=torch.bfloat16, device=DEV)
    B.dvdq_qlinear(x.to(DEV), q, w, None, 0, Y, ws)
    nat = torch.empty(M, K, dtype=torch.int8, device=DEV)
    B.dvdq_unpack_act_codes(ws, M, K, q, nat)
    assert_device_ok()
    nat = nat.cpu().numpy()
    # codes first (equal, or +-1 on a rounding tie), then the rest of the layer on the validated codes
    check_blockwise_codes(nat, out["codes"], out["xt"], out["scale64"], G)
    y_or = bf16_values(orc.combine_grouped(nat.astype(np.int32), u, z, out["scale32"], d, G))
    y = Y.to(torch.float64).cpu().numpy()
    assert np.abs(y - y_or).max() <= Y_MAXNORM_RTOL * np.abs(y_or).max()
    # and the static-scratch entry point takes the same option
    if B.dvdq_qlinear_workspace_bytes(M, K, q) <= B.STATIC_SCRATCH_BYTES:
        Y2 = torch.empty_like(Y)
        B.dvdq_qlinear_static(x.to(DEV), q, w, None, 0, Y2)
        assert_device_ok()
        assert torch.equal(Y, Y2)


@pytest.mark.parametrize("G", GROUPS)
@pytest.mark.parametrize("bits", [4, 6])
def test_blockwise_with_codes_kept_in_bytes_equals_packed(bits, G):
    """container_bits = 8 changes where a code is stored, not the code, the block scales or the output."""
    M, N, K, Bk = 200, 392, 2048, 256
    x = synth_x(M, K, seed=21 + bits).to(DEV)
    u, d, z = orc.prepare_weights(to_bits(synth_w(N, K, 22, "minmax")), Bk, "minmax")
    w, blob = gpu_pack_weights(u, d, z, Bk)
    ys = []
    for container in (0, 8):
        q = B.ActQuant(bits, Bk, G, container)
        ws = torch.empty(B.dvdq_qlinear_workspace_bytes(M, K, q), dtype=torch.uint8, device=DEV)
        Y = torch.empty(M, N, dtype=torch.bfloat16, device=DEV)
        B.dvdq_qlinear(x, q, w, None, 0, Y, ws)
        nat = torch.empty(M, K, dtype=torch.int8, device=DEV)
        B.dvdq_unpack_act_codes(ws, M, K, q, nat)
        assert_device_ok()
        ys.append((Y, nat))
    assert torch.equal(ys[0][1], ys[1][1]) and torch.equal(ys[0][0], ys[1][0])


@pytest.mark.parametrize("G", GROUPS)
def test_blockwise_scales_lower_the_quantization_error(G):
    """What the option is for: with outlier channels confined to one block, the other blocks get a
    finer grid, so the layer output is closer to the unquantized product than with one scale per token."""
    M, N, K, Bk, bits = 256, 256, 4096, 256, 4
    g = torch.Generator().manual_seed(11)
    x = torch.randn(M, K, generator=g)
    x[:, 5:9] *= 30.0                      # all outliers in the first rotation block
    x = x.to(torch.bfloat16)
    wb = synth_w(N, K, 12, "symmetric")
    u, d, z = orc.prepare_weights(to_bits(wb), Bk, "symmetric")
    w, blob = gpu_pack_weights(u, d, z, Bk)
    exact = orc.exact_linear(bf16_values(to_bits(x)), bf16_values(to_bits(wb)))
    errs = []
    for group in (0, G):
        q = B.ActQuant(bits, Bk, group)
        ws = torch.empty(B.dvdq_qlinear_workspace_bytes(M, K, q), dtype=torch.uint8, device=DEV)
        Y = torch.empty(M, N, dtype=torch.bfloat16, device=DEV)
        B.dvdq_qlinear(x.to(DEV), q, w, None, 0, Y, ws)
        assert_device_ok()
        errs.append(np.linalg.norm(Y.to(torch.float64).cpu().numpy() - exact))
    assert errs[1] < 0.85 * errs[0], errs


@pytest.mark.parametrize("G", GROUPS)
@pytest.mark.parametrize("layer_idx", [3, 0])
def test_full_size_blockwise_outputs_repeat_and_agree_across_layouts(layer_idx, G):
    """The benchmark's token count with block-wise scales: every launch gives the same bits, with
    the codes packed and kept in bytes (12 to 96 groups per token on the long layer)."""
    from paper_2505_18663_b200 import workloads as W
    wl = W.WORKLOADS["hunyuan"]
    layer = wl.layers[layer_idx]
    M = wl.M
    x = W.make_activations(wl, layer.K, device=DEV)
    u, d, z = W.make_weight_codes(layer, seed=layer_idx, device=DEV, symmetric=False)
    blob = torch.empty(B.dvdq_weight_blob_bytes(layer.N, layer.K), dtype=torch.uint8, device=DEV)
    w = B.dvdq_pack_weights(u, d, z, layer.rot_block, blob)
    ref = None
    for container in (0, 8):
        q = B.ActQuant(layer.bits, layer.rot_block, G, container)
        ws = torch.empty(B.dvdq_qlinear_workspace_bytes(M, layer.K, q), dtype=torch.uint8, device=DEV)
        for rep in range(4):
            Y = torch.empty(M, layer.N, dtype=torch.bfloat16, device=DEV)
            B.dvdq_qlinear(x, q, w, None, 0, Y, ws)
            assert_device_ok()
            if ref is None:
                ref = Y
            else:
                bad = int((Y != ref).sum())
                assert bad == 0, f"container_bits={container}, launch {rep}: {bad} outputs differ"
