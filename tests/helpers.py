"""Shared helpers of the tests: bf16 <-> raw bits, oracle <-> device plumbing."""
import numpy as np
import torch

from paper_2505_18663_b200 import binding as B


def to_bits(t: torch.Tensor) -> np.ndarray:
    """bf16 tensor (any device) -> numpy uint16 raw bits."""
    return t.detach().to("cpu").to(torch.bfloat16).contiguous().view(torch.int16).numpy().view(np.uint16)


def from_bits(bits: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(bits.view(np.int16).copy()).view(torch.bfloat16)


def bf16_values(bits: np.ndarray) -> np.ndarray:
    return from_bits(bits).to(torch.float64).numpy()


def act_quant(bits: int, rot_block: int, container: int = 0) -> B.ActQuant:
    return B.ActQuant(bits, rot_block, 0, container)


def gpu_rotate_quantize(x_dev: torch.Tensor, bits: int, rot_block: int, container: int = 0):
    """Runs the CUDA transform; returns (packed codes, scales, sums, natural-order int8 codes)."""
    M, K = x_dev.shape
    q = act_quant(bits, rot_block, container)
    codes = torch.empty(max(1, B.dvdq_act_codes_bytes_q(M, K, q)), dtype=torch.uint8, device=x_dev.device)
    scales = torch.empty(max(1, M), dtype=torch.float32, device=x_dev.device)
    sums = torch.empty(max(1, M), dtype=torch.int32, device=x_dev.device)
    B.dvdq_rotate_quantize(x_dev, q, codes, scales, sums)
    nat = torch.empty(M, K, dtype=torch.int8, device=x_dev.device)
    B.dvdq_unpack_act_codes(codes, M, K, q, nat)
    torch.cuda.synchronize()
    return codes, scales[:M], sums[:M], nat


def gpu_pack_weights(u: np.ndarray, delta: np.ndarray, z: np.ndarray, rot_block: int, device="cuda"):
    N, K = u.shape
    blob = torch.empty(B.dvdq_weight_blob_bytes(N, K), dtype=torch.uint8, device=device)
    w = B.dvdq_pack_weights(torch.from_numpy(u).to(device), torch.from_numpy(delta).to(device),
                            torch.from_numpy(z).to(device), rot_block, blob)
    return w, blob


def gpu_pack_codes(codes_np: np.ndarray, bits: int, rot_block: int, device="cuda", container: int = 0):
    M, K = codes_np.shape
    q = act_quant(bits, rot_block, container)
    nat = torch.from_numpy(codes_np.astype(np.int8)).to(device)
    packed = torch.empty(B.dvdq_act_codes_bytes_q(M, K, q), dtype=torch.uint8, device=device)
    sums = torch.empty(M, dtype=torch.int32, device=device)
    B.dvdq_pack_act_codes(nat, q, packed, sums)
    return packed, sums


def check_codes_against_oracle(nat_gpu: np.ndarray, codes_or: np.ndarray, xt: np.ndarray, s64: np.ndarray,
                               min_agree: float = 0.9999):
    """Codes agree on >= 99.99 % of the elements; every mismatch is +-1 and sits on a rounding
    tie: x~/s within 1e-4 of the half-way point between the two codes."""
    diff = nat_gpu.astype(np.int32) - codes_or
    mism = diff != 0
    frac = 1.0 - mism.mean() if mism.size else 1.0
    assert frac >= min_agree, f"only {frac:.6f} of the codes agree"
    if mism.any():
        assert np.abs(diff[mism]).max() == 1
        i, k = np.nonzero(mism)
        ratio = xt[i, k] / s64[i]
        mid = (nat_gpu[i, k].astype(np.float64) + codes_or[i, k]) / 2.0
        assert np.abs(ratio - mid).max() < 1e-4, np.abs(ratio - mid).max()
    return frac


def oracle_y_for_validated_codes(nat_gpu: np.ndarray, out: dict, u, d, z, bias_bits=None, act: int = 0) -> np.ndarray:
    """bf16 values the oracle gives for the layer output when its quantizer takes the GPU's side
    on rounding ties.  A code whose x~/s sits on a half-way point has two correct values (fp32
    and fp64 transforms land on different sides of it), and one flipped code moves a whole output
    row by s_i * Delta_n * (u - z): on a token with a large scale that alone can exceed the
    output tolerance.  So the codes are first validated (equal, or +-1 on a tie: see
    check_codes_against_oracle), and the rest of the path -- integer GEMM and epilogue, where
    nothing is ambiguous -- is then evaluated by the oracle on the validated codes."""
    from oracle import dvdq_oracle as orc
    check_codes_against_oracle(nat_gpu, out["codes"], out["xt"], out["scale64"])
    if np.array_equal(nat_gpu.astype(np.int32), out["codes"]):
        return bf16_values(out["y"])
    acc = orc.int_gemm(nat_gpu.astype(np.int32), u, z)
    return bf16_values(orc.epilogue(acc, out["scale32"], d, bias_bits, act))
