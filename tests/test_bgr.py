"""Bounded-init Grid Refinement (Alg. 1, Sec. 3.1): oracle pins (CPU) and the CUDA kernel against
the oracle (GPU)."""
import os

import numpy as np
import pytest
import torch

from oracle import dvdq_oracle as orc
from paper_2505_18663_b200 import binding as B

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "bgr_worked_example.txt")


def read_golden():
    out = {}
    for line in open(GOLDEN):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        key, *vals = line.split()
        out[key] = [float(v) for v in vals]
    return out


def gaussian_rows(N, K, seed, outliers=True):
    rng = np.random.default_rng(seed)
    w = rng.standard_normal((N, K)) * 0.02
    if outliers:                                   # a few far values per row, as rotated DiT weights have
        for n in range(N):
            w[n, rng.integers(0, K, 3)] *= 4.0
    return w


def quant_numpy(w, d, z, levels=15):
    """Quant / DeQuant of Sec. 3.1 written with numpy (round half to even), independent of the C code."""
    c = np.clip(np.rint(w / d[:, None]) + z[:, None], 0, levels)
    return c, d[:, None] * (c - z[:, None])


# ------------------------------------------------------------------ oracle pins

def test_oracle_matches_hand_worked_example():
    g = read_golden()
    w = np.array([g["w"]])
    u, d, z, e = orc.bgr_quantize(w, bits=int(g["bits"][0]), n_steps=int(g["n_steps"][0]), eps=g["eps"][0])
    assert u[0].tolist() == [int(v) for v in g["u"]]
    assert abs(d[0] - g["delta"][0]) < 1e-14 and z[0] == int(g["zero"][0])
    assert abs(e[0] ** 2 - g["err2"][0]) < 1e-14
    assert abs(orc.minmax_row_error(w, bits=2)[0] ** 2 - g["minmax_err2"][0]) < 1e-14


def test_oracle_output_is_a_valid_grid_and_reports_its_error():
    w = gaussian_rows(48, 1536, 1)
    u, d, z, e = orc.bgr_quantize(w)
    assert u.max() <= 15 and z.min() >= 0 and z.max() <= 15 and (d > 0).all()
    c, deq = quant_numpy(w, d, z.astype(np.float64))
    assert np.array_equal(c.astype(np.uint8), u)                     # codes follow from (Delta, z) by Quant
    assert np.allclose(np.linalg.norm(w - deq, axis=1), e, rtol=1e-12)


def test_oracle_never_worse_than_any_bounded_initialisation():
    """The result keeps the best grid seen, so its error is at most that of every clipped MinMax
    start (computed here with numpy), and in particular well below plain MinMax on bell-shaped rows."""
    w = gaussian_rows(32, 1024, 2)
    n_steps = 100
    u, d, z, e = orc.bgr_quantize(w, n_steps=n_steps)
    lo, hi = w.min(axis=1), w.max(axis=1)
    best_init = np.full(len(w), np.inf)
    for i in range(1, (n_steps + 1) // 2):
        lo_c, hi_c = lo + i * (hi - lo) / n_steps, hi - i * (hi - lo) / n_steps
        d0 = (hi_c - lo_c) / 15.0
        z0 = np.clip(-np.rint(lo_c / d0), 0, 15)
        _, deq = quant_numpy(w, d0, z0)
        best_init = np.minimum(best_init, np.linalg.norm(w - deq, axis=1))
    assert (e <= best_init * (1 + 1e-12)).all()
    em = orc.minmax_row_error(w)
    assert (e <= em).all() and (e / em).mean() < 0.85


def test_oracle_recovers_a_row_that_lies_on_a_grid():
    rng = np.random.default_rng(3)
    q = rng.integers(0, 16, size=(8, 512)).astype(np.float64)
    q[:, 0], q[:, 1] = 0, 15                                         # the row uses the whole range
    d_true = rng.random(8) * 0.01 + 0.001
    z_true = rng.integers(3, 12, size=8).astype(np.float64)
    w = d_true[:, None] * (q - z_true[:, None])
    u, d, z, e = orc.bgr_quantize(w, n_steps=100, eps=1e-12)
    # shrinking the range can only hurt such a row a little; refinement must pull the grid back
    assert (e <= 1e-9).all(), e
    assert np.allclose(d, d_true, rtol=1e-9) and np.array_equal(z, z_true.astype(np.int32))
    assert np.array_equal(u, q.astype(np.uint8))


# ------------------------------------------------------------------ CUDA kernel against the oracle

@pytest.mark.gpu
@pytest.mark.parametrize("N,K,seed", [(8, 64, 0), (40, 1536, 1), (24, 3072, 2), (9, 8960, 3)])
def test_bgr_kernel_matches_oracle(N, K, seed):
    w32 = gaussian_rows(N, K, seed).astype(np.float32)               # both sides start from these fp32 values
    w32[N // 2] = 0.25 if N > 8 else w32[N // 2]                      # a constant row
    u_or, d_or, z_or, e_or = orc.bgr_quantize(w32.astype(np.float64))
    wd = torch.from_numpy(w32).cuda()
    u = torch.empty(N, K, dtype=torch.uint8, device="cuda")
    d = torch.empty(N, dtype=torch.float32, device="cuda")
    z = torch.empty(N, dtype=torch.int32, device="cuda")
    B.dvdq_bgr_quantize(wd, 100, 1e-5, 50, u, d, z)
    # integer results are decided in fp64 on both sides: equal, up to a summation-order tie
    assert np.array_equal(z.cpu().numpy(), z_or)
    assert np.allclose(d.cpu().numpy().astype(np.float64), d_or, rtol=2e-7)     # stored as fp32
    assert (u.cpu().numpy() != u_or).mean() <= 1e-4
    # what is unique either way: the grid's error
    c, deq = quant_numpy(w32.astype(np.float64), d.cpu().numpy().astype(np.float64), z.cpu().numpy().astype(np.float64))
    e_gpu = np.linalg.norm(w32 - deq, axis=1)
    assert np.allclose(e_gpu, e_or, rtol=1e-5, atol=1e-12)


@pytest.mark.gpu
def test_bgr_weights_feed_the_quantized_layer():
    """rotate (GPU) -> BGR (GPU) -> pack -> qlinear, against the oracle run on the same grid."""
    from helpers import act_quant, bf16_values, to_bits, oracle_y_for_validated_codes
    M, N, K, Bk, bits = 130, 264, 1536, 512, 4
    g = torch.Generator().manual_seed(11)
    x = torch.randn(M, K, generator=g).to(torch.bfloat16)
    wb = (torch.randn(N, K, generator=g) * 0.02).to(torch.bfloat16)
    wt32 = torch.empty(N, K, dtype=torch.float32, device="cuda")
    B.dvdq_rotate_weights(wb.cuda(), Bk, wt32)                      # W~ = W R on the GPU: no CPU step feeds the GPU path
    u = torch.empty(N, K, dtype=torch.uint8, device="cuda")
    d = torch.empty(N, dtype=torch.float32, device="cuda")
    z = torch.empty(N, dtype=torch.int32, device="cuda")
    B.dvdq_bgr_quantize(wt32, 100, 1e-5, 50, u, d, z)
    # the grid the GPU chose is the oracle's for the same rotated weights
    u_or, d_or, z_or, _ = orc.bgr_quantize(wt32.cpu().numpy().astype(np.float64))
    assert np.array_equal(z.cpu().numpy(), z_or) and np.allclose(d.cpu().numpy().astype(np.float64), d_or, rtol=2e-7)
    assert (u.cpu().numpy() != u_or).mean() <= 1e-4
    blob = torch.empty(B.dvdq_weight_blob_bytes(N, K), dtype=torch.uint8, device="cuda")
    w = B.dvdq_pack_weights(u, d, z, Bk, blob)
    q = act_quant(bits, Bk)
    ws = torch.empty(B.dvdq_qlinear_workspace_bytes(M, K, q), dtype=torch.uint8, device="cuda")
    Y = torch.empty(M, N, dtype=torch.bfloat16, device="cuda")
    B.dvdq_qlinear(x.cuda(), q, w, None, 0, Y, ws)
    nat = torch.empty(M, K, dtype=torch.int8, device="cuda")
    B.dvdq_unpack_act_codes(ws, M, K, q, nat)
    un, dn, zn = u.cpu().numpy(), d.cpu().numpy(), z.cpu().numpy()
    out = orc.qlinear(to_bits(x), un, dn, zn, Bk, bits)
    y_or = oracle_y_for_validated_codes(nat.cpu().numpy(), out, un, dn, zn)
    y = Y.to(torch.float64).cpu().numpy()
    assert np.abs(y - y_or).max() <= 4e-3 * np.abs(y_or).max()
    # and the BGR grid is a better approximation of the rotated weights than plain MinMax
    exact = x.to(torch.float64).numpy() @ wb.to(torch.float64).numpy().T
    assert np.linalg.norm(y - exact) / np.linalg.norm(exact) < 0.5
