"""The allocation-free entry point dvdq_qlinear_static against dvdq_qlinear.

Some callers of the library may not allocate device memory at all (they run inside another
framework's engine or a loop that must never touch the allocator), so they cannot provide
the workspace dvdq_qlinear asks for.  dvdq_qlinear_static keeps that workspace in a fixed
array inside the library.  Both entry points launch the same kernels, so their outputs must
agree bit for bit; the second call checks that what the first call left in the shared array
does no harm.  This file is named so that pytest collects it last.
"""
import ctypes as C

import pytest
import torch

from paper_2505_18663_b200 import binding as B
from paper_2505_18663_b200 import workloads as W

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _layer(N, K, rot_block, seed, symmetric):
    layer = W.Layer(K=K, N=N, rot_block=rot_block, bits=4)
    u, d, z = W.make_weight_codes(layer, seed=seed, device=DEV, symmetric=symmetric)
    blob = torch.empty(B.dvdq_weight_blob_bytes(N, K), dtype=torch.uint8, device=DEV)
    return B.dvdq_pack_weights(u, d, z, rot_block, blob), blob


def _x(M, K, seed):
    g = torch.Generator(device=DEV).manual_seed(seed)
    return (torch.randn(M, K, generator=g, device=DEV) * 1.5).to(torch.bfloat16)


def test_static_scratch_entry_point_matches_qlinear_on_two_calls_in_a_row():
    cases = [
        # M, N, K, B, bits, act, bias, symmetric weights: the larger problem first, so that the
        # second call runs over stale codes of the first one
        (700, 512, 3072, 1024, 6, 1, True, False),
        (300, 264, 1536, 512, 4, 0, False, True),
    ]
    for i, (M, N, K, Bk, bits, act, has_bias, sym) in enumerate(cases):
        w, blob = _layer(N, K, Bk, seed=20 + i, symmetric=sym)
        q = B.ActQuant(bits, Bk, 0)
        x = _x(M, K, seed=30 + i)
        bias = (torch.randn(N, device=DEV) * 0.1).to(torch.bfloat16) if has_bias else None
        ws = torch.empty(B.dvdq_qlinear_workspace_bytes(M, K, q), dtype=torch.uint8, device=DEV)
        assert ws.numel() <= B.STATIC_SCRATCH_BYTES
        y_ref = torch.empty(M, N, dtype=torch.bfloat16, device=DEV)
        y_new = torch.full((M, N), float("nan"), dtype=torch.bfloat16, device=DEV)
        B.dvdq_qlinear(x, q, w, bias, act, y_ref, ws)
        B.dvdq_qlinear_static(x, q, w, bias, act, y_new)
        torch.cuda.synchronize()
        status, detail = B.dvdq_last_device_status()
        assert status == B.OK, (status, detail)
        assert bool(torch.isfinite(y_new).all())
        assert torch.equal(y_new, y_ref), f"call {i}: outputs differ"


def test_static_scratch_entry_point_refuses_problems_beyond_its_limit():
    K, N, Bk = 3072, 256, 1024
    w, blob = _layer(N, K, Bk, seed=5, symmetric=True)
    q = B.ActQuant(4, Bk, 0)
    M = 16384                                                    # 16384 * 1536 B of codes alone > 16 MiB
    assert B.dvdq_qlinear_workspace_bytes(M, K, q) > B.STATIC_SCRATCH_BYTES
    x = torch.zeros(8, K, dtype=torch.bfloat16, device=DEV)     # never read: the call must refuse first
    y = torch.zeros(8, N, dtype=torch.bfloat16, device=DEV)
    rc = B.load().dvdq_qlinear_static(C.c_void_p(x.data_ptr()), M, K, C.byref(q), C.byref(w), None, 0,
                                      C.c_void_p(y.data_ptr()), N, None)
    assert rc == B.ERR_WORKSPACE
    with pytest.raises(B.DvdqError):
        B.dvdq_qlinear_static(torch.zeros(M, K, dtype=torch.bfloat16, device=DEV), q, w, None, 0,
                              torch.zeros(M, N, dtype=torch.bfloat16, device=DEV))
