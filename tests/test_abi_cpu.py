"""Host-side checks that need no GPU: the library builds, loads, exports every symbol the
header declares, answers its size queries and rejects bad arguments before any CUDA call."""
import ctypes as C
import os
import re

import pytest
import torch

from paper_2505_18663_b200 import binding as B
from paper_2505_18663_b200 import build, workloads as W

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "dvdq.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(dvdq_[a-z0-9_]+)\s*\(", text)))


def test_library_builds_and_exports_every_declared_symbol():
    path = build.build_library()
    assert os.path.exists(path)
    lib = C.CDLL(path)
    names = declared_symbols()
    assert len(names) >= 14
    for n in names:
        assert hasattr(lib, n), f"{n} declared in dvdq.h but not exported"
    assert sorted(B.EXPORTS) == names
    assert B.dvdq_version() >= 1


def test_size_queries():
    assert B.dvdq_act_codes_bytes(256, 256, 4) == 256 * 128
    assert B.dvdq_act_codes_bytes(10, 3072, 6) == 10 * 2304
    assert B.dvdq_act_codes_bytes(10, 100, 4) == 0          # K not a multiple of 64
    assert B.dvdq_act_codes_bytes(10, 256, 5) == 0
    n = B.dvdq_weight_blob_bytes(3072, 3072)
    assert n >= 3072 * 1536 + 8 * 3072 and n % 256 == 0
    assert B.dvdq_weight_blob_bytes(3071, 3072) == 0
    assert B.dvdq_weight_operand_bytes(3072, 12288) == 3072 * 12288       # one int8 per code
    assert B.dvdq_weight_operand_bytes(3071, 3072) == 0 and B.dvdq_weight_operand_bytes(3072, 100) == 0
    q = B.ActQuant(4, 1024, 0)
    ws = B.dvdq_qlinear_workspace_bytes(1000, 3072, q)
    assert ws >= 1000 * 1536 + 8000 and ws % 256 == 0
    assert B.dvdq_qlinear_workspace_bytes(1000, 3072, B.ActQuant(4, 2048, 0)) == 0   # B does not divide K
    assert B.dvdq_qlinear_workspace_bytes(1000, 4096, B.ActQuant(4, 2048, 0)) > 0
    assert B.dvdq_qlinear_workspace_bytes(1000, 12288, B.ActQuant(4, 4096, 0)) > 0
    assert B.dvdq_qlinear_workspace_bytes(1000, 16384, B.ActQuant(4, 8192, 0)) == 0  # B > 4096
    assert B.dvdq_qlinear_workspace_bytes(1000, 1536, B.ActQuant(4, 1024, 0)) == 0   # B does not divide K
    assert B.dvdq_qlinear_workspace_bytes(1000, 3072, B.ActQuant(4, 1024, 64)) == 0  # granularity that is not built
    # block-wise scales: one scale and one code sum per token and group of 128, 256 or 1024 channels
    assert B.dvdq_act_scales_count(1000, 3072, B.ActQuant(4, 256, 256)) == 12000
    assert B.dvdq_act_scales_count(1000, 3072, B.ActQuant(4, 256, 128)) == 24000
    assert B.dvdq_act_scales_count(1000, 8960, B.ActQuant(4, 256, 256)) == 35000
    assert B.dvdq_act_scales_count(1000, 8960, B.ActQuant(4, 256, 1024)) == 0         # 8960 is not a multiple of 1024
    assert B.dvdq_act_scales_count(1000, 384, B.ActQuant(4, 64, 128)) == 0            # the GEMM takes k-blocks in pairs: K % 256
    qb = B.ActQuant(4, 256, 1024)
    assert B.dvdq_act_scales_count(1000, 3072, q) == 1000
    assert B.dvdq_act_scales_count(1000, 3072, qb) == 3000
    assert B.dvdq_act_scales_count(1000, 3200, qb) == 0                               # K is not a multiple of the block
    assert B.dvdq_qlinear_workspace_bytes(1000, 3072, qb) >= 1000 * 1536 + 2 * 3000 * 4
    assert B.dvdq_qlinear_workspace_bytes(1000, 3072, qb) > B.dvdq_qlinear_workspace_bytes(1000, 3072, B.ActQuant(4, 256, 0))


def test_status_strings():
    seen = set()
    for s in range(12):
        msg = B.status_string(s)
        assert msg and msg != "unknown status"
        seen.add(msg)
    assert len(seen) == 12
    assert B.status_string(99) == "unknown status"


def test_validation_happens_before_any_cuda_call():
    lib = B.load()
    q = B.ActQuant(5, 256, 0)
    one = C.c_void_p(256)   # never dereferenced: validation fails first
    assert lib.dvdq_rotate_quantize(one, 4, 256, 256, None, one, one, one, None) == B.ERR_NULL
    assert lib.dvdq_rotate_quantize(one, 4, 256, 256, C.byref(q), one, one, one, None) == B.ERR_BITS
    assert lib.dvdq_rotate_quantize(one, 4, 256, 256, C.byref(B.ActQuant(16, 256, 0)), one, one, one, None) == B.ERR_BITS
    assert B.dvdq_act_codes_bytes(3, 256, 8) == 3 * 256 and B.dvdq_act_codes_bytes(3, 256, 6) == 3 * 192
    assert lib.dvdq_rotate_quantize(one, 4, 250, 256, C.byref(B.ActQuant(4, 0, 0)), one, one, one, None) == B.ERR_SHAPE
    assert lib.dvdq_rotate_quantize(one, 4, 256, 128, C.byref(B.ActQuant(4, 256, 0)), one, one, one, None) == B.ERR_SHAPE
    assert lib.dvdq_rotate_quantize(one, 4, 256, 256, C.byref(B.ActQuant(4, 96, 0)), one, one, one, None) == B.ERR_ROT_BLOCK
    assert lib.dvdq_rotate_quantize(one, 4, 256, 256, C.byref(B.ActQuant(4, 512, 0)), one, one, one, None) == B.ERR_ROT_BLOCK
    assert lib.dvdq_rotate_quantize(one, 4, 16384, 16384, C.byref(B.ActQuant(4, 8192, 0)), one, one, one, None) == B.ERR_ROT_BLOCK
    assert lib.dvdq_rotate_quantize(one, 4, 256, 256, C.byref(B.ActQuant(4, 256, 1)), one, one, one, None) == B.ERR_UNSUPPORTED
    assert lib.dvdq_rotate_quantize(one, 4, 2048, 2048, C.byref(B.ActQuant(4, 256, 512)), one, one, one, None) == B.ERR_UNSUPPORTED
    assert lib.dvdq_rotate_quantize(one, 4, 1536, 1536, C.byref(B.ActQuant(4, 256, 1024)), one, one, one, None) == B.ERR_SHAPE
    assert lib.dvdq_rotate_quantize(one, 4, 384, 384, C.byref(B.ActQuant(4, 128, 128)), one, one, one, None) == B.ERR_SHAPE
    assert lib.dvdq_rotate_quantize(None, 4, 256, 256, C.byref(B.ActQuant(4, 256, 0)), one, one, one, None) == B.ERR_NULL
    assert lib.dvdq_rotate_quantize(C.c_void_p(8), 4, 256, 256, C.byref(B.ActQuant(4, 256, 0)), one, one, one, None) == B.ERR_ALIGN
    # weight handle checks
    w = B.Weights()
    assert lib.dvdq_qgemm(one, one, one, 4, C.byref(B.ActQuant(4, 256, 0)), C.byref(w), None, 0, one, 256, None) == B.ERR_BLOB
    assert lib.dvdq_qgemm(one, one, one, 4, C.byref(B.ActQuant(4, 256, 0)), None, None, 0, one, 256, None) == B.ERR_NULL
    w = B.Weights(0x51445644, 1, 256, 256, 256, 0, 4096, B.dvdq_weight_blob_bytes(256, 256))
    assert lib.dvdq_qgemm(one, one, one, 4, C.byref(B.ActQuant(4, 128, 0)), C.byref(w), None, 0, one, 256, None) == B.ERR_ROT_BLOCK
    assert lib.dvdq_qgemm(one, one, one, 4, C.byref(B.ActQuant(4, 256, 0)), C.byref(w), None, 7, one, 256, None) in (B.ERR_UNSUPPORTED, B.ERR_CUDA, B.ERR_ARCH)
    w.blob_bytes = 17
    assert lib.dvdq_qgemm(one, one, one, 4, C.byref(B.ActQuant(4, 256, 0)), C.byref(w), None, 0, one, 256, None) == B.ERR_BLOB
    assert lib.dvdq_pack_weights(one, one, one, 250, 256, 256, one, C.byref(w), None) == B.ERR_SHAPE
    assert lib.dvdq_qlinear(one, 4, 256, C.byref(B.ActQuant(4, 256, 0)), C.byref(B.Weights()), None, 0, one, 256, one, 0, None) == B.ERR_BLOB
    # dvdq_qlinear and dvdq_qlinear_static refuse everything dvdq_qgemm would refuse BEFORE their
    # first launch (the pointers here are never dereferenced, so nothing was launched)
    w = B.Weights(0x51445644, 1, 256, 256, 256, 0, 4096, B.dvdq_weight_blob_bytes(256, 256))
    big = 1 << 30
    for call in (lambda q, act, ldy, M=4: lib.dvdq_qlinear(one, M, 256, C.byref(q), C.byref(w), None, act, one, ldy, one, big, None),
                 lambda q, act, ldy, M=4: lib.dvdq_qlinear_static(one, M, 256, C.byref(q), C.byref(w), None, act, one, ldy, None)):
        assert call(B.ActQuant(4, 128, 0), 0, 256) == B.ERR_ROT_BLOCK       # activations and weights disagree on B
        assert call(B.ActQuant(4, 256, 0), 7, 256) == B.ERR_UNSUPPORTED     # unknown activation function
        assert call(B.ActQuant(4, 256, 0), 0, 250) == B.ERR_SHAPE           # ldy < N
        assert call(B.ActQuant(4, 256, 0), 0, 256, 0x7FFFFF01) == B.ERR_SHAPE
    assert lib.dvdq_qlinear(one, 4, 256, C.byref(B.ActQuant(4, 256, 0)), C.byref(w), None, 0, None, 256, one, big, None) == B.ERR_NULL
    assert lib.dvdq_qlinear(one, 4, 256, C.byref(B.ActQuant(4, 256, 0)), C.byref(w), None, 0, C.c_void_p(8), 256, one, big, None) == B.ERR_ALIGN
    # the offline weight entry points
    assert lib.dvdq_rotate_weights(one, 8, 250, 256, 0, one, None) == B.ERR_SHAPE
    assert lib.dvdq_rotate_weights(one, 8, 256, 128, 0, one, None) == B.ERR_SHAPE       # ldw < K
    assert lib.dvdq_rotate_weights(one, 8, 256, 256, 96, one, None) == B.ERR_ROT_BLOCK
    assert lib.dvdq_rotate_weights(None, 8, 256, 256, 64, one, None) == B.ERR_NULL
    assert lib.dvdq_quantize_weights_symmetric(one, 9, 256, 256, 64, one, C.byref(B.Weights()), None) == B.ERR_SHAPE   # N % 8
    assert lib.dvdq_quantize_weights_symmetric(one, 8, 256, 256, 64, one, None, None) == B.ERR_NULL
    assert lib.dvdq_quantize_weights_symmetric(one, 8, 256, 256, 64, C.c_void_p(64), C.byref(B.Weights()), None) == B.ERR_ALIGN
    # the int8 weight operand: the handle is validated first, then the caller's buffer
    wh = B.Weights(0x51445644, 1, 256, 256, 256, 0, 4096, B.dvdq_weight_blob_bytes(256, 256))
    wo = B.Weights()
    nk = 256 * 256
    assert lib.dvdq_widen_weights(C.byref(wh), C.c_void_p(4096), nk, None, None) == B.ERR_NULL
    assert lib.dvdq_widen_weights(None, C.c_void_p(4096), nk, C.byref(wo), None) == B.ERR_NULL
    assert lib.dvdq_widen_weights(C.byref(B.Weights()), C.c_void_p(4096), nk, C.byref(wo), None) == B.ERR_BLOB
    assert lib.dvdq_widen_weights(C.byref(wh), None, nk, C.byref(wo), None) == B.ERR_NULL
    assert lib.dvdq_widen_weights(C.byref(wh), C.c_void_p(4096), nk - 1, C.byref(wo), None) == B.ERR_WORKSPACE
    assert lib.dvdq_widen_weights(C.byref(wh), C.c_void_p(4096 + 16), nk, C.byref(wo), None) == B.ERR_ALIGN
    # a handle whose operand does not fit its shape, or is misaligned, is refused by the GEMM
    wh.operand, wh.operand_bytes = 8192, nk - 64
    assert lib.dvdq_qgemm(one, one, one, 4, C.byref(B.ActQuant(4, 256, 0)), C.byref(wh), None, 0, one, 256, None) == B.ERR_BLOB
    wh.operand, wh.operand_bytes = 8192 + 16, nk
    assert lib.dvdq_qgemm(one, one, one, 4, C.byref(B.ActQuant(4, 256, 0)), C.byref(wh), None, 0, one, 256, None) == B.ERR_ALIGN
    assert lib.dvdq_int8_mma_ceiling(0, None, None) == B.ERR_SHAPE
    assert lib.dvdq_debug_wait_timeout(0, None) == B.ERR_SHAPE


def test_binding_refuses_cpu_tensors():
    x = torch.zeros(4, 256, dtype=torch.bfloat16)
    with pytest.raises(TypeError):
        B.dvdq_rotate_quantize(x, B.ActQuant(4, 256, 0), torch.zeros(512, dtype=torch.uint8),
                               torch.zeros(4), torch.zeros(4, dtype=torch.int32))


def test_workloads_are_seeded_and_shaped():
    for name, wl in W.WORKLOADS.items():
        for layer in wl.layers:
            assert layer.K % layer.rot_block == 0 and layer.rot_block in (256, 512, 1024)
            assert layer.bits in (4, 6) and layer.N % 256 == 0
    wl = W.WORKLOADS["tiny"]
    a = W.make_activations(wl, 256)
    b = W.make_activations(wl, 256)
    assert a.shape == (256, 256) and a.dtype == torch.bfloat16 and torch.equal(a, b)
    col_rms = a.float().pow(2).mean(0).sqrt()
    assert int((col_rms > 10).sum()) == 4                      # four outlier channels x20
    hy = W.WORKLOADS["hunyuan"]
    assert sorted(l.bits for l in hy.layers) == [4, 4, 4, 6]   # 25 % of the layers at 6 bits
    assert hy.M == 65536 and W.WORKLOADS["ffn_chain"].M == 118800 and W.WORKLOADS["wan1p3b"].M == 21 * 30 * 52
    x = W.make_activations(W.WORKLOADS["wan14b"], 5120, M=64)
    rms = x.float().pow(2).mean(1).sqrt()
    assert rms.max() / rms.min() > 5                            # per-token magnitude spread
    rows = W.sample_rows(32760, 64)
    assert rows[0] == 0 and rows[-1] == 32759 and (rows >= 32640).sum() >= 100
    u, d, z = W.make_weight_codes(hy.layers[0], 3)
    assert u.dtype == torch.uint8 and int(u.max()) <= 15 and z.eq(8).all()
