"""Thin ctypes binding of the C ABI declared in ``include/dvdq.h``.

Argument marshalling only: every function takes torch CUDA tensors (device memory) and a
stream, checks dtypes, passes raw pointers and raises :class:`DvdqError` on a non-zero
status.  No step of the path runs in Python or on the CPU, and there is no fallback: if the
CUDA library is missing, importing the functions fails loudly.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional

import torch

from . import build as _build

# status codes of include/dvdq.h
OK, ERR_NULL, ERR_SHAPE, ERR_BITS, ERR_ROT_BLOCK, ERR_ALIGN, ERR_WORKSPACE, ERR_BLOB, ERR_ARCH, \
    ERR_CUDA, ERR_DEVICE_TIMEOUT, ERR_UNSUPPORTED = range(12)

EXPORTS = [
    "dvdq_status_string", "dvdq_version", "dvdq_act_codes_bytes", "dvdq_act_codes_bytes_q", "dvdq_act_scales_count", "dvdq_weight_blob_bytes",
    "dvdq_qlinear_workspace_bytes", "dvdq_rotate_quantize", "dvdq_pack_weights", "dvdq_qgemm",
    "dvdq_qlinear", "dvdq_qlinear_static", "dvdq_qgemm_fused_rq", "dvdq_qgemm_int32", "dvdq_pack_act_codes", "dvdq_unpack_act_codes",
    "dvdq_unpack_weights", "dvdq_last_device_status",
    "dvdq_rotate_weights", "dvdq_quantize_weights_symmetric", "dvdq_int8_mma_ceiling", "dvdq_debug_wait_timeout",
    "dvdq_weight_operand_bytes", "dvdq_widen_weights",
    "dvdq_bgr_quantize", "dvdq_gbs_l1_terms", "dvdq_gbs_init", "dvdq_gbs_next_bits", "dvdq_gbs_observe",
]


class DvdqError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: status {status} ({status_string(status)})")


class ActQuant(C.Structure):
    """dvdq_act_quant: the activation quantizer of Eq. 10 (bits, rotation block, scale granularity)
    and how its codes are stored (container_bits: 0 = packed, 8 = one int8 per code)."""
    _fields_ = [("bits", C.c_int32), ("rot_block", C.c_int32), ("scale_group", C.c_int32),
                ("container_bits", C.c_int32)]


class Weights(C.Structure):
    """dvdq_weights: host handle of a packed weight blob."""
    _fields_ = [("magic", C.c_uint32), ("version", C.c_uint32), ("N", C.c_int64), ("K", C.c_int64),
                ("rot_block", C.c_int32), ("k_layout", C.c_int32), ("blob", C.c_void_p),
                ("blob_bytes", C.c_uint64), ("operand", C.c_void_p), ("operand_bytes", C.c_uint64)]


class GbsState(C.Structure):
    """dvdq_gbs_state: host-side state of the delta-guided bit switching (Sec. 3.3)."""
    _fields_ = [("delta", C.c_double), ("b_low", C.c_int32), ("b_high", C.c_int32), ("accumulated", C.c_double),
                ("steps", C.c_int64), ("high_steps", C.c_int64)]


_lib = None


def lib_path() -> str:
    return _build.LIB_PATH


def load():
    """dlopen the in-tree library (building it first if the sources are newer)."""
    global _lib
    if _lib is not None:
        return _lib
    path = _build.LIB_PATH
    if _build.is_stale():
        try:
            path = _build.build_library()
        except Exception as e:  # no nvcc on this machine and no prebuilt library
            if not os.path.exists(path):
                raise RuntimeError(f"CUDA library {path} is missing and cannot be built: {e}") from e
    lib = C.CDLL(path)
    i32, i64, p, sz = C.c_int32, C.c_int64, C.c_void_p, C.c_size_t
    aq, wp = C.POINTER(ActQuant), C.POINTER(Weights)
    sig = {
        "dvdq_status_string": (C.c_char_p, [C.c_int]),
        "dvdq_version": (i32, []),
        "dvdq_act_codes_bytes": (sz, [i64, i64, i32]),
        "dvdq_act_codes_bytes_q": (sz, [i64, i64, aq]),
        "dvdq_act_scales_count": (sz, [i64, i64, aq]),
        "dvdq_weight_blob_bytes": (sz, [i64, i64]),
        "dvdq_weight_operand_bytes": (sz, [i64, i64]),
        "dvdq_widen_weights": (C.c_int, [wp, p, sz, wp, p]),
        "dvdq_qlinear_workspace_bytes": (sz, [i64, i64, aq]),
        "dvdq_rotate_quantize": (C.c_int, [p, i64, i64, i64, aq, p, p, p, p]),
        "dvdq_pack_weights": (C.c_int, [p, p, p, i64, i64, i32, p, wp, p]),
        "dvdq_qgemm": (C.c_int, [p, p, p, i64, aq, wp, p, i32, p, i64, p]),
        "dvdq_qlinear": (C.c_int, [p, i64, i64, aq, wp, p, i32, p, i64, p, sz, p]),
        "dvdq_qlinear_static": (C.c_int, [p, i64, i64, aq, wp, p, i32, p, i64, p]),
        "dvdq_qgemm_int32": (C.c_int, [p, p, i64, aq, wp, p, i64, p]),
        "dvdq_qgemm_fused_rq": (C.c_int, [p, p, p, i64, aq, wp, p, i32, aq, p, p, p, p, i64, p]),
        "dvdq_pack_act_codes": (C.c_int, [p, i64, i64, aq, p, p, p]),
        "dvdq_unpack_act_codes": (C.c_int, [p, i64, i64, aq, p, p]),
        "dvdq_unpack_weights": (C.c_int, [wp, p, p, p, p]),
        "dvdq_last_device_status": (C.c_int, [C.POINTER(C.c_uint32)]),
        "dvdq_bgr_quantize": (C.c_int, [p, i64, i64, i32, C.c_double, i32, p, p, p, p]),
        "dvdq_rotate_weights": (C.c_int, [p, i64, i64, i64, i32, p, p]),
        "dvdq_quantize_weights_symmetric": (C.c_int, [p, i64, i64, i64, i32, p, wp, p]),
        "dvdq_int8_mma_ceiling": (C.c_int, [i32, C.POINTER(C.c_int64), p]),
        "dvdq_debug_wait_timeout": (C.c_int, [C.c_uint64, p]),
        "dvdq_gbs_l1_terms": (C.c_int, [p, p, i64, p, p]),
        "dvdq_gbs_init": (C.c_int, [C.POINTER(GbsState), C.c_double, i32, i32]),
        "dvdq_gbs_next_bits": (i32, [C.POINTER(GbsState)]),
        "dvdq_gbs_observe": (C.c_int, [C.POINTER(GbsState), C.c_double, C.c_double]),
    }
    for name, (res, args) in sig.items():
        fn = getattr(lib, name)
        fn.restype = res
        fn.argtypes = args
    _lib = lib
    return lib


def status_string(status: int) -> str:
    return load().dvdq_status_string(int(status)).decode()


def _check(status: int, where: str):
    if status != OK:
        raise DvdqError(status, where)


def _ptr(t: Optional[torch.Tensor], dtype=None, name="tensor"):
    if t is None:
        return None
    if not t.is_cuda:
        raise TypeError(f"{name} must be a CUDA tensor")
    if dtype is not None and t.dtype != dtype:
        raise TypeError(f"{name} must be {dtype}, got {t.dtype}")
    return C.c_void_p(t.data_ptr())


def _stream(stream) -> C.c_void_p:
    if stream is None:
        stream = torch.cuda.current_stream()
    return C.c_void_p(stream.cuda_stream)


def _row_major(t: torch.Tensor, name: str) -> int:
    if t.dim() != 2 or t.stride(1) != 1:
        raise TypeError(f"{name} must be 2-D with unit inner stride")
    return t.stride(0)


# ------------------------------------------------------------------ size queries

def dvdq_version() -> int:
    return int(load().dvdq_version())


def dvdq_act_codes_bytes(M: int, K: int, bits: int) -> int:
    return int(load().dvdq_act_codes_bytes(M, K, bits))


def dvdq_act_codes_bytes_q(M: int, K: int, q: ActQuant) -> int:
    return int(load().dvdq_act_codes_bytes_q(M, K, C.byref(q)))


def dvdq_act_scales_count(M: int, K: int, q: ActQuant) -> int:
    return int(load().dvdq_act_scales_count(M, K, C.byref(q)))


def dvdq_weight_blob_bytes(N: int, K: int) -> int:
    return int(load().dvdq_weight_blob_bytes(N, K))


def dvdq_qlinear_workspace_bytes(M: int, K: int, q: ActQuant) -> int:
    return int(load().dvdq_qlinear_workspace_bytes(M, K, C.byref(q)))


# ------------------------------------------------------------------ the path

def dvdq_rotate_quantize(X: torch.Tensor, q: ActQuant, codes: torch.Tensor, scales: torch.Tensor,
                         code_sums: torch.Tensor, stream=None) -> None:
    ldx = _row_major(X, "X")
    M, K = X.shape
    _check(load().dvdq_rotate_quantize(_ptr(X, torch.bfloat16, "X"), M, K, ldx, C.byref(q),
                                       _ptr(codes, torch.uint8, "codes"), _ptr(scales, torch.float32, "scales"),
                                       _ptr(code_sums, torch.int32, "code_sums"), _stream(stream)),
           "dvdq_rotate_quantize")


def dvdq_pack_weights(Wq: torch.Tensor, delta: torch.Tensor, zero: torch.Tensor, rot_block: int,
                      blob: torch.Tensor, stream=None) -> Weights:
    N, K = Wq.shape
    if not Wq.is_contiguous():
        raise TypeError("Wq must be contiguous")
    w = Weights()
    _check(load().dvdq_pack_weights(_ptr(Wq, torch.uint8, "Wq"), _ptr(delta, torch.float32, "delta"),
                                    _ptr(zero, torch.int32, "zero"), N, K, rot_block,
                                    _ptr(blob, torch.uint8, "blob"), C.byref(w), _stream(stream)),
           "dvdq_pack_weights")
    return w


def dvdq_qgemm(codes: torch.Tensor, scales: torch.Tensor, code_sums: torch.Tensor, M: int, q: ActQuant,
               w: Weights, bias: Optional[torch.Tensor], act: int, Y: torch.Tensor, stream=None) -> None:
    ldy = _row_major(Y, "Y")
    _check(load().dvdq_qgemm(_ptr(codes, torch.uint8, "codes"), _ptr(scales, torch.float32, "scales"),
                             _ptr(code_sums, torch.int32, "code_sums"), M, C.byref(q), C.byref(w),
                             _ptr(bias, torch.bfloat16, "bias"), act, _ptr(Y, torch.bfloat16, "Y"), ldy,
                             _stream(stream)), "dvdq_qgemm")


def dvdq_qgemm_fused_rq(codes: torch.Tensor, scales: torch.Tensor, code_sums: torch.Tensor, M: int, q: ActQuant,
                        w: Weights, bias: Optional[torch.Tensor], act: int, q_next: ActQuant, codes_next: torch.Tensor,
                        scales_next: torch.Tensor, code_sums_next: torch.Tensor, Y: Optional[torch.Tensor] = None,
                        stream=None) -> None:
    """dvdq_qgemm whose epilogue writes the next layer's codes / scales / code sums
    (rot_block = scale_group = 256, one int8 per code) instead of bf16; Y, if given, also gets the bf16 output."""
    ldy = _row_major(Y, "Y") if Y is not None else 0
    _check(load().dvdq_qgemm_fused_rq(_ptr(codes, torch.uint8, "codes"), _ptr(scales, torch.float32, "scales"),
                                      _ptr(code_sums, torch.int32, "code_sums"), M, C.byref(q), C.byref(w),
                                      _ptr(bias, torch.bfloat16, "bias"), act, C.byref(q_next),
                                      _ptr(codes_next, torch.uint8, "codes_next"), _ptr(scales_next, torch.float32, "scales_next"),
                                      _ptr(code_sums_next, torch.int32, "code_sums_next"), _ptr(Y, torch.bfloat16, "Y"), ldy,
                                      _stream(stream)), "dvdq_qgemm_fused_rq")


def dvdq_qlinear(X: torch.Tensor, q: ActQuant, w: Weights, bias: Optional[torch.Tensor], act: int,
                 Y: torch.Tensor, workspace: torch.Tensor, stream=None) -> None:
    ldx = _row_major(X, "X")
    ldy = _row_major(Y, "Y")
    M = X.shape[0]
    _check(load().dvdq_qlinear(_ptr(X, torch.bfloat16, "X"), M, ldx, C.byref(q), C.byref(w),
                               _ptr(bias, torch.bfloat16, "bias"), act, _ptr(Y, torch.bfloat16, "Y"), ldy,
                               _ptr(workspace, torch.uint8, "workspace"), workspace.numel(), _stream(stream)),
           "dvdq_qlinear")


STATIC_SCRATCH_BYTES = 16 * 1024 * 1024


def dvdq_qlinear_static(X: torch.Tensor, q: ActQuant, w: Weights, bias: Optional[torch.Tensor], act: int,
                        Y: torch.Tensor, stream=None) -> None:
    """dvdq_qlinear for callers that cannot allocate: the intermediate codes live in a fixed
    STATIC_SCRATCH_BYTES array inside the library (shared by all calls on a device, so calls
    must not overlap; larger problems are refused with ERR_WORKSPACE)."""
    ldx = _row_major(X, "X")
    ldy = _row_major(Y, "Y")
    _check(load().dvdq_qlinear_static(_ptr(X, torch.bfloat16, "X"), X.shape[0], ldx, C.byref(q), C.byref(w),
                                      _ptr(bias, torch.bfloat16, "bias"), act, _ptr(Y, torch.bfloat16, "Y"), ldy,
                                      _stream(stream)), "dvdq_qlinear_static")


# ------------------------------------------------------------------ test / debug entry points

def dvdq_qgemm_int32(codes: torch.Tensor, code_sums: torch.Tensor, M: int, q: ActQuant, w: Weights,
                     acc: torch.Tensor, stream=None) -> None:
    ld = _row_major(acc, "acc")
    _check(load().dvdq_qgemm_int32(_ptr(codes, torch.uint8, "codes"), _ptr(code_sums, torch.int32, "code_sums"),
                                   M, C.byref(q), C.byref(w), _ptr(acc, torch.int32, "acc"), ld, _stream(stream)),
           "dvdq_qgemm_int32")


def dvdq_pack_act_codes(codes_nat: torch.Tensor, q: ActQuant, codes: torch.Tensor, code_sums: torch.Tensor,
                        stream=None) -> None:
    M, K = codes_nat.shape
    if not codes_nat.is_contiguous():
        raise TypeError("codes_nat must be contiguous")
    _check(load().dvdq_pack_act_codes(_ptr(codes_nat, torch.int8, "codes_nat"), M, K, C.byref(q),
                                      _ptr(codes, torch.uint8, "codes"), _ptr(code_sums, torch.int32, "code_sums"),
                                      _stream(stream)), "dvdq_pack_act_codes")


def dvdq_unpack_act_codes(codes: torch.Tensor, M: int, K: int, q: ActQuant, codes_nat: torch.Tensor,
                          stream=None) -> None:
    if not codes_nat.is_contiguous() or tuple(codes_nat.shape) != (M, K):
        raise TypeError("codes_nat must be contiguous [M, K]")
    _check(load().dvdq_unpack_act_codes(_ptr(codes, torch.uint8, "codes"), M, K, C.byref(q),
                                        _ptr(codes_nat, torch.int8, "codes_nat"), _stream(stream)),
           "dvdq_unpack_act_codes")


def dvdq_unpack_weights(w: Weights, Wq: torch.Tensor, delta: torch.Tensor, zero: torch.Tensor, stream=None) -> None:
    if not Wq.is_contiguous():
        raise TypeError("Wq must be contiguous")
    _check(load().dvdq_unpack_weights(C.byref(w), _ptr(Wq, torch.uint8, "Wq"), _ptr(delta, torch.float32, "delta"),
                                      _ptr(zero, torch.int32, "zero"), _stream(stream)), "dvdq_unpack_weights")


def dvdq_rotate_weights(W: torch.Tensor, rot_block: int, W_rot: torch.Tensor, stream=None) -> None:
    """W~ = W R along K: bf16 [N, K] -> dense fp32 [N, K]."""
    ldw = _row_major(W, "W")
    N, K = W.shape
    if not W_rot.is_contiguous() or tuple(W_rot.shape) != (N, K):
        raise TypeError("W_rot must be dense [N, K]")
    _check(load().dvdq_rotate_weights(_ptr(W, torch.bfloat16, "W"), N, K, ldw, rot_block,
                                      _ptr(W_rot, torch.float32, "W_rot"), _stream(stream)), "dvdq_rotate_weights")


def dvdq_quantize_weights_symmetric(W: torch.Tensor, rot_block: int, blob: torch.Tensor, stream=None) -> Weights:
    """bf16 [N, K] weights -> rotated, symmetric 4-bit codes (z = 8, Delta = absmax / 7) in a blob."""
    ldw = _row_major(W, "W")
    N, K = W.shape
    w = Weights()
    _check(load().dvdq_quantize_weights_symmetric(_ptr(W, torch.bfloat16, "W"), N, K, ldw, rot_block,
                                                  _ptr(blob, torch.uint8, "blob"), C.byref(w), _stream(stream)),
           "dvdq_quantize_weights_symmetric")
    return w


def dvdq_weight_operand_bytes(N: int, K: int) -> int:
    return int(load().dvdq_weight_operand_bytes(N, K))


def dvdq_widen_weights(w: Weights, operand: torch.Tensor, stream=None) -> Weights:
    """Writes the 4-bit codes of `w` one int8 each into `operand` (uint8, >= N * K bytes) and returns
    a handle that refers to both; GEMMs given it read the weight operand with TMA."""
    out = Weights()
    _check(load().dvdq_widen_weights(C.byref(w), _ptr(operand, torch.uint8, "operand"), operand.numel(), C.byref(out),
                                     _stream(stream)), "dvdq_widen_weights")
    return out


def dvdq_int8_mma_ceiling(iters: int, stream=None) -> int:
    """Launches the int8 tensor-pipe issue loop; returns the integer operations of the launch."""
    ops = C.c_int64(0)
    _check(load().dvdq_int8_mma_ceiling(iters, C.byref(ops), _stream(stream)), "dvdq_int8_mma_ceiling")
    return int(ops.value)


def dvdq_debug_wait_timeout(limit_ns: int, stream=None) -> None:
    _check(load().dvdq_debug_wait_timeout(int(limit_ns), _stream(stream)), "dvdq_debug_wait_timeout")


def dvdq_bgr_quantize(W_rot: torch.Tensor, n_steps: int, eps: float, max_iter: int, Wq: torch.Tensor,
                      delta: torch.Tensor, zero: torch.Tensor, stream=None) -> None:
    """Bounded-init Grid Refinement of rotated fp32 weights [N, K] -> (Wq uint8, delta fp32, zero int32)."""
    if W_rot.dim() != 2 or not W_rot.is_contiguous() or not Wq.is_contiguous():
        raise TypeError("W_rot and Wq must be dense [N, K]")
    N, K = W_rot.shape
    _check(load().dvdq_bgr_quantize(_ptr(W_rot, torch.float32, "W_rot"), N, K, n_steps, float(eps), max_iter,
                                    _ptr(Wq, torch.uint8, "Wq"), _ptr(delta, torch.float32, "delta"),
                                    _ptr(zero, torch.int32, "zero"), _stream(stream)), "dvdq_bgr_quantize")


def dvdq_gbs_l1_terms(F_t: torch.Tensor, F_prev: torch.Tensor, terms: torch.Tensor, stream=None) -> None:
    """terms (float64[2], device) <- (||F_t - F_prev||_1, ||F_prev||_1) of two bf16 tensors of equal size."""
    if F_t.numel() != F_prev.numel() or not F_t.is_contiguous() or not F_prev.is_contiguous():
        raise TypeError("F_t and F_prev must be contiguous and of equal size")
    if terms.dtype != torch.float64 or terms.numel() < 2:
        raise TypeError("terms must hold two float64 values")
    _check(load().dvdq_gbs_l1_terms(_ptr(F_t, torch.bfloat16, "F_t"), _ptr(F_prev, torch.bfloat16, "F_prev"), F_t.numel(),
                                    _ptr(terms, torch.float64, "terms"), _stream(stream)), "dvdq_gbs_l1_terms")


def dvdq_gbs_init(delta: float, b_low: int, b_high: int) -> GbsState:
    g = GbsState()
    _check(load().dvdq_gbs_init(C.byref(g), float(delta), b_low, b_high), "dvdq_gbs_init")
    return g


def dvdq_gbs_next_bits(g: GbsState) -> int:
    return int(load().dvdq_gbs_next_bits(C.byref(g)))


def dvdq_gbs_observe(g: GbsState, l1_change: float, l1_prev: float) -> None:
    _check(load().dvdq_gbs_observe(C.byref(g), float(l1_change), float(l1_prev)), "dvdq_gbs_observe")


def dvdq_last_device_status():
    """(status, detail) of the device-side status word; synchronizes the device and clears it."""
    d = C.c_uint32(0)
    s = load().dvdq_last_device_status(C.byref(d))
    return int(s), int(d.value)
