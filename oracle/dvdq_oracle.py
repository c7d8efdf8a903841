"""ctypes front end of ``dvdq_oracle.c`` (TEST INFRASTRUCTURE ONLY).

The arithmetic lives in the C file, written from the paper (Sec. 3.1 Quant/DeQuant,
Sec. 3.2 Eq. 10).  This module only compiles it with gcc, marshals numpy arrays and
strings the steps together in the paper's order.  bf16 tensors are numpy ``uint16``
arrays holding the raw bits.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "dvdq_oracle.c")
_BUILD = os.path.join(_HERE, "_build")
_SO = os.path.join(_BUILD, "libdvdq_oracle.so")
_lock = threading.Lock()
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle (gcc -O2 -fopenmp) if the shared object is missing or stale."""
    os.makedirs(_BUILD, exist_ok=True)
    stale = force or (not os.path.exists(_SO)) or os.path.getmtime(_SO) < os.path.getmtime(_SRC)
    if stale:
        tmp = _SO + f".tmp{os.getpid()}"
        cmd = ["gcc", "-O2", "-std=c11", "-fopenmp", "-fPIC", "-shared", "-ffp-contract=off",
               "-o", tmp, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
        os.replace(tmp, _SO)
    return _SO


def _load():
    global _lib
    with _lock:
        if _lib is None:
            lib = C.CDLL(build())
            i64, p = C.c_int64, C.c_void_p
            lib.oracle_bf16_to_double.restype = C.c_double
            lib.oracle_bf16_to_double.argtypes = [C.c_uint16]
            lib.oracle_double_to_bf16.restype = C.c_uint16
            lib.oracle_double_to_bf16.argtypes = [C.c_double]
            lib.oracle_hadamard_matrix.restype = None
            lib.oracle_hadamard_matrix.argtypes = [i64, p]
            lib.oracle_rotate_rows.restype = C.c_int
            lib.oracle_rotate_rows.argtypes = [p, i64, i64, i64, i64, p]
            lib.oracle_act_quantize.restype = C.c_int
            lib.oracle_act_quantize.argtypes = [p, i64, i64, C.c_int, p, p, p]
            lib.oracle_weight_quantize_minmax.restype = None
            lib.oracle_weight_quantize_minmax.argtypes = [p, i64, i64, p, p, p]
            lib.oracle_weight_quantize_symmetric.restype = None
            lib.oracle_weight_quantize_symmetric.argtypes = [p, i64, i64, p, p, p]
            lib.oracle_bgr_quantize.restype = None
            lib.oracle_bgr_quantize.argtypes = [p, i64, i64, C.c_int, C.c_int, C.c_double, C.c_int, p, p, p, p]
            lib.oracle_minmax_row_error.restype = None
            lib.oracle_minmax_row_error.argtypes = [p, i64, i64, C.c_int, p]
            lib.oracle_int_gemm.restype = i64
            lib.oracle_int_gemm.argtypes = [p, p, p, i64, i64, i64, p]
            lib.oracle_gelu_tanh.restype = C.c_double
            lib.oracle_gelu_tanh.argtypes = [C.c_double]
            lib.oracle_epilogue.restype = None
            lib.oracle_epilogue.argtypes = [p, p, p, p, C.c_int, i64, i64, p]
            lib.oracle_round_output.restype = None
            lib.oracle_round_output.argtypes = [p, p, C.c_int, i64, i64, p]
            lib.oracle_exact_linear.restype = None
            lib.oracle_exact_linear.argtypes = [p, p, i64, i64, i64, p]
            _lib = lib
    return _lib


def _ptr(a: np.ndarray):
    return a.ctypes.data_as(C.c_void_p)


def _c(a, dtype) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=dtype)


def num_threads() -> int:
    """Threads the OpenMP loops of the oracle use (rows are spread over them)."""
    env = os.environ.get("OMP_NUM_THREADS")
    if env:
        return int(env)
    return len(os.sched_getaffinity(0)) if hasattr(os, "sched_getaffinity") else (os.cpu_count() or 1)


# ---------------------------------------------------------------- scalar helpers

def bf16_to_double(bits: int) -> float:
    return float(_load().oracle_bf16_to_double(int(bits)))


def double_to_bf16(v: float) -> int:
    return int(_load().oracle_double_to_bf16(float(v)))


def bf16_array_to_double(a: np.ndarray) -> np.ndarray:
    """Exact widening of raw bf16 bits (a bf16 is the top half of a binary32)."""
    a = _c(a, np.uint16)
    return (a.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def gelu_tanh(v: float) -> float:
    return float(_load().oracle_gelu_tanh(float(v)))


# ---------------------------------------------------------------- steps, in the paper's order

def hadamard(B: int) -> np.ndarray:
    """Orthonormal Sylvester Hadamard matrix H_B / sqrt(B) (closed-form entries)."""
    H = np.empty((B, B), dtype=np.float64)
    _load().oracle_hadamard_matrix(B, _ptr(H))
    return H


def rotate(x_bf16: np.ndarray, B: int) -> np.ndarray:
    """X~ = X (I (x) H_B/sqrt(B)) by the dense definition, fp64.  B = 0: no rotation."""
    x = _c(x_bf16, np.uint16)
    rows, K = x.shape
    out = np.empty((rows, K), dtype=np.float64)
    rc = _load().oracle_rotate_rows(_ptr(x), rows, K, K, B, _ptr(out))
    if rc != 0:
        raise ValueError(f"rotation block {B} invalid for K={K} (rc={rc})")
    return out


def act_quantize(xt: np.ndarray, bits: int):
    """Per-token absmax quantizer -> (codes int32 [M,K], scale fp64 [M], scale fp32 [M])."""
    xt = _c(xt, np.float64)
    rows, K = xt.shape
    codes = np.empty((rows, K), dtype=np.int32)
    s64 = np.empty(rows, dtype=np.float64)
    s32 = np.empty(rows, dtype=np.float32)
    rc = _load().oracle_act_quantize(_ptr(xt), rows, K, bits, _ptr(codes), _ptr(s64), _ptr(s32))
    if rc != 0:
        raise ValueError(f"bits={bits} unsupported")
    return codes, s64, s32


def rotate_quantize(x_bf16: np.ndarray, B: int, bits: int):
    """rotate -> auto-scale -> quantize; returns (codes, scale64, scale32, xt)."""
    xt = rotate(x_bf16, B)
    codes, s64, s32 = act_quantize(xt, bits)
    return codes, s64, s32, xt


def weight_quantize(wt: np.ndarray, mode: str = "symmetric"):
    """4-bit per-output-channel weight codes -> (u uint8 [N,K] in 0..15, delta fp32 [N], z int32 [N])."""
    wt = _c(wt, np.float64)
    N, K = wt.shape
    u = np.empty((N, K), dtype=np.uint8)
    d = np.empty(N, dtype=np.float32)
    z = np.empty(N, dtype=np.int32)
    fn = {"symmetric": _load().oracle_weight_quantize_symmetric,
          "minmax": _load().oracle_weight_quantize_minmax}[mode]
    fn(_ptr(wt), N, K, _ptr(u), _ptr(d), _ptr(z))
    return u, d, z


def bgr_quantize(wt: np.ndarray, bits: int = 4, n_steps: int = 100, eps: float = 1e-5, max_iter: int = 50):
    """Bounded-init Grid Refinement (Alg. 1) per output channel ->
    (u uint8 [N,K], delta fp64 [N], z int32 [N], err fp64 [N] = || w - Delta (u - z) ||_2 per row)."""
    wt = _c(wt, np.float64)
    N, K = wt.shape
    u = np.empty((N, K), dtype=np.uint8)
    d = np.empty(N, dtype=np.float64)
    z = np.empty(N, dtype=np.int32)
    e = np.empty(N, dtype=np.float64)
    _load().oracle_bgr_quantize(_ptr(wt), N, K, bits, n_steps, float(eps), max_iter, _ptr(u), _ptr(d), _ptr(z), _ptr(e))
    return u, d, z, e


def minmax_row_error(wt: np.ndarray, bits: int = 4) -> np.ndarray:
    """|| w - Delta (W_q - z) ||_2 per row for the plain MinMax grid of Sec. 3.1."""
    wt = _c(wt, np.float64)
    N, K = wt.shape
    e = np.empty(N, dtype=np.float64)
    _load().oracle_minmax_row_error(_ptr(wt), N, K, bits, _ptr(e))
    return e


def int_gemm(codes: np.ndarray, u: np.ndarray, z: np.ndarray) -> np.ndarray:
    """acc[i,n] = sum_k codes[i,k] * (u[n,k] - z[n]) in 64-bit, checked to fit int32."""
    c = _c(codes, np.int32)
    u = _c(u, np.uint8)
    z = _c(z, np.int32)
    M, K = c.shape
    N = u.shape[0]
    assert u.shape[1] == K and z.shape[0] == N
    acc = np.empty((M, N), dtype=np.int32)
    bad = _load().oracle_int_gemm(_ptr(c), _ptr(u), _ptr(z), M, N, K, _ptr(acc))
    if bad:
        raise OverflowError(f"{bad} accumulators do not fit int32")
    return acc


def epilogue(acc: np.ndarray, scale32: np.ndarray, delta32: np.ndarray, bias_bf16=None, act: int = 0) -> np.ndarray:
    """y = bf16(acc * s_i * Delta_n + bias_n) [then GELU-tanh and a second bf16 rounding if act == 1]."""
    acc = _c(acc, np.int32)
    M, N = acc.shape
    s = _c(scale32, np.float32)
    d = _c(delta32, np.float32)
    b = None if bias_bf16 is None else _c(bias_bf16, np.uint16)
    y = np.empty((M, N), dtype=np.uint16)
    _load().oracle_epilogue(_ptr(acc), _ptr(s), _ptr(d), None if b is None else _ptr(b), act, M, N, _ptr(y))
    return y


def round_output(v: np.ndarray, bias_bf16=None, act: int = 0) -> np.ndarray:
    """The tail of the epilogue on values already dequantized in fp64:
    y = bf16(v + bias_n) [then GELU-tanh and a second bf16 rounding if act == 1].  bf16 bits [M,N]."""
    v = _c(v, np.float64)
    M, N = v.shape
    b = None if bias_bf16 is None else _c(bias_bf16, np.uint16)
    y = np.empty((M, N), dtype=np.uint16)
    _load().oracle_round_output(_ptr(v), None if b is None else _ptr(b), act, M, N, _ptr(y))
    return y


def exact_linear(x: np.ndarray, w: np.ndarray) -> np.ndarray:
    """Y = X W^T in fp64 (the product the method approximates)."""
    x = _c(x, np.float64)
    w = _c(w, np.float64)
    M, K = x.shape
    N = w.shape[0]
    y = np.empty((M, N), dtype=np.float64)
    _load().oracle_exact_linear(_ptr(x), _ptr(w), M, N, K, _ptr(y))
    return y


def prepare_weights(w_bf16: np.ndarray, B: int, mode: str = "symmetric"):
    """Offline side of Eq. 10: W~ = W (I (x) H_B/sqrt(B)) along K, then 4-bit codes."""
    wt = rotate(w_bf16, B)
    return weight_quantize(wt, mode)


def qlinear(x_bf16, u, delta32, z, B: int, bits: int, bias_bf16=None, act: int = 0):
    """The whole hot path for already-prepared weights; returns a dict of every stage."""
    codes, s64, s32, xt = rotate_quantize(x_bf16, B, bits)
    acc = int_gemm(codes, u, z)
    y = epilogue(acc, s32, delta32, bias_bf16, act)
    return {"xt": xt, "codes": codes, "scale64": s64, "scale32": s32, "acc": acc, "y": y}


# ---------------------------------------------------------------- delta-guided bit switching (Sec. 3.3)

def gbs_l1_terms(F_t_bf16: np.ndarray, F_prev_bf16: np.ndarray):
    """(||F_t - F_{t-1}||_1, ||F_{t-1}||_1) in fp64 from raw bf16 bits: the two norms of
    L1(F, t) = ||F_t - F_{t-1}||_1 / ||F_{t-1}||_1  (Sec. 3.3)."""
    a = bf16_array_to_double(F_t_bf16).ravel()
    b = bf16_array_to_double(F_prev_bf16).ravel()
    assert a.shape == b.shape
    return float(np.abs(a - b).sum()), float(np.abs(b).sum())


def gbs_schedule(l1_values, delta: float, b_low: int, b_high: int):
    """Bit width of every step of a run, given L1(F, t) of each finished step, by the rule of
    Sec. 3.3: step i runs at b_low while the changes summed since the last reset stay below
    delta; once the sum reaches delta the step runs at b_high and the sum restarts from zero.
    l1_values[i] is the change measured after step i; the decision for step i only sees the
    values of earlier steps (the sum is empty, i.e. 0, before the first step).  Returns one
    entry per step, len(l1_values) + 1 decisions for len(l1_values) observed changes."""
    bits = []
    acc = 0.0
    for i in range(len(l1_values) + 1):
        if acc >= delta:
            bits.append(b_high)
            acc = 0.0
        else:
            bits.append(b_low)
        if i < len(l1_values):
            acc += float(l1_values[i])
    return bits


# ---------------------------------------------------------------- block-wise scales (Sec. 3.2, last paragraph)

def act_quantize_grouped(xt: np.ndarray, bits: int, group: int):
    """The block-wise variant of the auto-scaling: one absmax scale per token AND per block of
    `group` consecutive rotated channels (the quantizer of Eq. 10 applied to every block on its
    own).  Returns (codes int32 [M,K], scale fp64 [M,K/group], scale fp32 [M,K/group])."""
    xt = _c(xt, np.float64)
    M, K = xt.shape
    assert group > 0 and K % group == 0
    G = K // group
    codes = np.empty((M, K), dtype=np.int32)
    s64 = np.empty((M, G), dtype=np.float64)
    s32 = np.empty((M, G), dtype=np.float32)
    for g in range(G):
        c, a, b = act_quantize(xt[:, g * group:(g + 1) * group], bits)
        codes[:, g * group:(g + 1) * group] = c
        s64[:, g] = a
        s32[:, g] = b
    return codes, s64, s32


def combine_grouped(codes, u, z, s32, delta32, group: int, bias_bf16=None, act: int = 0) -> np.ndarray:
    """Given codes and block scales, the output of the layer with block-wise activation scales:
        y_in = bf16( Delta_n * sum_g s_ig * sum_{k in block g} c_ik (u_nk - z_n) + bias_n ),
    every block's integer GEMM on its own, combined in fp64 (scales and Delta are their stored
    binary32 values), then the same rounding / GELU as the per-token path.  bf16 bits [M,N]."""
    codes = _c(codes, np.int32)
    M, K = codes.shape
    N = u.shape[0]
    v = np.zeros((M, N), dtype=np.float64)
    for g in range(K // group):
        sl = slice(g * group, (g + 1) * group)
        acc = int_gemm(np.ascontiguousarray(codes[:, sl]), np.ascontiguousarray(u[:, sl]), z)
        v += acc.astype(np.float64) * s32[:, g].astype(np.float64)[:, None]
    v *= np.asarray(delta32, dtype=np.float32).astype(np.float64)[None, :]
    return round_output(v, bias_bf16, act)


def qlinear_grouped(x_bf16, u, delta32, z, B: int, bits: int, group: int, bias_bf16=None, act: int = 0):
    """The layer with block-wise activation scales: rotation, the block-wise quantizer, then
    combine_grouped."""
    xt = rotate(x_bf16, B)
    codes, s64, s32 = act_quantize_grouped(xt, bits, group)
    y = combine_grouped(codes, u, z, s32, delta32, group, bias_bf16, act)
    return {"xt": xt, "codes": codes, "scale64": s64, "scale32": s32, "y": y}
