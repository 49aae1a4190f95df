"""ctypes front end of the RMSMP CPU oracle (TEST INFRASTRUCTURE, not a product path).

Only the test-suite, the smoke check and the benchmark's CPU-baseline leg import this
module.  It compiles ``rmsmp_oracle.c`` with gcc on first use and exposes its functions on
numpy arrays.  Nothing here touches the CUDA library.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "rmsmp_oracle.c")
_LIB = os.path.join(_HERE, "librmsmp_oracle.so")

SCHEME_POT, SCHEME_FIXED = 0, 1
ACT_U4, ACT_S4 = 0, 1
POT_NEAREST, POT_LOG2 = 0, 1


def build(force: bool = False) -> str:
    """Compile the oracle (gcc, -O2, no FMA contraction, OpenMP over rows/pixels)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".%d.tmp" % os.getpid()
        subprocess.check_call(
            ["gcc", "-O2", "-std=c99", "-ffp-contract=off", "-fopenmp", "-shared", "-fPIC",
             _SRC, "-lm", "-o", tmp])
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def lib() -> C.CDLL:
    global _lib
    if _lib is None:
        L = C.CDLL(build())
        L.rmsmp_o_fixed_q.argtypes = [C.c_float, C.c_float, C.c_int]
        L.rmsmp_o_pot_nibble.argtypes = [C.c_float, C.c_float, C.c_int]
        L.rmsmp_o_pot_value.argtypes = [C.c_int]
        L.rmsmp_o_wstep.argtypes = [C.c_float, C.c_int, C.c_int]
        L.rmsmp_o_wstep.restype = C.c_float
        L.rmsmp_o_row_variance.restype = C.c_double
        L.rmsmp_o_row_variance.argtypes = [C.c_void_p, C.c_int]
        _lib = L
    return _lib


def _p(a: np.ndarray) -> C.c_void_p:
    return C.c_void_p(a.ctypes.data)


def _c(a, dt) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=dt)


def fixed_q(w: float, alpha: float, bits: int) -> int:
    return lib().rmsmp_o_fixed_q(np.float32(w), np.float32(alpha), bits)


def pot_nibble(w: float, alpha: float, mode: int = POT_NEAREST) -> int:
    return lib().rmsmp_o_pot_nibble(np.float32(w), np.float32(alpha), mode)


def pot_value(nibble: int) -> int:
    return lib().rmsmp_o_pot_value(nibble)


def wstep(alpha: float, scheme: int, bits: int) -> np.float32:
    return np.float32(lib().rmsmp_o_wstep(np.float32(alpha), scheme, bits))


def quantize_rows(W, scheme, bits, alpha, pot_mode: int = POT_NEAREST):
    """W[M][K] fp32 -> (values int8 [M][K], wstep fp32 [M]).  Raises on an invalid menu/alpha."""
    W = _c(W, np.float32)
    M, K = W.shape
    scheme, bits, alpha = _c(scheme, np.uint8), _c(bits, np.uint8), _c(alpha, np.float32)
    values = np.empty((M, K), np.int8)
    ws = np.empty(M, np.float32)
    rc = lib().rmsmp_o_quantize_rows(_p(W), M, K, _p(scheme), _p(bits), _p(alpha), pot_mode,
                                     _p(values), _p(ws))
    if rc != 0:
        raise ValueError("invalid scheme/bits menu entry or alpha")
    return values, ws


def quantize_act(x, alpha_a: float, kind: int):
    """fp32 activations (any shape) -> (codes int8 same shape, act_step fp32)."""
    x = _c(x, np.float32)
    codes = np.empty(x.shape, np.int8)
    step = C.c_float(0)
    lib().rmsmp_o_quantize_act(_p(x), C.c_size_t(x.size), C.c_float(alpha_a), kind, _p(codes),
                               C.byref(step))
    return codes, np.float32(step.value)


def row_variance(w) -> float:
    w = _c(w, np.float32)
    return lib().rmsmp_o_row_variance(_p(w), w.size)


def ratio_counts(M: int, ratio):
    a, b, c = C.c_int(), C.c_int(), C.c_int()
    lib().rmsmp_o_ratio_counts(M, int(ratio[0]), int(ratio[1]), int(ratio[2]), C.byref(a),
                               C.byref(b), C.byref(c))
    return a.value, b.value, c.value


def assign_rows(W, ratio):
    """Scheme/precision map of a layer for ratio (PoT-4, Fixed-4, Fixed-8) -> (scheme, bits)."""
    W = _c(W, np.float32).reshape(W.shape[0], -1)
    M, K = W.shape
    scheme, bits = np.empty(M, np.uint8), np.empty(M, np.uint8)
    lib().rmsmp_o_assign_rows(_p(W), M, K, int(ratio[0]), int(ratio[1]), int(ratio[2]),
                              _p(scheme), _p(bits))
    return scheme, bits


def group_rows(scheme, bits) -> np.ndarray:
    scheme, bits = _c(scheme, np.uint8), _c(bits, np.uint8)
    perm = np.empty(scheme.size, np.int32)
    lib().rmsmp_o_group_rows(_p(scheme), _p(bits), scheme.size, _p(perm))
    return perm


def matmul(values, act) -> np.ndarray:
    """values[M][K] int8, act[N][K] int8 -> acc[N][M] int32."""
    values, act = _c(values, np.int8), _c(act, np.int8)
    M, K = values.shape
    N = act.shape[0]
    acc = np.empty((N, M), np.int32)
    lib().rmsmp_o_matmul(_p(values), _p(act), M, N, K, C.c_int64(K), _p(acc))
    return acc


def matmul_i64(values, act) -> np.ndarray:
    values, act = _c(values, np.int8), _c(act, np.int8)
    M, K = values.shape
    N = act.shape[0]
    acc = np.empty((N, M), np.int64)
    lib().rmsmp_o_matmul_i64(_p(values), _p(act), M, N, K, C.c_int64(K), _p(acc))
    return acc


def matmul_pot_shift(nibbles, act) -> np.ndarray:
    nibbles, act = _c(nibbles, np.uint8), _c(act, np.int8)
    M, K = nibbles.shape
    N = act.shape[0]
    acc = np.empty((N, M), np.int32)
    lib().rmsmp_o_matmul_pot_shift(_p(nibbles), _p(act), M, N, K, C.c_int64(K), _p(acc))
    return acc


def conv_out_hw(H, W, kh, kw, stride, pad):
    return (H + 2 * pad - kh) // stride + 1, (W + 2 * pad - kw) // stride + 1


def conv(values, act, stride: int, pad: int) -> np.ndarray:
    """values[M][Cin][kh][kw] int8, act[B][H][W][Cin] int8 -> acc[B][Ho][Wo][M] int32."""
    values, act = _c(values, np.int8), _c(act, np.int8)
    M, Cin, kh, kw = values.shape
    B, H, W, Ca = act.shape
    assert Ca == Cin
    Ho, Wo = conv_out_hw(H, W, kh, kw, stride, pad)
    acc = np.empty((B, Ho, Wo, M), np.int32)
    lib().rmsmp_o_conv(_p(values), _p(act), M, Cin, kh, kw, B, H, W, stride, pad, _p(acc))
    return acc


def im2col(act, kh: int, kw: int, stride: int, pad: int, ld: int | None = None) -> np.ndarray:
    """Patch matrix of act[B][H][W][C]: row (b, ho, wo) holds the kh x kw x C codes its output pixel sees, tap
    by tap with the channel fastest, zero outside the image and in the columns beyond kh*kw*C (up to ld).  A
    convolution is the matrix product of the filters, flattened in the same order, with these rows (the
    first layer of the networks of Section 4.1 is run that way)."""
    act = _c(act, np.int8)
    B, H, W, Cc = act.shape
    Ho, Wo = conv_out_hw(H, W, kh, kw, stride, pad)
    K = kh * kw * Cc
    cols = np.zeros((B, Ho, Wo, ld or K), np.int8)
    for b in range(B):
        for ho in range(Ho):
            for wo in range(Wo):
                for i in range(kh):
                    for j in range(kw):
                        y, x = ho * stride + i - pad, wo * stride + j - pad
                        if 0 <= y < H and 0 <= x < W:
                            cols[b, ho, wo, (i * kw + j) * Cc:(i * kw + j + 1) * Cc] = act[b, y, x]
    return cols.reshape(B * Ho * Wo, -1)


def conv_depthwise(values, act, stride: int, pad: int) -> np.ndarray:
    """values[C][kh][kw] int8, act[B][H][W][C] int8 -> acc[B][Ho][Wo][C] int32 (each channel with its own filter)."""
    values, act = _c(values, np.int8), _c(act, np.int8)
    Cc, kh, kw = values.shape
    B, H, W, Ca = act.shape
    assert Ca == Cc
    Ho, Wo = conv_out_hw(H, W, kh, kw, stride, pad)
    acc = np.empty((B, Ho, Wo, Cc), np.int32)
    lib().rmsmp_o_conv_depthwise(_p(values), _p(act), Cc, kh, kw, B, H, W, stride, pad, _p(acc))
    return acc


def conv_points(values, act, stride: int, pad: int, n_idx, r_idx) -> np.ndarray:
    values, act = _c(values, np.int8), _c(act, np.int8)
    M, Cin, kh, kw = values.shape
    B, H, W, _ = act.shape
    n_idx, r_idx = _c(n_idx, np.int64), _c(r_idx, np.int32)
    acc = np.empty(n_idx.size, np.int32)
    lib().rmsmp_o_conv_points(_p(values), _p(act), M, Cin, kh, kw, B, H, W, stride, pad,
                              _p(n_idx), _p(r_idx), C.c_int64(n_idx.size), _p(acc))
    return acc


def matmul_points(values, act, n_idx, r_idx) -> np.ndarray:
    values, act = _c(values, np.int8), _c(act, np.int8)
    K = values.shape[1]
    n_idx, r_idx = _c(n_idx, np.int64), _c(r_idx, np.int32)
    acc = np.empty(n_idx.size, np.int32)
    lib().rmsmp_o_matmul_points(_p(values), _p(act), K, C.c_int64(K), _p(n_idx), _p(r_idx),
                                C.c_int64(n_idx.size), _p(acc))
    return acc


def epilogue(acc, wstep_rows, act_step) -> np.ndarray:
    """acc[..., M] int32 -> y fp32 same shape: (float)acc * (wstep_r * act_step)."""
    acc = _c(acc, np.int32)
    M = acc.shape[-1]
    N = acc.size // M
    ws = _c(wstep_rows, np.float32)
    y = np.empty(acc.shape, np.float32)
    lib().rmsmp_o_epilogue(_p(acc), C.c_int64(N), M, _p(ws), C.c_float(act_step), _p(y))
    return y


def num_threads() -> int:
    return lib().rmsmp_o_num_threads()


def layer_linear(W, scheme, bits, alpha, act_codes, act_step, pot_mode=POT_NEAREST):
    """Whole linear layer: returns (values, wstep, acc[N][M], y[N][M])."""
    values, ws = quantize_rows(W, scheme, bits, alpha, pot_mode)
    acc = matmul(values, act_codes)
    return values, ws, acc, epilogue(acc, ws, act_step)


def layer_conv(W, scheme, bits, alpha, act_codes, act_step, stride, pad, pot_mode=POT_NEAREST):
    """Whole conv layer, W[M][Cin][kh][kw]: returns (values 4-D, wstep, acc, y) with NHWC-like [B][Ho][Wo][M]."""
    W = _c(W, np.float32)
    M = W.shape[0]
    values, ws = quantize_rows(W.reshape(M, -1), scheme, bits, alpha, pot_mode)
    values = values.reshape(W.shape)
    acc = conv(values, act_codes, stride, pad)
    return values, ws, acc, epilogue(acc, ws, act_step)
