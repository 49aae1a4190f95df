"""Thin ctypes binding of librmsmp.so: same names as include/rmsmp.h, argument marshalling only.

Device buffers are torch CUDA tensors (or raw integer device pointers); torch is used for
memory and streams, every step of the computation runs in the library's kernels.  There is no
CPU fallback: if the library cannot be loaded, every call raises.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "librmsmp.so")

# enums of rmsmp.h
OK = 0
SCHEME_POT, SCHEME_FIXED = 0, 1
ACT_U4, ACT_S4 = 0, 1
POT_NEAREST, POT_LOG2 = 0, 1
OUT_NM, OUT_MN = 0, 1
W_LINEAR, W_CONV_OIHW = 0, 1
VARIANT_AUTO, VARIANT_TENSOR, VARIANT_SIMT, VARIANT_SHIFTADD, VARIANT_SIMPLE = 0, 1, 2, 3, 4
(ERR_NULL, ERR_SHAPE, ERR_SCHEME, ERR_SCALE, ERR_ALIGN, ERR_BUFFER_TOO_SMALL, ERR_ARCH, ERR_CUDA,
 ERR_TIMEOUT, ERR_BAD_LAYER, ERR_VARIANT) = range(1, 12)

EXPORTS = (
    "rmsmp_status_string", "rmsmp_assign_rows", "rmsmp_layer_init", "rmsmp_quantize_pack",
    "rmsmp_unpack_codes", "rmsmp_quantize_act", "rmsmp_gemm", "rmsmp_gemm_variant",
    "rmsmp_conv_implicit", "rmsmp_conv_implicit_variant", "rmsmp_last_device_status",
    "rmsmp_measure_mma_peak", "rmsmp_workspace_bytes", "rmsmp_expand_weights", "rmsmp_gemm_workspace",
    "rmsmp_conv_implicit_workspace", "rmsmp_gemm_builtin_scratch", "rmsmp_grouped_table_bytes",
    "rmsmp_gemm_grouped", "rmsmp_gemm_workspace_requant", "rmsmp_conv_implicit_workspace_requant",
    "rmsmp_conv_depthwise", "rmsmp_im2col_codes", "rmsmp_layer_init_ratio", "rmsmp_assign_scratch_bytes", "rmsmp_assign_quantize_pack", "rmsmp_selftest_bounded_wait", "rmsmp_grouped_plan_bytes", "rmsmp_gemm_grouped_prepare", "rmsmp_gemm_grouped_launch",
)


class rmsmp_layer(C.Structure):
    _fields_ = [
        ("magic", C.c_uint32),
        ("M", C.c_int32), ("Cin", C.c_int32), ("kh", C.c_int32), ("kw", C.c_int32),
        ("Cp", C.c_int32), ("Kp", C.c_int32),
        ("nP", C.c_int32), ("nF4", C.c_int32), ("n8", C.c_int32),
        ("nblocks", C.c_int32), ("raw_stage_bytes", C.c_int32),
        ("off_perm", C.c_uint64), ("off_slot", C.c_uint64), ("off_wstep", C.c_uint64),
        ("off_alpha", C.c_uint64), ("off_kind", C.c_uint64), ("off_blocks", C.c_uint64),
        ("off_q4", C.c_uint64), ("off_q8", C.c_uint64),
        ("packed_bytes", C.c_uint64),
    ]

    @property
    def K(self) -> int:
        return self.Cin * self.kh * self.kw


class rmsmp_gemm_item(C.Structure):
    _fields_ = [
        ("layer", C.POINTER(rmsmp_layer)), ("d_packed", C.c_void_p), ("d_act", C.c_void_p),
        ("N", C.c_int64), ("ld_act", C.c_int64), ("act_step", C.c_float),
        ("d_out", C.c_void_p), ("ld_out", C.c_int64), ("d_acc", C.c_void_p), ("act_nonneg", C.c_int32),
    ]


class rmsmp_grouped_plan(C.Structure):
    _fields_ = [
        ("magic", C.c_uint32), ("count", C.c_int32), ("grid", C.c_int32), ("smem_bytes", C.c_uint32),
        ("device", C.c_int32), ("conv_grid", C.c_int32), ("d_table", C.c_void_p), ("table_bytes", C.c_uint64),
    ]


class RmsmpError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        try:
            msg = lib().rmsmp_status_string(status).decode()
        except Exception:
            msg = "?"
        super().__init__(f"{where}: status {status} ({msg})")


_lib = None


def lib() -> C.CDLL:
    """Load the CUDA library; fails loudly if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(
                f"{LIB_PATH} is missing: build it with `python -m paper_2111_00153_b200.build` "
                "(there is no CPU fallback)")
        L = C.CDLL(LIB_PATH)
        L.rmsmp_status_string.restype = C.c_char_p
        L.rmsmp_status_string.argtypes = [C.c_int]
        vp, i32, i64, f32 = C.c_void_p, C.c_int, C.c_int64, C.c_float
        L.rmsmp_assign_rows.argtypes = [vp, i32, i32, i32, i32, i32, vp, vp]
        L.rmsmp_layer_init.argtypes = [C.POINTER(rmsmp_layer), i32, i32, i32, i32, vp, vp]
        L.rmsmp_quantize_pack.argtypes = [vp, i32, C.POINTER(rmsmp_layer), vp, vp, vp, i32, vp,
                                          C.c_size_t, vp]
        L.rmsmp_unpack_codes.argtypes = [C.POINTER(rmsmp_layer), vp, vp, vp, vp, vp]
        L.rmsmp_quantize_act.argtypes = [vp, C.c_size_t, f32, i32, vp, C.POINTER(C.c_float), vp]
        L.rmsmp_gemm.argtypes = [C.POINTER(rmsmp_layer), vp, vp, i64, i64, f32, vp, i64, i32, vp, vp]
        L.rmsmp_gemm_variant.argtypes = [C.POINTER(rmsmp_layer), vp, vp, i64, i64, f32, vp, i64,
                                         i32, vp, i32, vp]
        L.rmsmp_conv_implicit.argtypes = [C.POINTER(rmsmp_layer), vp, vp, i32, i32, i32, i32, i32,
                                          f32, vp, i32, vp, vp]
        L.rmsmp_conv_implicit_variant.argtypes = [C.POINTER(rmsmp_layer), vp, vp, i32, i32, i32,
                                                  i32, i32, f32, vp, i32, vp, i32, vp]
        L.rmsmp_last_device_status.argtypes = [vp, vp]
        L.rmsmp_workspace_bytes.argtypes = [C.POINTER(rmsmp_layer), C.POINTER(C.c_size_t)]
        L.rmsmp_expand_weights.argtypes = [C.POINTER(rmsmp_layer), vp, vp, C.c_size_t, vp]
        L.rmsmp_gemm_workspace.argtypes = [C.POINTER(rmsmp_layer), vp, vp, vp, i64, i64, f32, vp, i64, i32, vp, vp]
        L.rmsmp_grouped_table_bytes.argtypes = [i32, C.POINTER(C.c_size_t)]
        L.rmsmp_gemm_grouped.argtypes = [C.POINTER(rmsmp_gemm_item), i32, i32, vp, C.c_size_t, vp]
        L.rmsmp_grouped_plan_bytes.argtypes = [C.POINTER(rmsmp_gemm_item), i32, C.POINTER(C.c_size_t)]
        L.rmsmp_gemm_grouped_prepare.argtypes = [C.POINTER(rmsmp_gemm_item), i32, i32, vp, C.c_size_t,
                                                 C.POINTER(rmsmp_grouped_plan), vp]
        L.rmsmp_gemm_grouped_launch.argtypes = [C.POINTER(rmsmp_grouped_plan), vp]
        L.rmsmp_gemm_builtin_scratch.argtypes = [C.POINTER(rmsmp_layer), vp, vp, i64, i64, f32, vp, i64, i32, vp, vp]
        L.rmsmp_conv_implicit_workspace.argtypes = [C.POINTER(rmsmp_layer), vp, vp, vp, i32, i32, i32, i32, i32,
                                                    f32, vp, i32, vp, vp]
        L.rmsmp_gemm_workspace_requant.argtypes = [C.POINTER(rmsmp_layer), vp, vp, vp, i64, i64, f32, f32, i32, vp, i64,
                                                   C.POINTER(C.c_float), vp]
        L.rmsmp_conv_implicit_workspace_requant.argtypes = [C.POINTER(rmsmp_layer), vp, vp, vp, i32, i32, i32, i32, i32,
                                                            f32, f32, i32, vp, C.POINTER(C.c_float), vp]
        L.rmsmp_conv_depthwise.argtypes = [C.POINTER(rmsmp_layer), vp, vp, i32, i32, i32, i32, i32, f32, vp, vp, vp]
        L.rmsmp_im2col_codes.argtypes = [vp, i32, i32, i32, i32, C.c_int64, i32, i32, i32, i32, vp, C.c_int64, vp]
        L.rmsmp_layer_init_ratio.argtypes = [C.POINTER(rmsmp_layer), i32, i32, i32, i32, i32, i32, i32]
        L.rmsmp_assign_scratch_bytes.argtypes = [i32, C.POINTER(C.c_size_t)]
        L.rmsmp_assign_quantize_pack.argtypes = [vp, i32, C.POINTER(rmsmp_layer), i32, i32, i32, vp, i32, vp, C.c_size_t,
                                                 vp, C.c_size_t, vp, vp, vp]
        L.rmsmp_selftest_bounded_wait.argtypes = [i64, vp, vp]
        L.rmsmp_measure_mma_peak.argtypes = [i32, i32, i32, vp, C.POINTER(C.c_float), C.POINTER(C.c_float), vp]
        _lib = L
    return _lib


def _dp(t):
    """Device pointer of a torch tensor, or pass an int / None through."""
    if t is None:
        return None
    if isinstance(t, int):
        return C.c_void_p(t)
    return C.c_void_p(t.data_ptr())


def _hp(a: np.ndarray):
    return C.c_void_p(a.ctypes.data)


def _stream(stream):
    if stream is None:
        import torch
        return C.c_void_p(torch.cuda.current_stream().cuda_stream)
    if isinstance(stream, int):
        return C.c_void_p(stream)
    return C.c_void_p(stream.cuda_stream)


def _check(st: int, where: str):
    if st != OK:
        raise RmsmpError(st, where)


def rmsmp_status_string(status: int) -> str:
    return lib().rmsmp_status_string(status).decode()


def rmsmp_assign_rows(h_W: np.ndarray, ratio):
    """Host helper: (scheme, bits) uint8 arrays for ratio (PoT-4, Fixed-4, Fixed-8)."""
    W = np.ascontiguousarray(h_W, dtype=np.float32)
    W = W.reshape(W.shape[0], -1)
    M, K = W.shape
    scheme, bits = np.empty(M, np.uint8), np.empty(M, np.uint8)
    _check(lib().rmsmp_assign_rows(_hp(W), M, K, int(ratio[0]), int(ratio[1]), int(ratio[2]),
                                   _hp(scheme), _hp(bits)), "rmsmp_assign_rows")
    return scheme, bits


def rmsmp_layer_init(M: int, Cin: int, kh: int, kw: int, h_scheme, h_bits) -> rmsmp_layer:
    scheme = np.ascontiguousarray(h_scheme, dtype=np.uint8)
    bits = np.ascontiguousarray(h_bits, dtype=np.uint8)
    if scheme.size != M or bits.size != M:
        raise ValueError("scheme/bits need M entries")
    layer = rmsmp_layer()
    _check(lib().rmsmp_layer_init(C.byref(layer), M, Cin, kh, kw, _hp(scheme), _hp(bits)),
           "rmsmp_layer_init")
    return layer


def rmsmp_quantize_pack(d_W, w_layout: int, layer: rmsmp_layer, h_scheme, h_bits, h_alpha,
                        pot_mode: int, d_packed, packed_bytes: int | None = None, stream=None):
    scheme = np.ascontiguousarray(h_scheme, dtype=np.uint8)
    bits = np.ascontiguousarray(h_bits, dtype=np.uint8)
    alpha = np.ascontiguousarray(h_alpha, dtype=np.float32)
    if not (scheme.size == bits.size == alpha.size == layer.M):
        raise ValueError("scheme/bits/alpha need M entries")
    if packed_bytes is None:
        packed_bytes = d_packed.numel() * d_packed.element_size()
    _check(lib().rmsmp_quantize_pack(_dp(d_W), w_layout, C.byref(layer), _hp(scheme), _hp(bits),
                                     _hp(alpha), pot_mode, _dp(d_packed), packed_bytes,
                                     _stream(stream)), "rmsmp_quantize_pack")


def rmsmp_unpack_codes(layer: rmsmp_layer, d_packed, d_values, d_perm=None, d_wstep=None,
                       stream=None):
    _check(lib().rmsmp_unpack_codes(C.byref(layer), _dp(d_packed), _dp(d_values), _dp(d_perm),
                                    _dp(d_wstep), _stream(stream)), "rmsmp_unpack_codes")


def rmsmp_quantize_act(d_X, count: int, alpha_a: float, kind: int, d_codes, stream=None) -> float:
    """Returns the activation step (alpha_a/15 or alpha_a/7) as a Python float (fp32 value)."""
    step = C.c_float(0.0)
    _check(lib().rmsmp_quantize_act(_dp(d_X), count, alpha_a, kind, _dp(d_codes), C.byref(step),
                                    _stream(stream)), "rmsmp_quantize_act")
    return step.value


def rmsmp_gemm(layer, d_packed, d_act, N: int, ld_act: int, act_step: float, d_out, ld_out: int,
               out_layout: int = OUT_NM, d_acc=None, stream=None):
    _check(lib().rmsmp_gemm(C.byref(layer), _dp(d_packed), _dp(d_act), N, ld_act, act_step,
                            _dp(d_out), ld_out, out_layout, _dp(d_acc), _stream(stream)),
           "rmsmp_gemm")


def rmsmp_gemm_variant(layer, d_packed, d_act, N: int, ld_act: int, act_step: float, d_out,
                       ld_out: int, out_layout: int, d_acc, variant: int, stream=None):
    _check(lib().rmsmp_gemm_variant(C.byref(layer), _dp(d_packed), _dp(d_act), N, ld_act, act_step,
                                    _dp(d_out), ld_out, out_layout, _dp(d_acc), variant,
                                    _stream(stream)), "rmsmp_gemm_variant")


def rmsmp_conv_implicit(layer, d_packed, d_act, B: int, H: int, W: int, stride: int, pad: int,
                        act_step: float, d_out, out_layout: int = OUT_NM, d_acc=None, stream=None):
    _check(lib().rmsmp_conv_implicit(C.byref(layer), _dp(d_packed), _dp(d_act), B, H, W, stride,
                                     pad, act_step, _dp(d_out), out_layout, _dp(d_acc),
                                     _stream(stream)), "rmsmp_conv_implicit")


def rmsmp_conv_implicit_variant(layer, d_packed, d_act, B: int, H: int, W: int, stride: int,
                                pad: int, act_step: float, d_out, out_layout: int, d_acc,
                                variant: int, stream=None):
    _check(lib().rmsmp_conv_implicit_variant(C.byref(layer), _dp(d_packed), _dp(d_act), B, H, W,
                                             stride, pad, act_step, _dp(d_out), out_layout,
                                             _dp(d_acc), variant, _stream(stream)),
           "rmsmp_conv_implicit_variant")


def rmsmp_gemm_workspace_requant(layer, d_packed, d_workspace, d_act, N: int, ld_act: int, act_step: float,
                                 next_alpha: float, next_kind: int, d_next_codes, ld_codes: int, stream=None) -> float:
    """Linear layer whose epilogue writes the next layer's 4-bit activation codes; returns their step."""
    step = C.c_float(0.0)
    _check(lib().rmsmp_gemm_workspace_requant(C.byref(layer), _dp(d_packed), _dp(d_workspace), _dp(d_act), N, ld_act,
                                              act_step, next_alpha, next_kind, _dp(d_next_codes), ld_codes,
                                              C.byref(step), _stream(stream)), "rmsmp_gemm_workspace_requant")
    return step.value


def rmsmp_conv_implicit_workspace_requant(layer, d_packed, d_workspace, d_act, B: int, H: int, W: int, stride: int,
                                          pad: int, act_step: float, next_alpha: float, next_kind: int,
                                          d_next_codes, stream=None) -> float:
    step = C.c_float(0.0)
    _check(lib().rmsmp_conv_implicit_workspace_requant(C.byref(layer), _dp(d_packed), _dp(d_workspace), _dp(d_act),
                                                       B, H, W, stride, pad, act_step, next_alpha, next_kind,
                                                       _dp(d_next_codes), C.byref(step), _stream(stream)),
           "rmsmp_conv_implicit_workspace_requant")
    return step.value


def rmsmp_workspace_bytes(layer) -> int:
    n = C.c_size_t(0)
    _check(lib().rmsmp_workspace_bytes(C.byref(layer), C.byref(n)), "rmsmp_workspace_bytes")
    return n.value


def rmsmp_expand_weights(layer, d_packed, d_workspace, workspace_bytes: int | None = None, stream=None):
    if workspace_bytes is None:
        workspace_bytes = d_workspace.numel() * d_workspace.element_size()
    _check(lib().rmsmp_expand_weights(C.byref(layer), _dp(d_packed), _dp(d_workspace), workspace_bytes,
                                      _stream(stream)), "rmsmp_expand_weights")


def rmsmp_gemm_workspace(layer, d_packed, d_workspace, d_act, N: int, ld_act: int, act_step: float,
                         d_out, ld_out: int, out_layout: int = OUT_NM, d_acc=None, stream=None):
    _check(lib().rmsmp_gemm_workspace(C.byref(layer), _dp(d_packed), _dp(d_workspace), _dp(d_act), N,
                                      ld_act, act_step, _dp(d_out), ld_out, out_layout, _dp(d_acc),
                                      _stream(stream)), "rmsmp_gemm_workspace")


def rmsmp_conv_implicit_workspace(layer, d_packed, d_workspace, d_act, B: int, H: int, W: int,
                                  stride: int, pad: int, act_step: float, d_out,
                                  out_layout: int = OUT_NM, d_acc=None, stream=None):
    _check(lib().rmsmp_conv_implicit_workspace(C.byref(layer), _dp(d_packed), _dp(d_workspace), _dp(d_act),
                                               B, H, W, stride, pad, act_step, _dp(d_out), out_layout,
                                               _dp(d_acc), _stream(stream)), "rmsmp_conv_implicit_workspace")


def rmsmp_gemm_builtin_scratch(layer, d_packed, d_act, N: int, ld_act: int, act_step: float, d_out,
                               ld_out: int, out_layout: int = OUT_NM, d_acc=None, stream=None):
    """Linear layer through the library's own 4 MiB scratch array: allocates nothing.  For callers
    that may not call cudaMalloc; calls must not overlap on the GPU (they share the array)."""
    _check(lib().rmsmp_gemm_builtin_scratch(C.byref(layer), _dp(d_packed), _dp(d_act), N, ld_act,
                                            act_step, _dp(d_out), ld_out, out_layout, _dp(d_acc),
                                            _stream(stream)), "rmsmp_gemm_builtin_scratch")


def rmsmp_grouped_table_bytes(count: int) -> int:
    n = C.c_size_t(0)
    _check(lib().rmsmp_grouped_table_bytes(count, C.byref(n)), "rmsmp_grouped_table_bytes")
    return n.value


def make_gemm_items(items):
    """items: iterable of (layer, d_packed, d_act, N, ld_act, act_step, d_out, ld_out, d_acc|None[, act_nonneg])
    -> ctypes array of rmsmp_gemm_item (keep the layers alive while it is in use)."""
    items = list(items)
    arr = (rmsmp_gemm_item * len(items))()
    for k, item in enumerate(items):
        layer, pk, act, N, ld_act, step, out, ld_out, acc = item[:9]
        arr[k].act_nonneg = int(item[9]) if len(item) > 9 else 0
        arr[k].layer = C.pointer(layer)
        arr[k].d_packed = pk.data_ptr(); arr[k].d_act = act.data_ptr()
        arr[k].N = N; arr[k].ld_act = ld_act; arr[k].act_step = step
        arr[k].d_out = out.data_ptr(); arr[k].ld_out = ld_out
        arr[k].d_acc = acc.data_ptr() if acc is not None else None
    return arr


def rmsmp_gemm_grouped(items_array, out_layout: int, d_table, table_bytes: int | None = None, stream=None):
    if table_bytes is None:
        table_bytes = d_table.numel() * d_table.element_size()
    _check(lib().rmsmp_gemm_grouped(items_array, len(items_array), out_layout, _dp(d_table), table_bytes,
                                    _stream(stream)), "rmsmp_gemm_grouped")


def rmsmp_grouped_plan_bytes(items_array) -> int:
    n = C.c_size_t(0)
    _check(lib().rmsmp_grouped_plan_bytes(items_array, len(items_array), C.byref(n)), "rmsmp_grouped_plan_bytes")
    return n.value


def rmsmp_gemm_grouped_prepare(items_array, out_layout: int, d_table, table_bytes: int | None = None, stream=None):
    """Builds the tensor-core grouped launch of these layers into d_table; returns the plan to launch."""
    if table_bytes is None:
        table_bytes = d_table.numel() * d_table.element_size()
    plan = rmsmp_grouped_plan()
    _check(lib().rmsmp_gemm_grouped_prepare(items_array, len(items_array), out_layout, _dp(d_table), table_bytes,
                                            C.byref(plan), _stream(stream)), "rmsmp_gemm_grouped_prepare")
    return plan


def rmsmp_gemm_grouped_launch(plan, stream=None):
    _check(lib().rmsmp_gemm_grouped_launch(C.byref(plan), _stream(stream)), "rmsmp_gemm_grouped_launch")


def rmsmp_last_device_status(d_packed, stream=None) -> int:
    return lib().rmsmp_last_device_status(_dp(d_packed), _stream(stream))


def rmsmp_conv_depthwise(layer, d_packed, d_act, B: int, H: int, W: int, stride: int, pad: int, act_step: float,
                         d_out, d_acc=None, stream=None):
    _check(lib().rmsmp_conv_depthwise(C.byref(layer), _dp(d_packed), _dp(d_act), B, H, W, stride, pad, act_step,
                                      _dp(d_out), _dp(d_acc), _stream(stream)), "rmsmp_conv_depthwise")


def rmsmp_im2col_codes(d_act, B: int, H: int, W: int, Cc: int, pix_pitch: int, kh: int, kw: int, stride: int, pad: int,
                       d_cols, ld_cols: int, stream=None):
    _check(lib().rmsmp_im2col_codes(_dp(d_act), B, H, W, Cc, pix_pitch, kh, kw, stride, pad, _dp(d_cols), ld_cols,
                                    _stream(stream)), "rmsmp_im2col_codes")


def rmsmp_layer_init_ratio(M: int, Cin: int, kh: int, kw: int, ratio) -> rmsmp_layer:
    layer = rmsmp_layer()
    _check(lib().rmsmp_layer_init_ratio(C.byref(layer), M, Cin, kh, kw, int(ratio[0]), int(ratio[1]), int(ratio[2])),
           "rmsmp_layer_init_ratio")
    return layer


def rmsmp_assign_scratch_bytes(M: int) -> int:
    n = C.c_size_t(0)
    _check(lib().rmsmp_assign_scratch_bytes(M, C.byref(n)), "rmsmp_assign_scratch_bytes")
    return n.value


def rmsmp_assign_quantize_pack(d_W, w_layout: int, layer, ratio, d_alpha, pot_mode: int, d_packed, d_scratch,
                               d_scheme=None, d_bits=None, stream=None):
    """Row assignment on the device + quantize + pack, from the ratio alone."""
    _check(lib().rmsmp_assign_quantize_pack(_dp(d_W), w_layout, C.byref(layer), int(ratio[0]), int(ratio[1]), int(ratio[2]),
                                            _dp(d_alpha), pot_mode, _dp(d_packed), d_packed.numel() * d_packed.element_size(),
                                            _dp(d_scratch), d_scratch.numel() * d_scratch.element_size(), _dp(d_scheme),
                                            _dp(d_bits), _stream(stream)), "rmsmp_assign_quantize_pack")


def rmsmp_selftest_bounded_wait(limit_cycles: int, d_status_word, stream=None):
    """Launches the one-warp kernel whose bounded wait must run out; the status word then holds ERR_TIMEOUT."""
    _check(lib().rmsmp_selftest_bounded_wait(limit_cycles, _dp(d_status_word), _stream(stream)),
           "rmsmp_selftest_bounded_wait")


def rmsmp_measure_mma_peak(d_status_word, use_bf16: bool = False, n_cols: int = 256,
                           iters: int = 20000, stream=None):
    """Tensor-pipe ceiling for the kernel's MMA shape: returns (tera-ops per second, milliseconds)."""
    tops, ms = C.c_float(0.0), C.c_float(0.0)
    _check(lib().rmsmp_measure_mma_peak(1 if use_bf16 else 0, n_cols, iters, _dp(d_status_word),
                                        C.byref(tops), C.byref(ms), _stream(stream)),
           "rmsmp_measure_mma_peak")
    return tops.value, ms.value
