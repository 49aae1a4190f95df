"""Host-side checks that need no GPU: the library loads, exports what the header declares,
validates its arguments before touching CUDA, and its host logic agrees with the oracle."""
import ctypes as C
import os
import re

import numpy as np
import pytest

from oracle import rmsmp_oracle as O
from paper_2111_00153_b200 import binding as R
from paper_2111_00153_b200 import build as B
from paper_2111_00153_b200 import synth

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def _built():
    B.build_library()


def test_library_exports_every_declared_symbol():
    hdr = open(os.path.join(ROOT, "include", "rmsmp.h")).read()
    declared = set(re.findall(r"\b(rmsmp_[a-z0-9_]+)\s*\(", hdr))
    assert declared, "no declarations found"
    assert declared == set(R.EXPORTS)
    lib = R.lib()
    for name in declared:
        assert hasattr(lib, name), name
    for name in R.EXPORTS:
        assert name in declared, name


def test_status_strings():
    seen = {R.rmsmp_status_string(i) for i in range(0, 12)}
    assert len(seen) == 12 and "ok" in seen


def test_assign_rows_matches_oracle_bit_for_bit():
    for idx, (M, K, ratio) in enumerate([(256, 512, (60, 35, 5)), (64, 576, (65, 30, 5)),
                                         (100, 33, (50, 40, 10)), (7, 5, (0, 100, 0)),
                                         (9, 12, (100, 0, 0))]):
        W = synth.weights_normal(synth.rng(90, idx), (M, K))
        s1, b1 = R.rmsmp_assign_rows(W, ratio)
        s2, b2 = O.assign_rows(W, ratio)
        assert np.array_equal(s1, s2) and np.array_equal(b1, b2)
    with pytest.raises(R.RmsmpError) as e:
        R.rmsmp_assign_rows(np.zeros((4, 4), np.float32), (50, 40, 5))
    assert e.value.status == R.ERR_SHAPE


def test_layer_init_layout():
    scheme = np.array([1, 0, 1, 0, 1, 0, 1], np.uint8)
    bits = np.array([4, 4, 8, 4, 4, 4, 8], np.uint8)
    L = R.rmsmp_layer_init(7, 70, 3, 3, scheme, bits)
    assert (L.nP, L.nF4, L.n8) == (3, 2, 2)
    assert L.Cp == 96 and L.Kp == 896 and L.nblocks == 1     # 9 taps * 96 = 864 -> 896
    offs = [L.off_perm, L.off_slot, L.off_wstep, L.off_alpha, L.off_kind, L.off_blocks, L.off_q4,
            L.off_q8, L.packed_bytes]
    assert all(o % 256 == 0 for o in offs) and offs == sorted(offs)
    assert L.off_q8 - L.off_q4 >= 5 * 896 // 2 and L.packed_bytes - L.off_q8 >= 2 * 896
    L2 = R.rmsmp_layer_init(300, 512, 1, 1, np.ones(300, np.uint8), np.full(300, 4, np.uint8))
    assert L2.nblocks == 3 and L2.Cp == 512 and L2.Kp == 512


def test_layer_init_rejects_bad_input():
    ok_s, ok_b = np.zeros(4, np.uint8), np.full(4, 4, np.uint8)
    for args, err in [((0, 8, 1, 1, ok_s, ok_b), R.ERR_SHAPE),
                      ((4, 0, 1, 1, ok_s, ok_b), R.ERR_SHAPE),
                      ((4, 1000001, 1, 1, ok_s, ok_b), R.ERR_SHAPE),
                      ((4, 8, 17, 1, ok_s, ok_b), R.ERR_SHAPE)]:
        layer = R.rmsmp_layer()
        st = R.lib().rmsmp_layer_init(C.byref(layer), *args[:4], C.c_void_p(args[4].ctypes.data),
                                      C.c_void_p(args[5].ctypes.data))
        assert st == err
    # PoT with 8 bits is not on the method's menu
    with pytest.raises(R.RmsmpError) as e:
        R.rmsmp_layer_init(4, 8, 1, 1, ok_s, np.array([4, 8, 4, 4], np.uint8))
    assert e.value.status == R.ERR_SCHEME
    with pytest.raises(R.RmsmpError) as e:
        R.rmsmp_layer_init(4, 8, 1, 1, np.array([0, 2, 0, 0], np.uint8), ok_b)
    assert e.value.status == R.ERR_SCHEME
    assert R.lib().rmsmp_layer_init(None, 4, 8, 1, 1, None, None) == R.ERR_NULL


def test_calls_validate_before_any_cuda_work():
    lib = R.lib()
    scheme, bits = np.array([0, 1, 1], np.uint8), np.array([4, 4, 8], np.uint8)
    L = R.rmsmp_layer_init(3, 64, 1, 1, scheme, bits)
    alpha = np.ones(3, np.float32)
    fake = C.c_void_p(0x10000)            # aligned, never dereferenced: validation fails first
    hp = lambda a: C.c_void_p(a.ctypes.data)

    def pack(layer=L, a=alpha, s=scheme, b=bits, dW=fake, dP=fake, nbytes=None, mode=0, layout=0):
        return lib.rmsmp_quantize_pack(dW, layout, C.byref(layer), hp(s), hp(b), hp(a), mode, dP,
                                       layer.packed_bytes if nbytes is None else nbytes, None)

    assert pack(dW=None) == R.ERR_NULL
    assert pack(a=np.array([1, 0, 1], np.float32)) == R.ERR_SCALE
    assert pack(a=np.array([1, np.inf, 1], np.float32)) == R.ERR_SCALE
    assert pack(a=np.array([1, np.nan, 1], np.float32)) == R.ERR_SCALE
    assert pack(a=np.array([1, -2, 1], np.float32)) == R.ERR_SCALE
    assert pack(b=np.array([8, 4, 8], np.uint8)) == R.ERR_SCHEME          # PoT-8
    assert pack(s=np.array([1, 1, 1], np.uint8)) == R.ERR_SCHEME          # differs from layer_init's map
    assert pack(nbytes=16) == R.ERR_BUFFER_TOO_SMALL
    assert pack(dW=C.c_void_p(0x10004)) == R.ERR_ALIGN
    assert pack(dP=C.c_void_p(0x10010)) == R.ERR_ALIGN
    assert pack(layout=1, layer=R.rmsmp_layer()) == R.ERR_BAD_LAYER
    assert pack(mode=7) == R.ERR_SCHEME

    step = C.c_float()
    assert lib.rmsmp_quantize_act(fake, 0, 1.0, 0, fake, C.byref(step), None) == R.ERR_SHAPE
    assert lib.rmsmp_quantize_act(fake, 8, 0.0, 0, fake, C.byref(step), None) == R.ERR_SCALE
    assert lib.rmsmp_quantize_act(None, 8, 1.0, 0, fake, C.byref(step), None) == R.ERR_NULL

    def gemm(N=8, ld=64, act=fake, out=fake, ld_out=3, layout=0, layer=L, packed=fake):
        return lib.rmsmp_gemm(C.byref(layer), packed, act, N, ld, 1.0, out, ld_out, layout, None, None)

    assert gemm(act=None) == R.ERR_NULL
    assert gemm(N=0) == R.ERR_SHAPE
    assert gemm(ld=48) == R.ERR_SHAPE          # shorter than K
    assert gemm(ld=72) == R.ERR_ALIGN          # not a multiple of 16
    assert gemm(ld_out=2) == R.ERR_SHAPE
    assert gemm(layout=1, ld_out=7) == R.ERR_SHAPE
    assert gemm(act=C.c_void_p(0x10001)) == R.ERR_ALIGN
    assert gemm(layer=R.rmsmp_layer()) == R.ERR_BAD_LAYER
    Lc = R.rmsmp_layer_init(3, 16, 3, 3, scheme, bits)
    assert gemm(layer=Lc) == R.ERR_SHAPE       # a conv layer is not a linear layer

    def conv(B=1, H=8, W=8, stride=1, pad=1, act=fake, layer=Lc):
        return lib.rmsmp_conv_implicit(C.byref(layer), fake, act, B, H, W, stride, pad, 1.0, fake, 0,
                                       None, None)

    assert conv(B=0) == R.ERR_SHAPE
    assert conv(stride=0) == R.ERR_SHAPE
    assert conv(H=1, pad=0) == R.ERR_SHAPE     # kernel larger than padded image
    assert conv(act=None) == R.ERR_NULL
    assert lib.rmsmp_last_device_status(None, None) == R.ERR_NULL


def test_no_gpu_means_loud_failure_not_fallback():
    import torch
    if torch.cuda.is_available():
        pytest.skip("GPU present")
    lib = R.lib()
    step = C.c_float()
    st = lib.rmsmp_quantize_act(C.c_void_p(0x10000), 16, 1.0, 0, C.c_void_p(0x20000), C.byref(step), None)
    assert st in (R.ERR_CUDA, R.ERR_ARCH)
