"""GPU parity: every step of the CUDA path against the CPU oracle, through the C ABI.

Integer results (codes, permutation, accumulators) must match bit for bit; fp32 outputs are a
single multiply of exactly converted integers and must match bit for bit too, and lie within
1e-6 relative of the double-precision value.
"""
import numpy as np
import pytest

from oracle import rmsmp_oracle as O
from paper_2111_00153_b200 import binding as R
from paper_2111_00153_b200 import synth
from tests import harness as Hn

pytestmark = pytest.mark.gpu

VARIANTS = [R.VARIANT_SIMPLE, R.VARIANT_SIMT, R.VARIANT_SHIFTADD, R.VARIANT_TENSOR, Hn.WORKSPACE]
VNAME = {R.VARIANT_SIMPLE: "simple", R.VARIANT_SIMT: "simt", R.VARIANT_SHIFTADD: "shiftadd",
         R.VARIANT_TENSOR: "tensor", R.VARIANT_AUTO: "auto", Hn.WORKSPACE: "workspace"}


def _mixed_map(M, seed, ratio=(60, 35, 5)):
    """A scheme map with the given ratio, rows shuffled (independent of weight values)."""
    nP, nF4, n8 = O.ratio_counts(M, ratio)
    kinds = np.array([0] * nP + [1] * nF4 + [2] * n8)
    np.random.default_rng(seed).shuffle(kinds)
    scheme = np.where(kinds == 0, 0, 1).astype(np.uint8)
    bits = np.where(kinds == 2, 8, 4).astype(np.uint8)
    return scheme, bits


def _check_layer_outputs(y, acc, acc_ref, ws, act_step, alpha, scheme, bits):
    assert np.array_equal(acc, acc_ref)
    y_ref = O.epilogue(acc_ref, ws, act_step)
    assert np.array_equal(y.view(np.uint32), y_ref.view(np.uint32))
    Qw = np.where(scheme == 0, 64.0, np.where(bits == 4, 7.0, 127.0))
    dbl = acc_ref.astype(np.float64) * (alpha.astype(np.float64) / Qw)[None, :] * float(act_step)
    nz = dbl != 0
    assert np.all(np.abs(y[nz] - dbl[nz]) <= 1e-6 * np.abs(dbl[nz]))


# ------------------------------------------------------------------ pack / unpack

@pytest.mark.parametrize("M,K,ratio", [(256, 512, (60, 35, 5)), (37, 200, (50, 40, 10)),
                                       (5, 3, (0, 100, 0)), (130, 1000, (100, 0, 0)),
                                       (64, 40000, (60, 35, 5)), (3, 7, (34, 33, 33))])
@pytest.mark.parametrize("mode", [R.POT_NEAREST, R.POT_LOG2])
def test_pack_codes_linear(M, K, ratio, mode):
    if mode == R.POT_LOG2 and K > 2000:
        pytest.skip("one large case per mode is enough")
    W = synth.weights_normal(synth.rng(70, M + K), (M, K))
    W[0, :min(K, 8)] = [0, 1e-9, -1e-9, 1, -1, 0.02, -0.02, 3e-4][:min(K, 8)]
    scheme, bits = O.assign_rows(W, ratio)
    alpha = synth.alpha_rows(W)
    layer, d_packed = Hn.pack_layer(W, scheme, bits, alpha, mode)
    vals, perm, ws = Hn.unpack(layer, d_packed)
    v_ref, ws_ref = O.quantize_rows(W, scheme, bits, alpha, mode)
    assert np.array_equal(vals, v_ref)
    assert np.array_equal(perm, O.group_rows(scheme, bits))
    assert np.array_equal(ws.view(np.uint32), ws_ref.view(np.uint32))


def test_pack_codes_on_rounding_ties_and_midpoints():
    # weights placed exactly on Fixed rounding ties and PoT decision points, alpha = 1
    ties4 = [np.float32((j + 0.5) / 7.0) for j in range(7)]
    ties8 = [np.float32((j + 0.5) / 127.0) for j in range(0, 127, 9)]
    mids = [2.0 ** -7] + [3 * 2.0 ** (k - 9) for k in range(2, 8)]
    geo = [2.0 ** -(j + 0.5) for j in range(7)]
    pts = []
    for v in ties4 + ties8 + mids + geo:
        f = np.float32(v)
        pts += [f, np.nextafter(f, np.float32(0)), np.nextafter(f, np.float32(2)), -f]
    K = len(pts)
    W = np.tile(np.array(pts, np.float32), (6, 1))
    scheme = np.array([0, 1, 1, 0, 1, 1], np.uint8)
    bits = np.array([4, 4, 8, 4, 4, 8], np.uint8)
    alpha = np.array([1, 1, 1, 0.5, 0.5, 0.5], np.float32)
    for mode in (R.POT_NEAREST, R.POT_LOG2):
        layer, d_packed = Hn.pack_layer(W, scheme, bits, alpha, mode)
        vals, _, _ = Hn.unpack(layer, d_packed)
        v_ref, _ = O.quantize_rows(W, scheme, bits, alpha, mode)
        assert np.array_equal(vals, v_ref)


@pytest.mark.parametrize("M,Cin,k", [(64, 64, 3), (20, 24, 3), (9, 5, 1), (12, 40, 5), (130, 16, 2)])
def test_pack_codes_conv(M, Cin, k):
    W = synth.weights_kaiming(synth.rng(71, M + Cin), M, Cin, k, k)
    scheme, bits = O.assign_rows(W, (60, 35, 5))
    alpha = synth.alpha_rows(W)
    layer, d_packed = Hn.pack_layer(W, scheme, bits, alpha)
    vals, perm, ws = Hn.unpack(layer, d_packed)
    v_ref, ws_ref = O.quantize_rows(W.reshape(M, -1), scheme, bits, alpha)
    assert np.array_equal(vals, v_ref)
    assert np.array_equal(perm, O.group_rows(scheme, bits))


# ------------------------------------------------------------------ activation quantizer

@pytest.mark.parametrize("count", [1, 15, 16, 1000, 4099, 1 << 20])
@pytest.mark.parametrize("kind", [R.ACT_U4, R.ACT_S4])
def test_quantize_act(count, kind):
    g = synth.rng(72, count)
    x = synth.act_halfnormal(g, count) if kind == R.ACT_U4 else synth.act_normal(g, count)
    x[: min(count, 6)] = [0.0, 0.1, 0.3, 3.0, 1.5, 2.9999][: min(count, 6)]
    codes, step = Hn.quantize_act(x, synth.ALPHA_ACT, kind)
    c_ref, s_ref = O.quantize_act(x, synth.ALPHA_ACT, kind)
    assert np.array_equal(codes, c_ref)
    assert step == s_ref


@pytest.mark.parametrize("alpha", [3.0, 2.9999998, 1.0, 1e-3, 7.3e5, 1e-35, 1e33])
@pytest.mark.parametrize("kind", [R.ACT_U4, R.ACT_S4])
def test_quantize_act_on_rounding_boundaries(alpha, kind):
    # Values on and a few ulps around every rounding boundary (k + 0.5) * alpha / Q and every level,
    # around the clip points, plus specials, repeated until the warp-wide vector path is used.
    # The code near a boundary depends on the single correctly rounded division x / alpha.
    Q = 15 if kind == R.ACT_U4 else 7
    a32 = np.float32(alpha)
    ks = np.arange(-2 * Q - 3, 2 * Q + 4, dtype=np.float64) / 2.0          # levels and half-levels, beyond the clips
    centre = (ks * np.float64(a32) / Q).astype(np.float32)
    pts = [centre]
    for d in range(1, 5):
        up, dn = centre.copy(), centre.copy()
        for _ in range(d):
            up = np.nextafter(up, np.float32(np.inf)); dn = np.nextafter(dn, np.float32(-np.inf))
        pts += [up, dn]
    special = np.array([0.0, -0.0, np.inf, -np.inf, np.finfo(np.float32).tiny, 1e-45, -1e-45,
                        np.finfo(np.float32).max], dtype=np.float32)
    x = np.concatenate(pts + [special]).astype(np.float32)
    g = synth.rng(72, 991)
    x = np.concatenate([x, g.permutation(np.tile(x, 8))])                  # > 4096 values, mixed inside each warp step
    codes, step = Hn.quantize_act(x, float(a32), kind)
    c_ref, s_ref = O.quantize_act(x, float(a32), kind)
    assert np.array_equal(codes, c_ref)
    assert step == s_ref


# ------------------------------------------------------------------ linear layer

LIN_CASES = [
    # M, K, N, ratio        spans several 128-row blocks / 256-token tiles with ragged tails
    (256, 512, 64, (60, 35, 5)),        # config 1
    (128, 128, 256, (60, 35, 5)),
    (300, 200, 77, (50, 40, 10)),
    (130, 96, 513, (60, 35, 5)),
    (64, 576, 300, (65, 30, 5)),
    (1, 32, 1, (0, 100, 0)),
    (200, 48, 40, (0, 0, 100)),
    (150, 1000, 33, (100, 0, 0)),
    (257, 2304, 260, (60, 35, 5)),
    (500, 640, 300, (60, 35, 5)),       # four row blocks: two per tile in the workspace variant, ragged last block
]


@pytest.mark.parametrize("variant", VARIANTS, ids=lambda v: VNAME[v])
@pytest.mark.parametrize("M,K,N,ratio", LIN_CASES)
def test_linear_layer(M, K, N, ratio, variant):
    g = synth.rng(73, M * 7 + K + N)
    W = synth.weights_normal(g, (M, K))
    scheme, bits = _mixed_map(M, M + K, ratio)
    alpha = synth.alpha_rows(W)
    signed = (M % 2 == 0)
    act = g.integers(-7, 8, (N, K), dtype=np.int8) if signed else synth.act_codes_uniform(g, (N, K))
    act_step = np.float32(0.1)
    layer, d_packed = Hn.pack_layer(W, scheme, bits, alpha)
    try:
        y, acc = Hn.gemm(layer, d_packed, act, act_step, variant)
    except R.RmsmpError as e:
        if e.status == R.ERR_VARIANT and variant in (R.VARIANT_TENSOR, Hn.WORKSPACE) and K % 16 != 0:
            pytest.skip("tensor variant needs K % 16 == 0")
        raise
    v_ref, ws = O.quantize_rows(W, scheme, bits, alpha)
    acc_ref = O.matmul(v_ref, act)
    _check_layer_outputs(y, acc, acc_ref, ws, act_step, alpha, scheme, bits)


@pytest.mark.parametrize("variant", [R.VARIANT_SIMT, R.VARIANT_TENSOR, R.VARIANT_AUTO, Hn.WORKSPACE], ids=lambda v: VNAME[v])
def test_linear_layer_mn_layout_and_padded_ld(variant):
    M, K, N = 140, 160, 70
    g = synth.rng(74, variant if isinstance(variant, int) else 9)
    W = synth.weights_normal(g, (M, K))
    scheme, bits = O.assign_rows(W, (60, 35, 5))
    alpha = synth.alpha_rows(W)
    act = synth.act_codes_uniform(g, (N, K))
    layer, d_packed = Hn.pack_layer(W, scheme, bits, alpha)
    y, acc = Hn.gemm(layer, d_packed, act, 0.25, variant, out_layout=R.OUT_MN, ld_act=192)
    v_ref, ws = O.quantize_rows(W, scheme, bits, alpha)
    _check_layer_outputs(y, acc, O.matmul(v_ref, act), ws, np.float32(0.25), alpha, scheme, bits)
    y2, _ = Hn.gemm(layer, d_packed, act, 0.25, variant, want_acc=False)
    assert np.array_equal(y2, y)


def test_extreme_codes_do_not_overflow_or_lose_bits():
    # every weight at full scale, every activation at 15: |acc| = K*127*15 on Fixed-8 rows
    M, K, N = 130, 4608, 40
    W = np.ones((M, K), np.float32)
    W[::2] = -1
    scheme, bits = _mixed_map(M, 5, (40, 30, 30))
    alpha = np.ones(M, np.float32)
    act = np.full((N, K), 15, np.int8)
    layer, d_packed = Hn.pack_layer(W, scheme, bits, alpha)
    v_ref, ws = O.quantize_rows(W, scheme, bits, alpha)
    acc_ref = O.matmul(v_ref, act)
    assert np.array_equal(acc_ref.astype(np.int64), O.matmul_i64(v_ref, act))
    assert np.abs(acc_ref).max() == K * 127 * 15
    for variant in VARIANTS:
        y, acc = Hn.gemm(layer, d_packed, act, 1.0, variant)
        _check_layer_outputs(y, acc, acc_ref, ws, np.float32(1.0), alpha, scheme, bits)


# ------------------------------------------------------------------ convolution

CONV_CASES = [
    # M, Cin, k, stride, pad, B, H, W
    (64, 64, 3, 1, 1, 2, 14, 14),
    (40, 32, 3, 2, 1, 3, 14, 14),
    (130, 128, 3, 1, 1, 2, 7, 7),
    (24, 16, 1, 2, 0, 2, 8, 8),
    (16, 16, 1, 1, 0, 1, 5, 9),
    (32, 48, 3, 2, 1, 2, 9, 12),      # odd sizes, non-square
    (140, 256, 3, 1, 1, 5, 7, 7),     # several images per tile, ragged last tile
    (20, 20, 3, 1, 1, 1, 6, 6),       # Cin not a multiple of 16: CUDA-core variants only
    (64, 64, 3, 1, 1, 1, 56, 56),
    (200, 64, 2, 1, 0, 2, 9, 9),      # 64-byte pixels, even tap count, two row blocks (weights through the ring)
    (96, 64, 3, 2, 1, 3, 7, 7),       # 64-byte pixels, several images per tile, stride 2
    (64, 48, 1, 1, 0, 2, 12, 12),     # 64-byte pixels, one tap
    (48, 32, 3, 2, 0, 2, 9, 11),      # stride 2 without padding, odd sizes: the parity sub-grids differ in extent
    (32, 64, 5, 2, 2, 2, 10, 7),      # stride 2, 5x5: taps two rows / columns outside the image
    (24, 32, 2, 2, 0, 3, 8, 6),       # stride 2, even kernel
    (40, 32, 3, 3, 1, 2, 10, 13),     # stride 3: element-strided boxes (no parity split)
    (300, 128, 3, 2, 1, 2, 28, 28),   # stride 2, three row blocks, tiles of whole output rows
    (48, 64, 3, 1, 1, 3, 16, 8),      # resident weights, width a multiple of 8: one activation stage per kernel column
    (64, 32, 3, 1, 1, 2, 24, 24),     # the same with one 32-code step per tap, tiles of several output rows
    (100, 64, 3, 1, 1, 2, 40, 56),    # the same, ragged last row block, non-square image
    (64, 16, 7, 2, 3, 2, 32, 32),     # first-layer shape: 7x7 stride 2 pad 3 (3 input channels stored as 16, the rest zero)
    (256, 64, 1, 1, 0, 2, 14, 14),    # bottleneck 1x1 expansions and reductions (ResNet-50 style)
    (64, 256, 1, 1, 0, 2, 14, 14),
    (32, 32, 3, 1, 1, 2, 16, 16),     # depthwise-separable networks' pointwise/3x3 sizes with few channels
]


@pytest.mark.parametrize("variant", VARIANTS, ids=lambda v: VNAME[v])
@pytest.mark.parametrize("M,Cin,k,stride,pad,B,H,W", CONV_CASES)
def test_conv_layer(M, Cin, k, stride, pad, B, H, W, variant):
    g = synth.rng(75, M + Cin + H)
    Wt = synth.weights_kaiming(g, M, Cin, k, k)
    scheme, bits = O.assign_rows(Wt, (60, 35, 5))
    alpha = synth.alpha_rows(Wt)
    x = synth.act_halfnormal(g, (B, H, W, Cin))
    codes, act_step = O.quantize_act(x, synth.ALPHA_ACT, O.ACT_U4)
    layer, d_packed = Hn.pack_layer(Wt, scheme, bits, alpha)
    try:
        y, acc = Hn.conv(layer, d_packed, codes, stride, pad, act_step, variant)
    except R.RmsmpError as e:
        if e.status == R.ERR_VARIANT and variant in (R.VARIANT_TENSOR, Hn.WORKSPACE) and Cin % 16 != 0:
            pytest.skip("tensor variant needs Cin % 16 == 0")
        raise
    v_ref, ws, acc_ref, y_ref = O.layer_conv(Wt, scheme, bits, alpha, codes, act_step, stride, pad)
    acc_ref = acc_ref.reshape(-1, M)
    _check_layer_outputs(y, acc, acc_ref, ws, act_step, alpha, scheme, bits)


def test_conv_mn_layout_auto():
    M, Cin, B, H = 72, 32, 2, 10
    g = synth.rng(76)
    Wt = synth.weights_kaiming(g, M, Cin, 3, 3)
    scheme, bits = O.assign_rows(Wt, (60, 35, 5))
    alpha = synth.alpha_rows(Wt)
    codes = synth.act_codes_uniform(g, (B, H, H, Cin))
    layer, d_packed = Hn.pack_layer(Wt, scheme, bits, alpha)
    y, acc = Hn.conv(layer, d_packed, codes, 1, 1, 0.2, R.VARIANT_AUTO, out_layout=R.OUT_MN)
    _, ws, acc_ref, _ = O.layer_conv(Wt, scheme, bits, alpha, codes, np.float32(0.2), 1, 1)
    _check_layer_outputs(y, acc, acc_ref.reshape(-1, M), ws, np.float32(0.2), alpha, scheme, bits)


# ------------------------------------------------------------------ the whole path, one call after the other

def test_full_path_fp32_in_fp32_out():
    """quantize_pack -> quantize_act -> conv, from fp32 tensors, as the benchmark runs it."""
    import torch
    L = synth.ConvShape("t", 96, 64, 3, 1, 1, 14)
    g = synth.rng(77)
    Wt = synth.weights_kaiming(g, L.M, L.Cin, 3, 3)
    x = synth.act_halfnormal(g, (4, 14, 14, 64))
    scheme, bits = R.rmsmp_assign_rows(Wt, synth.RATIO_RMSMP1)
    s2, b2 = O.assign_rows(Wt, synth.RATIO_RMSMP1)
    assert np.array_equal(scheme, s2) and np.array_equal(bits, b2)
    alpha = synth.alpha_rows(Wt)
    layer, d_packed = Hn.pack_layer(Wt, scheme, bits, alpha)
    dx = torch.from_numpy(x).cuda()
    dc = torch.empty(x.shape, dtype=torch.int8, device="cuda")
    step = R.rmsmp_quantize_act(dx, dx.numel(), synth.ALPHA_ACT, R.ACT_U4, dc)
    N = 4 * 14 * 14
    y = torch.empty((N, L.M), dtype=torch.float32, device="cuda")
    R.rmsmp_conv_implicit(layer, d_packed, dc, 4, 14, 14, 1, 1, step, y)
    torch.cuda.synchronize()
    codes, st_ref = O.quantize_act(x, synth.ALPHA_ACT, O.ACT_U4)
    assert np.float32(step) == st_ref
    _, _, _, y_ref = O.layer_conv(Wt, scheme, bits, alpha, codes, st_ref, 1, 1)
    assert np.array_equal(y.cpu().numpy().view(np.uint32), y_ref.reshape(N, L.M).view(np.uint32))


# ------------------------------------------------------------------ re-quantizing epilogue (layer chaining)
# The fused epilogue must give the codes of (this layer's fp32 output -> the activation quantizer),
# i.e. the oracle's layer followed by the oracle's quantizer, byte for byte.

def _next_alpha(y_ref):
    return float(np.float32(3.0 * float(np.std(y_ref))))


@pytest.mark.parametrize("kind", [R.ACT_U4, R.ACT_S4])
@pytest.mark.parametrize("M,K,N,ld_extra", [
    (256, 512, 300, 0),      # bulk stores, ragged last tile
    (200, 128, 77, 0),       # ld_codes = 200: not a multiple of 16 -> direct byte stores
    (130, 96, 513, 14),      # padded leading dimension (144), two row blocks, ragged rows
    (64, 576, 260, 0),       # duplicated rows, resident weights
])
def test_linear_requant_epilogue(M, K, N, ld_extra, kind):
    import torch
    g = synth.rng(81, M + K + N)
    Wt = synth.weights_normal(g, (M, K))
    codes = synth.act_codes_uniform(g, (N, K))
    act_step = np.float32(0.125)
    scheme, bits = O.assign_rows(Wt, (60, 35, 5))
    alpha = synth.alpha_rows(Wt)
    _, _, _, y_ref = O.layer_linear(Wt, scheme, bits, alpha, codes, act_step)
    na = _next_alpha(y_ref)
    want, want_step = O.quantize_act(y_ref.reshape(N, M), na, kind)
    layer, d_packed = Hn.pack_layer(Wt, scheme, bits, alpha)
    ws = torch.empty(R.rmsmp_workspace_bytes(layer), dtype=torch.int8, device="cuda")
    R.rmsmp_expand_weights(layer, d_packed, ws)
    ld = M + ld_extra
    out = torch.full((N, ld), 99, dtype=torch.int8, device="cuda")
    step = R.rmsmp_gemm_workspace_requant(layer, d_packed, ws, torch.from_numpy(codes).cuda(), N, K, float(act_step),
                                          na, kind, out, ld)
    torch.cuda.synchronize()
    assert R.rmsmp_last_device_status(d_packed) == R.OK
    got = out.cpu().numpy()
    assert np.float32(step) == want_step
    assert np.array_equal(got[:, :M], want)
    assert (got[:, M:] == 99).all()                      # padding columns untouched


@pytest.mark.parametrize("kind", [R.ACT_U4, R.ACT_S4])
@pytest.mark.parametrize("M,Cin,k,stride,pad,B,H,W", [
    (64, 64, 3, 1, 1, 2, 14, 14),
    (140, 256, 3, 1, 1, 5, 7, 7),      # several images per tile, ragged last tile, two row blocks
    (32, 48, 3, 2, 1, 2, 9, 12),
    (128, 64, 1, 2, 0, 2, 8, 8),
])
def test_conv_requant_epilogue(M, Cin, k, stride, pad, B, H, W, kind):
    import torch
    g = synth.rng(82, M + Cin + H)
    Wt = synth.weights_kaiming(g, M, Cin, k, k)
    scheme, bits = O.assign_rows(Wt, (60, 35, 5))
    alpha = synth.alpha_rows(Wt)
    x = synth.act_halfnormal(g, (B, H, W, Cin))
    codes, act_step = O.quantize_act(x, synth.ALPHA_ACT, O.ACT_U4)
    _, _, _, y_ref = O.layer_conv(Wt, scheme, bits, alpha, codes, act_step, stride, pad)
    y_ref = y_ref.reshape(-1, M)
    na = _next_alpha(y_ref)
    want, want_step = O.quantize_act(y_ref, na, kind)
    layer, d_packed = Hn.pack_layer(Wt, scheme, bits, alpha)
    ws = torch.empty(R.rmsmp_workspace_bytes(layer), dtype=torch.int8, device="cuda")
    R.rmsmp_expand_weights(layer, d_packed, ws)
    out = torch.full(y_ref.shape, 99, dtype=torch.int8, device="cuda")
    step = R.rmsmp_conv_implicit_workspace_requant(layer, d_packed, ws, torch.from_numpy(codes).cuda(), B, H, W,
                                                   stride, pad, float(act_step), na, kind, out)
    torch.cuda.synchronize()
    assert R.rmsmp_last_device_status(d_packed) == R.OK
    assert np.float32(step) == want_step
    assert np.array_equal(out.cpu().numpy(), want)


def _ulps(x, n):
    """fp32 value n units in the last place away from x."""
    v = np.float32(x)
    for _ in range(abs(n)):
        v = np.nextafter(v, np.float32(np.inf if n > 0 else -np.inf), dtype=np.float32)
    return v


@pytest.mark.parametrize("kind", [R.ACT_U4, R.ACT_S4])
@pytest.mark.parametrize("M,ld_extra", [(128, 0), (130, 14), (64, 0)], ids=["bulk", "direct", "dup"])
@pytest.mark.parametrize("step_ulps", [0, 1, -1, 4, -4])
def test_requant_epilogue_on_rounding_boundaries(M, ld_extra, step_ulps, kind):
    """The fused quantizer exactly ON, and a few units in the last place either side of, its
    rounding boundaries.  All rows are Fixed-8 with alpha = 127, so wstep = 1 and the weights are
    the integers they are given as; with act_step = 1 the layer output y equals the integer sum.
    next_alpha is chosen so that y / next_alpha * Q = y / 2: every odd sum lies exactly on a
    half-level (the tie goes to the even code), and an act_step a few ulps off 1 moves every value
    just off its level or half-level.  Expected codes: the oracle's epilogue followed by the
    oracle's quantizer, so its chain of fp32 roundings decides."""
    import torch
    K, N = 64, 700
    g = synth.rng(83, M + step_ulps + 10 * kind)
    lo = 0 if kind == R.ACT_U4 else -1
    Wt = g.integers(lo, 2, size=(M, K)).astype(np.float32)          # values in {0, 1} (U4) or {-1, 0, 1} (S4)
    Wt[g.random((M, K)) < (0.93 if kind == R.ACT_U4 else 0.8)] = 0.0  # sums of a few codes: mostly inside the clip range
    Wt[:, 0] = 127.0                                                  # one full-scale entry per row keeps the values exact ...
    scheme = np.ones(M, np.uint8)
    bits = np.full(M, 8, np.uint8)
    alpha = np.full(M, 127.0, np.float32)
    codes = synth.act_codes_uniform(g, (N, K))
    codes[:, 0] = 0                                                   # ... and never contributes to a sum
    if kind == R.ACT_S4:
        codes = (codes % 15 - 7).astype(np.int8)
        codes[:, 0] = 0
    act_step = _ulps(1.0, step_ulps)
    na = 30.0 if kind == R.ACT_U4 else 14.0
    values, wstep, acc_ref, y_ref = O.layer_linear(Wt, scheme, bits, alpha, codes, act_step)
    assert np.all(wstep == np.float32(1.0)) and np.array_equal(values, Wt.astype(np.int8))
    odd = (np.abs(acc_ref) % 2 == 1) & (np.abs(acc_ref) < 30)
    assert odd.mean() > 0.25                                           # a large share of outputs sits on a half-level
    want, _ = O.quantize_act(y_ref, na, kind)
    layer, d_packed = Hn.pack_layer(Wt, scheme, bits, alpha)
    ws = torch.empty(R.rmsmp_workspace_bytes(layer), dtype=torch.int8, device="cuda")
    R.rmsmp_expand_weights(layer, d_packed, ws)
    ld = M + ld_extra
    out = torch.full((N, ld), 99, dtype=torch.int8, device="cuda")
    R.rmsmp_gemm_workspace_requant(layer, d_packed, ws, torch.from_numpy(codes).cuda(), N, K, float(act_step),
                                   na, kind, out, ld)
    torch.cuda.synchronize()
    assert R.rmsmp_last_device_status(d_packed) == R.OK
    got = out.cpu().numpy()
    assert np.array_equal(got[:, :M], want)
    assert (got[:, M:] == 99).all()
    if step_ulps == 0:
        # with exact halves the expected code is the even neighbour, by the definition alone
        q = 15 if kind == R.ACT_U4 else 7
        t = np.clip(acc_ref.astype(np.float64) / na, 0.0 if kind == R.ACT_U4 else -1.0, 1.0) * q
        assert np.array_equal(want, np.rint(t).astype(np.int8))


def test_conv_requant_epilogue_on_rounding_boundaries():
    """The same construction through the convolution kernel's resident-weight form (3x3, 64 channels)."""
    import torch
    M, Cin, k, B, H = 64, 64, 3, 2, 12
    g = synth.rng(83, 999)
    Wt = g.integers(0, 2, size=(M, Cin, k, k)).astype(np.float32)
    Wt[g.random(Wt.shape) < 0.992] = 0.0
    Wt[:, 0, 0, 0] = 127.0
    scheme = np.ones(M, np.uint8)
    bits = np.full(M, 8, np.uint8)
    alpha = np.full(M, 127.0, np.float32)
    codes = synth.act_codes_uniform(g, (B, H, H, Cin))
    codes[..., 0] = 0
    for ulps in (0, 2, -2):
        act_step = _ulps(1.0, ulps)
        _, _, acc_ref, y_ref = O.layer_conv(Wt, scheme, bits, alpha, codes, act_step, 1, 1)
        assert ((acc_ref % 2 == 1) & (acc_ref < 30)).mean() > 0.2
        want, _ = O.quantize_act(y_ref.reshape(-1, M), 30.0, O.ACT_U4)
        layer, d_packed = Hn.pack_layer(Wt, scheme, bits, alpha)
        ws = torch.empty(R.rmsmp_workspace_bytes(layer), dtype=torch.int8, device="cuda")
        R.rmsmp_expand_weights(layer, d_packed, ws)
        out = torch.full(want.shape, 99, dtype=torch.int8, device="cuda")
        R.rmsmp_conv_implicit_workspace_requant(layer, d_packed, ws, torch.from_numpy(codes).cuda(), B, H, H, 1, 1,
                                                float(act_step), 30.0, R.ACT_U4, out)
        torch.cuda.synchronize()
        assert R.rmsmp_last_device_status(d_packed) == R.OK
        assert np.array_equal(out.cpu().numpy(), want)


def test_requant_rejects_bad_arguments():
    import torch
    g = synth.rng(83)
    Wt = synth.weights_normal(g, (32, 64))
    scheme, bits = O.assign_rows(Wt, (60, 35, 5))
    layer, d_packed = Hn.pack_layer(Wt, scheme, bits, synth.alpha_rows(Wt))
    ws = torch.empty(R.rmsmp_workspace_bytes(layer), dtype=torch.int8, device="cuda")
    R.rmsmp_expand_weights(layer, d_packed, ws)
    act = torch.zeros((40, 64), dtype=torch.int8, device="cuda")
    out = torch.zeros((40, 32), dtype=torch.int8, device="cuda")
    for bad_alpha in (0.0, -1.0, float("inf"), float("nan")):
        with pytest.raises(R.RmsmpError) as e:
            R.rmsmp_gemm_workspace_requant(layer, d_packed, ws, act, 40, 64, 0.1, bad_alpha, R.ACT_U4, out, 32)
        assert e.value.status == R.ERR_SCALE
    with pytest.raises(R.RmsmpError) as e:
        R.rmsmp_gemm_workspace_requant(layer, d_packed, ws, act, 40, 64, 0.1, 1.0, 7, out, 32)
    assert e.value.status == R.ERR_SCHEME
    with pytest.raises(R.RmsmpError) as e:
        R.rmsmp_gemm_workspace_requant(layer, d_packed, ws, act, 40, 64, 0.1, 1.0, R.ACT_U4, out, 16)   # ld < M
    assert e.value.status == R.ERR_SHAPE


def test_padded_output_rows_leave_the_padding_untouched():
    """[N][ld_out] fp32 output with ld_out > M and M not a multiple of 4: bulk stores clip in
    16-byte granules, so this shape must not go through them."""
    import torch
    M, K, N, ld = 130, 128, 300, 136
    g = synth.rng(84)
    Wt = synth.weights_normal(g, (M, K))
    codes = synth.act_codes_uniform(g, (N, K))
    scheme, bits = O.assign_rows(Wt, (60, 35, 5))
    alpha = synth.alpha_rows(Wt)
    layer, d_packed = Hn.pack_layer(Wt, scheme, bits, alpha)
    ws = torch.empty(R.rmsmp_workspace_bytes(layer), dtype=torch.int8, device="cuda")
    R.rmsmp_expand_weights(layer, d_packed, ws)
    d_codes = torch.from_numpy(codes).cuda()
    _, _, _, y_ref = O.layer_linear(Wt, scheme, bits, alpha, codes, np.float32(0.25))
    for fn in (lambda y: R.rmsmp_gemm_workspace(layer, d_packed, ws, d_codes, N, K, 0.25, y, ld),
               lambda y: R.rmsmp_gemm(layer, d_packed, d_codes, N, K, 0.25, y, ld)):
        y = torch.full((N, ld), -7.0, dtype=torch.float32, device="cuda")
        fn(y)
        torch.cuda.synchronize()
        got = y.cpu().numpy()
        assert np.array_equal(got[:, :M].view(np.uint32), y_ref.reshape(N, M).view(np.uint32))
        assert (got[:, M:] == -7.0).all()


def test_a_bounded_wait_that_runs_out_reports_timeout_and_leaves_the_context_usable():
    """The failure path, without a fault: one warp waits on a barrier nobody signals, with the
    kernels' own bounded wait and a limit of about a millisecond.  The status word must read
    ERR_TIMEOUT afterwards, and an ordinary layer on the same stream must still be bit-exact."""
    import torch
    status = torch.zeros(4, dtype=torch.int32, device="cuda")
    R.rmsmp_selftest_bounded_wait(2_000_000, status)
    torch.cuda.synchronize()
    assert int(status[0].item()) == R.ERR_TIMEOUT
    with pytest.raises(R.RmsmpError) as e:
        R.rmsmp_selftest_bounded_wait(10 ** 10, status)          # beyond the tenth of a second the call allows
    assert e.value.status == R.ERR_SHAPE
    g = synth.rng(84, 1)
    Wt = synth.weights_normal(g, (256, 512))
    scheme, bits = O.assign_rows(Wt, (60, 35, 5))
    alpha = synth.alpha_rows(Wt)
    act = synth.act_codes_uniform(g, (300, 512))
    layer, d_packed = Hn.pack_layer(Wt, scheme, bits, alpha)
    y, acc = Hn.gemm(layer, d_packed, act, 0.25, R.VARIANT_TENSOR)
    _, _, acc_ref, y_ref = O.layer_linear(Wt, scheme, bits, alpha, act, np.float32(0.25))
    assert np.array_equal(acc, acc_ref)
    assert np.array_equal(y.view(np.uint32), y_ref.view(np.uint32))


# ------------------------------------------------------------------ row assignment on the device

@pytest.mark.parametrize("ratio", [(60, 35, 5), (65, 30, 5), (0, 100, 0), (50, 40, 10)], ids=lambda r: "%d-%d-%d" % r)
@pytest.mark.parametrize("shape", [(256, 512), (130, 96), (1000, 2304), (64, 64, 3, 3), (160, 48, 3, 3)], ids=str)
def test_assignment_on_the_device_matches_oracle(shape, ratio):
    """Ratio in, packed layer out: the assignment (variance rank), the grouping, the per-row steps and every
    code must equal the oracle's assign_rows -> quantize_rows -> group_rows; then the layer runs."""
    import torch
    g = synth.rng(85, sum(shape) + ratio[0])
    conv = len(shape) == 4
    Wt = synth.weights_kaiming(g, *shape) if conv else synth.weights_normal(g, shape)
    if not conv:
        Wt[7] = Wt[3]                                   # two rows of equal variance: the row index decides
    M = shape[0]
    Cin, kh, kw = (shape[1], shape[2], shape[3]) if conv else (shape[1], 1, 1)
    layer = R.rmsmp_layer_init_ratio(M, Cin, kh, kw, ratio)
    d_W = torch.from_numpy(Wt).cuda()
    d_packed = torch.empty(layer.packed_bytes, dtype=torch.uint8, device="cuda")
    scratch = torch.empty(R.rmsmp_assign_scratch_bytes(M), dtype=torch.uint8, device="cuda")
    d_scheme = torch.empty(M, dtype=torch.uint8, device="cuda")
    d_bits = torch.empty(M, dtype=torch.uint8, device="cuda")
    R.rmsmp_assign_quantize_pack(d_W, R.W_CONV_OIHW if conv else R.W_LINEAR, layer, ratio, None, R.POT_NEAREST, d_packed,
                                 scratch, d_scheme, d_bits)
    torch.cuda.synchronize()
    scheme, bits = O.assign_rows(Wt, ratio)
    assert np.array_equal(d_scheme.cpu().numpy(), scheme) and np.array_equal(d_bits.cpu().numpy(), bits)
    alpha = synth.alpha_rows(Wt)
    v_ref, ws_ref = O.quantize_rows(Wt.reshape(M, -1), scheme, bits, alpha)
    vals, perm, ws = Hn.unpack(layer, d_packed)
    assert np.array_equal(perm, O.group_rows(scheme, bits))
    assert np.array_equal(ws.view(np.uint32), ws_ref.view(np.uint32))
    assert np.array_equal(vals, v_ref)
    # the same descriptor as the host route gives, and a layer run on top of it
    ref_layer = R.rmsmp_layer_init(M, Cin, kh, kw, scheme, bits)
    assert (layer.nP, layer.nF4, layer.n8, layer.packed_bytes) == (ref_layer.nP, ref_layer.nF4, ref_layer.n8, ref_layer.packed_bytes)
    if not conv:
        act = synth.act_codes_uniform(g, (77, shape[1]))
        for variant in (R.VARIANT_AUTO, R.VARIANT_TENSOR if shape[1] % 16 == 0 else R.VARIANT_SIMT, Hn.WORKSPACE if shape[1] % 16 == 0 else R.VARIANT_SIMT):
            y, acc = Hn.gemm(layer, d_packed, act, 0.05, variant)
            assert np.array_equal(acc, O.matmul(v_ref, act))


# ------------------------------------------------------------------ depthwise convolution

@pytest.mark.parametrize("C,k,stride,pad,B,H,W,kind", [
    (32, 3, 1, 1, 2, 14, 14, R.ACT_U4),
    (96, 3, 2, 1, 3, 15, 13, R.ACT_U4),        # MobileNet-v2 style stride-2 block, odd sizes
    (144, 3, 1, 1, 1, 28, 28, R.ACT_S4),
    (960, 3, 1, 1, 2, 7, 7, R.ACT_U4),         # the widest depthwise layer of MobileNet-v2
    (8, 5, 1, 2, 2, 6, 9, R.ACT_S4),
    (1280, 3, 1, 1, 1, 5, 6, R.ACT_S4),        # more channel quads than threads of a block
    (16, 3, 3, 0, 2, 11, 10, R.ACT_U4),        # a stride the run kernel does not take
])
def test_depthwise_conv_matches_oracle(C, k, stride, pad, B, H, W, kind):
    import torch
    g = synth.rng(86, C + k + H)
    Wt = synth.weights_kaiming(g, C, 1, k, k)
    scheme, bits = O.assign_rows(Wt, (60, 35, 5))
    alpha = synth.alpha_rows(Wt)
    x = synth.act_halfnormal(g, (B, H, W, C)) if kind == R.ACT_U4 else synth.act_normal(g, (B, H, W, C))
    codes, act_step = O.quantize_act(x, synth.ALPHA_ACT, kind)
    layer, d_packed = Hn.pack_layer(Wt, scheme, bits, alpha)
    v_ref, wstep = O.quantize_rows(Wt.reshape(C, -1), scheme, bits, alpha)
    acc_ref = O.conv_depthwise(v_ref.reshape(C, k, k), codes, stride, pad)
    y_ref = O.epilogue(acc_ref, wstep, act_step)
    Ho, Wo = O.conv_out_hw(H, W, k, k, stride, pad)
    y = torch.full((B, Ho, Wo, C), float("nan"), dtype=torch.float32, device="cuda")
    acc = torch.full((B, Ho, Wo, C), -5, dtype=torch.int32, device="cuda")
    R.rmsmp_conv_depthwise(layer, d_packed, torch.from_numpy(codes).cuda(), B, H, W, stride, pad, float(act_step), y, acc)
    torch.cuda.synchronize()
    assert np.array_equal(acc.cpu().numpy(), acc_ref)
    assert np.array_equal(y.cpu().numpy().view(np.uint32), y_ref.view(np.uint32))


def test_depthwise_conv_rejects_what_it_cannot_run():
    import torch
    g = synth.rng(86, 1)
    Wt = synth.weights_kaiming(g, 6, 1, 3, 3)            # 6 channels: not a multiple of 4
    scheme, bits = O.assign_rows(Wt, (60, 35, 5))
    layer, d_packed = Hn.pack_layer(Wt, scheme, bits, synth.alpha_rows(Wt))
    a = torch.zeros((1, 4, 4, 8), dtype=torch.int8, device="cuda")
    y = torch.zeros((1, 4, 4, 8), dtype=torch.float32, device="cuda")
    with pytest.raises(R.RmsmpError) as e:
        R.rmsmp_conv_depthwise(layer, d_packed, a, 1, 4, 4, 1, 1, 0.1, y)
    assert e.value.status == R.ERR_VARIANT
    Wd = synth.weights_kaiming(g, 8, 2, 3, 3)            # an ordinary layer is not a depthwise one
    scheme, bits = O.assign_rows(Wd, (60, 35, 5))
    layer, d_packed = Hn.pack_layer(Wd, scheme, bits, synth.alpha_rows(Wd))
    with pytest.raises(R.RmsmpError) as e:
        R.rmsmp_conv_depthwise(layer, d_packed, a, 1, 4, 4, 1, 1, 0.1, y)
    assert e.value.status == R.ERR_SHAPE


# ---------------------------------------------------------------- first layer (few channels) as a patch matrix
@pytest.mark.gpu
@pytest.mark.parametrize("M,Cin,k,stride,pad,B,H,W,pitch", [
    (64, 3, 7, 2, 3, 2, 30, 26, 3),        # the networks' first layer (Section 4.1): 3 channels, 7 x 7, stride 2
    (24, 3, 3, 1, 1, 1, 9, 7, 4),          # a padded pixel pitch
    (40, 1, 5, 1, 0, 2, 8, 8, 1),
    (16, 64, 3, 1, 1, 1, 4, 262, 64),      # input rows too wide for shared memory: the direct-gather form
])
def test_first_layer_patch_matrix_and_gemm_match_oracle_conv(M, Cin, k, stride, pad, B, H, W, pitch):
    import torch
    g = synth.rng(91, M + Cin + H)
    Wt = synth.weights_normal(g, (M, Cin, k, k))
    scheme, bits = O.assign_rows(Wt.reshape(M, -1), (60, 35, 5))
    alpha = synth.alpha_rows(Wt.reshape(M, -1))
    act = synth.act_codes_uniform(g, (B, H, W, Cin))
    K = k * k * Cin
    ld = (K + 15) // 16 * 16
    # patch matrix on the device against the oracle's
    a = torch.zeros((B, H, W, pitch), dtype=torch.int8, device="cuda")
    a[..., :Cin] = torch.from_numpy(act).cuda()
    Ho, Wo = O.conv_out_hw(H, W, k, k, stride, pad)
    N = B * Ho * Wo
    cols = torch.full((N, ld), 99, dtype=torch.int8, device="cuda")
    R.rmsmp_im2col_codes(a, B, H, W, Cin, pitch, k, k, stride, pad, cols, ld)
    torch.cuda.synchronize()
    assert np.array_equal(cols.cpu().numpy(), O.im2col(act, k, k, stride, pad, ld))
    # the layer as a linear layer over the patches, filters flattened tap-major with zero columns appended
    Wl = np.zeros((M, ld), np.float32)
    Wl[:, :K] = Wt.transpose(0, 2, 3, 1).reshape(M, K)
    layer, d_packed = Hn.pack_layer(Wl, scheme, bits, alpha)
    step = np.float32(0.05)
    y = torch.full((N, M), float("nan"), dtype=torch.float32, device="cuda")
    acc = torch.zeros((N, M), dtype=torch.int32, device="cuda")
    R.rmsmp_gemm_variant(layer, d_packed, cols, N, ld, float(step), y, M, R.OUT_NM, acc, R.VARIANT_AUTO)
    torch.cuda.synchronize()
    assert R.rmsmp_last_device_status(d_packed) == R.OK
    _, _, acc_ref, y_ref = O.layer_conv(Wt, scheme, bits, alpha, act, step, stride, pad)
    assert np.array_equal(acc.cpu().numpy(), acc_ref.reshape(N, M))
    assert np.array_equal(y.cpu().numpy().view(np.uint32), y_ref.reshape(N, M).view(np.uint32))


@pytest.mark.gpu
def test_patch_matrix_rejects_bad_arguments():
    import torch
    a = torch.zeros((1, 4, 4, 3), dtype=torch.int8, device="cuda")
    cols = torch.zeros((16, 32), dtype=torch.int8, device="cuda")
    for args, status in [((a, 1, 4, 4, 3, 3, 3, 3, 1, 1, cols, 16), R.ERR_SHAPE),       # ld_cols below kh*kw*C
                         ((a, 1, 4, 4, 3, 3, 3, 3, 1, 1, cols, 40), R.ERR_ALIGN),       # not a multiple of 16
                         ((a, 1, 4, 4, 3, 2, 3, 3, 1, 1, cols, 32), R.ERR_SHAPE),       # pitch below the channel count
                         ((a, 1, 4, 4, 3, 3, 7, 7, 1, 0, cols, 160), R.ERR_SHAPE)]:     # filter larger than the image
        with pytest.raises(R.RmsmpError) as e:
            R.rmsmp_im2col_codes(*args)
        assert e.value.status == status


# ---------------------------------------------------------------- resident weights expanded by the CTA itself
@pytest.mark.gpu
@pytest.mark.parametrize("M,K,N,layout", [
    (48, 192, 300, R.OUT_MN),       # duplicated rows (M <= 64), 64-byte k-blocks, [M][N] output
    (100, 64, 515, R.OUT_NM),       # rows beyond M in the block, one short k-block
    (128, 576, 77, R.OUT_NM),       # the largest resident stripe (72 KB expanded)
    (64, 448, 1000, R.OUT_NM),      # 64-byte k-blocks with a last chunk of 64 codes
])
def test_linear_layer_without_workspace_on_resident_weights(M, K, N, layout):
    """A layer of one row block whose expanded weights stay in shared memory is expanded once per CTA from the
    packed codes (no workspace): every kind of row, both output layouts, with the raw sums."""
    g = synth.rng(93, M + K + N)
    W = synth.weights_normal(g, (M, K))
    scheme, bits = _mixed_map(M, M + K, (50, 30, 20))
    alpha = synth.alpha_rows(W)
    act = g.integers(-8, 16, (N, K), dtype=np.int8)
    layer, d_packed = Hn.pack_layer(W, scheme, bits, alpha)
    y, acc = Hn.gemm(layer, d_packed, act, 0.125, R.VARIANT_TENSOR, out_layout=layout)
    v_ref, ws = O.quantize_rows(W, scheme, bits, alpha)
    _check_layer_outputs(y, acc, O.matmul(v_ref, act), ws, np.float32(0.125), alpha, scheme, bits)
