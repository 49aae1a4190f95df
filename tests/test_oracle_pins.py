"""Pins for the CPU oracle: what the paper and plain mathematics fix, checked without a GPU.

Each test is chosen so that a plausible mistake in the oracle (dropped term, wrong sign or
index, transposed operand, wrong level count, wrong tie rule) fails at least one of them.
"""
import os
from fractions import Fraction

import numpy as np
import pytest

from oracle import rmsmp_oracle as O
from paper_2111_00153_b200 import synth

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _golden_levels():
    out = {}
    for line in open(os.path.join(GOLD, "level_sets.txt")):
        if line.startswith("#") or not line.strip():
            continue
        k, *v = line.split()
        out[k] = v
    return out


# ----------------------------------------------------------------- level sets (Eq. 1, Eq. 4)

def test_fixed_level_set_and_count():
    g = _golden_levels()
    for bits, key in ((4, "fixed4_count"), (8, "fixed8_count")):
        Q = 2 ** (bits - 1) - 1
        ws = np.linspace(-1.3, 1.3, 20001, dtype=np.float32)
        qs = {O.fixed_q(w, 1.0, bits) for w in ws}
        assert qs == set(range(-Q, Q + 1))
        assert len(qs) == int(g[key][0])
    # the dequantized values are exactly Eq. 1's set
    lv = sorted(float(Fraction(s)) for s in g["fixed4"])
    deq = sorted({abs(O.fixed_q(w, 1.0, 4)) / 7.0 for w in np.linspace(0, 1, 2001)})
    assert np.allclose(deq, lv, rtol=0, atol=1e-15)


@pytest.mark.parametrize("mode", [O.POT_NEAREST, O.POT_LOG2])
def test_pot_level_set_and_count(mode):
    g = _golden_levels()
    ws = np.linspace(-1.3, 1.3, 40001, dtype=np.float32)
    vals = {O.pot_value(O.pot_nibble(w, 1.0, mode)) for w in ws}
    assert vals == {0} | {s * 2 ** j for j in range(7) for s in (-1, 1)}
    assert len(vals) == int(g["pot4_count"][0])
    lv = sorted(float(Fraction(s)) for s in g["pot4"])
    assert sorted({abs(v) / 64.0 for v in vals}) == lv
    # canonical zero: sign bit never set with e = 0
    assert O.pot_nibble(-1e-9, 1.0, mode) == 0


# ----------------------------------------------------------------- closed forms / special cases

@pytest.mark.parametrize("bits", [4, 8])
@pytest.mark.parametrize("alpha", [1.0, 0.37, 0.0613, 5.5])
def test_fixed_exact_levels_map_to_themselves(bits, alpha):
    Q = 2 ** (bits - 1) - 1
    a = np.float32(alpha)
    for j in range(-Q, Q + 1):
        w = np.float32(np.float64(a) * j / Q)
        assert O.fixed_q(w, a, bits) == j
    # clipping (Eq. 3): beyond alpha saturates
    assert O.fixed_q(np.float32(3 * alpha), a, bits) == Q
    assert O.fixed_q(np.float32(-3 * alpha), a, bits) == -Q
    assert O.fixed_q(0.0, a, bits) == 0


@pytest.mark.parametrize("mode", [O.POT_NEAREST, O.POT_LOG2])
@pytest.mark.parametrize("alpha", [1.0, 0.37, 0.0613])
def test_pot_exact_levels_map_to_themselves(mode, alpha):
    a = np.float32(alpha)
    for j in range(7):
        for s in (1, -1):
            w = np.float32(s * np.float64(a) * 2.0 ** -j)
            nib = O.pot_nibble(w, a, mode)
            assert nib & 7 == 7 - j and (nib >> 3) == (1 if s < 0 else 0)
            assert O.pot_value(nib) == s * 2 ** (6 - j)
    assert O.pot_nibble(np.float32(9 * alpha), a, mode) == 7
    assert O.pot_nibble(np.float32(-9 * alpha), a, mode) == 15
    assert O.pot_nibble(0.0, a, mode) == 0


def test_odd_symmetry_and_monotone():
    g = np.random.default_rng(5)
    ws = np.sort((g.standard_normal(4000) * 0.5).astype(np.float32))
    for bits in (4, 8):
        q = np.array([O.fixed_q(w, 0.9, bits) for w in ws])
        qn = np.array([O.fixed_q(-w, 0.9, bits) for w in ws])
        assert np.array_equal(q, -qn)
        assert np.all(np.diff(q) >= 0)
    for mode in (O.POT_NEAREST, O.POT_LOG2):
        v = np.array([O.pot_value(O.pot_nibble(w, 0.9, mode)) for w in ws])
        vn = np.array([O.pot_value(O.pot_nibble(-w, 0.9, mode)) for w in ws])
        assert np.array_equal(v, -vn)
        assert np.all(np.diff(v) >= 0)


def test_fixed_error_bound_half_step():
    g = np.random.default_rng(6)
    for bits in (4, 8):
        Q = 2 ** (bits - 1) - 1
        for alpha in (1.0, 0.0731):
            ws = (g.uniform(-1, 1, 3000) * alpha).astype(np.float32)
            step = alpha / Q
            for w in ws:
                q = O.fixed_q(w, alpha, bits)
                assert abs(q * step - float(w)) <= step / 2 * (1 + 1e-5)


def test_pot_nearest_error_is_half_local_gap():
    levels = np.array([0.0] + [2.0 ** -j for j in range(6, -1, -1)])
    g = np.random.default_rng(7)
    for w in g.uniform(0, 1, 3000).astype(np.float32):
        v = abs(O.pot_value(O.pot_nibble(w, 1.0, O.POT_NEAREST))) / 64.0
        i = int(np.searchsorted(levels, float(w), side="right")) - 1
        lo, hi = levels[i], levels[min(i + 1, 7)]
        assert abs(v - float(w)) <= (hi - lo) / 2 + 1e-12


@pytest.mark.parametrize("alpha", [1.0, 0.213, 7.0])
def test_idempotent_requantization(alpha):
    a = np.float32(alpha)
    for bits in (4, 8):
        Q = 2 ** (bits - 1) - 1
        step = O.wstep(a, O.SCHEME_FIXED, bits)
        for q in range(-Q, Q + 1):
            assert O.fixed_q(np.float32(q) * step, a, bits) == q
    step = O.wstep(a, O.SCHEME_POT, 4)
    for mode in (O.POT_NEAREST, O.POT_LOG2):
        for nib in list(range(0, 8)) + list(range(9, 16)):
            v = O.pot_value(nib)
            assert O.pot_nibble(np.float32(v) * step, a, mode) == nib


def test_wstep_definition():
    for alpha in (1.0, 0.3, 12.5):
        a = np.float32(alpha)
        assert O.wstep(a, O.SCHEME_FIXED, 4) == np.float32(a / np.float32(7))
        assert O.wstep(a, O.SCHEME_FIXED, 8) == np.float32(a / np.float32(127))
        assert O.wstep(a, O.SCHEME_POT, 4) == np.float32(a / np.float32(64))


# ----------------------------------------------------------------- brute force nearest level

def _brute_nearest(t, levels, tie_larger):
    """argmin over an explicit level list in double; tie -> larger magnitude or None."""
    d = np.abs(np.asarray(levels, dtype=np.float64) - float(t))
    m = d.min()
    cand = [levels[i] for i in np.flatnonzero(d == m)]
    if len(cand) > 1 and not tie_larger:
        return None
    return max(cand, key=abs)


def test_fixed_matches_brute_force_projection():
    g = np.random.default_rng(8)
    for bits in (4, 8):
        Q = 2 ** (bits - 1) - 1
        levels = [j / Q for j in range(-Q, Q + 1)]
        for alpha in (1.0, 0.05):
            W = (g.standard_normal((8, 8)) * alpha * 0.6).astype(np.float32)
            for w in W.ravel():
                t = float(np.clip(np.float32(w) / np.float32(alpha), -1, 1))
                if abs((t * Q) % 1 - 0.5) < 1e-4:     # fp32 near-tie: the tie rule decides, tested below
                    continue
                assert O.fixed_q(w, alpha, bits) == round(_brute_nearest(t, levels, True) * Q)


def test_pot_nearest_matches_brute_force_projection_including_midpoints():
    levels = [0.0] + [s * 2.0 ** -j for j in range(7) for s in (1, -1)]
    g = np.random.default_rng(9)
    W = g.uniform(-1.1, 1.1, (8, 8)).astype(np.float32)
    mids = [2.0 ** -7] + [3 * 2.0 ** (k - 9) for k in range(2, 8)]
    adversarial = []
    for m in mids:
        f = np.float32(m)
        adversarial += [f, np.nextafter(f, np.float32(0)), np.nextafter(f, np.float32(2)),
                        -f, -np.nextafter(f, np.float32(0))]
    for w in list(W.ravel()) + adversarial:
        t = float(np.clip(np.float32(w), -1, 1))
        want = _brute_nearest(t, levels, True)
        got = O.pot_value(O.pot_nibble(w, 1.0, O.POT_NEAREST)) / 64.0
        assert got == want, (w, got, want)


def test_pot_log2_matches_rounding_of_log2():
    g = np.random.default_rng(10)
    for w in g.uniform(2.0 ** -9, 1.0, 4000).astype(np.float32):
        r = int(np.floor(np.log2(float(w)) + 0.5))
        want = 0 if r < -6 else 2 ** (6 + min(r, 0))
        assert O.pot_value(O.pot_nibble(w, 1.0, O.POT_LOG2)) == want
    # the two modes differ between the arithmetic and the geometric midpoint (e.g. 0.72)
    assert O.pot_value(O.pot_nibble(0.72, 1.0, O.POT_NEAREST)) == 32
    assert O.pot_value(O.pot_nibble(0.72, 1.0, O.POT_LOG2)) == 64


def test_round_half_to_even_reading():
    # t*7 lands exactly on 2.5 in binary32 for this t; the documented reading rounds to even (2).
    t = np.float32(2.5 / 7.0)
    assert np.float32(t * np.float32(7)) == np.float32(2.5)
    assert O.fixed_q(t, 1.0, 4) == 2
    assert O.fixed_q(-t, 1.0, 4) == -2
    assert O.fixed_q(0.5, 1.0, 4) == 4      # 3.5 -> 4
    assert O.fixed_q(0.5, 1.0, 8) == 64     # 63.5 -> 64


def test_quantize_rows_rejects_pot8_and_bad_alpha():
    W = np.ones((2, 4), np.float32)
    with pytest.raises(ValueError):
        O.quantize_rows(W, [0, 1], [8, 4], [1.0, 1.0])      # PoT-8 is not on the menu
    with pytest.raises(ValueError):
        O.quantize_rows(W, [1, 1], [4, 4], [0.0, 1.0])
    with pytest.raises(ValueError):
        O.quantize_rows(W, [1, 1], [4, 3], [1.0, 1.0])


# ----------------------------------------------------------------- activations

def test_activation_quantizer():
    x = np.array([-1.0, 0.0, 0.1, 0.2, 1.5, 3.0, 4.0], np.float32)
    c, st = O.quantize_act(x, 3.0, O.ACT_U4)
    assert st == np.float32(np.float32(3.0) / np.float32(15))
    assert list(c) == [0, 0, 0, 1, 8, 15, 15]     # 0.5 -> 0 (even), 1.0 -> 1, 7.5 -> 8
    c, st = O.quantize_act(x, 3.0, O.ACT_S4)
    assert st == np.float32(np.float32(3.0) / np.float32(7))
    assert list(c) == [O.fixed_q(v, 3.0, 4) for v in x]
    g = np.random.default_rng(3)
    xs = np.abs(g.standard_normal(5000)).astype(np.float32)
    c, st = O.quantize_act(xs, 3.0, O.ACT_U4)
    assert c.min() >= 0 and c.max() == 15
    inside = xs <= 3.0
    assert np.all(np.abs(c[inside] * float(st) - xs[inside]) <= float(st) / 2 * (1 + 1e-5))


# ----------------------------------------------------------------- ratio and assignment

def test_ratio_counts_formula():
    assert O.ratio_counts(256, (60, 35, 5)) == (154, 89, 13)
    assert O.ratio_counts(64, (60, 35, 5)) == (38, 23, 3)
    assert O.ratio_counts(768, (60, 35, 5)) == (461, 269, 38)
    assert O.ratio_counts(512, (65, 30, 5)) == (333, 153, 26)
    assert O.ratio_counts(100, (0, 100, 0)) == (0, 100, 0)
    assert O.ratio_counts(100, (100, 0, 0)) == (100, 0, 0)
    for M in range(1, 300, 7):
        for r in synth.RATIO_SWEEP + ((65, 30, 5),):
            a, b, c = O.ratio_counts(M, r)
            assert a + b + c == M and min(a, b, c) >= 0
            assert abs(a - M * r[0] / 100) <= 0.5 + 1e-9 or a == M - c
            assert abs(c - M * r[2] / 100) <= 0.5 + 1e-9


def test_assignment_follows_variance_order_and_ratio():
    g = synth.rng(99, 1)
    W = synth.weights_kaiming(g, 96, 16, 3, 3)
    scheme, bits = O.assign_rows(W, (60, 35, 5))
    var = W.reshape(96, -1).astype(np.float64).var(axis=1)
    pot = (scheme == 0)
    f4 = (scheme == 1) & (bits == 4)
    f8 = (scheme == 1) & (bits == 8)
    assert (pot.sum(), f4.sum(), f8.sum()) == O.ratio_counts(96, (60, 35, 5))
    assert np.all(bits[pot] == 4)                         # PoT never takes the higher precision
    assert var[pot].max() <= var[f4].min() <= var[f4].max() <= var[f8].min()
    assert abs(O.row_variance(W[3]) - var[3]) <= 1e-12 * var[3]
    # ties: equal rows are ordered by index
    W2 = np.tile(W[:1].reshape(1, -1), (10, 1))
    s2, b2 = O.assign_rows(W2, (50, 40, 10))
    assert list(s2) == [0] * 5 + [1] * 5 and list(b2) == [4] * 9 + [8]


def test_grouping_is_a_stable_sort_by_scheme():
    scheme = np.array([1, 0, 1, 0, 1, 0, 1], np.uint8)
    bits = np.array([4, 4, 8, 4, 4, 4, 8], np.uint8)
    perm = O.group_rows(scheme, bits)
    assert list(perm) == [1, 3, 5, 0, 4, 2, 6]


# ----------------------------------------------------------------- contraction

def _tiny_layer(seed, M=7, K=13, N=5, ratio=(60, 30, 10)):
    g = np.random.default_rng(seed)
    W = (g.standard_normal((M, K)) * 0.02).astype(np.float32)
    scheme, bits = O.assign_rows(W, ratio)
    alpha = synth.alpha_rows(W)
    act = g.integers(0, 16, (N, K), dtype=np.int8)
    return W, scheme, bits, alpha, act


def test_matmul_brute_force_python_loops():
    W, scheme, bits, alpha, act = _tiny_layer(11)
    v, ws, acc, y = O.layer_linear(W, scheme, bits, alpha, act, np.float32(0.1))
    M, K = W.shape
    for n in range(act.shape[0]):
        for r in range(M):
            s = 0
            for k in range(K):
                s += int(v[r, k]) * int(act[n, k])
            assert acc[n, r] == s
            c = np.float32(ws[r] * np.float32(0.1))
            assert y[n, r] == np.float32(np.float32(s) * c)


def test_matmul_equals_numpy_int64_and_no_overflow():
    g = np.random.default_rng(12)
    v = g.integers(-127, 128, (33, 257), dtype=np.int8)
    a = g.integers(-7, 16, (19, 257), dtype=np.int8)
    want = a.astype(np.int64) @ v.astype(np.int64).T
    assert np.array_equal(O.matmul(v, a).astype(np.int64), want)
    assert np.array_equal(O.matmul_i64(v, a), want)
    # all-Fixed-8 rows with alpha = 127 and unit activation step is a textbook integer matmul
    W = v.astype(np.float32)
    vals, ws, acc, y = O.layer_linear(W, np.ones(33, np.uint8), np.full(33, 8, np.uint8),
                                      np.full(33, 127.0, np.float32), a, np.float32(1.0))
    assert np.array_equal(vals, v) and np.all(ws == 1.0)
    assert np.array_equal(y.astype(np.int64), want)


def test_pot_rows_by_shift_add_equal_multiply_form():
    g = np.random.default_rng(13)
    nib = g.integers(0, 16, (9, 40), dtype=np.uint8)
    nib[nib == 8] = 0
    vals = np.array([[O.pot_value(int(c)) for c in row] for row in nib], np.int8)
    a = g.integers(-7, 16, (6, 40), dtype=np.int8)
    assert np.array_equal(O.matmul_pot_shift(nib, a), O.matmul(vals, a))


def test_one_hot_activations_return_weight_columns_and_linearity():
    W, scheme, bits, alpha, act = _tiny_layer(14, M=10, K=12, N=12)
    eye = np.eye(12, dtype=np.int8)
    v, ws, acc, y = O.layer_linear(W, scheme, bits, alpha, eye, np.float32(1.0))
    assert np.array_equal(acc, v.T.astype(np.int32))
    # dequantized weights lie within half a step (Fixed) of the originals
    fx = scheme == 1
    assert np.all(np.abs(y.T[fx] - W[fx]) <= ws[fx, None] / 2 * (1 + 1e-5))
    a1 = act[:5]
    a2 = np.random.default_rng(1).integers(0, 8, a1.shape, dtype=np.int8)
    assert np.array_equal(O.matmul(v, a1 + a2), O.matmul(v, a1) + O.matmul(v, a2))


def test_output_close_to_double_precision_product():
    W, scheme, bits, alpha, act = _tiny_layer(15, M=24, K=300, N=9)
    v, ws, acc, y = O.layer_linear(W, scheme, bits, alpha, act, np.float32(3.0 / 15))
    Qw = np.where(scheme == 0, 64.0, np.where(bits == 4, 7.0, 127.0))
    ref = acc.astype(np.float64) * (alpha.astype(np.float64) / Qw)[None, :] * (3.0 / 15)
    nz = ref != 0
    assert np.all(np.abs(y[nz] - ref[nz]) <= 1e-6 * np.abs(ref[nz]))


# ----------------------------------------------------------------- convolution

def _im2col(act, kh, kw, stride, pad):
    B, H, W, Cc = act.shape
    Ho, Wo = O.conv_out_hw(H, W, kh, kw, stride, pad)
    ap = np.zeros((B, H + 2 * pad, W + 2 * pad, Cc), act.dtype)
    ap[:, pad:pad + H, pad:pad + W] = act
    cols = np.empty((B, Ho, Wo, Cc, kh, kw), act.dtype)
    for i in range(kh):
        for j in range(kw):
            cols[..., i, j] = ap[:, i:i + stride * Ho:stride, j:j + stride * Wo:stride]
    return cols.reshape(B * Ho * Wo, Cc * kh * kw)


@pytest.mark.parametrize("k,stride,pad,H", [(3, 1, 1, 6), (3, 2, 1, 7), (1, 2, 0, 6), (1, 1, 0, 4),
                                             (3, 2, 1, 8)])
def test_conv_equals_im2col_times_matmul(k, stride, pad, H):
    g = np.random.default_rng(16 + k + stride)
    v = g.integers(-127, 128, (5, 6, k, k), dtype=np.int8)
    a = g.integers(0, 16, (2, H, H + 1, 6), dtype=np.int8)
    acc = O.conv(v, a, stride, pad)
    cols = _im2col(a, k, k, stride, pad)
    want = cols.astype(np.int64) @ v.reshape(5, -1).astype(np.int64).T
    assert np.array_equal(acc.reshape(-1, 5).astype(np.int64), want)
    n_idx = np.array([0, 3, acc.size // 5 - 1])
    r_idx = np.array([4, 0, 2], np.int32)
    assert np.array_equal(O.conv_points(v, a, stride, pad, n_idx, r_idx),
                          acc.reshape(-1, 5)[n_idx, r_idx])


def test_conv_1x1_stride1_is_the_linear_layer():
    g = np.random.default_rng(17)
    v = g.integers(-7, 8, (6, 10, 1, 1), dtype=np.int8)
    a = g.integers(0, 16, (3, 4, 5, 10), dtype=np.int8)
    acc = O.conv(v, a, 1, 0)
    lin = O.matmul(v.reshape(6, 10), a.reshape(-1, 10))
    assert np.array_equal(acc.reshape(-1, 6), lin)
    n_idx, r_idx = np.array([0, 7, 59]), np.array([1, 5, 0], np.int32)
    assert np.array_equal(O.matmul_points(v.reshape(6, 10), a.reshape(-1, 10), n_idx, r_idx),
                          lin[n_idx, r_idx])


# ----------------------------------------------------------------- operation count convention

def test_op_count_convention_matches_table6():
    """Table 6: throughput x latency is the operation count of one ResNet-18 image; with two
    operations per multiply-accumulate the layer list must give the same number."""
    prods = []
    for line in open(os.path.join(GOLD, "table6_fpga.txt")):
        if line.startswith("#") or not line.strip():
            continue
        f = line.split()
        prods.append(float(f[3]) * float(f[4]) / 1e3)        # GOP per image
    assert len(prods) == 16
    assert 3.55 < min(prods) and max(prods) < 3.70
    macs = sum(L.macs(1) * L.count for L in synth.resnet18_convs())
    macs += synth.RESNET18_CONV1.macs(1) + synth.RESNET18_FC_MACS
    assert abs(2 * macs / 1e9 - float(np.median(prods))) < 0.03
    assert sum(L.count for L in synth.resnet18_convs()) == 19


def test_depthwise_conv_is_the_dense_conv_with_block_diagonal_filters():
    """Pin of the depthwise oracle: the same sums as the ordinary convolution when filter c is zero on
    every input channel but c (the definition of a depthwise layer), at three geometries; and one
    output re-added by hand."""
    g = np.random.default_rng(11)
    for (Cc, k, stride, pad, B, H, W) in ((8, 3, 1, 1, 2, 6, 7), (12, 3, 2, 1, 1, 9, 8), (4, 5, 1, 2, 2, 5, 5)):
        v = g.integers(-127, 128, size=(Cc, k, k)).astype(np.int8)
        a = g.integers(-7, 16, size=(B, H, W, Cc)).astype(np.int8)
        dense = np.zeros((Cc, Cc, k, k), np.int8)
        for c in range(Cc):
            dense[c, c] = v[c]
        got = O.conv_depthwise(v, a, stride, pad)
        assert np.array_equal(got, O.conv(dense, a, stride, pad))
        b, ho, wo, c = B - 1, 1, 2, Cc - 1
        s = 0
        for i in range(k):
            for j in range(k):
                y, x = ho * stride + i - pad, wo * stride + j - pad
                if 0 <= y < H and 0 <= x < W:
                    s += int(v[c, i, j]) * int(a[b, y, x, c])
        assert got[b, ho, wo, c] == s


def test_patch_matrix_times_flattened_filters_is_the_convolution():
    """im2col against the direct convolution (a different code path: the C loop nest), over stride, padding and
    an odd channel count; and its zero padding and column order on a hand-made case."""
    g = np.random.default_rng(41)
    for (Cin, k, stride, pad, H, W) in [(3, 7, 2, 3, 11, 9), (3, 3, 1, 1, 5, 6), (5, 2, 2, 0, 6, 6), (1, 3, 1, 2, 4, 4)]:
        V = g.integers(-7, 8, (6, Cin, k, k), dtype=np.int8)
        act = g.integers(-8, 16, (2, H, W, Cin), dtype=np.int8)
        cols = O.im2col(act, k, k, stride, pad, ld=(k * k * Cin + 15) // 16 * 16)
        Vl = np.zeros((6, cols.shape[1]), np.int8)
        Vl[:, :k * k * Cin] = V.transpose(0, 2, 3, 1).reshape(6, -1)
        assert np.array_equal(O.matmul(Vl, cols), O.conv(V, act, stride, pad).reshape(-1, 6))
        assert not cols[:, k * k * Cin:].any()
    # one pixel, 2 channels (codes 5, 6), 2 x 2 filter, pad 1: four output pixels, each seeing the pixel at another tap
    cols = O.im2col(np.array([[[[5, 6]]]], np.int8), 2, 2, 1, 1)
    assert cols.tolist() == [[0, 0, 0, 0, 0, 0, 5, 6], [0, 0, 0, 0, 5, 6, 0, 0], [0, 0, 5, 6, 0, 0, 0, 0], [5, 6, 0, 0, 0, 0, 0, 0]]
