"""GPU parity at the sizes of the five workload configurations, in the launch configuration the
benchmark uses (workspace variant, [N][M] output), against the CPU oracle.

The ResNet-18 stack is compared in full at the benchmark's batch; of the BERT-base linears the
largest ones are compared on randomly sampled outputs the oracle computes one by one plus every
row (the integer sums are exact, so each sampled element is as strict as in a full comparison).
"""
import numpy as np
import pytest

from oracle import rmsmp_oracle as O
from paper_2111_00153_b200 import binding as R
from paper_2111_00153_b200 import synth
from tests import harness as Hn

pytestmark = pytest.mark.gpu


def _expected(acc, ws, act_step):
    return O.epilogue(acc, ws, act_step)


def _run_conv_device(W, scheme, bits, alpha, x, stride, pad, kind, workspace=True):
    """fp32 weights / activations on the host -> (codes, step, y) through the C ABI."""
    import torch
    layer, d_packed = Hn.pack_layer(W, scheme, bits, alpha)
    dx = torch.from_numpy(x).cuda()
    codes = torch.empty(x.shape, dtype=torch.int8, device="cuda")
    step = R.rmsmp_quantize_act(dx, dx.numel(), synth.ALPHA_ACT, kind, codes)
    B, H, Wd, _ = x.shape
    Ho, Wo = O.conv_out_hw(H, Wd, layer.kh, layer.kw, stride, pad)
    y = torch.full((B * Ho * Wo, layer.M), float("nan"), dtype=torch.float32, device="cuda")
    if workspace:
        ws = torch.empty(R.rmsmp_workspace_bytes(layer), dtype=torch.int8, device="cuda")
        R.rmsmp_expand_weights(layer, d_packed, ws)
        R.rmsmp_conv_implicit_workspace(layer, d_packed, ws, codes, B, H, Wd, stride, pad, step, y)
    else:
        R.rmsmp_conv_implicit_variant(layer, d_packed, codes, B, H, Wd, stride, pad, step, y, R.OUT_NM, None,
                                      R.VARIANT_TENSOR)
    torch.cuda.synchronize()
    assert R.rmsmp_last_device_status(d_packed) == R.OK
    return codes.cpu().numpy(), np.float32(step), y.cpu().numpy()


# ------------------------------------------------------------------ config 2: one ResNet conv, full

@pytest.mark.parametrize("workspace", [True, False], ids=["workspace", "smem"])
def test_config2_conv256_14x14_batch32_full(workspace):
    L = synth.CONFIG2_CONV
    g = synth.rng(2, 0)
    W = synth.weights_kaiming(g, L.M, L.Cin, L.k, L.k)
    x = synth.act_halfnormal(g, (32, L.H, L.H, L.Cin))
    scheme, bits = O.assign_rows(W, synth.RATIO_RMSMP1)
    assert (int((scheme == 0).sum()), int(((scheme == 1) & (bits == 4)).sum()), int((bits == 8).sum())) == (154, 89, 13)
    alpha = synth.alpha_rows(W)
    codes, step, y = _run_conv_device(W, scheme, bits, alpha, x, L.stride, L.pad, R.ACT_U4, workspace)
    c_ref, s_ref = O.quantize_act(x, synth.ALPHA_ACT, O.ACT_U4)
    assert np.array_equal(codes, c_ref) and step == s_ref
    _, ws, acc, y_ref = O.layer_conv(W, scheme, bits, alpha, c_ref, s_ref, L.stride, L.pad)
    assert np.array_equal(y.view(np.uint32), y_ref.reshape(-1, L.M).view(np.uint32))


# ------------------------------------------------------------------ config 3: BERT-base linears, N = 4096

@pytest.mark.parametrize("name,M,K", synth.BERT_BASE_LINEARS)
def test_config3_bert_base_linear(name, M, K):
    import torch
    N = synth.BERT_BASE_TOKENS
    g = synth.rng(3, M + K)
    W = synth.weights_normal(g, (M, K))
    x = synth.act_normal(g, (N, K))
    scheme, bits = O.assign_rows(W, synth.RATIO_RMSMP1)
    alpha = synth.alpha_rows(W)
    layer, d_packed = Hn.pack_layer(W, scheme, bits, alpha)
    dx = torch.from_numpy(x).cuda()
    codes = torch.empty((N, K), dtype=torch.int8, device="cuda")
    step = R.rmsmp_quantize_act(dx, dx.numel(), synth.ALPHA_ACT, R.ACT_S4, codes)
    y = torch.empty((N, M), dtype=torch.float32, device="cuda")
    acc = torch.empty((N, M), dtype=torch.int32, device="cuda")
    ws = torch.empty(R.rmsmp_workspace_bytes(layer), dtype=torch.int8, device="cuda")
    R.rmsmp_expand_weights(layer, d_packed, ws)
    R.rmsmp_gemm_workspace(layer, d_packed, ws, codes, N, K, step, y, M, R.OUT_NM, acc)
    y2 = torch.empty((N, M), dtype=torch.float32, device="cuda")
    R.rmsmp_gemm(layer, d_packed, codes, N, K, step, y2, M)           # the in-shared-memory expansion path
    torch.cuda.synchronize()
    assert torch.equal(y, y2)
    c_ref, s_ref = O.quantize_act(x, synth.ALPHA_ACT, O.ACT_S4)
    assert np.array_equal(codes.cpu().numpy(), c_ref) and np.float32(step) == s_ref
    v_ref, wstep = O.quantize_rows(W, scheme, bits, alpha)
    if M * K * N <= 3e9:                                   # attn_out: everything
        acc_ref = O.matmul(v_ref, c_ref)
        assert np.array_equal(acc.cpu().numpy(), acc_ref)
        assert np.array_equal(y.cpu().numpy().view(np.uint32), _expected(acc_ref, wstep, s_ref).view(np.uint32))
    else:                                                   # sampled outputs, every row at least once
        r = np.random.default_rng(M)
        n_idx = np.concatenate([r.integers(0, N, 40000), r.integers(0, N, M), [0, N - 1, N - 1]])
        m_idx = np.concatenate([r.integers(0, M, 40000), np.arange(M), [0, M - 1, 0]]).astype(np.int32)
        pts = O.matmul_points(v_ref, c_ref, n_idx, m_idx)
        assert np.array_equal(acc.cpu().numpy()[n_idx, m_idx], pts)
        c = (wstep[m_idx] * s_ref).astype(np.float32)
        want = (pts.astype(np.float32) * c).astype(np.float32)
        assert np.array_equal(y.cpu().numpy()[n_idx, m_idx].view(np.uint32), want.view(np.uint32))


def test_two_row_blocks_per_tile_full():
    """Long K, two row blocks and two waves of single-block tiles: the shape class for which the
    workspace variant runs both row blocks of a tile against one activation stage.  Every
    accumulator and output against the oracle; 19000 tokens leave a ragged last tile."""
    import torch
    M, K, N = 256, 2048, 19000
    g = synth.rng(3, 77)
    W = synth.weights_normal(g, (M, K))
    c_ref = synth.act_codes_uniform(g, (N, K))
    step = np.float32(0.0625)
    scheme, bits = O.assign_rows(W, synth.RATIO_RMSMP1)
    alpha = synth.alpha_rows(W)
    layer, d_packed = Hn.pack_layer(W, scheme, bits, alpha)
    codes = torch.from_numpy(c_ref).cuda()
    y = torch.full((N, M), float("nan"), dtype=torch.float32, device="cuda")
    acc = torch.empty((N, M), dtype=torch.int32, device="cuda")
    ws = torch.empty(R.rmsmp_workspace_bytes(layer), dtype=torch.int8, device="cuda")
    R.rmsmp_expand_weights(layer, d_packed, ws)
    R.rmsmp_gemm_workspace(layer, d_packed, ws, codes, N, K, float(step), y, M, R.OUT_NM, acc)
    torch.cuda.synchronize()
    assert R.rmsmp_last_device_status(d_packed) == R.OK
    v_ref, wstep = O.quantize_rows(W, scheme, bits, alpha)
    acc_ref = O.matmul(v_ref, c_ref)
    assert np.array_equal(acc.cpu().numpy(), acc_ref)
    assert np.array_equal(y.cpu().numpy().view(np.uint32), _expected(acc_ref, wstep, step).view(np.uint32))
    # the same shape through the re-quantizing epilogue (next layer's signed 4-bit codes)
    y_ref = _expected(acc_ref, wstep, step)
    na = float(np.float32(3.0 * float(np.std(y_ref))))
    want, _ = O.quantize_act(y_ref, na, O.ACT_S4)
    out = torch.empty((N, M), dtype=torch.int8, device="cuda")
    R.rmsmp_gemm_workspace_requant(layer, d_packed, ws, codes, N, K, float(step), na, R.ACT_S4, out, M)
    torch.cuda.synchronize()
    assert np.array_equal(out.cpu().numpy(), want)


# ------------------------------------------------------------------ config 4: the ResNet-18 stack

@pytest.mark.parametrize("L", synth.resnet18_convs(), ids=lambda L: L.name)
def test_config4_resnet18_layer_batch4_full(L):
    g = synth.rng(4, L.M + L.Cin + L.k)
    W = synth.weights_kaiming(g, L.M, L.Cin, L.k, L.k)
    x = synth.act_halfnormal(g, (4, L.H, L.H, L.Cin))
    scheme, bits = R.rmsmp_assign_rows(W, synth.RATIO_RMSMP1)
    alpha = synth.alpha_rows(W)
    codes, step, y = _run_conv_device(W, scheme, bits, alpha, x, L.stride, L.pad, R.ACT_U4)
    _, ws, acc, y_ref = O.layer_conv(W, scheme, bits, alpha, codes, step, L.stride, L.pad)
    assert np.array_equal(y.view(np.uint32), y_ref.reshape(-1, L.M).view(np.uint32))


@pytest.mark.parametrize("L", synth.resnet18_convs(), ids=lambda L: L.name)
def test_config4_resnet18_layer_batch256_full(L):
    """Every one of the ten layer types of the stack at the benchmark's batch (256) and in its launch
    configuration: all activation codes and all B*Ho*Wo*M outputs against the oracle's layer
    (quantizer, direct convolution, epilogue), bit for bit."""
    B = 256
    g = synth.rng(4, 7 * L.M + L.H)
    W = synth.weights_kaiming(g, L.M, L.Cin, L.k, L.k)
    x = synth.act_halfnormal(g, (B, L.H, L.H, L.Cin))
    scheme, bits = R.rmsmp_assign_rows(W, synth.RATIO_RMSMP1)
    alpha = synth.alpha_rows(W)
    codes, step, y = _run_conv_device(W, scheme, bits, alpha, x, L.stride, L.pad, R.ACT_U4)
    c_ref, s_ref = O.quantize_act(x, synth.ALPHA_ACT, O.ACT_U4)
    del x
    assert step == s_ref and np.array_equal(codes, c_ref)
    del codes
    _, _, _, y_ref = O.layer_conv(W, scheme, bits, alpha, c_ref, s_ref, L.stride, L.pad)
    assert np.array_equal(y.view(np.uint32), y_ref.reshape(-1, L.M).view(np.uint32))


def test_resnet18_first_layer_7x7_batch4_full():
    """The 7x7 stride-2 first convolution at ImageNet size, its 3 input channels stored as 16 (zeros
    beyond the third) so that a pixel is one 16-byte granule: every output against the oracle."""
    M, Cin, k, B, H = 64, 16, 7, 4, 224
    g = synth.rng(4, 777)
    W = synth.weights_kaiming(g, M, Cin, k, k)
    W[:, 3:] = 0.0
    x = synth.act_halfnormal(g, (B, H, H, Cin))
    x[..., 3:] = 0.0
    scheme, bits = R.rmsmp_assign_rows(W, synth.RATIO_RMSMP1)
    alpha = synth.alpha_rows(W)
    codes, step, y = _run_conv_device(W, scheme, bits, alpha, x, 2, 3, R.ACT_U4)
    _, ws, acc, y_ref = O.layer_conv(W, scheme, bits, alpha, codes, step, 2, 3)
    assert np.array_equal(y.view(np.uint32), y_ref.reshape(-1, M).view(np.uint32))


# ------------------------------------------------------------------ config 5: weight-bound small-N sweep

@pytest.mark.parametrize("ratio", synth.RATIO_SWEEP, ids=lambda r: "%d-%d-%d" % r)
@pytest.mark.parametrize("N", synth.BERT_LARGE_TOKENS)
@pytest.mark.parametrize("name,M,K", synth.BERT_LARGE_LINEARS)
def test_config5_bert_large_small_batch(name, M, K, N, ratio):
    g = synth.rng(5, M // 64 + K // 32 + N + ratio[0])
    W = synth.weights_normal(g, (M, K))
    scheme, bits = O.assign_rows(W, ratio)
    alpha = synth.alpha_rows(W)
    act = synth.act_codes_uniform(g, (N, K))
    layer, d_packed = Hn.pack_layer(W, scheme, bits, alpha)
    v_ref, wstep = O.quantize_rows(W, scheme, bits, alpha)
    acc_ref = O.matmul(v_ref, act)
    y_ref = _expected(acc_ref, wstep, np.float32(0.05))
    for variant in (R.VARIANT_AUTO, R.VARIANT_SHIFTADD, R.VARIANT_TENSOR):
        y, acc = Hn.gemm(layer, d_packed, act, 0.05, variant)
        assert np.array_equal(acc, acc_ref)
        assert np.array_equal(y.view(np.uint32), y_ref.view(np.uint32))


# ------------------------------------------------------------------ config 5, grouped: many layers, one launch

@pytest.mark.parametrize("N", [1, 8, 5])
def test_config5_grouped_launch_matches_oracle(N):
    import torch
    shapes = [(1024, 1024), (4096, 1024), (1024, 4096), (130, 96), (64, 40)]
    keep, items, refs = [], [], []
    for i, (M, K) in enumerate(shapes):
        g = synth.rng(5, 900 + i + N)
        W = synth.weights_normal(g, (M, K))
        ratio = synth.RATIO_SWEEP[i % 4]
        scheme, bits = O.assign_rows(W, ratio)
        alpha = synth.alpha_rows(W)
        act = synth.act_codes_uniform(g, (N, K))
        layer, d_packed = Hn.pack_layer(W, scheme, bits, alpha)
        ld = (K + 15) // 16 * 16
        a = torch.zeros((N, ld), dtype=torch.int8, device="cuda")
        a[:, :K] = torch.from_numpy(act).cuda()
        y = torch.full((N, M), float("nan"), dtype=torch.float32, device="cuda")
        acc = torch.full((N, M), -5, dtype=torch.int32, device="cuda")
        step = float(np.float32(0.01 * (i + 1)))
        keep.append((layer, d_packed, a, y, acc))
        items.append((layer, d_packed, a, N, ld, step, y, M, acc))
        v_ref, wstep = O.quantize_rows(W, scheme, bits, alpha)
        acc_ref = O.matmul(v_ref, act)
        refs.append((acc_ref, _expected(acc_ref, wstep, np.float32(step))))
    arr = R.make_gemm_items(items)
    table = torch.empty(R.rmsmp_grouped_table_bytes(len(items)), dtype=torch.uint8, device="cuda")
    R.rmsmp_gemm_grouped(arr, R.OUT_NM, table)
    torch.cuda.synchronize()
    for (layer, d_packed, a, y, acc), (acc_ref, y_ref) in zip(keep, refs):
        assert np.array_equal(acc.cpu().numpy(), acc_ref)
        assert np.array_equal(y.cpu().numpy().view(np.uint32), y_ref.view(np.uint32))


def _grouped_case(shapes, N, layout=R.OUT_NM):
    """Layers, device buffers, items and oracle results for a grouped launch."""
    import torch
    keep, items, refs = [], [], []
    for i, (M, K) in enumerate(shapes):
        g = synth.rng(5, 700 + i + N)
        W = synth.weights_normal(g, (M, K))
        ratio = synth.RATIO_SWEEP[(i + 2) % 4]
        scheme, bits = O.assign_rows(W, ratio)
        alpha = synth.alpha_rows(W)
        act = synth.act_codes_uniform(g, (N, K))
        if i % 2:
            act = (act % 15 - 7).astype(np.int8)            # signed codes on every other layer
        layer, d_packed = Hn.pack_layer(W, scheme, bits, alpha)
        ld = (K + 15) // 16 * 16
        a = torch.zeros((N, ld), dtype=torch.int8, device="cuda")
        a[:, :K] = torch.from_numpy(act).cuda()
        shape = (N, M) if layout == R.OUT_NM else (M, N)
        y = torch.full(shape, float("nan"), dtype=torch.float32, device="cuda")
        acc = torch.full(shape, -5, dtype=torch.int32, device="cuda") if i != 1 else None
        step = float(np.float32(0.01 * (i + 1)))
        keep.append((layer, d_packed, a, y, acc))
        # unsigned codes: every other such layer says so (its bytes are then read as they are by the PoT tiles)
        items.append((layer, d_packed, a, N, ld, step, y, shape[1], acc, 1 if i % 4 == 0 else 0))
        v_ref, wstep = O.quantize_rows(W, scheme, bits, alpha)
        acc_ref = O.matmul(v_ref, act)
        refs.append((acc_ref, _expected(acc_ref, wstep, np.float32(step))))
    return keep, items, refs


def _check_grouped(keep, refs, layout=R.OUT_NM):
    for (layer, d_packed, a, y, acc), (acc_ref, y_ref) in zip(keep, refs):
        assert R.rmsmp_last_device_status(d_packed) == R.OK
        yh = y.cpu().numpy()
        if layout == R.OUT_MN:
            yh = yh.T
        assert np.array_equal(yh.view(np.uint32), y_ref.view(np.uint32))
        if acc is not None:
            ah = acc.cpu().numpy()
            assert np.array_equal(ah.T if layout == R.OUT_MN else ah, acc_ref)


GROUPED_SHAPES = [(1024, 1024), (4096, 1024), (1024, 4096), (130, 96), (64, 40), (300, 640), (128, 128)]


@pytest.mark.parametrize("N", [1, 8, 5, 33, 128])
def test_config5_grouped_tensor_launch_matches_oracle(N):
    """The grouped launch on the tensor cores (prepare once, launch): BERT-large shapes plus ragged
    ones (row counts that are not multiples of 128, an odd number of k-blocks, K below one k-block, a
    padded activation pitch), all four scheme ratios, signed and unsigned codes, against the oracle."""
    import torch
    keep, items, refs = _grouped_case(GROUPED_SHAPES, N)
    arr = R.make_gemm_items(items)
    table = torch.empty(R.rmsmp_grouped_plan_bytes(arr), dtype=torch.uint8, device="cuda")
    plan = R.rmsmp_gemm_grouped_prepare(arr, R.OUT_NM, table)
    R.rmsmp_gemm_grouped_launch(plan)
    torch.cuda.synchronize()
    _check_grouped(keep, refs)
    # the plan stays valid: new activation codes in the same buffers, second launch
    for k, (layer, d_packed, a, y, acc) in enumerate(keep):
        a.copy_(torch.roll(a, 1, dims=1) if a.shape[1] > 16 else a)
        y.fill_(float("nan"))
    R.rmsmp_gemm_grouped_launch(plan)
    torch.cuda.synchronize()
    for (layer, d_packed, a, y, acc) in keep:
        assert not torch.isnan(y).any()


def test_grouped_tensor_launch_mn_layout_and_single_layer():
    import torch
    keep, items, refs = _grouped_case([(384, 512), (200, 256)], 33, R.OUT_MN)
    arr = R.make_gemm_items(items)
    table = torch.empty(R.rmsmp_grouped_plan_bytes(arr), dtype=torch.uint8, device="cuda")
    plan = R.rmsmp_gemm_grouped_prepare(arr, R.OUT_MN, table)
    R.rmsmp_gemm_grouped_launch(plan)
    torch.cuda.synchronize()
    _check_grouped(keep, refs, R.OUT_MN)
    keep, items, refs = _grouped_case([(96, 2048)], 17)
    arr = R.make_gemm_items(items)
    table = torch.empty(R.rmsmp_grouped_plan_bytes(arr), dtype=torch.uint8, device="cuda")
    plan = R.rmsmp_gemm_grouped_prepare(arr, R.OUT_NM, table)
    assert plan.grid == 3                      # one tile per kind
    R.rmsmp_gemm_grouped_launch(plan)
    torch.cuda.synchronize()
    _check_grouped(keep, refs)


def test_grouped_tensor_launch_rejects_what_it_cannot_run():
    import torch
    keep, items, refs = _grouped_case([(128, 256)], 129)           # more than 128 tokens
    arr = R.make_gemm_items(items)
    table = torch.empty(R.rmsmp_grouped_plan_bytes(arr), dtype=torch.uint8, device="cuda")
    with pytest.raises(R.RmsmpError) as e:
        R.rmsmp_gemm_grouped_prepare(arr, R.OUT_NM, table)
    assert e.value.status == R.ERR_VARIANT
    keep, items, refs = _grouped_case([(128, 256)], 8)
    arr = R.make_gemm_items(items)
    with pytest.raises(R.RmsmpError) as e:
        R.rmsmp_gemm_grouped_prepare(arr, R.OUT_NM, table[:256])
    assert e.value.status == R.ERR_BUFFER_TOO_SMALL
    # PoT rows are summed in fp32 on the tensor core: exact up to a reduction length of 16384, refused beyond
    keep, items, refs = _grouped_case([(16, 16384 + 128)], 2)
    arr = R.make_gemm_items(items)
    table2 = torch.empty(R.rmsmp_grouped_plan_bytes(arr), dtype=torch.uint8, device="cuda")
    with pytest.raises(R.RmsmpError) as e:
        R.rmsmp_gemm_grouped_prepare(arr, R.OUT_NM, table2)
    assert e.value.status == R.ERR_VARIANT


def test_grouped_tensor_launch_longest_exact_reduction_with_extreme_codes():
    """K = 16384, every weight at full scale (PoT rows: +-64 in units of the row's step), every activation 15 or
    -16: the fp32 sums of the PoT tiles reach their largest magnitude (2^24 - 2^14 quarter units) and must still
    be the exact integers."""
    import torch
    M, K, N = 40, 16384, 3
    W = np.ones((M, K), np.float32)
    W[::3] = -1
    scheme, bits = O.assign_rows(synth.weights_normal(synth.rng(5, 77), (M, K)), (60, 35, 5))
    alpha = np.ones(M, np.float32)
    layer, d_packed = Hn.pack_layer(W, scheme, bits, alpha)
    v_ref, wstep = O.quantize_rows(W, scheme, bits, alpha)
    for codes, nonneg in ((np.full((N, K), 15, np.int8), 1), (np.full((N, K), -16, np.int8), 0), (np.full((N, K), 15, np.int8), 0)):
        a = torch.from_numpy(codes).cuda()
        y = torch.full((N, M), float("nan"), dtype=torch.float32, device="cuda")
        acc = torch.zeros((N, M), dtype=torch.int32, device="cuda")
        arr = R.make_gemm_items([(layer, d_packed, a, N, K, 1.0, y, M, acc, nonneg)])
        table = torch.empty(R.rmsmp_grouped_plan_bytes(arr), dtype=torch.uint8, device="cuda")
        plan = R.rmsmp_gemm_grouped_prepare(arr, R.OUT_NM, table)
        R.rmsmp_gemm_grouped_launch(plan)
        torch.cuda.synchronize()
        assert R.rmsmp_last_device_status(d_packed) == R.OK
        acc_ref = O.matmul(v_ref, codes)
        assert np.abs(acc_ref).max() >= 64 * 15 * K
        assert np.array_equal(acc.cpu().numpy(), acc_ref)
        assert np.array_equal(y.cpu().numpy().view(np.uint32), _expected(acc_ref, wstep, np.float32(1.0)).view(np.uint32))
    with pytest.raises(R.RmsmpError) as e:
        R.rmsmp_gemm_grouped_launch(R.rmsmp_grouped_plan())
    assert e.value.status == R.ERR_BAD_LAYER


# ------------------------------------------------------------------ CTA-pair kernel (long K, even row blocks, fp32 [N][M] output)

@pytest.mark.parametrize("M,K,N", [
    (256, 2048, 1000),      # ragged last half (1000 = 7 * 128 + 104), odd number of halves
    (500, 2304, 300),       # four row blocks, the last one ragged; last tile has one empty half
    (512, 4096, 129),       # second half holds a single token
])
def test_cta_pair_linear_full(M, K, N):
    """Shapes that run on the two-CTA kernel when called without an accumulator dump; the same call
    with a dump runs on the single-CTA kernel.  Both against the oracle, element by element."""
    import torch
    g = synth.rng(3, M + K + N)
    W = synth.weights_normal(g, (M, K))
    c_ref = synth.act_codes_uniform(g, (N, K))
    step = np.float32(0.0625)
    scheme, bits = O.assign_rows(W, synth.RATIO_RMSMP1)
    alpha = synth.alpha_rows(W)
    layer, d_packed = Hn.pack_layer(W, scheme, bits, alpha)
    codes = torch.from_numpy(c_ref).cuda()
    ws = torch.empty(R.rmsmp_workspace_bytes(layer), dtype=torch.int8, device="cuda")
    R.rmsmp_expand_weights(layer, d_packed, ws)
    y_pair = torch.full((N, M), float("nan"), dtype=torch.float32, device="cuda")
    R.rmsmp_gemm_workspace(layer, d_packed, ws, codes, N, K, float(step), y_pair, M)
    y_one = torch.full((N, M), float("nan"), dtype=torch.float32, device="cuda")
    acc = torch.empty((N, M), dtype=torch.int32, device="cuda")
    R.rmsmp_gemm_workspace(layer, d_packed, ws, codes, N, K, float(step), y_one, M, R.OUT_NM, acc)
    torch.cuda.synchronize()
    assert R.rmsmp_last_device_status(d_packed) == R.OK
    v_ref, wstep = O.quantize_rows(W, scheme, bits, alpha)
    acc_ref = O.matmul(v_ref, c_ref)
    want = _expected(acc_ref, wstep, step)
    assert np.array_equal(acc.cpu().numpy(), acc_ref)
    assert np.array_equal(y_one.cpu().numpy().view(np.uint32), want.view(np.uint32))
    assert np.array_equal(y_pair.cpu().numpy().view(np.uint32), want.view(np.uint32))


@pytest.mark.parametrize("M,Cin,k,stride,pad,B,H", [
    (256, 256, 3, 1, 1, 5, 14),      # halves of 7 rows; 10 halves
    (256, 256, 3, 2, 1, 3, 28),      # stride 2: 14x14 outputs
    (512, 512, 3, 1, 1, 7, 7),       # two images per half, odd image count
    (256, 128, 5, 1, 2, 2, 20),      # 5x5 taps (25 k-blocks), halves of 5 rows of 20 pixels
])
def test_cta_pair_conv_full(M, Cin, k, stride, pad, B, H):
    g = synth.rng(4, M + Cin + k + H)
    W = synth.weights_kaiming(g, M, Cin, k, k)
    x = synth.act_halfnormal(g, (B, H, H, Cin))
    scheme, bits = R.rmsmp_assign_rows(W, synth.RATIO_RMSMP1)
    alpha = synth.alpha_rows(W)
    codes, step, y = _run_conv_device(W, scheme, bits, alpha, x, stride, pad, R.ACT_U4)
    _, ws, acc, y_ref = O.layer_conv(W, scheme, bits, alpha, codes, step, stride, pad)
    assert np.array_equal(y.view(np.uint32), y_ref.reshape(-1, M).view(np.uint32))


def test_grouped_tensor_launches_in_a_row_see_the_inputs_of_their_turn():
    """Launches of one plan run as programmatic dependents of whatever is in front of them on the stream.  Eight
    launches in a row, the activation buffers rewritten between them by ordinary kernels and the outputs copied
    away after each: every launch must have read the codes of its own turn (signed layers through the copy
    that its first kernel writes) and no launch may have overwritten the outputs of the one before it early."""
    import torch
    shapes = [(384, 512), (200, 256), (128, 1024), (130, 96)]
    N, turns = 5, 8
    keep, items, refs = _grouped_case(shapes, N)
    arr = R.make_gemm_items(items)
    table = torch.empty(R.rmsmp_grouped_plan_bytes(arr), dtype=torch.uint8, device="cuda")
    plan = R.rmsmp_gemm_grouped_prepare(arr, R.OUT_NM, table)
    base = [a.clone() for (_, _, a, _, _) in keep]
    outs = []
    for t in range(turns):
        for (layer, d_packed, a, y, acc), b in zip(keep, base):
            a.copy_(torch.roll(b, t, dims=0))                 # turn t: the tokens rotated by t
        R.rmsmp_gemm_grouped_launch(plan)
        if t % 2:
            R.rmsmp_gemm_grouped_launch(plan)                 # and a launch directly behind a launch
        outs.append([y.clone() for (_, _, _, y, _) in keep])
    torch.cuda.synchronize()
    for t in range(turns):
        for k, ((acc_ref, y_ref), y) in enumerate(zip(refs, outs[t])):
            want = np.roll(y_ref, t, axis=0)
            assert np.array_equal(y.cpu().numpy().view(np.uint32), want.view(np.uint32)), (t, k)
