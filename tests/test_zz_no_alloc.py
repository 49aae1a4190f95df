"""The allocation-free linear layer (rmsmp_gemm_builtin_scratch) against the workspace path.

Some callers of the library may not allocate device memory when they call it (a plugin inside
a runtime with a fixed arena, a latency-critical loop); for them the scratch of the workspace
variant is an array inside the library.  The test runs the entry point twice in a row through
the C ABI -- a large layer first, then a smaller one, so the second call finds the first call's
bytes still in the shared array -- and requires the same bits as the caller-scratch path and
as the CPU oracle's linear layer.  A call that is refused (bad argument, shape the tensor kernel
cannot run) must not have touched the array.  This file is collected last on purpose.
"""
import numpy as np
import pytest

from oracle import rmsmp_oracle as O
from paper_2111_00153_b200 import binding as R
from paper_2111_00153_b200 import synth
from tests import harness as Hn

pytestmark = pytest.mark.gpu


def _run(M, K, N, seed):
    import torch
    g = synth.rng(80, seed)
    W = synth.weights_normal(g, (M, K))
    scheme, bits = R.rmsmp_assign_rows(W, synth.RATIO_RMSMP1)
    alpha = synth.alpha_rows(W)
    act = synth.act_codes_uniform(g, (N, K))
    layer, d_packed = Hn.pack_layer(W, scheme, bits, alpha)
    a = torch.from_numpy(act).cuda()
    step = float(np.float32(0.2))

    y_ref = torch.empty((N, M), dtype=torch.float32, device="cuda")
    acc_ref = torch.empty((N, M), dtype=torch.int32, device="cuda")
    ws = torch.empty(R.rmsmp_workspace_bytes(layer), dtype=torch.int8, device="cuda")
    R.rmsmp_expand_weights(layer, d_packed, ws)
    R.rmsmp_gemm_workspace(layer, d_packed, ws, a, N, K, step, y_ref, M, R.OUT_NM, acc_ref)

    y = torch.full((N, M), float("nan"), dtype=torch.float32, device="cuda")
    acc = torch.full((N, M), -1, dtype=torch.int32, device="cuda")
    R.rmsmp_gemm_builtin_scratch(layer, d_packed, a, N, K, step, y, M, R.OUT_NM, acc)
    torch.cuda.synchronize()
    assert R.rmsmp_last_device_status(d_packed) == R.OK
    assert torch.equal(acc, acc_ref)
    assert np.array_equal(y.cpu().numpy().view(np.uint32), y_ref.cpu().numpy().view(np.uint32))
    _, _, acc_o, y_o = O.layer_linear(W, scheme, bits, alpha, act, np.float32(step))
    assert np.array_equal(acc.cpu().numpy(), acc_o)
    assert np.array_equal(y.cpu().numpy().view(np.uint32), y_o.view(np.uint32))


def test_two_calls_in_a_row_match_the_workspace_path():
    _run(768, 3072, 300, 1)      # 2.25 MiB of the array
    _run(130, 512, 77, 2)        # a smaller layer on top of the first call's leftovers


def test_layer_beyond_the_built_in_scratch_is_rejected():
    import torch
    M, K = 2048, 4096             # 8 MiB of expanded weights: over the 4 MiB limit
    scheme = np.ones(M, np.uint8)
    bits = np.full(M, 4, np.uint8)
    layer = R.rmsmp_layer_init(M, K, 1, 1, scheme, bits)
    buf = torch.zeros(4096, dtype=torch.uint8, device="cuda")
    with pytest.raises(R.RmsmpError) as e:
        R.rmsmp_gemm_builtin_scratch(layer, buf, buf, 16, K, 1.0, buf, M)
    assert e.value.status == R.ERR_BUFFER_TOO_SMALL


def test_refused_calls_leave_the_shared_array_alone():
    """A good call, then calls that must be refused before anything is queued, then the good call
    again: the refusals return their documented codes and the repeated call is still bit-exact."""
    import torch
    _run(256, 512, 64, 3)
    # K = 40 is not a multiple of 16: only the tensor-core kernel exists behind this entry point
    g = synth.rng(80, 4)
    W = synth.weights_normal(g, (64, 40))
    scheme, bits = R.rmsmp_assign_rows(W, synth.RATIO_RMSMP1)
    layer, d_packed = Hn.pack_layer(W, scheme, bits, synth.alpha_rows(W))
    a = torch.zeros((8, 48), dtype=torch.int8, device="cuda")
    y = torch.zeros((8, 64), dtype=torch.float32, device="cuda")
    with pytest.raises(R.RmsmpError) as e:
        R.rmsmp_gemm_builtin_scratch(layer, d_packed, a, 8, 48, 0.1, y, 64)
    assert e.value.status == R.ERR_VARIANT
    # output leading dimension smaller than M, and a misaligned activation pointer
    g = synth.rng(80, 5)
    W = synth.weights_normal(g, (128, 256))
    scheme, bits = R.rmsmp_assign_rows(W, synth.RATIO_RMSMP1)
    layer, d_packed = Hn.pack_layer(W, scheme, bits, synth.alpha_rows(W))
    a = torch.zeros((8 * 256 + 16,), dtype=torch.int8, device="cuda")
    y = torch.zeros((8, 128), dtype=torch.float32, device="cuda")
    with pytest.raises(R.RmsmpError) as e:
        R.rmsmp_gemm_builtin_scratch(layer, d_packed, a, 8, 256, 0.1, y, 64)
    assert e.value.status == R.ERR_SHAPE
    with pytest.raises(R.RmsmpError) as e:
        R.rmsmp_gemm_builtin_scratch(layer, d_packed, a[1:], 8, 256, 0.1, y, 128)
    assert e.value.status == R.ERR_ALIGN
    torch.cuda.synchronize()
    _run(256, 512, 64, 3)
