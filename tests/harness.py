"""Helpers shared by the GPU parity tests: run a layer through the C ABI and fetch results."""
from __future__ import annotations

import numpy as np

from paper_2111_00153_b200 import binding as R


def torch_mod():
    import torch
    return torch


def pack_layer(W: np.ndarray, scheme, bits, alpha, pot_mode=R.POT_NEAREST):
    """W: [M][K] or [M][Cin][kh][kw] fp32 (host).  Returns (layer, d_packed)."""
    torch = torch_mod()
    W = np.ascontiguousarray(W, np.float32)
    if W.ndim == 4:
        M, Cin, kh, kw = W.shape
        layout = R.W_CONV_OIHW
    else:
        M, Cin = W.shape
        kh = kw = 1
        layout = R.W_LINEAR
    layer = R.rmsmp_layer_init(M, Cin, kh, kw, scheme, bits)
    d_W = torch.from_numpy(W).cuda()
    d_packed = torch.empty(layer.packed_bytes, dtype=torch.uint8, device="cuda")
    R.rmsmp_quantize_pack(d_W, layout, layer, scheme, bits, alpha, pot_mode, d_packed)
    torch.cuda.synchronize()
    return layer, d_packed


def unpack(layer, d_packed):
    torch = torch_mod()
    M, K = layer.M, layer.K
    vals = torch.empty((M, K), dtype=torch.int8, device="cuda")
    perm = torch.empty(M, dtype=torch.int32, device="cuda")
    ws = torch.empty(M, dtype=torch.float32, device="cuda")
    R.rmsmp_unpack_codes(layer, d_packed, vals, perm, ws)
    torch.cuda.synchronize()
    return vals.cpu().numpy(), perm.cpu().numpy(), ws.cpu().numpy()


WORKSPACE = "workspace"     # pseudo-variant: expand once into scratch memory, then the tensor kernel


def _workspace(layer, d_packed):
    torch = torch_mod()
    ws = torch.empty(R.rmsmp_workspace_bytes(layer), dtype=torch.int8, device="cuda")
    R.rmsmp_expand_weights(layer, d_packed, ws)
    return ws


def gemm(layer, d_packed, act: np.ndarray, act_step, variant=R.VARIANT_AUTO, out_layout=R.OUT_NM,
         ld_act=None, want_acc=True, canary=True):
    """act: [N][K] int8 host.  Returns (y, acc) as numpy in [N][M] orientation."""
    torch = torch_mod()
    N, K = act.shape
    M = layer.M
    ld = ld_act or ((K + 15) // 16 * 16)
    a = torch.zeros((N, ld), dtype=torch.int8, device="cuda")
    a[:, :K] = torch.from_numpy(np.ascontiguousarray(act)).cuda()
    shape = (N, M) if out_layout == R.OUT_NM else (M, N)
    pad = 64 if canary else 0
    ybuf = torch.full((shape[0] * shape[1] + 2 * pad,), float("nan"), dtype=torch.float32, device="cuda")
    abuf = torch.full((shape[0] * shape[1] + 2 * pad,), -77777, dtype=torch.int32, device="cuda")
    y = ybuf[pad:pad + shape[0] * shape[1]].view(shape)
    acc = abuf[pad:pad + shape[0] * shape[1]].view(shape)
    if variant == WORKSPACE:
        R.rmsmp_gemm_workspace(layer, d_packed, _workspace(layer, d_packed), a, N, ld,
                               float(np.float32(act_step)), y, shape[1], out_layout, acc if want_acc else None)
    else:
        R.rmsmp_gemm_variant(layer, d_packed, a, N, ld, float(np.float32(act_step)), y, shape[1], out_layout,
                             acc if want_acc else None, variant)
    torch.cuda.synchronize()
    assert R.rmsmp_last_device_status(d_packed) == R.OK
    if canary:   # nothing written outside the output
        assert torch.isnan(ybuf[:pad]).all() and torch.isnan(ybuf[-pad:]).all()
        assert (abuf[:pad] == -77777).all() and (abuf[-pad:] == -77777).all()
    yh, ah = y.cpu().numpy(), acc.cpu().numpy()
    if out_layout == R.OUT_MN:
        yh, ah = yh.T, ah.T
    return yh, (ah if want_acc else None)


def conv(layer, d_packed, act: np.ndarray, stride, pad, act_step, variant=R.VARIANT_AUTO,
         out_layout=R.OUT_NM, want_acc=True):
    """act: [B][H][W][Cin] int8 host.  Returns (y, acc) as numpy [B*Ho*Wo][M]."""
    torch = torch_mod()
    B, H, W, Cin = act.shape
    M = layer.M
    Ho = (H + 2 * pad - layer.kh) // stride + 1
    Wo = (W + 2 * pad - layer.kw) // stride + 1
    N = B * Ho * Wo
    a = torch.from_numpy(np.ascontiguousarray(act)).cuda()
    shape = (N, M) if out_layout == R.OUT_NM else (M, N)
    cpad = 64
    ybuf = torch.full((N * M + 2 * cpad,), float("nan"), dtype=torch.float32, device="cuda")
    abuf = torch.full((N * M + 2 * cpad,), -77777, dtype=torch.int32, device="cuda")
    y = ybuf[cpad:cpad + N * M].view(shape)
    acc = abuf[cpad:cpad + N * M].view(shape)
    if variant == WORKSPACE:
        R.rmsmp_conv_implicit_workspace(layer, d_packed, _workspace(layer, d_packed), a, B, H, W, stride, pad,
                                        float(np.float32(act_step)), y, out_layout, acc if want_acc else None)
    else:
        R.rmsmp_conv_implicit_variant(layer, d_packed, a, B, H, W, stride, pad, float(np.float32(act_step)),
                                      y, out_layout, acc if want_acc else None, variant)
    torch.cuda.synchronize()
    assert R.rmsmp_last_device_status(d_packed) == R.OK
    assert torch.isnan(ybuf[:cpad]).all() and torch.isnan(ybuf[-cpad:]).all()
    assert (abuf[:cpad] == -77777).all() and (abuf[-cpad:] == -77777).all()
    yh, ah = y.cpu().numpy(), acc.cpu().numpy()
    if out_layout == R.OUT_MN:
        yh, ah = yh.T, ah.T
    return yh, (ah if want_acc else None)


def quantize_act(x: np.ndarray, alpha_a, kind):
    torch = torch_mod()
    d = torch.from_numpy(np.ascontiguousarray(x, np.float32)).cuda()
    codes = torch.empty(d.shape, dtype=torch.int8, device="cuda")
    step = R.rmsmp_quantize_act(d, d.numel(), alpha_a, kind, codes)
    torch.cuda.synchronize()
    return codes.cpu().numpy(), np.float32(step)
