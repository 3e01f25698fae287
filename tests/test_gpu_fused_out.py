"""GPU parity of the fusion on the output side of the layer (Section 3 / Appendix A: the next layer quantizes this
layer's output token-wise): `zq_w4a8_linear_fused_out` applies the ReLU of the MLP and collects every token's
max |y| in its epilogue, and `zq_quantize_act_fp8_scaled` then quantizes y in one pass.

What is checked: y against the oracle (1e-3 of max |y|, ReLU applied to the oracle's y); the collected maxima
against the maxima of the y the GPU stored, exactly (a maximum has no rounding); the one-pass quantizer fed with
them against the oracle's quantizer on that same y, bit for bit, and against the two-pass kernel."""
import numpy as np
import pytest
import torch

import oracle
from paper_2307_09782_b200 import binding, synth
from tests.gpu_util import TOL_REL, host, to_bf16, up
from tests.test_gpu_parity import _layer

pytestmark = pytest.mark.gpu


def _bits(t: torch.Tensor) -> np.ndarray:
    return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


@pytest.mark.parametrize("M,N,K,r,mode,layout,out_dtype,relu,raw_x", [
    (8, 640, 2048, 8, "M2", "mx", torch.bfloat16, True, True),        # decode: quantizer inside the kernel, shared tiles
    (8, 640, 2048, 8, "M2", "mx", torch.float32, False, False),       # FP32 y, shared tiles: partial sums, not adds
    (40, 128 * 30, 1024, 8, "M1", "mx", torch.bfloat16, True, False),  # 64-token tiles dealt out as unit ranges
    (100, 128 * 20, 1024, 8, "M2", "mx", torch.bfloat16, True, False),  # a pair plan with shared positions: single CTAs
    (500, 768, 2048, 0, "M2", "mx", torch.bfloat16, True, False),
    (1120, 128 * 120, 256, 8, "M2", "mx", torch.bfloat16, True, False),  # CTA pairs, whole positions
    (1000, 128 * 120 - 37, 384, 16, "M1", "mx", torch.float32, True, False),  # ragged channels, generic rank
    (1120, 128 * 119, 512, 8, "M2", "mx", torch.bfloat16, False, False),  # odd channel-tile count: persistent single CTAs
    (300, 384, 512, 8, "none", "mx", torch.bfloat16, True, False),    # unconstrained scales in the block-scaled kernel
    (100, 640, 1024, 8, "M2", "cast", torch.bfloat16, True, False),   # the kernel that casts: split K
    (300, 384, 512, 8, "none", "cast", torch.bfloat16, True, False),
    (700, 1000, 1024, 8, "M2", "mx_fp8", torch.bfloat16, True, False),
])
def test_fused_output_and_one_pass_quantizer(M, N, K, r, mode, layout, out_dtype, relu, raw_x):
    x_bits, W, U, V = _layer(700 + M, M, N, K, r)
    q_o, sx_o, t_o = oracle.quantize_act_fp8(x_bits, V)
    if layout == "mx_fp8":
        c_o, sh_o, sc_o = oracle.pack_weight(W, 128, mode, "e4m3", 127)
        y_o = oracle.linear_general(q_o, sx_o, c_o, sh_o, sc_o, 128, mode, "e4m3", U, t_o)
    else:
        c_o, sh_o, sc_o = oracle.pack_weight_fp4(W, 128, mode)
        y_o = oracle.w4a8_linear(q_o, sx_o, c_o, sh_o, sc_o, 128, mode, U, t_o)
    if relu:
        y_o = np.maximum(y_o, 0.0)
    pw = binding.pack_weight_fp4(up(W), 128, mode, binding.LAYOUTS[layout])
    ws = binding.make_workspace(binding.linear_workspace_bytes(M, N, K, r))
    amax = torch.full((M,), float("nan"), dtype=torch.float32, device="cuda")
    Ud, Vd = up(U), up(V)
    for _ in range(2):   # the second call must find flags and scratch as the first did
        if raw_x:
            y = binding.w4a8_linear(pw, x=to_bf16(x_bits), U=Ud, V=Vd, out_dtype=out_dtype, workspace=ws, relu=relu,
                                    y_absmax=amax)
        else:
            q, sx, t = binding.quantize_act_fp8(to_bf16(x_bits), Vd)
            y = binding.w4a8_linear(pw, q=q, sx=sx, t=t, U=Ud, out_dtype=out_dtype, workspace=ws, relu=relu,
                                    y_absmax=amax)
        assert binding.device_status(ws) == (0, 0)
        yh = host(y.float()).astype(np.float64)
        tol = TOL_REL * np.abs(y_o).max()
        if out_dtype == torch.bfloat16:
            tol = tol + 2.0 ** (np.floor(np.log2(np.maximum(np.abs(y_o), 1e-30))) - 7)
        assert np.all(np.abs(yh - y_o) <= tol)
        if relu:
            assert (yh >= 0).all()
        # the maxima are those of the stored values, exactly
        assert torch.equal(amax, y.float().abs().amax(dim=1))
    if out_dtype != torch.bfloat16:
        return
    # the next layer's quantizer in one pass, on the y the GPU produced
    _, V2 = synth.make_lorc(900 + M, 8, N, 8) if N % 16 == 0 else (None, None)
    if N % 16:
        return
    y_bits = _bits(y)
    q2_o, sx2_o, t2_o = oracle.quantize_act_fp8(y_bits, V2)
    q2, sx2, t2 = binding.quantize_act_fp8(y, up(V2), absmax=amax)
    assert np.array_equal(host(q2), q2_o)
    assert np.array_equal(host(sx2).view(np.uint32), sx2_o.view(np.uint32))
    assert np.abs(host(t2) - t2_o).max() <= 1e-4 * max(np.abs(t2_o).max(), 1e-30)
    q3, sx3, _ = binding.quantize_act_fp8(y, up(V2))
    assert torch.equal(q2, q3) and torch.equal(sx2, sx3)


@pytest.mark.parametrize("M,K,r", [(1, 16, 0), (5, 4096, 8), (100, 7168, 8), (517, 28672, 8), (300, 2048, 16),
                                   (2000, 1024, 0), (9, 28704, 8)])
def test_one_pass_quantizer_alone(M, K, r):
    """Every token count and rank through `zq_quantize_act_fp8_scaled`, the maxima taken from torch."""
    x_bits = synth.make_x(800 + M, M, K, max(1, K // 100), 20.0)
    x_bits[min(3, M - 1)] = 0
    V = synth.make_lorc(800 + M, 8, K, r)[1] if r else None
    x = to_bf16(x_bits)
    amax = x.float().abs().amax(dim=1).contiguous()
    q_o, sx_o, t_o = oracle.quantize_act_fp8(x_bits, V)
    q, sx, t = binding.quantize_act_fp8(x, up(V), absmax=amax)
    assert np.array_equal(host(q), q_o)
    assert np.array_equal(host(sx).view(np.uint32), sx_o.view(np.uint32))
    if r:
        assert np.abs(host(t) - t_o).max() <= 1e-4 * np.abs(t_o).max()
