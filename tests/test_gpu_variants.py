"""GPU parity of the operand variants and of the group size 320: FP8-E4M3 weights (the W8A8 FP - FP rows of
Table 2) through the block-scaled kernel, E5M2 as the target of the cast FP4 -> FP8 (Section 3, footnote; shifts
to 13), and groups of 320 input features (Appendix A: the paper's choice for a hidden size of 3200).
Codes, shifts and scales bit for bit against the oracle, outputs within 1e-3 of max |y|."""
import numpy as np
import pytest
import torch

import oracle
from paper_2307_09782_b200 import binding, synth
from tests.gpu_util import TOL_REL, check_packed, host, to_bf16, untile_codes, up
from tests.test_gpu_parity import _layer

pytestmark = pytest.mark.gpu
FP8, E5M2, MX, CAST = binding.WEIGHTS_MX_FP8, binding.WEIGHTS_CAST_E5M2, binding.WEIGHTS_MX, binding.WEIGHTS_CAST


def _wild_rows(W, group):
    """Rows whose groups differ by up to 2^-11 in magnitude: shifts beyond 5."""
    W = W.copy()
    W[1, :group] *= 2.0 ** -7
    W[2, group:2 * group] *= 2.0 ** -11
    W[3, :group] = 0.0
    return W


def _check_y(pw, x_bits, U, V, y_o, out_dtype=torch.float32, rows=None):
    M, K = x_bits.shape
    r = 0 if U is None else U.shape[1]
    ws = binding.make_workspace(binding.linear_workspace_bytes(M, pw.N, K, r))
    y = binding.w4a8_linear(pw, x=to_bf16(x_bits), U=up(U), V=up(V), out_dtype=out_dtype, workspace=ws)
    assert binding.device_status(ws) == (0, 0)
    yh = host(y.float()).astype(np.float64)
    if rows is not None:
        yh = yh[rows]
    ymax = np.abs(y_o).max()
    if out_dtype == torch.float32:
        assert np.abs(yh - y_o).max() <= TOL_REL * ymax
    else:
        ulp = 2.0 ** (np.floor(np.log2(np.maximum(np.abs(y_o), 1e-30))) - 7)
        assert np.all(np.abs(yh - y_o) <= ulp + TOL_REL * ymax)
    return yh


# ---- FP8 weights ------------------------------------------------------------------------------------------
@pytest.mark.parametrize("mode", ["M1", "M2"])
@pytest.mark.parametrize("group", [64, 128, 256, 320])
def test_pack_fp8_weights_bit_exact(mode, group):
    K = 1280
    W = _wild_rows(synth.make_w(21, 200, K), group)
    c_o, sh_o, sc_o = oracle.pack_weight(W, group, mode, "e4m3", 127)
    pw = binding.pack_weight_fp4(up(W), group, mode, FP8)
    codes, sh32 = untile_codes(host(pw.codes), 200, K, FP8)
    assert np.array_equal(codes, c_o)
    assert np.array_equal(host(pw.shift), sh_o) and np.array_equal(sh32, np.repeat(sh_o, group // 32, axis=1))
    assert np.array_equal(host(pw.scale).view(np.uint32), sc_o.view(np.uint32))
    assert sh_o.max() > 5      # the case really goes beyond the FP4 clamp


@pytest.mark.parametrize("M,N,K,r,mode", [(1, 384, 1024, 8, "M2"), (16, 256, 8192, 8, "M1"), (40, 200, 2048, 0, "M2"),
                                          (130, 384, 512, 8, "M2"), (300, 1000, 1024, 16, "M1"),
                                          (1120, 128 * 120, 512, 8, "M2")])
def test_linear_fp8_weights(M, N, K, r, mode):
    x_bits, W, U, V = _layer(500 + M, M, N, K, r)
    q_o, sx_o, t_o = oracle.quantize_act_fp8(x_bits, V)
    c_o, sh_o, sc_o = oracle.pack_weight(W, 128, mode, "e4m3", 127)
    rows = None if M <= 300 else [0, 191, 192, 223, 224, 447, 448, 700, M - 1]
    y_o = oracle.linear_general(q_o, sx_o, c_o, sh_o, sc_o, 128, mode, "e4m3", U, t_o, rows=rows)
    pw = binding.pack_weight_fp4(up(W), 128, mode, FP8)
    _check_y(pw, x_bits, U, V, y_o, rows=rows)
    if M == 40:
        _check_y(pw, x_bits, U, V, y_o, out_dtype=torch.bfloat16)


def test_linear_fp8_weights_exact_on_power_of_two_data():
    M, N, K = 16, 256, 512
    rng = np.random.default_rng(5)
    x = rng.choice([0.0, 0.25, 0.5, 1.0, -1.0, 2.0], (M, K)).astype(np.float32)
    x[:, 0] = 7.0
    W = rng.choice([0.0, 0.5, -1.0, 1.75, 3.5, -4.0], (N, K)).astype(np.float32)
    W[:, ::128] = 7.0
    W[3, 128:256] *= 2.0 ** -9
    bits = synth.f32_to_bf16_bits(x)
    q_o, sx_o, _ = oracle.quantize_act_fp8(bits)
    for mode in ("M1", "M2"):
        c_o, sh_o, sc_o = oracle.pack_weight(W, 128, mode, "e4m3", 127)
        y_o = oracle.linear_general(q_o, sx_o, c_o, sh_o, sc_o, 128, mode, "e4m3")
        yh = _check_y(binding.pack_weight_fp4(up(W), 128, mode, FP8), bits, None, None, y_o)
        assert np.array_equal(yh, y_o), mode


# ---- E5M2 as the cast target ------------------------------------------------------------------------------
@pytest.mark.parametrize("mode", ["M1", "M2"])
def test_cast_to_e5m2_keeps_shifts_to_13(mode):
    M, N, K = 24, 300, 1024
    x_bits, W, U, V = _layer(601, M, N, K, 8)
    W = _wild_rows(W, 128)
    c_o, sh_o, sc_o = oracle.pack_weight(W, 128, mode, "e2m1", 13)
    assert 5 < sh_o.max() <= 13
    pw = binding.pack_weight_fp4(up(W), 128, mode, E5M2)
    codes, sh32 = untile_codes(host(pw.codes), N, K, CAST)        # the same tiling as the E4M3 cast layout
    c_plain = (c_o[:, 0::2] | (c_o[:, 1::2] << 4)).astype(np.uint8)
    assert np.array_equal(codes, c_plain)
    assert np.array_equal(host(pw.shift), sh_o) and np.array_equal(sh32, np.repeat(sh_o, 4, axis=1))
    assert np.array_equal(host(pw.scale).view(np.uint32), sc_o.view(np.uint32))
    q_o, sx_o, t_o = oracle.quantize_act_fp8(x_bits, V)
    y_o = oracle.linear_general(q_o, sx_o, c_o, sh_o, sc_o, 128, mode, "e2m1", U, t_o)
    _check_y(pw, x_bits, U, V, y_o)
    # with the E4M3 target the same weight is packed with the shifts clamped at 5: other codes in the wild rows
    pw5 = binding.pack_weight_fp4(up(W), 128, mode, CAST)
    assert host(pw5.shift).max() == 5


@pytest.mark.parametrize("M", [1, 64, 300])
def test_cast_to_e5m2_equals_cast_to_e4m3_within_shift_5(M):
    # both casts are exact there: same products, same accumulation order, the same bits in y
    x_bits, _, U, V = _layer(602 + M, M, 384, 2048, 8)
    W = synth.make_w(602, 384, 2048)     # plain Gaussian rows: shifts 0 .. 2
    x, Ud, Vd = to_bf16(x_bits), up(U), up(V)
    q, sx, t = binding.quantize_act_fp8(x, Vd)
    ys = []
    for layout in (CAST, E5M2):
        pw = binding.pack_weight_fp4(up(W), 128, "M2", layout)
        assert host(pw.shift).max() <= 5
        ys.append(host(binding.w4a8_linear(pw, q=q, sx=sx, t=t, U=Ud)))
    assert np.abs(ys[0] - ys[1]).max() <= 1e-6 * np.abs(ys[0]).max()


# ---- groups of 320 ----------------------------------------------------------------------------------------
@pytest.mark.parametrize("layout", [CAST, MX])
@pytest.mark.parametrize("mode", ["M1", "M2"])
def test_group_320(layout, mode):
    # a 3200 -> 3200 layer (the hidden size the paper uses groups of 320 for), decode and prefill token counts
    N = K = 3200
    x_bits, W, U, V = _layer(700, 300, N, K, 8)
    c_o, sh_o, sc_o = oracle.pack_weight_fp4(W, 320, mode)
    pw = binding.pack_weight_fp4(up(W), 320, mode, layout)
    check_packed(pw, c_o, sh_o, sc_o, 320)
    q_o, sx_o, t_o = oracle.quantize_act_fp8(x_bits, V)
    for M in (8, 300):
        rows = list(range(M)) if M == 8 else [0, 127, 128, 191, 192, 255, 256, 299]
        y_o = oracle.w4a8_linear(q_o[:M], sx_o[:M], c_o, sh_o, sc_o, 320, mode, U, t_o[:M], rows=rows)
        _check_y(pw, x_bits[:M], U, V, y_o, rows=rows)


def test_group_320_is_refused_for_unconstrained_scales():
    W = up(synth.make_w(1, 128, 640))
    with pytest.raises(binding.ZqError) as e:
        binding.pack_weight_fp4(W, 320, "none", CAST)
    assert e.value.status == -2
