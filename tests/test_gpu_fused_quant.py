"""GPU parity of the decode path in which the block-scaled GEMM kernel quantizes its activations itself
(Section 3: token-wise FP8 activation quantization; LoRC down-projection t = V x with the raw x), taken by
zq_w4a8_linear for raw bf16 activations of at most 16 tokens and weights in a block-scaled layout (the cases
with more tokens check the hand-over to the two-kernel path right above that limit).

The kernel leaves its FP8 codes in the workspace, out of the caller's sight; the stand-alone quantizer's
bit-exact tests cover the shared cast arithmetic, and here y is compared with the oracle (1e-3 of max |y|)
and with the two-kernel path (quantizer kernel, then GEMM), which computes the same products from the same
codes and so differs only in summation order.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2307_09782_b200 import binding, synth
from tests.gpu_util import TOL_REL, host, to_bf16, up
from tests.test_gpu_parity import _layer

pytestmark = pytest.mark.gpu
MX = binding.WEIGHTS_MX


def _oracle(x_bits, W, U, V, group, mode):
    q_o, sx_o, t_o = oracle.quantize_act_fp8(x_bits, V)
    c_o, sh_o, sc_o = oracle.pack_weight_fp4(W, group, mode)
    return oracle.w4a8_linear(q_o, sx_o, c_o, sh_o, sc_o, group, mode, U, t_o)


def _check(x_bits, W, U, V, group=128, mode="M2", out_dtype=torch.float32, calls=1):
    M, K = x_bits.shape
    N = W.shape[0]
    r = 0 if U is None else U.shape[1]
    y_o = _oracle(x_bits, W, U, V, group, mode)
    pw = binding.pack_weight_fp4(up(W), group, mode, MX)
    ws = binding.make_workspace(binding.linear_workspace_bytes(M, N, K, r))
    x, Ud, Vd = to_bf16(x_bits), up(U), up(V)
    launches0 = binding.launch_count()
    for _ in range(calls):  # the scratch the CTAs meet in must be left clean for the next call
        y = binding.w4a8_linear(pw, x=x, U=Ud, V=Vd, out_dtype=out_dtype, workspace=ws)
        assert binding.device_status(ws) == (0, 0)
        yh = host(y.float()).astype(np.float64)
        ymax = np.abs(y_o).max()
        if out_dtype == torch.float32:
            assert np.abs(yh - y_o).max() <= TOL_REL * ymax
        else:
            ulp = 2.0 ** (np.floor(np.log2(np.maximum(np.abs(y_o), 1e-30))) - 7)
            assert np.all(np.abs(yh - y_o) <= ulp + TOL_REL * ymax)
    # up to 16 tokens the layer is one launch (quantizer and GEMM are one kernel), beyond that two
    assert binding.launch_count() - launches0 == (calls if M <= 16 else 2 * calls)
    # the two-kernel path on the same workspace: same codes, same products
    q, sx, t = binding.quantize_act_fp8(x, Vd)
    y2 = binding.w4a8_linear(pw, q=q, sx=sx, t=t, U=Ud, out_dtype=out_dtype, workspace=ws)
    assert binding.device_status(ws) == (0, 0)
    tol2 = 1e-5 if out_dtype == torch.float32 else 2.0 ** -7
    assert np.abs(host(y2.float()) - host(y.float())).max() <= tol2 * np.abs(host(y2.float())).max()
    return yh, y_o


@pytest.mark.parametrize("M", [1, 2, 7, 8, 15, 16, 17, 32])
def test_every_token_count(M):
    x_bits, W, U, V = _layer(300 + M, M, 384, 1024, 8)
    _check(x_bits, W, U, V, calls=2)


@pytest.mark.parametrize("M,N,K,r", [
    (8, 128 * 40, 1024, 8),    # more K blocks and tiles than one wave's share: several segments per CTA
    (16, 256, 8192, 8),        # few tiles, long K: tiles shared by many CTAs (store / flag / add)
    (5, 200, 256, 0),          # ragged N, no LoRC
    (16, 129, 4096, 16),       # a full 16-token tile, rank 16
    (3, 1, 384, 8),            # a single output channel
    (9, 128 * 230, 256, 8),    # two K blocks of x only: most CTAs have no share of the quantizer's work
    (12, 640, 128, 8),         # a single K block: the split path (fewer than 8 units)
    (13, 1000, 2048, 64),      # the largest rank
    (1, 128 * 224, 896, 8),    # the decode shape of a wide layer
])
def test_plan_branches(M, N, K, r):
    x_bits, W, U, V = _layer(400 + M + r, M, N, K, r)
    _check(x_bits, W, U, V, calls=2)


@pytest.mark.parametrize("mode,group", [("M1", 64), ("M1", 128), ("M2", 256)])
def test_modes_and_groups(mode, group):
    x_bits, W, U, V = _layer(77, 11, 512, 2048, 8)
    _check(x_bits, W, U, V, group=group, mode=mode)


def test_bf16_output():
    x_bits, W, U, V = _layer(78, 16, 256, 4096, 8)
    _check(x_bits, W, U, V, out_dtype=torch.bfloat16, calls=2)
    x_bits, W, U, V = _layer(79, 6, 128 * 20, 512, 8)
    _check(x_bits, W, U, V, out_dtype=torch.bfloat16)


def test_fp8_weights():
    M, N, K, r = 8, 640, 2048, 8
    x_bits, W, U, V = _layer(83, M, N, K, r)
    q_o, sx_o, t_o = oracle.quantize_act_fp8(x_bits, V)
    c_o, sh_o, sc_o = oracle.pack_weight(W, 128, "M2", "e4m3", 127)
    y_o = oracle.linear_general(q_o, sx_o, c_o, sh_o, sc_o, 128, "M2", "e4m3", U, t_o)
    pw = binding.pack_weight_fp4(up(W), 128, "M2", binding.WEIGHTS_MX_FP8)
    ws = binding.make_workspace(binding.linear_workspace_bytes(M, N, K, r))
    l0 = binding.launch_count()
    y = binding.w4a8_linear(pw, x=to_bf16(x_bits), U=up(U), V=up(V), workspace=ws)
    assert binding.device_status(ws) == (0, 0) and binding.launch_count() - l0 == 1
    assert np.abs(host(y).astype(np.float64) - y_o).max() <= TOL_REL * np.abs(y_o).max()


def test_zero_tokens_outliers_and_tiny_rows():
    # an all-zero token (scale 1, codes 0), a token whose absmax sits in the last K block, a tiny-magnitude token
    M, N, K, r = 8, 384, 1024, 8
    x_bits, W, U, V = _layer(80, M, N, K, r)
    x = synth.bf16_bits_to_f32(x_bits)
    x[2] = 0.0
    x[3] *= 1e-3
    x[3, K - 1] = 300.0
    x[5] *= 2.0 ** -100
    _check(synth.f32_to_bf16_bits(x), W, U, V)


def test_exact_on_power_of_two_data():
    M, N, K = 16, 256, 512
    rng = np.random.default_rng(5)
    x = rng.choice([0.0, 0.25, 0.5, 1.0, -1.0, 2.0], (M, K)).astype(np.float32)
    x[:, 0] = 7.0
    W = rng.choice([0.0, 0.5, -1.0, 1.5, 3.0, -4.0], (N, K)).astype(np.float32)
    W[:, ::128] = 6.0
    W[3, 128:256] *= 0.125
    yh, y_o = _check(synth.f32_to_bf16_bits(x), W, None, None, mode="M1")
    assert np.array_equal(yh, y_o)


def test_strided_activations_and_output():
    M, N, K, r = 8, 640, 2048, 8
    x_bits, W, U, V = _layer(81, M, N, K, r)
    y_o = _oracle(x_bits, W, U, V, 128, "M2")
    pw = binding.pack_weight_fp4(up(W), 128, "M2", MX)
    xbuf = torch.full((M, K + 64), float("nan"), dtype=torch.bfloat16, device="cuda")
    xbuf[:, :K] = to_bf16(x_bits)
    ybuf = torch.full((M, N + 24), float("nan"), dtype=torch.float32, device="cuda")
    ws = binding.make_workspace(binding.linear_workspace_bytes(M, N, K, r))
    binding.w4a8_linear(pw, x=xbuf[:, :K], U=up(U), V=up(V), y=ybuf[:, :N], workspace=ws)
    assert binding.device_status(ws) == (0, 0)
    assert torch.isnan(ybuf[:, N:]).all()
    assert np.abs(host(ybuf[:, :N]).astype(np.float64) - y_o).max() <= TOL_REL * np.abs(y_o).max()


def test_interleaved_with_larger_calls_on_one_workspace():
    # decode and prefill calls alternate on one workspace: each must find the scratch as it needs it
    N, K, r = 512, 2048, 8
    x_bits, W, U, V = _layer(82, 300, N, K, r)
    pw = binding.pack_weight_fp4(up(W), 128, "M1", MX)
    ws = binding.make_workspace(binding.linear_workspace_bytes(300, N, K, r))
    x, Ud, Vd = to_bf16(x_bits), up(U), up(V)
    y_o = _oracle(x_bits, W, U, V, 128, "M1")
    for M in (4, 300, 16, 17, 300, 1):
        y = binding.w4a8_linear(pw, x=x[:M], U=Ud, V=Vd, workspace=ws)
        assert binding.device_status(ws) == (0, 0)
        assert np.abs(host(y).astype(np.float64) - y_o[:M]).max() <= TOL_REL * np.abs(y_o[:M]).max(), M


@pytest.mark.parametrize("M,N,K,r", [(8, 128 * 40, 1024, 8), (1, 128 * 224, 896, 8), (16, 256, 8192, 8), (40, 128 * 30, 1024, 8),
                                     (500, 640, 2048, 8)])
def test_plain_launches_on_an_exclusive_device(M, N, K, r):
    """After zq_set_exclusive_device(1) the launches whose CTAs hand tiles over to one another are plain ones
    instead of cooperative ones: same results, and the default comes back afterwards."""
    x_bits, W, U, V = _layer(600 + M, M, N, K, r)
    was = binding.set_exclusive_device(True)
    try:
        assert binding.set_exclusive_device(True) is True
        _check(x_bits, W, U, V, calls=3)
    finally:
        binding.set_exclusive_device(was)
    assert binding.set_exclusive_device(was) == was
