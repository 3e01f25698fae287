"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle on the same seeded inputs.

Bit-exact for FP8 activation codes, FP4 weight codes, shifts and scales; outputs within
1e-3 * max|y| (FP32 accumulation order differs).
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2307_09782_b200 import binding, synth
from gpu_util import TOL_REL, check_linear, check_packed, dev, host, to_bf16, up

pytestmark = pytest.mark.gpu


# ---------------------------------------------------------------------------------------------- quantizer
@pytest.mark.parametrize("M,K", [(1, 16), (3, 48), (16, 768), (17, 2048), (5, 11008), (4, 28672), (2, 40960)])
def test_act_quant_bit_exact(M, K):
    x_bits = synth.make_x(100 + M, M, K, max(1, K // 100), 20.0)
    _, V = synth.make_lorc(100 + M, 8, K, 8)
    q_o, sx_o, t_o = oracle.quantize_act_fp8(x_bits, V)
    q, sx, t = binding.quantize_act_fp8(to_bf16(x_bits), up(V))
    assert np.array_equal(host(q), q_o)
    assert np.array_equal(host(sx).view(np.uint32), sx_o.view(np.uint32))
    assert np.abs(host(t) - t_o).max() <= 1e-4 * np.abs(t_o).max()


@pytest.mark.parametrize("M,K,lorc", [(1187, 768, True), (1184, 2048, False), (2500, 256, True), (385, 4096, True),
                                      (384, 48, True), (300, 16384, True), (1030, 7168, True), (520, 28672, True),
                                      (400, 3584, False), (390, 14336, True), (386, 28704, True),
                                      (388, 33024, True), (391, 4112, True), (8192, 1024, True)])
def test_act_quant_many_rows_kernel(M, K, lorc):
    """Token counts large enough for the eight-rows kernels (one pass with the rows in shared memory, split over a
    cluster of 1 / 2 / 4 / 8 CTAs by row length; two passes beyond 32768 columns), with a ragged last row group and
    ragged last slices."""
    x_bits = synth.make_x(300 + M, M, K, max(1, K // 100), 20.0)
    x_bits[5] = 0                                 # an all-zero token
    V = synth.make_lorc(300 + M, 8, K, 8)[1] if lorc else None
    q_o, sx_o, t_o = oracle.quantize_act_fp8(x_bits, V)
    q, sx, t = binding.quantize_act_fp8(to_bf16(x_bits), up(V))
    assert np.array_equal(host(q), q_o)
    assert np.array_equal(host(sx).view(np.uint32), sx_o.view(np.uint32))
    if lorc:
        assert np.abs(host(t) - t_o).max() <= 1e-4 * np.abs(t_o).max()


@pytest.mark.parametrize("M,K,lorc", [(64, 1024, True), (100, 7168, True), (128, 28672, True), (383, 4096, True),
                                      (200, 28704, True), (65, 2048, False), (130, 16, True), (72, 40960, True),
                                      (63, 7168, True), (77, 3600, True), (32, 7168, True), (31, 7168, True),
                                      (40, 28672, True)])
def test_act_quant_a_few_hundred_rows(M, K, lorc):
    """Token counts between the cluster-per-row kernel and the eight-row CTAs: eight rows per cluster with the rows
    in shared memory (and, outside its limits on K, the kernels around it)."""
    x_bits = synth.make_x(500 + M, M, K, max(1, K // 100), 20.0)
    x_bits[min(5, M - 1)] = 0                      # an all-zero token
    V = synth.make_lorc(500 + M, 8, K, 8)[1] if lorc else None
    q_o, sx_o, t_o = oracle.quantize_act_fp8(x_bits, V)
    q, sx, t = binding.quantize_act_fp8(to_bf16(x_bits), up(V))
    assert np.array_equal(host(q), q_o)
    assert np.array_equal(host(sx).view(np.uint32), sx_o.view(np.uint32))
    if lorc:
        assert np.abs(host(t) - t_o).max() <= 1e-4 * np.abs(t_o).max()


def test_act_quant_many_rows_strided_input():
    _strided_quant_case(517, 7168)
    _strided_quant_case(150, 7168)


def _strided_quant_case(M, K):
    x_bits = synth.make_x(77, M, K, 70, 20.0)
    V = synth.make_lorc(77, 8, K, 8)[1]
    wide = torch.full((M, K + 264), 1e30, dtype=torch.bfloat16, device=dev())
    wide[:, :K] = to_bf16(x_bits)
    q_o, sx_o, t_o = oracle.quantize_act_fp8(x_bits, V)
    q, sx, t = binding.quantize_act_fp8(wide[:, :K], up(V))
    assert np.array_equal(host(q), q_o) and np.array_equal(host(sx).view(np.uint32), sx_o.view(np.uint32))
    assert np.abs(host(t) - t_o).max() <= 1e-4 * np.abs(t_o).max()


def test_act_quant_edge_rows_and_strided_input():
    K = 256
    x = np.zeros((6, K), dtype=np.float32)
    x[1] = np.linspace(-3, 3, K)
    x[2, 7] = -1e-30                      # tiny absmax
    x[3] = 3.0e38                         # near the top of bf16
    x[4] = np.random.default_rng(0).standard_normal(K) * 1e-3
    x[4, 9] = 77.0                        # one outlier: the rest lands in the subnormal range of E4M3
    x[5] = -0.0
    bits = synth.f32_to_bf16_bits(x)
    q_o, sx_o, _ = oracle.quantize_act_fp8(bits)
    q, sx, _ = binding.quantize_act_fp8(to_bf16(bits))
    assert np.array_equal(host(q), q_o) and np.array_equal(host(sx).view(np.uint32), sx_o.view(np.uint32))
    # rank-16 LoRC and a padded leading dimension
    wide = torch.zeros((6, K + 64), dtype=torch.bfloat16, device=dev())
    wide[:, :K] = to_bf16(bits)
    _, V = synth.make_lorc(3, 8, K, 16)
    q2, sx2, t2 = binding.quantize_act_fp8(wide[:, :K], up(V))
    _, _, t_o = oracle.quantize_act_fp8(bits, V)
    assert np.array_equal(host(q2), q_o) and np.array_equal(host(sx2), sx_o)
    assert np.abs(host(t2) - t_o).max() <= 1e-4 * np.abs(t_o).max()
    # empty input is a no-op
    q3, sx3, _ = binding.quantize_act_fp8(torch.empty((0, K), dtype=torch.bfloat16, device=dev()))
    assert q3.shape == (0, K) and sx3.shape == (0,)


# ---------------------------------------------------------------------------------------------- packer
def _special_weights(N, K, seed):
    W = synth.make_w(seed, N, K, 0.02)
    assert N >= 7
    W[0, :128] = 0.0                                   # all-zero group
    W[1, 128:256] *= np.float32(2.0 ** -9)             # needs a shift beyond the clamp
    W[2, :] = 0.0                                      # all-zero row
    W[3, 0:64] = np.float32(6.0 * 2.0 ** -7) * np.sign(W[3, 0:64] + 1e-9)  # scale exactly a power of two
    W[4, 5] = -0.0
    W[5, 256:384] *= 0.3
    if N > 6:
        W[6, :] *= np.float32(1e-36)                   # scales in the subnormal range
    return W


@pytest.mark.parametrize("mode", ["none", "M1", "M2"])
@pytest.mark.parametrize("group", [64, 128, 256])
def test_pack_weight_bit_exact(mode, group):
    W = _special_weights(9, 1024, 31)
    c_o, sh_o, sc_o = oracle.pack_weight_fp4(W, group, mode)
    check_packed(binding.pack_weight_fp4(up(W), group, mode), c_o, sh_o, sc_o, group)


@pytest.mark.parametrize("mode", ["none", "M1", "M2"])
def test_pack_weight_layer_shape(mode):
    W = synth.make_w(2, 1000, 4096, 0.02)
    c_o, sh_o, sc_o = oracle.pack_weight_fp4(W, 128, mode)
    check_packed(binding.pack_weight_fp4(up(W), 128, mode), c_o, sh_o, sc_o, 128)


# ---------------------------------------------------------------------------------------------- linear
def _layer(seed, M, N, K, r, outliers=0.01):
    x_bits = synth.make_x(seed, M, K, max(1, int(outliers * K)), 20.0)
    W = synth.make_w(seed, N, K, 0.02)
    W[min(3, N - 1), :128] *= 0.1           # make the shifts non-trivial
    W[min(5, N - 1), K - 128:] *= 0.02
    U = V = None
    if r:
        U, V = synth.make_lorc(seed, N, K, r)
    return x_bits, W, U, V


@pytest.mark.parametrize("mode", ["M1", "M2", "none"])
@pytest.mark.parametrize("M", [1, 16, 17, 100, 130, 300])
def test_linear_small(mode, M):
    x_bits, W, U, V = _layer(40 + M, M, 384, 512, 8)
    check_linear(x_bits, W, U, V, 128, mode)


@pytest.mark.parametrize("mode", ["M2", "none"])
@pytest.mark.parametrize("M,N,K,r", [(3, 200, 256, 0), (33, 128, 128, 16), (64, 129, 1024, 8), (7, 1, 384, 8)])
def test_linear_ragged_tiles(mode, M, N, K, r):
    x_bits, W, U, V = _layer(60 + M, M, N, K, r)
    check_linear(x_bits, W, U, V, 128, mode)


@pytest.mark.parametrize("mode,group", [("M1", 64), ("M2", 256), ("none", 256), ("none", 64)])
def test_linear_other_group_sizes(mode, group):
    x_bits, W, U, V = _layer(71, 20, 256, 1024, 8)
    check_linear(x_bits, W, U, V, group, mode)


@pytest.mark.parametrize("mode", ["M1", "none"])
def test_linear_split_k_long_rows(mode):
    # few output tiles and a long K: several CTAs share an output tile through the workspace
    x_bits, W, U, V = _layer(81, 16, 256, 8192, 8)
    check_linear(x_bits, W, U, V, 128, mode)


def test_linear_bf16_output_and_fused_quantizer():
    x_bits, W, U, V = _layer(91, 48, 512, 1024, 8)
    check_linear(x_bits, W, U, V, 128, "M2", out_dtype=torch.bfloat16)
    check_linear(x_bits, W, U, V, 128, "M2", fused_quant=True)
    check_linear(x_bits, W, None, None, 128, "M1", fused_quant=True)


def test_linear_exact_on_power_of_two_data_and_deterministic():
    M, N, K = 16, 256, 512
    rng = np.random.default_rng(5)
    x = rng.choice([0.0, 0.25, 0.5, 1.0, -1.0, 2.0], (M, K)).astype(np.float32)
    x[:, 0] = 7.0
    W = rng.choice([0.0, 0.5, -1.0, 1.5, 3.0, -4.0], (N, K)).astype(np.float32)
    W[:, ::128] = 6.0
    bits = synth.f32_to_bf16_bits(x)
    for mode in ("none", "M1", "M2"):
        y, y_o = check_linear(bits, W, None, None, 128, mode)
        assert np.array_equal(y, y_o), mode
        y2, _ = check_linear(bits, W, None, None, 128, mode)
        assert np.array_equal(y, y2)


def test_workspace_reuse_across_calls_and_token_counts():
    N, K, r = 384, 2048, 8
    ws = binding.make_workspace(binding.linear_workspace_bytes(256, N, K, r))
    W = synth.make_w(7, N, K)
    U, V = synth.make_lorc(7, N, K, r)
    c_o, sh_o, sc_o = oracle.pack_weight_fp4(W, 128, "M2")
    pw = binding.pack_weight_fp4(up(W), 128, "M2")
    for M in (256, 16, 1, 100, 16):
        x_bits = synth.make_x(7 + M, M, K, 20)
        q_o, sx_o, t_o = oracle.quantize_act_fp8(x_bits, V)
        y_o = oracle.w4a8_linear(q_o, sx_o, c_o, sh_o, sc_o, 128, "M2", U, t_o)
        y = binding.w4a8_linear(pw, x=to_bf16(x_bits), U=up(U), V=up(V), workspace=ws)
        assert binding.device_status(ws) == (0, 0)
        assert np.abs(host(y) - y_o).max() <= TOL_REL * np.abs(y_o).max()


def test_host_buffer_entry_point():
    M, N, K, r = 24, 256, 512, 8
    x_bits, W, U, V = _layer(95, M, N, K, r)
    pw = binding.pack_weight_fp4(up(W), 128, "M1")
    ws = binding.make_workspace(binding.linear_host_workspace_bytes(M, N, K, r))
    xh = torch.from_numpy(x_bits.view(np.int16)).view(torch.bfloat16).pin_memory()
    yh = torch.empty((M, N), dtype=torch.float32).pin_memory()
    binding.w4a8_linear_host(xh, yh, pw, U=up(U), V=up(V), workspace=ws)
    q_o, sx_o, t_o = oracle.quantize_act_fp8(x_bits, V)
    c_o, sh_o, sc_o = oracle.pack_weight_fp4(W, 128, "M1")
    y_o = oracle.w4a8_linear(q_o, sx_o, c_o, sh_o, sc_o, 128, "M1", U, t_o)
    assert np.abs(yh.numpy() - y_o).max() <= TOL_REL * np.abs(y_o).max()


def test_a_bounded_wait_that_runs_out_is_reported_and_the_context_stays_usable():
    # the failure path of every in-kernel wait: record ZQ_ERR_DEVICE_TIMEOUT, return, nothing hangs or faults
    x_bits, W, U, V = _layer(7, 16, 256, 512, 8)
    ws = binding.make_workspace(binding.linear_workspace_bytes(16, 256, 512, 8))
    binding.selftest_bounded_wait(ws, limit_us=1000)
    assert binding.device_status(ws) == (-8, 100)
    assert binding.device_status(ws)[0] == 0          # reading the status cleared it
    binding.lib().zq_workspace_init(ws.data_ptr(), ws.numel(), None)
    for layout in (binding.WEIGHTS_CAST, binding.WEIGHTS_MX):   # a normal call on the re-initialized workspace
        pw = binding.pack_weight_fp4(up(W), 128, "M2", layout)
        y = binding.w4a8_linear(pw, x=to_bf16(x_bits), U=up(U), V=up(V), workspace=ws)
        assert binding.device_status(ws) == (0, 0)
        q_o, sx_o, t_o = oracle.quantize_act_fp8(x_bits, V)
        c_o, sh_o, sc_o = oracle.pack_weight_fp4(W, 128, "M2")
        y_o = oracle.w4a8_linear(q_o, sx_o, c_o, sh_o, sc_o, 128, "M2", U, t_o)
        assert np.abs(host(y).astype(np.float64) - y_o).max() <= TOL_REL * np.abs(y_o).max()
