"""GPU parity of the layout in which the tensor core performs the cast FP4 -> FP8 (Section 3, "Casting the
FP4 to FP8"): E2M1 codes as the MMA's own operand, the power-of-two group shift as its E8M0 block scale.
Same oracle, same tolerances as the casting kernel: packed codes / shifts / scales bit-exact, outputs within
1e-3 of max |y|, and exact where every product and sum is exactly representable."""
import numpy as np
import pytest
import torch

import oracle
from paper_2307_09782_b200 import binding, synth
from tests.gpu_util import TOL_REL, check_linear, check_packed, host, to_bf16, up
from tests.test_gpu_parity import _layer, _special_weights

pytestmark = pytest.mark.gpu
MX = binding.WEIGHTS_MX


@pytest.mark.parametrize("mode", ["M1", "M2"])
@pytest.mark.parametrize("group", [64, 128, 256])
def test_pack_weight_mx_bit_exact(mode, group):
    W = _special_weights(9, 1024, 31)
    c_o, sh_o, sc_o = oracle.pack_weight_fp4(W, group, mode)
    check_packed(binding.pack_weight_fp4(up(W), group, mode, MX), c_o, sh_o, sc_o, group)


@pytest.mark.parametrize("group", [64, 128, 256])
def test_pack_weight_mx_unconstrained_scales(group):
    # mode none in the block-scaled arrangement: the same codes, unit block scales, FP32 scales beside them
    W = _special_weights(9, 512, 31)
    c_o, sh_o, sc_o = oracle.pack_weight_fp4(W, group, "none")
    check_packed(binding.pack_weight_fp4(up(W), group, "none", MX), c_o, sh_o, sc_o, group)


@pytest.mark.parametrize("group", [64, 128, 256])
@pytest.mark.parametrize("M,N,K,r", [(1, 384, 1024, 8), (16, 256, 8192, 8), (40, 200, 2048, 0), (100, 640, 512, 8),
                                     (128, 128 * 9, 768, 16), (300, 1000, 1024, 8), (700, 128 * 150, 512, 8)])
def test_linear_unconstrained_scales(M, N, K, r, group):
    # per-group promotion with the FP32 group scale (Section 3: what M1 / M2 remove) in the block-scaled kernel:
    # unit ranges with shared tiles, whole tiles, several token tiles of 128, groups of half / one / two K blocks
    x_bits, W, U, V = _layer(900 + M, M, N, K, r)
    rows = None if M <= 300 else [0, 127, 128, 255, 256, 511, 512, M - 1]
    check_linear(x_bits, W, U, V, group, "none", layout=MX, rows=rows)


def test_linear_unconstrained_scales_bf16_and_exact():
    x_bits, W, U, V = _layer(950, 48, 512, 1024, 8)
    check_linear(x_bits, W, U, V, 128, "none", out_dtype=torch.bfloat16, layout=MX)
    M, N, K = 16, 256, 512
    rng = np.random.default_rng(5)
    x = rng.choice([0.0, 0.25, 0.5, 1.0, -1.0, 2.0], (M, K)).astype(np.float32)
    x[:, 0] = 7.0
    W = rng.choice([0.0, 0.5, -1.0, 1.5, 3.0, -4.0], (N, K)).astype(np.float32)
    W[:, ::128] = 6.0
    W[3, 128:256] *= 0.125
    y, y_o = check_linear(synth.f32_to_bf16_bits(x), W, None, None, 128, "none", layout=MX)
    assert np.array_equal(y, y_o)


@pytest.mark.parametrize("mode", ["M1", "M2"])
@pytest.mark.parametrize("M", [1, 16, 17, 100, 130, 300])
def test_linear_small(mode, M):
    x_bits, W, U, V = _layer(40 + M, M, 384, 512, 8)
    check_linear(x_bits, W, U, V, 128, mode, layout=MX)


@pytest.mark.parametrize("M,N,K,r", [(3, 200, 256, 0), (33, 128, 128, 16), (64, 129, 1024, 8), (7, 1, 384, 8),
                                     (192, 256, 512, 8), (200, 300, 512, 8), (256, 128, 256, 0),
                                     (700, 1000, 1024, 8), (1153, 2000, 256, 8)])
def test_linear_ragged_tiles(M, N, K, r):
    x_bits, W, U, V = _layer(60 + M, M, N, K, r)
    check_linear(x_bits, W, U, V, 128, "M2", layout=MX)


@pytest.mark.parametrize("mode,group", [("M1", 64), ("M2", 256), ("M2", 64)])
def test_linear_other_group_sizes(mode, group):
    x_bits, W, U, V = _layer(71, 20, 256, 1024, 8)
    check_linear(x_bits, W, U, V, group, mode, layout=MX)


@pytest.mark.parametrize("M", [16, 40, 200])
def test_linear_split_k_long_rows(M):
    # few output tiles and a long K: several CTAs share an output tile (atomics or the workspace)
    x_bits, W, U, V = _layer(81, M, 256, 8192, 8)
    check_linear(x_bits, W, U, V, 128, "M1", layout=MX)


def test_linear_many_tiles_per_cta():
    # more output tiles than resident CTAs at 16 tokens: every CTA walks several segments, both accumulators
    x_bits, W, U, V = _layer(83, 9, 128 * 40, 1024, 8)
    check_linear(x_bits, W, U, V, 128, "M2", layout=MX)


def test_linear_many_token_tiles_per_cta():
    # more 192-token tiles than SMs: the persistent CTAs walk several tiles with different tokens, and the
    # launch order runs through groups of token tiles
    x_bits, W, U, V = _layer(85, 192 * 11 + 5, 128 * 20, 256, 8)
    rows = [0, 191, 192, 383, 1000, 192 * 8 - 1, 192 * 8, 192 * 11, 192 * 11 + 4]
    check_linear(x_bits, W, U, V, 128, "M1", layout=MX, rows=rows)


@pytest.mark.parametrize("M", [1120, 1000])
def test_linear_persistent_whole_tiles(M):
    # 600 or 720 output tiles, more than four per SM: every CTA walks whole tiles (224 or 192 tokens wide) of
    # different token rows with both accumulator buffers
    x_bits, W, U, V = _layer(89, M, 128 * 120, 512, 8)
    rows = [0, 191, 192, 223, 224, 447, 448, 700, M - 2, M - 1]
    check_linear(x_bits, W, U, V, 128, "M2", layout=MX, rows=rows)


@pytest.mark.parametrize("M,N,K,r,mode,layout,out_dtype", [
    (1120, 128 * 120, 512, 8, "M2", MX, torch.bfloat16),           # 224-token tiles, bf16 y
    (1000, 128 * 120 - 37, 384, 8, "M1", MX, torch.float32),       # 208-token tiles, ragged last channel tile
    (1100, 128 * 120, 256, 0, "M2", MX, torch.float32),            # no LoRC
    (1120, 128 * 120, 256, 16, "M2", MX, torch.float32),           # a rank the epilogue reads through the cache
    (896, 128 * 148, 256, 8, "M2", MX, torch.float32),             # four whole rounds of 74 pairs
    (528, 128 * 200, 256, 8, "M2", MX, torch.float32),             # three tiles of 176 tokens
    (1040, 128 * 120, 384, 8, "M1", MX, torch.bfloat16),           # five tiles of 208 tokens
])
def test_linear_cta_pairs(M, N, K, r, mode, layout, out_dtype):
    """Many tokens and an even number of channel tiles: two CTAs share each token tile (one MMA of 256 channels
    over both CTAs' tensor memory), whole tiles only."""
    pl = binding.linear_plan(M, N, K, mode, layout)
    assert pl["pair"] == 1 and pl["bm"] in (176, 192, 208, 224)
    x_bits, W, U, V = _layer(91 + r, M, N, K, r)
    bm = pl["bm"]
    rows = sorted({min(v, M - 1) for v in (0, bm // 2 - 1, bm // 2, bm - 1, bm, bm + bm // 2, 2 * bm - 1, 3 * bm + 5,
                                           M - bm // 2 - 1, M - 2, M - 1)})
    check_linear(x_bits, W, U, V, 128, mode, layout=layout, rows=rows, out_dtype=out_dtype)


@pytest.mark.parametrize("M,N,K,out_dtype", [
    (500, 128 * 6, 2048, torch.float32),      # 3 x 3 positions x 16 K blocks dealt out as ranges: most positions shared
    (500, 128 * 6, 2048, torch.bfloat16),     # bf16 y with shared tiles: the single CTAs take it (workspace partial sums)
    (192, 128 * 150, 512, torch.float32),     # one row of 192-token tiles
    (100, 128 * 20, 1024, torch.float32),     # one row of 128-token tiles, 20 pairs
    (128, 128 * 150, 256, torch.float32),     # one row of 128-token tiles, all 74 pairs
    (1120, 128 * 120, 9216, torch.float32),   # four whole rounds, then four positions dealt out to all 74 pairs
])
def test_linear_cta_pairs_shared_positions(M, N, K, out_dtype):
    """Pair positions whose K range is split between pairs: the last contributor stores, the others wait for its
    flag and add; a second call on the same workspace must find the flags as the first one did."""
    pl = binding.linear_plan(M, N, K, "M2", MX)
    assert pl["pair"] == 1 and (pl["stream"] == 1 or pl["tail_pos0"] < pl["m_tiles"] * pl["n_tiles"] // 2)
    x_bits, W, U, V = _layer(93, M, N, K, 8)
    bm = pl["bm"]
    rows = sorted({min(v, M - 1) for v in (0, bm // 2 - 1, bm // 2, bm - 1, bm, M // 2, M - 2, M - 1)})
    q_o, sx_o, t_o = oracle.quantize_act_fp8(x_bits, V)
    c_o, sh_o, sc_o = oracle.pack_weight_fp4(W, 128, "M2")
    y_o = oracle.w4a8_linear(q_o, sx_o, c_o, sh_o, sc_o, 128, "M2", U, t_o, rows=rows)
    pw = binding.pack_weight_fp4(up(W), 128, "M2", MX)
    ws = binding.make_workspace(binding.linear_workspace_bytes(M, N, K, 8))
    q, sx, t = binding.quantize_act_fp8(to_bf16(x_bits), up(V))
    for _ in range(3):
        y = binding.w4a8_linear(pw, q=q, sx=sx, t=t, U=up(U), out_dtype=out_dtype, workspace=ws)
        assert binding.device_status(ws) == (0, 0)
        yh = host(y.float()).astype(np.float64)[rows]
        tol = TOL_REL * np.abs(y_o).max()
        if out_dtype == torch.bfloat16:
            tol = tol + 2.0 ** (np.floor(np.log2(np.maximum(np.abs(y_o), 1e-30))) - 7)
        assert np.all(np.abs(yh - y_o) <= tol)


@pytest.mark.parametrize("seed", range(12))
def test_linear_cta_pairs_seeded_random_shapes(seed):
    """Seeded random shapes with an even number of channel tiles (ragged last tile, any K, ranks 0 / 8 / 16, both
    output types): whatever partition the plan picks, sampled rows must match the oracle, twice on one workspace."""
    rng = np.random.default_rng(4242 + seed)
    M = int(rng.choice([rng.integers(65, 129), rng.integers(129, 600), rng.integers(600, 2600)]))
    N = 256 * int(rng.integers(1, 80)) - int(rng.integers(0, 128))
    K = 128 * int(rng.integers(1, 40))
    r = int(rng.choice([0, 8, 8, 16]))
    mode = str(rng.choice(["M1", "M2"]))
    out_dtype = torch.float32 if rng.random() < 0.75 else torch.bfloat16
    assert binding.linear_plan(M, N, K, mode, MX)["pair"] == 1 or M > 224
    x_bits, W, U, V = _layer(2000 + seed, M, N, K, r)
    rows = sorted(set(int(v) for v in rng.integers(0, M, 10)) | {0, M - 1})
    q_o, sx_o, t_o = oracle.quantize_act_fp8(x_bits, V)
    c_o, sh_o, sc_o = oracle.pack_weight_fp4(W, 128, mode)
    y_o = oracle.w4a8_linear(q_o, sx_o, c_o, sh_o, sc_o, 128, mode, U, t_o, rows=rows)
    pw = binding.pack_weight_fp4(up(W), 128, mode, MX)
    ws = binding.make_workspace(binding.linear_workspace_bytes(M, N, K, r))
    q, sx, t = binding.quantize_act_fp8(to_bf16(x_bits), up(V))
    tol = TOL_REL * np.abs(y_o).max()
    if out_dtype == torch.bfloat16:
        tol = tol + 2.0 ** (np.floor(np.log2(np.maximum(np.abs(y_o), 1e-30))) - 7)
    for _ in range(2):
        y = binding.w4a8_linear(pw, q=q, sx=sx, t=t, U=up(U), out_dtype=out_dtype, workspace=ws)
        assert binding.device_status(ws) == (0, 0)
        assert np.all(np.abs(host(y.float()).astype(np.float64)[rows] - y_o) <= tol)


def test_linear_cta_pairs_fp8_weights():
    M, N, K, r = 1120, 128 * 120, 384, 8
    assert binding.linear_plan(M, N, K, "M2", binding.WEIGHTS_MX_FP8)["pair"] == 1
    x_bits, W, U, V = _layer(97, M, N, K, r)
    rows = [0, 111, 112, 223, 224, 500, M - 113, M - 1]
    q_o, sx_o, t_o = oracle.quantize_act_fp8(x_bits, V)
    c_o, sh_o, sc_o = oracle.pack_weight(W, 128, "M2", "e4m3", 127)
    y_o = oracle.linear_general(q_o[rows], sx_o[rows], c_o, sh_o, sc_o, 128, "M2", "e4m3", U, t_o[rows])
    pw = binding.pack_weight_fp4(up(W), 128, "M2", binding.WEIGHTS_MX_FP8)
    ws = binding.make_workspace(binding.linear_workspace_bytes(M, N, K, r))
    q, sx, t = binding.quantize_act_fp8(to_bf16(x_bits), up(V))
    y = binding.w4a8_linear(pw, q=q, sx=sx, t=t, U=up(U), workspace=ws)
    assert binding.device_status(ws) == (0, 0)
    assert np.abs(host(y).astype(np.float64)[rows] - y_o).max() <= TOL_REL * np.abs(y_o).max()


@pytest.mark.parametrize("out_dtype", [torch.float32, torch.bfloat16])
def test_linear_persistent_last_round_shared(out_dtype):
    # 600 tiles of 72 K blocks on 148 SMs: four whole rounds, then the 8 tiles of the last round are dealt
    # out as unit ranges to all CTAs (FP32 y: cleared in the kernel and added into; bf16 y: partial sums
    # through the workspace)
    M = 1120
    x_bits, W, U, V = _layer(90, M, 128 * 120, 9216, 8)
    rows = [0, 223, 224, 700, M - 1]
    check_linear(x_bits, W, U, V, 128, "M2", layout=MX, rows=rows, out_dtype=out_dtype)


def test_linear_several_token_tiles_dealt_out_as_unit_ranges():
    # fewer 192-token tiles than four per SM: contiguous unit ranges across token tiles, shared tiles added
    # with atomics (FP32 y) or handed over through the workspace (bf16 y)
    x_bits, W, U, V = _layer(87, 500, 640, 2048, 8)
    rows = [0, 191, 192, 383, 384, 499]
    check_linear(x_bits, W, U, V, 128, "M2", layout=MX, rows=rows)
    check_linear(x_bits, W, U, V, 128, "M2", layout=MX, rows=rows, out_dtype=torch.bfloat16)


def test_linear_bf16_output_and_fused_quantizer():
    x_bits, W, U, V = _layer(91, 48, 512, 1024, 8)
    check_linear(x_bits, W, U, V, 128, "M2", out_dtype=torch.bfloat16, layout=MX)
    check_linear(x_bits, W, U, V, 128, "M2", fused_quant=True, layout=MX)
    check_linear(x_bits, W, None, None, 128, "M1", fused_quant=True, layout=MX)


def test_linear_exact_on_power_of_two_data():
    M, N, K = 16, 256, 512
    rng = np.random.default_rng(5)
    x = rng.choice([0.0, 0.25, 0.5, 1.0, -1.0, 2.0], (M, K)).astype(np.float32)
    x[:, 0] = 7.0
    W = rng.choice([0.0, 0.5, -1.0, 1.5, 3.0, -4.0], (N, K)).astype(np.float32)
    W[:, ::128] = 6.0
    W[3, 128:256] *= 0.125   # a group with shift 3
    W[200, 256:] *= 0.25     # shift 2 over two groups
    bits = synth.f32_to_bf16_bits(x)
    for mode in ("M1", "M2"):
        y, y_o = check_linear(bits, W, None, None, 128, mode, layout=MX)
        assert np.array_equal(y, y_o), mode


def test_both_layouts_agree():
    # same codes, same products: the two kernels differ only in summation order
    M, N, K, r = 64, 384, 2048, 8
    x_bits, W, U, V = _layer(97, M, N, K, r)
    x = to_bf16(x_bits)
    q, sx, t = binding.quantize_act_fp8(x, up(V))
    ys = []
    for layout in (binding.WEIGHTS_CAST, MX):
        pw = binding.pack_weight_fp4(up(W), 128, "M2", layout)
        ys.append(host(binding.w4a8_linear(pw, q=q, sx=sx, t=t, U=up(U))))
    assert np.abs(ys[0] - ys[1]).max() <= 1e-5 * np.abs(ys[0]).max()


def _fuzz_cases():
    rng = np.random.default_rng(20230719)
    cases = []
    for i in range(28):
        kind = i % 4
        if kind == 0:      # decode-like: one narrow row of tiles, long K (unit ranges, shared tiles)
            M, N, K = int(rng.integers(1, 65)), 128 * int(rng.integers(1, 12)) - int(rng.integers(0, 100)), \
                128 * int(rng.integers(8, 72))
        elif kind == 1:    # one row of wide tiles
            M, N, K = int(rng.integers(65, 257)), 128 * int(rng.integers(1, 40)), 128 * int(rng.integers(1, 20))
        elif kind == 2:    # several token tiles, few output tiles (unit ranges across token tiles)
            M, N, K = int(rng.integers(257, 1500)), 128 * int(rng.integers(1, 6)) - int(rng.integers(0, 60)), \
                128 * int(rng.integers(2, 40))
        else:              # many tiles: persistent launch, with and without a shared last round
            M, N, K = int(rng.integers(700, 2400)), 128 * int(rng.integers(60, 130)), 128 * int(rng.integers(1, 4))
        N = max(N, 1)
        cases.append((M, N, K, ["M1", "M2"][i % 2], [64, 128, 256][i % 3], [0, 8, 8, 16][i % 4],
                      torch.float32 if i % 5 else torch.bfloat16))
    return cases


@pytest.mark.parametrize("M,N,K,mode,group,r,out_dtype", _fuzz_cases())
def test_linear_seeded_random_shapes(M, N, K, mode, group, r, out_dtype):
    """Seeded random shapes through every branch of the launch plan; sampled token rows against the oracle."""
    if K % group:
        K += group - K % group
    x_bits, W, U, V = _layer(1000 + M + N, M, N, K, r)
    rng = np.random.default_rng(M * 7 + N)
    rows = sorted(set([0, M - 1] + [int(v) for v in rng.integers(0, M, 6)] +
                      [b for b in (191, 192, 223, 224, 255, 256) if b < M]))
    check_linear(x_bits, W, U, V, group, mode, layout=MX, rows=rows, out_dtype=out_dtype)


@pytest.mark.parametrize("layout", [binding.WEIGHTS_CAST, MX])
def test_host_buffer_entry_point_in_row_chunks(layout):
    # more than 1024 tokens: the host entry uploads, computes and downloads in overlapping row chunks
    M, N, K, r = 2600, 384, 512, 8
    x_bits, W, U, V = _layer(96, M, N, K, r)
    pw = binding.pack_weight_fp4(up(W), 128, "M2", layout)
    ws = binding.make_workspace(binding.linear_host_workspace_bytes(M, N, K, r))
    xh = torch.from_numpy(x_bits.view(np.int16)).view(torch.bfloat16).pin_memory()
    yh = torch.full((M, N), float("nan"), dtype=torch.float32).pin_memory()
    for _ in range(2):   # the second call reuses the copy streams
        binding.w4a8_linear_host(xh, yh, pw, U=up(U), V=up(V), workspace=ws)
    assert binding.device_status(ws) == (0, 0)
    q_o, sx_o, t_o = oracle.quantize_act_fp8(x_bits, V)
    c_o, sh_o, sc_o = oracle.pack_weight_fp4(W, 128, "M2")
    rows = [0, 1023, 1024, 2047, 2048, 2599] + list(range(1000, 1100, 7))
    y_o = oracle.w4a8_linear(q_o, sx_o, c_o, sh_o, sc_o, 128, "M2", U, t_o, rows=rows)
    assert not np.isnan(yh.numpy()).any()
    assert np.abs(yh.numpy()[rows] - y_o).max() <= TOL_REL * np.abs(y_o).max()
    # the same numbers as the device entry point up to summation order
    y_d = host(binding.w4a8_linear(pw, x=to_bf16(x_bits), U=up(U), V=up(V)))
    assert np.abs(yh.numpy() - y_d).max() <= 1e-5 * np.abs(y_d).max()


@pytest.mark.parametrize("M,N,K", [(8, 640, 4096), (40, 200, 2048), (300, 384, 512), (1120, 15360, 256), (500, 768, 2048)])
def test_strided_output_leaves_the_gaps_alone(M, N, K):
    # y with a leading dimension larger than N: shared tiles (store / flag / add), whole tiles, the persistent
    # launch and the CTA pairs (whole and shared positions) must write exactly the M x N block
    x_bits, W, U, V = _layer(98, M, N, K, 8)
    pw = binding.pack_weight_fp4(up(W), 128, "M2", MX)
    q, sx, t = binding.quantize_act_fp8(to_bf16(x_bits), up(V))
    pad = 24
    buf = torch.full((M, N + pad), float("nan"), dtype=torch.float32, device="cuda")
    y = buf[:, :N]
    binding.w4a8_linear(pw, q=q, sx=sx, t=t, U=up(U), y=y)
    ref = binding.w4a8_linear(pw, q=q, sx=sx, t=t, U=up(U))
    assert torch.isnan(buf[:, N:]).all()
    assert np.abs(host(y) - host(ref)).max() <= 1e-5 * np.abs(host(ref)).max()
