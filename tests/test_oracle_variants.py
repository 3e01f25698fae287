"""Pins of the oracle's variant functions: the E5M2 and E3M0 formats (Section 2; Appendix A, Table A.1), E5M2 as
the cast target (Section 3, footnote), FP8 weights (Table 2, W8A8), the integer quantizer of Eq. 1, and the
LoRC factors (Section 3).  Each is checked against something other than itself: hand-typed code tables,
torch's own FP8 casts, closed forms, brute-force nearest-value searches, numpy's SVD."""
import numpy as np
import pytest
import torch

import oracle
from paper_2307_09782_b200 import synth


# ---- formats -----------------------------------------------------------------------------------------
def test_e3m0_all_sixteen_codes():
    # 1 sign, 3 exponent bits (bias 3), no mantissa: zero and the powers of two 2^-2 .. 2^4
    want = [0.0, 0.25, 0.5, 1.0, 2.0, 4.0, 8.0, 16.0]
    for c in range(8):
        assert oracle.e3m0_decode(c) == want[c]
        assert oracle.e3m0_decode(c | 8) == -want[c]
    for c in range(16):
        if c != 8:
            assert oracle.e3m0_encode(oracle.e3m0_decode(c)) == c
    # rounding: nearest power of two in value, saturating at 16, everything below half the smallest to zero
    assert oracle.e3m0_encode(3.1) == 5 and oracle.e3m0_encode(2.9) == 4
    assert oracle.e3m0_encode(100.0) == 7 and oracle.e3m0_encode(-1e9) == 15
    assert oracle.e3m0_encode(0.1) == 0 and oracle.e3m0_encode(0.13) == 1


def test_e5m2_landmarks_and_all_codes_against_torch():
    landmarks = {0x00: 0.0, 0x01: 2.0 ** -16, 0x03: 3 * 2.0 ** -16, 0x04: 2.0 ** -14, 0x3C: 1.0, 0x3D: 1.25,
                 0x3E: 1.5, 0x3F: 1.75, 0x40: 2.0, 0x7B: 57344.0, 0xBC: -1.0}
    for code, v in landmarks.items():
        assert oracle.e5m2_decode(code) == v
        assert oracle.e5m2_encode(v) == code
    t = torch.arange(256, dtype=torch.uint8).view(torch.float8_e5m2).float().numpy()
    for c in range(256):
        d = oracle.e5m2_decode(c)
        assert (np.isnan(d) and np.isnan(t[c])) or d == t[c], c
    assert oracle.e5m2_encode(1e9) == 0x7B and oracle.e5m2_encode(-1e9) == 0xFB   # saturating, no infinity


def test_e5m2_encode_against_torch_cast_on_every_bf16_value_in_range():
    bits = np.arange(0, 1 << 16, dtype=np.uint16)
    v = synth.bf16_bits_to_f32(bits)
    ok = np.isfinite(v) & (np.abs(v) <= 57344.0)
    want = torch.from_numpy(v[ok]).to(torch.float8_e5m2).view(torch.uint8).numpy()
    got = np.array([oracle.e5m2_encode(float(x)) for x in v[ok]], dtype=np.uint8)
    same = got == want
    # torch keeps the sign of a value that rounds to zero; so does the oracle
    assert same.all(), (v[ok][~same][:5], got[~same][:5], want[~same][:5])


def test_cast_to_e5m2_is_a_subtraction_in_the_exponent_field_down_to_shift_13():
    for c in range(16):
        base = oracle.widen_e5m2(c, 0)
        for d in range(0, 14):
            w = oracle.widen_e5m2(c, d)
            assert oracle.e5m2_decode(w) == oracle.e2m1_decode(c) * 2.0 ** -d     # exact: no rounding
            if c & 7:
                assert w == base - 4 * d, (c, d)                                   # exponent field starts at bit 2
    # one step further the smallest magnitude leaves the normal range: the byte is no longer base - 4 d
    assert oracle.widen_e5m2(1, 14) != oracle.widen_e5m2(1, 0) - 4 * 14
    # within shift <= 5 both cast targets hold the same values
    for c in range(16):
        for d in range(6):
            assert oracle.e5m2_decode(oracle.widen_e5m2(c, d)) == oracle.e4m3_decode(oracle.widen(c, d))


# ---- weights in other formats ------------------------------------------------------------------------
def _unpack_nibbles(codes):
    out = np.empty((codes.shape[0], codes.shape[1] * 2), dtype=np.uint8)
    out[:, 0::2] = codes & 0xF
    out[:, 1::2] = codes >> 4
    return out


@pytest.mark.parametrize("mode", ["none", "M1", "M2"])
def test_general_pack_reduces_to_the_fp4_pack(mode):
    W = synth.make_w(3, 24, 512)
    W[2, :128] *= 2.0 ** -9
    c4, sh4, sc4 = oracle.pack_weight_fp4(W, 128, mode)
    c, sh, sc = oracle.pack_weight(W, 128, mode, "e2m1", 5)
    assert np.array_equal(_unpack_nibbles(c4), c)
    assert np.array_equal(sc4.view(np.uint32), sc.view(np.uint32))
    assert (sh4 is None and sh is None) or np.array_equal(sh4, sh)
    x_bits = synth.make_x(3, 4, 512, 5, 20.0)
    q, sx, _ = oracle.quantize_act_fp8(x_bits)
    assert np.array_equal(oracle.w4a8_linear(q, sx, c4, sh4, sc4, 128, mode),
                          oracle.linear_general(q, sx, c, sh, sc, 128, mode, "e2m1"))


@pytest.mark.parametrize("mode", ["none", "M1", "M2"])
@pytest.mark.parametrize("group", [64, 128, 320])
def test_fp8_weights_closed_forms(mode, group):
    K = 640
    W = synth.make_w(5, 16, K)
    W[1, :group] *= 2.0 ** -7        # a shift of 7: beyond the FP4 clamp, fine for a block scale
    c, sh, sc = oracle.pack_weight(W, group, mode, "e4m3", 127)
    G = K // group
    S = (np.abs(W).reshape(16, G, group).max(axis=2) / np.float32(448.0)).astype(np.float32)
    if mode == "none":
        assert np.array_equal(sc, S)
        shat = S.astype(np.float64)
    elif mode == "M1":
        p = np.ceil(np.log2(S.astype(np.float64)))
        assert np.array_equal(sc.astype(np.float64), 2.0 ** p.max(axis=1))
        assert np.array_equal(sh, (p.max(axis=1, keepdims=True) - p).astype(np.uint8))
        shat = 2.0 ** p
    else:
        smax = S.max(axis=1, keepdims=True).astype(np.float64)
        d = np.ceil(np.log2(smax / S.astype(np.float64)))
        assert np.array_equal(sc, S.max(axis=1)) and np.array_equal(sh, d.astype(np.uint8))
        shat = smax / 2.0 ** d
        assert sh[1, 0] >= 7
    # codes: torch's own saturating-free cast of fl32(W / S^) where in range, +-448 where the ratio exceeds it
    ratio = (W.reshape(16, G, group) / shat[:, :, None].astype(np.float32)).astype(np.float32).reshape(16, K)
    want = torch.from_numpy(np.clip(ratio, -448, 448)).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    assert np.array_equal(c, want)
    # the linear over these weights equals numpy's matmul of the dequantized operands
    x_bits = synth.make_x(5, 3, K, 6, 20.0)
    q, sx, _ = oracle.quantize_act_fp8(x_bits)
    xh = np.array([[oracle.e4m3_decode(v) for v in row] for row in q]) * sx[:, None].astype(np.float64)
    wh = np.array([[oracle.e4m3_decode(v) for v in row] for row in c]) * np.repeat(shat, group, axis=1)
    y = oracle.linear_general(q, sx, c, sh, sc, group, mode, "e4m3")
    assert np.abs(y - xh @ wh.T).max() <= 1e-12 * np.abs(y).max()


def test_group_320_fp4_and_e3m0_weights():
    # the group size the paper uses for the model whose hidden size is 3200 (Appendix A), and the E3M0 codes
    W = synth.make_w(6, 8, 640)
    for fmt, vmax in (("e2m1", 6.0), ("e3m0", 16.0)):
        c, sh, sc = oracle.pack_weight(W, 320, "none", fmt, 5)
        S = np.abs(W).reshape(8, 2, 320).max(axis=2) / np.float32(vmax)
        assert np.array_equal(sc, S.astype(np.float32))
        dec = oracle.e2m1_decode if fmt == "e2m1" else oracle.e3m0_decode
        grid = np.array(sorted({dec(k) for k in range(16)}))
        what = np.array([[dec(v) for v in row] for row in c])
        ratio = W / np.repeat(S, 320, axis=1)
        # every code is a nearest grid value of its ratio
        best = np.abs(ratio[:, :, None] - grid[None, None, :]).min(axis=2)
        assert np.all(np.abs(ratio - what) <= best + 1e-6)
        # the arg-max of every group lands on +-vmax
        for n in range(8):
            for g in range(2):
                k = np.abs(W[n, g * 320:(g + 1) * 320]).argmax() + g * 320
                assert abs(what[n, k]) == vmax


# ---- Eq. 1 and the FP-versus-INT comparison -------------------------------------------------------------
def test_integer_quantizer_closed_forms_and_brute_force():
    rng = np.random.default_rng(0)
    x = rng.normal(size=257)
    x[17] = 9.0
    for bits in (4, 8):
        ys = oracle.int_fake_quant(x, bits, True)
        qmax = 2 ** (bits - 1) - 1
        S = np.abs(x).max() / qmax
        grid = np.arange(-qmax, qmax + 1) * S
        assert np.allclose(ys, grid[np.abs(x[:, None] - grid[None, :]).argmin(axis=1)], rtol=0, atol=1e-12)
        assert ys[17] == pytest.approx(9.0, abs=1e-12)
        ya = oracle.int_fake_quant(x, bits, False)
        S = (x.max() - x.min()) / (2 ** bits - 1)
        grid = x.min() + np.arange(2 ** bits) * S
        assert np.allclose(ya, grid[np.abs(x[:, None] - grid[None, :]).argmin(axis=1)], rtol=0, atol=1e-12)
        assert ya.min() == x.min() and ya.max() == pytest.approx(x.max(), abs=1e-12)
    assert np.array_equal(oracle.int_fake_quant(np.zeros(5), 8, True), np.zeros(5))


def test_fp_fake_quant_is_nearest_on_the_scaled_grid():
    rng = np.random.default_rng(1)
    x = rng.normal(size=300)
    for fmt, dec, ncodes, vmax in (("e2m1", oracle.e2m1_decode, 16, 6.0), ("e3m0", oracle.e3m0_decode, 16, 16.0),
                                   ("e4m3", oracle.e4m3_decode, 256, 448.0), ("e5m2", oracle.e5m2_decode, 256, 57344.0)):
        grid = np.array(sorted({dec(c) for c in range(ncodes) if np.isfinite(dec(c))}))
        S = np.abs(x).max() / vmax
        y = oracle.fp_fake_quant(x, fmt)
        best = np.abs(x[:, None] - grid[None, :] * S).min(axis=1)
        assert np.all(np.abs(x - y) <= best * (1 + 1e-6) + 1e-12), fmt


def test_formats_on_activations_with_outlier_channels_and_on_gaussian_weights():
    # Section 2's argument, on the synthetic stand-ins: with a few large channels in a token, the uniform INT8
    # grid spends its levels on the outliers and the bulk of the values is represented worse than by FP8-E4M3;
    # for near-Gaussian weights E2M1 beats E3M0 (Table A.1's ranking), and E4M3 beats E5M2 as an 8-bit code.
    x = synth.bf16_bits_to_f32(synth.make_x(4, 64, 4096, 41, 20.0)).astype(np.float64)
    out = synth.outlier_channels(4, 4096, 41)
    bulk = np.ones(4096, dtype=bool)
    bulk[out] = False
    err = {}
    for name, fn in (("int8_sym", lambda r: oracle.int_fake_quant(r, 8, True)),
                     ("int8_asym", lambda r: oracle.int_fake_quant(r, 8, False)),
                     ("e4m3", lambda r: oracle.fp_fake_quant(r, "e4m3")),
                     ("e5m2", lambda r: oracle.fp_fake_quant(r, "e5m2"))):
        e = np.stack([fn(row) - row for row in x])
        err[name] = float((e[:, bulk] ** 2).mean())
    assert err["e4m3"] < 0.25 * err["int8_sym"] and err["e4m3"] < 0.25 * err["int8_asym"]
    assert err["e4m3"] < err["e5m2"]
    W = synth.make_w(4, 64, 1024).astype(np.float64)
    werr = {}
    for name, fn in (("e2m1", lambda g: oracle.fp_fake_quant(g, "e2m1")), ("e3m0", lambda g: oracle.fp_fake_quant(g, "e3m0")),
                     ("int4_sym", lambda g: oracle.int_fake_quant(g, 4, True))):
        e = np.concatenate([fn(g) - g for g in W.reshape(-1, 128)])
        werr[name] = float((e ** 2).mean())
    assert werr["e2m1"] < werr["e3m0"]
    assert 0.5 < werr["e2m1"] / werr["int4_sym"] < 2.0      # comparable, as the paper finds for FP4 against INT4


# ---- LoRC factors ---------------------------------------------------------------------------------------
@pytest.mark.parametrize("N,K,r", [(96, 64, 8), (48, 160, 16), (64, 64, 5)])
def test_lorc_factors_against_numpy_svd(N, K, r):
    rng = np.random.default_rng(N + K)
    E = rng.normal(size=(N, K)) * np.geomspace(1.0, 1e-3, K)[None, :]
    U, V, sg = oracle.lorc_factors(E, r)
    s_np = np.linalg.svd(E, compute_uv=False)
    assert np.allclose(sg, s_np, rtol=1e-10, atol=1e-12)
    # best rank-r approximation: the squared Frobenius error is the sum of the dropped singular values squared
    assert np.linalg.norm(E - U @ V) ** 2 == pytest.approx((s_np[r:] ** 2).sum(), rel=1e-9)
    # the two factors share sigma evenly: U^T U = V V^T = diag(sigma_r)
    assert np.allclose(U.T @ U, np.diag(s_np[:r]), atol=1e-9 * s_np[0])
    assert np.allclose(V @ V.T, np.diag(s_np[:r]), atol=1e-9 * s_np[0])


def test_lorc_factors_recover_a_low_rank_error_exactly_and_reduce_the_weight_error():
    rng = np.random.default_rng(9)
    A, B = rng.normal(size=(40, 4)), rng.normal(size=(4, 72))
    U, V, sg = oracle.lorc_factors(A @ B, 4)
    assert np.abs(U @ V - A @ B).max() <= 1e-10 and sg[4] <= 1e-10
    # on a quantized weight: W^ + U^ V^ is closer to W than W^ is, by exactly the captured singular values
    W = synth.make_w(9, 64, 256)
    c, sh, sc = oracle.pack_weight(W, 128, "M2", "e2m1", 5)
    what = np.array([[oracle.e2m1_decode(v) for v in row] for row in c]) * \
        np.repeat(sc[:, None].astype(np.float64) / 2.0 ** sh, 128, axis=1)
    E = W.astype(np.float64) - what
    U, V, sg = oracle.lorc_factors(E, 8)
    assert np.linalg.norm(E - U @ V) ** 2 == pytest.approx(np.linalg.norm(E) ** 2 - (sg[:8] ** 2).sum(), rel=1e-9)
