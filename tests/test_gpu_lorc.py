"""GPU check of the LoRC factor construction (Section 3: SVD of the error matrix E = W - W^, rank r, singular
values split between the two factors) against the oracle's Jacobi SVD.  The device finds the leading subspace by
randomized subspace iteration, and any orthogonal re-mixing of the factors is equally valid, so the comparison is
on what is unique: the product U^ V^ (through the residual ||E - U^ V^||_F against the optimum the oracle's
singular values give), the singular values, and the spanned subspace where a spectral gap defines it."""
import numpy as np
import pytest
import torch

import oracle
from paper_2307_09782_b200 import binding, synth
from tests.gpu_util import TOL_REL, host, to_bf16, up

pytestmark = pytest.mark.gpu


def _dequant(W, group, mode):
    c, sh, sc = oracle.pack_weight(W, group, mode, "e2m1", 5)
    dec = np.array([oracle.e2m1_decode(v) for v in range(16)])
    G = W.shape[1] // group
    shat = sc.astype(np.float64) if mode == "none" else sc[:, None].astype(np.float64) / 2.0 ** sh
    return dec[c] * np.repeat(shat.reshape(W.shape[0], G), group, axis=1)


def _omega(seed, K, l):
    return torch.from_numpy(np.random.default_rng(seed).standard_normal((K, l)).astype(np.float32)).cuda()


@pytest.mark.parametrize("r", [8, 16])
def test_error_with_a_spectral_gap_is_recovered(r):
    # W = grid values + a small rank-4 matrix: every code and scale is that of the grid part, so E is the rank-4
    # matrix exactly and the device must find it whatever the rank asked for
    N, K, g = 384, 512, 128
    rng = np.random.default_rng(3)
    grid = np.array([0.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0])
    Gm = rng.choice(grid, (N, K)) * rng.choice([-1.0, 1.0], (N, K))
    Gm[:, 0::g] = 6.0                       # every group's maximum, so that its scale is exactly 1
    A, B = rng.normal(size=(N, 4)), rng.normal(size=(4, K))
    B[:, 0::g] = 0.0                        # the perturbation leaves the maxima alone
    L = A @ B
    L *= 0.1 / np.abs(L).max()              # far inside half a grid step
    W = (Gm + L).astype(np.float32)
    E = W.astype(np.float64) - _dequant(W, g, "none")
    assert np.abs(E - (W.astype(np.float64) - Gm)).max() == 0.0
    U_o, V_o, sg = oracle.lorc_factors(E, r)
    pw = binding.pack_weight_fp4(up(W), g, "none")
    U, V, s2 = binding.lorc_factors(up(W), pw, r, _omega(1, K, r + 8), iters=2)
    U, V, s2 = host(U).astype(np.float64), host(V).astype(np.float64), host(s2).astype(np.float64)
    assert np.allclose(np.sqrt(np.maximum(s2[:4], 0)), sg[:4], rtol=1e-3)
    assert np.all(s2[4:] <= 1e-6 * s2[0])
    assert np.linalg.norm(E - U @ V) <= 2e-3 * np.linalg.norm(E)          # fp16 storage of the factors
    # the subspace: projector onto span(U^[:, :4]) against the oracle's
    Qd, _ = np.linalg.qr(U[:, :4])
    Qo, _ = np.linalg.qr(U_o[:, :4])
    assert np.linalg.norm(Qd @ Qd.T - Qo @ Qo.T, 2) <= 5e-3


@pytest.mark.parametrize("mode,r", [("M2", 8), ("M1", 16), ("none", 32), ("M2", 56)])
def test_quantization_error_of_a_gaussian_weight(mode, r):
    # the real use: E is the (nearly white) quantization error; the residual must be close to the optimum
    N, K, g = 512, 768, 128
    W = synth.make_w(11, N, K)
    W[:, :8] *= 6.0                          # a few heavy input channels give E some structure
    E = W.astype(np.float64) - _dequant(W, g, mode)
    _, _, sg = oracle.lorc_factors(E, r)
    opt_res2 = (sg[r:] ** 2).sum()
    opt_cap2 = (sg[:r] ** 2).sum()
    pw = binding.pack_weight_fp4(up(W), g, mode)
    U, V, s2 = binding.lorc_factors(up(W), pw, r, _omega(2, K, r + 8), iters=4)
    U, V = host(U).astype(np.float64), host(V).astype(np.float64)
    res2 = np.linalg.norm(E - U @ V) ** 2
    assert res2 >= opt_res2 * (1 - 1e-6)                      # nothing beats the truncated SVD
    cap2 = np.linalg.norm(E) ** 2 - res2
    assert cap2 >= 0.80 * opt_cap2, (cap2 / opt_cap2)
    assert np.all(host(s2).astype(np.float64)[:r] <= sg[:r] ** 2 * (1 + 1e-3))   # Ritz values from below
    # the factors share sigma: U^T U and V V^T are (nearly) the same diagonal matrix
    d1, d2 = np.diag(U.T @ U), np.diag(V @ V.T)
    assert np.allclose(d1, d2, rtol=2e-2)


def test_factors_feed_the_linear_layer():
    # the rank-56 epilogue on constructed factors: y against the oracle with the same fp16 U^, V^
    M, N, K, r = 48, 384, 1024, 56
    x_bits = synth.make_x(12, M, K, 10, 20.0)
    W = synth.make_w(12, N, K)
    for layout in (binding.WEIGHTS_CAST, binding.WEIGHTS_MX):
        pw = binding.pack_weight_fp4(up(W), 128, "M2", layout)
        U, V, _ = binding.lorc_factors(up(W), pw, r, _omega(3, K, r + 8), iters=2)
        ws = binding.make_workspace(binding.linear_workspace_bytes(M, N, K, r))
        y = binding.w4a8_linear(pw, x=to_bf16(x_bits), U=U, V=V, workspace=ws)
        assert binding.device_status(ws) == (0, 0)
        q_o, sx_o, t_o = oracle.quantize_act_fp8(x_bits, host(V))
        c_o, sh_o, sc_o = oracle.pack_weight_fp4(W, 128, "M2")
        y_o = oracle.w4a8_linear(q_o, sx_o, c_o, sh_o, sc_o, 128, "M2", host(U), t_o)
        assert np.abs(host(y).astype(np.float64) - y_o).max() <= TOL_REL * np.abs(y_o).max()
    # and the compensated weight is closer to W than the quantized one (Section 3's purpose of LoRC)
    E = W.astype(np.float64) - _dequant(W, 128, "M2")
    Uh, Vh = host(U).astype(np.float64), host(V).astype(np.float64)
    assert np.linalg.norm(E - Uh @ Vh) < np.linalg.norm(E)
