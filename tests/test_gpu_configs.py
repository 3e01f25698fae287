"""GPU parity at the full sizes of the five workload configurations, in the launch shapes bench.py times.

Every packed FP4 code, shift, scale, FP8 activation code and token scale is compared bit for bit with the
oracle on the whole tensor.  Outputs are compared on sampled token rows (first, last, tile boundaries, a few
seeded random rows; all N columns of each) within 1e-3 * max|y| over the sampled rows, because the FP64
oracle needs about a second per row at these sizes.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2307_09782_b200 import binding, synth
from gpu_util import TOL_REL, check_packed, host, to_bf16, up

pytestmark = pytest.mark.gpu


def _sample_rows(M, bm, k, seed):
    rows = {0, M - 1}
    for b in (bm, 2 * bm):
        for r in (b - 1, b):
            if 0 <= r < M:
                rows.add(r)
    rng = np.random.default_rng(seed)
    while len(rows) < min(k, M):
        rows.add(int(rng.integers(0, M)))
    return sorted(rows)[:max(k, 1)] if M > k else sorted(rows)


def _run_layer(wl, shape, modes, Ms, rows_per_case, lorc_variants=(True,)):
    K, N = shape.K, shape.N
    Mmax = max(Ms)
    x_bits = synth.make_x(wl.seed, Mmax, K, wl.n_outliers(K), wl.outlier_factor)
    W = synth.make_w(wl.seed, N, K, wl.sigma_w)
    r = wl.lorc_rank
    U = V = None
    if r:
        U, V = synth.make_lorc(wl.seed, N, K, r)
    # quantizer on the whole activation tensor (this also goes through the many-rows kernel when M is large)
    q_o, sx_o, t_o = oracle.quantize_act_fp8(x_bits, V)
    x_d, U_d, V_d = to_bf16(x_bits), up(U), up(V)
    q, sx, t = binding.quantize_act_fp8(x_d, V_d)
    assert np.array_equal(host(q), q_o), "FP8 codes"
    assert np.array_equal(host(sx).view(np.uint32), sx_o.view(np.uint32)), "token scales"
    if r:
        assert np.abs(host(t) - t_o).max() <= 1e-4 * np.abs(t_o).max()
    del q, sx, t
    W_d = up(W)
    ws = binding.make_workspace(binding.linear_workspace_bytes(Mmax, N, K, r))
    for mode in modes:
        c_o, sh_o, sc_o = oracle.pack_weight_fp4(W, wl.group, mode)
        # both weight layouts for the constrained modes: the kernel that casts and the block-scaled one
        layouts = [binding.WEIGHTS_CAST] + ([binding.WEIGHTS_MX] if mode != "none" else [])
        pws = []
        for layout in layouts:
            pw = binding.pack_weight_fp4(W_d, wl.group, mode, layout)
            check_packed(pw, c_o, sh_o, sc_o, wl.group)
            pws.append(pw)
        for M in Ms:
            for with_lorc in lorc_variants:
                use = bool(r) and with_lorc
                bm = 16
                while bm < 256 and bm < M:
                    bm *= 2
                rows = sorted(set(_sample_rows(M, bm, rows_per_case, 1000 + M)) |
                              {r_ for r_ in (191, 192) if r_ < M})
                y_o = oracle.w4a8_linear(q_o[:M], sx_o[:M], c_o, sh_o, sc_o, wl.group, mode, U if use else None,
                                         t_o[:M] if use else None, rows=rows)
                for pw in pws:
                    y = binding.w4a8_linear(pw, x=x_d[:M], U=U_d if use else None, V=V_d if use else None,
                                            workspace=ws)
                    assert binding.device_status(ws) == (0, 0)
                    err = np.abs(host(y[rows]).astype(np.float64) - y_o).max()
                    assert err <= TOL_REL * np.abs(y_o).max(), (shape, mode, pw.layout, M, use, err, np.abs(y_o).max())
                    del y
        del pws


def test_config_opt125m():
    wl = synth.WORKLOADS["opt125m"]
    _run_layer(wl, wl.shapes[0], wl.modes, wl.Ms, rows_per_case=16)


@pytest.mark.parametrize("i", [0, 1, 2])
def test_config_opt1_3b(i):
    wl = synth.WORKLOADS["opt1.3b"]
    _run_layer(wl, wl.shapes[i], wl.modes, wl.Ms, rows_per_case=8)


@pytest.mark.parametrize("i", [0, 1, 2])
def test_config_llama7b(i):
    wl = synth.WORKLOADS["llama7b"]
    _run_layer(wl, wl.shapes[i], wl.modes, wl.Ms, rows_per_case=5)


@pytest.mark.parametrize("i", [0, 1])
def test_config_llama30b(i):
    wl = synth.WORKLOADS["llama30b"]
    _run_layer(wl, wl.shapes[i], wl.modes, wl.Ms, rows_per_case=4)


@pytest.mark.parametrize("i", [0, 1])
def test_config_opt30b(i):
    wl = synth.WORKLOADS["opt30b"]
    _run_layer(wl, wl.shapes[i], wl.modes, wl.Ms, rows_per_case=5, lorc_variants=(True, False))
