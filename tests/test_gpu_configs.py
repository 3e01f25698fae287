"""GPU parity at the full sizes of the five workload configurations, in the launch shapes bench.py times.

Every packed FP4 code, shift, scale, FP8 activation code and token scale is compared bit for bit with the
oracle on the whole tensor.  Outputs are compared on sampled token rows, all N columns of each, within
1e-3 * max|y| over the sampled rows, because the FP64 oracle needs a fraction of a second per row at these
sizes.  The sample of a case is built from the token-tile width the launch plan really picks for each weight
layout (asked from zq_w4a8_linear_plan): the first and the last row, both rows at every tile boundary, one
seeded row inside every token tile, and 32 further seeded rows; up to 64 tokens every row is compared.
The LoRC-off variant of a case runs the same kernels with another epilogue branch, so it takes the
boundaries of the first two and the last tile plus 8 seeded rows.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2307_09782_b200 import binding, synth
from gpu_util import TOL_REL, check_packed, host, to_bf16, up

pytestmark = pytest.mark.gpu


def _sample_rows(M, bms, seed, full=True):
    """Token rows to compare: see the module docstring.  `bms`: tile widths in use (one per weight layout)."""
    if M <= 64:
        return list(range(M))
    rng = np.random.default_rng(seed)
    rows = {0, M - 1}
    for bm in bms:
        n_tiles = (M + bm - 1) // bm
        tiles = range(n_tiles) if full else sorted({0, min(1, n_tiles - 1), n_tiles - 1})
        for ti in tiles:
            lo, hi = ti * bm, min((ti + 1) * bm, M)
            rows.update((lo, hi - 1))
            if lo > 0:
                rows.add(lo - 1)
            if full:
                rows.add(int(rng.integers(lo, hi)))
    rows.update(int(v) for v in rng.integers(0, M, size=32 if full else 8))
    assert all(0 <= v < M for v in rows)
    return sorted(rows)


def _run_layer(wl, shape, modes, Ms, lorc_variants=(True,)):
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
        # both weight layouts: the kernel that casts and the block-scaled one
        layouts = [binding.WEIGHTS_CAST, binding.WEIGHTS_MX]
        pws = []
        for layout in layouts:
            pw = binding.pack_weight_fp4(W_d, wl.group, mode, layout)
            check_packed(pw, c_o, sh_o, sc_o, wl.group)
            pws.append(pw)
        for M in Ms:
            for with_lorc in lorc_variants:
                use = bool(r) and with_lorc
                bms = sorted({binding.linear_plan(M, N, K, mode, pw.layout)["bm"] for pw in pws})
                rows = _sample_rows(M, bms, 1000 + M, full=with_lorc or not r)
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
    _run_layer(wl, wl.shapes[0], wl.modes, wl.Ms)


@pytest.mark.parametrize("i", [0, 1, 2])
def test_config_opt1_3b(i):
    wl = synth.WORKLOADS["opt1.3b"]
    _run_layer(wl, wl.shapes[i], wl.modes, wl.Ms)


@pytest.mark.parametrize("i", [0, 1, 2])
def test_config_llama7b(i):
    wl = synth.WORKLOADS["llama7b"]
    _run_layer(wl, wl.shapes[i], wl.modes, wl.Ms)


@pytest.mark.parametrize("i", [0, 1])
def test_config_llama30b(i):
    wl = synth.WORKLOADS["llama30b"]
    _run_layer(wl, wl.shapes[i], wl.modes, wl.Ms)


@pytest.mark.parametrize("i", [0, 1])
def test_config_opt30b(i):
    wl = synth.WORKLOADS["opt30b"]
    _run_layer(wl, wl.shapes[i], wl.modes, wl.Ms, lorc_variants=(True, False))
