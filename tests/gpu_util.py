"""Helpers shared by the GPU parity tests: upload seeded inputs, run the oracle beside the CUDA path."""
import numpy as np
import torch

import oracle
from paper_2307_09782_b200 import binding, synth

TOL_REL = 1e-3  # max |err| <= TOL_REL * max |y_oracle|  (FP32 accumulation, order-dependent)


def dev():
    return torch.device("cuda:0")


def to_bf16(bits: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).to(dev()).view(torch.bfloat16)


def up(a):
    return None if a is None else torch.from_numpy(np.ascontiguousarray(a)).to(dev())


def host(t):
    return None if t is None else t.cpu().numpy()


def check_linear(x_bits, W, U, V, group, mode, out_dtype=torch.float32, rows=None, fused_quant=False):
    """Runs oracle and CUDA path on the same inputs; asserts bit-exact codes / scales and y within tolerance."""
    M, K = x_bits.shape
    N = W.shape[0]
    r = 0 if U is None else U.shape[1]
    q_o, sx_o, t_o = oracle.quantize_act_fp8(x_bits, V)
    c_o, sh_o, sc_o = oracle.pack_weight_fp4(W, group, mode)
    y_o = oracle.w4a8_linear(q_o, sx_o, c_o, sh_o, sc_o, group, mode, U, t_o, rows=rows)

    x = to_bf16(x_bits)
    Wd, Ud, Vd = up(W), up(U), up(V)
    codes, shift, scale = binding.pack_weight_fp4(Wd, group, mode)
    assert np.array_equal(host(codes), c_o), "FP4 codes"
    if sh_o is not None:
        assert np.array_equal(host(shift), sh_o), "shifts"
    assert np.array_equal(host(scale).view(np.uint32), sc_o.view(np.uint32)), "scales"
    ws = binding.make_workspace(binding.linear_workspace_bytes(M, N, K, r))
    if fused_quant:
        y = binding.w4a8_linear(codes, shift, scale, group, mode, x=x, U=Ud, V=Vd, out_dtype=out_dtype, workspace=ws)
    else:
        q, sx, t = binding.quantize_act_fp8(x, Vd)
        assert np.array_equal(host(q), q_o), "FP8 codes"
        assert np.array_equal(host(sx).view(np.uint32), sx_o.view(np.uint32)), "token scales"
        if r:
            assert np.abs(host(t) - t_o).max() <= 1e-4 * max(np.abs(t_o).max(), 1e-30), "LoRC down-projection"
        y = binding.w4a8_linear(codes, shift, scale, group, mode, q=q, sx=sx, t=t, U=Ud, out_dtype=out_dtype,
                                workspace=ws)
    st, detail = binding.device_status(ws)
    assert st == 0, f"device status {st} detail {detail}"
    yh = y.float().cpu().numpy().astype(np.float64)
    if rows is not None:
        yh = yh[np.asarray(rows)]
    ymax = np.abs(y_o).max()
    if out_dtype == torch.float32:
        err = np.abs(yh - y_o).max()
        assert err <= TOL_REL * ymax, f"max|err| {err:.3e} > {TOL_REL * ymax:.3e}"
    else:
        # bf16 output: the rounding of a value that is itself within the FP32 tolerance
        ulp = 2.0 ** (np.floor(np.log2(np.maximum(np.abs(y_o), 1e-30))) - 7)
        assert np.all(np.abs(yh - y_o) <= ulp + TOL_REL * ymax)
    return yh, y_o
