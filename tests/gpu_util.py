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


def untile_codes(tiles: np.ndarray, N: int, K: int, layout=binding.WEIGHTS_CAST):
    """Decodes either tiled weight format (include/zqfp.h) back to plain form:
    returns (codes uint8 [N, K/2] with element 2b in the low nibble of byte b, shifts uint8 [N, K/32])."""
    nt, kb = (N + 127) // 128, K // 128
    if layout == binding.WEIGHTS_MX_FP8:
        # a block of 128 output rows: E4M3 bytes of all K blocks (row r of a K block at r * 128), then the scales
        t = np.ascontiguousarray(tiles, dtype=np.uint8).reshape(nt, kb * 16896)
        codes = t[:, :kb * 16384].reshape(nt, kb, 128, 128).transpose(0, 2, 1, 3).reshape(nt * 128, K)
        sf = t[:, kb * 16384:].reshape(nt, kb, 32, 4, 4).transpose(0, 3, 2, 1, 4).reshape(nt * 128, kb * 4)
        assert not codes[N:].any() and np.all(sf[N:] == 127), "padding rows: zero codes, unit scales"
        return codes[:N], (127 - sf[:N].astype(np.int32)).astype(np.uint8)
    if layout == binding.WEIGHTS_MX:
        t = np.ascontiguousarray(tiles, dtype=np.uint8).reshape(nt, kb * 8704)   # a block of 128 output rows:
        codes = t[:, :kb * 8192].reshape(nt, kb, 128, 64).transpose(0, 2, 1, 3).reshape(nt * 128, K // 2)
        sf = t[:, kb * 8192:].reshape(nt, kb, 32, 4, 4)  # codes of all K blocks, then scales [kb, r % 32, r / 32, s]
        sf = sf.transpose(0, 3, 2, 1, 4).reshape(nt * 128, kb * 4)      # [n, K / 32]
        assert not codes[N:].any() and np.all(sf[N:] == 127), "padding rows: zero codes, unit scales"
        assert np.all(sf <= 127) and np.all(sf >= 122)   # shifts 0 .. 5
        return codes[:N], (127 - sf[:N]).astype(np.uint8)
    t = np.ascontiguousarray(tiles, dtype=np.uint8).reshape(nt, kb, 8448)
    words = t[:, :, :8192].copy().view(np.uint32).reshape(nt, kb, 4, 128, 4)     # [nt, kb, chunk, row, word]
    el = np.empty((nt, kb, 4, 128, 4, 8), dtype=np.uint8)                         # 4-bit codes per element
    for i in range(8):
        mag = (words >> np.uint32(4 * i)) & np.uint32(7)
        sbit = 8 * i + 7 if i < 4 else 8 * (i - 4) + 3
        sgn = (words >> np.uint32(sbit)) & np.uint32(1)
        el[..., i] = (mag | (sgn << np.uint32(3))).astype(np.uint8)
    # -> [nt, row, kb, chunk, word, i] = [n, k]
    el = el.transpose(0, 3, 1, 2, 4, 5).reshape(nt * 128, K)
    codes = (el[:, 0::2] | (el[:, 1::2] << 4)).astype(np.uint8)
    sh = t[:, :, 8192:].reshape(nt, kb, 128, 2).transpose(0, 2, 1, 3).reshape(nt * 128, kb * 2)
    assert not codes[N:].any() and not sh[N:].any(), "padding rows must be zero"
    return codes[:N], np.repeat(sh[:N], 2, axis=1)


def check_packed(pw, c_o, sh_o, sc_o, group):
    """Bit-exact comparison of a PackedWeight with the oracle's plain codes / shifts / scales."""
    codes, sh32 = untile_codes(host(pw.codes), pw.N, pw.K, pw.layout)
    assert np.array_equal(codes, c_o), "FP4 codes"
    if sh_o is not None:
        assert np.array_equal(host(pw.shift), sh_o), "shifts"
        assert np.array_equal(sh32, np.repeat(sh_o, group // 32, axis=1)), "shifts inside the tiles"
    else:
        assert not sh32.any()
    assert np.array_equal(host(pw.scale).view(np.uint32), sc_o.view(np.uint32)), "scales"


def check_linear(x_bits, W, U, V, group, mode, out_dtype=torch.float32, rows=None, fused_quant=False,
                 layout=binding.WEIGHTS_CAST):
    """Runs oracle and CUDA path on the same inputs; asserts bit-exact codes / scales and y within tolerance."""
    M, K = x_bits.shape
    N = W.shape[0]
    r = 0 if U is None else U.shape[1]
    q_o, sx_o, t_o = oracle.quantize_act_fp8(x_bits, V)
    c_o, sh_o, sc_o = oracle.pack_weight_fp4(W, group, mode)
    y_o = oracle.w4a8_linear(q_o, sx_o, c_o, sh_o, sc_o, group, mode, U, t_o, rows=rows)

    x = to_bf16(x_bits)
    Wd, Ud, Vd = up(W), up(U), up(V)
    pw = binding.pack_weight_fp4(Wd, group, mode, layout)
    check_packed(pw, c_o, sh_o, sc_o, group)
    ws = binding.make_workspace(binding.linear_workspace_bytes(M, N, K, r))
    if fused_quant:
        y = binding.w4a8_linear(pw, x=x, U=Ud, V=Vd, out_dtype=out_dtype, workspace=ws)
    else:
        q, sx, t = binding.quantize_act_fp8(x, Vd)
        assert np.array_equal(host(q), q_o), "FP8 codes"
        assert np.array_equal(host(sx).view(np.uint32), sx_o.view(np.uint32)), "token scales"
        if r:
            assert np.abs(host(t) - t_o).max() <= 1e-4 * max(np.abs(t_o).max(), 1e-30), "LoRC down-projection"
        y = binding.w4a8_linear(pw, q=q, sx=sx, t=t, U=Ud, out_dtype=out_dtype,
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
