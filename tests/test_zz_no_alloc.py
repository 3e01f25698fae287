"""zq_w4a8_linear_noalloc: the entry point for callers that cannot allocate device memory (a serving
loop with a frozen memory plan, a plug-in without an allocator) and so cannot provide a workspace.
Its split-K scratch is a fixed array inside the library.  The result must equal the regular entry
point's (and the CPU oracle's), call after call, since the shared array keeps the previous call's
contents.

Collected last on purpose: a failure here cannot hide a failure of any other test in a run that stops
at the first one.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2307_09782_b200 import binding, synth
from gpu_util import TOL_REL, host, to_bf16, up

pytestmark = pytest.mark.gpu


def _inputs(seed, M, N, K, r):
    x_bits = synth.make_x(seed, M, K, max(1, K // 100), 20.0)
    W = synth.make_w(seed, N, K, 0.02)
    U, V = synth.make_lorc(seed, N, K, r)
    return x_bits, W, U, V


def _case(seed, M, N, K, r, mode):
    x_bits, W, U, V = _inputs(seed, M, N, K, r)
    q, sx, t = binding.quantize_act_fp8(to_bf16(x_bits), up(V))
    return q, sx, t, up(U), binding.pack_weight_fp4(up(W), 128, mode)


def _oracle_y(seed, M, N, K, r, mode):
    x_bits, W, U, V = _inputs(seed, M, N, K, r)
    q, sx, t = oracle.quantize_act_fp8(x_bits, V)
    c, sh, sc = oracle.pack_weight_fp4(W, 128, mode)
    return oracle.w4a8_linear(q, sx, c, sh, sc, 128, mode, U, t)


def test_noalloc_matches_workspace_entry_point_twice_in_a_row():
    # a split-K shape (few output tiles, long K): the scratch array is really used
    M, N, K, r, mode = 16, 256, 8192, 8, "M2"
    q, sx, t, U, pw = _case(201, M, N, K, r, mode)
    ws = binding.make_workspace(binding.linear_workspace_bytes(M, N, K, r))
    y_ref = binding.w4a8_linear(pw, q=q, sx=sx, t=t, U=U, workspace=ws)
    assert binding.device_status(ws) == (0, 0)
    ref = host(y_ref).astype(np.float64)
    tol = TOL_REL * np.abs(ref).max()
    y_o = _oracle_y(201, M, N, K, r, mode)
    for _ in range(2):
        y = binding.w4a8_linear_noalloc(pw, q=q, sx=sx, t=t, U=U)
        assert binding.noalloc_status() == (0, 0)
        assert np.abs(host(y).astype(np.float64) - ref).max() <= tol
        assert np.abs(host(y).astype(np.float64) - y_o).max() <= TOL_REL * np.abs(y_o).max()
    # a different problem right after (other tile shape, mode none, no split) reuses the same array
    M2, N2, K2 = 200, 384, 512
    q2, sx2, t2, U2, pw2 = _case(202, M2, N2, K2, r, "none")
    ws2 = binding.make_workspace(binding.linear_workspace_bytes(M2, N2, K2, r))
    ref2 = host(binding.w4a8_linear(pw2, q=q2, sx=sx2, t=t2, U=U2, workspace=ws2))
    y2_o = _oracle_y(202, M2, N2, K2, r, "none")
    for _ in range(2):
        y2 = binding.w4a8_linear_noalloc(pw2, q=q2, sx=sx2, t=t2, U=U2)
        torch.cuda.synchronize()
        assert np.abs(host(y2).astype(np.float64) - ref2).max() <= TOL_REL * np.abs(ref2).max()
        assert np.abs(host(y2).astype(np.float64) - y2_o).max() <= TOL_REL * np.abs(y2_o).max()
    # and the first problem again
    y = binding.w4a8_linear_noalloc(pw, q=q, sx=sx, t=t, U=U)
    assert binding.noalloc_status() == (0, 0)
    assert np.abs(host(y).astype(np.float64) - ref).max() <= tol
    assert np.abs(host(y).astype(np.float64) - y_o).max() <= TOL_REL * np.abs(y_o).max()


def test_noalloc_rejects_problems_beyond_the_fixed_scratch():
    limit = binding.lib().zq_w4a8_linear_noalloc_max_scratch_bytes()
    assert limit == 32 << 20
    # 256 tokens x 4096 outputs with a very long K splits into partial sums far beyond 32 MiB
    M, N, K = 256, 4096, 65536
    q = torch.zeros((M, K), dtype=torch.uint8, device="cuda")
    sx = torch.ones((M,), dtype=torch.float32, device="cuda")
    nbytes = binding.packed_weight_sizes(N, K, 128, "M1")[0]
    pw = binding.PackedWeight(torch.zeros((nbytes,), dtype=torch.uint8, device="cuda"),
                              torch.zeros((N, K // 128), dtype=torch.uint8, device="cuda"),
                              torch.ones((N,), dtype=torch.float32, device="cuda"), N, K, 128, binding.SCALE_M1)
    with pytest.raises(binding.ZqError) as e:
        binding.w4a8_linear_noalloc(pw, q=q, sx=sx)
    assert e.value.status == -5
