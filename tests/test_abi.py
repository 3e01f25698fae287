"""The C-ABI library: it loads without a GPU, exports every symbol the header declares, and its
host-side validation returns the documented error codes before anything is launched."""
import ctypes as C
import os
import re

import pytest

import __graft_entry__ as entry
from paper_2307_09782_b200 import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def L():
    entry.build()
    return binding.lib()


def test_exports_match_header(L):
    text = open(os.path.join(ROOT, "include", "zqfp.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    declared = set(re.findall(r"\b(zq_[a-z0-9_]+)\s*\(", text))
    assert declared == set(binding.EXPORTS)
    for name in declared:
        assert hasattr(L, name), name


def test_status_strings(L):
    assert binding.status_string(0) == "ok"
    for code in range(-8, 0):
        assert binding.status_string(code) not in ("ok", "unknown status")


def test_size_queries(L):
    assert binding.packed_weight_sizes(768, 768, 128, "none") == (6 * 6 * 8448, 0, 768 * 6 * 4)
    assert binding.packed_weight_sizes(768, 768, 128, "M2") == (6 * 6 * 8448, 768 * 6, 768 * 4)
    assert binding.packed_weight_sizes(129, 256, 64, "M1") == (2 * 2 * 8448, 129 * 4, 129 * 4)
    assert binding.packed_weight_sizes(129, 256, 64, "M1", "mx") == (2 * 2 * 8704, 129 * 4, 129 * 4)
    assert binding.packed_weight_sizes(129, 256, 64, "M1", "mx_fp8") == (2 * 2 * 16896, 129 * 4, 129 * 4)
    assert binding.packed_weight_sizes(129, 256, 64, "M2", "cast_e5m2") == (2 * 2 * 8448, 129 * 4, 129 * 4)
    assert binding.packed_weight_sizes(8, 640, 320, "M2") == (5 * 8448, 8 * 2, 8 * 4)
    with pytest.raises(binding.ZqError) as e:
        binding.packed_weight_sizes(8, 100, 128, "M1")
    assert e.value.status == -2
    with pytest.raises(binding.ZqError) as e:
        binding.packed_weight_sizes(8, 128, 128, 7)
    assert e.value.status == -4
    small = binding.linear_workspace_bytes(16, 768, 768, 0)
    assert small >= 256 + 4 * 16384
    assert binding.linear_workspace_bytes(8192, 28672, 7168, 8) >= 8192 * 7168
    assert binding.linear_host_workspace_bytes(16, 768, 768, 0) >= small + 16 * 768 * 2 + 16 * 768 * 4
    # sizes the linear entry points refuse give 0, and degenerate ones do not crash the host process
    for fn in (binding.linear_workspace_bytes, binding.linear_host_workspace_bytes):
        assert fn(16, 128, 64, 0) == 0       # K below one 128-element block
        assert fn(16, 128, 192, 0) == 0      # K not a multiple of 128
        assert fn(16, 128, 256, 12) == 0     # rank not a multiple of 8
        assert fn(-1, 128, 256, 0) == 0
        assert fn(16, 0, 128, 0) >= 256 + 4 * 16384    # N == 0 is a no-op of the linear call: head only
        assert fn(0, 128, 128, 0) >= 256 + 4 * 16384


def test_workspace_serves_every_smaller_token_count(L):
    # a workspace sized for M tokens must hold the split-K scratch of every plan up to M tokens
    for (N, K) in [(7552, 1024), (7168, 28672), (2048, 8192), (640, 4096)]:
        big = binding.linear_workspace_bytes(8192, N, K, 8)
        for M in [1, 16, 17, 100, 128, 129, 192, 193, 256, 257, 448, 449, 1280, 1281, 2047, 4097, 8191]:
            assert binding.linear_workspace_bytes(M, N, K, 8) <= big, (N, K, M)
            for mode, layout in (("none", "cast"), ("M1", "cast"), ("M1", "mx")):
                pl = binding.linear_plan(M, N, K, mode, layout)
                # head + partial sums + q + sx + t for M tokens fit the 8192-token workspace
                need = 256 + 4 * 16384 + 4 * pl["partial_floats"] + M * K + 4 * M + 32 * M
                assert need <= big, (N, K, M, mode, layout)


def test_validation_before_launch(L):
    null = C.c_void_p(None)
    fake = C.c_void_p(0x1000)  # never dereferenced: validation fails first
    # quantizer
    assert L.zq_quantize_act_fp8(null, 4, 64, 64, fake, fake, null, 0, null, null) == -1
    assert L.zq_quantize_act_fp8(fake, 4, 60, 64, fake, fake, null, 0, null, null) == -2
    assert L.zq_quantize_act_fp8(fake, 4, 64, 32, fake, fake, null, 0, null, null) == -2
    assert L.zq_quantize_act_fp8(C.c_void_p(0x1004), 4, 64, 64, fake, fake, null, 0, null, null) == -3
    assert L.zq_quantize_act_fp8(fake, 4, 64, 64, fake, fake, fake, 65, fake, null) == -2
    assert L.zq_quantize_act_fp8(fake, 0, 64, 64, fake, fake, null, 0, null, null) == 0
    # packer
    assert L.zq_pack_weight_fp4(fake, 4, 256, 100, 1, 0, fake, fake, fake, null) == -2
    assert L.zq_pack_weight_fp4(fake, 4, 256, 128, 3, 0, fake, fake, fake, null) == -4
    assert L.zq_pack_weight_fp4(fake, 4, 256, 128, 1, 4, fake, fake, fake, null) == -4   # unknown layout
    assert L.zq_pack_weight_fp4(fake, 4, 256, 128, 0, 2, fake, fake, fake, null) == -4   # FP8 codes need M1 / M2
    assert L.zq_pack_weight_fp4(fake, 4, 256, 128, 0, 3, fake, fake, fake, null) == -4   # so does the E5M2 target
    assert L.zq_pack_weight_fp4(fake, 4, 640, 320, 0, 0, fake, fake, fake, null) == -2   # groups of 320: M1 / M2 only
    assert L.zq_pack_weight_fp4(fake, 4, 256, 128, 1, 0, fake, null, fake, null) == -1
    assert L.zq_pack_weight_fp4(fake, 0, 256, 128, 1, 1, fake, fake, fake, null) == 0
    # linear
    args = dict(q=fake, sx=fake, x=null, ldx=0, M=4, N=128, K=256, group=128, mode=1, layout=0, codes=fake, shift=fake,
                scale=fake, U=null, V=null, t=null, r=0, y=fake, ydt=0, ldy=128, ws=fake, wsb=1 << 30, st=null)

    def call(**kw):
        a = dict(args, **kw)
        return L.zq_w4a8_linear(a["q"], a["sx"], a["x"], a["ldx"], a["M"], a["N"], a["K"], a["group"], a["mode"],
                                a["layout"], a["codes"], a["shift"], a["scale"], a["U"], a["V"], a["t"], a["r"], a["y"], a["ydt"],
                                a["ldy"], a["ws"], a["wsb"], a["st"])

    assert call(K=192) == -2
    assert call(group=96) == -2
    assert call(r=12, U=fake, t=fake) == -2
    assert call(mode=5) == -4
    assert call(ydt=2) == -4
    assert call(codes=null) == -1
    assert call(q=null) == -1
    assert call(r=8, U=fake) == -1          # t missing
    assert call(ldy=64) == -2
    assert call(codes=C.c_void_p(0x1008)) == -3
    assert call(layout=1, codes=C.c_void_p(0x1010)) == -3   # the 4-bit tensor map wants 32-byte alignment
    assert call(layout=2, mode=0) == -4
    assert call(layout=4) == -4
    assert call(ws=null) == -5
    assert call(wsb=1024) == -5
    assert call(M=0) == 0
    assert call(N=0, ldy=0) == 0
    # the host-buffer entry point validates the same way
    def host_call(**kw):
        a = dict(args, **kw)
        return L.zq_w4a8_linear_host(fake, a["M"], a["N"], a["K"], a["group"], a["mode"], a["layout"], a["codes"],
                                     a["shift"], a["scale"], a["U"], a["V"], a["r"], fake, a["ws"], a["wsb"], a["st"])
    assert host_call(K=64) == -2
    assert host_call(N=0) == 0
    assert host_call(group=96) == -2
    assert host_call(mode=9) == -4
    assert host_call(ws=null) == -5
    assert L.zq_workspace_init(null, 1 << 20, null) == -1
    assert L.zq_workspace_init(fake, 16, null) == -5
