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
    assert L.zq_pack_weight_fp4(fake, 4, 256, 128, 1, 2, fake, fake, fake, null) == -4   # unknown layout
    assert L.zq_pack_weight_fp4(fake, 4, 256, 128, 0, 1, fake, fake, fake, null) == -4   # block scales need M1 / M2
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
    assert call(layout=1, mode=0) == -4
    assert call(layout=3) == -4
    assert call(ws=null) == -5
    assert call(wsb=1024) == -5
    assert call(M=0) == 0
    assert L.zq_workspace_init(null, 1 << 20, null) == -1
    assert L.zq_workspace_init(fake, 16, null) == -5
