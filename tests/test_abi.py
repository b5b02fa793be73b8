"""The C-ABI library: it loads without a GPU, exports every symbol the header
declares, and rejects host-detectable misuse before touching the device."""
import ctypes
import os
import re

import pytest

from paper_2609_04098_b200 import binding as nv
from paper_2609_04098_b200 import build as nvbuild

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def L():
    nvbuild.build()
    return nv.lib()


def _declared():
    text = open(os.path.join(ROOT, "include", "nvfp4.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(nvfp4_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(L):
    names = _declared()
    assert set(names) == set(nv.EXPORTS)
    for n in names:
        assert getattr(L, n) is not None


def test_sf_bytes_and_strings(L):
    assert nv.sf_bytes(128, 64, nv.SF_MMA) == 512
    assert nv.sf_bytes(1, 16, nv.SF_MMA) == 512
    assert nv.sf_bytes(129, 5120, nv.SF_MMA) == 2 * 80 * 512
    assert nv.sf_bytes(8192, 5120, nv.SF_MMA) == 8192 * 320
    assert nv.sf_bytes(7, 48, nv.SF_LINEAR) == 21
    assert nv.sf_bytes(7, 40, nv.SF_LINEAR) == 0          # K not a multiple of 16
    assert nv.status_string(0) == "ok"
    assert "segment" in nv.status_string(4)
    assert b"128" in L.nvfp4_gemm_variants()
    assert L.nvfp4_launch_count() == 0 or L.nvfp4_launch_count() > 0


def test_host_side_argument_checks_need_no_gpu(L):
    vp = ctypes.c_void_p
    p = vp(0x1000)                 # never dereferenced: every call below fails its checks first
    seg = (nv._Segment * 2)()
    seg[0].col_begin, seg[0].col_count = 0, 8
    seg[1].col_begin, seg[1].col_count = 8, 8
    assert L.nvfp4_calibrate(None, 4, 16, 16, p, None, None) == 1
    assert L.nvfp4_calibrate(p, 4, 16, 8, p, None, None) == 2                      # ld < cols
    assert L.nvfp4_quantize_act(p, 4, 24, 24, p, p, p, nv.SF_MMA, None) == 2      # K % 16
    assert L.nvfp4_quantize_act(None, 4, 32, 32, p, p, p, nv.SF_MMA, None) == 1
    assert L.nvfp4_quantize_act(p, 4, 32, 40, p, p, p, nv.SF_MMA, None) == 3      # ld % 16
    assert L.nvfp4_quantize_act(vp(0x1010), 4, 32, 32, p, p, p, nv.SF_MMA, None) == 3   # 16- but not 32-byte aligned
    assert L.nvfp4_quantize_act(p, 4, 32, 32, p, p, p, 7, None) == 9
    assert L.nvfp4_quantize_weight(p, 16, 32, 32, seg, 2, p, 0, p, p, nv.SF_MMA, None) != 4
    seg[1].col_begin = 9
    assert L.nvfp4_quantize_weight(p, 16, 32, 32, seg, 2, p, 0, p, p, nv.SF_MMA, None) == 4
    seg[1].col_begin = 8
    assert L.nvfp4_quantize_weight(p, 17, 32, 32, seg, 2, p, 0, p, p, nv.SF_MMA, None) == 4
    assert L.nvfp4_quantize_weight(p, 16, 32, 32, seg, 0, p, 0, p, p, nv.SF_MMA, None) == 4
    lin = lambda **kw: L.nvfp4_linear(kw.get("a", p), p, p, kw.get("M", 8), kw.get("K", 64), p, p, kw.get("N", 16),
                                      kw.get("segs", seg), p, kw.get("nseg", 2), p, kw.get("ldy", 16),
                                      kw.get("flags", 0), kw.get("ws", p), kw.get("wsb", 256), None)
    assert lin(a=None) == 1
    assert lin(K=48) == 2
    assert lin(ldy=8) == 2
    assert lin(N=24, ldy=32) == 4
    assert lin(ws=None) == 5
    assert lin(wsb=8) == 5
    assert lin(a=vp(0x1004)) == 3
    assert lin(flags=8) == 2 and lin(flags=14) == 2
    assert L.nvfp4_workspace_reset(None, 256, None) == 1
    assert L.nvfp4_workspace_reset(p, 8, None) == 5
    assert L.nvfp4_device_status(None, None) == 1
    assert L.nvfp4_set_gemm_variant(3) == 2 and L.nvfp4_set_gemm_variant(0) == 0
    assert L.nvfp4_linear_workspace_bytes(8, 16, 64, 2) >= 4
    assert L.nvfp4_linear_bf16_workspace_bytes(8, 16, 64, 2) >= 256 + nv.SPLIT_RESERVE_BYTES + 128 * 32 + 512
    assert L.nvfp4_linear_workspace_bytes(16, 6144, 8192, 1) <= 256 + nv.SPLIT_RESERVE_BYTES
    # the fused entry points check every argument before anything is enqueued
    fused = lambda **kw: L.nvfp4_linear_bf16(kw.get("x", p), kw.get("ldx", 64), p, kw.get("M", 8), kw.get("K", 64), p, p,
                                             kw.get("N", 16), kw.get("segs", seg), p, kw.get("nseg", 2), p,
                                             kw.get("ldy", 16), kw.get("flags", 0), kw.get("ws", p),
                                             kw.get("wsb", 1 << 24), None)
    assert fused(x=None) == 1
    assert fused(K=48) == 2
    assert fused(ldx=32) == 2
    assert fused(ldy=8) == 2
    assert fused(flags=8) == 2
    assert fused(N=24, ldy=32) == 4
    assert fused(ws=None) == 5
    assert fused(wsb=4096) == 5
    assert fused(x=vp(0x1010)) == 3
    assert fused(M=1, x=None) == 1 and fused(M=1, N=24, ldy=32) == 4        # the single-token route checks the same
    static = lambda **kw: L.nvfp4_linear_bf16_static(p, 64, p, kw.get("M", 8), kw.get("K", 64), p, p, 16, seg, p, 2, p, 16,
                                                     0, None)
    assert static(K=48) == 2 and static(M=-1) == 2
    assert static(M=4096, K=5120) == 5                                       # beyond the fixed array
    assert nv.STATIC_SCRATCH_BYTES == 12 * 1024 * 1024
