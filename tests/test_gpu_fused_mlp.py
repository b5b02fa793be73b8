"""GPU parity of the MLP's fused gate/up projection: SwiGLU and the quantization of the down
projection's input inside the GEMM epilogue (``nvfp4_linear_swiglu``), through the C ABI.

Every link is checked against the oracle on its own:
  weights   codes and scale bytes of the interleaved layout = the oracle's, rows permuted (bit-exact);
  link 1    gate/up as the epilogue rounds them to bf16 (testing output) vs the oracle's exact GEMM,
            within the GEMM tolerance;
  link 2    h the epilogue forms (testing output) vs the float64 definition of silu(gate) * up applied to
            those gate/up values, rounded once: at most one bf16 ulp apart, equal almost everywhere;
  link 3    codes and scale bytes of h bit-exact vs the oracle's quantization of that h.
The fused call must also equal the two-kernel path (GEMM, then nvfp4_swiglu_quantize) bit for bit.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2609_04098_b200 import binding as nv
from paper_2609_04098_b200 import synth
from tests import gpu_util as gu

pytestmark = pytest.mark.gpu


@pytest.fixture(autouse=True)
def _auto_variant():
    yield
    nv.set_gemm_variant(0)


def il_rows(inner):
    """Interleaved row order: position p holds original row il[p] of [gate rows | up rows]."""
    p = np.arange(2 * inner)
    b, r = p // 32, p % 32
    return np.where(r < 16, b * 16 + r, inner + b * 16 + (r - 16))


def _operands(seed, M, inner, K):
    segs = synth.make_segments((("gate", inner, 0.02), ("up", inner, 0.03)))
    x = synth.prefill_activations(seed, 901, M, K)
    w = synth.weights(seed, 902, segs, K)
    ac, asf, ga, _ = gu.oracle_quantized(x)
    wc, wsf, gs, _ = gu.oracle_quantized(w, segments=segs)
    return segs, x, w, ac, asf, ga, wc, wsf, gs


def _check_fused(seed, M, inner, K, rows=None):
    segs, x, w, ac, asf, ga, wc, wsf, gs = _operands(seed, M, inner, K)
    il = il_rows(inner)
    # weights: interleaved layout on the device = the oracle's rows, permuted
    w_codes, w_sf, g_gu = nv.nvfp4_quantize_weight_gate_up(gu.dev_bf16(w))
    torch.cuda.synchronize()
    assert np.array_equal(g_gu.cpu().numpy(), gs)
    gu.check_quantized(w_codes, w_sf, nv.SF_MMA, wc[il], wsf[il], K)
    # the fused call on the oracle's activation codes
    a_codes, a_sf, g_a = gu.dev_u8(ac), gu.dev_u8(oracle.sf_to_mma(asf, K)), gu.dev_f32(ga)
    ws = nv.alloc_workspace(gu.DEV)
    # static scale of h: from the oracle's own chain on a few rows, with head-room
    probe = np.arange(min(M, 32))
    y_probe = oracle.gemm(ac, asf, ga, wc, wsf, oracle.col_scales(2 * inner, segs, gs), rows=probe)
    _, gh = oracle.calibrate(oracle.swiglu_bf16(oracle.f64_to_bf16_bits(y_probe)))
    gh = np.float32(gh * 2.0)
    g_h = gu.dev_f32(gh)
    dbg_y = torch.empty((M, 2 * inner), dtype=torch.bfloat16, device=gu.DEV)
    dbg_h = torch.empty((M, inner), dtype=torch.bfloat16, device=gu.DEV)
    h_codes, h_sf = nv.nvfp4_linear_swiglu(a_codes, a_sf, g_a, w_codes, w_sf, g_gu, g_h, ws, dbg_y=dbg_y, dbg_h=dbg_h)
    assert nv.device_status(ws) == 0
    # without the testing outputs: same codes and scales
    h_codes2, h_sf2 = nv.nvfp4_linear_swiglu(a_codes, a_sf, g_a, w_codes, w_sf, g_gu, g_h, ws)
    assert nv.device_status(ws) == 0
    assert torch.equal(h_codes, h_codes2) and torch.equal(h_sf, h_sf2)
    ri = np.arange(M) if rows is None else rows
    rt = torch.from_numpy(ri).to(gu.DEV)
    inv = np.argsort(il)                                   # original column -> interleaved position
    y_il = dbg_y[rt].contiguous()
    y_rows = y_il[:, torch.from_numpy(inv).to(gu.DEV)].contiguous()          # gate | up in original order
    # link 1
    gcol = oracle.col_scales(2 * inner, segs, gs)
    y_ref = oracle.gemm(ac, asf, ga, wc, wsf, gcol, rows=ri)
    gu.check_gemm(y_rows, y_ref, gu.gemm_bounds(ac, asf, ga, wc, wsf, gcol, rows=ri), "gate/up")
    # link 2
    h_def = oracle.swiglu_bf16(gu.host_bits(y_rows))
    h_gpu = gu.host_bits(dbg_h[rt].contiguous())
    gu.check_bf16_close_to_definition(h_gpu, h_def, 0.995, "h")
    # link 3
    hc, hsf = oracle.quantize(h_gpu, oracle.row_scales(len(ri), g=gh))
    if rows is None:
        gu.check_quantized(h_codes, h_sf, nv.SF_MMA, hc, hsf, inner)
    else:
        sf_lin, pad_zero = oracle.sf_from_mma(h_sf.cpu().numpy(), M, inner)
        assert pad_zero
        assert np.array_equal(h_codes[rt].cpu().numpy(), hc) and np.array_equal(sf_lin[ri], hsf)
    # the two-kernel path on the plain (not interleaved) weights gives the same bytes
    w_codes_p, w_sf_p, g_p = nv.nvfp4_quantize_weight(gu.dev_bf16(w), segs)
    y_plain = nv.nvfp4_linear(a_codes, a_sf, g_a, w_codes_p, w_sf_p, segs, g_p, ws)
    c2, s2 = nv.nvfp4_swiglu_quantize(y_plain, g_h)
    assert nv.device_status(ws) == 0
    assert torch.equal(c2, h_codes) and torch.equal(s2, h_sf)
    return h_codes, h_sf


@pytest.mark.parametrize("variant", [256, 2, 0])
@pytest.mark.parametrize("M,inner,K", [(130, 128, 512), (1, 64, 64), (257, 320, 320), (200, 448, 1088), (384, 1024, 256)])
def test_fused_swiglu_epilogue_small_shapes(variant, M, inner, K):
    nv.set_gemm_variant(variant)
    _check_fused(3, M, inner, K)


def test_fused_swiglu_epilogue_full_size_mlp():
    # configs[2]: M = 8192, K = 5120, inner = 17408; oracle links on one row in every 128-row band
    M, inner, K = 8192, synth.MLP_INNER, synth.HIDDEN
    rng = np.random.default_rng(9)
    rows = np.unique(np.array([t * 128 + rng.integers(0, 128) for t in range(M // 128)] + [0, M - 1]))
    _check_fused(4, M, inner, K, rows=rows)
