"""GPU parity for the checkpoint-side repair: re-rounded scale bytes bit-exact against the
oracle in both layouts, and the single-scale GEMM on the repaired checkpoint close to the exact
per-segment epilogue (and far from the unrepaired defect)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2609_04098_b200 import binding as nv
from paper_2609_04098_b200 import synth
from tests import gpu_util as gu
from tests.golden.load import paper_constants

pytestmark = pytest.mark.gpu
PC = paper_constants()


def _group(seed, spec, K, ratios):
    segs = synth.make_segments(spec)
    w = synth.weights(seed, 2, segs, K)
    g0 = oracle.calibrate(w[:segs[0].count])[1]
    gs = np.array([g0 / np.float32(r) for r in ratios], np.float32)
    N = w.shape[0]
    wc, wsf = oracle.quantize(w, oracle.row_scales(N, segs, gs))
    return segs, gs, wc, wsf, N


@pytest.mark.parametrize("layout", [nv.SF_MMA, nv.SF_LINEAR])
@pytest.mark.parametrize("N_spec,K", [((("qkv", 96, 0.02), ("z", 96, 0.02)), 512),
                                       ((("b", 48, 0.2), ("a", 48, 0.2), ("c", 37, 0.02)), 1040)])
def test_scale_bytes_bit_exact(layout, N_spec, K):
    ratios = [1.0, PC["ratio_b_a"], PC["ratio_worst"]][:len(N_spec)]
    segs, gs, wc, wsf, N = _group(4, N_spec, K, ratios)
    want, gstar = oracle.harmonize_scales(wsf, oracle.row_scales(N, segs, gs))
    sf_in = gu.dev_u8(oracle.sf_to_mma(wsf, K) if layout == nv.SF_MMA else wsf.ravel())
    out, g_shared = nv.nvfp4_harmonize_scales(sf_in, N, K, segs, gu.dev_f32(gs), layout)
    torch.cuda.synchronize()
    assert g_shared.item() == gstar
    got = out.cpu().numpy()
    if layout == nv.SF_MMA:
        lin, pad_zero = oracle.sf_from_mma(got, N, K)
        assert pad_zero
    else:
        lin = got.reshape(N, K // 16)
    assert np.array_equal(lin, want)


def test_single_scale_gemm_on_the_repaired_checkpoint():
    spec = (("qkv", 256, 0.02), ("z", 256, 0.02))
    K, M = 1024, 192
    segs, gs, wc, wsf, N = _group(5, spec, K, [1.0, PC["ratio_qkv_z"]])
    x = synth.prefill_activations(5, 1, M, K)
    ac, asf, ga, _ = gu.oracle_quantized(x)
    a_codes, a_sf, g_a = gu.dev_u8(ac), gu.dev_u8(oracle.sf_to_mma(asf, K)), gu.dev_f32(ga)
    w_codes, w_sf = gu.dev_u8(wc), gu.dev_u8(oracle.sf_to_mma(wsf, K))
    ws = nv.alloc_workspace(gu.DEV)
    exact = nv.nvfp4_linear(a_codes, a_sf, g_a, w_codes, w_sf, segs, gu.dev_f32(gs), ws, out_f32=True)
    sf_h, g_shared = nv.nvfp4_harmonize_scales(w_sf, N, K, segs, gu.dev_f32(gs))
    repaired = nv.nvfp4_linear(a_codes, a_sf, g_a, w_codes, sf_h, [(0, N)], g_shared, ws, out_f32=True)
    defect = nv.nvfp4_linear(a_codes, a_sf, g_a, w_codes, w_sf, [(0, N)], g_shared, ws, out_f32=True)
    assert nv.device_status(ws) == 0
    # against the oracle's GEMM on the oracle's harmonised scales
    want_sf, gstar = oracle.harmonize_scales(wsf, oracle.row_scales(N, segs, gs))
    gcol = np.full(N, gstar, np.float32)
    gu.check_gemm(repaired, oracle.gemm(ac, asf, ga, wc, want_sf, gcol), gu.gemm_bounds(ac, asf, ga, wc, want_sf, gcol))
    e, r, d = exact.double().cpu().numpy(), repaired.double().cpu().numpy(), defect.double().cpu().numpy()
    z = slice(256, 512)
    assert np.array_equal(r[:, :256], e[:, :256])
    assert np.linalg.norm(r[:, z] - e[:, z]) / np.linalg.norm(e[:, z]) < 0.04
    assert abs(np.linalg.norm(d[:, z] - e[:, z]) / np.linalg.norm(e[:, z]) - (PC["ratio_qkv_z"] - 1.0)) < 1e-3
