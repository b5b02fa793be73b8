"""Pins for the checkpoint-side repair (shared global scale, ratio folded into the E4M3 block
scales): identities, the re-rounding bound the paper states, a library cast, and its effect on
the GEMM compared with the exact per-segment epilogue."""
import numpy as np
import torch

import oracle
from paper_2609_04098_b200 import synth
from tests.golden.load import paper_constants

PC = paper_constants()


def _weights(seed, spec, K):
    segs = synth.make_segments(spec)
    w = synth.weights(seed, 2, segs, K)
    gs = np.array([oracle.calibrate(w[s.begin:s.begin + s.count])[1] for s in segs], np.float32)
    N = w.shape[0]
    wc, wsf = oracle.quantize(w, oracle.row_scales(N, segs, gs))
    return segs, gs, wc, wsf


def test_equal_scales_change_nothing_and_power_of_two_ratios_are_exact_shifts():
    segs, gs, wc, wsf = _weights(0, (("a", 16, 0.02), ("b", 16, 0.02)), 256)
    g_same = np.full(32, gs[0], np.float32)
    out, gstar = oracle.harmonize_scales(wsf, g_same)
    assert gstar == gs[0] and np.array_equal(out, wsf)
    # second module's scale = first / 4: its bytes move down two binades (exponent field - 2)
    g_row = np.concatenate([np.full(16, gs[0]), np.full(16, gs[0] / 4)]).astype(np.float32)
    out, gstar = oracle.harmonize_scales(wsf, g_row)
    assert gstar == gs[0]
    assert np.array_equal(out[:16], wsf[:16])
    big = wsf[16:] >= 0x18                       # stays normal after two binades down
    assert np.array_equal(out[16:][big], wsf[16:][big] - 0x10)


def test_matches_library_cast_of_the_product():
    segs, gs, wc, wsf = _weights(1, (("qkv", 24, 0.02), ("z", 24, 0.02)), 512)
    g_row = oracle.row_scales(48, segs, [gs[0], np.float32(gs[0] / PC["ratio_qkv_z"])])
    out, gstar = oracle.harmonize_scales(wsf, g_row)
    dec = torch.from_numpy(wsf.copy()).view(torch.float8_e4m3fn).to(torch.float32).numpy()
    ratio = (g_row / gstar).astype(np.float32)[:, None]
    ref = torch.from_numpy((dec * ratio).astype(np.float32)).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    assert np.array_equal(out, ref)


def test_rerounding_error_is_within_the_papers_bound():
    # "re-rounding error <= 6.2 % on affected local scales": half an ulp of a 3-bit mantissa
    worst = []
    for ratio in (PC["ratio_qkv_z"], PC["ratio_b_a"], PC["ratio_worst"]):
        segs, gs, wc, wsf = _weights(2, (("m0", 32, 0.02), ("m1", 32, 0.02)), 512)
        g_row = oracle.row_scales(64, segs, [gs[0], np.float32(gs[0] / ratio)])
        out, gstar = oracle.harmonize_scales(wsf, g_row)
        dec_in = np.array([[oracle.e4m3_decode(b) for b in row] for row in wsf[32:]], np.float64)
        dec_out = np.array([[oracle.e4m3_decode(b) for b in row] for row in out[32:]], np.float64)
        want = dec_in * float(g_row[32]) / float(gstar)               # what the new scale should represent
        ok = dec_out >= 2.0 ** -6                                     # normal results
        rel = np.abs(dec_out[ok] - want[ok]) / dec_out[ok]
        assert rel.max() <= 2.0 ** -4 + 1e-7
        worst.append(rel.max())
    assert max(worst) > 0.03                       # the re-rounding is real (a fixed ratio meets only 8 mantissas)
    assert abs(2.0 ** -4 - PC["rerounding_error_max"]) < 1e-3


def test_gemm_after_harmonisation_is_close_to_the_exact_repair_and_far_from_the_defect():
    spec = (("qkv", 64, 0.02), ("z", 64, 0.02))
    segs, gs, wc, wsf = _weights(3, spec, 512)
    gs = np.array([gs[0], gs[0] / np.float32(PC["ratio_qkv_z"])], np.float32)     # the paper's qkv/z ratio
    x = synth.prefill_activations(3, 1, 32, 512)
    _, ga = oracle.calibrate(x)
    ac, asf = oracle.quantize(x, oracle.row_scales(32, g=ga))
    exact = oracle.gemm(ac, asf, ga, wc, wsf, oracle.col_scales(128, segs, gs))           # per-segment epilogue
    out, gstar = oracle.harmonize_scales(wsf, oracle.row_scales(128, segs, gs))
    shared = oracle.gemm(ac, asf, ga, wc, out, np.full(128, gstar, np.float32))           # repaired checkpoint
    defect = oracle.gemm(ac, asf, ga, wc, wsf, np.full(128, gstar, np.float32))           # max scale, scales untouched
    z = slice(64, 128)
    err_repair = np.linalg.norm(shared[:, z] - exact[:, z]) / np.linalg.norm(exact[:, z])
    err_defect = np.linalg.norm(defect[:, z] - exact[:, z]) / np.linalg.norm(exact[:, z])
    assert np.array_equal(shared[:, :64], exact[:, :64])              # the module that owns g* is untouched
    assert err_repair < 0.04                                          # re-rounded scales: a few per cent at most
    assert abs(err_defect - (PC["ratio_qkv_z"] - 1.0)) < 1e-3          # the defect: off by the ratio
