"""Helpers shared by the GPU parity tests: host<->device marshalling and the
tolerance checks for GEMM outputs.  The oracle side of every comparison is
computed from the same seeded host inputs; nothing here comes from the CUDA path.
"""
import numpy as np
import torch

import oracle
from paper_2609_04098_b200 import binding as nv
from paper_2609_04098_b200 import synth

DEV = "cuda:0"


def dev_bf16(bits: np.ndarray) -> torch.Tensor:
    return synth.to_torch_bf16(bits).to(DEV)


def dev_u8(a: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.uint8)).to(DEV)


def dev_f32(a) -> torch.Tensor:
    return torch.from_numpy(np.atleast_1d(np.asarray(a, dtype=np.float32))).to(DEV)


def host_bits(t: torch.Tensor) -> np.ndarray:
    """bf16 device tensor -> uint16 bit patterns on the host."""
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16)


def oracle_quantized(x_bits, g=None, segments=None, g_seg=None):
    """Oracle (codes, linear scales, row scales) for an activation (g) or weight (segments)."""
    R = x_bits.shape[0]
    if segments is None:
        if g is None:
            _, g = oracle.calibrate(x_bits)
        grow = oracle.row_scales(R, g=g)
        gs = g
    else:
        if g_seg is None:
            g_seg = [oracle.calibrate(x_bits[s.begin:s.begin + s.count])[1] for s in segments]
        grow = oracle.row_scales(R, segments, g_seg)
        gs = np.asarray(g_seg, dtype=np.float32)
    codes, sf = oracle.quantize(x_bits, grow)
    return codes, sf, gs, grow


def check_quantized(codes_gpu, sf_gpu, layout, codes_ref, sf_ref, K):
    """Bit-exact comparison of packed codes and scale bytes (padding must be zero)."""
    cg = codes_gpu.cpu().numpy()
    assert cg.shape == codes_ref.shape
    bad = np.argwhere(cg != codes_ref)
    assert bad.size == 0, "codes differ at %d bytes, first %s: gpu %02x oracle %02x" % (
        len(bad), bad[0], cg[tuple(bad[0])], codes_ref[tuple(bad[0])])
    sg = sf_gpu.cpu().numpy()
    rows = codes_ref.shape[0]
    if layout == nv.SF_MMA:
        assert sg.size == oracle.sf_mma_bytes(rows, K)
        lin, pad_zero = oracle.sf_from_mma(sg, rows, K)
        assert pad_zero, "padding bytes of the scale buffer are not zero"
    else:
        lin = sg[:rows * (K // 16)].reshape(rows, K // 16)
    bad = np.argwhere(lin != sf_ref)
    assert bad.size == 0, "scale bytes differ at %d places, first %s: gpu %02x oracle %02x" % (
        len(bad), bad[0], lin[tuple(bad[0])], sf_ref[tuple(bad[0])])


def gemm_bounds(a_codes, a_sf, g_a, w_codes, w_sf, gcol, rows=None, cols=None):
    """Per-element tolerance 1e-2 * ||a_hat_m|| * ||w_hat_n|| / sqrt(K)."""
    M, K = a_codes.shape[0], a_codes.shape[1] * 2
    ri = np.arange(M) if rows is None else np.asarray(rows)
    ci = np.arange(w_codes.shape[0]) if cols is None else np.asarray(cols)
    a_hat = oracle.dequantize(a_codes[ri], a_sf[ri], oracle.row_scales(len(ri), g=g_a))
    w_hat = oracle.dequantize(w_codes[ci], w_sf[ci], gcol[ci])
    return 1e-2 * np.linalg.norm(a_hat, axis=1)[:, None] * np.linalg.norm(w_hat, axis=1)[None, :] / np.sqrt(K)


def check_gemm(y_gpu: torch.Tensor, y_ref: np.ndarray, bound: np.ndarray, what=""):
    """The GEMM bar: relative Frobenius error <= 2e-3 against the exact result and no
    element further than `bound`; for bf16 output an element may instead be within one
    bf16 ulp of the correctly rounded exact result (a large output's half-ulp can
    exceed the bound)."""
    if y_gpu.dtype == torch.bfloat16:
        yg = oracle.bf16_bits_to_f64(host_bits(y_gpu))
    else:
        yg = y_gpu.detach().cpu().numpy().astype(np.float64)
    assert yg.shape == y_ref.shape
    assert np.all(np.isfinite(yg)), what
    nrm = np.linalg.norm(y_ref)
    rel = np.linalg.norm(yg - y_ref) / nrm if nrm > 0 else np.linalg.norm(yg)
    assert rel <= 2e-3, "%s relative Frobenius error %.3e" % (what, rel)
    err = np.abs(yg - y_ref)
    over = err > bound
    if y_gpu.dtype == torch.bfloat16 and over.any():
        ref_b = oracle.f64_to_bf16_bits(y_ref)
        ref_v = oracle.bf16_bits_to_f64(ref_b)
        ulp = np.abs(oracle.bf16_bits_to_f64((ref_b & np.uint16(0x7FFF)) + np.uint16(1)) -
                     oracle.bf16_bits_to_f64(ref_b & np.uint16(0x7FFF)))
        over &= np.abs(yg - ref_v) > ulp
    assert not over.any(), "%s %d elements outside the bound (worst %.3e x bound)" % (
        what, int(over.sum()), float((err / np.maximum(bound, 1e-300)).max()))
    return rel


def check_bf16_close_to_definition(got_bits: np.ndarray, want_bits: np.ndarray, min_equal=0.995, what=""):
    """A bf16 tensor formed on the device in binary32 against the same tensor from the float64
    definition rounded once: never more than one bf16 ulp apart (with an absolute floor of 2^-100:
    below it the device may return a zero), and equal (up to the sign of a zero) for at least
    `min_equal` of the elements."""
    assert got_bits.shape == want_bits.shape, what
    gv, wv = oracle.bf16_bits_to_f64(got_bits), oracle.bf16_bits_to_f64(want_bits)
    assert np.all(np.isfinite(gv)), what
    mag = want_bits & np.uint16(0x7FFF)
    ulp = np.abs(oracle.bf16_bits_to_f64(mag + np.uint16(1)) - oracle.bf16_bits_to_f64(mag))
    far = np.abs(gv - wv) > np.maximum(ulp, 2.0 ** -100)
    assert not far.any(), "%s: %d elements more than one bf16 ulp from the definition" % (what, int(far.sum()))
    same = float(((gv == wv) | ((np.abs(gv) < 2.0 ** -100) & (np.abs(wv) < 2.0 ** -100))).mean()) if gv.size else 1.0
    assert same >= min_equal, "%s: only %.4f of the elements equal the rounded definition" % (what, same)
    return same
