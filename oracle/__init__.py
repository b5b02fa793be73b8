"""CPU oracle for the NVFP4 W4A4 linear layer -- TEST INFRASTRUCTURE ONLY.

A thin numpy/ctypes front for ``nvfp4_oracle.c`` (plain C, compiled with
``gcc -O2 -ffp-contract=off -fopenmp``).  It is imported by ``tests/``, by the
smoke check and by the benchmark's CPU-baseline leg, and by nothing else: the
CUDA library and its Python binding never import it, and it never imports them.

Every function follows the paper's definition of NVFP4 (Background, "NVFP4")
and of the per-module global scales that meet in one fused GEMM (Section 6,
"Per-module calibration vs. fused-GEMM scaling"); the C file states the
operation order that the bit-exact comparison relies on.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "nvfp4_oracle.c")
_LIB = os.path.join(_HERE, "libnvfp4_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the C oracle next to its source (no-op when up to date)."""
    if (not force and os.path.exists(_LIB)
            and os.path.getmtime(_LIB) >= os.path.getmtime(_SRC)):
        return _LIB
    tmp = _LIB + ".tmp%d" % os.getpid()
    cmd = ["gcc", "-O2", "-ffp-contract=off", "-fno-fast-math", "-fopenmp", "-shared", "-fPIC",
           "-o", tmp, _SRC, "-lm"]
    subprocess.run(cmd, check=True)
    os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is not None:
        return _lib
    build()
    L = ctypes.CDLL(_LIB)
    i64, u8p, u16p, f32p, f64p, i64p = (ctypes.c_int64, ctypes.c_void_p, ctypes.c_void_p,
                                       ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p)
    L.orc_f64_to_bf16.restype = ctypes.c_uint16
    L.orc_f64_to_bf16.argtypes = [ctypes.c_double]
    L.orc_f64_to_bf16_n.restype = None
    L.orc_f64_to_bf16_n.argtypes = [f64p, i64, u16p]
    L.orc_e2m1_decode.restype = ctypes.c_float
    L.orc_e2m1_decode.argtypes = [ctypes.c_uint8]
    L.orc_e2m1_encode.restype = ctypes.c_uint8
    L.orc_e2m1_encode.argtypes = [ctypes.c_float]
    L.orc_e4m3_decode.restype = ctypes.c_float
    L.orc_e4m3_decode.argtypes = [ctypes.c_uint8]
    L.orc_e4m3_encode.restype = ctypes.c_uint8
    L.orc_e4m3_encode.argtypes = [ctypes.c_float]
    L.orc_calibrate.restype = None
    L.orc_calibrate.argtypes = [u16p, i64, i64, i64, f32p, f32p]
    L.orc_quantize.restype = ctypes.c_int
    L.orc_quantize.argtypes = [u16p, i64, i64, i64, f32p, u8p, u8p]
    L.orc_silu_mul.restype = ctypes.c_double
    L.orc_silu_mul.argtypes = [ctypes.c_double, ctypes.c_double]
    L.orc_swiglu_bf16.restype = None
    L.orc_swiglu_bf16.argtypes = [u16p, i64, i64, i64, u16p]
    L.orc_rmsnorm_bf16.restype = None
    L.orc_rmsnorm_bf16.argtypes = [u16p, i64, i64, i64, u16p, ctypes.c_double, u16p]
    L.orc_dequantize.restype = None
    L.orc_dequantize.argtypes = [u8p, u8p, f32p, i64, i64, f64p]
    L.orc_harmonize_scales.restype = ctypes.c_float
    L.orc_harmonize_scales.argtypes = [u8p, i64, i64, f32p, u8p]
    L.orc_stats.restype = ctypes.c_int
    L.orc_stats.argtypes = [u16p, i64, i64, i64, ctypes.c_float, f64p]
    L.orc_sf_mma_bytes.restype = i64
    L.orc_sf_mma_bytes.argtypes = [i64, i64]
    L.orc_sf_mma_index.restype = i64
    L.orc_sf_mma_index.argtypes = [i64, i64, i64]
    L.orc_sf_to_mma.restype = None
    L.orc_sf_to_mma.argtypes = [u8p, i64, i64, u8p]
    L.orc_gemm.restype = ctypes.c_int
    L.orc_gemm.argtypes = [u8p, u8p, ctypes.c_float, i64, i64, u8p, u8p, f32p, i64,
                           i64p, i64, i64p, i64, f64p]
    L.orc_num_threads.restype = ctypes.c_int
    L.orc_num_threads.argtypes = []
    _lib = L
    return L


def _p(a: np.ndarray):
    return a.ctypes.data_as(ctypes.c_void_p)


def _c(a, dtype) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=dtype)


def num_threads() -> int:
    return int(_load().orc_num_threads())


# -- element codecs ----------------------------------------------------------
def e2m1_decode(code: int) -> float:
    return float(_load().orc_e2m1_decode(int(code) & 0xF))


def e2m1_encode(y: float) -> int:
    return int(_load().orc_e2m1_encode(np.float32(y)))


def e4m3_decode(byte: int) -> float:
    return float(_load().orc_e4m3_decode(int(byte) & 0xFF))


def e4m3_encode(v: float) -> int:
    return int(_load().orc_e4m3_encode(np.float32(v)))


def f64_to_bf16_bits(y: np.ndarray) -> np.ndarray:
    L = _load()
    flat = _c(y, np.float64).ravel()
    out = np.empty(flat.size, np.uint16)
    L.orc_f64_to_bf16_n(_p(flat), flat.size, _p(out))
    return out.reshape(np.shape(y))


def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    """bf16 bit patterns -> float64 (exact)."""
    u = np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)
    return u.view(np.float32).astype(np.float64)


# -- the path ------------------------------------------------------------------
def calibrate(x_bits: np.ndarray):
    """(amax, g) with g = amax / (6*448) in binary32; all-zero tensor -> g = 1."""
    x = _c(x_bits, np.uint16)
    assert x.ndim == 2
    amax = np.zeros(1, np.float32)
    g = np.zeros(1, np.float32)
    _load().orc_calibrate(_p(x), x.shape[0], x.shape[1], x.shape[1], _p(amax), _p(g))
    return np.float32(amax[0]), np.float32(g[0])


def row_scales(rows: int, segments: Optional[Sequence] = None, g=None) -> np.ndarray:
    """Expand one scale (activations) or per-segment scales (weights) to one per row.
    ``segments`` items need ``.begin`` and ``.count``."""
    if segments is None:
        return np.full(rows, np.float32(g), dtype=np.float32)
    out = np.zeros(rows, np.float32)
    for s, gs in zip(segments, g):
        out[s.begin:s.begin + s.count] = np.float32(gs)
    return out


def quantize(x_bits: np.ndarray, g_row: np.ndarray):
    """bf16 [R, C] -> (codes u8 [R, C/2], scale bytes u8 [R, C/16] row-major)."""
    x = _c(x_bits, np.uint16)
    R, C = x.shape
    g_row = _c(g_row, np.float32)
    assert g_row.shape == (R,)
    codes = np.empty((R, C // 2), np.uint8)
    sf = np.empty((R, C // 16), np.uint8)
    rc = _load().orc_quantize(_p(x), R, C, C, _p(g_row), _p(codes), _p(sf))
    if rc != 0:
        raise ValueError("columns must be a multiple of 16")
    return codes, sf


def silu_mul(g: float, u: float) -> float:
    """silu(g) * u = g / (1 + exp(-g)) * u in double (before the bf16 rounding)."""
    return float(_load().orc_silu_mul(float(g), float(u)))


def swiglu_bf16(gate_up_bits: np.ndarray) -> np.ndarray:
    """bf16 [R, 2I] (gate | up) -> h = bf16(silu(gate) * up), bf16 bit patterns [R, I]: the
    definition evaluated in double and rounded once."""
    gu = _c(gate_up_bits, np.uint16)
    R, two_i = gu.shape
    assert two_i % 2 == 0
    h = np.empty((R, two_i // 2), np.uint16)
    _load().orc_swiglu_bf16(_p(gu), R, two_i // 2, two_i, _p(h))
    return h


def rmsnorm_bf16(x_bits: np.ndarray, w_bits: np.ndarray, eps: float) -> np.ndarray:
    """bf16 [R, C], weight bf16 [C] -> bf16( x / sqrt(mean(x^2) + eps) * w ), bit patterns [R, C]."""
    x = _c(x_bits, np.uint16)
    w = _c(w_bits, np.uint16)
    R, C = x.shape
    assert w.shape == (C,)
    y = np.empty((R, C), np.uint16)
    _load().orc_rmsnorm_bf16(_p(x), R, C, C, _p(w), ctypes.c_double(float(np.float32(eps))), _p(y))
    return y


def dequantize(codes: np.ndarray, sf: np.ndarray, g_row: np.ndarray) -> np.ndarray:
    codes = _c(codes, np.uint8)
    sf = _c(sf, np.uint8)
    R, C = codes.shape[0], codes.shape[1] * 2
    out = np.empty((R, C), np.float64)
    _load().orc_dequantize(_p(codes), _p(sf), _p(_c(g_row, np.float32)), R, C, _p(out))
    return out


def harmonize_scales(sf_linear: np.ndarray, g_row: np.ndarray):
    """Shared global scale for a fused group: returns (re-rounded scale bytes, g* = max g)."""
    sf = _c(sf_linear, np.uint8)
    g_row = _c(g_row, np.float32)
    out = np.empty_like(sf)
    gstar = _load().orc_harmonize_scales(_p(sf), sf.shape[0], sf.shape[1], _p(g_row), _p(out))
    return out, np.float32(gstar)


def derive_stats(raw, n_elements: int) -> dict:
    """{sum x^2, sum x^4, sum err^2, amax, blocks, 1-hot blocks} -> the table's columns."""
    s2, s4, se, amax, nb, hot = [float(v) for v in raw]
    rms = (s2 / n_elements) ** 0.5 if n_elements else 0.0
    return {"max_over_rms": amax / rms if rms > 0 else 0.0,
            "kurtosis": n_elements * s4 / (s2 * s2) if s2 > 0 else 0.0,
            "onehot_share": hot / nb if nb else 0.0,
            "rel_error": (se / s2) ** 0.5 if s2 > 0 else 0.0}


def stats_raw(x_bits: np.ndarray, g) -> np.ndarray:
    x = _c(x_bits, np.uint16)
    out = np.zeros(6, np.float64)
    rc = _load().orc_stats(_p(x), x.shape[0], x.shape[1], x.shape[1], ctypes.c_float(float(np.float32(g))), _p(out))
    if rc != 0:
        raise ValueError("columns must be a multiple of 16")
    return out


def stats(x_bits: np.ndarray, g) -> dict:
    """max/RMS, kurtosis, 1-hot block share and quantization error of a bf16 tensor at NVFP4 granularity."""
    x = _c(x_bits, np.uint16)
    return derive_stats(stats_raw(x, g), x.size)


def sf_mma_bytes(rows: int, cols: int) -> int:
    return int(_load().orc_sf_mma_bytes(rows, cols))


def sf_mma_index(r: int, b: int, cols: int) -> int:
    return int(_load().orc_sf_mma_index(r, b, cols))


def sf_to_mma(sf_linear: np.ndarray, cols: int) -> np.ndarray:
    sf = _c(sf_linear, np.uint8)
    out = np.empty(sf_mma_bytes(sf.shape[0], cols), np.uint8)
    _load().orc_sf_to_mma(_p(sf), sf.shape[0], cols, _p(out))
    return out


def sf_from_mma(sf_mma: np.ndarray, rows: int, cols: int):
    """Inverse of ``sf_to_mma``: returns (linear [rows, cols/16], True if every
    padding byte is zero)."""
    nb = cols // 16
    r = np.arange(rows, dtype=np.int64)[:, None]
    b = np.arange(nb, dtype=np.int64)[None, :]
    katoms = (nb + 3) // 4
    idx = ((r // 128) * katoms + b // 4) * 512 + ((r % 128) % 32) * 16 + ((r % 128) // 32) * 4 + b % 4
    flat = np.ascontiguousarray(sf_mma, dtype=np.uint8).ravel()
    lin = flat[idx]
    mask = np.ones(flat.size, dtype=bool)
    mask[idx.ravel()] = False
    return lin, bool(np.all(flat[mask] == 0))


def col_scales(N: int, segments: Sequence, g_seg) -> np.ndarray:
    out = np.zeros(N, np.float32)
    for s, gs in zip(segments, g_seg):
        out[s.begin:s.begin + s.count] = np.float32(gs)
    return out


def gemm(a_codes, a_sf, g_a, w_codes, w_sf, g_col, rows=None, cols=None) -> np.ndarray:
    """Exact Y = (A_hat . W_hat^T) with per-column global scale; float64.
    ``rows`` / ``cols``: optional index arrays selecting which outputs to compute."""
    a_codes = _c(a_codes, np.uint8)
    a_sf = _c(a_sf, np.uint8)
    w_codes = _c(w_codes, np.uint8)
    w_sf = _c(w_sf, np.uint8)
    M, K = a_codes.shape[0], a_codes.shape[1] * 2
    N = w_codes.shape[0]
    assert w_codes.shape[1] * 2 == K
    g_col = _c(g_col, np.float32)
    assert g_col.shape == (N,)
    ri = None if rows is None else _c(rows, np.int64)
    ci = None if cols is None else _c(cols, np.int64)
    R = M if ri is None else ri.size
    C = N if ci is None else ci.size
    out = np.empty((R, C), np.float64)
    rc = _load().orc_gemm(_p(a_codes), _p(a_sf), ctypes.c_float(float(np.float32(g_a))), M, K,
                          _p(w_codes), _p(w_sf), _p(g_col), N,
                          None if ri is None else _p(ri), R,
                          None if ci is None else _p(ci), C, _p(out))
    if rc != 0:
        raise RuntimeError("oracle gemm failed (%d)" % rc)
    return out


# -- gated delta-rule recurrence (paper: Background, Eq. 1-2; Section 5.3 lockstep study) ------------
def gdn_gates(a: np.ndarray, b: np.ndarray, A_log: np.ndarray, dt_bias: np.ndarray):
    """Eq. 1: g = -exp(A_log) * softplus(a + dt_bias); alpha = exp(g) in (0, 1); beta = sigmoid(b)."""
    a = np.asarray(a, np.float64)
    z = a + np.asarray(dt_bias, np.float64)
    softplus = np.logaddexp(0.0, z)
    alpha = np.exp(-np.exp(np.asarray(A_log, np.float64)) * softplus)
    bb = np.asarray(b, np.float64)
    e = np.exp(-np.abs(bb))                                    # sigmoid without overflow: e in (0, 1]
    beta = np.where(bb >= 0, 1.0 / (1.0 + e), e / (1.0 + e))
    return alpha, beta


def gdn_recurrence(q, k, v, a, b, A_log, dt_bias, impulse_step: int = -1, impulse_rel: float = 0.0):
    """Eq. 2 in float64, token by token: S_t = alpha_t S_{t-1} + beta_t k_t (v_t - S_{t-1}^T k_t)^T and
    o_t = S_t^T (q_t / sqrt(K)), S_0 = 0.  q, k: [T, Hk, K]; v: [T, Hv, V]; a, b: [T, Hv]; value head h
    reads query/key head h // (Hv // Hk).  Returns (states [T, Hv, K, V], outputs [T, Hv, V]).
    `impulse_step` >= 0 scales the state by (1 + impulse_rel) once, after that token."""
    q, k, v = (np.asarray(t, np.float64) for t in (q, k, v))
    T, Hk, K = q.shape
    Hv, V = v.shape[1], v.shape[2]
    alpha, beta = gdn_gates(a, b, A_log, dt_bias)
    rep = Hv // Hk
    S = np.zeros((Hv, K, V))
    states = np.empty((T, Hv, K, V))
    outs = np.empty((T, Hv, V))
    for t in range(T):
        for h in range(Hv):
            kt, qt = k[t, h // rep], q[t, h // rep]
            pred = S[h].T @ kt                                   # what the state predicts for this key
            S[h] = alpha[t, h] * S[h] + beta[t, h] * np.outer(kt, v[t, h] - pred)
            outs[t, h] = S[h].T @ (qt / np.sqrt(K))
            if t == impulse_step:
                S[h] = S[h] * (1.0 + impulse_rel)
        states[t] = S
    return states, outs


def gdn_lockstep(clean, other, A_log, dt_bias, sample_every: int, impulse_step: int = -1, impulse_rel: float = 0.0):
    """Clean and second trajectory on their own inputs; relative state and output error at the sampled
    tokens (sample_every - 1, 2 * sample_every - 1, ...): ([ns, Hv], [ns, Hv])."""
    S0, o0 = gdn_recurrence(*clean, A_log, dt_bias)
    S1, o1 = gdn_recurrence(*other, A_log, dt_bias, impulse_step, impulse_rel)
    idx = np.arange(sample_every - 1, S0.shape[0], sample_every)
    ds = np.sqrt(((S1[idx] - S0[idx]) ** 2).sum(axis=(2, 3)))
    rs = np.sqrt((S0[idx] ** 2).sum(axis=(2, 3)))
    do = np.sqrt(((o1[idx] - o0[idx]) ** 2).sum(axis=2))
    ro = np.sqrt((o0[idx] ** 2).sum(axis=2))
    with np.errstate(divide="ignore", invalid="ignore"):
        return np.where(rs > 0, ds / rs, 0.0), np.where(ro > 0, do / ro, 0.0)
