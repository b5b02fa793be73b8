"""Python binding of the C ABI in ``include/nvfp4.h``: argument marshalling only.

Every function takes torch CUDA tensors (device memory and streams are all that
torch provides here), passes raw pointers and sizes to the library and raises
``Nvfp4Error`` on a non-zero status.  There is no CPU or torch fallback: if the
library has not been built the first call fails.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Sequence, Tuple

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.environ.get("NVFP4_B200_LIB", os.path.join(_HERE, "libnvfp4_b200.so"))

SF_LINEAR = 0
SF_MMA = 1
OUT_BF16 = 0
OUT_F32 = 1
WS_ZEROED = 2        # workspaces from alloc_workspace are zero-filled, so the binding always promises this
W_RESIDENT = 4       # the weights were complete before the preceding work of the stream was submitted
MAX_SEGMENTS = 32

EXPORTS = (
    "nvfp4_sf_bytes", "nvfp4_calibrate", "nvfp4_quantize_act", "nvfp4_swiglu_quantize", "nvfp4_rmsnorm_quantize",
    "nvfp4_quantize_weight", "nvfp4_quantize_weight_gate_up", "nvfp4_linear_swiglu",
    "nvfp4_harmonize_scales", "nvfp4_tensor_stats", "nvfp4_linear", "nvfp4_linear_workspace_bytes", "nvfp4_linear_bf16",
    "nvfp4_linear_bf16_workspace_bytes", "nvfp4_linear_bf16_static", "nvfp4_static_status", "nvfp4_workspace_reset", "nvfp4_device_status",
    "nvfp4_gdn_lockstep", "nvfp4_last_gemm_clock", "nvfp4_set_wait_limit_ns", "nvfp4_selftest_bounded_wait", "nvfp4_launch_count", "nvfp4_set_gemm_variant", "nvfp4_gemm_variants", "nvfp4_status_string",
)


class Nvfp4Error(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__("%s: status %d (%s)" % (where, status, status_string(status)))


class _Segment(ctypes.Structure):
    _fields_ = [("col_begin", ctypes.c_int64), ("col_count", ctypes.c_int64)]


_lib = None


def lib() -> ctypes.CDLL:
    """Load the CUDA library (built by ``paper_2609_04098_b200.build``); no fallback."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError("CUDA library missing: %s -- run `python -m paper_2609_04098_b200.build`" % LIB_PATH)
    L = ctypes.CDLL(LIB_PATH)
    vp, i64, i32, u32, sz = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int, ctypes.c_uint32, ctypes.c_size_t
    segp = ctypes.POINTER(_Segment)
    L.nvfp4_sf_bytes.restype = sz
    L.nvfp4_sf_bytes.argtypes = [i64, i64, i32]
    L.nvfp4_calibrate.restype = i32
    L.nvfp4_calibrate.argtypes = [vp, i64, i64, i64, vp, vp, vp]
    L.nvfp4_quantize_act.restype = i32
    L.nvfp4_quantize_act.argtypes = [vp, i64, i64, i64, vp, vp, vp, i32, vp]
    L.nvfp4_swiglu_quantize.restype = i32
    L.nvfp4_swiglu_quantize.argtypes = [vp, i64, i64, i64, vp, vp, vp, i32, vp, vp]
    L.nvfp4_rmsnorm_quantize.restype = i32
    L.nvfp4_rmsnorm_quantize.argtypes = [vp, i64, i64, i64, vp, ctypes.c_float, vp, vp, vp, i32, vp, vp]
    L.nvfp4_quantize_weight.restype = i32
    L.nvfp4_quantize_weight.argtypes = [vp, i64, i64, i64, segp, i32, vp, i32, vp, vp, i32, vp]
    L.nvfp4_quantize_weight_gate_up.restype = i32
    L.nvfp4_quantize_weight_gate_up.argtypes = [vp, i64, i64, i64, vp, i32, vp, vp, vp]
    L.nvfp4_linear_swiglu.restype = i32
    L.nvfp4_linear_swiglu.argtypes = [vp, vp, vp, i64, i64, vp, vp, i64, vp, vp, vp, vp, vp, vp, vp, sz, vp]
    L.nvfp4_harmonize_scales.restype = i32
    L.nvfp4_harmonize_scales.argtypes = [vp, i64, i64, i32, segp, vp, i32, vp, vp, vp]
    L.nvfp4_tensor_stats.restype = i32
    L.nvfp4_tensor_stats.argtypes = [vp, i64, i64, i64, vp, vp, vp]
    L.nvfp4_linear.restype = i32
    L.nvfp4_linear.argtypes = [vp, vp, vp, i64, i64, vp, vp, i64, segp, vp, i32, vp, i64, u32, vp, sz, vp]
    L.nvfp4_linear_workspace_bytes.restype = sz
    L.nvfp4_linear_workspace_bytes.argtypes = [i64, i64, i64, i32]
    L.nvfp4_linear_bf16.restype = i32
    L.nvfp4_linear_bf16.argtypes = [vp, i64, vp, i64, i64, vp, vp, i64, segp, vp, i32, vp, i64, u32, vp, sz, vp]
    L.nvfp4_linear_bf16_workspace_bytes.restype = sz
    L.nvfp4_linear_bf16_workspace_bytes.argtypes = [i64, i64, i64, i32]
    L.nvfp4_linear_bf16_static.restype = i32
    L.nvfp4_linear_bf16_static.argtypes = [vp, i64, vp, i64, i64, vp, vp, i64, segp, vp, i32, vp, i64, u32, vp]
    L.nvfp4_static_status.restype = i32
    L.nvfp4_static_status.argtypes = [vp]
    L.nvfp4_workspace_reset.restype = i32
    L.nvfp4_workspace_reset.argtypes = [vp, sz, vp]
    L.nvfp4_device_status.restype = i32
    L.nvfp4_device_status.argtypes = [vp, vp]
    L.nvfp4_gdn_lockstep.restype = i32
    L.nvfp4_gdn_lockstep.argtypes = [vp] * 12 + [i64, i32, i32, i64, ctypes.c_float, i64, vp, vp, vp, vp]
    L.nvfp4_last_gemm_clock.restype = i32
    L.nvfp4_last_gemm_clock.argtypes = [vp, ctypes.POINTER(ctypes.c_double), ctypes.POINTER(ctypes.c_double), vp]
    L.nvfp4_set_wait_limit_ns.restype = i32
    L.nvfp4_set_wait_limit_ns.argtypes = [ctypes.c_uint64]
    L.nvfp4_selftest_bounded_wait.restype = i32
    L.nvfp4_selftest_bounded_wait.argtypes = [vp, sz, ctypes.c_uint64, vp]
    L.nvfp4_launch_count.restype = ctypes.c_uint64
    L.nvfp4_launch_count.argtypes = []
    L.nvfp4_set_gemm_variant.restype = i32
    L.nvfp4_set_gemm_variant.argtypes = [i32]
    L.nvfp4_gemm_variants.restype = ctypes.c_char_p
    L.nvfp4_gemm_variants.argtypes = []
    L.nvfp4_status_string.restype = ctypes.c_char_p
    L.nvfp4_status_string.argtypes = [i32]
    _lib = L
    return L


def status_string(status: int) -> str:
    return lib().nvfp4_status_string(int(status)).decode()


def _check(status: int, where: str) -> None:
    if status != 0:
        raise Nvfp4Error(status, where)


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream(stream) -> ctypes.c_void_p:
    s = torch.cuda.current_stream() if stream is None else stream
    return ctypes.c_void_p(s.cuda_stream)


def _segments(segments: Sequence[Tuple[int, int]]):
    arr = (_Segment * max(1, len(segments)))()
    for i, (b, c) in enumerate(segments):
        arr[i].col_begin, arr[i].col_count = int(b), int(c)
    return arr


def seg_pairs(segments) -> Sequence[Tuple[int, int]]:
    """Accept (begin, count) pairs or objects with .begin/.count."""
    return [(s.begin, s.count) if hasattr(s, "begin") else (int(s[0]), int(s[1])) for s in segments]


def launch_count() -> int:
    return int(lib().nvfp4_launch_count())


def set_gemm_variant(variant: int) -> None:
    _check(lib().nvfp4_set_gemm_variant(int(variant)), "nvfp4_set_gemm_variant")


def set_wait_limit_ns(limit_ns: int) -> None:
    """Limit of every in-kernel wait of the GEMM (0 = default 2 s)."""
    _check(lib().nvfp4_set_wait_limit_ns(int(limit_ns)), "nvfp4_set_wait_limit_ns")


def selftest_bounded_wait(workspace: torch.Tensor, limit_ns: int, stream=None) -> None:
    """Enqueue the failure-path self-test (a wait that nothing completes); read device_status after."""
    _check(lib().nvfp4_selftest_bounded_wait(_ptr(workspace), workspace.numel(), int(limit_ns), _stream(stream)),
           "nvfp4_selftest_bounded_wait")


def sf_bytes(rows: int, K: int, layout: int = SF_MMA) -> int:
    return int(lib().nvfp4_sf_bytes(rows, K, layout))


def nvfp4_calibrate(x: torch.Tensor, g: Optional[torch.Tensor] = None, amax: Optional[torch.Tensor] = None,
                    stream=None) -> torch.Tensor:
    """amax -> global scale g = amax/(6*448) (device scalar, float32)."""
    assert x.is_cuda and x.dtype == torch.bfloat16 and x.dim() == 2 and x.stride(1) == 1
    if g is None:
        g = torch.empty(1, dtype=torch.float32, device=x.device)
    _check(lib().nvfp4_calibrate(_ptr(x), x.shape[0], x.shape[1], x.stride(0), _ptr(g), _ptr(amax),
                                 _stream(stream)), "nvfp4_calibrate")
    return g


def alloc_quantized(rows: int, K: int, device, layout: int = SF_MMA):
    codes = torch.empty((rows, K // 2), dtype=torch.uint8, device=device)
    sf = torch.empty(max(1, sf_bytes(rows, K, layout)), dtype=torch.uint8, device=device)
    return codes, sf


def nvfp4_quantize_act(x: torch.Tensor, g: torch.Tensor, layout: int = SF_MMA, out=None, stream=None):
    """bf16 [M, K] -> (codes u8 [M, K/2], scale bytes u8 [nvfp4_sf_bytes])."""
    assert x.is_cuda and x.dtype == torch.bfloat16 and x.dim() == 2 and x.stride(1) == 1
    M, K = x.shape
    codes, sf = out if out is not None else alloc_quantized(M, K, x.device, layout)
    _check(lib().nvfp4_quantize_act(_ptr(x), M, K, x.stride(0), _ptr(g), _ptr(codes), _ptr(sf), layout,
                                    _stream(stream)), "nvfp4_quantize_act")
    return codes, sf


def nvfp4_swiglu_quantize(gate_up: torch.Tensor, g: torch.Tensor, layout: int = SF_MMA, out=None, stream=None,
                          h_out: Optional[torch.Tensor] = None):
    """bf16 [M, 2I] (gate | up) -> NVFP4 of bf16(silu(gate) * up): (codes u8 [M, I/2], scale bytes).
    ``h_out`` (bf16 [M, I], contiguous; testing aid) also receives the tensor that was quantized."""
    assert gate_up.is_cuda and gate_up.dtype == torch.bfloat16 and gate_up.dim() == 2 and gate_up.stride(1) == 1
    M, two_i = gate_up.shape
    inner = two_i // 2
    assert h_out is None or (h_out.dtype == torch.bfloat16 and h_out.shape == (M, inner) and h_out.is_contiguous())
    codes, sf = out if out is not None else alloc_quantized(M, inner, gate_up.device, layout)
    _check(lib().nvfp4_swiglu_quantize(_ptr(gate_up), M, inner, gate_up.stride(0), _ptr(g), _ptr(codes), _ptr(sf),
                                       layout, _ptr(h_out), _stream(stream)), "nvfp4_swiglu_quantize")
    return codes, sf


def nvfp4_rmsnorm_quantize(x: torch.Tensor, weight: torch.Tensor, eps: float, g: torch.Tensor, layout: int = SF_MMA,
                           out=None, stream=None, y_out: Optional[torch.Tensor] = None):
    """bf16 [M, K], gain bf16 [K] -> NVFP4 of bf16(RMSNorm(x) * weight): (codes, scale bytes).
    ``y_out`` (bf16 [M, K], contiguous; testing aid) also receives the tensor that was quantized."""
    assert x.is_cuda and x.dtype == torch.bfloat16 and x.dim() == 2 and x.stride(1) == 1
    assert weight.dtype == torch.bfloat16 and weight.numel() == x.shape[1] and weight.is_contiguous()
    M, K = x.shape
    assert y_out is None or (y_out.dtype == torch.bfloat16 and y_out.shape == (M, K) and y_out.is_contiguous())
    codes, sf = out if out is not None else alloc_quantized(M, K, x.device, layout)
    _check(lib().nvfp4_rmsnorm_quantize(_ptr(x), M, K, x.stride(0), _ptr(weight), ctypes.c_float(eps), _ptr(g),
                                        _ptr(codes), _ptr(sf), layout, _ptr(y_out), _stream(stream)),
           "nvfp4_rmsnorm_quantize")
    return codes, sf


def nvfp4_quantize_weight(w: torch.Tensor, segments, g_seg: Optional[torch.Tensor] = None,
                          layout: int = SF_MMA, out=None, stream=None):
    """bf16 [N, K] -> (codes, scale bytes, g_seg).  ``g_seg=None`` calibrates each
    segment (amax/2688) on the device; otherwise the given per-segment scales are used."""
    assert w.is_cuda and w.dtype == torch.bfloat16 and w.dim() == 2 and w.stride(1) == 1
    N, K = w.shape
    pairs = seg_pairs(segments)
    calibrate = 0
    if g_seg is None:
        g_seg = torch.empty(len(pairs), dtype=torch.float32, device=w.device)
        calibrate = 1
    codes, sf = out if out is not None else alloc_quantized(N, K, w.device, layout)
    _check(lib().nvfp4_quantize_weight(_ptr(w), N, K, w.stride(0), _segments(pairs), len(pairs), _ptr(g_seg),
                                       calibrate, _ptr(codes), _ptr(sf), layout, _stream(stream)),
           "nvfp4_quantize_weight")
    return codes, sf, g_seg


def nvfp4_quantize_weight_gate_up(w: torch.Tensor, g_gate_up: Optional[torch.Tensor] = None, out=None, stream=None):
    """bf16 [2I, K] (gate rows, then up rows) -> (codes, scale bytes, g[2]) with the rows interleaved 16 by 16,
    the order ``nvfp4_linear_swiglu`` expects.  ``g_gate_up=None`` calibrates each module on the device."""
    assert w.is_cuda and w.dtype == torch.bfloat16 and w.dim() == 2 and w.stride(1) == 1 and w.shape[0] % 2 == 0
    N, K = w.shape
    calibrate = 0
    if g_gate_up is None:
        g_gate_up = torch.empty(2, dtype=torch.float32, device=w.device)
        calibrate = 1
    codes, sf = out if out is not None else alloc_quantized(N, K, w.device, SF_MMA)
    _check(lib().nvfp4_quantize_weight_gate_up(_ptr(w), N // 2, K, w.stride(0), _ptr(g_gate_up), calibrate, _ptr(codes),
                                               _ptr(sf), _stream(stream)), "nvfp4_quantize_weight_gate_up")
    return codes, sf, g_gate_up


def nvfp4_linear_swiglu(a_codes, a_sf, g_a, w_codes, w_sf, g_gate_up, g_h, workspace, out=None, stream=None,
                        dbg_y: Optional[torch.Tensor] = None, dbg_h: Optional[torch.Tensor] = None):
    """Gate/up GEMM with SwiGLU and the quantization of h = silu(gate) * up in its epilogue: returns
    (codes u8 [M, I/2], scale bytes) of h, ready for the down projection.  ``dbg_y`` (bf16 [M, 2I], interleaved
    columns) and ``dbg_h`` (bf16 [M, I]) are optional testing outputs."""
    M, K = a_codes.shape[0], a_codes.shape[1] * 2
    inner = w_codes.shape[0] // 2
    codes, sf = out if out is not None else alloc_quantized(M, inner, a_codes.device, SF_MMA)
    _check(lib().nvfp4_linear_swiglu(_ptr(a_codes), _ptr(a_sf), _ptr(g_a), M, K, _ptr(w_codes), _ptr(w_sf), inner,
                                     _ptr(g_gate_up), _ptr(g_h), _ptr(codes), _ptr(sf), _ptr(dbg_y), _ptr(dbg_h),
                                     _ptr(workspace), workspace.numel(), _stream(stream)), "nvfp4_linear_swiglu")
    return codes, sf


def nvfp4_harmonize_scales(w_sf: torch.Tensor, N: int, K: int, segments, g_seg: torch.Tensor,
                           layout: int = SF_MMA, stream=None):
    """Shared global scale for a fused group: returns (re-rounded scale bytes, g* device scalar)."""
    pairs = seg_pairs(segments)
    out = torch.empty_like(w_sf)
    g_shared = torch.empty(1, dtype=torch.float32, device=w_sf.device)
    _check(lib().nvfp4_harmonize_scales(_ptr(w_sf), N, K, layout, _segments(pairs), _ptr(g_seg), len(pairs),
                                        _ptr(out), _ptr(g_shared), _stream(stream)), "nvfp4_harmonize_scales")
    return out, g_shared


def nvfp4_tensor_stats(x: torch.Tensor, g: torch.Tensor, stream=None) -> torch.Tensor:
    """Seven float64 accumulators (see include/nvfp4.h): sums of x^2, x^4, err^2, amax, blocks, 1-hot blocks."""
    assert x.is_cuda and x.dtype == torch.bfloat16 and x.dim() == 2 and x.stride(1) == 1
    out = torch.empty(7, dtype=torch.float64, device=x.device)
    _check(lib().nvfp4_tensor_stats(_ptr(x), x.shape[0], x.shape[1], x.stride(0), _ptr(g), _ptr(out), _stream(stream)),
           "nvfp4_tensor_stats")
    return out


def alloc_workspace(device, M: int = 0, N: int = 0, K: int = 0, nseg: int = 1, fused: bool = False) -> torch.Tensor:
    n = (lib().nvfp4_linear_bf16_workspace_bytes(M, N, K, nseg) if fused
         else lib().nvfp4_linear_workspace_bytes(M, N, K, nseg))
    ws = torch.zeros(int(n), dtype=torch.uint8, device=device)
    return ws


def nvfp4_linear(a_codes, a_sf, g_a, w_codes, w_sf, segments, g_seg, workspace, out=None,
                 out_f32: bool = False, stream=None, w_resident: bool = False) -> torch.Tensor:
    """Y[M, N] = (A_q . W_q^T) * g_a * g_seg[segment of n]; bf16 (or float32) output.
    ``w_resident``: the weights (codes, scales, ``g_seg``) were complete before the work in front of
    this call was submitted to the stream, so the kernel may fetch them while that work still runs."""
    M, K = a_codes.shape[0], a_codes.shape[1] * 2
    N = w_codes.shape[0]
    pairs = seg_pairs(segments)
    if out is None:
        out = torch.empty((M, N), dtype=torch.float32 if out_f32 else torch.bfloat16, device=a_codes.device)
    flags = (OUT_F32 if out.dtype == torch.float32 else OUT_BF16) | WS_ZEROED | (W_RESIDENT if w_resident else 0)
    _check(lib().nvfp4_linear(_ptr(a_codes), _ptr(a_sf), _ptr(g_a), M, K, _ptr(w_codes), _ptr(w_sf), N,
                              _segments(pairs), _ptr(g_seg), len(pairs), _ptr(out), out.stride(0), flags,
                              _ptr(workspace), workspace.numel(), _stream(stream)), "nvfp4_linear")
    return out


def nvfp4_linear_bf16(x, g_a, w_codes, w_sf, segments, g_seg, workspace, out=None, out_f32: bool = False,
                      stream=None, w_resident: bool = False) -> torch.Tensor:
    """Same layer fed with bf16 activations; quantization happens inside the call."""
    assert x.is_cuda and x.dtype == torch.bfloat16 and x.dim() == 2 and x.stride(1) == 1
    M, K = x.shape
    N = w_codes.shape[0]
    pairs = seg_pairs(segments)
    if out is None:
        out = torch.empty((M, N), dtype=torch.float32 if out_f32 else torch.bfloat16, device=x.device)
    flags = (OUT_F32 if out.dtype == torch.float32 else OUT_BF16) | WS_ZEROED | (W_RESIDENT if w_resident else 0)
    _check(lib().nvfp4_linear_bf16(_ptr(x), x.stride(0), _ptr(g_a), M, K, _ptr(w_codes), _ptr(w_sf), N,
                                   _segments(pairs), _ptr(g_seg), len(pairs), _ptr(out), out.stride(0), flags,
                                   _ptr(workspace), workspace.numel(), _stream(stream)), "nvfp4_linear_bf16")
    return out


STATIC_SCRATCH_BYTES = 12 * 1024 * 1024
SPLIT_RESERVE_BYTES = 5 * 1024 * 1024      # split-K part of every workspace, directly behind the 256-byte status block


def nvfp4_linear_bf16_static(x, g_a, w_codes, w_sf, segments, g_seg, out=None, out_f32: bool = False,
                             stream=None) -> torch.Tensor:
    """``nvfp4_linear_bf16`` without a caller-provided workspace, for hosts that may not allocate
    device memory when they run a layer (a server whose memory pool owns the whole device, a
    plug-in inside another framework's callback).  The quantized activations go to a fixed
    ``STATIC_SCRATCH_BYTES`` array inside the library; larger problems raise ``Nvfp4Error``
    (workspace).  Calls share that array, so calls that overlap on the GPU must be serialised;
    make the first call on a device outside of stream capture.  ``out`` must be passed in by a
    caller that really cannot allocate (otherwise it is allocated here, by torch)."""
    assert x.is_cuda and x.dtype == torch.bfloat16 and x.dim() == 2 and x.stride(1) == 1
    M, K = x.shape
    N = w_codes.shape[0]
    pairs = seg_pairs(segments)
    if out is None:
        out = torch.empty((M, N), dtype=torch.float32 if out_f32 else torch.bfloat16, device=x.device)
    flags = OUT_F32 if out.dtype == torch.float32 else OUT_BF16
    _check(lib().nvfp4_linear_bf16_static(_ptr(x), x.stride(0), _ptr(g_a), M, K, _ptr(w_codes), _ptr(w_sf), N,
                                          _segments(pairs), _ptr(g_seg), len(pairs), _ptr(out), out.stride(0),
                                          flags, _stream(stream)), "nvfp4_linear_bf16_static")
    return out


def static_status(stream=None) -> int:
    """Status word of the library's static scratch (synchronises the stream); a failure also
    clears the word and re-zeroes the split-K part of the array."""
    return int(lib().nvfp4_static_status(_stream(stream)))


def nvfp4_gdn_lockstep(clean, other, A_log, dt_bias, sample_every: int, impulse_step: int = -1,
                       impulse_rel: float = 0.0, final_state: bool = False, stream=None):
    """Gated delta-rule recurrence on two input sets in lockstep.  ``clean`` and ``other`` are tuples
    (q [T,Hk,128], k [T,Hk,128], v [T,Hv,128], a [T,Hv], b [T,Hv]) of float32 CUDA tensors.
    Returns (rel_state [T // sample_every, Hv], rel_out, final states [2,Hv,128,128] or None)."""
    q, k, v, a, b = clean
    T, Hk = q.shape[0], q.shape[1]
    Hv = v.shape[1]
    for t in tuple(clean) + tuple(other) + (A_log, dt_bias):
        assert t.is_cuda and t.dtype == torch.float32 and t.is_contiguous()
    ns = T // sample_every
    rel_state = torch.zeros((max(ns, 1), Hv), dtype=torch.float32, device=q.device)
    rel_out = torch.zeros_like(rel_state)
    fs = torch.empty((2, Hv, 128, 128), dtype=torch.float32, device=q.device) if final_state else None
    _check(lib().nvfp4_gdn_lockstep(*[_ptr(t) for t in clean], *[_ptr(t) for t in other], _ptr(A_log), _ptr(dt_bias),
                                    T, Hk, Hv, int(impulse_step), ctypes.c_float(impulse_rel), int(sample_every),
                                    _ptr(rel_state), _ptr(rel_out), _ptr(fs), _stream(stream)), "nvfp4_gdn_lockstep")
    return rel_state[:ns], rel_out[:ns], fs


def last_gemm_clock(workspace: torch.Tensor, stream=None) -> Tuple[float, float]:
    """(SM clock in MHz, lifetime in us) of the first CTA of the last tensor-core GEMM launched on this
    workspace, from the kernel's own cycle counter and wall clock.  Synchronises the stream."""
    mhz, us = ctypes.c_double(0.0), ctypes.c_double(0.0)
    _check(lib().nvfp4_last_gemm_clock(_ptr(workspace), ctypes.byref(mhz), ctypes.byref(us), _stream(stream)),
           "nvfp4_last_gemm_clock")
    return mhz.value, us.value


def workspace_reset(workspace: torch.Tensor, stream=None) -> None:
    _check(lib().nvfp4_workspace_reset(_ptr(workspace), workspace.numel(), _stream(stream)), "nvfp4_workspace_reset")


def device_status(workspace: torch.Tensor, stream=None) -> int:
    """Synchronises the stream; 0 = ok, 8 = a bounded in-kernel wait ran out, 10 = a global scale
    read on the device was not finite and positive."""
    return int(lib().nvfp4_device_status(_ptr(workspace), _stream(stream)))
