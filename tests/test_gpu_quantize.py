"""GPU parity: calibrate / quantize_act / quantize_weight against the CPU oracle,
bit-exact on packed codes and scale bytes, through the C ABI."""
import numpy as np
import pytest
import torch

import oracle
from paper_2609_04098_b200 import binding as nv
from paper_2609_04098_b200 import synth
from tests import gpu_util as gu

pytestmark = pytest.mark.gpu


def _act_case(x_bits, g=None, layout=nv.SF_MMA, ld_pad=0):
    M, K = x_bits.shape
    xt = gu.dev_bf16(x_bits)
    if ld_pad:
        buf = torch.zeros((M, K + ld_pad), dtype=torch.bfloat16, device=gu.DEV)
        buf[:, :K] = xt
        xt = buf[:, :K]
    if g is None:
        amax_d = torch.zeros(1, dtype=torch.float32, device=gu.DEV)
        g_d = nv.nvfp4_calibrate(xt, amax=amax_d)
        amax_o, g_o = oracle.calibrate(x_bits)
        assert amax_d.item() == amax_o and g_d.item() == g_o
    else:
        g_d = gu.dev_f32(g)
        g_o = np.float32(g)
    codes_d, sf_d = nv.nvfp4_quantize_act(xt, g_d, layout)
    torch.cuda.synchronize()
    codes_o, sf_o, _, _ = gu.oracle_quantized(x_bits, g=g_o)
    gu.check_quantized(codes_d, sf_d, layout, codes_o, sf_o, K)
    return codes_d, sf_d


@pytest.mark.parametrize("layout", [nv.SF_MMA, nv.SF_LINEAR])
def test_config1_activations(layout):
    x, _, _ = synth.config1(0)
    _act_case(x, layout=layout)


@pytest.mark.parametrize("M,K", [(1, 16), (1, 5120), (3, 48), (16, 64), (17, 80), (127, 272), (129, 256),
                                 (130, 1040), (257, 512), (300, 2064)])
@pytest.mark.parametrize("layout", [nv.SF_MMA, nv.SF_LINEAR])
def test_ragged_shapes(M, K, layout):
    x = synth.config2_activations(7, M=M, K=K)
    _act_case(x, layout=layout)


def test_strided_input():
    x = synth.prefill_activations(1, 3, 70, 320)
    _act_case(x, ld_pad=48)


def test_every_finite_bf16_pattern_at_several_scales():
    # all 2^16 bit patterns minus NaN/Inf, laid out so that blocks mix magnitudes
    pats = np.arange(65536, dtype=np.uint16)
    finite = pats[(pats & 0x7F80) != 0x7F80]
    rng = np.random.default_rng(0)
    for g in (1.0, 0.37, 2.0 ** -20, 3.1e4):
        x = rng.permutation(finite)[: (finite.size // 256) * 256].reshape(-1, 256)
        _act_case(x, g=g)
    # sorted order: neighbouring values share blocks, so codes span the whole grid incl. ties
    x = finite[: (finite.size // 512) * 512].reshape(-1, 512)
    _act_case(x, g=2.0 ** -3)
    _act_case(x)


def test_ties_zeros_signs_and_saturation():
    vals = np.array([6.0, 0.25, 0.75, 1.25, 1.75, 2.5, 3.5, 5.0, -0.25, -0.75, -1.25, -1.75, -2.5, -3.5, -5.0, 0.0,
                     0.0] * 1 + [-0.0] * 15 + [1e6, -1e6] + [1.0] * 14 + [1e-30, -1e-30] * 8)
    x = synth.f64_to_bf16_bits(vals).reshape(1, 64)
    _act_case(x, g=1.0)
    _act_case(x, g=1e-3)        # static scale far too small: scale bytes and codes saturate
    _act_case(np.zeros((5, 64), np.uint16))               # all-zero tensor: g = 1, everything 0
    _act_case(np.full((5, 64), 0x8000, np.uint16))        # all -0


def test_config2_full_size_bit_exact():
    x = synth.config2_activations(0)
    assert x.shape == (8192, 5120)
    _act_case(x)


def test_repeat_runs_are_identical():
    x = synth.config2_activations(3, M=1024, K=5120)
    xt = gu.dev_bf16(x)
    g = nv.nvfp4_calibrate(xt)
    c1, s1 = nv.nvfp4_quantize_act(xt, g)
    c2, s2 = nv.nvfp4_quantize_act(xt, g)
    torch.cuda.synchronize()
    assert torch.equal(c1, c2) and torch.equal(s1, s2)


@pytest.mark.parametrize("layout", [nv.SF_MMA, nv.SF_LINEAR])
def test_weight_segments_calibrated_on_device(layout):
    segs = synth.make_segments((("q", 64, 0.02), ("k", 40, 0.02), ("a", 48, 0.2), ("b", 9, 0.2)))
    w = synth.weights(0, 5, segs, 320)
    codes_d, sf_d, g_d = nv.nvfp4_quantize_weight(gu.dev_bf16(w), segs, None, layout)
    torch.cuda.synchronize()
    codes_o, sf_o, g_o, _ = gu.oracle_quantized(w, segments=segs)
    assert np.array_equal(g_d.cpu().numpy(), g_o)
    gu.check_quantized(codes_d, sf_d, layout, codes_o, sf_o, 320)


def test_weight_segments_given_scales():
    segs = synth.make_segments((("qkv", 96, 0.02), ("z", 96, 0.02)))
    w = synth.weights(2, 5, segs, 256)
    g_seg = np.float32([3.1e-5, 3.1e-5 / 1.82])
    codes_d, sf_d, _ = nv.nvfp4_quantize_weight(gu.dev_bf16(w), segs, gu.dev_f32(g_seg), nv.SF_MMA)
    torch.cuda.synchronize()
    codes_o, sf_o, _, _ = gu.oracle_quantized(w, segments=segs, g_seg=g_seg)
    gu.check_quantized(codes_d, sf_d, nv.SF_MMA, codes_o, sf_o, 256)


def test_gdn_weight_full_size():
    segs = synth.make_segments(synth.GDN_SEGMENTS)
    w = synth.weights(0, 402, segs, synth.HIDDEN)
    codes_d, sf_d, g_d = nv.nvfp4_quantize_weight(gu.dev_bf16(w), segs, None, nv.SF_MMA)
    torch.cuda.synchronize()
    codes_o, sf_o, g_o, _ = gu.oracle_quantized(w, segments=segs)
    assert np.array_equal(g_d.cpu().numpy(), g_o)
    gu.check_quantized(codes_d, sf_d, nv.SF_MMA, codes_o, sf_o, synth.HIDDEN)


# ---- producer fusion: silu(gate) * up -> quantize in one pass -------------------------------
# Two independent links, both against the oracle: (1) the bf16 tensor h the kernel forms (testing
# output) against the float64 definition rounded once -- at most one bf16 ulp apart, equal almost
# everywhere; (2) codes and scale bytes bit-exact against oracle.quantize of THAT tensor.
def _swiglu_input(M, inner, seed=9):
    segs = synth.make_segments((("gate", M, 1.0),))
    gate_up = synth.weights(seed, 60, segs, 2 * inner)                 # bf16 [M, 2*inner] ~ N(0, 1): gate | up
    # a few hot entries, as after a projection of outlier channels
    gate_up[:, 7] = synth.f64_to_bf16_bits(synth.bf16_bits_to_f32(gate_up[:, 7]).astype(np.float64) * 12.0)
    return gate_up


def _swiglu_check(gate_up, layout=nv.SF_MMA, ld_pad=0, min_equal=0.995):
    M, inner = gate_up.shape[0], gate_up.shape[1] // 2
    h_def = oracle.swiglu_bf16(gate_up)                                # the definition, float64, rounded once
    _, g = oracle.calibrate(h_def)
    t = synth.to_torch_bf16(gate_up).to(gu.DEV)
    if ld_pad:
        buf = torch.zeros((M, 2 * inner + ld_pad), dtype=torch.bfloat16, device=gu.DEV)
        buf[:, :2 * inner] = t
        t = buf[:, :2 * inner]
    h_d = torch.empty((M, inner), dtype=torch.bfloat16, device=gu.DEV)
    codes_d, sf_d = nv.nvfp4_swiglu_quantize(t, gu.dev_f32(g), layout, h_out=h_d)
    torch.cuda.synchronize()
    h_gpu = gu.host_bits(h_d)
    gu.check_bf16_close_to_definition(h_gpu, h_def, min_equal, "swiglu %s" % ((M, inner),))
    codes_o, sf_o, _, _ = gu.oracle_quantized(h_gpu, g=g)
    gu.check_quantized(codes_d, sf_d, layout, codes_o, sf_o, inner)
    # without the testing output the kernel writes the same codes and scales
    codes_2, sf_2 = nv.nvfp4_swiglu_quantize(t, gu.dev_f32(g), layout)
    torch.cuda.synchronize()
    assert torch.equal(codes_2, codes_d) and torch.equal(sf_2, sf_d)
    return t, g, codes_d, sf_d, h_d


@pytest.mark.parametrize("M,inner", [(1, 16), (5, 48), (128, 512), (130, 1040), (300, 17408 // 4)])
@pytest.mark.parametrize("layout", [nv.SF_MMA, nv.SF_LINEAR])
def test_swiglu_quantize_two_links_to_the_oracle(M, inner, layout):
    _swiglu_check(_swiglu_input(M, inner), layout)


def test_swiglu_quantize_strided_and_equal_to_unfused_path():
    t, g, codes_d, sf_d, h_d = _swiglu_check(_swiglu_input(96, 2048), ld_pad=64)
    # the same result as calling nvfp4_quantize_act on the h the kernel formed
    c2, s2 = nv.nvfp4_quantize_act(h_d, gu.dev_f32(g))
    torch.cuda.synchronize()
    assert torch.equal(c2, codes_d) and torch.equal(s2, sf_d)


def test_swiglu_extreme_gates():
    M, inner = 4, 64
    vals = np.zeros((M, 2 * inner))
    vals[:, :inner] = np.linspace(-120, 120, inner)[None, :] * np.array([1.0, 0.5, 0.01, -1.0])[:, None]
    vals[:, inner:] = np.array([1.0, -3.0, 250.0, 0.125])[:, None]
    _swiglu_check(synth.f64_to_bf16_bits(vals).reshape(M, 2 * inner), min_equal=0.98)


def test_swiglu_quantize_just_above_the_two_chunk_switch():
    # M * chunks > 2 * (148 SMs x 40 resident warps): the launch shape of the large tensors
    _swiglu_check(_swiglu_input(352, 17408, seed=10))


def test_swiglu_quantize_full_size_mlp_inner():
    # the benchmark's own launch: [8192, 2 x 17408] bf16 in, every code and scale byte compared
    _swiglu_check(_swiglu_input(8192, 17408, seed=11))


# ---- producer fusion: RMSNorm(x) * w -> quantize in one pass ----------------------------------
def _rmsnorm_case(M, K, layout=nv.SF_MMA, seed=12, eps=1e-6, ld_pad=0):
    x = synth.prefill_activations(seed, 80, M, K)
    w = synth.f64_to_bf16_bits(1.0 + 0.25 * np.cos(0.37 * np.arange(K)))
    y_def = oracle.rmsnorm_bf16(x, w, eps)                             # the definition, float64, rounded once
    _, g = oracle.calibrate(y_def)
    t = gu.dev_bf16(x)
    if ld_pad:
        buf = torch.zeros((M, K + ld_pad), dtype=torch.bfloat16, device=gu.DEV)
        buf[:, :K] = t
        t = buf[:, :K]
    y_d = torch.empty((M, K), dtype=torch.bfloat16, device=gu.DEV)
    codes_d, sf_d = nv.nvfp4_rmsnorm_quantize(t, gu.dev_bf16(w), eps, gu.dev_f32(g), layout, y_out=y_d)
    torch.cuda.synchronize()
    y_gpu = gu.host_bits(y_d)
    gu.check_bf16_close_to_definition(y_gpu, y_def, 0.995, "rmsnorm %s" % ((M, K),))
    codes_o, sf_o, _, _ = gu.oracle_quantized(y_gpu, g=g)
    gu.check_quantized(codes_d, sf_d, layout, codes_o, sf_o, K)
    codes_2, sf_2 = nv.nvfp4_rmsnorm_quantize(t, gu.dev_bf16(w), eps, gu.dev_f32(g), layout)
    torch.cuda.synchronize()
    assert torch.equal(codes_2, codes_d) and torch.equal(sf_2, sf_d)


# K = 16 .. 2560: one warp per row; 5120: two; 17408: eight; 20992: beyond the register-resident
# kernel (two passes over the row)
@pytest.mark.parametrize("M,K", [(1, 16), (3, 528), (130, 5120), (64, 17408), (257, 1040), (200, 2560), (9, 20992)])
@pytest.mark.parametrize("layout", [nv.SF_MMA, nv.SF_LINEAR])
def test_rmsnorm_quantize_two_links_to_the_oracle(M, K, layout):
    _rmsnorm_case(M, K, layout)


def test_rmsnorm_quantize_strided_and_eps_zero():
    _rmsnorm_case(40, 2048, ld_pad=32, eps=0.0)
    _rmsnorm_case(2048, 5120, seed=13)


def test_rmsnorm_quantize_full_size_hidden():
    _rmsnorm_case(8192, 5120, seed=14)
