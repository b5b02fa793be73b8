"""The no-allocation entry point ``nvfp4_linear_bf16_static``.

It serves hosts that may not allocate device memory when they run a layer -- a server
whose own pool holds the whole device, a plug-in called from inside another framework --
by keeping the quantized-activation scratch in a fixed array inside the library.  The
tests drive it through the C ABI.  It must give the same output as ``nvfp4_linear_bf16``
with a caller-provided workspace on two calls in a row (the second reuses the array with
different inputs and a different shape); a sequence of shapes whose quantized activations
reach far into the array must not disturb later calls that split K (the split-K part of
the array sits at a fixed place in front of them), checked against the oracle; and sizes
beyond the array are refused.

This file sorts last on purpose: a run that stops at the first failure has then already
run every other test.
"""
import pytest
import torch

import oracle
from paper_2609_04098_b200 import binding as nv
from paper_2609_04098_b200 import synth
from tests import gpu_util as gu

pytestmark = pytest.mark.gpu


def _case(seed, M, K, segspec):
    segs = synth.make_segments(segspec)
    x = gu.dev_bf16(synth.prefill_activations(seed, 1, M, K))
    w = gu.dev_bf16(synth.weights(seed, 2, segs, K))
    g_a = nv.nvfp4_calibrate(x)
    w_codes, w_sf, g_seg = nv.nvfp4_quantize_weight(w, segs)
    return segs, x, g_a, w_codes, w_sf, g_seg


def test_static_scratch_matches_workspace_entry_point_twice():
    for seed, M, K, spec in ((21, 48, 1024, (("p", 200, 0.02), ("q", 120, 0.2))),
                             (22, 130, 512, (("a", 96, 0.02), ("b", 48, 0.2), ("c", 8, 0.02)))):
        segs, x, g_a, w_codes, w_sf, g_seg = _case(seed, M, K, spec)
        N = w_codes.shape[0]
        ws = nv.alloc_workspace(gu.DEV, M, N, K, len(segs), fused=True)
        want = nv.nvfp4_linear_bf16(x, g_a, w_codes, w_sf, segs, g_seg, ws)
        assert nv.device_status(ws) == 0
        out = torch.empty((M, N), dtype=torch.bfloat16, device=gu.DEV)     # caller-owned output
        got = nv.nvfp4_linear_bf16_static(x, g_a, w_codes, w_sf, segs, g_seg, out=out)
        assert nv.static_status() == 0
        # same kernels on the same quantized activations: the tolerance is equality
        assert torch.equal(got, want), (seed, M, K)


def _oracle_case(seed, M, N, K):
    segs = synth.make_segments((("w", N, 0.02),))
    x = synth.prefill_activations(seed, 3, M, K)
    w = synth.weights(seed, 4, segs, K)
    ac, asf, ga, _ = gu.oracle_quantized(x)
    wc, wsf, gs, _ = gu.oracle_quantized(w, segments=segs)
    gcol = oracle.col_scales(N, segs, gs)
    dev = (gu.dev_bf16(x), gu.dev_f32(ga), gu.dev_u8(wc), gu.dev_u8(oracle.sf_to_mma(wsf, K)), segs, gu.dev_f32(gs))
    return dev, oracle.gemm(ac, asf, ga, wc, wsf, gcol), gu.gemm_bounds(ac, asf, ga, wc, wsf, gcol)


def test_static_scratch_shape_sequence_against_the_oracle():
    # many rows at a long K first (their codes and scales fill ~0.9 MB of the array), then
    # decode-sized calls at the same K that split K over several CTAs, then a single token
    for seed, (M, N, K) in enumerate(((200, 1024, 8192), (16, 6144, 8192), (256, 1024, 8192), (16, 1024, 8192),
                                      (1, 6144, 8192), (16, 6144, 8192))):
        dev, y_ref, bound = _oracle_case(50 + seed, M, N, K)
        y = nv.nvfp4_linear_bf16_static(*dev)
        assert nv.static_status() == 0, (M, N, K)
        gu.check_gemm(y, y_ref, bound, "static %s" % ((M, N, K),))


def test_static_scratch_rejects_sizes_beyond_the_array():
    M, K = 4096, 5120                      # 4096 x 5120 / 2 bytes of codes alone exceed what the array holds
    assert nv.lib().nvfp4_linear_bf16_workspace_bytes(M, 256, K, 1) > nv.STATIC_SCRATCH_BYTES
    segs, x, g_a, w_codes, w_sf, g_seg = _case(23, 8, K, (("w", 256, 0.02),))
    big = torch.zeros((M, K), dtype=torch.bfloat16, device=gu.DEV)
    with pytest.raises(nv.Nvfp4Error) as err:
        nv.nvfp4_linear_bf16_static(big, g_a, w_codes, w_sf, segs, g_seg)
    assert err.value.status == 5 and "workspace" in str(err.value)
