"""Failure detection without faulting a GPU: bounded waits run out, the kernel returns, the
host reads a status, the context stays usable."""
import time

import pytest
import torch

import oracle
from paper_2609_04098_b200 import binding as nv
from paper_2609_04098_b200 import synth
from tests import gpu_util as gu

pytestmark = pytest.mark.gpu


def test_wait_on_a_barrier_nothing_completes_times_out():
    ws = nv.alloc_workspace(gu.DEV)
    t0 = time.perf_counter()
    nv.selftest_bounded_wait(ws, 2_000_000)            # 2 ms
    assert nv.device_status(ws) == 8                   # NVFP4_ERR_TIMEOUT
    assert time.perf_counter() - t0 < 5.0
    # the context is alive and the status word can be cleared and reused
    nv.workspace_reset(ws)
    assert nv.device_status(ws) == 0
    assert float(torch.ones(4, device=gu.DEV).sum().item()) == 4.0


@pytest.mark.parametrize("variant", [256, 2])
def test_gemm_gives_up_cleanly_when_its_waits_are_cut_short(variant):
    # A 1 ns limit makes a correct launch run out of patience on its first real wait: every role
    # winds down, the status word says so, and the next launch (default limit) is correct.
    nv.set_gemm_variant(variant)
    M, N, K = 512, 512, 5120
    segs = synth.make_segments((("w", N, 0.02),))
    x = synth.prefill_activations(31, 1, M, K)
    w = synth.weights(31, 2, segs, K)
    ac, asf, ga, _ = gu.oracle_quantized(x)
    wc, wsf, gs, _ = gu.oracle_quantized(w, segments=segs)
    args = (gu.dev_u8(ac), gu.dev_u8(oracle.sf_to_mma(asf, K)), gu.dev_f32(ga), gu.dev_u8(wc),
            gu.dev_u8(oracle.sf_to_mma(wsf, K)), segs, gu.dev_f32(gs))
    ws = nv.alloc_workspace(gu.DEV)
    try:
        nv.set_wait_limit_ns(1)
        nv.nvfp4_linear(*args, ws)
        assert nv.device_status(ws) == 8
    finally:
        nv.set_wait_limit_ns(0)
        nv.set_gemm_variant(0)
    nv.workspace_reset(ws)
    nv.set_gemm_variant(variant)
    y = nv.nvfp4_linear(*args, ws)
    nv.set_gemm_variant(0)
    assert nv.device_status(ws) == 0
    gcol = oracle.col_scales(N, segs, gs)
    gu.check_gemm(y, oracle.gemm(ac, asf, ga, wc, wsf, gcol), gu.gemm_bounds(ac, asf, ga, wc, wsf, gcol), "after timeout")
