"""GPU parity for the NVFP4-granularity statistics against the oracle's float64 definition.  The
block count and the maximum are exact.  The kernel forms each block's sums in binary32 (16 fused
multiply-adds: relative error below 16 * 2^-24 ~ 1e-6 per block, less in the total) and its
dequantized value through one extra binary32 rounding of e4m3 * g (2^-24 relative on x_hat, i.e.
about 1e-6 on an error that is a tenth of x): tolerances 5e-6 on sum x^2 and sum x^4, 2e-5 on
sum err^2.  The 1-hot count compares bmax^2 * 16 with 9 * (binary32 block sum): a block within
1e-6 of the threshold may fall on the other side, so the count may differ by a few in a million."""
import numpy as np
import pytest
import torch

import oracle
from paper_2609_04098_b200 import binding as nv
from paper_2609_04098_b200 import synth
from tests import gpu_util as gu

pytestmark = pytest.mark.gpu


def _case(x_bits, g=None):
    if g is None:
        _, g = oracle.calibrate(x_bits)
    want = oracle.stats_raw(x_bits, g)
    got = nv.nvfp4_tensor_stats(gu.dev_bf16(x_bits), gu.dev_f32(g)).cpu().numpy()
    assert got[3] == want[3] and got[4] == want[4], (got, want)
    assert abs(got[5] - want[5]) <= 1 + 5e-6 * want[4], (got, want)
    for i, tol in ((0, 5e-6), (1, 5e-6), (2, 2e-5)):
        assert abs(got[i] - want[i]) <= tol * abs(want[i]) + 1e-300, (i, got[i], want[i])
    return oracle.derive_stats(got[:6], x_bits.size)


def test_heavy_tailed_activations():
    st = _case(synth.config2_activations(0, M=1024, K=5120))
    assert st["max_over_rms"] > 40 and 0.0 < st["onehot_share"] < 0.5


def test_weights_and_ragged_shapes_and_static_scale():
    segs = synth.make_segments((("w", 300, 0.02),))
    st = _case(synth.weights(0, 31, segs, 1040))
    assert abs(st["kurtosis"] - 3.0) < 0.2 and 0.08 < st["rel_error"] < 0.13
    _case(synth.prefill_activations(2, 32, 7, 48), g=0.37)
    _case(np.zeros((3, 64), np.uint16))
    x = np.zeros((1, 32))
    x[0, 3] = 7.0
    st = _case(synth.f64_to_bf16_bits(x).reshape(1, 32), g=1.0)
    assert st["onehot_share"] == 0.5
