"""GPU parity of the lockstep gated delta-rule recurrence (binary32 on the device) against the oracle's
float64 recurrence, and the synthetic version of the paper's lockstep study: the in-projections of a
GDN layer computed exactly and through the NVFP4 W4A4 layer feed two trajectories; the state error
must plateau instead of growing, and a one-off 1 % state impulse must be forgotten."""
import numpy as np
import pytest
import torch

import oracle
from paper_2609_04098_b200 import binding as nv
from paper_2609_04098_b200 import synth
from tests import gpu_util as gu

pytestmark = pytest.mark.gpu


def _inputs(seed, T, Hk, Hv, noise):
    rng = np.random.default_rng(seed)
    def unit(*shape):
        x = rng.standard_normal(shape)
        return x / np.linalg.norm(x, axis=-1, keepdims=True)
    q, k = unit(T, Hk, 128), unit(T, Hk, 128)
    v = rng.standard_normal((T, Hv, 128))
    a, b = rng.standard_normal((T, Hv)) * 2.0, rng.standard_normal((T, Hv))
    clean = [t.astype(np.float32) for t in (q, k, v, a, b)]
    other = [(t + noise * np.abs(t).mean() * rng.standard_normal(t.shape)).astype(np.float32) for t in (q, k, v, a, b)]
    for i in (0, 1):      # keep queries and keys on the unit sphere, as the layer does
        other[i] = (other[i] / np.linalg.norm(other[i], axis=-1, keepdims=True)).astype(np.float32)
    A_log = (np.log(rng.uniform(0.005, 0.2, Hv))).astype(np.float32)
    dtb = (rng.standard_normal(Hv) * 0.1).astype(np.float32)
    return clean, other, A_log, dtb


def _dev(ts):
    return tuple(torch.from_numpy(np.ascontiguousarray(t)).to(gu.DEV) for t in ts)


@pytest.mark.parametrize("T,Hk,Hv,every", [(257, 2, 6, 16), (64, 1, 1, 1), (300, 3, 3, 50)])
def test_lockstep_matches_the_float64_recurrence(T, Hk, Hv, every):
    clean, other, A_log, dtb = _inputs(1, T, Hk, Hv, 0.05)
    rs_o, ro_o = oracle.gdn_lockstep(clean, other, A_log, dtb, every)
    rs, ro, fs = nv.nvfp4_gdn_lockstep(_dev(clean), _dev(other), *_dev((A_log, dtb)), every, final_state=True)
    torch.cuda.synchronize()
    # two binary32 trajectories against two float64 ones: the errors of each (~1e-6 relative per state)
    # are far below the differences being measured (~5e-2)
    assert np.allclose(rs.cpu().numpy(), rs_o, rtol=2e-3, atol=1e-6)
    assert np.allclose(ro.cpu().numpy(), ro_o, rtol=5e-3, atol=1e-5)
    S0, _ = oracle.gdn_recurrence(*clean, A_log, dtb)
    S1, _ = oracle.gdn_recurrence(*other, A_log, dtb)
    f = fs.cpu().numpy().astype(np.float64)
    for got, want in ((f[0], S0[-1]), (f[1], S1[-1])):
        assert np.linalg.norm(got - want) <= 2e-5 * np.linalg.norm(want)


def test_impulse_is_one_percent_at_its_step_and_decays():
    T, Hk, Hv = 200, 2, 4
    clean, _, A_log, dtb = _inputs(2, T, Hk, Hv, 0.0)
    rs_o, _ = oracle.gdn_lockstep(clean, clean, A_log, dtb, 1, impulse_step=40, impulse_rel=0.01)
    rs, _, _ = nv.nvfp4_gdn_lockstep(_dev(clean), _dev(clean), *_dev((A_log, dtb)), 1, impulse_step=40, impulse_rel=0.01)
    got = rs.cpu().numpy()
    assert np.all(got[:40] == 0) and np.allclose(got[40], 0.01, rtol=1e-4)
    assert np.allclose(got, rs_o, rtol=2e-2, atol=2e-6)          # binary32 noise floor matters once the impulse has faded
    assert np.all(got[-1] < 0.5 * got[40])


def test_synthetic_lockstep_study_with_nvfp4_projections():
    # T tokens through the fused GDN in-projection (q 2048 | k 2048 | v 6144 | z 6144 | a 48 | b 48), once
    # exactly (float32 matmul of the bf16 operands) and once through the NVFP4 W4A4 layer
    T, K = 4096, synth.HIDDEN
    segs = synth.make_segments(synth.GDN_SEGMENTS)
    x = gu.dev_bf16(synth.prefill_activations(11, 1001, T, K))
    w = gu.dev_bf16(synth.weights(11, 1002, segs, K))
    y_ref = x.float() @ w.float().t()
    w_codes, w_sf, g_seg = nv.nvfp4_quantize_weight(w, segs)
    g_a = nv.nvfp4_calibrate(x)
    ws = nv.alloc_workspace(gu.DEV, T, 16480, K, 6, fused=True)
    y_q = nv.nvfp4_linear_bf16(x, g_a, w_codes, w_sf, segs, g_seg, ws, out_f32=True)
    assert nv.device_status(ws) == 0

    def split(y):
        def unit(t):
            return (t / t.norm(dim=-1, keepdim=True)).contiguous()
        q = unit(y[:, 0:2048].reshape(T, 16, 128))
        k = unit(y[:, 2048:4096].reshape(T, 16, 128))
        v = y[:, 4096:10240].reshape(T, 48, 128).contiguous()
        a = (0.05 * y[:, 16384:16432]).contiguous()           # gate temperature of the synthetic layer
        b = (0.05 * y[:, 16432:16480]).contiguous()
        return q, k, v, a, b

    rng = np.random.default_rng(3)
    A_log = torch.from_numpy(np.log(rng.uniform(0.002, 0.3, 48)).astype(np.float32)).to(gu.DEV)
    dtb = torch.zeros(48, dtype=torch.float32, device=gu.DEV)
    every = 256
    rs, ro, _ = nv.nvfp4_gdn_lockstep(split(y_ref), split(y_q), A_log, dtb, every)
    rel = np.median(rs.cpu().numpy(), axis=1)                   # median over heads, one value per 256 tokens
    assert 0.01 < rel[-1] < 0.6
    # the paper's finding, in shape: the error is there from the first sample on and does not accumulate
    assert rel[-1] < 1.5 * rel[0] and rel.max() < 2.0 * np.median(rel)
    # a one-off 1 % state impulse on otherwise identical inputs is forgotten
    clean = split(y_ref)
    ri, _, _ = nv.nvfp4_gdn_lockstep(clean, clean, A_log, dtb, every, impulse_step=1023, impulse_rel=0.01)
    imp = np.median(ri.cpu().numpy(), axis=1)
    assert abs(imp[3] - 0.01) < 1e-4 and np.all(imp[:3] == 0)
    assert imp[-1] < 0.3 * imp[3]
