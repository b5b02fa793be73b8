"""GPU parity: the block-scaled FP4 GEMM with per-segment global scales against the
oracle's exact GEMM, through the C ABI.  Tolerance: relative Frobenius error <= 2e-3
and the per-element bound of tests/gpu_util.check_gemm."""
import numpy as np
import pytest
import torch

import oracle
from paper_2609_04098_b200 import binding as nv
from paper_2609_04098_b200 import synth
from tests import gpu_util as gu

pytestmark = pytest.mark.gpu

VARIANTS = [128, 256, 2]


@pytest.fixture(autouse=True)
def _auto_variant():
    yield
    nv.set_gemm_variant(0)


def _ws():
    return nv.alloc_workspace(gu.DEV)


def _oracle_operands(seed, M, K, segspec, hot=2):
    segs = synth.make_segments(segspec)
    x = synth.activations(seed, 1, M, K, n_hot=min(hot, K), hot_scale=50.0)
    w = synth.weights(seed, 2, segs, K)
    ac, asf, ga, _ = gu.oracle_quantized(x)
    wc, wsf, gs, _ = gu.oracle_quantized(w, segments=segs)
    return segs, x, w, ac, asf, ga, wc, wsf, gs


def _run_from_oracle_operands(segs, ac, asf, ga, wc, wsf, gs, K, out_f32=False, ws=None):
    """Feed the ORACLE's codes and scales (re-ordered by the oracle's own layout map) to
    the GPU GEMM: a layout disagreement with the hardware shows up as a wrong product."""
    ws = ws if ws is not None else _ws()
    y = nv.nvfp4_linear(gu.dev_u8(ac), gu.dev_u8(oracle.sf_to_mma(asf, K)), gu.dev_f32(ga),
                        gu.dev_u8(wc), gu.dev_u8(oracle.sf_to_mma(wsf, K)), segs, gu.dev_f32(gs), ws,
                        out_f32=out_f32)
    assert nv.device_status(ws) == 0
    return y


@pytest.mark.parametrize("variant", VARIANTS)
@pytest.mark.parametrize("K", [64, 512, 5120])
def test_all_ones_gives_K_exactly(variant, K):
    nv.set_gemm_variant(variant)
    M, N = 130, 264
    ac = np.full((M, K // 2), 0x22, np.uint8)
    wc = np.full((N, K // 2), 0x22, np.uint8)
    asf = np.full((M, K // 16), 0x38, np.uint8)
    wsf = np.full((N, K // 16), 0x38, np.uint8)
    segs = [(0, N)]
    for f32 in (True, False):
        y = _run_from_oracle_operands(segs, ac, asf, 1.0, wc, wsf, [1.0], K, out_f32=f32)
        assert torch.all(y.float() == float(K)), (variant, K, f32)


@pytest.mark.parametrize("variant", VARIANTS)
def test_one_hot_scale_bytes_move_the_right_outputs(variant):
    # one scale byte doubled at a time: exactly one row (A) or one column (W) of the product
    # doubles its contribution from that 16-element block
    nv.set_gemm_variant(variant)
    M, N, K = 128, 256, 256
    ac = np.full((M, K // 2), 0x22, np.uint8)
    wc = np.full((N, K // 2), 0x22, np.uint8)
    for (who, r, b) in (("a", 0, 0), ("a", 37, 5), ("a", 127, 15), ("w", 1, 3), ("w", 130, 8), ("w", 255, 15)):
        asf = np.full((M, K // 16), 0x38, np.uint8)
        wsf = np.full((N, K // 16), 0x38, np.uint8)
        (asf if who == "a" else wsf)[r, b] = 0x40                       # 2.0
        y = _run_from_oracle_operands([(0, N)], ac, asf, 1.0, wc, wsf, [1.0], K, out_f32=True).cpu().numpy()
        want = np.full((M, N), float(K))
        if who == "a":
            want[r, :] += 16
        else:
            want[:, r] += 16
        assert np.array_equal(y, want), (who, r, b)


@pytest.mark.parametrize("variant", VARIANTS)
@pytest.mark.parametrize("out_f32", [False, True])
def test_config1_full_output(variant, out_f32):
    nv.set_gemm_variant(variant)
    x, w, segs = synth.config1(0)
    ac, asf, ga, _ = gu.oracle_quantized(x)
    wc, wsf, gs, _ = gu.oracle_quantized(w, segments=segs)
    gcol = oracle.col_scales(256, segs, gs)
    y_ref = oracle.gemm(ac, asf, ga, wc, wsf, gcol)
    # whole GPU path: calibrate + quantize + GEMM on the device
    xt, wt = gu.dev_bf16(x), gu.dev_bf16(w)
    g_a = nv.nvfp4_calibrate(xt)
    a_codes, a_sf = nv.nvfp4_quantize_act(xt, g_a)
    w_codes, w_sf, g_seg = nv.nvfp4_quantize_weight(wt, segs)
    ws = _ws()
    y = nv.nvfp4_linear(a_codes, a_sf, g_a, w_codes, w_sf, segs, g_seg, ws, out_f32=out_f32)
    assert nv.device_status(ws) == 0
    gu.check_gemm(y, y_ref, gu.gemm_bounds(ac, asf, ga, wc, wsf, gcol), "config1")
    # and from the oracle's operands
    y2 = _run_from_oracle_operands(segs, ac, asf, ga, wc, wsf, gs, 512, out_f32=out_f32)
    assert torch.equal(y, y2)


@pytest.mark.parametrize("variant", VARIANTS)
@pytest.mark.parametrize("M,N,K", [(1, 48, 64), (16, 130, 192), (129, 272, 320), (200, 520, 1088),
                                   (128, 50, 256), (257, 16480 // 8, 576)])
def test_ragged_shapes(variant, M, N, K):
    nv.set_gemm_variant(variant)
    n1 = max(1, N // 3)
    segs, x, w, ac, asf, ga, wc, wsf, gs = _oracle_operands(11, M, K, (("p", n1, 0.02), ("q", N - n1, 0.2)))
    gcol = oracle.col_scales(N, segs, gs)
    y_ref = oracle.gemm(ac, asf, ga, wc, wsf, gcol)
    bound = gu.gemm_bounds(ac, asf, ga, wc, wsf, gcol)
    for f32 in (False, True):            # N % 8 != 0 exercises the scalar store path
        y = _run_from_oracle_operands(segs, ac, asf, ga, wc, wsf, gs, K, out_f32=f32)
        gu.check_gemm(y, y_ref, bound, "ragged %s" % ((M, N, K),))


def test_output_padding_is_untouched():
    # ldy > N: the columns between N and ldy must keep their canary
    M, N, K = 70, 200, 256
    segs, x, w, ac, asf, ga, wc, wsf, gs = _oracle_operands(12, M, K, (("p", N, 0.02),))
    out = torch.full((M + 3, N + 24), 7.0, dtype=torch.bfloat16, device=gu.DEV)
    ws = _ws()
    nv.nvfp4_linear(gu.dev_u8(ac), gu.dev_u8(oracle.sf_to_mma(asf, K)), gu.dev_f32(ga), gu.dev_u8(wc),
                    gu.dev_u8(oracle.sf_to_mma(wsf, K)), segs, gu.dev_f32(gs), ws, out=out[:M, :N])
    assert nv.device_status(ws) == 0
    assert torch.all(out[:, N:] == 7.0) and torch.all(out[M:, :] == 7.0)
    y_ref = oracle.gemm(ac, asf, ga, wc, wsf, oracle.col_scales(N, segs, gs))
    gu.check_gemm(out[:M, :N].contiguous(), y_ref, gu.gemm_bounds(ac, asf, ga, wc, wsf, oracle.col_scales(N, segs, gs)))


@pytest.mark.parametrize("variant", VARIANTS)
def test_segment_epilogue_and_single_scale_defect(variant):
    # small copy of the fused GDN in-projection: boundaries inside one tile, tiny segments
    nv.set_gemm_variant(variant)
    spec = (("q", 64, 0.02), ("k", 64, 0.02), ("v", 192, 0.02), ("z", 192, 0.02), ("a", 48, 0.2), ("b", 48, 0.2))
    M, K = 256, 512
    segs, x, w, ac, asf, ga, wc, wsf, gs = _oracle_operands(13, M, K, spec)
    N = 608
    gcol = oracle.col_scales(N, segs, gs)
    y_ref = oracle.gemm(ac, asf, ga, wc, wsf, gcol)
    y = _run_from_oracle_operands(segs, ac, asf, ga, wc, wsf, gs, K, out_f32=True)
    gu.check_gemm(y, y_ref, gu.gemm_bounds(ac, asf, ga, wc, wsf, gcol), "gdn-small")
    # doubling one segment's scale doubles that segment bit-exactly and nothing else
    gs2 = np.array(gs, dtype=np.float32)
    gs2[4] *= 2
    y2 = _run_from_oracle_operands(segs, ac, asf, ga, wc, wsf, gs2, K, out_f32=True)
    b, e = segs[4].begin, segs[4].begin + segs[4].count
    assert torch.equal(y2[:, b:e], 2 * y[:, b:e])
    assert torch.equal(y2[:, :b], y[:, :b]) and torch.equal(y2[:, e:], y[:, e:])
    # the defect: one global scale (max of the constituents) for the whole fused GEMM
    gmax = float(np.max(gs))
    y_bad = _run_from_oracle_operands([(0, N)], ac, asf, ga, wc, wsf, [gmax], K, out_f32=True).cpu().numpy()
    yg = y.cpu().numpy()
    for s, g in zip(segs, gs):
        sl = slice(s.begin, s.begin + s.count)
        rel = np.linalg.norm(y_bad[:, sl] - yg[:, sl]) / np.linalg.norm(yg[:, sl])
        assert abs(rel - abs(gmax / float(g) - 1.0)) < 1e-5, s.name


def test_fused_entry_point_equals_two_step_path():
    M, K = 300, 1024
    segs = synth.make_segments((("p", 200, 0.02), ("q", 120, 0.2)))
    x = synth.prefill_activations(5, 1, M, K)
    w = synth.weights(5, 2, segs, K)
    xt = gu.dev_bf16(x)
    g_a = nv.nvfp4_calibrate(xt)
    w_codes, w_sf, g_seg = nv.nvfp4_quantize_weight(gu.dev_bf16(w), segs)
    a_codes, a_sf = nv.nvfp4_quantize_act(xt, g_a)
    ws = _ws()
    y1 = nv.nvfp4_linear(a_codes, a_sf, g_a, w_codes, w_sf, segs, g_seg, ws)
    ws2 = nv.alloc_workspace(gu.DEV, M, 320, K, 2, fused=True)
    y2 = nv.nvfp4_linear_bf16(xt, g_a, w_codes, w_sf, segs, g_seg, ws2)
    assert nv.device_status(ws) == 0 and nv.device_status(ws2) == 0
    assert torch.equal(y1, y2)


@pytest.mark.parametrize("variant", VARIANTS)
def test_gdn_in_projection_full_size_sampled(variant):
    # M=8192, K=5120, N=16480 in six segments; the oracle computes sampled rows and
    # columns, and a random-sign projection covers every tile
    nv.set_gemm_variant(variant)
    M, K = 8192, synth.HIDDEN
    segs = synth.make_segments(synth.GDN_SEGMENTS)
    N = 16480
    x = synth.prefill_activations(0, 401, M, K)
    w = synth.weights(0, 402, segs, K)
    ac, asf, ga, _ = gu.oracle_quantized(x)
    wc, wsf, gs, _ = gu.oracle_quantized(w, segments=segs)
    gcol = oracle.col_scales(N, segs, gs)
    xt, wt = gu.dev_bf16(x), gu.dev_bf16(w)
    g_a = nv.nvfp4_calibrate(xt)
    a_codes, a_sf = nv.nvfp4_quantize_act(xt, g_a)
    w_codes, w_sf, g_seg = nv.nvfp4_quantize_weight(wt, segs)
    gu.check_quantized(a_codes, a_sf, nv.SF_MMA, ac, asf, K)
    gu.check_quantized(w_codes, w_sf, nv.SF_MMA, wc, wsf, K)
    ws = _ws()
    y = nv.nvfp4_linear(a_codes, a_sf, g_a, w_codes, w_sf, segs, g_seg, ws)
    assert nv.device_status(ws) == 0
    rng = np.random.default_rng(0)
    rows = np.sort(np.array([t * 128 + rng.integers(0, 128) for t in range(0, M // 128, 4)] + [0, M - 1]))
    y_rows = oracle.gemm(ac, asf, ga, wc, wsf, gcol, rows=rows)
    gu.check_gemm(y[torch.from_numpy(rows).to(gu.DEV)], y_rows,
                  gu.gemm_bounds(ac, asf, ga, wc, wsf, gcol, rows=rows), "gdn rows")
    edge = sorted({c for s in segs for c in (s.begin, s.begin + s.count - 1)} | {N - 1, 0})
    cols = np.array(sorted(set(edge) | set(rng.integers(0, N, 24).tolist())))
    y_cols = oracle.gemm(ac, asf, ga, wc, wsf, gcol, cols=cols)
    gu.check_gemm(y[:, torch.from_numpy(cols).to(gu.DEV)].contiguous(), y_cols,
                  gu.gemm_bounds(ac, asf, ga, wc, wsf, gcol, cols=cols), "gdn cols")
    # Freivalds-style projection over the whole output: Y r against A_hat (W_hat^T r) in float64
    r = rng.choice([-1.0, 1.0], N)
    a_hat = oracle.dequantize(ac, asf, oracle.row_scales(M, g=ga))
    w_hat = oracle.dequantize(wc, wsf, gcol)
    want = a_hat @ (w_hat.T @ r)
    got = y.double().cpu().numpy() @ r
    scale = np.linalg.norm(a_hat, axis=1) * np.linalg.norm(w_hat) / np.sqrt(K)
    # bf16 rounding of N outputs: random-walk error ~ 2^-9 * |y| * sqrt(N)
    assert np.max(np.abs(got - want) / scale) < 2e-2


# ---- decode-sized batches: split-K over a self-cleaning workspace -----------------------------
@pytest.mark.parametrize("M,N,K", [(1, 6144, 5120), (16, 520, 8192), (100, 2064, 8448), (128, 1000, 9216), (3, 136, 17408)])
@pytest.mark.parametrize("out_f32", [False, True])
def test_small_m_split_k(M, N, K, out_f32):
    n1 = N // 3
    segs, x, w, ac, asf, ga, wc, wsf, gs = _oracle_operands(17, M, K, (("p", n1, 0.02), ("q", N - n1, 0.2)))
    gcol = oracle.col_scales(N, segs, gs)
    y_ref = oracle.gemm(ac, asf, ga, wc, wsf, gcol)
    bound = gu.gemm_bounds(ac, asf, ga, wc, wsf, gcol)
    ws = nv.alloc_workspace(gu.DEV, M, N, K, 2)            # zero-filled, large enough for the split-K area
    assert ws.numel() > 256
    first = None
    for _ in range(3):                                      # the same workspace every time: it must come back clean
        y = _run_from_oracle_operands(segs, ac, asf, ga, wc, wsf, gs, K, out_f32=out_f32, ws=ws)
        gu.check_gemm(y, y_ref, bound, "split-K %s" % ((M, N, K),))
        if first is None:
            first = y.clone()
        elif out_f32:
            # fp32 atomics add in arrival order: equal up to summation order
            assert torch.allclose(y, first, rtol=1e-5, atol=1e-6 * float(first.abs().max()))
    assert bool((ws[256:] == 0).all())                     # counters and partial sums left at zero
    # and the one-tile-per-CTA kernel gives the same answer (within summation order)
    y1 = _run_from_oracle_operands(segs, ac, asf, ga, wc, wsf, gs, K, out_f32=out_f32)    # 256-byte workspace: no split
    gu.check_gemm(y1, y_ref, bound, "no split")


# ---- the benchmark's own shapes at full size (whole device path, auto tile choice) ------------
def _full_size_sampled(M, K, spec, seed, n_rows=16, n_cols=24):
    """Device path end to end (calibrate, quantize, GEMM) at full size; the oracle checks the
    quantized operands in full, the GEMM on sampled rows, sampled columns (every segment edge and
    the last column among them) and a random-sign projection of the whole output."""
    segs = synth.make_segments(spec)
    N = sum(s.count for s in segs)
    x = synth.prefill_activations(seed, 501, M, K)
    w = synth.weights(seed, 502, segs, K)
    ac, asf, ga, _ = gu.oracle_quantized(x)
    wc, wsf, gs, _ = gu.oracle_quantized(w, segments=segs)
    gcol = oracle.col_scales(N, segs, gs)
    xt, wt = gu.dev_bf16(x), gu.dev_bf16(w)
    g_a = nv.nvfp4_calibrate(xt)
    a_codes, a_sf = nv.nvfp4_quantize_act(xt, g_a)
    w_codes, w_sf, g_seg = nv.nvfp4_quantize_weight(wt, segs)
    del xt, wt
    gu.check_quantized(a_codes, a_sf, nv.SF_MMA, ac, asf, K)
    gu.check_quantized(w_codes, w_sf, nv.SF_MMA, wc, wsf, K)
    ws = _ws()
    y = nv.nvfp4_linear(a_codes, a_sf, g_a, w_codes, w_sf, segs, g_seg, ws)
    assert nv.device_status(ws) == 0
    rng = np.random.default_rng(seed)
    step = max(1, (M // 128) // n_rows)
    rows = np.unique(np.array([t * 128 + rng.integers(0, 128) for t in range(0, M // 128, step)] + [0, M - 1]))
    y_rows = oracle.gemm(ac, asf, ga, wc, wsf, gcol, rows=rows)
    gu.check_gemm(y[torch.from_numpy(rows).to(gu.DEV)], y_rows,
                  gu.gemm_bounds(ac, asf, ga, wc, wsf, gcol, rows=rows), "rows")
    edge = {c for s in segs for c in (s.begin, s.begin + s.count - 1)} | {0, N - 1}
    cols = np.array(sorted(edge | set(rng.integers(0, N, n_cols).tolist())))
    y_cols = oracle.gemm(ac, asf, ga, wc, wsf, gcol, cols=cols)
    gu.check_gemm(y[:, torch.from_numpy(cols).to(gu.DEV)].contiguous(), y_cols,
                  gu.gemm_bounds(ac, asf, ga, wc, wsf, gcol, cols=cols), "cols")
    # projection of the whole output on a random sign vector, operands dequantized in row chunks
    r = rng.choice([-1.0, 1.0], N)
    wr = np.zeros(K)
    w_norm2 = 0.0
    for b in range(0, N, 4096):
        w_hat = oracle.dequantize(wc[b:b + 4096], wsf[b:b + 4096], gcol[b:b + 4096])
        wr += w_hat.T @ r[b:b + 4096]
        w_norm2 += float((w_hat ** 2).sum())
    worst = 0.0
    r_dev = torch.from_numpy(r).to(gu.DEV)
    got = (y.double() @ r_dev).cpu().numpy()
    for b in range(0, M, 2048):
        a_hat = oracle.dequantize(ac[b:b + 2048], asf[b:b + 2048], oracle.row_scales(min(2048, M - b), g=ga))
        want = a_hat @ wr
        scale = np.linalg.norm(a_hat, axis=1) * np.sqrt(w_norm2) / np.sqrt(K)
        worst = max(worst, float(np.max(np.abs(got[b:b + 2048] - want) / scale)))
    assert worst < 2e-2, worst


def test_mlp_gate_up_full_size_sampled():
    _full_size_sampled(8192, synth.HIDDEN, (("gate", synth.MLP_INNER, 0.02), ("up", synth.MLP_INNER, 0.02)), 1)


def test_mlp_down_full_size_sampled():
    _full_size_sampled(8192, synth.MLP_INNER, (("down", synth.HIDDEN, 0.02),), 2)


def test_long_prefill_32k_tokens_sampled():
    _full_size_sampled(32768, synth.HIDDEN, (("w", 6144, 0.02),), 3, n_rows=32)


# ---- 1 or 2 tokens: the weight-streaming decode kernel behind nvfp4_linear_bf16 (3, 4: tensor cores) ------------------
@pytest.mark.parametrize("M", [1, 2, 3, 4])
@pytest.mark.parametrize("N,K", [(6144, 5120), (1000, 1088), (5120, 17408), (50, 64)])
@pytest.mark.parametrize("out_f32", [False, True])
def test_decode_batches(M, N, K, out_f32):
    n1 = max(1, N // 3)
    segs = synth.make_segments((("p", n1, 0.02), ("q", N - n1, 0.2)))
    x = synth.activations(19, 1, M, K, n_hot=2, hot_scale=50.0)
    w = synth.weights(19, 2, segs, K)
    ac, asf, ga, _ = gu.oracle_quantized(x)
    wc, wsf, gs, _ = gu.oracle_quantized(w, segments=segs)
    gcol = oracle.col_scales(N, segs, gs)
    y_ref = oracle.gemm(ac, asf, ga, wc, wsf, gcol)
    ws = nv.alloc_workspace(gu.DEV, M, N, K, 2, fused=True)
    launches = nv.launch_count()
    y = nv.nvfp4_linear_bf16(gu.dev_bf16(x), gu.dev_f32(ga), gu.dev_u8(wc), gu.dev_u8(oracle.sf_to_mma(wsf, K)), segs,
                             gu.dev_f32(gs), ws, out_f32=out_f32)
    torch.cuda.synchronize()
    assert nv.launch_count() - launches == (1 if M <= 2 else 2)     # 1-2 tokens: one kernel, quantization included
    gu.check_gemm(y, y_ref, gu.gemm_bounds(ac, asf, ga, wc, wsf, gcol), "decode %s" % ((M, N, K),))
    if out_f32 and M <= 2:
        # no output rounding and exact block sums: only fp32 accumulation order separates it from the oracle
        assert np.max(np.abs(y.cpu().numpy().astype(np.float64) - y_ref)) <= 2e-6 * np.max(np.abs(y_ref)) + 1e-30
    # the tensor-core path (forced) agrees within the same bounds
    nv.set_gemm_variant(128)
    y2 = nv.nvfp4_linear_bf16(gu.dev_bf16(x), gu.dev_f32(ga), gu.dev_u8(wc), gu.dev_u8(oracle.sf_to_mma(wsf, K)), segs,
                              gu.dev_f32(gs), ws, out_f32=out_f32)
    nv.set_gemm_variant(0)
    gu.check_gemm(y2, y_ref, gu.gemm_bounds(ac, asf, ga, wc, wsf, gcol), "tensor-core path")
