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


def _run_from_oracle_operands(segs, ac, asf, ga, wc, wsf, gs, K, out_f32=False, ws=None, w_resident=False):
    """Feed the ORACLE's codes and scales (re-ordered by the oracle's own layout map) to
    the GPU GEMM: a layout disagreement with the hardware shows up as a wrong product."""
    ws = ws if ws is not None else _ws()
    y = nv.nvfp4_linear(gu.dev_u8(ac), gu.dev_u8(oracle.sf_to_mma(asf, K)), gu.dev_f32(ga),
                        gu.dev_u8(wc), gu.dev_u8(oracle.sf_to_mma(wsf, K)), segs, gu.dev_f32(gs), ws,
                        out_f32=out_f32, w_resident=w_resident)
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
    _check_sampled(y, M, N, K, segs, ac, asf, ga, wc, wsf, gcol, np.random.default_rng(0), "gdn")


# ---- decode-sized batches: K shared by the CTAs of a cluster, or split over a self-cleaning workspace ----
# automatic choice: clusters whose CTAs meet in shared memory (every shape below has few enough tiles);
# variant 128 forced: one CTA per tile, K split through the workspace where K is long enough
@pytest.mark.parametrize("M,N,K", [(1, 6144, 5120), (16, 520, 8192), (33, 1100, 5120), (64, 6144, 5120), (100, 2064, 8448),
                                   (128, 1000, 9216), (3, 136, 17408), (7, 128, 512)])
@pytest.mark.parametrize("out_f32", [False, True])
@pytest.mark.parametrize("variant", [0, 128])
def test_small_m_split_k(M, N, K, out_f32, variant):
    nv.set_gemm_variant(variant)
    n1 = N // 3
    segs, x, w, ac, asf, ga, wc, wsf, gs = _oracle_operands(17, M, K, (("p", n1, 0.02), ("q", N - n1, 0.2)))
    gcol = oracle.col_scales(N, segs, gs)
    y_ref = oracle.gemm(ac, asf, ga, wc, wsf, gcol)
    bound = gu.gemm_bounds(ac, asf, ga, wc, wsf, gcol)
    ws = nv.alloc_workspace(gu.DEV, M, N, K, 2)            # zero-filled, large enough for the split-K area
    assert ws.numel() > 256
    first = None
    for rep in range(3):                                    # the same workspace every time: it must come back clean
        y = _run_from_oracle_operands(segs, ac, asf, ga, wc, wsf, gs, K, out_f32=out_f32, ws=ws, w_resident=rep == 2)
        gu.check_gemm(y, y_ref, bound, "split-K %s" % ((M, N, K),))
        if first is None:
            first = y.clone()
        elif variant == 0:
            assert torch.equal(y, first)                    # the cluster adds its partial sums in a fixed order
        elif out_f32:
            # fp32 atomics add in arrival order: equal up to summation order
            assert torch.allclose(y, first, rtol=1e-5, atol=1e-6 * float(first.abs().max()))
    assert bool((ws[256:] == 0).all())                     # counters and partial sums left at zero
    # and the one-tile-per-CTA kernel gives the same answer (within summation order)
    nv.set_gemm_variant(128)
    y1 = _run_from_oracle_operands(segs, ac, asf, ga, wc, wsf, gs, K, out_f32=out_f32)    # 256-byte workspace: no split
    nv.set_gemm_variant(0)
    gu.check_gemm(y1, y_ref, bound, "no split")


# ---- the benchmark's own shapes at full size (whole device path, auto tile choice) ------------
def _sample_rows_cols(M, N, segs, rng, n_cols=64):
    """One row inside every 128-row band (plus the first and last row); at least `n_cols` columns,
    among them both neighbours of every segment edge and the last column."""
    rows = np.unique(np.array([t * 128 + rng.integers(0, min(128, M - t * 128)) for t in range((M + 127) // 128)]
                              + [0, M - 1]))
    edge = set()
    for s_ in segs:
        for c in (s_.begin - 1, s_.begin, s_.begin + s_.count - 1, s_.begin + s_.count):
            if 0 <= c < N:
                edge.add(int(c))
    edge |= {0, N - 1}
    extra = set(rng.integers(0, N, max(0, n_cols - len(edge)) + 8).tolist())
    cols = np.array(sorted(edge | extra))
    assert len(cols) >= min(n_cols, N)
    return rows, cols


def _check_sampled(y, M, N, K, segs, ac, asf, ga, wc, wsf, gcol, rng, what):
    """Oracle comparison of a full-size output on sampled rows and columns plus a random-sign
    projection of the whole output (operands dequantized in chunks)."""
    rows, cols = _sample_rows_cols(M, N, segs, rng)
    y_rows = oracle.gemm(ac, asf, ga, wc, wsf, gcol, rows=rows)
    gu.check_gemm(y[torch.from_numpy(rows).to(gu.DEV)], y_rows,
                  gu.gemm_bounds(ac, asf, ga, wc, wsf, gcol, rows=rows), what + " rows")
    y_cols = oracle.gemm(ac, asf, ga, wc, wsf, gcol, cols=cols)
    gu.check_gemm(y[:, torch.from_numpy(cols).to(gu.DEV)].contiguous(), y_cols,
                  gu.gemm_bounds(ac, asf, ga, wc, wsf, gcol, cols=cols), what + " cols")
    r = rng.choice([-1.0, 1.0], N)
    wr = np.zeros(K)
    w_norm2 = 0.0
    for b in range(0, N, 4096):
        w_hat = oracle.dequantize(wc[b:b + 4096], wsf[b:b + 4096], gcol[b:b + 4096])
        wr += w_hat.T @ r[b:b + 4096]
        w_norm2 += float((w_hat ** 2).sum())
    worst = 0.0
    got = (y.double() @ torch.from_numpy(r).to(gu.DEV)).cpu().numpy()
    for b in range(0, M, 2048):
        a_hat = oracle.dequantize(ac[b:b + 2048], asf[b:b + 2048], oracle.row_scales(min(2048, M - b), g=ga))
        want = a_hat @ wr
        scale = np.linalg.norm(a_hat, axis=1) * np.sqrt(w_norm2) / np.sqrt(K)
        worst = max(worst, float(np.max(np.abs(got[b:b + 2048] - want) / scale)))
    # bf16 rounding of N outputs: random-walk error ~ 2^-9 * |y| * sqrt(N)
    assert worst < 2e-2, (what, worst)


def _full_size_sampled(M, K, spec, seed):
    """Device path end to end (calibrate, quantize, GEMM) at full size; the oracle checks the
    quantized operands in full and the GEMM as _check_sampled describes."""
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
    _check_sampled(y, M, N, K, segs, ac, asf, ga, wc, wsf, gcol, np.random.default_rng(seed), "full size %s" % ((M, N, K),))


def test_mlp_gate_up_full_size_sampled():
    _full_size_sampled(8192, synth.HIDDEN, (("gate", synth.MLP_INNER, 0.02), ("up", synth.MLP_INNER, 0.02)), 1)


def test_mlp_down_full_size_sampled():
    _full_size_sampled(8192, synth.MLP_INNER, (("down", synth.HIDDEN, 0.02),), 2)


def test_long_prefill_32k_tokens_sampled():
    _full_size_sampled(32768, synth.HIDDEN, (("w", 6144, 0.02),), 3)


# ---- 1 token (2 where K is not a multiple of 256): the weight-streaming decode kernel behind nvfp4_linear_bf16; up to
# 8 tokens (K a multiple of 256): one tensor-core kernel that quantizes the activations itself; otherwise quantize
# kernel + GEMM
@pytest.mark.parametrize("M", [1, 2, 3, 4, 8, 9, 16, 17])
@pytest.mark.parametrize("N,K", [(6144, 5120), (1000, 1088), (5120, 17408), (50, 64), (34816, 512), (300, 256), (129, 768)])
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
    assert nv.launch_count() - launches == (1 if M <= 2 or (M <= 8 and K % 256 == 0) else 2)
    gu.check_gemm(y, y_ref, gu.gemm_bounds(ac, asf, ga, wc, wsf, gcol), "decode %s" % ((M, N, K),))
    if out_f32 and (M == 1 or (M == 2 and K % 256 != 0)):             # the weight-streaming kernel
        # no output rounding and exact block sums: only fp32 accumulation order separates it from the oracle
        assert np.max(np.abs(y.cpu().numpy().astype(np.float64) - y_ref)) <= 2e-6 * np.max(np.abs(y_ref)) + 1e-30
    # the tensor-core path (forced) agrees within the same bounds
    nv.set_gemm_variant(128)
    y2 = nv.nvfp4_linear_bf16(gu.dev_bf16(x), gu.dev_f32(ga), gu.dev_u8(wc), gu.dev_u8(oracle.sf_to_mma(wsf, K)), segs,
                              gu.dev_f32(gs), ws, out_f32=out_f32)
    nv.set_gemm_variant(0)
    gu.check_gemm(y2, y_ref, gu.gemm_bounds(ac, asf, ga, wc, wsf, gcol), "tensor-core path")


# ---- the M sweep's own entry point: quantize inside the call, K=5120 -> N=6144 -----------------
@pytest.mark.parametrize("M", [16, 128, 1024, 8192])
def test_m_sweep_layer_through_the_fused_entry_point(M):
    K, N = synth.HIDDEN, 6144
    segs = synth.make_segments((("w", N, 0.02),))
    x = synth.prefill_activations(7, 601, M, K)
    w = synth.weights(7, 602, segs, K)
    ac, asf, ga, _ = gu.oracle_quantized(x)
    wc, wsf, gs, _ = gu.oracle_quantized(w, segments=segs)
    gcol = oracle.col_scales(N, segs, gs)
    ws = nv.alloc_workspace(gu.DEV, M, N, K, 1, fused=True)
    y = nv.nvfp4_linear_bf16(gu.dev_bf16(x), gu.dev_f32(ga), gu.dev_u8(wc), gu.dev_u8(oracle.sf_to_mma(wsf, K)), segs,
                             gu.dev_f32(gs), ws)
    assert nv.device_status(ws) == 0
    if M <= 1024:
        gu.check_gemm(y, oracle.gemm(ac, asf, ga, wc, wsf, gcol), gu.gemm_bounds(ac, asf, ga, wc, wsf, gcol), "M=%d" % M)
    else:
        _check_sampled(y, M, N, K, segs, ac, asf, ga, wc, wsf, gcol, np.random.default_rng(M), "M=%d" % M)
    assert bool((ws[256:256 + nv.SPLIT_RESERVE_BYTES] == 0).all())


# ---- one workspace across layers of different K: the split-K part sits at a fixed place ---------
def _decode_layer(seed, M, N, K):
    segs = synth.make_segments((("w", N, 0.02),))
    x = synth.prefill_activations(seed, 701, M, K)
    w = synth.weights(seed, 702, segs, K)
    ac, asf, ga, _ = gu.oracle_quantized(x)
    wc, wsf, gs, _ = gu.oracle_quantized(w, segments=segs)
    gcol = oracle.col_scales(N, segs, gs)
    y_ref = oracle.gemm(ac, asf, ga, wc, wsf, gcol)
    bound = gu.gemm_bounds(ac, asf, ga, wc, wsf, gcol)
    dev = (gu.dev_bf16(x), gu.dev_f32(ga), gu.dev_u8(wc), gu.dev_u8(oracle.sf_to_mma(wsf, K)), segs, gu.dev_f32(gs))
    return dev, y_ref, bound


def test_one_workspace_reused_across_layers_of_different_k():
    # the model's own pair: K = 5120 (no split-K) and K = 17408 (split-K), alternating on one
    # zero-filled workspace sized for the larger; every result against the oracle
    M = 16
    a, a_ref, a_bound = _decode_layer(31, M, 6144, synth.HIDDEN)
    b, b_ref, b_bound = _decode_layer(32, M, synth.HIDDEN, synth.MLP_INNER)
    big, big_ref, big_bound = _decode_layer(33, 200, 1024, 8192)          # many rows: codes reach far into the workspace
    small, small_ref, small_bound = _decode_layer(34, 16, 6144, 8192)      # split-K again after it
    n = max(nv.lib().nvfp4_linear_bf16_workspace_bytes(m, nn, k, 1)
            for (m, nn, k) in ((M, 6144, synth.HIDDEN), (M, synth.HIDDEN, synth.MLP_INNER), (200, 1024, 8192), (16, 6144, 8192)))
    ws = torch.zeros(int(n), dtype=torch.uint8, device=gu.DEV)
    for dev, ref, bound, what in ((a, a_ref, a_bound, "K=5120"), (b, b_ref, b_bound, "K=17408"),
                                  (big, big_ref, big_bound, "M=200 K=8192"), (small, small_ref, small_bound, "M=16 K=8192"),
                                  (a, a_ref, a_bound, "K=5120 again"), (b, b_ref, b_bound, "K=17408 again")):
        y = nv.nvfp4_linear_bf16(*dev, ws)
        assert nv.device_status(ws) == 0, what
        gu.check_gemm(y, ref, bound, what)
        assert bool((ws[256:256 + nv.SPLIT_RESERVE_BYTES] == 0).all()), what      # split-K part left at zero


def test_bad_global_scale_is_reported_on_the_device():
    # g must be finite and > 0: the kernel reports it in the status word instead of repairing it
    M, N, K = 64, 256, 256
    segs, x, w, ac, asf, ga, wc, wsf, gs = _oracle_operands(41, M, K, (("p", 128, 0.02), ("q", 128, 0.2)))
    for bad_ga, bad_gs in ((0.0, gs), (float("inf"), gs), (ga, [gs[0], -1.0]), (ga, [float("nan"), gs[1]])):
        ws = _ws()
        nv.nvfp4_linear(gu.dev_u8(ac), gu.dev_u8(oracle.sf_to_mma(asf, K)), gu.dev_f32(bad_ga), gu.dev_u8(wc),
                        gu.dev_u8(oracle.sf_to_mma(wsf, K)), segs, gu.dev_f32(bad_gs), ws)
        assert nv.device_status(ws) == 10
    # the decode kernel (1 token, bf16 in) reports it too
    ws = nv.alloc_workspace(gu.DEV, 1, N, K, 2, fused=True)
    nv.nvfp4_linear_bf16(gu.dev_bf16(x[:1]), gu.dev_f32(0.0), gu.dev_u8(wc), gu.dev_u8(oracle.sf_to_mma(wsf, K)), segs,
                         gu.dev_f32(gs), ws)
    assert nv.device_status(ws) == 10
    ws = _ws()
    y = _run_from_oracle_operands(segs, ac, asf, ga, wc, wsf, gs, K, ws=ws)       # good scales: status stays 0
    gu.check_gemm(y, oracle.gemm(ac, asf, ga, wc, wsf, oracle.col_scales(N, segs, gs)),
                  gu.gemm_bounds(ac, asf, ga, wc, wsf, oracle.col_scales(N, segs, gs)), "good scales")


# ---- the MLP as served: gate/up GEMM -> silu(gate)*up quantized by the producer-fused kernel -> down GEMM ----
def test_mlp_chain_with_fused_producer_link_by_link():
    M, K, INNER = 8192, synth.HIDDEN, synth.MLP_INNER
    seg_gu = synth.make_segments((("gate", INNER, 0.02), ("up", INNER, 0.02)))
    seg_d = synth.make_segments((("down", K, 0.02),))
    x = synth.prefill_activations(5, 801, M, K)
    w_gu = synth.weights(5, 802, seg_gu, K)
    w_d = synth.weights(5, 803, seg_d, INNER)
    ac, asf, ga, _ = gu.oracle_quantized(x)
    wgc, wgsf, ggs, _ = gu.oracle_quantized(w_gu, segments=seg_gu)
    wdc, wdsf, gds, _ = gu.oracle_quantized(w_d, segments=seg_d)
    gcol_gu = oracle.col_scales(2 * INNER, seg_gu, ggs)
    gcol_d = oracle.col_scales(K, seg_d, gds)
    rng = np.random.default_rng(5)
    rows = np.unique(np.array([t * 128 + rng.integers(0, 128) for t in range(M // 128)] + [0, M - 1]))
    rows_t = torch.from_numpy(rows).to(gu.DEV)
    # device chain
    xt = gu.dev_bf16(x)
    g1 = gu.dev_f32(ga)
    q1 = nv.nvfp4_quantize_act(xt, g1)
    w_gu_c, w_gu_sf, g_gu = nv.nvfp4_quantize_weight(gu.dev_bf16(w_gu), seg_gu)
    w_d_c, w_d_sf, g_d = nv.nvfp4_quantize_weight(gu.dev_bf16(w_d), seg_d)
    ws = _ws()
    y1 = nv.nvfp4_linear(q1[0], q1[1], g1, w_gu_c, w_gu_sf, seg_gu, g_gu, ws)
    # link 1: gate/up GEMM rows against the exact GEMM
    y1_rows_ref = oracle.gemm(ac, asf, ga, wgc, wgsf, gcol_gu, rows=rows)
    gu.check_gemm(y1[rows_t], y1_rows_ref, gu.gemm_bounds(ac, asf, ga, wgc, wgsf, gcol_gu, rows=rows), "gate/up rows")
    # the activation scale of h is static (offline calibration): here from the definition on the sampled rows
    y1_rows_bits = gu.host_bits(y1[rows_t].contiguous())
    h_rows_def = oracle.swiglu_bf16(y1_rows_bits)
    _, gh = oracle.calibrate(h_rows_def)
    gh = np.float32(gh * 2.0)                                              # head-room for the rows not sampled
    g2 = gu.dev_f32(gh)
    h_d = torch.empty((M, INNER), dtype=torch.bfloat16, device=gu.DEV)
    q2 = nv.nvfp4_swiglu_quantize(y1, g2, h_out=h_d)
    y2 = nv.nvfp4_linear(q2[0], q2[1], g2, w_d_c, w_d_sf, seg_d, g_d, ws)
    assert nv.device_status(ws) == 0
    # link 2: h the kernel formed against the definition applied to the device's own gate/up rows
    h_rows_gpu = gu.host_bits(h_d[rows_t].contiguous())
    gu.check_bf16_close_to_definition(h_rows_gpu, h_rows_def, 0.995, "h rows")
    # link 3: codes and scales bit-exact against the oracle's quantization of that h
    hc, hsf = oracle.quantize(h_rows_gpu, oracle.row_scales(len(rows), g=gh))
    sf_lin, pad_zero = oracle.sf_from_mma(q2[1].cpu().numpy(), M, INNER)
    assert pad_zero
    assert np.array_equal(q2[0][rows_t].cpu().numpy(), hc) and np.array_equal(sf_lin[rows], hsf)
    # link 4: down GEMM rows against the exact GEMM on those codes
    y2_rows_ref = oracle.gemm(hc, hsf, gh, wdc, wdsf, gcol_d)
    bound = gu.gemm_bounds(hc, hsf, gh, wdc, wdsf, gcol_d)
    gu.check_gemm(y2[rows_t], y2_rows_ref, bound, "down rows")
    # end to end: the oracle's own chain (exact GEMM -> bf16 -> definition -> quantize -> exact GEMM) on the
    # same rows; the device differs where a gate/up output or an h rounded the other way (rare, one ulp)
    y1_bits_ref = oracle.f64_to_bf16_bits(y1_rows_ref)
    h_ref = oracle.swiglu_bf16(y1_bits_ref)
    hc_ref, hsf_ref = oracle.quantize(h_ref, oracle.row_scales(len(rows), g=gh))
    y2_chain_ref = oracle.gemm(hc_ref, hsf_ref, gh, wdc, wdsf, gcol_d)
    got = oracle.bf16_bits_to_f64(gu.host_bits(y2[rows_t].contiguous()))
    assert np.linalg.norm(got - y2_chain_ref) / np.linalg.norm(y2_chain_ref) <= 3e-3
    assert (hc_ref == hc).mean() > 0.999


# ---- kernels that start under their predecessor: a chain of dependent layers, back to back ----------------
# Every GEMM releases the kernel behind it at once and, with the weights flagged resident, fetches weights
# while the kernel in front still runs; what it reads from (and writes over) its predecessors is ordered by
# waits inside the kernels.  A chain in which each layer's input IS the previous layer's output, run back to
# back on a stream and as a CUDA-graph replay, must give bit for bit what the same chain gives with a device
# synchronisation after every call -- an ordering mistake shows up as a changed result.
@pytest.mark.parametrize("M", [1, 4, 64, 300])
def test_dependent_chain_back_to_back_equals_synchronised(M):
    K = 2048                                       # square layers: each output feeds the next call
    depth = 8
    segs = synth.make_segments((("w", K, 0.02),))
    ws = nv.alloc_workspace(gu.DEV, M, K, K, 1, fused=True)
    layers = []
    for i in range(depth):
        w_c, w_sf, g_w = nv.nvfp4_quantize_weight(gu.dev_bf16(synth.weights(31, 900 + i, segs, K)), segs)
        layers.append((w_c, w_sf, g_w))
    x0 = gu.dev_bf16(synth.activations(31, 1, M, K, n_hot=2, hot_scale=20.0))
    g_a = gu.dev_f32(np.float32(0.05))            # one static activation scale for every layer
    bufs = [torch.empty((M, K), dtype=torch.bfloat16, device=gu.DEV) for _ in range(2)]
    torch.cuda.synchronize()

    def chain(sync):
        src = x0
        for i, (w_c, w_sf, g_w) in enumerate(layers):
            dst = bufs[i & 1]                      # ping-pong: layer i+1 overwrites what layer i read
            nv.nvfp4_linear_bf16(src, g_a, w_c, w_sf, segs, g_w, ws, out=dst, w_resident=True)
            if sync:
                torch.cuda.synchronize()
            src = dst
        return src

    want = chain(sync=True).clone()
    assert nv.device_status(ws) == 0
    assert bool(torch.isfinite(want.float()).all()) and float(want.float().abs().max()) > 0.0
    for _ in range(3):
        got = chain(sync=False)
        torch.cuda.synchronize()
        assert torch.equal(got, want)
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            out = chain(sync=False)
        for _ in range(3):
            graph.replay()
        side.synchronize()
    assert torch.equal(out, want)
    assert nv.device_status(ws) == 0


# ---- more distinct output buffers than the table of encoded tensor maps holds ------------------------------
def test_many_distinct_output_pointers():
    M, N, K = 130, 64, 64                                   # the TMA-store path (bf16, aligned rows)
    segs, x, w, ac, asf, ga, wc, wsf, gs = _oracle_operands(41, M, K, (("p", N, 0.02),))
    y_ref = oracle.gemm(ac, asf, ga, wc, wsf, oracle.col_scales(N, segs, gs))
    bound = gu.gemm_bounds(ac, asf, ga, wc, wsf, oracle.col_scales(N, segs, gs))
    a_c, a_sf, g_a = gu.dev_u8(ac), gu.dev_u8(oracle.sf_to_mma(asf, K)), gu.dev_f32(ga)
    w_c, w_sf, g_w = gu.dev_u8(wc), gu.dev_u8(oracle.sf_to_mma(wsf, K)), gu.dev_f32(gs)
    ws = _ws()
    n_bufs = 4500
    pool = torch.zeros((n_bufs, M, N), dtype=torch.bfloat16, device=gu.DEV)
    for i in range(n_bufs):
        nv.nvfp4_linear(a_c, a_sf, g_a, w_c, w_sf, segs, g_w, ws, out=pool[i])
    nv.nvfp4_linear(a_c, a_sf, g_a, w_c, w_sf, segs, g_w, ws, out=pool[0])     # an entry that was evicted long ago
    torch.cuda.synchronize()
    assert nv.device_status(ws) == 0
    for i in (0, 1, 2047, 2048, 4095, 4096, n_bufs - 1):
        gu.check_gemm(pool[i], y_ref, bound, "buffer %d" % i)
    assert torch.equal(pool[0], pool[n_bufs - 1]) and torch.equal(pool[17], pool[4321])
