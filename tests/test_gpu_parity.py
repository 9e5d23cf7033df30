"""GPU parity: the CUDA path (through the C ABI) against the fp64 CPU oracle, element by
element, on the same seeded inputs.  Tolerances are the stated ones:
    bf16 outputs : |err| <= 1e-2 + 1e-2 |ref|
    fp32 outputs and lse : |err| <= 1e-3 + 1e-3 |ref|
Outputs are pre-filled with NaN and surrounded by canaries, so an element the
kernel never wrote, or a write outside the output, fails the test."""
import numpy as np
import pytest
import torch

from oracle import ref
from paper_2511_20100_b200 import inputs
from paper_2511_20100_b200 import binding as B

pytestmark = pytest.mark.gpu

TOL = {"bf16": (1e-2, 1e-2), "fp32": (1e-3, 1e-3)}
PAD = 512   # canary elements before and after every output


def _guarded(shape, dtype):
    n = int(np.prod(shape))
    buf = torch.full((n + 2 * PAD,), float("nan"), dtype=dtype, device="cuda")
    buf[:PAD] = 7.0
    buf[PAD + n:] = 7.0
    return buf, buf[PAD:PAD + n].view(*shape)


def _canaries_intact(buf, n):
    return bool((buf[:PAD] == 7.0).all()) and bool((buf[PAD + n:] == 7.0).all())


def _assert_close(got, want, tol, what):
    r = ref.compare(got, want, *tol)
    assert r["ok"], "%s: %d/%d outside tolerance, max |err| %.3e, worst ratio %.2f at flat index %d" % (
        what, r["violations"], r["count"], r["max_abs_err"], r["max_ratio"], r["worst_index"])
    return r


def run_linear(M, N, K, act, odt, seed, bias=True):
    li = inputs.linear_inputs(M, N, K, seed, bias=bias)
    buf, out = _guarded((M, N), torch.bfloat16 if odt == "bf16" else torch.float32)
    B.mtmc_fused_linear(li.X.cuda(), li.W.cuda(), None if li.b is None else li.b.cuda(), act, odt, out=out)
    B.mtmc_check_status()
    assert _canaries_intact(buf, M * N)
    return li, out


# ------------------------------------------------------------------ small shapes, full oracle
SMALL = [
    # M, N, K  -- several tiles, ragged tails in every dimension, K not a multiple of 64
    (1, 8, 8), (17, 8, 64), (100, 72, 136), (128, 128, 64), (129, 257, 72), (136, 384, 256),
    (256, 100, 1024), (384, 640, 512), (300, 520, 200), (64, 1000, 320),
]


@pytest.mark.parametrize("M,N,K", SMALL)
@pytest.mark.parametrize("act", ["none", "relu", "gelu_tanh", "silu"])
@pytest.mark.parametrize("odt", ["fp32", "bf16"])
def test_fused_linear_small(M, N, K, act, odt):
    li, out = run_linear(M, N, K, act, odt, seed=1000 + M + N + K)
    want = ref.fused_linear(inputs.bf16_bits(li.X), inputs.bf16_bits(li.W), inputs.f32(li.b), B.ACT[act])
    _assert_close(inputs.to_f64(out), want, TOL[odt], "fused_linear %dx%dx%d %s %s" % (M, N, K, act, odt))


@pytest.mark.parametrize("tile_n", [128, 256])
def test_fused_linear_both_tile_widths(tile_n):
    B.mtmc_set_tuning(tile_n=tile_n)
    try:
        li, out = run_linear(260, 392, 328, "gelu_tanh", "fp32", seed=77)
    finally:
        B.mtmc_set_tuning()
    want = ref.fused_linear(inputs.bf16_bits(li.X), inputs.bf16_bits(li.W), inputs.f32(li.b), B.ACT["gelu_tanh"])
    _assert_close(inputs.to_f64(out), want, TOL["fp32"], "tile_n %d" % tile_n)


@pytest.mark.parametrize("cta_pair", [1, -1])
def test_cta_pair_and_single_cta_kernels_agree_with_the_oracle(cta_pair):
    """Both tiled kernels on the same ragged shapes: 256-row CTA-pair tiles and 128-row single-CTA tiles."""
    B.mtmc_set_tuning(cta_pair=cta_pair)
    try:
        li, out = run_linear(600, 1000, 328, "gelu_tanh", "bf16", seed=81)
        si = inputs.swiglu_inputs(520, 648, 256, seed=82)
        sw = B.mtmc_swiglu(si.X.cuda(), si.Wg.cuda(), si.Wu.cuda())
        ll = inputs.linear_inputs(700, 3000, 192, seed=83)
        lse = B.mtmc_linear_lse(ll.X.cuda(), ll.W.cuda(), ll.b.cuda())
        one = inputs.linear_inputs(129, 257, 72, seed=84)             # second CTA of the pair almost empty
        o1 = B.mtmc_fused_linear(one.X.cuda(), one.W.cuda(), one.b.cuda(), "relu", "fp32")
        B.mtmc_check_status()
    finally:
        B.mtmc_set_tuning()
    _assert_close(inputs.to_f64(out), ref.fused_linear(inputs.bf16_bits(li.X), inputs.bf16_bits(li.W), inputs.f32(li.b),
                                                       ref.ACT_GELU_TANH), TOL["bf16"], "fused_linear")
    _assert_close(inputs.to_f64(sw), ref.swiglu(inputs.bf16_bits(si.X), inputs.bf16_bits(si.Wg), inputs.bf16_bits(si.Wu)),
                  TOL["bf16"], "swiglu")
    _assert_close(inputs.to_f64(lse), ref.linear_lse(inputs.bf16_bits(ll.X), inputs.bf16_bits(ll.W), inputs.f32(ll.b)),
                  TOL["fp32"], "linear_lse")
    _assert_close(inputs.to_f64(o1), ref.fused_linear(inputs.bf16_bits(one.X), inputs.bf16_bits(one.W), inputs.f32(one.b),
                                                      ref.ACT_RELU), TOL["fp32"], "129x257x72")



@pytest.mark.parametrize("M,N,K", [(100, 72, 136), (512, 256, 64), (600, 520, 328), (1100, 1300, 1024), (2048, 1000, 200)])
@pytest.mark.parametrize("act,odt", [("gelu_tanh", "bf16"), ("relu", "fp32")])
def test_large_tile_pair_kernel_forced(M, N, K, act, odt):
    """The CTA-pair kernel with 512 x 256 tiles (two 128-row halves per CTA, eight epilogue warps), forced by the
    tuning hook on shapes that leave rows, columns and k-blocks ragged."""
    li = inputs.linear_inputs(M, N, K, seed=8800 + M + N)
    want = ref.fused_linear(inputs.bf16_bits(li.X), inputs.bf16_bits(li.W), inputs.f32(li.b), B.ACT[act])
    buf, out = _guarded((M, N), torch.bfloat16 if odt == "bf16" else torch.float32)
    B.mtmc_set_tuning(cta_pair=2)
    try:
        B.mtmc_fused_linear(li.X.cuda(), li.W.cuda(), li.b.cuda(), act, odt, out=out)
        B.mtmc_check_status()
        again = B.mtmc_fused_linear(li.X.cuda(), li.W.cuda(), li.b.cuda(), act, odt)
    finally:
        B.mtmc_set_tuning()
    assert _canaries_intact(buf, M * N)
    assert torch.equal(again, out)
    _assert_close(inputs.to_f64(out), want, TOL[odt], "512-row tiles %dx%dx%d %s %s" % (M, N, K, act, odt))


@pytest.mark.parametrize("M,N,K", [(100, 72, 136), (600, 520, 328), (1100, 1300, 1024)])
def test_large_tile_pair_kernel_row_reductions(M, N, K):
    """logsumexp, row max and cross entropy on the 512 x 256 tiles (forced), bias staged in shared memory."""
    li = inputs.linear_inputs(M, N, K, seed=8950 + M)
    Xb, Wb, bf = inputs.bf16_bits(li.X), inputs.bf16_bits(li.W), inputs.f32(li.b)
    Xd, Wd, bd = li.X.cuda(), li.W.cuda(), li.b.cuda()
    tgt = torch.from_numpy(np.random.default_rng(M).integers(0, N, size=M))
    B.mtmc_set_tuning(cta_pair=2)
    try:
        lse = B.mtmc_linear_lse(Xd, Wd, bd)
        lse_nobias = B.mtmc_linear_lse(Xd, Wd, None)
        mx, arg = B.mtmc_linear_rowmax(Xd, Wd, bd)
        loss = B.mtmc_linear_cross_entropy(Xd, Wd, bd, tgt.cuda())
        B.mtmc_check_status()
    finally:
        B.mtmc_set_tuning()
    fi = inputs.fp8_linear_inputs(M, N, 2 * K, seed=8960 + M)           # E4M3 operands through the same kernel
    B.mtmc_set_tuning(cta_pair=2)
    try:
        lse8 = B.mtmc_linear_lse_fp8(fi.X.cuda(), fi.W.cuda(), fi.b.cuda(), fi.scale_x, fi.scale_w)
        B.mtmc_check_status()
    finally:
        B.mtmc_set_tuning()
    _assert_close(inputs.to_f64(lse8), ref.linear_lse_fp8(inputs.fp8_bits(fi.X), inputs.fp8_bits(fi.W), inputs.f32(fi.b),
                                                          fi.scale_x, fi.scale_w), TOL["fp32"], "fp8 lse, 512-row tiles")
    si = inputs.swiglu_inputs(M, N, K, seed=8970 + M)                   # and the SwiGLU gate, which only the hook sends there
    B.mtmc_set_tuning(cta_pair=2)
    try:
        sw = B.mtmc_swiglu(si.X.cuda(), si.Wg.cuda(), si.Wu.cuda())
        B.mtmc_check_status()
    finally:
        B.mtmc_set_tuning()
    _assert_close(inputs.to_f64(sw), ref.swiglu(inputs.bf16_bits(si.X), inputs.bf16_bits(si.Wg), inputs.bf16_bits(si.Wu)),
                  TOL["bf16"], "swiglu, 512-row tiles")
    _assert_close(inputs.to_f64(lse), ref.linear_lse(Xb, Wb, bf), TOL["fp32"], "lse, 512-row tiles")
    _assert_close(inputs.to_f64(lse_nobias), ref.linear_lse(Xb, Wb, None), TOL["fp32"], "lse without bias, 512-row tiles")
    _check_rowmax(li, mx, arg, "rowmax, 512-row tiles")
    want_loss, _ = ref.linear_cross_entropy(Xb, Wb, bf, tgt.numpy())
    _assert_close(inputs.to_f64(loss), want_loss, TOL["fp32"], "cross entropy, 512-row tiles")


@pytest.mark.parametrize("M,N,K,padx,padw,pado", [(5, 300, 512, 64, 8, 20), (100, 72, 136, 8, 24, 3), (300, 520, 328, 16, 8, 8),
                                                  (128, 1024, 4096, 64, 64, 1024), (1100, 1300, 1024, 8, 8, 4), (600, 520, 6144, 8, 16, 0)])
@pytest.mark.parametrize("act,odt", [("gelu_tanh", "bf16"), ("none", "fp32")])
def test_fused_linear_strided_views(M, N, K, padx, padw, pado, act, odt):
    """Column slices of wider matrices as X, W and out, on the weight-streaming, single-CTA, cluster split-K and
    CTA-pair kernels; the columns of the wide output outside the slice must stay untouched."""
    li = inputs.linear_inputs(M, N, K, seed=9000 + M + N)
    want = ref.fused_linear(inputs.bf16_bits(li.X), inputs.bf16_bits(li.W), inputs.f32(li.b), B.ACT[act])
    tdt = torch.bfloat16 if odt == "bf16" else torch.float32
    Xw = torch.full((M, K + padx), 3.0, dtype=torch.bfloat16, device="cuda")
    Ww = torch.full((N, K + padw), -2.0, dtype=torch.bfloat16, device="cuda")
    Ow = torch.full((M, N + pado), 7.0, dtype=tdt, device="cuda")
    offx, offw, offo = (8 if padx >= 16 else 0), (8 if padw >= 16 else 0), (8 if pado >= 16 else 0)
    Xv, Wv, Ov = Xw[:, offx:offx + K], Ww[:, offw:offw + K], Ow[:, offo:offo + N]
    Xv.copy_(li.X.cuda()); Wv.copy_(li.W.cuda())
    B.mtmc_fused_linear_strided(Xv, Wv, li.b.cuda(), act, odt, out=Ov)
    B.mtmc_check_status()
    _assert_close(inputs.to_f64(Ov.contiguous()), want, TOL[odt], "strided %dx%dx%d %s" % (M, N, K, odt))
    assert bool((Ow[:, :offo] == 7.0).all()) and bool((Ow[:, offo + N:] == 7.0).all())
    dense = B.mtmc_fused_linear(li.X.cuda(), li.W.cuda(), li.b.cuda(), act, odt)
    assert torch.equal(dense, Ov.contiguous())              # the same kernels on the same values


@pytest.mark.parametrize("M,N,K,padx,padw,pado", [(100, 72, 136, 8, 24, 3), (300, 520, 328, 16, 8, 8), (128, 1024, 4096, 64, 64, 1024),
                                                  (1100, 1300, 1024, 8, 16, 4)])
def test_other_operators_on_strided_views(M, N, K, padx, padw, pado):
    """SwiGLU and the three row reductions on column slices of wider matrices (single-CTA, cluster split-K and
    CTA-pair kernels): the same bits as the dense calls, within tolerance of the oracle, neighbours untouched."""
    si = inputs.swiglu_inputs(M, N, K, seed=9050 + M + N)
    li = inputs.linear_inputs(M, N, K, seed=9060 + M + N)
    tgt = torch.from_numpy(np.random.default_rng(M + N).integers(0, N, size=M)).cuda()
    Xw = torch.full((M, K + padx), 3.0, dtype=torch.bfloat16, device="cuda")
    GU = torch.full((N, 2 * K + padw), -2.0, dtype=torch.bfloat16, device="cuda")       # gate and up side by side in one matrix
    Ow = torch.full((M, N + pado), 7.0, dtype=torch.bfloat16, device="cuda")
    offx, offo = (8 if padx >= 16 else 0), (8 if pado >= 16 else 0)
    Xv, Gv, Uv, Ov = Xw[:, offx:offx + K], GU[:, :K], GU[:, K:2 * K], Ow[:, offo:offo + N]
    Xv.copy_(si.X.cuda()); Gv.copy_(si.Wg.cuda()); Uv.copy_(si.Wu.cuda())
    B.mtmc_swiglu_strided(Xv, Gv, Uv, out=Ov)
    B.mtmc_check_status()
    want = ref.swiglu(inputs.bf16_bits(si.X), inputs.bf16_bits(si.Wg), inputs.bf16_bits(si.Wu))
    _assert_close(inputs.to_f64(Ov.contiguous()), want, TOL["bf16"], "strided swiglu %dx%dx%d" % (M, N, K))
    assert bool((Ow[:, :offo] == 7.0).all()) and bool((Ow[:, offo + N:] == 7.0).all())
    assert torch.equal(B.mtmc_swiglu(si.X.cuda(), si.Wg.cuda(), si.Wu.cuda()), Ov.contiguous())
    # the row reductions: X as above, W as the left half of the wide matrix
    Xv.copy_(li.X.cuda()); Gv.copy_(li.W.cuda())
    bd = li.b.cuda()
    lse = B.mtmc_linear_lse_strided(Xv, Gv, bd)
    mx, arg = B.mtmc_linear_rowmax_strided(Xv, Gv, bd)
    loss = B.mtmc_linear_cross_entropy_strided(Xv, Gv, bd, tgt)
    B.mtmc_check_status()
    Xd, Wd = li.X.cuda(), li.W.cuda()
    assert torch.equal(lse, B.mtmc_linear_lse(Xd, Wd, bd))
    dmx, darg = B.mtmc_linear_rowmax(Xd, Wd, bd)
    assert torch.equal(mx, dmx) and torch.equal(arg, darg)
    assert torch.equal(loss, B.mtmc_linear_cross_entropy(Xd, Wd, bd, tgt))
    Xb, Wb, bf = inputs.bf16_bits(li.X), inputs.bf16_bits(li.W), inputs.f32(li.b)
    _assert_close(inputs.to_f64(lse), ref.linear_lse(Xb, Wb, bf), TOL["fp32"], "strided lse")
    _check_rowmax(li, mx, arg, "strided rowmax")
    want_loss, _ = ref.linear_cross_entropy(Xb, Wb, bf, tgt.cpu().numpy())
    _assert_close(inputs.to_f64(loss), want_loss, TOL["fp32"], "strided cross entropy")


def test_large_tile_pair_kernel_chosen_for_long_k():
    """From 256 k-blocks on the 512 x 256 tiles are the default when their waves cost no more than the 256 x 256 pair
    tiles' (1024 x 9472 x 16384: 74 large tiles, one wave).  That shape against the oracle on sampled points (every pair
    tile, tile edges); a small one (15 tiles: cluster split-K by default) in full on each kernel family the hooks select."""
    M, N, K = 1024, 9472, 16384
    li = inputs.linear_inputs(M, N, K, seed=8899)
    out = B.mtmc_fused_linear(li.X.cuda(), li.W.cuda(), li.b.cuda(), "silu", "bf16")
    assert "gemm_big_kernel" in B.mtmc_last_kernel_name(), "ran %s" % B.mtmc_last_kernel_name()
    B.mtmc_check_status()
    rows, cols = inputs.sample_points(M, N, 3000, seed=7, tile_m=256, tile_n=256)
    want = ref.fused_linear_points(inputs.bf16_bits(li.X), inputs.bf16_bits(li.W), inputs.f32(li.b), ref.ACT_SILU, rows, cols)
    _assert_close(inputs.to_f64(out[torch.from_numpy(rows).cuda(), torch.from_numpy(cols).cuda()]), want, TOL["bf16"], "1024 x 9472 x 16384 sampled")
    assert bool(torch.isfinite(out.float()).all())
    del out, li

    M, N, K = 600, 520, 6144
    li = inputs.linear_inputs(M, N, K, seed=8900)
    Xb, Wb, bf = inputs.bf16_bits(li.X), inputs.bf16_bits(li.W), inputs.f32(li.b)
    Xd, Wd, bd = li.X.cuda(), li.W.cuda(), li.b.cuda()
    want = ref.fused_linear(Xb, Wb, bf, ref.ACT_SILU)
    for tune, family in ((dict(), "gemm_ksplit_kernel"), (dict(cta_pair=1), "gemm_pair_kernel"), (dict(cta_pair=2), "gemm_big_kernel"),
                         (dict(cta_pair=-1, split_k=1), "gemm_tiled_kernel")):
        B.mtmc_set_tuning(**tune)
        try:
            out = B.mtmc_fused_linear(Xd, Wd, bd, "silu", "fp32")
            assert family in B.mtmc_last_kernel_name(), "%r ran %s" % (tune, B.mtmc_last_kernel_name())
        finally:
            B.mtmc_set_tuning()
        _assert_close(inputs.to_f64(out), want, TOL["fp32"], "long K, %s" % family)
    R = torch.randn(M, N, generator=torch.Generator().manual_seed(5)).bfloat16()
    res = B.mtmc_fused_linear_residual(Xd, Wd, bd, R.cuda(), "none", "bf16")
    _assert_close(inputs.to_f64(res), ref.fused_linear_residual(Xb, Wb, bf, inputs.bf16_bits(R), ref.ACT_NONE), TOL["bf16"],
                  "long K residual")
    fi = inputs.fp8_linear_inputs(M, N, 2 * K, seed=8901)
    f8 = B.mtmc_fused_linear_fp8(fi.X.cuda(), fi.W.cuda(), fi.b.cuda(), fi.scale_x, fi.scale_w, "gelu_tanh", "bf16")
    want8 = ref.fused_linear_fp8(inputs.fp8_bits(fi.X), inputs.fp8_bits(fi.W), inputs.f32(fi.b), fi.scale_x, fi.scale_w, ref.ACT_GELU_TANH)
    _assert_close(inputs.to_f64(f8), want8, TOL["bf16"], "long K fp8")
    B.mtmc_check_status()


@pytest.mark.parametrize("M,N,K,want", [(100, 1000, 2304, "(128-column tiles)<EPI_ACT, 4>"), (200, 392, 1152, "(128-column tiles)<EPI_ACT, 2>"),
                                        (128, 4096, 4096, "(128-column tiles)<EPI_ACT, 4>")])
def test_cluster_split_k_on_128_column_tiles(M, N, K, want):
    """Activation epilogues take the cluster split-K kernel on 128-column tiles when that halves the cluster: clusters of
    four and of two, each CTA walking an odd number of k-blocks (9: the ring is handed over two at a time and ends with
    half a stage), ragged N, fp32 and bf16 outputs, the residual form and E4M3 operands."""
    li = inputs.linear_inputs(M, N, K, seed=9400 + M)
    Xb, Wb, bf = inputs.bf16_bits(li.X), inputs.bf16_bits(li.W), inputs.f32(li.b)
    Xd, Wd, bd = li.X.cuda(), li.W.cuda(), li.b.cuda()
    buf, out = _guarded((M, N), torch.float32)
    B.mtmc_fused_linear(Xd, Wd, bd, "gelu_tanh", "fp32", out=out)
    assert want in B.mtmc_last_kernel_name(), "ran %s" % B.mtmc_last_kernel_name()
    B.mtmc_check_status()
    assert _canaries_intact(buf, M * N)
    _assert_close(inputs.to_f64(out), ref.fused_linear(Xb, Wb, bf, ref.ACT_GELU_TANH), TOL["fp32"], "narrow split-K %dx%dx%d" % (M, N, K))
    assert torch.equal(B.mtmc_fused_linear(Xd, Wd, bd, "gelu_tanh", "fp32"), out)          # bit-reproducible
    R = torch.randn(M, N, generator=torch.Generator().manual_seed(M + N)).bfloat16()
    res = B.mtmc_fused_linear_residual(Xd, Wd, bd, R.cuda(), "silu", "bf16")
    assert want in B.mtmc_last_kernel_name()
    _assert_close(inputs.to_f64(res), ref.fused_linear_residual(Xb, Wb, bf, inputs.bf16_bits(R), ref.ACT_SILU), TOL["bf16"], "narrow split-K residual")
    fi = inputs.fp8_linear_inputs(M, N, 2 * K, seed=9500 + M)
    f8 = B.mtmc_fused_linear_fp8(fi.X.cuda(), fi.W.cuda(), fi.b.cuda(), fi.scale_x, fi.scale_w, "relu", "bf16")
    assert want in B.mtmc_last_kernel_name(), "fp8 ran %s" % B.mtmc_last_kernel_name()
    want8 = ref.fused_linear_fp8(inputs.fp8_bits(fi.X), inputs.fp8_bits(fi.W), inputs.f32(fi.b), fi.scale_x, fi.scale_w, ref.ACT_RELU)
    _assert_close(inputs.to_f64(f8), want8, TOL["bf16"], "narrow split-K fp8")
    B.mtmc_check_status()


@pytest.mark.parametrize("K", [40, 136, 264, 456, 520])
def test_pair_kernel_odd_and_even_k_block_counts(K):
    """The pair kernel hands its ring over two k-blocks at a time; a walk of 1, 3, 5 or 7 k-blocks ends with half a
    stage (K = 40, 136, 264, 456; 520 is 9 k-blocks and wraps the three-stage ring).  All epilogues, bf16 and E4M3
    operands, and tail pieces (300 x 520 leaves a partial wave that is cut into column pieces)."""
    M, N = 300, 520
    li = inputs.linear_inputs(M, N, K, seed=9100 + K)
    si = inputs.swiglu_inputs(M, N, K, seed=9200 + K)
    fi = inputs.fp8_linear_inputs(M, N, 2 * K, seed=9300 + K)
    Xb, Wb, bf = inputs.bf16_bits(li.X), inputs.bf16_bits(li.W), inputs.f32(li.b)
    B.mtmc_set_tuning(cta_pair=1)
    try:
        out = B.mtmc_fused_linear(li.X.cuda(), li.W.cuda(), li.b.cuda(), "gelu_tanh", "fp32")
        assert "gemm_pair_kernel" in B.mtmc_last_kernel_name()
        sw = B.mtmc_swiglu(si.X.cuda(), si.Wg.cuda(), si.Wu.cuda())
        assert "gemm_pair_kernel" in B.mtmc_last_kernel_name()
        lse = B.mtmc_linear_lse(li.X.cuda(), li.W.cuda(), li.b.cuda())
        f8 = B.mtmc_fused_linear_fp8(fi.X.cuda(), fi.W.cuda(), fi.b.cuda(), fi.scale_x, fi.scale_w, "relu", "fp32")
        assert "gemm_pair_kernel" in B.mtmc_last_kernel_name()
    finally:
        B.mtmc_set_tuning()
    B.mtmc_check_status()
    _assert_close(inputs.to_f64(out), ref.fused_linear(Xb, Wb, bf, ref.ACT_GELU_TANH), TOL["fp32"], "pair, K = %d" % K)
    _assert_close(inputs.to_f64(sw), ref.swiglu(inputs.bf16_bits(si.X), inputs.bf16_bits(si.Wg), inputs.bf16_bits(si.Wu)), TOL["bf16"],
                  "pair swiglu, K = %d" % K)
    _assert_close(inputs.to_f64(lse), ref.linear_lse(Xb, Wb, bf), TOL["fp32"], "pair lse, K = %d" % K)
    want8 = ref.fused_linear_fp8(inputs.fp8_bits(fi.X), inputs.fp8_bits(fi.W), inputs.f32(fi.b), fi.scale_x, fi.scale_w, ref.ACT_RELU)
    _assert_close(inputs.to_f64(f8), want8, TOL["fp32"], "pair fp8, K = %d" % (2 * K))


@pytest.mark.parametrize("M,N,K", [(9, 520, 392), (16, 4096, 512), (129, 257, 72), (300, 520, 200), (600, 1000, 328)])
@pytest.mark.parametrize("odt", ["fp32", "bf16"])
def test_fused_linear_residual(M, N, K, odt):
    """Skip connection joined to the epilogue, on the skinny, single-CTA and CTA-pair paths; also in place."""
    li = inputs.linear_inputs(M, N, K, seed=6000 + M + N)
    tdt = torch.bfloat16 if odt == "bf16" else torch.float32
    R = torch.randn(M, N, generator=torch.Generator().manual_seed(M * N)).to(tdt)
    Rnp = inputs.bf16_bits(R) if odt == "bf16" else R.numpy()
    want = ref.fused_linear_residual(inputs.bf16_bits(li.X), inputs.bf16_bits(li.W), inputs.f32(li.b), Rnp, ref.ACT_SILU)
    buf, out = _guarded((M, N), tdt)
    Xd, Wd, bd, Rd = li.X.cuda(), li.W.cuda(), li.b.cuda(), R.cuda()
    B.mtmc_fused_linear_residual(Xd, Wd, bd, Rd, "silu", odt, out=out)
    B.mtmc_check_status()
    assert _canaries_intact(buf, M * N)
    _assert_close(inputs.to_f64(out), want, TOL[odt], "residual %dx%dx%d %s" % (M, N, K, odt))
    B.mtmc_fused_linear_residual(Xd, Wd, bd, Rd, "silu", odt, out=Rd)          # in place
    B.mtmc_check_status()
    assert torch.equal(Rd, out)


@pytest.mark.parametrize("M,N,K", [(1, 16, 16), (17, 8, 128), (100, 72, 144), (129, 257, 272), (300, 520, 400),
                                   (600, 1000, 656), (1024, 2048, 1024)])
@pytest.mark.parametrize("act,odt", [("none", "fp32"), ("gelu_tanh", "bf16"), ("relu", "fp32")])
def test_fused_linear_fp8(M, N, K, act, odt):
    """E4M3 operands with per-tensor scales on the single-CTA and CTA-pair kernels (K = 32 per MMA)."""
    fi = inputs.fp8_linear_inputs(M, N, K, seed=7000 + M + N)
    buf, out = _guarded((M, N), torch.bfloat16 if odt == "bf16" else torch.float32)
    B.mtmc_fused_linear_fp8(fi.X.cuda(), fi.W.cuda(), fi.b.cuda(), fi.scale_x, fi.scale_w, act, odt, out=out)
    B.mtmc_check_status()
    assert _canaries_intact(buf, M * N)
    want = ref.fused_linear_fp8(inputs.fp8_bits(fi.X), inputs.fp8_bits(fi.W), inputs.f32(fi.b), fi.scale_x, fi.scale_w, B.ACT[act])
    _assert_close(inputs.to_f64(out), want, TOL[odt], "fp8 %dx%dx%d %s %s" % (M, N, K, act, odt))


@pytest.mark.parametrize("M,N,K,split_k", [(1, 4096, 4096, 0), (8, 8192, 2064, 0), (16, 4736, 1024, 0), (17, 5000, 4112, 0),
                                           (33, 9472, 528, 0), (64, 16384, 4096, 0), (4, 1024, 4096, 4), (48, 640, 2192, 3),
                                           (2, 300, 16, 0), (64, 96, 8192, 0)])
@pytest.mark.parametrize("act,odt", [("none", "fp32"), ("silu", "bf16")])
def test_fused_linear_fp8_skinny(M, N, K, split_k, act, odt):
    """E4M3 weights streamed once on the split-K path (M <= 64): CTA-pair and ticket plans, ragged K and N."""
    fi = inputs.fp8_linear_inputs(M, N, K, seed=7100 + M + N)
    buf, out = _guarded((M, N), torch.bfloat16 if odt == "bf16" else torch.float32)
    B.mtmc_set_tuning(split_k=split_k)
    try:
        B.mtmc_fused_linear_fp8(fi.X.cuda(), fi.W.cuda(), fi.b.cuda(), fi.scale_x, fi.scale_w, act, odt, out=out)
        B.mtmc_check_status()
    finally:
        B.mtmc_set_tuning()
    assert _canaries_intact(buf, M * N)
    want = ref.fused_linear_fp8(inputs.fp8_bits(fi.X), inputs.fp8_bits(fi.W), inputs.f32(fi.b), fi.scale_x, fi.scale_w, B.ACT[act])
    _assert_close(inputs.to_f64(out), want, TOL[odt], "fp8 skinny %dx%dx%d %s %s" % (M, N, K, act, odt))


@pytest.mark.parametrize("M,N,K", [(1, 16, 16), (100, 72, 144), (300, 392, 272), (128, 1024, 4096), (600, 1000, 656), (1024, 2048, 1024)])
def test_swiglu_fp8(M, N, K):
    """E4M3 SwiGLU with separate gate / up scales on the single-CTA, cluster split-K and CTA-pair kernels."""
    X8, Wg8, Wu8, sx, sg, su = inputs.fp8_swiglu_inputs(M, N, K, seed=7200 + M + N)
    buf, out = _guarded((M, N), torch.bfloat16)
    B.mtmc_swiglu_fp8(X8.cuda(), Wg8.cuda(), Wu8.cuda(), sx, sg, su, out=out)
    B.mtmc_check_status()
    assert _canaries_intact(buf, M * N)
    want = ref.swiglu_fp8(inputs.fp8_bits(X8), inputs.fp8_bits(Wg8), inputs.fp8_bits(Wu8), sx, sg, su)
    _assert_close(inputs.to_f64(out), want, TOL["bf16"], "swiglu fp8 %dx%dx%d" % (M, N, K))


@pytest.mark.parametrize("M,N,K", [(1, 1, 16), (5, 8, 64), (200, 1000, 256), (129, 257, 80), (128, 1024, 4096), (600, 3000, 128),
                                   (1024, 4096, 512)])
def test_linear_lse_fp8(M, N, K):
    fi = inputs.fp8_linear_inputs(M, N, K, seed=7300 + M + N)
    buf, out = _guarded((M,), torch.float32)
    B.mtmc_linear_lse_fp8(fi.X.cuda(), fi.W.cuda(), fi.b.cuda(), fi.scale_x, fi.scale_w, lse_out=out)
    B.mtmc_check_status()
    assert _canaries_intact(buf, M)
    want = ref.linear_lse_fp8(inputs.fp8_bits(fi.X), inputs.fp8_bits(fi.W), inputs.f32(fi.b), fi.scale_x, fi.scale_w)
    _assert_close(inputs.to_f64(out), want, TOL["fp32"], "lse fp8 %dx%dx%d" % (M, N, K))


@pytest.mark.parametrize("M,N,K", [(5, 8, 64), (200, 1000, 256), (129, 257, 80), (128, 1024, 4096), (600, 1100, 192)])
def test_linear_rowmax_and_cross_entropy_fp8(M, N, K):
    fi = inputs.fp8_linear_inputs(M, N, K, seed=7400 + M + N)
    X8, W8, bf = inputs.fp8_bits(fi.X), inputs.fp8_bits(fi.W), inputs.f32(fi.b)
    Xd, Wd, bd = fi.X.cuda(), fi.W.cuda(), fi.b.cuda()
    mx, arg = B.mtmc_linear_rowmax_fp8(Xd, Wd, bd, fi.scale_x, fi.scale_w)
    want_mx, want_arg = ref.linear_rowmax_fp8(X8, W8, bf, fi.scale_x, fi.scale_w)
    _assert_close(inputs.to_f64(mx), want_mx, TOL["fp32"], "fp8 rowmax %dx%dx%d" % (M, N, K))
    z = ref.fused_linear_fp8(X8, W8, bf, fi.scale_x, fi.scale_w, ref.ACT_NONE)
    a = arg.cpu().numpy().astype(np.int64)
    assert np.all((a >= 0) & (a < N))
    assert np.all(np.abs(z[np.arange(M), a] - want_mx) <= 1e-3 + 1e-3 * np.abs(want_mx))       # the named column holds the maximum
    if N > 1:
        clear = (want_mx - np.partition(z, -2, axis=1)[:, -2]) > 1e-2
        assert np.array_equal(a[clear], want_arg[clear])
    tgt = torch.from_numpy(np.random.default_rng(M + N).integers(0, N, size=M))
    loss, lse = B.mtmc_linear_cross_entropy_fp8(Xd, Wd, bd, fi.scale_x, fi.scale_w, tgt.cuda(), want_lse=True)
    B.mtmc_check_status()
    want_loss, want_lse = ref.linear_cross_entropy_fp8(X8, W8, bf, fi.scale_x, fi.scale_w, tgt.numpy())
    _assert_close(inputs.to_f64(loss), want_loss, TOL["fp32"], "fp8 cross entropy %dx%dx%d" % (M, N, K))
    _assert_close(inputs.to_f64(lse), want_lse, TOL["fp32"], "fp8 lse of cross entropy")


# ------------------------------------------------------------------ block-scaled E4M3 (MXFP8)
def _mx_dev(mi):
    return mi.X.cuda(), mi.SX.cuda(), mi.W.cuda(), mi.SW.cuda(), None if mi.b is None else mi.b.cuda()


def _mx_np(mi):
    return inputs.fp8_bits(mi.X), mi.SX.numpy(), inputs.fp8_bits(mi.W), mi.SW.numpy(), inputs.f32(mi.b)


@pytest.mark.parametrize("kernel", ["single-CTA tiles", "CTA pairs"])
@pytest.mark.parametrize("vary", ["none", "x_rows", "w_rows", "x_kblocks", "w_kblocks", "all"])
def test_mxfp8_scale_placement_exact(vary, kernel):
    """Integer-valued elements and power-of-two scales: every product and fp32 partial sum is exact, so the result
    must equal the oracle bit for bit.  Each case lets the scales vary along one axis only (rows of X, rows of W,
    k-blocks of X, k-blocks of W), so that a scale read from the wrong row, quadrant or k-block fails its own case."""
    M, N, K = (256, 384, 512) if kernel == "single-CTA tiles" else (600, 700, 512)     # pairs: 256 x 224 tiles, ragged in M and N
    g = torch.Generator().manual_seed(60)
    X = torch.randint(-2, 3, (M, K), generator=g).float().to(torch.float8_e4m3fn)
    W = torch.randint(-2, 3, (N, K), generator=g).float().to(torch.float8_e4m3fn)
    SX = torch.full((M, K // 32), 127, dtype=torch.uint8)
    SW = torch.full((N, K // 32), 127, dtype=torch.uint8)
    if vary in ("x_rows", "all"):
        SX += (torch.arange(M) % 7).to(torch.uint8)[:, None]
    if vary in ("w_rows", "all"):
        SW += (torch.arange(N) % 5).to(torch.uint8)[:, None]
    if vary in ("x_kblocks", "all"):
        SX -= (torch.arange(K // 32) % 6).to(torch.uint8)[None, :]
    if vary in ("w_kblocks", "all"):
        SW -= (torch.arange(K // 32) % 4).to(torch.uint8)[None, :]
    B.mtmc_set_tuning(cta_pair=-1 if kernel == "single-CTA tiles" else 1)
    try:
        out = B.mtmc_fused_linear_mxfp8(X.cuda(), SX.cuda(), W.cuda(), SW.cuda(), None, "none", "fp32")
        B.mtmc_check_status()
    finally:
        B.mtmc_set_tuning()
    assert ("gemm_mx_kernel" if kernel == "single-CTA tiles" else "gemm_mx_pair_kernel") in B.mtmc_last_kernel_name()
    want = ref.fused_linear_mxfp8(inputs.fp8_bits(X), SX.numpy(), inputs.fp8_bits(W), SW.numpy(), None, ref.ACT_NONE)
    got = inputs.to_f64(out)
    bad = np.argwhere(got != want)
    assert len(bad) == 0, "%s, %s: %d mismatches, first at %r: got %r want %r; mismatching rows %r.., columns %r.." % (
        vary, kernel, len(bad), tuple(bad[0]), got[tuple(bad[0])], want[tuple(bad[0])], sorted(set(bad[:, 0]))[:8], sorted(set(bad[:, 1]))[:8])


@pytest.mark.parametrize("M,N,K", [(1, 8, 32), (17, 8, 128), (100, 72, 160), (129, 257, 288), (300, 520, 416), (600, 1000, 672),
                                   (1024, 2048, 1024)])
@pytest.mark.parametrize("act,odt", [("none", "fp32"), ("gelu_tanh", "bf16"), ("relu", "fp32")])
def test_fused_linear_mxfp8(M, N, K, act, odt):
    """Seeded N(0,1) draws with block magnitudes spread over 2^-6 .. 2^6, quantised to MXFP8; ragged M, N and K (K not a
    multiple of the 128-element ring stage)."""
    mi = inputs.mx_linear_inputs(M, N, K, seed=7500 + M + N, spread=6)
    buf, out = _guarded((M, N), torch.bfloat16 if odt == "bf16" else torch.float32)
    Xd, SXd, Wd, SWd, bd = _mx_dev(mi)
    B.mtmc_fused_linear_mxfp8(Xd, SXd, Wd, SWd, bd, act, odt, out=out)
    B.mtmc_check_status()
    assert _canaries_intact(buf, M * N)
    X8, SX, W8, SW, b = _mx_np(mi)
    _assert_close(inputs.to_f64(out), ref.fused_linear_mxfp8(X8, SX, W8, SW, b, B.ACT[act]), TOL[odt], "mxfp8 %dx%dx%d %s %s" % (M, N, K, act, odt))
    assert torch.equal(B.mtmc_fused_linear_mxfp8(Xd, SXd, Wd, SWd, bd, act, odt), out)


@pytest.mark.parametrize("M,N,K", [(5, 8, 64), (100, 72, 160), (300, 392, 288), (600, 1000, 672), (1100, 520, 1056)])
def test_swiglu_and_lse_mxfp8(M, N, K):
    mi = inputs.mx_linear_inputs(M, N, K, seed=7600 + M + N, spread=4)
    up = inputs.mx_linear_inputs(M, N, K, seed=7650 + M + N, spread=4)
    Xd, SXd, Gd, SGd, bd = _mx_dev(mi)
    buf, out = _guarded((M, N), torch.bfloat16)
    B.mtmc_swiglu_mxfp8(Xd, SXd, Gd, SGd, up.W.cuda(), up.SW.cuda(), out=out)
    lse = B.mtmc_linear_lse_mxfp8(Xd, SXd, Gd, SGd, bd)
    B.mtmc_check_status()
    assert _canaries_intact(buf, M * N)
    X8, SX, G8, SG, b = _mx_np(mi)
    want = ref.swiglu_mxfp8(X8, SX, G8, SG, inputs.fp8_bits(up.W), up.SW.numpy())
    _assert_close(inputs.to_f64(out), want, TOL["bf16"], "mxfp8 swiglu %dx%dx%d" % (M, N, K))
    _assert_close(inputs.to_f64(lse), ref.linear_lse_mxfp8(X8, SX, G8, SG, b), TOL["fp32"], "mxfp8 lse %dx%dx%d" % (M, N, K))


def test_mxfp8_with_caller_workspace_and_full_size_sample():
    """4096^3 in a caller workspace of exactly mtmc_workspace_bytes; the first and last rows against the oracle."""
    M = N = K = 4096
    mi = inputs.mx_linear_inputs(M, N, K, seed=1, spread=3)
    need = B.mtmc_workspace_bytes("fused_linear_mxfp8", M, N, K)
    guard = torch.full((need + 8192,), 0x5A, dtype=torch.uint8, device="cuda")
    off = (-guard.data_ptr()) % 256 + 3840
    B.mtmc_set_workspace(guard[off:off + need])
    try:
        out = B.mtmc_fused_linear_mxfp8(*_mx_dev(mi), "gelu_tanh", "bf16")
        B.mtmc_check_status()
    finally:
        B.mtmc_set_workspace(None)
    assert bool((guard[:off] == 0x5A).all()) and bool((guard[off + need:] == 0x5A).all())
    rows = np.array([0, 1, 127, 128, 2047, 4095])
    X8, SX, W8, SW, b = _mx_np(mi)
    want = ref.fused_linear_mxfp8(np.ascontiguousarray(X8[rows]), np.ascontiguousarray(SX[rows]), W8, SW, b, ref.ACT_GELU_TANH)
    _assert_close(inputs.to_f64(out[torch.from_numpy(rows).cuda()]), want, TOL["bf16"], "mxfp8 4096^3 sampled rows")
    assert bool(torch.isfinite(out.float()).all())


def test_fused_linear_fp8_exact_small_integers():
    # operands in {-2..2} are exact in E4M3 and every fp32 partial sum is exact: the result must be exact too
    g = torch.Generator().manual_seed(6)
    X = torch.randint(-2, 3, (200, 256), generator=g).float().to(torch.float8_e4m3fn)
    W = torch.randint(-2, 3, (264, 256), generator=g).float().to(torch.float8_e4m3fn)
    out = B.mtmc_fused_linear_fp8(X.cuda(), W.cuda(), None, 1.0, 1.0, "none", "fp32")
    B.mtmc_check_status()
    want = ref.fused_linear_fp8(inputs.fp8_bits(X), inputs.fp8_bits(W), None, 1.0, 1.0, ref.ACT_NONE)
    assert np.array_equal(inputs.to_f64(out), want)


def test_fused_linear_fp8_at_full_size_on_sampled_points():
    fi = inputs.fp8_linear_inputs(4096, 4096, 4096, seed=1)
    out = B.mtmc_fused_linear_fp8(fi.X.cuda(), fi.W.cuda(), fi.b.cuda(), fi.scale_x, fi.scale_w, "gelu_tanh", "bf16")
    B.mtmc_check_status()
    rows, cols = inputs.sample_points(4096, 4096, 4000, seed=5, tile_m=256, tile_n=256)
    want = ref.fused_linear_fp8_points(inputs.fp8_bits(fi.X), inputs.fp8_bits(fi.W), inputs.f32(fi.b), fi.scale_x, fi.scale_w,
                                       ref.ACT_GELU_TANH, rows, cols)
    got = inputs.to_f64(out[torch.from_numpy(rows).cuda(), torch.from_numpy(cols).cuda()])
    _assert_close(got, want, TOL["bf16"], "fp8 4096^3 sampled")
    assert bool(torch.isfinite(out.float()).all())


def test_fused_linear_exact_integers_and_no_bias():
    # integer-valued operands: every product and fp32 partial sum is exact, so the result must be too
    g = torch.Generator().manual_seed(5)
    X = torch.randint(-3, 4, (200, 192), generator=g).to(torch.bfloat16)
    W = torch.randint(-3, 4, (264, 192), generator=g).to(torch.bfloat16)
    out = B.mtmc_fused_linear(X.cuda(), W.cuda(), None, "none", "fp32")
    B.mtmc_check_status()
    want = ref.fused_linear(inputs.bf16_bits(X), inputs.bf16_bits(W), None, ref.ACT_NONE)
    assert np.array_equal(inputs.to_f64(out), want)


def test_identity_weight_and_zero_input():
    li = inputs.linear_inputs(130, 192, 192, seed=3)
    eye = torch.eye(192).to(torch.bfloat16)
    out = B.mtmc_fused_linear(li.X.cuda(), eye.cuda(), li.b.cuda(), "silu", "fp32")
    want = ref.fused_linear(inputs.bf16_bits(li.X), inputs.bf16_bits(eye), inputs.f32(li.b), ref.ACT_SILU)
    _assert_close(inputs.to_f64(out), want, TOL["fp32"], "W = I")
    zero = torch.zeros_like(li.X)
    out0 = B.mtmc_fused_linear(zero.cuda(), li.W.cuda(), li.b.cuda(), "gelu_tanh", "fp32")
    B.mtmc_check_status()
    want0 = np.array([ref.act(ref.ACT_GELU_TANH, float(v)) for v in li.b])
    _assert_close(inputs.to_f64(out0), np.broadcast_to(want0, (130, 192)), TOL["fp32"], "X = 0")


@pytest.mark.parametrize("M,N,K", [(1, 8, 8), (100, 72, 136), (300, 392, 256), (128, 1000, 512), (513, 136, 64)])
def test_swiglu_small(M, N, K):
    si = inputs.swiglu_inputs(M, N, K, seed=2000 + M + N)
    buf, out = _guarded((M, N), torch.bfloat16)
    B.mtmc_swiglu(si.X.cuda(), si.Wg.cuda(), si.Wu.cuda(), out=out)
    B.mtmc_check_status()
    assert _canaries_intact(buf, M * N)
    want = ref.swiglu(inputs.bf16_bits(si.X), inputs.bf16_bits(si.Wg), inputs.bf16_bits(si.Wu))
    _assert_close(inputs.to_f64(out), want, TOL["bf16"], "swiglu %dx%dx%d" % (M, N, K))


def test_swiglu_equal_weights_is_silu_z_times_z():
    si = inputs.swiglu_inputs(140, 256, 192, seed=31)
    out = B.mtmc_swiglu(si.X.cuda(), si.Wg.cuda(), si.Wg.cuda())
    B.mtmc_check_status()
    z = ref.fused_linear(inputs.bf16_bits(si.X), inputs.bf16_bits(si.Wg), None, ref.ACT_NONE)
    want = np.vectorize(lambda v: ref.act(ref.ACT_SILU, v) * v)(z)
    _assert_close(inputs.to_f64(out), want, TOL["bf16"], "Wg = Wu")


@pytest.mark.parametrize("M,N,K", [(1, 1, 8), (5, 8, 64), (200, 1000, 256), (129, 257, 72), (64, 3000, 128), (260, 512, 320)])
@pytest.mark.parametrize("bias", [True, False])
def test_linear_lse_small(M, N, K, bias):
    li = inputs.linear_inputs(M, N, K, seed=3000 + M + N, bias=bias)
    buf, out = _guarded((M,), torch.float32)
    B.mtmc_linear_lse(li.X.cuda(), li.W.cuda(), None if li.b is None else li.b.cuda(), lse_out=out)
    B.mtmc_check_status()
    assert _canaries_intact(buf, M)
    want = ref.linear_lse(inputs.bf16_bits(li.X), inputs.bf16_bits(li.W), inputs.f32(li.b))
    _assert_close(inputs.to_f64(out), want, TOL["fp32"], "lse %dx%dx%d" % (M, N, K))


def test_linear_lse_shift_law():
    li = inputs.linear_inputs(150, 700, 128, seed=41)
    a = B.mtmc_linear_lse(li.X.cuda(), li.W.cuda(), li.b.cuda())
    b = B.mtmc_linear_lse(li.X.cuda(), li.W.cuda(), (li.b + 3.0).cuda())
    B.mtmc_check_status()
    assert torch.allclose(b - a, torch.full_like(a, 3.0), atol=2e-3)
    for c in (700.0, -900.0):       # lse(z + c) = lse(z) + c where exp(z + c) itself overflows / underflows in fp32
        far = B.mtmc_linear_lse(li.X.cuda(), li.W.cuda(), (li.b + c).cuda())
        want = ref.linear_lse(inputs.bf16_bits(li.X), inputs.bf16_bits(li.W), inputs.f32(li.b + c))
        _assert_close(inputs.to_f64(far), want, TOL["fp32"], "shift %g" % c)
    B.mtmc_check_status()


# ------------------------------------------------------------------ numeric edge cases, on every kernel family
# (tuning that forces the family, a shape that lands on it)
FAMILIES = [("single-CTA tiles", dict(cta_pair=-1), (300, 1000, 328)), ("256 x 256 pair tiles", dict(cta_pair=1), (600, 1000, 328)),
            ("512 x 256 pair tiles", dict(cta_pair=2), (600, 1000, 328)), ("cluster split-K", dict(), (128, 1024, 4096))]


def _expect_family(name):
    want = {"single-CTA tiles": "gemm_tiled_kernel", "256 x 256 pair tiles": "gemm_pair_kernel",
            "512 x 256 pair tiles": "gemm_big_kernel", "cluster split-K": "gemm_ksplit_kernel"}[name]
    assert want in B.mtmc_last_kernel_name(), "%s: ran %s" % (name, B.mtmc_last_kernel_name())


@pytest.mark.parametrize("family,tune,shape", FAMILIES, ids=[f[0] for f in FAMILIES])
def test_lse_edge_cases(family, tune, shape):
    """All-equal logits (W = 0: lse = lse(b), without bias ln N), one dominant logit (a weight row scaled by 64),
    and the shift law at +-500 -- where exp of the unshifted logits would overflow or vanish in fp32."""
    M, N, K = shape
    li = inputs.linear_inputs(M, N, K, seed=9500 + M)
    Xb, Wb, bf = inputs.bf16_bits(li.X), inputs.bf16_bits(li.W), inputs.f32(li.b)
    Xd, Wd, bd = li.X.cuda(), li.W.cuda(), li.b.cuda()
    W0 = torch.zeros_like(li.W)
    Wdom = li.W.clone()
    Wdom[N // 3] = (Wdom[N // 3].float() * 64.0).bfloat16()           # exact: a power of two
    B.mtmc_set_tuning(**tune)
    try:
        zero_b = B.mtmc_linear_lse(Xd, W0.cuda(), bd)
        _expect_family(family)
        zero_nob = B.mtmc_linear_lse(Xd, W0.cuda(), None)
        dom = B.mtmc_linear_lse(Xd, Wdom.cuda(), bd)
        up = B.mtmc_linear_lse(Xd, Wd, (li.b + 500.0).cuda())
        down = B.mtmc_linear_lse(Xd, Wd, (li.b - 500.0).cuda())
        mx, arg = B.mtmc_linear_rowmax(Xd, Wdom.cuda(), bd)
        B.mtmc_check_status()
    finally:
        B.mtmc_set_tuning()
    _assert_close(inputs.to_f64(zero_b), ref.linear_lse(Xb, inputs.bf16_bits(W0), bf), TOL["fp32"], family + ": W = 0")
    _assert_close(inputs.to_f64(zero_nob), np.full(M, np.log(N)), TOL["fp32"], family + ": W = 0, no bias = ln N")
    _assert_close(inputs.to_f64(dom), ref.linear_lse(Xb, inputs.bf16_bits(Wdom), bf), TOL["fp32"], family + ": dominant logit")
    _assert_close(inputs.to_f64(up), ref.linear_lse(Xb, Wb, inputs.f32(li.b + 500.0)), TOL["fp32"], family + ": bias + 500")
    _assert_close(inputs.to_f64(down), ref.linear_lse(Xb, Wb, inputs.f32(li.b - 500.0)), TOL["fp32"], family + ": bias - 500")
    want_mx, _ = ref.linear_rowmax(Xb, inputs.bf16_bits(Wdom), bf)
    _assert_close(inputs.to_f64(mx), want_mx, TOL["fp32"], family + ": row max with a dominant column")


@pytest.mark.parametrize("family,tune,shape", FAMILIES, ids=[f[0] for f in FAMILIES])
def test_swiglu_zero_gate_and_zero_up_are_exact_zeros(family, tune, shape):
    M, N, K = shape
    si = inputs.swiglu_inputs(M, N, K, seed=9600 + M)
    Z = torch.zeros_like(si.Wg)
    B.mtmc_set_tuning(**tune)
    try:
        zero_gate = B.mtmc_swiglu(si.X.cuda(), Z.cuda(), si.Wu.cuda())
        _expect_family(family)
        zero_up = B.mtmc_swiglu(si.X.cuda(), si.Wg.cuda(), Z.cuda())
        B.mtmc_check_status()
    finally:
        B.mtmc_set_tuning()
    assert bool((zero_gate.float() == 0).all()), family + ": Wg = 0"
    assert bool((zero_up.float() == 0).all()), family + ": Wu = 0"


def _signed_zeros_and_denormals(M, K, seed):
    """bf16 X [M,K]: row blocks of +0, of -0, of bf16 denormals (both signs), and ordinary rows with zeros and
    denormals sprinkled in."""
    g = torch.Generator().manual_seed(seed)
    X = torch.randn(M, K, generator=g).bfloat16()
    bits = X.view(torch.int16).clone()
    q = max(1, M // 4)
    bits[:q] = 0                                            # +0
    bits[q:2 * q] = -32768                                  # -0 (0x8000)
    den = torch.randint(1, 128, (q, K), generator=g, dtype=torch.int16)        # denormals: exponent 0, mantissa 1..127
    sign = torch.randint(0, 2, (q, K), generator=g, dtype=torch.int16) * -32768
    bits[2 * q:3 * q] = den | sign
    mask = torch.rand(M - 3 * q, K, generator=g) < 0.05
    tail = bits[3 * q:]
    tail[mask] = (den[:1].expand(M - 3 * q, K))[mask]
    return bits.view(torch.bfloat16)


@pytest.mark.parametrize("family,tune,shape", FAMILIES + [("weight streaming", dict(), (16, 640, 1024))],
                         ids=[f[0] for f in FAMILIES] + ["weight streaming"])
def test_signed_zero_and_denormal_inputs(family, tune, shape):
    """Rows of +0, -0 and bf16 denormals in X: the outputs are act(b) (up to products far below the tolerance),
    finite, and the ordinary rows are unaffected by their neighbours."""
    M, N, K = shape
    li = inputs.linear_inputs(M, N, K, seed=9700 + M)
    X = _signed_zeros_and_denormals(M, K, seed=9701 + M)
    B.mtmc_set_tuning(**tune)
    try:
        out = B.mtmc_fused_linear(X.cuda(), li.W.cuda(), li.b.cuda(), "gelu_tanh", "fp32")
        if family != "weight streaming":
            _expect_family(family)
        lse = B.mtmc_linear_lse(X.cuda(), li.W.cuda(), li.b.cuda()) if family != "weight streaming" else None
        B.mtmc_check_status()
    finally:
        B.mtmc_set_tuning()
    Xb, Wb, bf = inputs.bf16_bits(X), inputs.bf16_bits(li.W), inputs.f32(li.b)
    _assert_close(inputs.to_f64(out), ref.fused_linear(Xb, Wb, bf, ref.ACT_GELU_TANH), TOL["fp32"], family + ": zeros and denormals")
    if lse is not None:
        _assert_close(inputs.to_f64(lse), ref.linear_lse(Xb, Wb, bf), TOL["fp32"], family + ": lse with zeros and denormals")


# ------------------------------------------------------------------ row max and cross entropy of the fused logits
def _check_rowmax(li, mx_gpu, arg_gpu, what):
    X, W, b = inputs.bf16_bits(li.X), inputs.bf16_bits(li.W), inputs.f32(li.b)
    want_mx, want_arg = ref.linear_rowmax(X, W, b)
    _assert_close(inputs.to_f64(mx_gpu), want_mx, TOL["fp32"], what + " max")
    _, logits = ref.linear_lse(X, W, b, want_logits=True)
    arg = arg_gpu.cpu().numpy().astype(np.int64)
    assert np.all((arg >= 0) & (arg < logits.shape[1]))
    # fp32 and fp64 may order near-ties differently: the column the GPU names must hold the maximum within
    # tolerance, and wherever the runner-up is clearly lower the two must name the same column
    picked = logits[np.arange(logits.shape[0]), arg]
    assert np.all(np.abs(picked - want_mx) <= 1e-3 + 1e-3 * np.abs(want_mx)), what + " argmax validity"
    if logits.shape[1] > 1:
        second = np.partition(logits, -2, axis=1)[:, -2]
        clear = (want_mx - second) > 1e-2
        assert np.array_equal(arg[clear], want_arg[clear]), what + " argmax"


@pytest.mark.parametrize("M,N,K", [(1, 1, 8), (5, 8, 64), (200, 1000, 256), (129, 257, 72), (64, 3000, 128), (600, 1100, 192)])
def test_linear_rowmax_small(M, N, K):
    li = inputs.linear_inputs(M, N, K, seed=5000 + M + N)
    bufm, mx = _guarded((M,), torch.float32)
    arg = torch.full((M,), -7, dtype=torch.int32, device="cuda")
    B.mtmc_linear_rowmax(li.X.cuda(), li.W.cuda(), li.b.cuda(), max_out=mx, argmax_out=arg)
    B.mtmc_check_status()
    assert _canaries_intact(bufm, M)
    _check_rowmax(li, mx, arg, "rowmax %dx%dx%d" % (M, N, K))
    only_max, none = B.mtmc_linear_rowmax(li.X.cuda(), li.W.cuda(), li.b.cuda(), want_argmax=False)
    assert none is None and torch.equal(only_max, mx)


def test_linear_rowmax_ties_go_to_the_lowest_column():
    li = inputs.linear_inputs(140, 700, 64, seed=5100)
    W = li.W.clone(); b = li.b.clone()
    W[650] = W[13]; b[650] = b[13]; W[300] = W[13]; b[300] = b[13]        # three identical columns
    _, arg = B.mtmc_linear_rowmax(li.X.cuda(), W.cuda(), b.cuda())
    B.mtmc_check_status()
    a = arg.cpu().numpy()
    assert not np.any((a == 650) | (a == 300))


@pytest.mark.parametrize("M,N,K", [(1, 1, 8), (5, 8, 64), (200, 1000, 256), (129, 257, 72), (64, 3000, 128), (600, 1100, 192)])
def test_linear_cross_entropy_small(M, N, K):
    li = inputs.linear_inputs(M, N, K, seed=5200 + M + N)
    tgt = torch.from_numpy(np.random.default_rng(M + N).integers(0, N, size=M))
    bufl, loss = _guarded((M,), torch.float32)
    _, lse = B.mtmc_linear_cross_entropy(li.X.cuda(), li.W.cuda(), li.b.cuda(), tgt.cuda(), loss_out=loss, want_lse=True)
    B.mtmc_check_status()
    assert _canaries_intact(bufl, M)
    want_loss, want_lse = ref.linear_cross_entropy(inputs.bf16_bits(li.X), inputs.bf16_bits(li.W), inputs.f32(li.b), tgt.numpy())
    _assert_close(inputs.to_f64(loss), want_loss, TOL["fp32"], "cross entropy %dx%dx%d" % (M, N, K))
    _assert_close(inputs.to_f64(lse), want_lse, TOL["fp32"], "lse of cross entropy")
    assert torch.equal(B.mtmc_linear_cross_entropy(li.X.cuda(), li.W.cuda(), li.b.cuda(), tgt.cuda()), loss)


def test_cross_entropy_target_out_of_range_gives_nan_for_that_row_only():
    li = inputs.linear_inputs(40, 300, 64, seed=5300)
    tgt = torch.arange(40, dtype=torch.int64) % 300
    tgt[7] = 300
    tgt[19] = -1
    loss = B.mtmc_linear_cross_entropy(li.X.cuda(), li.W.cuda(), li.b.cuda(), tgt.cuda())
    B.mtmc_check_status()
    bad = torch.isnan(loss).cpu().numpy()
    assert bad[7] and bad[19] and bad.sum() == 2


def test_rowmax_and_cross_entropy_at_lm_head_size_on_sampled_rows():
    c = inputs.CONFIGS["C4"]
    li = inputs.linear_inputs(c["M"], c["N"], c["K"], c["seed"])
    tgt = torch.from_numpy(np.random.default_rng(9).integers(0, c["N"], size=c["M"]))
    Xd, Wd, bd = li.X.cuda(), li.W.cuda(), li.b.cuda()
    mx, arg = B.mtmc_linear_rowmax(Xd, Wd, bd)
    loss, lse = B.mtmc_linear_cross_entropy(Xd, Wd, bd, tgt.cuda(), want_lse=True)
    B.mtmc_check_status()
    rows = np.unique(np.concatenate([[0, 127, 128, 255, 256, c["M"] - 1], np.random.default_rng(4).integers(0, c["M"], size=10)]))
    sub = inputs.LinearInputs(li.X[rows].contiguous(), li.W, li.b)
    idx = torch.from_numpy(rows).cuda()
    _check_rowmax(sub, mx[idx], arg[idx], "C4 rowmax sampled rows")
    want_loss, want_lse = ref.linear_cross_entropy(inputs.bf16_bits(sub.X), inputs.bf16_bits(sub.W), inputs.f32(sub.b), tgt.numpy()[rows])
    _assert_close(inputs.to_f64(loss[idx]), want_loss, TOL["fp32"], "C4 cross entropy sampled rows")
    _assert_close(inputs.to_f64(lse[idx]), want_lse, TOL["fp32"], "C4 lse sampled rows")
    # properties at full size: max <= lse <= max + ln N and loss >= lse - max >= 0 for every row
    assert bool((mx <= lse + 1e-3).all()) and bool((lse <= mx + np.log(c["N"]) + 1e-3).all())
    assert bool((loss >= lse - mx - 2e-3).all())


def test_decode_and_prefill_sweep_at_full_size():
    """M = 64 ... 512 rows against one 8192 x 8192 weight matrix (bias + GELU-tanh, bf16), every output against the
    oracle, and the kernel family that each batch size lands on: weight streaming up to 64 rows, cluster split-K
    up to 256, CTA pairs from there."""
    N = K = 8192
    li = inputs.linear_inputs(512, N, K, seed=8100)
    Wd, bd = li.W.cuda(), li.b.cuda()
    Wb, bf = inputs.bf16_bits(li.W), inputs.f32(li.b)
    for M, family in ((64, "skinny_splitk_kernel"), (65, "gemm_ksplit_kernel"), (96, "gemm_ksplit_kernel"), (128, "gemm_ksplit_kernel"),
                      (192, "gemm_ksplit_kernel"), (256, "gemm_ksplit_kernel"), (384, "gemm_pair_kernel"), (512, "gemm_pair_kernel")):
        X = li.X[:M].contiguous()
        buf, out = _guarded((M, N), torch.bfloat16)
        B.mtmc_fused_linear(X.cuda(), Wd, bd, "gelu_tanh", "bf16", out=out)
        ran = B.mtmc_last_kernel_name()
        B.mtmc_check_status()
        assert family in ran, "M = %d: ran %s" % (M, ran)
        assert _canaries_intact(buf, M * N)
        want = ref.fused_linear(inputs.bf16_bits(X), Wb, bf, ref.ACT_GELU_TANH)
        _assert_close(inputs.to_f64(out), want, TOL["bf16"], "%d x 8192 x 8192 on %s" % (M, ran))


# ------------------------------------------------------------------ row softmax written out as probabilities
# Probabilities are compared relative to their own size (a row of N of them averages 1/N, far below any absolute
# tolerance that suits activations): logit error (bf16 products, fp32 sums) and the hardware exp2 give a few 1e-4;
# a bf16 result adds two roundings of a value in [0, 1], 2^-8 together.  The absolute term only covers results that
# fp32 flushes to zero (below 2^-126).
SOFTMAX_TOL = {"fp32": (1e-30, 2e-3), "bf16": (1e-30, 1e-2)}


def _check_softmax(li, prob, lse, odt, what):
    Xb, Wb, bf = inputs.bf16_bits(li.X), inputs.bf16_bits(li.W), inputs.f32(li.b)
    want = ref.linear_softmax(Xb, Wb, bf)
    _assert_close(inputs.to_f64(prob), want, SOFTMAX_TOL[odt], what)
    if lse is not None:
        _assert_close(inputs.to_f64(lse), ref.linear_lse(Xb, Wb, bf), TOL["fp32"], what + ": lse")
    sums = prob.double().sum(dim=1).cpu().numpy()
    np.testing.assert_allclose(sums, np.ones_like(sums), rtol=0, atol=4e-3 if odt == "bf16" else 1e-4, err_msg=what + ": row sums")


@pytest.mark.parametrize("M,N,K", [(1, 1, 8), (5, 8, 64), (200, 1000, 256), (129, 257, 72), (64, 3000, 128), (260, 512, 320),
                                   (300, 2304, 2048), (130, 4100, 512), (700, 1300, 328),
                                   (128, 300, 4096), (200, 1100, 4096), (64, 2048, 2048), (16, 520, 1024)])
@pytest.mark.parametrize("odt", ["fp32", "bf16"])
def test_linear_softmax_small(M, N, K, odt):
    """Single-CTA tiles, pair tiles and cluster split-K (clusters of two, four and eight, also with pieces that lie
    wholly past N), whole and split wave tails, N a multiple of 32, of 8, of 4 and odd."""
    li = inputs.linear_inputs(M, N, K, seed=5400 + M + N, bias=(M % 2 == 0))
    buf, out = _guarded((M, N), torch.bfloat16 if odt == "bf16" else torch.float32)
    bufl, lse = _guarded((M,), torch.float32)
    B.mtmc_linear_softmax(li.X.cuda(), li.W.cuda(), None if li.b is None else li.b.cuda(), odt, prob_out=out, lse_out=lse)
    B.mtmc_check_status()
    assert _canaries_intact(buf, M * N) and _canaries_intact(bufl, M)
    _check_softmax(li, out, lse, odt, "softmax %dx%dx%d %s" % (M, N, K, odt))
    again = B.mtmc_linear_softmax(li.X.cuda(), li.W.cuda(), None if li.b is None else li.b.cuda(), odt)   # lse in the workspace
    B.mtmc_check_status()
    assert torch.equal(again, out), "run-to-run bits"


SOFTMAX_FAMILIES = [("single-CTA tiles", dict(cta_pair=-1), 0, (300, 1000, 328)), ("128-column tiles", dict(tile_n=128), 0, (300, 1000, 328)),
                    ("256 x 256 pair tiles", dict(cta_pair=1), -1, (600, 1000, 328)), ("pair tiles, stream-K", dict(cta_pair=1), 1, (600, 2304, 328)),
                    ("cluster split-K", dict(), 0, (128, 1024, 4096))]


@pytest.mark.parametrize("family,tune,sk,shape", SOFTMAX_FAMILIES, ids=[f[0] for f in SOFTMAX_FAMILIES])
@pytest.mark.parametrize("odt", ["fp32", "bf16"])
def test_linear_softmax_edge_cases(family, tune, sk, shape, odt):
    """On every kernel that carries the epilogue: equal logits (W = 0: softmax(b), without bias 1/N), one dominant logit
    (a weight row scaled by 64: one probability near 1, the rest tiny but right), and shifts of +-500 in the bias,
    which leave the probabilities alone although exp of the logits themselves overflows or vanishes in fp32."""
    M, N, K = shape
    li = inputs.linear_inputs(M, N, K, seed=9800 + M)
    Xd, Wd, bd = li.X.cuda(), li.W.cuda(), li.b.cuda()
    W0 = torch.zeros_like(li.W)
    Wdom = li.W.clone()
    Wdom[N // 3] = (Wdom[N // 3].float() * 64.0).bfloat16()
    B.mtmc_set_tuning(**tune)
    B.mtmc_set_schedule(sk)
    try:
        plain = B.mtmc_linear_softmax(Xd, Wd, bd, odt)
        want_kernel = "gemm_pair_kernel" if "pair" in family else "gemm_ksplit_kernel" if "split-K" in family else "gemm_tiled_kernel"
        assert want_kernel in B.mtmc_last_kernel_name(), "%s: ran %s" % (family, B.mtmc_last_kernel_name())
        zero_b = B.mtmc_linear_softmax(Xd, W0.cuda(), bd, odt)
        zero_nob = B.mtmc_linear_softmax(Xd, W0.cuda(), None, odt)
        dom = B.mtmc_linear_softmax(Xd, Wdom.cuda(), bd, odt)
        up = B.mtmc_linear_softmax(Xd, Wd, (li.b + 500.0).cuda(), odt)
        down = B.mtmc_linear_softmax(Xd, Wd, (li.b - 500.0).cuda(), odt)
        B.mtmc_check_status()
    finally:
        B.mtmc_set_schedule(0)
        B.mtmc_set_tuning()
    tol = SOFTMAX_TOL[odt]
    _check_softmax(li, plain, None, odt, family)
    _check_softmax(inputs.LinearInputs(li.X, W0, li.b), zero_b, None, odt, family + ": W = 0")
    _assert_close(inputs.to_f64(zero_nob), np.full((M, N), 1.0 / N), tol, family + ": W = 0, no bias = 1/N")
    _check_softmax(inputs.LinearInputs(li.X, Wdom, li.b), dom, None, odt, family + ": dominant logit")
    _check_softmax(inputs.LinearInputs(li.X, li.W, li.b + 500.0), up, None, odt, family + ": bias + 500")
    _check_softmax(inputs.LinearInputs(li.X, li.W, li.b - 500.0), down, None, odt, family + ": bias - 500")


def test_linear_softmax_with_caller_workspace_and_bad_arguments():
    M, N, K = 300, 2304, 2048
    li = inputs.linear_inputs(M, N, K, seed=5500)
    Xd, Wd, bd = li.X.cuda(), li.W.cuda(), li.b.cuda()
    for sk in (1, -1):
        B.mtmc_set_schedule(sk)
        try:
            need = B.mtmc_workspace_bytes("linear_softmax", M, N, K)      # under the schedule that the call will run with
            assert need >= B.mtmc_workspace_bytes("linear_lse", M, N, K) > 0
            guard = torch.full((need + 8192,), 0x5A, dtype=torch.uint8, device="cuda")
            off = (-guard.data_ptr()) % 256 + 3840
            B.mtmc_set_workspace(guard[off:off + need])
            prob = B.mtmc_linear_softmax(Xd, Wd, bd, "bf16")
            B.mtmc_check_status()
        finally:
            B.mtmc_set_schedule(0)
            B.mtmc_set_workspace(None)
        assert bool((guard[:off] == 0x5A).all()) and bool((guard[off + need:] == 0x5A).all())
        _check_softmax(li, prob, None, "bf16", "softmax, caller workspace, schedule %d" % sk)
    L = B.load()
    assert L.mtmc_linear_softmax(Xd.data_ptr(), Wd.data_ptr(), None, M, N, K, 7, prob.data_ptr(), None) == B.ERR_INVALID_ARG
    assert L.mtmc_linear_softmax(Xd.data_ptr(), Wd.data_ptr(), None, M, N, K, 0, None, None) == B.ERR_INVALID_ARG
    assert L.mtmc_linear_softmax(Xd.data_ptr(), Wd.data_ptr(), None, M, N, K + 4, 0, prob.data_ptr(), None) == B.ERR_UNSUPPORTED_SHAPE
    B.mtmc_check_status()


@pytest.mark.parametrize("M,N,K,padx,padw,pado", [(100, 72, 136, 8, 24, 3), (300, 520, 328, 16, 8, 8), (300, 2304, 2048, 64, 64, 1024),
                                                  (1100, 1300, 1024, 8, 16, 4)])
@pytest.mark.parametrize("odt", ["fp32", "bf16"])
def test_linear_softmax_on_strided_views(M, N, K, padx, padw, pado, odt):
    """X, W and the probabilities as column slices of wider matrices (single-CTA and pair kernels; pitches that allow
    16-byte accesses and pitches that do not): the dense call's bits, the neighbours untouched."""
    li = inputs.linear_inputs(M, N, K, seed=9070 + M + N)
    tdt = torch.bfloat16 if odt == "bf16" else torch.float32
    Xw = torch.full((M, K + padx), 3.0, dtype=torch.bfloat16, device="cuda")
    Ww = torch.full((N, K + padw), -2.0, dtype=torch.bfloat16, device="cuda")
    Ow = torch.full((M, N + pado), 7.0, dtype=tdt, device="cuda")
    offx, offw, offo = (8 if padx >= 16 else 0), (8 if padw >= 16 else 0), (8 if pado >= 16 else 0)
    Xv, Wv, Ov = Xw[:, offx:offx + K], Ww[:, offw:offw + K], Ow[:, offo:offo + N]
    Xv.copy_(li.X.cuda()); Wv.copy_(li.W.cuda())
    B.mtmc_linear_softmax_strided(Xv, Wv, li.b.cuda(), odt, prob_out=Ov)
    B.mtmc_check_status()
    _check_softmax(li, Ov.contiguous(), None, odt, "strided softmax %dx%dx%d %s" % (M, N, K, odt))
    assert bool((Ow[:, :offo] == 7.0).all()) and bool((Ow[:, offo + N:] == 7.0).all())
    assert torch.equal(B.mtmc_linear_softmax(li.X.cuda(), li.W.cuda(), li.b.cuda(), odt), Ov.contiguous())


@pytest.mark.parametrize("M,N,K", [(5, 8, 64), (200, 1000, 256), (129, 257, 80), (600, 3000, 128), (1024, 4096, 512)])
@pytest.mark.parametrize("odt", ["fp32", "bf16"])
def test_linear_softmax_fp8(M, N, K, odt):
    fi = inputs.fp8_linear_inputs(M, N, K, seed=7500 + M + N)
    buf, out = _guarded((M, N), torch.bfloat16 if odt == "bf16" else torch.float32)
    _, lse = B.mtmc_linear_softmax_fp8(fi.X.cuda(), fi.W.cuda(), fi.b.cuda(), fi.scale_x, fi.scale_w, odt, prob_out=out, want_lse=True)
    B.mtmc_check_status()
    assert _canaries_intact(buf, M * N)
    X8, W8, bf = inputs.fp8_bits(fi.X), inputs.fp8_bits(fi.W), inputs.f32(fi.b)
    _assert_close(inputs.to_f64(out), ref.linear_softmax_fp8(X8, W8, bf, fi.scale_x, fi.scale_w), SOFTMAX_TOL[odt],
                  "softmax fp8 %dx%dx%d %s" % (M, N, K, odt))
    _assert_close(inputs.to_f64(lse), ref.linear_lse_fp8(X8, W8, bf, fi.scale_x, fi.scale_w), TOL["fp32"], "lse of softmax fp8")


def test_linear_softmax_random_shapes_kernels_and_schedules():
    """Seeded sweep: 60 shapes (M to 900, N to 6000, K to 2560) over output types, bias or none, logits spread by a
    bias forty times as wide, the kernel choices of the tuning hook, the stream-K schedule and E4M3 operands."""
    rng = np.random.default_rng(20261)
    for it in range(60):
        M, N = int(rng.integers(1, 900)), int(rng.integers(1, 6000))
        K = int(rng.integers(1, 160)) * 8 if rng.random() < 0.7 else int(rng.integers(1, 40)) * 64
        odt = "bf16" if rng.random() < 0.5 else "fp32"
        bias = rng.random() < 0.7
        r = rng.random()
        tune = dict(cta_pair=1) if r < 0.2 else dict(cta_pair=-1) if r < 0.35 else dict(tile_n=128) if r < 0.45 else {}
        sk = int(rng.choice([0, 1, -1]))
        fp8 = rng.random() < 0.25
        what = "case %d: %dx%dx%d %s bias=%s %r stream_k=%d fp8=%s" % (it, M, N, K, odt, bias, tune, sk, fp8)
        B.mtmc_set_tuning(**tune)
        B.mtmc_set_schedule(sk)
        try:
            if fp8:
                K = max(16, K // 16 * 16)
                fi = inputs.fp8_linear_inputs(M, N, K, seed=it)
                out = B.mtmc_linear_softmax_fp8(fi.X.cuda(), fi.W.cuda(), fi.b.cuda() if bias else None, fi.scale_x, fi.scale_w, odt)
                want = ref.linear_softmax_fp8(inputs.fp8_bits(fi.X), inputs.fp8_bits(fi.W), inputs.f32(fi.b) if bias else None,
                                              fi.scale_x, fi.scale_w)
            else:
                li = inputs.linear_inputs(M, N, K, seed=it, bias=bias)
                if bias and rng.random() < 0.3:
                    li.b = li.b * 40.0
                out = B.mtmc_linear_softmax(li.X.cuda(), li.W.cuda(), None if li.b is None else li.b.cuda(), odt)
                want = ref.linear_softmax(inputs.bf16_bits(li.X), inputs.bf16_bits(li.W), inputs.f32(li.b))
            B.mtmc_check_status()
        finally:
            B.mtmc_set_schedule(0)
            B.mtmc_set_tuning()
        _assert_close(inputs.to_f64(out), want, SOFTMAX_TOL[odt], what)
        sums = out.double().sum(dim=1)
        assert bool(((sums - 1.0).abs() <= (4e-3 if odt == "bf16" else 1e-4)).all()), what + ": row sums"


def test_linear_softmax_at_lm_head_size_on_sampled_rows():
    c = inputs.CONFIGS["C4"]
    li = inputs.linear_inputs(c["M"], c["N"], c["K"], c["seed"])
    Xd, Wd, bd = li.X.cuda(), li.W.cuda(), li.b.cuda()
    prob, lse = B.mtmc_linear_softmax(Xd, Wd, bd, "bf16", want_lse=True)
    assert "gemm_pair_kernel" in B.mtmc_last_kernel_name()
    lse_alone = B.mtmc_linear_lse(Xd, Wd, bd)
    B.mtmc_check_status()
    rows = np.unique(np.concatenate([[0, 127, 128, 255, 256, c["M"] - 1], np.random.default_rng(6).integers(0, c["M"], size=4)]))
    want = ref.linear_softmax_rows(inputs.bf16_bits(li.X), inputs.bf16_bits(li.W), inputs.f32(li.b), rows)
    idx = torch.from_numpy(rows).cuda()
    _assert_close(inputs.to_f64(prob[idx]), want, SOFTMAX_TOL["bf16"], "C4 softmax sampled rows")
    # properties at full size: every row sums to one, no probability above one or below zero, lse as the reduction alone
    sums = prob.float().sum(dim=1)
    assert bool(((sums - 1.0).abs() <= 4e-3).all()), "row sums %.5f .. %.5f" % (float(sums.min()), float(sums.max()))
    assert bool((prob >= 0).all()) and bool((prob <= 1).all())
    assert torch.allclose(lse, lse_alone, rtol=0, atol=1e-4)


# ------------------------------------------------------------------ cluster split-K (few tiles, long K)
# Problems of at most half a wave of 128 x 256 tiles: a cluster of 2, 4 or 8 CTAs per tile, reduce-scatter through
# distributed shared memory.  Ragged in every dimension, k-blocks that do not divide evenly among the CTAs,
# column groups that lie wholly past N.
KSPLIT = [(128, 1024, 4096), (100, 520, 1096), (300, 1000, 2056), (512, 2048, 2048), (700, 1100, 1160), (65, 8192, 1024),
          (128, 300, 2048), (200, 4096, 4096)]


@pytest.mark.parametrize("M,N,K", KSPLIT)
@pytest.mark.parametrize("act,odt", [("gelu_tanh", "bf16"), ("none", "fp32")])
def test_cluster_split_k_fused_linear(M, N, K, act, odt):
    li = inputs.linear_inputs(M, N, K, seed=8000 + M + N)
    want = ref.fused_linear(inputs.bf16_bits(li.X), inputs.bf16_bits(li.W), inputs.f32(li.b), B.ACT[act])
    Xd, Wd, bd = li.X.cuda(), li.W.cuda(), li.b.cuda()
    buf, out = _guarded((M, N), torch.bfloat16 if odt == "bf16" else torch.float32)
    B.mtmc_fused_linear(Xd, Wd, bd, act, odt, out=out)
    B.mtmc_check_status()
    assert _canaries_intact(buf, M * N)
    _assert_close(inputs.to_f64(out), want, TOL[odt], "cluster split-K %dx%dx%d %s" % (M, N, K, odt))
    # the partials are added in rank order: every launch gives the same bits
    for _ in range(5):
        assert torch.equal(B.mtmc_fused_linear(Xd, Wd, bd, act, odt), out)
    # smaller clusters, and the tiled kernel without any split, stay within tolerance as well
    for cap in (4, 2, 1):
        B.mtmc_set_tuning(split_k=cap)
        try:
            other = B.mtmc_fused_linear(Xd, Wd, bd, act, odt)
            B.mtmc_check_status()
        finally:
            B.mtmc_set_tuning()
        _assert_close(inputs.to_f64(other), want, TOL[odt], "split_k cap %d %dx%dx%d %s" % (cap, M, N, K, odt))


@pytest.mark.parametrize("M,N,K", [(128, 1024, 4096), (300, 1000, 2056), (512, 2048, 2048), (700, 1100, 1160), (128, 300, 2048)])
def test_cluster_split_k_other_epilogues(M, N, K):
    li = inputs.linear_inputs(M, N, K, seed=8100 + M + N)
    Xb, Wb, bf = inputs.bf16_bits(li.X), inputs.bf16_bits(li.W), inputs.f32(li.b)
    Xd, Wd, bd = li.X.cuda(), li.W.cuda(), li.b.cuda()
    lse = B.mtmc_linear_lse(Xd, Wd, bd)
    _assert_close(inputs.to_f64(lse), ref.linear_lse(Xb, Wb, bf), TOL["fp32"], "split-K lse %dx%dx%d" % (M, N, K))
    mx, arg = B.mtmc_linear_rowmax(Xd, Wd, bd)
    _check_rowmax(li, mx, arg, "split-K rowmax %dx%dx%d" % (M, N, K))
    tgt = torch.from_numpy(np.random.default_rng(M + N).integers(0, N, size=M))
    loss = B.mtmc_linear_cross_entropy(Xd, Wd, bd, tgt.cuda())
    want_loss, _ = ref.linear_cross_entropy(Xb, Wb, bf, tgt.numpy())
    _assert_close(inputs.to_f64(loss), want_loss, TOL["fp32"], "split-K cross entropy")
    R = torch.randn(M, N, generator=torch.Generator().manual_seed(M * N)).bfloat16()
    res = B.mtmc_fused_linear_residual(Xd, Wd, bd, R.cuda(), "silu", "bf16")
    _assert_close(inputs.to_f64(res), ref.fused_linear_residual(Xb, Wb, bf, inputs.bf16_bits(R), ref.ACT_SILU), TOL["bf16"],
                  "split-K residual")
    B.mtmc_check_status()
    si = inputs.swiglu_inputs(M, N, K, seed=8200 + M)
    sw = B.mtmc_swiglu(si.X.cuda(), si.Wg.cuda(), si.Wu.cuda())
    _assert_close(inputs.to_f64(sw), ref.swiglu(inputs.bf16_bits(si.X), inputs.bf16_bits(si.Wg), inputs.bf16_bits(si.Wu)),
                  TOL["bf16"], "split-K swiglu")
    fi = inputs.fp8_linear_inputs(M, N, 2 * K, seed=8300 + M)
    f8 = B.mtmc_fused_linear_fp8(fi.X.cuda(), fi.W.cuda(), fi.b.cuda(), fi.scale_x, fi.scale_w, "gelu_tanh", "bf16")
    want8 = ref.fused_linear_fp8(inputs.fp8_bits(fi.X), inputs.fp8_bits(fi.W), inputs.f32(fi.b), fi.scale_x, fi.scale_w, ref.ACT_GELU_TANH)
    _assert_close(inputs.to_f64(f8), want8, TOL["bf16"], "split-K fp8")
    B.mtmc_check_status()


@pytest.mark.parametrize("M,N,K", [(128, 300, 4096), (200, 1100, 4096)])
@pytest.mark.parametrize("own_workspace", [False, True])
def test_row_reductions_on_clusters_of_eight_with_a_ragged_last_tile(M, N, K, own_workspace):
    """Clusters of eight CTAs per 256-column tile leave eight partials per tile, also for a last tile that lies
    mostly past N: the workspace must hold ceil(N/256) * 8 pieces per row.  Run on the library's scratch and on a
    caller workspace of exactly mtmc_workspace_bytes inside a canary-guarded buffer; bf16 and E4M3 operands."""
    li = inputs.linear_inputs(M, N, K, seed=8400 + M + N)
    fi = inputs.fp8_linear_inputs(M, N, 2 * K, seed=8450 + M + N)
    Xb, Wb, bf = inputs.bf16_bits(li.X), inputs.bf16_bits(li.W), inputs.f32(li.b)
    X8, W8, b8 = inputs.fp8_bits(fi.X), inputs.fp8_bits(fi.W), inputs.f32(fi.b)
    tgt = torch.from_numpy(np.random.default_rng(M + N).integers(0, N, size=M))
    Xd, Wd, bd, td = li.X.cuda(), li.W.cuda(), li.b.cuda(), tgt.cuda()
    X8d, W8d, b8d = fi.X.cuda(), fi.W.cuda(), fi.b.cuda()
    guard = None
    if own_workspace:
        need = max(B.mtmc_workspace_bytes(op, M, N, K) for op in ("linear_lse", "linear_rowmax", "linear_cross_entropy"))
        assert need == B.mtmc_workspace_bytes("linear_cross_entropy", M, N, 2 * K)        # the figure does not depend on K
        guard = torch.full((need + 2 * 4096,), 0x5A, dtype=torch.uint8, device="cuda")
        off = (-guard.data_ptr()) % 256 + 3840              # a 256-byte aligned start with canary bytes on both sides
        assert (guard.data_ptr() + off) % 256 == 0
        B.mtmc_set_workspace(guard[off:off + need])
    try:
        lse = B.mtmc_linear_lse(Xd, Wd, bd)
        assert "gemm_ksplit_kernel<EPI_LSE, 8>" in B.mtmc_last_kernel_name(), B.mtmc_last_kernel_name()
        mx, arg = B.mtmc_linear_rowmax(Xd, Wd, bd)
        loss, lse2 = B.mtmc_linear_cross_entropy(Xd, Wd, bd, td, want_lse=True)
        lse8 = B.mtmc_linear_lse_fp8(X8d, W8d, b8d, fi.scale_x, fi.scale_w)
        mx8, _ = B.mtmc_linear_rowmax_fp8(X8d, W8d, b8d, fi.scale_x, fi.scale_w)
        loss8 = B.mtmc_linear_cross_entropy_fp8(X8d, W8d, b8d, fi.scale_x, fi.scale_w, td)
        B.mtmc_check_status()
    finally:
        B.mtmc_set_workspace(None)
    if guard is not None:
        assert bool((guard[:off] == 0x5A).all()) and bool((guard[off + need:] == 0x5A).all()), "write outside the workspace"
    want_loss, want_lse = ref.linear_cross_entropy(Xb, Wb, bf, tgt.numpy())
    _assert_close(inputs.to_f64(lse), want_lse, TOL["fp32"], "lse")
    _assert_close(inputs.to_f64(lse2), want_lse, TOL["fp32"], "lse of cross entropy")
    _assert_close(inputs.to_f64(loss), want_loss, TOL["fp32"], "cross entropy")
    _check_rowmax(li, mx, arg, "rowmax")
    want_loss8, want_lse8 = ref.linear_cross_entropy_fp8(X8, W8, b8, fi.scale_x, fi.scale_w, tgt.numpy())
    _assert_close(inputs.to_f64(lse8), want_lse8, TOL["fp32"], "fp8 lse")
    _assert_close(inputs.to_f64(loss8), want_loss8, TOL["fp32"], "fp8 cross entropy")
    want_mx8, _ = ref.linear_rowmax_fp8(X8, W8, b8, fi.scale_x, fi.scale_w)
    _assert_close(inputs.to_f64(mx8), want_mx8, TOL["fp32"], "fp8 rowmax")


def test_calls_on_two_streams_keep_their_scratch_apart():
    """Library-owned scratch is per stream: logsumexp calls of different shapes issued alternately on two streams,
    without any synchronisation between them, each match the oracle."""
    a = inputs.linear_inputs(700, 3000, 512, seed=8500)
    b = inputs.linear_inputs(520, 5000, 256, seed=8501)
    dev = [(t.X.cuda(), t.W.cuda(), t.b.cuda()) for t in (a, b)]
    streams = [torch.cuda.Stream(), torch.cuda.Stream()]
    torch.cuda.synchronize()
    outs = [[], []]
    for rep in range(6):
        for i in (0, 1):
            with torch.cuda.stream(streams[i]):
                outs[i].append(B.mtmc_linear_lse(*dev[i]))
    torch.cuda.synchronize()
    B.mtmc_check_status()
    for i, t in enumerate((a, b)):
        want = ref.linear_lse(inputs.bf16_bits(t.X), inputs.bf16_bits(t.W), inputs.f32(t.b))
        for o in outs[i]:
            _assert_close(inputs.to_f64(o), want, TOL["fp32"], "stream %d" % i)


# ------------------------------------------------------------------ stream-K schedule of the 256 x 256 pair kernel
# Forced by the schedule hook: problems with somewhat more tiles than CTA pairs (81 to 100 tiles on 74 pairs: the last
# full wave and the remainder are dealt by k-blocks, two holders per shared tile) and with fewer tiles than pairs
# (everything is dealt by k-blocks); shares that begin and end inside tiles, k-block counts that do not divide,
# ragged rows / columns / K.
STREAMK = [(2304, 2304, 328), (2304, 2400, 4096), (2500, 2200, 72), (2304, 2304, 64),
           # fewer tiles than pairs: every tile has several holders (up to five), some pairs' shares lie inside one tile
           (300, 2304, 4096), (128, 8192, 2048), (520, 1000, 1096), (300, 520, 72)]


def _streamk(fn):
    B.mtmc_set_tuning(cta_pair=1)
    B.mtmc_set_schedule(1)
    try:
        return fn()
    finally:
        B.mtmc_set_schedule(0)
        B.mtmc_set_tuning()


@pytest.mark.parametrize("M,N,K", STREAMK)
@pytest.mark.parametrize("act,odt", [("gelu_tanh", "bf16"), ("none", "fp32")])
def test_stream_k_fused_linear(M, N, K, act, odt):
    li = inputs.linear_inputs(M, N, K, seed=8600 + M + N + K)
    want = ref.fused_linear(inputs.bf16_bits(li.X), inputs.bf16_bits(li.W), inputs.f32(li.b), B.ACT[act])
    Xd, Wd, bd = li.X.cuda(), li.W.cuda(), li.b.cuda()
    buf, out = _guarded((M, N), torch.bfloat16 if odt == "bf16" else torch.float32)

    def run():
        B.mtmc_fused_linear(Xd, Wd, bd, act, odt, out=out)
        assert "gemm_pair_kernel" in B.mtmc_last_kernel_name()
        B.mtmc_check_status()
        return [B.mtmc_fused_linear(Xd, Wd, bd, act, odt) for _ in range(4)]
    again = _streamk(run)
    B.mtmc_check_status()
    assert _canaries_intact(buf, M * N)
    _assert_close(inputs.to_f64(out), want, TOL[odt], "stream-K %dx%dx%d %s" % (M, N, K, odt))
    for o in again:                    # whoever of a shared tile's two holders finishes it, the bits are the same
        assert torch.equal(o, out)


@pytest.mark.parametrize("M,N,K", [(2304, 1160, 328), (2304, 2400, 1096)])
def test_stream_k_other_epilogues(M, N, K):
    li = inputs.linear_inputs(M, N, K, seed=8700 + M + N)
    Xb, Wb, bf = inputs.bf16_bits(li.X), inputs.bf16_bits(li.W), inputs.f32(li.b)
    Xd, Wd, bd = li.X.cuda(), li.W.cuda(), li.b.cuda()
    tgt = torch.from_numpy(np.random.default_rng(M + N).integers(0, N, size=M))
    si = inputs.swiglu_inputs(M, N, K, seed=8710 + M)
    fi = inputs.fp8_linear_inputs(M, N, 2 * K, seed=8720 + M)
    R = torch.randn(M, N, generator=torch.Generator().manual_seed(M + N)).bfloat16()

    def run():
        r = {}
        r["lse"] = B.mtmc_linear_lse(Xd, Wd, bd)
        r["rowmax"] = B.mtmc_linear_rowmax(Xd, Wd, bd)
        r["xent"] = B.mtmc_linear_cross_entropy(Xd, Wd, bd, tgt.cuda())
        r["swiglu"] = B.mtmc_swiglu(si.X.cuda(), si.Wg.cuda(), si.Wu.cuda())
        r["res"] = B.mtmc_fused_linear_residual(Xd, Wd, bd, R.cuda(), "silu", "bf16")
        r["fp8"] = B.mtmc_fused_linear_fp8(fi.X.cuda(), fi.W.cuda(), fi.b.cuda(), fi.scale_x, fi.scale_w, "gelu_tanh", "bf16")
        assert "gemm_pair_kernel" in B.mtmc_last_kernel_name()
        B.mtmc_check_status()
        return r
    r = _streamk(run)
    _assert_close(inputs.to_f64(r["lse"]), ref.linear_lse(Xb, Wb, bf), TOL["fp32"], "stream-K lse")
    _check_rowmax(li, r["rowmax"][0], r["rowmax"][1], "stream-K rowmax")
    want_loss, _ = ref.linear_cross_entropy(Xb, Wb, bf, tgt.numpy())
    _assert_close(inputs.to_f64(r["xent"]), want_loss, TOL["fp32"], "stream-K cross entropy")
    _assert_close(inputs.to_f64(r["swiglu"]), ref.swiglu(inputs.bf16_bits(si.X), inputs.bf16_bits(si.Wg), inputs.bf16_bits(si.Wu)),
                  TOL["bf16"], "stream-K swiglu")
    _assert_close(inputs.to_f64(r["res"]), ref.fused_linear_residual(Xb, Wb, bf, inputs.bf16_bits(R), ref.ACT_SILU), TOL["bf16"],
                  "stream-K residual")
    want8 = ref.fused_linear_fp8(inputs.fp8_bits(fi.X), inputs.fp8_bits(fi.W), inputs.f32(fi.b), fi.scale_x, fi.scale_w, ref.ACT_GELU_TANH)
    _assert_close(inputs.to_f64(r["fp8"]), want8, TOL["bf16"], "stream-K fp8")


@pytest.mark.parametrize("M,N,K", [(2304, 2304, 328), (300, 2304, 2048)])
def test_stream_k_with_caller_workspace(M, N, K):
    """The accumulator parts and flag words in a caller's workspace of exactly mtmc_workspace_bytes, canaries around it
    (also below 512 rows, where the pair kernel now starts)."""
    li = inputs.linear_inputs(M, N, K, seed=8800 + M)
    Xd, Wd, bd = li.X.cuda(), li.W.cuda(), li.b.cuda()

    def run():
        need = B.mtmc_workspace_bytes("linear_lse", M, N, K)
        assert need >= B.mtmc_workspace_bytes("fused_linear", M, N, K) > 0
        guard = torch.full((need + 8192,), 0x5A, dtype=torch.uint8, device="cuda")
        off = (-guard.data_ptr()) % 256 + 3840
        B.mtmc_set_workspace(guard[off:off + need])
        try:
            out = B.mtmc_fused_linear(Xd, Wd, bd, "relu", "fp32")
            lse = B.mtmc_linear_lse(Xd, Wd, bd)
            B.mtmc_check_status()
        finally:
            B.mtmc_set_workspace(None)
        assert bool((guard[:off] == 0x5A).all()) and bool((guard[off + need:] == 0x5A).all())
        return out, lse
    out, lse = _streamk(run)
    Xb, Wb, bf = inputs.bf16_bits(li.X), inputs.bf16_bits(li.W), inputs.f32(li.b)
    _assert_close(inputs.to_f64(out), ref.fused_linear(Xb, Wb, bf, ref.ACT_RELU), TOL["fp32"], "stream-K, caller workspace")
    _assert_close(inputs.to_f64(lse), ref.linear_lse(Xb, Wb, bf), TOL["fp32"], "stream-K lse, caller workspace")


# ------------------------------------------------------------------ skinny / split-K path
@pytest.mark.parametrize("M,N,K", [
    (16, 512, 1024), (1, 128, 64), (5, 300, 2048), (16, 136, 8192), (9, 1032, 392),   # few rows: ticketed split-K
    (16, 4096, 512), (7, 2400, 1096), (3, 9472, 72), (16, 2368, 128),                  # cluster-pair split-K
    (16, 20000, 256), (2, 9480, 64),                                                   # many rows / one k-block
    (17, 520, 392), (32, 4096, 512), (33, 2400, 1096), (64, 9472, 136), (50, 300, 2048), (64, 20000, 128),   # decode batches up to 64
])
@pytest.mark.parametrize("odt", ["fp32", "bf16"])
def test_skinny_small(M, N, K, odt):
    li, out = run_linear(M, N, K, "gelu_tanh", odt, seed=4000 + M + N)
    want = ref.fused_linear(inputs.bf16_bits(li.X), inputs.bf16_bits(li.W), inputs.f32(li.b), ref.ACT_GELU_TANH)
    _assert_close(inputs.to_f64(out), want, TOL[odt], "skinny %dx%dx%d %s" % (M, N, K, odt))


@pytest.mark.parametrize("M,N,K,split_k", [(16, 8192, 8192, 0), (1, 4096, 1024, 0), (64, 9472, 136, 0), (5, 300, 2048, 0),
                                           (16, 512, 1024, 4), (33, 2400, 1096, 0), (7, 128, 64, 0),
                                           (128, 4096, 4096, 0), (100, 8192, 4160, 0), (200, 1000, 1152, 0)])
def test_skinny_static_weights_same_bits(M, N, K, split_k):
    """With the static-weights promise the first ring of W loads goes out before the wait on the preceding kernel, in the
    weight-streaming kernel and in the cluster split-K kernel (the last three shapes and the short-band ones: 128- and
    256-column tiles, an odd walk): same bits as without it, launch after launch (each launch follows one of this
    library's own kernels)."""
    li = inputs.linear_inputs(M, N, K, seed=4100 + M + N)
    Xd, Wd, bd = li.X.cuda(), li.W.cuda(), li.b.cuda()
    B.mtmc_set_tuning(split_k=split_k)
    try:
        plain = B.mtmc_fused_linear(Xd, Wd, bd, "gelu_tanh", "fp32")
        B.mtmc_set_static_weights(True)
        outs = [B.mtmc_fused_linear(Xd, Wd, bd, "gelu_tanh", "fp32") for _ in range(12)]
        lse = B.mtmc_linear_lse(Xd, Wd, bd)                      # a merge kernel right before the next skinny launch
        after_merge = B.mtmc_fused_linear(Xd, Wd, bd, "gelu_tanh", "fp32")
        B.mtmc_check_status()
    finally:
        B.mtmc_set_static_weights(False)
        B.mtmc_set_tuning()
    for o in outs + [after_merge]:
        assert torch.equal(o, plain)
    want = ref.fused_linear(inputs.bf16_bits(li.X), inputs.bf16_bits(li.W), inputs.f32(li.b), ref.ACT_GELU_TANH)
    _assert_close(inputs.to_f64(plain), want, TOL["fp32"], "static weights %dx%dx%d" % (M, N, K))
    assert torch.isfinite(lse).all()


@pytest.mark.parametrize("M", [24, 64])
@pytest.mark.parametrize("split_k", [1, 3])
def test_skinny_decode_batch_forced_split(M, split_k):
    li = inputs.linear_inputs(M, 640, 2048, seed=46)
    want = ref.fused_linear(inputs.bf16_bits(li.X), inputs.bf16_bits(li.W), inputs.f32(li.b), ref.ACT_SILU)
    B.mtmc_set_tuning(split_k=split_k)
    try:
        Xd, Wd, bd = li.X.cuda(), li.W.cuda(), li.b.cuda()
        first = B.mtmc_fused_linear(Xd, Wd, bd, "silu", "fp32")
        again = B.mtmc_fused_linear(Xd, Wd, bd, "silu", "fp32")
        B.mtmc_check_status()
    finally:
        B.mtmc_set_tuning()
    _assert_close(inputs.to_f64(first), want, TOL["fp32"], "M %d split_k %d" % (M, split_k))
    assert torch.equal(first, again)


@pytest.mark.parametrize("split_k", [1, 2, 8, 37])
def test_skinny_result_independent_of_split(split_k):
    li = inputs.linear_inputs(16, 640, 4096, seed=44)
    want = ref.fused_linear(inputs.bf16_bits(li.X), inputs.bf16_bits(li.W), inputs.f32(li.b), ref.ACT_GELU_TANH)
    B.mtmc_set_tuning(split_k=split_k)
    try:
        Xd, Wd, bd = li.X.cuda(), li.W.cuda(), li.b.cuda()
        first = B.mtmc_fused_linear(Xd, Wd, bd, "gelu_tanh", "fp32")
        again = B.mtmc_fused_linear(Xd, Wd, bd, "gelu_tanh", "fp32")
        B.mtmc_check_status()
    finally:
        B.mtmc_set_tuning()
    _assert_close(inputs.to_f64(first), want, TOL["fp32"], "split_k %d" % split_k)
    assert torch.equal(first, again), "split-K result must be bit-stable run to run"


def test_skinny_with_caller_workspace():
    """The weight-streaming kernel's ticket plan (forced: a shape this small goes to the cluster split-K kernel by itself)
    with partials and tickets in a caller's workspace; too small a workspace is refused before anything is launched."""
    li = inputs.linear_inputs(16, 512, 2048, seed=45)
    B.mtmc_set_tuning(split_k=4)
    need = B.mtmc_workspace_bytes("fused_linear", 16, 512, 2048)
    assert need > 0
    ws = torch.full((need + 256,), 255, dtype=torch.uint8, device="cuda")   # dirty on purpose
    off = (-ws.data_ptr()) % 256
    B.mtmc_set_workspace(ws[off:off + need])
    try:
        out = B.mtmc_fused_linear(li.X.cuda(), li.W.cuda(), li.b.cuda(), "gelu_tanh", "bf16")
        assert "ticket plan" in B.mtmc_last_kernel_name()
        B.mtmc_check_status()
        with pytest.raises(B.MtmcError) as e:
            B.mtmc_set_workspace(ws[off:off + 1024])
            B.mtmc_fused_linear(li.X.cuda(), li.W.cuda(), li.b.cuda(), "gelu_tanh", "bf16")
        assert e.value.status == B.ERR_WORKSPACE
    finally:
        B.mtmc_set_workspace(None)
        B.mtmc_set_tuning()
    want = ref.fused_linear(inputs.bf16_bits(li.X), inputs.bf16_bits(li.W), inputs.f32(li.b), ref.ACT_GELU_TANH)
    _assert_close(inputs.to_f64(out), want, TOL["bf16"], "caller workspace")


# ------------------------------------------------------------------ the five benchmark configurations
def test_config_c1_full():
    c = inputs.CONFIGS["C1"]
    li, out = run_linear(c["M"], c["N"], c["K"], c["act"], c["out_dtype"], c["seed"])
    want = ref.fused_linear(inputs.bf16_bits(li.X), inputs.bf16_bits(li.W), inputs.f32(li.b), B.ACT[c["act"]])
    _assert_close(inputs.to_f64(out), want, TOL["fp32"], "C1")


def test_config_c2_full_output():
    """Every one of the 4096 x 4096 outputs of C2 against the oracle (68.7 GMAC on the host cores)."""
    c = inputs.CONFIGS["C2"]
    li, out = run_linear(c["M"], c["N"], c["K"], c["act"], c["out_dtype"], c["seed"])
    assert "gemm_big_kernel" in B.mtmc_last_kernel_name() or "gemm_pair_kernel" in B.mtmc_last_kernel_name()
    want = ref.fused_linear(inputs.bf16_bits(li.X), inputs.bf16_bits(li.W), inputs.f32(li.b), B.ACT[c["act"]])
    _assert_close(inputs.to_f64(out), want, TOL["bf16"], "C2 full output")


def test_config_c3_full_output():
    """Every one of the 8192 x 11008 outputs of C3 against the oracle, in blocks of 1024 rows (the oracle's
    fp64 result of the whole matrix would be 0.7 GB)."""
    c = inputs.CONFIGS["C3"]
    si = inputs.swiglu_inputs(c["M"], c["N"], c["K"], c["seed"])
    buf, out = _guarded((c["M"], c["N"]), torch.bfloat16)
    B.mtmc_swiglu(si.X.cuda(), si.Wg.cuda(), si.Wu.cuda(), out=out)
    B.mtmc_check_status()
    assert "gemm_pair_kernel" in B.mtmc_last_kernel_name()
    assert _canaries_intact(buf, c["M"] * c["N"])
    Wg, Wu = inputs.bf16_bits(si.Wg), inputs.bf16_bits(si.Wu)
    host = out.cpu()
    for r0 in range(0, c["M"], 1024):
        want = ref.swiglu(inputs.bf16_bits(si.X[r0:r0 + 1024].contiguous()), Wg, Wu)
        _assert_close(inputs.to_f64(host[r0:r0 + 1024]), want, TOL["bf16"], "C3 full output, rows %d.." % r0)


def test_config_c4_full_output():
    """All 4096 logsumexp values of C4 against the oracle (537 GMAC on the host cores)."""
    c = inputs.CONFIGS["C4"]
    li = inputs.linear_inputs(c["M"], c["N"], c["K"], c["seed"])
    buf, out = _guarded((c["M"],), torch.float32)
    B.mtmc_linear_lse(li.X.cuda(), li.W.cuda(), li.b.cuda(), lse_out=out)
    B.mtmc_check_status()
    assert _canaries_intact(buf, c["M"])
    want = ref.linear_lse(inputs.bf16_bits(li.X), inputs.bf16_bits(li.W), inputs.f32(li.b))
    _assert_close(inputs.to_f64(out), want, TOL["fp32"], "C4 full output")


def test_config_c5_full():
    c = inputs.CONFIGS["C5"]
    li, out = run_linear(c["M"], c["N"], c["K"], c["act"], c["out_dtype"], c["seed"])
    want = ref.fused_linear(inputs.bf16_bits(li.X), inputs.bf16_bits(li.W), inputs.f32(li.b), B.ACT[c["act"]])
    _assert_close(inputs.to_f64(out), want, TOL["bf16"], "C5")


# ------------------------------------------------------------------ determinism, errors
def test_bit_reproducible():
    li = inputs.linear_inputs(300, 520, 448, seed=9)
    Xd, Wd, bd = li.X.cuda(), li.W.cuda(), li.b.cuda()
    first = B.mtmc_fused_linear(Xd, Wd, bd, "gelu_tanh", "bf16")
    l0 = B.mtmc_linear_lse(Xd, Wd, bd)
    for _ in range(10):
        assert torch.equal(first, B.mtmc_fused_linear(Xd, Wd, bd, "gelu_tanh", "bf16"))
        assert torch.equal(l0, B.mtmc_linear_lse(Xd, Wd, bd))
    B.mtmc_check_status()


def test_argument_errors_enqueue_nothing():
    L = B.load()
    x = torch.zeros(64, 64, dtype=torch.bfloat16, device="cuda")
    o = torch.zeros(64, 64, dtype=torch.float32, device="cuda")
    before = B.mtmc_launch_count()
    assert L.mtmc_fused_linear(None, x.data_ptr(), None, 64, 64, 64, 0, 0, o.data_ptr()) == B.ERR_INVALID_ARG
    assert L.mtmc_fused_linear(x.data_ptr(), x.data_ptr(), None, 64, 64, 0, 0, 0, o.data_ptr()) == B.ERR_INVALID_ARG
    assert L.mtmc_fused_linear(x.data_ptr(), x.data_ptr(), None, 64, 64, 64, 9, 0, o.data_ptr()) == B.ERR_INVALID_ARG
    assert L.mtmc_fused_linear(x.data_ptr(), x.data_ptr(), None, 64, 64, 64, 0, 5, o.data_ptr()) == B.ERR_INVALID_ARG
    assert L.mtmc_fused_linear(x.data_ptr(), x.data_ptr(), None, 64, 64, 60, 0, 0, o.data_ptr()) == B.ERR_UNSUPPORTED_SHAPE
    assert L.mtmc_fused_linear(x.data_ptr() + 2, x.data_ptr(), None, 32, 64, 64, 0, 0, o.data_ptr()) == B.ERR_INVALID_ARG
    assert L.mtmc_swiglu(x.data_ptr(), x.data_ptr(), None, 64, 64, 64, o.data_ptr()) == B.ERR_INVALID_ARG
    assert L.mtmc_linear_lse(x.data_ptr(), x.data_ptr(), None, 64, 64, 64, None) == B.ERR_INVALID_ARG
    assert B.mtmc_launch_count() == before
    assert len(L.mtmc_last_error()) > 0
    B.mtmc_check_status()


def test_bounded_wait_reports_a_timeout_and_the_context_stays_usable():
    """Failure detection without a fault: a wait that nothing will satisfy gives up after its limit,
    the kernel returns, the status surfaces once on the host, and the library keeps working."""
    B.mtmc_check_status()
    B.mtmc_selftest_timeout()
    with pytest.raises(B.MtmcError) as e:
        B.mtmc_check_status()
    assert e.value.status == B.ERR_DEVICE_TIMEOUT
    B.mtmc_check_status()                                   # sticky status was cleared by the report
    li, out = run_linear(140, 264, 192, "relu", "fp32", seed=91)
    want = ref.fused_linear(inputs.bf16_bits(li.X), inputs.bf16_bits(li.W), inputs.f32(li.b), ref.ACT_RELU)
    _assert_close(inputs.to_f64(out), want, TOL["fp32"], "after the self-test")
    sk, so = run_linear(16, 640, 1024, "gelu_tanh", "bf16", seed=92)     # ticket path after tickets were marked dirty
    _assert_close(inputs.to_f64(so), ref.fused_linear(inputs.bf16_bits(sk.X), inputs.bf16_bits(sk.W), inputs.f32(sk.b),
                                                     ref.ACT_GELU_TANH), TOL["bf16"], "skinny after the self-test")


def test_host_pointer_entry_points():
    li = inputs.linear_inputs(150, 264, 128, seed=61)
    out = B.mtmc_fused_linear_host(li.X, li.W, li.b, "relu", "fp32")
    want = ref.fused_linear(inputs.bf16_bits(li.X), inputs.bf16_bits(li.W), inputs.f32(li.b), ref.ACT_RELU)
    _assert_close(inputs.to_f64(out), want, TOL["fp32"], "fused_linear_host")
    lse = B.mtmc_linear_lse_host(li.X, li.W, li.b)
    _assert_close(inputs.to_f64(lse), ref.linear_lse(inputs.bf16_bits(li.X), inputs.bf16_bits(li.W), inputs.f32(li.b)),
                  TOL["fp32"], "linear_lse_host")
    si = inputs.swiglu_inputs(150, 264, 128, seed=62)
    sw = B.mtmc_swiglu_host(si.X, si.Wg, si.Wu)
    _assert_close(inputs.to_f64(sw), ref.swiglu(inputs.bf16_bits(si.X), inputs.bf16_bits(si.Wg), inputs.bf16_bits(si.Wu)),
                  TOL["bf16"], "swiglu_host")


def test_host_pointer_calls_without_waiting():
    """Ten calls of mixed shapes through the host-pointer pipeline without waiting in between (more than its six slots,
    so slots are reused while earlier calls are in flight), one wait at the end; every result against the oracle."""
    shapes = [(150, 264, 128), (64, 1024, 512), (300, 520, 200), (16, 512, 1024), (129, 257, 72)]
    jobs = []
    for rep in range(2):
        for i, (M, N, K) in enumerate(shapes):
            li = inputs.linear_inputs(M, N, K, seed=9100 + 10 * rep + i)
            X, W, b = li.X.pin_memory(), li.W.pin_memory(), li.b.pin_memory()
            if i % 3 == 2:
                out = torch.full((M,), float("nan")).pin_memory()
                B.mtmc_linear_lse_host(X, W, b, lse_out=out, blocking=False)
                want, tol = ref.linear_lse(inputs.bf16_bits(li.X), inputs.bf16_bits(li.W), inputs.f32(li.b)), TOL["fp32"]
            else:
                out = torch.full((M, N), float("nan")).pin_memory()
                B.mtmc_fused_linear_host(X, W, b, "silu", "fp32", out=out, blocking=False)
                want, tol = ref.fused_linear(inputs.bf16_bits(li.X), inputs.bf16_bits(li.W), inputs.f32(li.b), ref.ACT_SILU), TOL["fp32"]
            jobs.append((out, want, tol, (X, W, b)))
    si = inputs.swiglu_inputs(200, 392, 256, seed=9190)
    sX, sG, sU = si.X.pin_memory(), si.Wg.pin_memory(), si.Wu.pin_memory()
    sw = torch.zeros((200, 392), dtype=torch.bfloat16).pin_memory()
    B.mtmc_swiglu_host(sX, sG, sU, out=sw, blocking=False)
    B.mtmc_host_sync()
    B.mtmc_check_status()
    for n, (out, want, tol, _) in enumerate(jobs):
        _assert_close(inputs.to_f64(out), want, tol, "pipelined host call %d" % n)
    _assert_close(inputs.to_f64(sw), ref.swiglu(inputs.bf16_bits(si.X), inputs.bf16_bits(si.Wg), inputs.bf16_bits(si.Wu)),
                  TOL["bf16"], "pipelined swiglu_host")


def test_random_shapes_long_k_schedules_and_switches():
    """Seeded sweep of 160 shapes with K up to 4480 (the cluster split-K kernels on 256- and 128-column tiles, odd and
    even k-walks on the pair kernels' two-k-block ring), row counts on both sides of every kernel boundary, the
    stream-K schedule and the static-weights switch on and off, bf16 and E4M3 operands, against the oracle."""
    rng = np.random.default_rng(20251126)
    tunings = [dict(), dict(), dict(cta_pair=1), dict(cta_pair=2), dict(cta_pair=-1), dict(split_k=1), dict(tile_n=128)]
    seen = set()
    for case in range(160):
        M = int([rng.integers(1, 65), rng.integers(65, 300), rng.integers(257, 700), 128, 256, 512][case % 6])
        N = 8 * int(rng.integers(1, 150))
        K = 8 * int([rng.integers(1, 40), rng.integers(40, 560), 64, 128, 256, 264][int(rng.integers(0, 6))])
        op = ["linear", "swiglu", "lse", "fp8", "linear", "residual", "rowmax"][int(rng.integers(0, 7))]
        tune = tunings[int(rng.integers(0, len(tunings)))]
        sk = int(rng.integers(0, 4) == 0)
        static = bool(rng.integers(0, 2))
        act = ["none", "relu", "gelu_tanh", "silu"][int(rng.integers(0, 4))]
        odt = "bf16" if rng.integers(0, 2) else "fp32"
        what = "case %d: %s %dx%dx%d %s %s %r stream-K %d static %d" % (case, op, M, N, K, act, odt, tune, sk, static)
        B.mtmc_set_tuning(**tune)
        B.mtmc_set_schedule(sk)
        B.mtmc_set_static_weights(static)
        try:
            if op == "swiglu":
                si = inputs.swiglu_inputs(M, N, K, seed=9800 + case)
                got = B.mtmc_swiglu(si.X.cuda(), si.Wg.cuda(), si.Wu.cuda())
                _assert_close(inputs.to_f64(got), ref.swiglu(inputs.bf16_bits(si.X), inputs.bf16_bits(si.Wg), inputs.bf16_bits(si.Wu)),
                              TOL["bf16"], what)
            elif op == "fp8":
                K8 = (K + 15) // 16 * 16
                fi = inputs.fp8_linear_inputs(M, N, K8, seed=9800 + case)
                got = B.mtmc_fused_linear_fp8(fi.X.cuda(), fi.W.cuda(), fi.b.cuda(), fi.scale_x, fi.scale_w, act, odt)
                want = ref.fused_linear_fp8(inputs.fp8_bits(fi.X), inputs.fp8_bits(fi.W), inputs.f32(fi.b), fi.scale_x, fi.scale_w, B.ACT[act])
                _assert_close(inputs.to_f64(got), want, TOL[odt], what)
            else:
                li = inputs.linear_inputs(M, N, K, seed=9800 + case)
                Xb, Wb, bf = inputs.bf16_bits(li.X), inputs.bf16_bits(li.W), inputs.f32(li.b)
                Xd, Wd, bd = li.X.cuda(), li.W.cuda(), li.b.cuda()
                if op == "linear":
                    buf, out = _guarded((M, N), torch.bfloat16 if odt == "bf16" else torch.float32)
                    B.mtmc_fused_linear(Xd, Wd, bd, act, odt, out=out)
                    B.mtmc_check_status()
                    assert _canaries_intact(buf, M * N), what
                    _assert_close(inputs.to_f64(out), ref.fused_linear(Xb, Wb, bf, B.ACT[act]), TOL[odt], what)
                elif op == "residual":
                    R = torch.randn(M, N, generator=torch.Generator().manual_seed(case)).bfloat16()
                    got = B.mtmc_fused_linear_residual(Xd, Wd, bd, R.cuda(), act, "bf16")
                    _assert_close(inputs.to_f64(got), ref.fused_linear_residual(Xb, Wb, bf, inputs.bf16_bits(R), B.ACT[act]), TOL["bf16"], what)
                elif op == "lse":
                    _assert_close(inputs.to_f64(B.mtmc_linear_lse(Xd, Wd, bd)), ref.linear_lse(Xb, Wb, bf), TOL["fp32"], what)
                else:
                    mx, arg = B.mtmc_linear_rowmax(Xd, Wd, bd)
                    _check_rowmax(li, mx, arg, what)
            B.mtmc_check_status()
            seen.add(B.mtmc_last_kernel_name().split("<")[0])
        finally:
            B.mtmc_set_tuning()
            B.mtmc_set_schedule(0)
            B.mtmc_set_static_weights(False)
    for family in ("gemm_tiled_kernel", "gemm_pair_kernel", "gemm_big_kernel", "gemm_ksplit_kernel", "gemm_ksplit_kernel (128-column tiles)"):
        assert family in seen, "the sweep never reached %s (ran %r)" % (family, sorted(seen))


def test_random_shapes_all_operators_and_kernels():
    """Seeded sweep: 60 random shapes (ragged M, N, K; K a multiple of 8), each through a randomly chosen operator and
    kernel choice (automatic, 256 x 256 pairs, 512 x 256 pairs, single-CTA tiles of either width), against the oracle."""
    rng = np.random.default_rng(20251125)
    tunings = [dict(), dict(cta_pair=1), dict(cta_pair=2), dict(cta_pair=-1), dict(tile_n=128), dict(split_k=2)]
    for case in range(60):
        M = int(rng.integers(1, 700))
        N = int(rng.integers(1, 900))
        K = 8 * int(rng.integers(1, 260))
        while M * N * K > 4e8:
            K = max(8, K // 2 // 8 * 8)
        op = ["linear", "lse", "swiglu", "rowmax", "xent", "residual"][case % 6]
        tune = tunings[int(rng.integers(0, len(tunings)))]
        what = "case %d: %s %dx%dx%d %r" % (case, op, M, N, K, tune)
        li = inputs.linear_inputs(M, N, K, seed=9300 + case)
        Xb, Wb, bf = inputs.bf16_bits(li.X), inputs.bf16_bits(li.W), inputs.f32(li.b)
        Xd, Wd, bd = li.X.cuda(), li.W.cuda(), li.b.cuda()
        B.mtmc_set_tuning(**tune)
        try:
            if op == "linear":
                act = ["none", "relu", "gelu_tanh", "silu"][case // 6 % 4]
                odt = "bf16" if case % 2 else "fp32"
                buf, out = _guarded((M, N), torch.bfloat16 if odt == "bf16" else torch.float32)
                B.mtmc_fused_linear(Xd, Wd, bd, act, odt, out=out)
                B.mtmc_check_status()
                assert _canaries_intact(buf, M * N), what
                _assert_close(inputs.to_f64(out), ref.fused_linear(Xb, Wb, bf, B.ACT[act]), TOL[odt], what)
            elif op == "lse":
                _assert_close(inputs.to_f64(B.mtmc_linear_lse(Xd, Wd, bd)), ref.linear_lse(Xb, Wb, bf), TOL["fp32"], what)
            elif op == "swiglu":
                si = inputs.swiglu_inputs(M, N, K, seed=9400 + case)
                got = B.mtmc_swiglu(si.X.cuda(), si.Wg.cuda(), si.Wu.cuda())
                _assert_close(inputs.to_f64(got), ref.swiglu(inputs.bf16_bits(si.X), inputs.bf16_bits(si.Wg), inputs.bf16_bits(si.Wu)),
                              TOL["bf16"], what)
            elif op == "rowmax":
                mx, arg = B.mtmc_linear_rowmax(Xd, Wd, bd)
                _check_rowmax(li, mx, arg, what)
            elif op == "xent":
                tgt = torch.from_numpy(rng.integers(0, N, size=M))
                loss = B.mtmc_linear_cross_entropy(Xd, Wd, bd, tgt.cuda())
                want, _ = ref.linear_cross_entropy(Xb, Wb, bf, tgt.numpy())
                _assert_close(inputs.to_f64(loss), want, TOL["fp32"], what)
            else:
                R = torch.randn(M, N, generator=torch.Generator().manual_seed(case)).bfloat16()
                got = B.mtmc_fused_linear_residual(Xd, Wd, bd, R.cuda(), "silu", "bf16")
                _assert_close(inputs.to_f64(got), ref.fused_linear_residual(Xb, Wb, bf, inputs.bf16_bits(R), ref.ACT_SILU),
                              TOL["bf16"], what)
            B.mtmc_check_status()
        finally:
            B.mtmc_set_tuning()

