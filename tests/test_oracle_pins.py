"""Pins for the fp64 CPU oracle: every check here is against something OTHER than the
oracle itself -- exact rational brute force, hand-worked values, 40-digit closed
forms, algebraic laws of the operators, and torch's fp64 library routines.  A
dropped term, a wrong sign or index, or a transposed operand fails at least one.
CPU only."""
import math
import os
from fractions import Fraction

import numpy as np
import pytest
import torch

from oracle import ref
from paper_2511_20100_b200 import inputs

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")
ACTS = [ref.ACT_NONE, ref.ACT_RELU, ref.ACT_GELU_TANH, ref.ACT_SILU]


def bits(a) -> np.ndarray:
    """float array (values exactly representable in bf16, or to be RNE-rounded) -> uint16 bit patterns."""
    return inputs.bf16_bits(torch.as_tensor(np.asarray(a, dtype=np.float32)).to(torch.bfloat16))


def widen(b16: np.ndarray) -> np.ndarray:
    return inputs.bits_to_bf16(b16).to(torch.float64).numpy()


def py_act(kind, z):
    """Independent scalar restatement used only where the GEMM part is under test."""
    if kind == ref.ACT_NONE:
        return z
    if kind == ref.ACT_RELU:
        return max(z, 0.0)
    if kind == ref.ACT_GELU_TANH:
        return float(torch.nn.functional.gelu(torch.tensor(z, dtype=torch.float64), approximate="tanh"))
    return float(torch.nn.functional.silu(torch.tensor(z, dtype=torch.float64)))


# ---------------------------------------------------------------- bf16 decode
def test_bf16_decode_known_patterns():
    # 0x3F80 = 1, 0xC000 = -2, 0x3FC0 = 1.5, 0x0001 = 2^-133 (denormal), 0x8000 = -0
    pats = np.array([[0x3F80, 0xC000, 0x3FC0, 0x0001, 0x8000]], dtype=np.uint16).T.copy()  # X [5,1]
    one = np.array([[0x3F80]], dtype=np.uint16)                                                # W [1,1] = 1
    z = ref.fused_linear(pats, one, None, ref.ACT_NONE)[:, 0]
    assert z.tolist() == [1.0, -2.0, 1.5, 2.0 ** -133, 0.0]


# ---------------------------------------------------------------- GEMM core
def test_hand_worked_example():
    blocks, cur = {}, None
    for line in open(os.path.join(GOLDEN, "gemm_2x3x4.txt")):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        tok = line.split()
        if tok[0] in ("X", "W", "b", "Z"):
            cur = tok[0]
            blocks[cur] = []
        else:
            blocks[cur].append([float(t) for t in tok])
    X, W, b, Z = (np.array(blocks[k]) for k in ("X", "W", "b", "Z"))
    got = ref.fused_linear(bits(X), bits(W), b[0].astype(np.float32), ref.ACT_NONE)
    assert got.shape == (2, 3)
    assert np.array_equal(got, Z)
    # and through the sampled entry point
    rows, cols = np.array([0, 1, 1]), np.array([2, 0, 2])
    pts = ref.fused_linear_points(bits(X), bits(W), b[0].astype(np.float32), ref.ACT_NONE, rows, cols)
    assert pts.tolist() == [Z[0, 2], Z[1, 0], Z[1, 2]]


@pytest.mark.parametrize("M,N,K", [(4, 4, 4), (3, 5, 7), (1, 1, 1), (2, 6, 3)])
def test_exact_rational_brute_force(M, N, K):
    vals = [0.0, 0.5, -0.5, 1.0, -1.0, 1.5, -1.5, 2.0, -2.0, 3.0, -3.0]
    rng = np.random.default_rng(100 + M * 49 + N * 7 + K)
    X = rng.choice(vals, size=(M, K))
    W = rng.choice(vals, size=(N, K))
    b = rng.choice([0.0, 0.25, -0.75, 1.0], size=N).astype(np.float32)
    got = ref.fused_linear(bits(X), bits(W), b, ref.ACT_NONE)
    for m in range(M):
        for n in range(N):
            exact = sum((Fraction(X[m, k]) * Fraction(W[n, k]) for k in range(K)), Fraction(float(b[n])))
            assert Fraction(got[m, n]) == exact, (m, n)


def test_identity_weight_gives_act_of_x_plus_b():
    li = inputs.linear_inputs(9, 16, 16, seed=11)
    eye = bits(np.eye(16))
    Xd, b = widen(inputs.bf16_bits(li.X)), inputs.f32(li.b)
    for kind in ACTS:
        got = ref.fused_linear(inputs.bf16_bits(li.X), eye, b, kind)
        want = np.array([[py_act(kind, Xd[m, n] + float(b[n])) for n in range(16)] for m in range(9)])
        np.testing.assert_allclose(got, want, rtol=1e-14, atol=1e-15)


def test_zero_input_gives_act_of_bias():
    li = inputs.linear_inputs(5, 12, 24, seed=12)
    X0 = np.zeros((5, 24), dtype=np.uint16)
    b = inputs.f32(li.b)
    for kind in ACTS:
        got = ref.fused_linear(X0, inputs.bf16_bits(li.W), b, kind)
        want = np.array([py_act(kind, float(v)) for v in b])
        for m in range(5):
            np.testing.assert_allclose(got[m], want, rtol=1e-14, atol=1e-16)


def test_k_split_additivity_permutation_and_scaling():
    li = inputs.linear_inputs(6, 10, 40, seed=13)
    X, W, b = inputs.bf16_bits(li.X), inputs.bf16_bits(li.W), inputs.f32(li.b)
    z = ref.fused_linear(X, W, None, ref.ACT_NONE)
    z1 = ref.fused_linear(X[:, :24].copy(), W[:, :24].copy(), None, ref.ACT_NONE)
    z2 = ref.fused_linear(X[:, 24:].copy(), W[:, 24:].copy(), None, ref.ACT_NONE)
    np.testing.assert_allclose(z, z1 + z2, rtol=0, atol=1e-13)
    perm = np.random.default_rng(5).permutation(40)
    zp = ref.fused_linear(X[:, perm].copy(), W[:, perm].copy(), None, ref.ACT_NONE)
    np.testing.assert_allclose(z, zp, rtol=0, atol=1e-13)
    nperm = np.random.default_rng(6).permutation(10)
    zb = ref.fused_linear(X, W, b, ref.ACT_NONE)
    zn = ref.fused_linear(X, W[nperm].copy(), b[nperm].copy(), ref.ACT_NONE)
    assert np.array_equal(zn, zb[:, nperm])
    W2 = bits(2.0 * widen(W))                      # doubling is exact in bf16
    assert np.array_equal(ref.fused_linear(X, W2, None, ref.ACT_NONE), 2.0 * z)
    # bias enters once, after the sum
    np.testing.assert_allclose(zb - z, np.broadcast_to(b.astype(np.float64), z.shape), rtol=0, atol=1e-14)


@pytest.mark.parametrize("M,N,K,seed", [(7, 13, 64, 21), (33, 5, 129, 22)])
def test_against_torch_fp64_matmul(M, N, K, seed):
    li = inputs.linear_inputs(M, N, K, seed=seed)
    want = li.X.double() @ li.W.double().T + li.b.double()
    got = ref.fused_linear(inputs.bf16_bits(li.X), inputs.bf16_bits(li.W), inputs.f32(li.b), ref.ACT_NONE)
    np.testing.assert_allclose(got, want.numpy(), rtol=0, atol=1e-12)
    for kind, fn in [(ref.ACT_RELU, torch.relu),
                     (ref.ACT_GELU_TANH, lambda t: torch.nn.functional.gelu(t, approximate="tanh")),
                     (ref.ACT_SILU, torch.nn.functional.silu)]:
        got = ref.fused_linear(inputs.bf16_bits(li.X), inputs.bf16_bits(li.W), inputs.f32(li.b), kind)
        np.testing.assert_allclose(got, fn(want).numpy(), rtol=1e-12, atol=1e-13)


def test_residual_is_added_after_the_activation():
    li = inputs.linear_inputs(6, 11, 40, seed=14)
    X, W, b = inputs.bf16_bits(li.X), inputs.bf16_bits(li.W), inputs.f32(li.b)
    rng = np.random.default_rng(8)
    R32 = rng.normal(size=(6, 11)).astype(np.float32)
    Rb = bits(R32)
    for kind in ACTS:
        base = ref.fused_linear(X, W, b, kind)
        assert np.array_equal(ref.fused_linear_residual(X, W, b, R32, kind), base + R32.astype(np.float64))
        assert np.array_equal(ref.fused_linear_residual(X, W, b, Rb, kind), base + widen(Rb))
        assert np.array_equal(ref.fused_linear_residual(X, W, b, np.zeros_like(R32), kind), base)
    # torch: relu(z) + r, not relu(z + r)
    z = li.X.double() @ li.W.double().T + li.b.double()
    want = torch.relu(z) + torch.from_numpy(R32).double()
    np.testing.assert_allclose(ref.fused_linear_residual(X, W, b, R32, ref.ACT_RELU), want.numpy(), rtol=0, atol=1e-12)


# ---------------------------------------------------------------- FP8 (E4M3) operands
def test_e4m3_decode_every_pattern():
    # known values of the format: 0x38 = 1, 0x7E = 448 (largest), 0x01 = 2^-9 (smallest subnormal), 0x08 = 2^-6
    assert ref.e4m3(0x38) == 1.0 and ref.e4m3(0x7E) == 448.0 and ref.e4m3(0x01) == 2.0 ** -9 and ref.e4m3(0x08) == 2.0 ** -6
    assert ref.e4m3(0xB8) == -1.0 and ref.e4m3(0x00) == 0.0 and math.isnan(ref.e4m3(0x7F)) and math.isnan(ref.e4m3(0xFF))
    # and all 256 against torch's float8_e4m3fn conversion
    pats = torch.arange(256, dtype=torch.int32).to(torch.uint8)
    want = pats.view(torch.float8_e4m3fn).to(torch.float64).numpy()
    for i in range(256):
        got = ref.e4m3(i)
        assert (math.isnan(got) and math.isnan(want[i])) or got == want[i], i
    # monotone in the positive half
    vals = [ref.e4m3(i) for i in range(0x7F)]
    assert all(a < b for a, b in zip(vals, vals[1:]))


def test_fp8_linear_pins():
    fi = inputs.fp8_linear_inputs(7, 13, 96, seed=71)
    X8, W8, b = inputs.fp8_bits(fi.X), inputs.fp8_bits(fi.W), inputs.f32(fi.b)
    got = ref.fused_linear_fp8(X8, W8, b, fi.scale_x, fi.scale_w, ref.ACT_NONE)
    scale = float(np.float32(fi.scale_x)) * float(np.float32(fi.scale_w))
    want = scale * (fi.X.to(torch.float64) @ fi.W.to(torch.float64).T) + fi.b.double()
    np.testing.assert_allclose(got, want.numpy(), rtol=1e-13, atol=1e-13)
    # exact brute force: every E4M3 value is a multiple of 2^-9, so products are multiples of 2^-18
    xi = (fi.X.to(torch.float64) * 512).numpy().astype(np.int64)
    wi = (fi.W.to(torch.float64) * 512).numpy().astype(np.int64)
    raw = ref.fused_linear_fp8(X8, W8, None, 1.0, 1.0, ref.ACT_NONE)
    for m in range(7):
        for n in range(13):
            assert Fraction(raw[m, n]) == Fraction(int((xi[m] * wi[n]).sum()), 512 * 512)
    # scales multiply the sum, not the bias; activation applied last
    twice = ref.fused_linear_fp8(X8, W8, b, 2.0 * fi.scale_x, fi.scale_w, ref.ACT_NONE)
    np.testing.assert_allclose(twice - b.astype(np.float64), 2.0 * (got - b.astype(np.float64)), rtol=1e-13, atol=1e-13)
    g = ref.fused_linear_fp8(X8, W8, b, fi.scale_x, fi.scale_w, ref.ACT_GELU_TANH)
    np.testing.assert_allclose(g, torch.nn.functional.gelu(want, approximate="tanh").numpy(), rtol=1e-12, atol=1e-13)
    rows, cols = np.array([0, 6, 3]), np.array([12, 0, 5])
    assert np.array_equal(ref.fused_linear_fp8_points(X8, W8, b, fi.scale_x, fi.scale_w, ref.ACT_GELU_TANH, rows, cols), g[rows, cols])
    # quantisation recipe: the largest magnitude lands on the format's maximum
    assert float(fi.X.to(torch.float32).abs().max()) == 448.0 and float(fi.W.to(torch.float32).abs().max()) == 448.0


def _as_bf16_bits(t8, factor):
    """E4M3 tensor times a power of two, as bf16 bit patterns: exact, every E4M3 value has 4 significant bits."""
    v = t8.to(torch.float32) * factor
    b = v.to(torch.bfloat16)
    assert torch.equal(b.to(torch.float32), v)
    return inputs.bf16_bits(b)


def test_fp8_swiglu_pins():
    X8, Wg8, Wu8, sx, sg, su = inputs.fp8_swiglu_inputs(6, 11, 80, seed=72)
    xb, gb, ub = inputs.fp8_bits(X8), inputs.fp8_bits(Wg8), inputs.fp8_bits(Wu8)
    got = ref.swiglu_fp8(xb, gb, ub, sx, sg, su)
    f = lambda v: float(np.float32(v))
    g = f(sx) * f(sg) * (X8.to(torch.float64) @ Wg8.to(torch.float64).T)
    u = f(sx) * f(su) * (X8.to(torch.float64) @ Wu8.to(torch.float64).T)
    np.testing.assert_allclose(got, (torch.nn.functional.silu(g) * u).numpy(), rtol=1e-12, atol=1e-13)
    # gate and up carry their own scales: the product of the two linear layers, each pinned on its own
    prod = ref.fused_linear_fp8(xb, gb, None, sx, sg, ref.ACT_SILU) * ref.fused_linear_fp8(xb, ub, None, sx, su, ref.ACT_NONE)
    np.testing.assert_allclose(got, prod, rtol=1e-14, atol=0)
    # with power-of-two scales folded into bf16 copies of the operands it is the bf16 function, bit for bit
    folded = ref.swiglu(_as_bf16_bits(X8, 2.0 ** -3), _as_bf16_bits(Wg8, 2.0 ** -7), _as_bf16_bits(Wu8, 2.0 ** -5))
    assert np.array_equal(ref.swiglu_fp8(xb, gb, ub, 2.0 ** -3, 2.0 ** -7, 2.0 ** -5), folded)
    # linear in the up scale, zero for a zero up projection, and the gate scale is inside the silu
    np.testing.assert_allclose(ref.swiglu_fp8(xb, gb, ub, sx, sg, 2.0 * su), 2.0 * got, rtol=1e-14, atol=0)
    assert not np.any(ref.swiglu_fp8(xb, gb, np.zeros_like(ub), sx, sg, su))
    assert not np.allclose(ref.swiglu_fp8(xb, gb, ub, sx, 2.0 * sg, su), 2.0 * got)


def test_fp8_linear_lse_pins():
    fi = inputs.fp8_linear_inputs(5, 37, 64, seed=73)
    X8, W8, b = inputs.fp8_bits(fi.X), inputs.fp8_bits(fi.W), inputs.f32(fi.b)
    lse, logits = ref.linear_lse_fp8(X8, W8, b, fi.scale_x, fi.scale_w, want_logits=True)
    scale = float(np.float32(fi.scale_x)) * float(np.float32(fi.scale_w))
    z = scale * (fi.X.to(torch.float64) @ fi.W.to(torch.float64).T) + fi.b.double()
    np.testing.assert_allclose(logits, z.numpy(), rtol=1e-13, atol=1e-13)
    np.testing.assert_allclose(lse, torch.logsumexp(z, dim=-1).numpy(), rtol=1e-13, atol=0)
    # the logits are those of the pinned FP8 linear layer, and the row reduction is the pinned one
    assert np.array_equal(logits, ref.fused_linear_fp8(X8, W8, b, fi.scale_x, fi.scale_w, ref.ACT_NONE))
    assert np.array_equal(lse, np.array([ref.lse_vector(row) for row in logits]))
    # shift law through the bias, and the bf16 function on operands with the power-of-two scales folded in
    np.testing.assert_allclose(ref.linear_lse_fp8(X8, W8, b + np.float32(0.5), fi.scale_x, fi.scale_w), lse + 0.5, rtol=0, atol=2e-7)   # b + 0.5 rounds in fp32
    folded = ref.linear_lse(_as_bf16_bits(fi.X, 2.0 ** -4), _as_bf16_bits(fi.W, 2.0 ** -8), b)
    assert np.array_equal(ref.linear_lse_fp8(X8, W8, b, 2.0 ** -4, 2.0 ** -8), folded)


def test_fp8_rowmax_and_cross_entropy_pins():
    fi = inputs.fp8_linear_inputs(6, 41, 48, seed=74)
    X8, W8, b = inputs.fp8_bits(fi.X), inputs.fp8_bits(fi.W), inputs.f32(fi.b)
    z = ref.fused_linear_fp8(X8, W8, b, fi.scale_x, fi.scale_w, ref.ACT_NONE)          # the pinned FP8 logits
    mx, arg = ref.linear_rowmax_fp8(X8, W8, b, fi.scale_x, fi.scale_w)
    assert np.array_equal(mx, z.max(axis=1)) and np.array_equal(arg, z.argmax(axis=1))
    tv, ti = torch.from_numpy(z).max(dim=1)
    assert np.array_equal(mx, tv.numpy()) and np.array_equal(arg, ti.numpy())
    # ties go to the lowest column: duplicate the winning weight row (and its bias) further right
    W2, b2 = W8.copy(), b.copy()
    for m in range(1):
        src, dst = int(arg[0]), 40 if arg[0] != 40 else 39
        W2[dst], b2[dst] = W2[src], b2[src]
    mx2, arg2 = ref.linear_rowmax_fp8(X8, W2, b2, fi.scale_x, fi.scale_w)
    assert mx2[0] == mx[0] and arg2[0] == min(int(arg[0]), dst)
    tgt = np.array([0, 40, 7, 7, 13, 22])
    loss, lse = ref.linear_cross_entropy_fp8(X8, W8, b, fi.scale_x, fi.scale_w, tgt)
    assert np.array_equal(lse, ref.linear_lse_fp8(X8, W8, b, fi.scale_x, fi.scale_w))
    assert np.array_equal(loss, lse - z[np.arange(6), tgt])
    want = torch.nn.functional.cross_entropy(torch.from_numpy(z), torch.from_numpy(tgt), reduction="none")
    np.testing.assert_allclose(loss, want.numpy(), rtol=1e-12, atol=1e-12)
    # with power-of-two scales folded into bf16 copies of the operands: the bf16 functions, bit for bit
    fmx, farg = ref.linear_rowmax(_as_bf16_bits(fi.X, 2.0 ** -4), _as_bf16_bits(fi.W, 2.0 ** -8), b)
    gmx, garg = ref.linear_rowmax_fp8(X8, W8, b, 2.0 ** -4, 2.0 ** -8)
    assert np.array_equal(fmx, gmx) and np.array_equal(farg, garg)
    floss, _ = ref.linear_cross_entropy(_as_bf16_bits(fi.X, 2.0 ** -4), _as_bf16_bits(fi.W, 2.0 ** -8), b, tgt)
    gloss, _ = ref.linear_cross_entropy_fp8(X8, W8, b, 2.0 ** -4, 2.0 ** -8, tgt)
    assert np.array_equal(floss, gloss)


def test_fp8_softmax_pins():
    fi = inputs.fp8_linear_inputs(6, 41, 48, seed=75)
    X8, W8, b = inputs.fp8_bits(fi.X), inputs.fp8_bits(fi.W), inputs.f32(fi.b)
    P = ref.linear_softmax_fp8(X8, W8, b, fi.scale_x, fi.scale_w)
    z = ref.fused_linear_fp8(X8, W8, b, fi.scale_x, fi.scale_w, ref.ACT_NONE)          # the pinned FP8 logits
    np.testing.assert_allclose(P, torch.softmax(torch.from_numpy(z), dim=-1).numpy(), rtol=1e-13, atol=0)
    assert np.array_equal(P, np.stack([ref.softmax_vector(row) for row in z]))         # the pinned row routine on them
    lse = ref.linear_lse_fp8(X8, W8, b, fi.scale_x, fi.scale_w)
    np.testing.assert_allclose(P, np.exp(z - lse[:, None]), rtol=1e-12)
    np.testing.assert_allclose(P.sum(axis=1), np.ones(6), rtol=0, atol=1e-13)
    # doubling one scale and halving the other changes nothing; doubling one doubles the logits' spread
    assert np.array_equal(ref.linear_softmax_fp8(X8, W8, b, 2.0 * fi.scale_x, 0.5 * fi.scale_w), P)
    P2 = ref.linear_softmax_fp8(X8, W8, None, 2.0 * fi.scale_x, fi.scale_w)
    z0 = ref.fused_linear_fp8(X8, W8, None, fi.scale_x, fi.scale_w, ref.ACT_NONE)
    np.testing.assert_allclose(P2, torch.softmax(torch.from_numpy(2.0 * z0), dim=-1).numpy(), rtol=1e-12)
    # with power-of-two scales folded into bf16 copies of the operands: the bf16 function, bit for bit
    folded = ref.linear_softmax(_as_bf16_bits(fi.X, 2.0 ** -4), _as_bf16_bits(fi.W, 2.0 ** -8), b)
    assert np.array_equal(ref.linear_softmax_fp8(X8, W8, b, 2.0 ** -4, 2.0 ** -8), folded)


# ---------------------------------------------------------------- activations
def _closed_forms():
    rows = []
    for line in open(os.path.join(GOLDEN, "closed_forms.txt")):
        if line.startswith("#") or not line.strip():
            continue
        kind, arg, val = line.split()
        rows.append((kind, arg, float(val)))
    return rows


def test_e8m0_decode_every_code():
    # the scale byte is a biased exponent: 127 = 1, 0 = 2^-127, 254 = 2^127, 255 = NaN
    assert ref.e8m0(127) == 1.0 and ref.e8m0(128) == 2.0 and ref.e8m0(126) == 0.5
    assert ref.e8m0(0) == 2.0 ** -127 and ref.e8m0(254) == 2.0 ** 127 and math.isnan(ref.e8m0(255))
    for e in range(255):
        assert ref.e8m0(e) == math.ldexp(1.0, e - 127), e
        if e:
            assert ref.e8m0(e) == 2.0 * ref.e8m0(e - 1)


def _mx_dequant(X8, SX):
    """fp64 torch tensor of the block-scaled values (every element times its block's power of two)."""
    scale = torch.exp2(SX.to(torch.float64) - 127.0).repeat_interleave(32, dim=1)
    return X8.to(torch.float64) * scale


def test_mxfp8_linear_pins():
    mi = inputs.mx_linear_inputs(6, 11, 128, seed=81, spread=5)          # neighbouring blocks with very different scales
    X8, W8, b = inputs.fp8_bits(mi.X), inputs.fp8_bits(mi.W), inputs.f32(mi.b)
    SX, SW = mi.SX.numpy(), mi.SW.numpy()
    assert len(np.unique(SX)) > 4 and len(np.unique(SW)) > 4
    got = ref.fused_linear_mxfp8(X8, SX, W8, SW, b, ref.ACT_NONE)
    # library pin: dequantise in torch fp64, then a plain matmul
    want = _mx_dequant(mi.X, mi.SX) @ _mx_dequant(mi.W, mi.SW).T + mi.b.double()
    np.testing.assert_allclose(got, want.numpy(), rtol=1e-13, atol=1e-13)
    # exact brute force with rationals: element = integer / 512, scale = 2^(byte - 127)
    raw = ref.fused_linear_mxfp8(X8, SX, W8, SW, None, ref.ACT_NONE)
    xi = (mi.X.to(torch.float64) * 512).numpy().astype(np.int64)
    wi = (mi.W.to(torch.float64) * 512).numpy().astype(np.int64)
    for m in range(3):
        for n in range(4):
            acc = Fraction(0)
            for k in range(128):
                acc += Fraction(int(xi[m, k]), 512) * Fraction(2) ** (int(SX[m, k // 32]) - 127) * \
                       Fraction(int(wi[n, k]), 512) * Fraction(2) ** (int(SW[n, k // 32]) - 127)
            assert abs(raw[m, n] - float(acc)) <= 1e-13 * max(1.0, abs(float(acc)))
    # equal block scales reduce to the per-tensor form, bit for bit (powers of two are exact per-tensor scales)
    SXc, SWc = np.full_like(SX, 121), np.full_like(SW, 130)
    same = ref.fused_linear_mxfp8(X8, SXc, W8, SWc, b, ref.ACT_SILU)
    per_tensor = ref.fused_linear_fp8(X8, W8, b, 2.0 ** (121 - 127), 2.0 ** (130 - 127), ref.ACT_SILU)
    assert np.array_equal(same, per_tensor)
    # one more on every X scale doubles z; the contribution of a block depends on its own scales only
    doubled = ref.fused_linear_mxfp8(X8, SX + 1, W8, SW, None, ref.ACT_NONE)
    np.testing.assert_allclose(doubled, 2.0 * raw, rtol=1e-15, atol=0)
    parts = np.zeros_like(raw)
    for blk in range(4):
        ks = slice(32 * blk, 32 * blk + 32)
        parts += ref.fused_linear_mxfp8(np.ascontiguousarray(X8[:, ks]), np.ascontiguousarray(SX[:, blk:blk + 1]),
                                        np.ascontiguousarray(W8[:, ks]), np.ascontiguousarray(SW[:, blk:blk + 1]), None, ref.ACT_NONE)
    np.testing.assert_allclose(parts, raw, rtol=1e-13, atol=1e-13)
    # swapping the scales of two blocks of one row changes that row only, and not into the same value
    SX2 = SX.copy()
    SX2[0, 0], SX2[0, 1] = SX[0, 1] + 3, SX[0, 0]
    swapped = ref.fused_linear_mxfp8(X8, SX2, W8, SW, None, ref.ACT_NONE)
    assert np.array_equal(swapped[1:], raw[1:]) and not np.allclose(swapped[0], raw[0])


def test_mxfp8_swiglu_and_lse_pins():
    mi = inputs.mx_linear_inputs(5, 9, 96, seed=82, spread=4)
    up = inputs.mx_linear_inputs(5, 9, 96, seed=83, spread=4)
    X8, SX = inputs.fp8_bits(mi.X), mi.SX.numpy()
    G8, SG, U8, SU = inputs.fp8_bits(mi.W), mi.SW.numpy(), inputs.fp8_bits(up.W), up.SW.numpy()
    got = ref.swiglu_mxfp8(X8, SX, G8, SG, U8, SU)
    g = ref.fused_linear_mxfp8(X8, SX, G8, SG, None, ref.ACT_SILU)          # product of the two pinned layers
    u = ref.fused_linear_mxfp8(X8, SX, U8, SU, None, ref.ACT_NONE)
    np.testing.assert_allclose(got, g * u, rtol=1e-14, atol=0)
    xd = _mx_dequant(mi.X, mi.SX)
    want = torch.nn.functional.silu(xd @ _mx_dequant(mi.W, mi.SW).T) * (xd @ _mx_dequant(up.W, up.SW).T)
    np.testing.assert_allclose(got, want.numpy(), rtol=1e-12, atol=1e-13)
    assert np.all(ref.swiglu_mxfp8(X8, SX, np.zeros_like(G8), SG, U8, SU) == 0)
    b = inputs.f32(mi.b)
    lse = ref.linear_lse_mxfp8(X8, SX, G8, SG, b)
    z = xd @ _mx_dequant(mi.W, mi.SW).T + mi.b.double()
    np.testing.assert_allclose(lse, torch.logsumexp(z, dim=-1).numpy(), rtol=1e-13, atol=1e-13)
    shifted = ref.linear_lse_mxfp8(X8, SX, G8, SG, b + np.float32(2.0))
    np.testing.assert_allclose(shifted - lse, 2.0, rtol=0, atol=1e-6)       # b + 2 is rounded to fp32 before it is used


def test_activation_closed_forms():
    ids = {"relu": ref.ACT_RELU, "gelu_tanh": ref.ACT_GELU_TANH, "silu": ref.ACT_SILU}
    seen = 0
    for kind, arg, val in _closed_forms():
        if kind in ids:
            got = ref.act(ids[kind], float(arg))
            # 1 + tanh(.) cancels for very negative z: the formula in double carries ~1e-16 absolute error there
            assert got == pytest.approx(val, rel=4e-15, abs=1e-15), (kind, arg)
            seen += 1
    assert seen == 39


def test_activation_identities():
    zs = np.linspace(-9.0, 9.0, 181)
    for kind in (ref.ACT_RELU, ref.ACT_GELU_TANH, ref.ACT_SILU):
        for z in zs:
            # act(z) - act(-z) = z for ReLU, GELU-tanh (tanh odd) and SiLU (sigma(z)+sigma(-z)=1)
            assert ref.act(kind, z) - ref.act(kind, -z) == pytest.approx(z, abs=1e-14)
        assert ref.act(kind, 0.0) == 0.0
        assert ref.act(kind, 40.0) == pytest.approx(40.0, rel=1e-15)
        assert abs(ref.act(kind, -40.0)) < 1e-15
    h = 1e-6   # slope one half at the origin for the two smooth activations
    for kind in (ref.ACT_GELU_TANH, ref.ACT_SILU):
        assert (ref.act(kind, h) - ref.act(kind, -h)) / (2 * h) == pytest.approx(0.5, abs=1e-9)
    assert ref.act(ref.ACT_RELU, 2 * 1.7) == 2 * ref.act(ref.ACT_RELU, 1.7)
    assert ref.act(ref.ACT_NONE, -3.25) == -3.25


# ---------------------------------------------------------------- SwiGLU
def test_swiglu_laws():
    si = inputs.swiglu_inputs(6, 9, 32, seed=31)
    X, Wg, Wu = (inputs.bf16_bits(t) for t in (si.X, si.Wg, si.Wu))
    out = ref.swiglu(X, Wg, Wu)
    # equal weights: silu(z) * z
    z = ref.fused_linear(X, Wg, None, ref.ACT_NONE)
    same = ref.swiglu(X, Wg, Wg)
    want = torch.nn.functional.silu(torch.from_numpy(z)) * torch.from_numpy(z)
    np.testing.assert_allclose(same, want.numpy(), rtol=1e-13, atol=1e-15)
    zero = np.zeros_like(Wu)
    assert np.all(ref.swiglu(X, Wg, zero) == 0.0)        # up = 0
    assert np.all(ref.swiglu(X, zero, Wu) == 0.0)        # silu(0) = 0
    Wu2 = bits(2.0 * widen(Wu))
    assert np.array_equal(ref.swiglu(X, Wg, Wu2), 2.0 * out)
    gate = ref.fused_linear(X, Wg, None, ref.ACT_SILU)
    up = ref.fused_linear(X, Wu, None, ref.ACT_NONE)
    assert np.array_equal(out, gate * up)
    tw = torch.nn.functional.silu(si.X.double() @ si.Wg.double().T) * (si.X.double() @ si.Wu.double().T)
    np.testing.assert_allclose(out, tw.numpy(), rtol=1e-12, atol=1e-13)
    # gate and up are not interchangeable
    assert not np.allclose(out, ref.swiglu(X, Wu, Wg))
    rows, cols = np.array([0, 5, 3]), np.array([8, 0, 4])
    assert np.array_equal(ref.swiglu_points(X, Wg, Wu, rows, cols), out[rows, cols])


# ---------------------------------------------------------------- logsumexp
def test_lse_closed_forms():
    seen = 0
    for kind, arg, val in _closed_forms():
        if kind == "lse":
            v = [float(t) for t in arg.split(",")]
            assert ref.lse_vector(v) == pytest.approx(val, rel=4e-15), arg
            seen += 1
    assert seen == 6
    assert ref.lse_vector([0, 0, 0, 0]) == pytest.approx(math.log(4.0), rel=1e-15)


def test_lse_laws_on_vectors():
    rng = np.random.default_rng(41)
    z = rng.normal(size=200)
    base = ref.lse_vector(z)
    for c in (-700.0, -3.5, 12.25, 900.0):
        assert ref.lse_vector(z + c) == pytest.approx(base + c, abs=1e-12 * max(1.0, abs(c)))   # shift law
    assert np.sum(np.exp(z - base)) == pytest.approx(1.0, abs=1e-13)                           # softmax sums to 1
    assert z.max() <= base <= z.max() + math.log(z.size)
    assert ref.lse_vector(np.full(37, -2.5)) == pytest.approx(-2.5 + math.log(37), rel=1e-15)
    assert ref.lse_vector([4.75]) == 4.75
    assert ref.lse_vector(z[rng.permutation(200)]) == pytest.approx(base, abs=1e-13)
    a, b = ref.lse_vector(z[:77]), ref.lse_vector(z[77:])                                     # merge law
    assert math.log(math.exp(a) + math.exp(b)) == pytest.approx(base, abs=1e-13)
    assert base == pytest.approx(float(torch.logsumexp(torch.from_numpy(z), 0)), abs=1e-13)


def test_linear_lse_end_to_end():
    li = inputs.linear_inputs(5, 300, 48, seed=42)
    X, W, b = inputs.bf16_bits(li.X), inputs.bf16_bits(li.W), inputs.f32(li.b)
    lse, logits = ref.linear_lse(X, W, b, want_logits=True)
    z = (li.X.double() @ li.W.double().T + li.b.double())
    np.testing.assert_allclose(logits, z.numpy(), rtol=0, atol=1e-12)
    np.testing.assert_allclose(lse, torch.logsumexp(z, -1).numpy(), rtol=0, atol=1e-12)
    np.testing.assert_allclose(np.exp(logits - lse[:, None]).sum(axis=1), np.ones(5), rtol=0, atol=1e-12)
    # adding c to every bias shifts every lse by c (c exactly representable)
    b_shift = (li.b.double() + 2.0).float().numpy()
    exact_shift = b_shift.astype(np.float64) - b.astype(np.float64)   # what fp32 rounding really added per column
    lse_s = ref.linear_lse(X, W, b_shift, False)
    assert np.all(np.abs(lse_s - lse - 2.0) <= np.abs(exact_shift - 2.0).max() + 1e-12)
    # zero weights: lse = lse(b); no bias and zero weights: ln N
    W0 = np.zeros_like(W)
    assert ref.linear_lse(X, W0, b, False)[0] == pytest.approx(ref.lse_vector(b.astype(np.float64)), abs=1e-13)
    assert ref.linear_lse(X, W0, None, False)[3] == pytest.approx(math.log(300), rel=1e-15)
    # N = 1: lse = z
    l1 = ref.linear_lse(X, W[:1].copy(), b[:1].copy(), False)
    np.testing.assert_allclose(l1, z.numpy()[:, 0], rtol=0, atol=1e-12)
    rows = np.array([4, 0, 2])
    np.testing.assert_array_equal(ref.linear_lse_rows(X, W, b, rows), lse[rows])


def test_softmax_golden_values():
    """40-digit values of exp(z_i - lse(z)) for five logit vectors (moderate, spread over 40 units, offset by 1000)."""
    seen = 0
    for kind, arg, val in _closed_forms():
        if kind == "softmax":
            logits, idx = arg.split("|")
            p = ref.softmax_vector([float(t) for t in logits.split(",")])
            assert p[int(idx)] == pytest.approx(val, rel=2e-13), arg      # exp(-20) near 1e-9: fp64 keeps 13 digits of it
            seen += 1
    assert seen == 19


def test_softmax_closed_forms_and_laws():
    # logits ln(a_i) for integers a_i: p_i = a_i / sum(a) exactly in the rationals
    a = [1, 2, 3, 10, 48]
    p = ref.softmax_vector([math.log(v) for v in a])
    for got, v in zip(p, a):
        assert got == pytest.approx(float(Fraction(v, sum(a))), rel=4e-15)
    # equal logits: 1/N; one logit: 1; far-apart and huge logits neither overflow nor lose the winner
    np.testing.assert_allclose(ref.softmax_vector(np.full(37, -2.5)), np.full(37, 1.0 / 37), rtol=1e-15)
    assert ref.softmax_vector([4.75])[0] == 1.0
    np.testing.assert_array_equal(ref.softmax_vector([1000.0, 1000.0]), [0.5, 0.5])
    np.testing.assert_array_equal(ref.softmax_vector([-1000.0, 0.0]), [0.0, 1.0])
    # two classes: softmax([z, 0])[0] is the logistic function 1 / (1 + exp(-z))
    for z in (-30.0, -2.25, 0.0, 0.5, 7.0, 40.0):
        assert ref.softmax_vector([z, 0.0])[0] == pytest.approx(1.0 / (1.0 + math.exp(-z)), rel=4e-16, abs=0)
    rng = np.random.default_rng(43)
    z = rng.normal(size=200) * 3.0
    p = ref.softmax_vector(z)
    assert p.sum() == pytest.approx(1.0, abs=1e-14) and np.all(p > 0)
    for c in (-700.0, -3.5, 12.25, 900.0):                                   # shift invariance
        np.testing.assert_allclose(ref.softmax_vector(z + c), p, rtol=1e-12 * max(1.0, abs(c)))
    perm = rng.permutation(200)                                              # permutation equivariance
    np.testing.assert_allclose(ref.softmax_vector(z[perm]), p[perm], rtol=1e-13)
    np.testing.assert_array_equal(np.argsort(p, kind="stable"), np.argsort(z, kind="stable"))   # monotone in the logits
    i, j = 17, 133                                                           # ratios: p_i / p_j = exp(z_i - z_j)
    assert p[i] / p[j] == pytest.approx(math.exp(z[i] - z[j]), rel=1e-13)
    np.testing.assert_allclose(p, np.exp(z - ref.lse_vector(z)), rtol=1e-12)                  # the logsumexp form
    np.testing.assert_allclose(p, torch.softmax(torch.from_numpy(z), 0).numpy(), rtol=1e-13)  # library routine


def test_linear_softmax_end_to_end():
    li = inputs.linear_inputs(5, 300, 48, seed=44)
    X, W, b = inputs.bf16_bits(li.X), inputs.bf16_bits(li.W), inputs.f32(li.b)
    P = ref.linear_softmax(X, W, b)
    z = li.X.double() @ li.W.double().T + li.b.double()
    np.testing.assert_allclose(P, torch.softmax(z, -1).numpy(), rtol=1e-12, atol=0)
    np.testing.assert_allclose(P.sum(axis=1), np.ones(5), rtol=0, atol=1e-13)
    # consistent with the other oracle routes to the same logits: exp(z - lse), and act = none pre-activations
    lse = ref.linear_lse(X, W, b)
    np.testing.assert_allclose(P, np.exp(ref.fused_linear(X, W, b, ref.ACT_NONE) - lse[:, None]), rtol=1e-12)
    # the expected negative log-probability of a column is the cross entropy with that target
    tgt = np.array([0, 299, 17, 150, 42])
    loss, _ = ref.linear_cross_entropy(X, W, b, tgt)
    np.testing.assert_allclose(-np.log(P[np.arange(5), tgt]), loss, rtol=0, atol=1e-12)
    # zero weights: softmax(b) in every row; zero weights and no bias: 1/N; N = 1: all ones
    W0 = np.zeros_like(W)
    np.testing.assert_allclose(ref.linear_softmax(X, W0, b)[3], ref.softmax_vector(b.astype(np.float64)), rtol=1e-14)
    np.testing.assert_array_equal(ref.linear_softmax(X, W0, None), np.full((5, 300), 1.0 / 300))
    np.testing.assert_array_equal(ref.linear_softmax(X, W[:1].copy(), b[:1].copy()), np.ones((5, 1)))
    # a transposed operand or a dropped bias would move the row maximum's place
    assert np.array_equal(P.argmax(axis=1), z.numpy().argmax(axis=1))
    rows = np.array([4, 0, 2])
    np.testing.assert_array_equal(ref.linear_softmax_rows(X, W, b, rows), P[rows])


def test_lse_expected_level_for_unit_variance_logits():
    # logits ~ N(0,1) + small bias over N columns: lse ~ ln N + 1/2 (lognormal mean)
    li = inputs.linear_inputs(4, 4000, 256, seed=43)
    lse = ref.linear_lse(inputs.bf16_bits(li.X), inputs.bf16_bits(li.W), inputs.f32(li.b))
    assert np.all(np.abs(lse - (math.log(4000) + 0.5)) < 0.15)


# ---------------------------------------------------------------- row max, cross entropy
def test_rowmax_pins():
    li = inputs.linear_inputs(7, 300, 48, seed=61)
    X, W, b = inputs.bf16_bits(li.X), inputs.bf16_bits(li.W), inputs.f32(li.b)
    mx, arg = ref.linear_rowmax(X, W, b)
    z = li.X.double() @ li.W.double().T + li.b.double()
    tmax, targ = z.max(dim=-1)
    np.testing.assert_allclose(mx, tmax.numpy(), rtol=0, atol=1e-12)
    assert np.array_equal(arg, targ.numpy())
    # zero weights: the row max is max(b), attained at argmax(b), for every row
    mx0, arg0 = ref.linear_rowmax(X, np.zeros_like(W), b)
    assert np.all(mx0 == float(b.max())) and np.all(arg0 == int(b.argmax()))
    # ties go to the lowest index: two identical weight rows and biases
    W2 = W.copy(); W2[200] = W2[17]; b2 = b.copy(); b2[200] = b2[17]
    _, arg2 = ref.linear_rowmax(X, W2, b2)
    assert not np.any(arg2 == 200)
    # the maximum bounds logsumexp from below within ln N
    lse = ref.linear_lse(X, W, b)
    assert np.all(mx <= lse) and np.all(lse <= mx + math.log(300))
    # permuting the columns permutes the argmax and leaves the max unchanged
    perm = np.random.default_rng(2).permutation(300)
    mxp, argp = ref.linear_rowmax(X, W[perm].copy(), b[perm].copy())
    assert np.array_equal(mxp, mx) and np.array_equal(perm[argp], arg)


def test_cross_entropy_pins():
    li = inputs.linear_inputs(9, 250, 64, seed=62)
    X, W, b = inputs.bf16_bits(li.X), inputs.bf16_bits(li.W), inputs.f32(li.b)
    tgt = np.random.default_rng(3).integers(0, 250, size=9)
    loss, lse = ref.linear_cross_entropy(X, W, b, tgt)
    z = li.X.double() @ li.W.double().T + li.b.double()
    want = torch.nn.functional.cross_entropy(z, torch.from_numpy(tgt), reduction="none")
    np.testing.assert_allclose(loss, want.numpy(), rtol=0, atol=1e-12)
    np.testing.assert_array_equal(lse, ref.linear_lse(X, W, b))
    assert np.all(loss >= 0.0)
    # -log softmax: exp(-loss) is the softmax probability of the target, and the probabilities of a row sum to 1
    row = [float(np.exp(-ref.linear_cross_entropy(X[:1], W, b, np.array([n]))[0][0])) for n in range(250)]
    assert sum(row) == pytest.approx(1.0, abs=1e-12)
    # all logits equal: loss = ln N whatever the target
    l0, _ = ref.linear_cross_entropy(X, np.zeros_like(W), None, tgt)
    np.testing.assert_allclose(l0, np.full(9, math.log(250)), rtol=1e-15)
    # adding a constant to every bias changes lse but not the loss (2.0 keeps b's low bits only approximately: bound it)
    b_shift = (li.b.double() + 2.0).float().numpy()
    ls, _ = ref.linear_cross_entropy(X, W, b_shift, tgt)
    assert np.all(np.abs(ls - loss) <= 2 * np.abs((b_shift.astype(np.float64) - b.astype(np.float64)) - 2.0).max() + 1e-12)
    # target = argmax gives the smallest loss of the row: lse - max
    mx, arg = ref.linear_rowmax(X, W, b)
    la, _ = ref.linear_cross_entropy(X, W, b, arg)
    np.testing.assert_allclose(la, lse - mx, rtol=0, atol=1e-12)
    assert np.all(la <= loss + 1e-12)
    with pytest.raises(ValueError):
        ref.linear_cross_entropy(X, W, b, np.full(9, 250))


# ---------------------------------------------------------------- sampled variants, threads, comparator
def test_points_match_full_and_threads_do_not_matter():
    li = inputs.linear_inputs(20, 31, 72, seed=51)
    X, W, b = inputs.bf16_bits(li.X), inputs.bf16_bits(li.W), inputs.f32(li.b)
    rows, cols = inputs.sample_points(20, 31, 25, seed=3, tile_m=8, tile_n=8)
    full = ref.fused_linear(X, W, b, ref.ACT_GELU_TANH)
    assert np.array_equal(ref.fused_linear_points(X, W, b, ref.ACT_GELU_TANH, rows, cols), full[rows, cols])
    ref.set_threads(1)
    try:
        assert np.array_equal(ref.fused_linear(X, W, b, ref.ACT_GELU_TANH), full)
    finally:
        ref.set_threads(0)
    assert ref.get_threads() >= 1


def test_bad_arguments_are_rejected():
    X = np.zeros((2, 4), dtype=np.uint16)
    W = np.zeros((3, 4), dtype=np.uint16)
    with pytest.raises(ValueError):
        ref.fused_linear(X, W, None, 7)
    with pytest.raises(ValueError):
        ref.fused_linear_points(X, W, None, 0, [2], [0])
    with pytest.raises(TypeError):
        ref.fused_linear(X.astype(np.float32), W, None, 0)


def test_comparator():
    refv = np.array([1.0, -2.0, 0.0, 100.0])
    ok = ref.compare(refv + np.array([0.019, -0.029, 0.0099, 1.0]), refv, 1e-2, 1e-2)
    assert ok["ok"] and ok["violations"] == 0 and ok["max_abs_err"] == pytest.approx(1.0)
    bad = ref.compare(refv + np.array([0.021, 0.0, 0.0, 0.0]), refv, 1e-2, 1e-2)
    assert not bad["ok"] and bad["violations"] == 1 and bad["worst_index"] == 0
    nan = ref.compare(np.array([np.nan, 1.0]), np.array([0.0, 1.0]), 1.0, 1.0)
    assert nan["violations"] == 1
    inf = ref.compare(np.array([np.inf]), np.array([np.inf]), 1.0, 1.0)
    assert inf["violations"] == 1
