"""Seeded synthetic inputs shared by the CUDA tests, the oracle tests and the benchmark.

This module holds none of the method's arithmetic: it only draws random tensors
with the stated distributions and rounds them to bf16.  Both the CUDA path and
the CPU oracle receive the very same arrays, so parity never depends on the
generator.

Recipe ("seed s"): a torch CPU generator seeded with s; fp32 draws in the fixed
order X, W (or Wg then Wu), b:
    X  = randn(M, K)                 -> bf16 (round to nearest even)
    W  = randn(N, K) * K**-0.5       -> bf16   (variance 1/K, so X.W^T ~ N(0,1))
    b  = rand(N) * 0.2 - 0.1         (fp32, U(-0.1, 0.1), not rounded)
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np
import torch

# The five benchmark configurations (shape, call, seed).
CONFIGS = {
    "C1": dict(op="fused_linear", M=256, N=256, K=256, act="relu", out_dtype="fp32", seed=0),
    "C2": dict(op="fused_linear", M=4096, N=4096, K=4096, act="gelu_tanh", out_dtype="bf16", seed=1),
    "C3": dict(op="swiglu", M=8192, N=11008, K=4096, seed=2),
    "C4": dict(op="linear_lse", M=4096, N=32000, K=4096, seed=3),
    "C5": dict(op="fused_linear", M=16, N=8192, K=8192, act="gelu_tanh", out_dtype="bf16", seed=4),
}

# Further operators of the same family (measured beside the five, not part of the benchmark step).
EXTRA_CONFIGS = {
    "X1": dict(op="linear_rowmax", M=4096, N=32000, K=4096, seed=3),
    "X2": dict(op="linear_cross_entropy", M=4096, N=32000, K=4096, seed=3),
    # the MLP down-projection that follows C3, with the skip connection joined to the epilogue
    "X3": dict(op="fused_linear_residual", M=8192, N=4096, K=11008, act="none", out_dtype="bf16", seed=5),
    # C2 and the SwiGLU-sized GEMM with E4M3 operands (tensor peak is twice the bf16 one)
    "X4": dict(op="fused_linear_fp8", M=4096, N=4096, K=4096, act="gelu_tanh", out_dtype="bf16", seed=1),
    "X5": dict(op="fused_linear_fp8", M=8192, N=8192, K=8192, act="gelu_tanh", out_dtype="bf16", seed=6),
    # the decode GEMM of C5 with E4M3 weights and activations: half the bytes to stream
    "X6": dict(op="fused_linear_fp8", M=16, N=8192, K=8192, act="gelu_tanh", out_dtype="bf16", seed=4),
    # a decode batch of 128 rows against the same weights: too many rows for the weight-streaming kernel, one
    # row block of 32 tiles for the tiled one -> clusters of four CTAs per tile, split along K
    "X7": dict(op="fused_linear", M=128, N=8192, K=8192, act="gelu_tanh", out_dtype="bf16", seed=7),
    # C2 and the 8192-cube with block-scaled E4M3 operands (MXFP8: one power-of-two scale per 32 elements of K)
    "X8": dict(op="fused_linear_mxfp8", M=4096, N=4096, K=4096, act="gelu_tanh", out_dtype="bf16", seed=1),
    "X9": dict(op="fused_linear_mxfp8", M=8192, N=8192, K=8192, act="gelu_tanh", out_dtype="bf16", seed=6),
    # a decode batch against a 4096-wide layer: 32 tiles of 128 x 128, clusters of four CTAs per tile split along K
    "X10": dict(op="fused_linear", M=128, N=4096, K=4096, act="gelu_tanh", out_dtype="bf16", seed=8),
    # X7's 8192-wide layer against 256 rows (clusters of two CTAs per tile) and 512 rows (64 pair tiles on 74 pairs)
    "X12": dict(op="fused_linear", M=256, N=8192, K=8192, act="gelu_tanh", out_dtype="bf16", seed=9),
    "X13": dict(op="fused_linear", M=512, N=8192, K=8192, act="gelu_tanh", out_dtype="bf16", seed=10),
    # C4's logits as probabilities: the row softmax written out in bf16 (the logits themselves never are)
    "X11": dict(op="linear_softmax", M=4096, N=32000, K=4096, out_dtype="bf16", seed=3),
}


def residual(M: int, N: int, seed: int, dtype=torch.bfloat16) -> torch.Tensor:
    """Seeded N(0,1) residual stream [M,N] in the output dtype."""
    return torch.randn(M, N, generator=_gen(seed + 1000), dtype=torch.float32).to(dtype)


def targets(M: int, N: int, seed: int) -> torch.Tensor:
    """Seeded uniform target columns, int64 [M]."""
    return torch.from_numpy(np.random.default_rng(seed).integers(0, N, size=M))


@dataclass
class LinearInputs:
    X: torch.Tensor            # [M, K] bf16, CPU
    W: torch.Tensor            # [N, K] bf16, CPU
    b: torch.Tensor | None     # [N] fp32, CPU


@dataclass
class SwigluInputs:
    X: torch.Tensor            # [M, K] bf16
    Wg: torch.Tensor           # [N, K] bf16
    Wu: torch.Tensor           # [N, K] bf16


def _gen(seed: int) -> torch.Generator:
    g = torch.Generator(device="cpu")
    g.manual_seed(int(seed))
    return g


def linear_inputs(M: int, N: int, K: int, seed: int, bias: bool = True) -> LinearInputs:
    g = _gen(seed)
    X = torch.randn(M, K, generator=g, dtype=torch.float32).to(torch.bfloat16)
    W = (torch.randn(N, K, generator=g, dtype=torch.float32) * (float(K) ** -0.5)).to(torch.bfloat16)
    b = (torch.rand(N, generator=g, dtype=torch.float32) * 0.2 - 0.1) if bias else None
    return LinearInputs(X, W, b)


def swiglu_inputs(M: int, N: int, K: int, seed: int) -> SwigluInputs:
    g = _gen(seed)
    X = torch.randn(M, K, generator=g, dtype=torch.float32).to(torch.bfloat16)
    Wg = (torch.randn(N, K, generator=g, dtype=torch.float32) * (float(K) ** -0.5)).to(torch.bfloat16)
    Wu = (torch.randn(N, K, generator=g, dtype=torch.float32) * (float(K) ** -0.5)).to(torch.bfloat16)
    return SwigluInputs(X, Wg, Wu)


@dataclass
class Fp8LinearInputs:
    X: torch.Tensor            # [M, K] float8_e4m3fn, CPU
    W: torch.Tensor            # [N, K] float8_e4m3fn, CPU
    b: torch.Tensor | None     # [N] fp32
    scale_x: float             # per-tensor scales: real value = scale * stored value
    scale_w: float


def fp8_linear_inputs(M: int, N: int, K: int, seed: int, bias: bool = True) -> Fp8LinearInputs:
    """The bf16 recipe's draws, quantised per tensor to E4M3 with the scale that maps the largest
    magnitude to 448 (the format's maximum); scales are rounded to fp32."""
    li = linear_inputs(M, N, K, seed, bias)
    out = []
    for t in (li.X.float(), li.W.float()):
        scale = float(torch.tensor(float(t.abs().max()) / 448.0, dtype=torch.float32)) or 1.0
        out.append(((t / scale).to(torch.float8_e4m3fn), scale))
    return Fp8LinearInputs(out[0][0], out[1][0], li.b, out[0][1], out[1][1])


def fp8_swiglu_inputs(M: int, N: int, K: int, seed: int):
    """The SwiGLU recipe's draws quantised per tensor to E4M3: (X8, Wg8, Wu8, scale_x, scale_g, scale_u)."""
    si = swiglu_inputs(M, N, K, seed)
    out = []
    for t in (si.X.float(), si.Wg.float(), si.Wu.float()):
        scale = float(torch.tensor(float(t.abs().max()) / 448.0, dtype=torch.float32)) or 1.0
        out.append(((t / scale).to(torch.float8_e4m3fn), scale))
    return out[0][0], out[1][0], out[2][0], out[0][1], out[1][1], out[2][1]


def mx_quantize(t: torch.Tensor):
    """Block-scaled E4M3 (MXFP8) quantisation of a 2-D fp32/bf16 tensor [R, K], K % 32 == 0: per row and block of
    32 consecutive columns a shared power-of-two scale 2^e with e = floor(log2(max |block|)) - 8 (8 = the exponent
    of the largest E4M3 binade, as in the OCP microscaling recipe; an all-zero block takes e = 0), elements
    rounded to E4M3 after division by the scale (saturating at 448).  Returns (float8_e4m3fn [R,K], uint8
    scales [R,K/32] holding e + 127)."""
    R, K = t.shape
    assert K % 32 == 0
    blocks = t.float().reshape(R, K // 32, 32)
    amax = blocks.abs().amax(dim=-1)
    e = torch.where(amax > 0, torch.floor(torch.log2(amax.clamp_min(1e-38))) - 8.0, torch.zeros_like(amax)).clamp(-127.0, 127.0)
    scaled = (blocks / torch.exp2(e).unsqueeze(-1)).clamp(-448.0, 448.0)
    return scaled.reshape(R, K).to(torch.float8_e4m3fn), (e + 127.0).to(torch.uint8)


@dataclass
class MxLinearInputs:
    X: torch.Tensor            # [M, K] float8_e4m3fn, CPU
    SX: torch.Tensor           # [M, K/32] uint8 (UE8M0), CPU
    W: torch.Tensor            # [N, K] float8_e4m3fn
    SW: torch.Tensor           # [N, K/32] uint8
    b: torch.Tensor | None     # [N] fp32


def mx_linear_inputs(M: int, N: int, K: int, seed: int, bias: bool = True, spread: float = 0.0) -> MxLinearInputs:
    """The bf16 recipe's draws quantised to MXFP8.  spread > 0 multiplies every 32-block of X and of W by its own
    seeded power of two in [2^-spread, 2^spread] first, so that neighbouring blocks carry very different scales."""
    li = linear_inputs(M, N, K, seed, bias)
    X, W = li.X.float(), li.W.float()
    if spread > 0:
        g = _gen(seed + 77)
        ex = torch.randint(-int(spread), int(spread) + 1, (M, K // 32), generator=g).float()
        ew = torch.randint(-int(spread), int(spread) + 1, (N, K // 32), generator=g).float()
        X = (X.reshape(M, K // 32, 32) * torch.exp2(ex).unsqueeze(-1)).reshape(M, K)
        W = (W.reshape(N, K // 32, 32) * torch.exp2(ew).unsqueeze(-1)).reshape(N, K)
    X8, SX = mx_quantize(X)
    W8, SW = mx_quantize(W)
    return MxLinearInputs(X8, SX, W8, SW, li.b)


def fp8_bits(t: torch.Tensor) -> np.ndarray:
    """float8_e4m3fn tensor (CPU) -> uint8 numpy array of the raw bit patterns."""
    assert t.dtype == torch.float8_e4m3fn
    return t.detach().cpu().contiguous().view(torch.uint8).numpy()


def bf16_bits(t: torch.Tensor) -> np.ndarray:
    """bf16 tensor (CPU) -> uint16 numpy array of the same shape holding the raw bit patterns."""
    assert t.dtype == torch.bfloat16
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16)


def bits_to_bf16(a: np.ndarray) -> torch.Tensor:
    """uint16 bit patterns -> bf16 torch tensor (CPU) of the same shape."""
    assert a.dtype == np.uint16
    return torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).view(torch.bfloat16)


def f32(t: torch.Tensor | None) -> np.ndarray | None:
    return None if t is None else t.detach().cpu().contiguous().numpy()


def to_f64(t: torch.Tensor) -> np.ndarray:
    """Exact widening of a result tensor (fp32 or bf16, any device) to float64 numpy."""
    return t.detach().to("cpu").to(torch.float64).numpy()


def sample_points(M: int, N: int, count: int, seed: int, tile_m: int = 128, tile_n: int = 128):
    """(rows, cols) for sampled parity: the four corners of the output, first/last
    element of tile-edge rows and columns, plus `count` seeded uniform positions."""
    rng = np.random.default_rng(seed)
    rows = list(rng.integers(0, M, size=count))
    cols = list(rng.integers(0, N, size=count))
    edge_r = sorted({0, M - 1, min(tile_m - 1, M - 1), min(tile_m, M - 1), (M // tile_m) * tile_m - 1 if M >= tile_m else 0,
                     min((M // tile_m) * tile_m, M - 1)})
    edge_c = sorted({0, N - 1, min(tile_n - 1, N - 1), min(tile_n, N - 1), (N // tile_n) * tile_n - 1 if N >= tile_n else 0,
                     min((N // tile_n) * tile_n, N - 1)})
    for r in edge_r:
        for c in edge_c:
            rows.append(r)
            cols.append(c)
    return np.asarray(rows, dtype=np.int64), np.asarray(cols, dtype=np.int64)
