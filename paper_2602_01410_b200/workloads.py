"""Seeded synthetic inputs for the mixed-precision linear layer.

This module only draws numbers and lists shapes.  It holds none of the method's arithmetic
(no scaling rule, no rounding to FP8/FP4, no GEMM), so both the CPU oracle's tests and the CUDA
path's tests can take their inputs from it: the same bf16 bytes go to both sides.

Recipe (stands in for the paper's real training tensors, which need checkpoints and datasets):
  X   ~ N(0,1); a seeded subset of the feature columns (the "outlier channels") is multiplied
        by a constant, as LLM activations show a few large-magnitude channels;
  W   ~ N(0, 0.02);
  dY  ~ N(0, 1e-3) times a per-row log-normal(0,1) factor (token-dependent gradient scale).
Values are drawn in float32 and rounded once, to nearest-even, to bf16.
Shapes are the Llama-like linears (Q/K/V fused, O, gate, up, down) of Fig. 4 of the paper.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np

BASE_SEED = 260201410
FMT_BF16, FMT_FP8, FMT_FP4 = 0, 1, 2
FMT_NAMES = {FMT_BF16: "bf16", FMT_FP8: "fp8_e4m3", FMT_FP4: "fp4_e2m1"}
TENSOR_IDS = {"X": 0, "W": 1, "dY": 2, "tags": 3, "aux": 4}


def to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """float32 -> bf16 bit patterns (uint16), round-to-nearest ties-to-even; finite inputs."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    lsb = (u >> np.uint32(16)) & np.uint32(1)
    return ((u + np.uint32(0x7FFF) + lsb) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def rng_for(config: int, layer: int, linear: int, tensor: str) -> np.random.Generator:
    ss = np.random.SeedSequence([BASE_SEED, config, layer, linear, TENSOR_IDS[tensor]])
    return np.random.Generator(np.random.Philox(ss))


def _normal_f32(rng, shape):
    return rng.standard_normal(shape, dtype=np.float32)


def make_x(rng, M, K, outlier_frac=0.01, outlier_scale=20.0) -> np.ndarray:
    x = _normal_f32(rng, (M, K))
    n_out = int(np.ceil(outlier_frac * K)) if outlier_frac > 0 else 0
    if n_out:
        cols = rng.permutation(K)[:n_out]
        x[:, cols] *= np.float32(outlier_scale)
    return to_bf16_bits(x)


def make_w(rng, N, K) -> np.ndarray:
    return to_bf16_bits(_normal_f32(rng, (N, K)) * np.float32(0.02))


def make_dy(rng, M, N) -> np.ndarray:
    g = _normal_f32(rng, (M, N)) * np.float32(1e-3)
    row = np.exp(_normal_f32(rng, (M, 1)))
    return to_bf16_bits(g * row)


@dataclass(frozen=True)
class Linear:
    name: str
    K: int  # in-features
    N: int  # out-features


@dataclass(frozen=True)
class Config:
    index: int
    name: str
    M: int                      # tokens per step
    linears: tuple              # Linear entries of one transformer block
    layers: int
    outlier_frac: float
    outlier_scale: float
    tag_rule: str               # how precision tags are drawn, see precision_tags()


def _block(hidden, ffn, qkv_out):
    return (Linear("qkv", hidden, qkv_out), Linear("o", hidden, hidden),
            Linear("gate", hidden, ffn), Linear("up", hidden, ffn), Linear("down", ffn, hidden))


CONFIGS = (
    Config(0, "single-512", 512, (Linear("lin", 512, 512),), 1, 0.01, 20.0, "fixed-fp8-fp8-fp4"),
    Config(1, "llama-1b", 8192,
           (Linear("q", 2048, 2048), Linear("k", 2048, 256), Linear("v", 2048, 256),
            Linear("o", 2048, 2048), Linear("gate", 2048, 5632), Linear("up", 2048, 5632),
            Linear("down", 5632, 2048)), 1, 0.01, 20.0, "uniform"),
    Config(2, "llama-3b", 8192, _block(3200, 8640, 9600), 26, 0.005, 50.0, "p50-30-20"),
    Config(3, "llama-7b", 16384, _block(4096, 11008, 12288), 32, 0.01, 20.0, "all-fp4-then-fp8"),
    Config(4, "llama-70b-slice", 8192, _block(8192, 28672, 10240), 4, 0.005, 50.0, "fp4-80pct-flops"),
)


def linear_inputs(cfg: Config, layer: int, linear: int, M: int | None = None):
    """bf16 bit patterns (X[M,K], W[N,K], dY[M,N]) of one linear of a config."""
    lin = cfg.linears[linear]
    M = cfg.M if M is None else M
    x = make_x(rng_for(cfg.index, layer, linear, "X"), M, lin.K, cfg.outlier_frac, cfg.outlier_scale)
    w = make_w(rng_for(cfg.index, layer, linear, "W"), lin.N, lin.K)
    dy = make_dy(rng_for(cfg.index, layer, linear, "dY"), M, lin.N)
    return x, w, dy


def precision_tags(cfg: Config):
    """Precision tag per (layer, linear, gemm) with gemm in (fwd, dgrad, wgrad).

    Returns an int array [layers, n_linears, 3].  Rules:
      fixed-fp8-fp8-fp4 : fwd FP8, dgrad FP8, wgrad FP4
      uniform           : each tag uniform over {BF16, FP8, FP4}
      p50-30-20         : each GEMM independently FP4 w.p. .5, FP8 w.p. .3, BF16 w.p. .2
      all-fp4-then-fp8  : returns the all-FP4 table (the sweep repeats it with FP8)
      fp4-80pct-flops   : GEMMs visited in a seeded order get FP4 until at least 80 % of the
                          linear-layer FLOPs are FP4 (the paper's efficiency metric, Sec. 6.1),
                          the rest FP8
    """
    L, n = cfg.layers, len(cfg.linears)
    rng = rng_for(cfg.index, 0, 0, "tags")
    tags = np.empty((L, n, 3), dtype=np.int64)
    if cfg.tag_rule == "fixed-fp8-fp8-fp4":
        tags[...] = np.array([FMT_FP8, FMT_FP8, FMT_FP4])
    elif cfg.tag_rule == "uniform":
        tags[...] = rng.integers(0, 3, size=tags.shape)
    elif cfg.tag_rule == "p50-30-20":
        tags[...] = rng.choice([FMT_FP4, FMT_FP8, FMT_BF16], size=tags.shape, p=[0.5, 0.3, 0.2])
    elif cfg.tag_rule == "all-fp4-then-fp8":
        tags[...] = FMT_FP4
    elif cfg.tag_rule == "fp4-80pct-flops":
        flops = np.empty((L, n, 3), dtype=np.float64)
        for j, lin in enumerate(cfg.linears):
            flops[:, j, :] = 2.0 * cfg.M * lin.K * lin.N
        order = rng.permutation(flops.size)
        flat = np.full(flops.size, FMT_FP8, dtype=np.int64)
        total, acc = flops.sum(), 0.0
        for idx in order:
            if acc >= 0.8 * total:
                break
            flat[idx] = FMT_FP4
            acc += flops.reshape(-1)[idx]
        tags[...] = flat.reshape(tags.shape)
    else:
        raise ValueError(cfg.tag_rule)
    return tags
