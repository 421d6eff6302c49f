"""Seeded synthetic inputs for the tile-hybrid linear layer.

This module only *draws* inputs (weights, activations, tile flags, per-matrix
2:4-tile fractions) and names the workloads.  It contains none of the method's
arithmetic (no masking, packing or matmul), so both the CPU oracle's tests and
the CUDA path's tests can feed from it without sharing any computation.

Everything is drawn from numpy's counter-based Philox generator keyed by
``(seed, stream)``, where ``stream`` is a tuple of small integers / strings
naming what is drawn (config, layer, matrix, role).  Values are rounded once to
bf16 (round-to-nearest-even) and returned as ``uint16`` bit patterns: those
bit patterns *are* the inputs.

The workloads stand in for the LLaMA-2 7B / 13B checkpoints the paper
evaluates (Appendix A, throughput tables): same linear-layer shapes
(q, k, v, o, gate, up, down), Gaussian weights of initialiser width
(std 0.02), unit-Gaussian activations, independent Bernoulli tile flags.
"""
from __future__ import annotations

import numpy as np

MASTER_SEED = 23410
TILE = 128

ROLE_W, ROLE_X, ROLE_FLAGS, ROLE_FRACTION = 1, 2, 3, 4


def _stream_key(seed: int, stream) -> list[int]:
    """Stable 2x64-bit Philox key from a seed and a tuple naming the stream (FNV-1a)."""
    h = 0xCBF29CE484222325
    for item in stream:
        for b in str(item).encode() + b"\x1f":
            h ^= b
            h = (h * 0x100000001B3) & 0xFFFFFFFFFFFFFFFF
    return [seed & 0xFFFFFFFFFFFFFFFF, h]


def generator(seed: int, *stream) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=_stream_key(seed, stream)))


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """float32 -> bf16 bit patterns (uint16), round-to-nearest-even; finite inputs."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    rounded = u + (np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1)))
    return (rounded >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def normal_bf16(shape, std: float, seed: int, *stream) -> np.ndarray:
    """N(0, std^2) samples rounded to bf16, as uint16 bit patterns of the given shape."""
    g = generator(seed, *stream)
    x = g.standard_normal(int(np.prod(shape)), dtype=np.float32)
    if std != 1.0:
        x *= np.float32(std)
    return f32_to_bf16_bits(x).reshape(shape)


def weight(N: int, K: int, seed: int = MASTER_SEED, *stream) -> np.ndarray:
    """W [N x K] ~ N(0, 0.02^2), bf16 bits."""
    return normal_bf16((N, K), 0.02, seed, ROLE_W, *stream)


def activation(M: int, K: int, seed: int = MASTER_SEED, *stream) -> np.ndarray:
    """X [M x K] ~ N(0, 1), bf16 bits."""
    return normal_bf16((M, K), 1.0, seed, ROLE_X, *stream)


def tile_flags(N: int, K: int, p_sparse: float, seed: int = MASTER_SEED, *stream,
               tile_n: int = TILE, tile_k: int = TILE) -> np.ndarray:
    """Per-tile kind flags [N/tile_n x K/tile_k] uint8: 1 = stored 2:4 with probability p_sparse, 0 = dense.

    p_sparse = 0 and 1 are exact (all dense / all 2:4).
    """
    tn, tk = N // tile_n, K // tile_k
    if p_sparse <= 0.0:
        return np.zeros((tn, tk), np.uint8)
    if p_sparse >= 1.0:
        return np.ones((tn, tk), np.uint8)
    g = generator(seed, ROLE_FLAGS, *stream)
    return (g.random(tn * tk) < p_sparse).astype(np.uint8).reshape(tn, tk)


def fraction(lo: float, hi: float, seed: int = MASTER_SEED, *stream) -> float:
    """One per-matrix 2:4-tile fraction drawn uniformly from [lo, hi]."""
    g = generator(seed, ROLE_FRACTION, *stream)
    return float(lo + (hi - lo) * g.random())


# --------------------------------------------------------------------------------------
# Workloads (shapes are [N out-features, K in-features]).

LLAMA2_7B_SHAPES = {
    "attn_qkvo": (4096, 4096),
    "mlp_gate_up": (11008, 4096),
    "mlp_down": (4096, 11008),
}
LLAMA2_13B_SHAPES = {
    "attn_qkvo": (5120, 5120),
    "mlp_gate_up": (13824, 5120),
    "mlp_down": (5120, 13824),
}
# one transformer block = q, k, v, o, gate, up, down
LLAMA2_7B_BLOCK = [("q", 4096, 4096), ("k", 4096, 4096), ("v", 4096, 4096), ("o", 4096, 4096),
                   ("gate", 11008, 4096), ("up", 11008, 4096), ("down", 4096, 11008)]


def single_gemm_case():
    """Small case: X [16 x 1024], W [1024 x 1024], Bernoulli(0.5) tiles."""
    return dict(name="single", N=1024, K=1024, M=16, p=0.5, stream=("single",))


def decode_cases():
    """7B decode linears: 3 shapes x M in {1,16} x p in {0, .35, .7, 1}."""
    out = []
    for sname, (N, K) in LLAMA2_7B_SHAPES.items():
        for p in (0.0, 0.35, 0.7, 1.0):
            for M in (1, 16):
                out.append(dict(name=f"7b.{sname}.p{p}.M{M}", N=N, K=K, M=M, p=p,
                                stream=("decode", sname, p)))
    return out


def decode_q4_cases():
    """The decode linears with every tile stored with 4-bit values (tile kinds 2 and 3): the same shapes, 2:4-tile
    fractions and seeded streams as decode_cases(), so the two workloads differ only in the payload format."""
    return [dict(c, name=c["name"] + ".q4", q4=True) for c in decode_cases()]


def prefill_cases():
    """7B prefill linears: 3 shapes x M in {512,2048,4096} x p in {0, .5, 1}."""
    out = []
    for sname, (N, K) in LLAMA2_7B_SHAPES.items():
        for p in (0.0, 0.5, 1.0):
            for M in (512, 2048, 4096):
                out.append(dict(name=f"7b.{sname}.p{p}.M{M}", N=N, K=K, M=M, p=p,
                                stream=("prefill", sname, p)))
    return out


def llama13b_cases(seed: int = MASTER_SEED):
    """13B linears: 3 shapes x M in {1,8,64,512,4096}, per-matrix p ~ U[0.2, 1.0]."""
    out = []
    for sname, (N, K) in LLAMA2_13B_SHAPES.items():
        p = fraction(0.2, 1.0, seed, "13b", sname)
        for M in (1, 8, 64, 512, 4096):
            out.append(dict(name=f"13b.{sname}.p{p:.3f}.M{M}", N=N, K=K, M=M, p=p,
                            stream=("13b", sname)))
    return out


def stack_cases(seed: int = MASTER_SEED, n_blocks: int = 32):
    """Full 7B-shaped linear stack: n_blocks x 7 matrices, per-matrix p ~ U[0,1]."""
    out = []
    for b in range(n_blocks):
        for role, N, K in LLAMA2_7B_BLOCK:
            p = fraction(0.0, 1.0, seed, "stack", b, role)
            out.append(dict(name=f"stack.{b}.{role}", N=N, K=K, p=p, stream=("stack", b, role)))
    return out


def stack_fused_cases(seed: int = MASTER_SEED, n_blocks: int = 32):
    """The same stack with the linears that share an input stored as one matrix each: q/k/v stacked along N
    (12288 x 4096) and gate/up stacked (22016 x 4096); 4 GEMMs per block instead of 7.  Every part keeps
    the 2:4-tile fraction and the flag stream of its own matrix in ``stack_cases``."""
    groups = [("qkv", ("q", "k", "v")), ("o", ("o",)), ("gate_up", ("gate", "up")), ("down", ("down",))]
    shapes = {role: (N, K) for role, N, K in LLAMA2_7B_BLOCK}
    out = []
    for b in range(n_blocks):
        for name, roles in groups:
            K = shapes[roles[0]][1]
            parts = [dict(N=shapes[r][0], p=fraction(0.0, 1.0, seed, "stack", b, r), stream=("stack", b, r)) for r in roles]
            N = sum(q["N"] for q in parts)
            p = sum(q["p"] * q["N"] for q in parts) / N
            out.append(dict(name=f"stack.{b}.{name}", N=N, K=K, p=p, stream=("stack", b, name), parts=parts))
    return out


def case_flags(case: dict, seed: int = MASTER_SEED) -> np.ndarray:
    """Tile flags of a case; a case made of stacked matrices concatenates its parts' flags along N."""
    if "parts" in case:
        return np.concatenate([tile_flags(q["N"], case["K"], q["p"], seed, *q["stream"]) for q in case["parts"]], axis=0)
    flags = tile_flags(case["N"], case["K"], case["p"], seed, *case["stream"])
    return flags | 2 if case.get("q4") else flags          # bit 1: the tile's stored values are 4-bit codes


def make_case_inputs(case: dict, seed: int = MASTER_SEED, M: int | None = None):
    """(W bits [N x K], flags [TN x TK], X bits [M x K]) for a case dict from the lists above."""
    N, K = case["N"], case["K"]
    M = case.get("M") if M is None else M
    W = weight(N, K, seed, *case["stream"])
    flags = case_flags(case, seed)
    X = activation(M, K, seed, *case["stream"], M)
    return W, flags, X


# ---------------------------------------------------------------------------------------------
# Mask-learning inputs (logits of Algorithm 1).  Draws only: no softmax, no masks here.

ROLE_P_TILE, ROLE_P_24 = 5, 6
LOGIT_STD = 0.014                # "Logits Init N(0, 0.014)" of the hyper-parameter table
PRIOR_STRENGTH = 3.0             # "Prior(Strength) SparseGPT(3)"
# (tau, kappa) at the start and at the end of the schedules of the hyper-parameter table
SCHEDULE_START, SCHEDULE_END = (2.0, 25.0), (0.05, 350.0)


def tile_logits(TN: int, TK: int, p_dense: float, seed: int, *stream) -> np.ndarray:
    """P_tile [TN x TK] float32: N(0, LOGIT_STD^2) plus a prior of +-PRIOR_STRENGTH, positive
    (dense) with probability ``p_dense`` -- the shape of the paper's prior-initialised logits."""
    g = generator(seed, ROLE_P_TILE, *stream)
    base = g.standard_normal(TN * TK, dtype=np.float32) * np.float32(LOGIT_STD)
    sign = np.where(g.random(TN * TK) < p_dense, np.float32(1), np.float32(-1))
    return (base + np.float32(PRIOR_STRENGTH) * sign).reshape(TN, TK).astype(np.float32)


def pattern_logits(N: int, K: int, seed: int, *stream, std: float = LOGIT_STD) -> np.ndarray:
    """P_2:4 [6 x N*K/4] float32 ~ N(0, std^2); row c = candidate c, column = n*(K/4) + g."""
    g = generator(seed, ROLE_P_24, *stream)
    return (g.standard_normal(6 * (N * K // 4), dtype=np.float32) * np.float32(std)).reshape(6, N * K // 4)
