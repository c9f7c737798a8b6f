"""Seeded synthetic inputs for the LowRA quantized-LoRA linear-layer hot path.

This module only *draws inputs*: weights, per-row precisions, activations, LoRA
factors and a stand-in codebook.  It holds none of the method's arithmetic (no
absmax, bucketing, packing, decoding, Lloyd-Max or GEMM) so that both the CPU
oracle's tests and the CUDA path's tests / benchmark can be fed identical bits
without sharing any code of the method itself.

Every value is a pure function of (seed, matrix id, stream, element index)
through a counter-based splitmix64 hash, so any sub-block can be regenerated
independently and in any order.

Shapes follow the linear layers of Llama-2-7B / 13B, which the paper fine-tunes
(Section 7.1 "Evaluation Setup"; 4096 / 11008 are the layer sizes named in Section 6.1
"Preprocessing for the Pipeline"); the real checkpoints are replaced by the recipe below.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import Dict, List, Tuple

import numpy as np

BASE_SEED = 20250208
_GOLDEN = np.uint64(0x9E3779B97F4A7C15)
_M1 = np.uint64(0xBF58476D1CE4E5B9)
_M2 = np.uint64(0x94D049BB133111EB)
_TWO_M53 = 2.0 ** -53

# stream ids (one independent sequence per purpose)
_S_NORMAL, _S_OUTLIER_PICK, _S_T0, _S_SIGMA, _S_PREC, _S_CB = 0, 1, 2, 7, 8, 9
_S_ACT, _S_LORA_A, _S_LORA_B, _S_GRAD = 16, 17, 18, 19


def _mix(z: np.ndarray) -> np.ndarray:
    z = (z ^ (z >> np.uint64(30))) * _M1
    z = (z ^ (z >> np.uint64(27))) * _M2
    return z ^ (z >> np.uint64(31))


def _key(seed: int, matrix_id: int, stream: int) -> np.uint64:
    with np.errstate(over="ignore"):
        k = np.uint64(seed & 0xFFFFFFFFFFFFFFFF)
        k = _mix(np.asarray(k + _GOLDEN * np.uint64(matrix_id + 1)))
        k = _mix(np.asarray(k + _GOLDEN * np.uint64(stream + 1)))
    return np.uint64(k)


def hash_u64(seed: int, matrix_id: int, stream: int, idx: np.ndarray) -> np.ndarray:
    """splitmix64 finaliser of key(seed, matrix, stream) + idx * golden."""
    idx = np.asarray(idx, dtype=np.uint64)
    with np.errstate(over="ignore"):
        return _mix(_key(seed, matrix_id, stream) + (idx + np.uint64(1)) * _GOLDEN)


def uniform01(seed: int, matrix_id: int, stream: int, idx: np.ndarray) -> np.ndarray:
    """Uniform in [0, 1), 53 bits."""
    return (hash_u64(seed, matrix_id, stream, idx) >> np.uint64(11)).astype(np.float64) * _TWO_M53


def normal(seed: int, matrix_id: int, stream: int, idx: np.ndarray) -> np.ndarray:
    """Standard normal by Box-Muller in fp64 from counters 2*idx and 2*idx+1."""
    idx = np.asarray(idx, dtype=np.uint64)
    h1 = hash_u64(seed, matrix_id, stream, idx * np.uint64(2))
    h2 = hash_u64(seed, matrix_id, stream, idx * np.uint64(2) + np.uint64(1))
    u1 = ((h1 >> np.uint64(11)).astype(np.float64) + 1.0) * _TWO_M53  # (0, 1]
    u2 = (h2 >> np.uint64(11)).astype(np.float64) * _TWO_M53
    return np.sqrt(-2.0 * np.log(u1)) * np.cos((2.0 * math.pi) * u2)


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even fp32 -> bf16, returned as uint16 bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    r = (u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) >> np.uint32(16)
    return r.astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.asarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


# ----------------------------------------------------------------------------
# weights
# ----------------------------------------------------------------------------
def weights(N: int, K: int, *, matrix_id: int = 0, seed: int = BASE_SEED,
            kind: str = "llama", row_chunk: int = 512) -> np.ndarray:
    """fp32 [N, K] weight matrix.

    kind="llama": row r has sigma_r log-uniform in [0.005, 0.05]; entry = sigma_r * Z;
        independently with probability 1e-3 an entry is replaced by
        10 * sigma_r * t4, t4 Student-t with 4 degrees of freedom.
    kind="tiny":  every entry 0.02 * Z, no outliers.
    """
    out = np.empty((N, K), dtype=np.float32)
    if kind == "tiny":
        sig = np.full(N, 0.02)
    else:
        u = uniform01(seed, matrix_id, _S_SIGMA, np.arange(N))
        sig = np.exp(math.log(0.005) + u * (math.log(0.05) - math.log(0.005)))
    for r0 in range(0, N, row_chunk):
        r1 = min(N, r0 + row_chunk)
        idx = (np.arange(r0, r1, dtype=np.uint64)[:, None] * np.uint64(K)
               + np.arange(K, dtype=np.uint64)[None, :])
        z = normal(seed, matrix_id, _S_NORMAL, idx)
        blk = z * sig[r0:r1, None]
        if kind != "tiny":
            pick = uniform01(seed, matrix_id, _S_OUTLIER_PICK, idx) < 1e-3
            if pick.any():
                sel = idx[pick]
                z0 = normal(seed, matrix_id, _S_T0, sel)
                chi = np.zeros_like(z0)
                for j in range(1, 5):
                    zj = normal(seed, matrix_id, _S_T0 + j, sel)
                    chi += zj * zj
                t4 = z0 / np.sqrt(chi / 4.0)
                rows = np.nonzero(pick)[0]
                blk[pick] = 10.0 * sig[r0 + rows] * t4
        out[r0:r1] = blk.astype(np.float32)
    return out


def precisions(N: int, mix: Dict[int, float], *, matrix_id: int = 0,
               seed: int = BASE_SEED) -> np.ndarray:
    """uint8 [N] with exact class counts round(f_b * N); the largest class absorbs the
    remainder; positions by a seeded shuffle."""
    bits = sorted(mix)
    counts = {b: int(round(mix[b] * N)) for b in bits}
    big = max(bits, key=lambda b: (mix[b], b))
    counts[big] += N - sum(counts.values())
    assert all(c >= 0 for c in counts.values())
    labels = np.concatenate([np.full(counts[b], b, dtype=np.uint8) for b in bits])
    order = np.argsort(hash_u64(seed, matrix_id, _S_PREC, np.arange(N)), kind="stable")
    out = np.empty(N, dtype=np.uint8)
    out[order] = labels
    return out


def bf16_normal(shape: Tuple[int, int], scale: float, *, stream: int, matrix_id: int = 0,
                seed: int = BASE_SEED) -> np.ndarray:
    """bf16 bit patterns (uint16) of scale * Z, shape [rows, cols]."""
    rows, cols = shape
    out = np.empty((rows, cols), dtype=np.uint16)
    step = max(1, (1 << 22) // max(cols, 1))
    for r0 in range(0, rows, step):
        r1 = min(rows, r0 + step)
        idx = (np.arange(r0, r1, dtype=np.uint64)[:, None] * np.uint64(cols)
               + np.arange(cols, dtype=np.uint64)[None, :])
        out[r0:r1] = f32_to_bf16_bits((normal(seed, matrix_id, stream, idx) * scale).astype(np.float32))
    return out


def activations(M: int, K: int, *, matrix_id: int = 0, seed: int = BASE_SEED) -> np.ndarray:
    return bf16_normal((M, K), 1.0, stream=_S_ACT, matrix_id=matrix_id, seed=seed)


def out_grads(M: int, N: int, *, matrix_id: int = 0, seed: int = BASE_SEED) -> np.ndarray:
    return bf16_normal((M, N), 1.0, stream=_S_GRAD, matrix_id=matrix_id, seed=seed)


def lora_factors(K: int, N: int, r: int, *, matrix_id: int = 0, seed: int = BASE_SEED):
    """A bf16 [K, r], B bf16 [r, N], both 0.01 * Z."""
    A = bf16_normal((K, r), 0.01, stream=_S_LORA_A, matrix_id=matrix_id, seed=seed)
    B = bf16_normal((r, N), 0.01, stream=_S_LORA_B, matrix_id=matrix_id, seed=seed)
    return A, B


# ----------------------------------------------------------------------------
# stand-in codebooks (for runs that may not execute the Lloyd-Max learner)
# ----------------------------------------------------------------------------
# Initial levels printed in the paper's Appendix F listing (4-, 2- and 1-bit).
_LEVELS = {
    4: [-1.0, -0.6961928, -0.5250731, -0.3949175, -0.28444138, -0.18477343, -0.09105, 0.0,
        0.0795803, 0.1609302, 0.2461123, 0.33791524, 0.44070983, 0.562617, 0.72295684, 1.0],
    2: [-1.0, 0.0, 0.3379, 1.0],
    1: [-1.0, 1.0],
}


# Initial thresholds printed in the same listing (it prints none for 4 bits).
_THRESHOLDS = {2: [-0.5, 0.16895762, 0.66895762], 1: [0.0]}


def initial_codebooks():
    """Starting tables of a codebook learner, as inputs: the levels and thresholds printed in the paper's
    Appendix F listing; for 4 bits, where it prints no thresholds, the points halfway between neighbouring
    levels.  -> (levels, thresholds), float64 [3, 16] each, rows = 1-, 2-, 4-bit tables, unused entries 0."""
    y0 = np.zeros((3, 16), dtype=np.float64)
    t0 = np.zeros((3, 16), dtype=np.float64)
    for c, b in enumerate((1, 2, 4)):
        lv = np.asarray(_LEVELS[b], dtype=np.float64)
        y0[c, :lv.size] = lv
        th = np.asarray(_THRESHOLDS[b], dtype=np.float64) if b in _THRESHOLDS else 0.5 * (lv[:-1] + lv[1:])
        t0[c, :th.size] = th
    return y0, t0


def standin_codebooks(precs: np.ndarray, *, matrix_id: int = 0, seed: int = BASE_SEED):
    """Per-row tables without running the learner: the listed initial levels, each moved by
    a seeded amount of up to +-20 % of the gap to its neighbour (so rows differ and levels stay
    sorted), thresholds halfway between neighbouring levels.

    Returns maps fp32 [N, 16] (unused = 0) and thresholds fp32 [N, 16] (unused = +inf).
    """
    N = precs.shape[0]
    maps = np.zeros((N, 16), dtype=np.float32)
    thr = np.full((N, 16), np.inf, dtype=np.float32)
    u = uniform01(seed, matrix_id, _S_CB, np.arange(N * 16)).reshape(N, 16)
    for b in (1, 2, 4):
        rows = np.nonzero(precs == b)[0]
        if rows.size == 0:
            continue
        lv = np.asarray(_LEVELS[b], dtype=np.float64)
        L = lv.size
        gap_lo = np.diff(lv, prepend=lv[0] - (lv[1] - lv[0]))
        gap_hi = np.diff(lv, append=lv[-1] + (lv[-1] - lv[-2]))
        gap = np.minimum(gap_lo, gap_hi)
        m = lv[None, :] + (u[rows, :L] - 0.5) * 0.4 * gap[None, :]
        m32 = m.astype(np.float32)
        maps[rows[:, None], np.arange(L)[None, :]] = m32
        mid = ((m32[:, :-1].astype(np.float64) + m32[:, 1:].astype(np.float64)) * 0.5).astype(np.float32)
        thr[rows[:, None], np.arange(L - 1)[None, :]] = mid
    return maps, thr


# ----------------------------------------------------------------------------
# workload configurations
# ----------------------------------------------------------------------------
@dataclass(frozen=True)
class Matrix:
    name: str
    N: int       # out_features (rows, output channels)
    K: int       # in_features
    matrix_id: int


@dataclass(frozen=True)
class Config:
    name: str
    matrices: Tuple[Matrix, ...]
    mix: Dict[int, float]
    tokens: Tuple[int, ...]
    rank: int
    s: float
    weight_kind: str = "llama"
    lloyd_iters: int = 10
    ops: Tuple[str, ...] = ("encode", "decode", "forward", "backward")


def _layer(h: int, f: int, layer: int = 0) -> Tuple[Matrix, ...]:
    names = (("q_proj", h, h), ("k_proj", h, h), ("v_proj", h, h), ("o_proj", h, h),
             ("gate_proj", f, h), ("up_proj", f, h), ("down_proj", h, f))
    return tuple(Matrix(n, N, K, layer * 7 + i) for i, (n, N, K) in enumerate(names))


def config(i: int) -> Config:
    """The five workload configurations (1-based, as numbered in the benchmark spec)."""
    if i == 1:
        return Config("tiny-512", (Matrix("w", 512, 512, 0),), {1: 0.5, 2: 0.5}, (16,), 16, 2.0,
                      weight_kind="tiny")
    if i == 2:
        return Config("q_proj-4096", (Matrix("q_proj", 4096, 4096, 0),), {1: 0.3, 2: 0.5, 4: 0.2},
                      (2048,), 64, 2.0)
    if i == 3:
        return Config("llama7b-layer", _layer(4096, 11008), {1: 0.60, 2: 0.35, 4: 0.05},
                      (4096,), 64, 2.0)
    if i == 4:
        return Config("llama13b-layer", _layer(5120, 13824), {1: 0.85, 2: 0.15}, (4096,), 64, 2.0)
    if i == 5:
        mats: List[Matrix] = []
        for layer in range(32):
            mats.extend(_layer(4096, 11008, layer))
        return Config("llama7b-model", tuple(mats), {2: 0.75, 4: 0.25}, (1024, 4096, 8192), 64, 2.0,
                      ops=("encode", "decode", "forward"))
    raise ValueError(f"no config {i}")


def avg_bits(mix: Dict[int, float]) -> float:
    return sum(b * f for b, f in mix.items())
