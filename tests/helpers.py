"""Shared builders for the parity tests: one seeded problem, the oracle's answers, device copies."""
from __future__ import annotations

from dataclasses import dataclass
from typing import Dict, Optional

import numpy as np

import oracle
import synth_inputs as si


@dataclass
class Case:
    N: int
    K: int
    W: np.ndarray            # fp32 [N, K]
    precs: np.ndarray        # uint8 [N]
    maps: np.ndarray         # fp32 [N, 16]
    thr: np.ndarray          # fp32 [N, 16]
    packed: np.ndarray       # oracle's packed bytes
    absmax: np.ndarray       # oracle's absmax, stored order
    W_hat: np.ndarray        # oracle's decode, bf16 bits [N, K]


def make_case(N: int, K: int, mix: Dict[int, float], *, matrix_id: int = 0, kind: str = "llama",
              lloyd_iters: int = 10, precs: Optional[np.ndarray] = None) -> Case:
    W = si.weights(N, K, matrix_id=matrix_id, kind=kind)
    if precs is None:
        precs = si.precisions(N, mix, matrix_id=matrix_id)
    maps, thr = oracle.lloyd_max(W, precs, T=lloyd_iters)
    packed, a = oracle.encode(W, precs, thr)
    W_hat = oracle.decode(packed, a, maps, precs, K)
    return Case(N, K, W, precs, maps, thr, packed, a, W_hat)


def gemm_errors(got: np.ndarray, ref: np.ndarray):
    """(max |got - ref| / max |ref|,  ||got - ref||_F / ||ref||_F)."""
    d = got.astype(np.float64) - ref
    return float(np.abs(d).max() / np.abs(ref).max()), float(np.linalg.norm(d) / np.linalg.norm(ref))


MAX_TOL = 1e-2    # max|Y - Y_ref| <= 1e-2 * max|Y_ref|
FRO_TOL = 5e-3    # ||Y - Y_ref||_F <= 5e-3 * ||Y_ref||_F
