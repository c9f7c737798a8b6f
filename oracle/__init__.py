"""CPU oracle for the LowRA quantized-LoRA linear-layer hot path (Python face).

TEST INFRASTRUCTURE ONLY: imported by tests, by the smoke check and by the benchmark's CPU
baseline leg; the product never routes through it.  The encoding steps (absmax, normalise,
bucket, pack, decode, Lloyd-Max) are scalar C in ``lowra_oracle.c``; the two LoRA products are
the definition written out with numpy float64 matmuls (no blocking, no intermediate rounding):

    Y  = X . W_hat^T + s * ((X . A) . B)                 forward
    dX = dY . W_hat  + s * ((dY . B^T) . A^T)            input gradient

with W_hat the decoded bf16 weights (Appendix A.2 of the paper) and all operands promoted
from bf16 to float64.  The base weights are frozen and only the low-rank factors are trained
(Section 3), so dX is the only gradient that flows through the quantised weight.

Pins: tests/test_oracle_*.py (printed constants, brute force, closed forms, invariants).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "lowra_oracle.c")
_LIB = os.path.join(_HERE, "liblowra_oracle.so")
_lib = None

TABLE_STRIDE = 16


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (no CUDA involved)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-fopenmp", "-ffp-contract=off", "-fno-fast-math", "-shared", "-fPIC",
               "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        L = ctypes.CDLL(_LIB)
        i64, vp, ci = ctypes.c_int64, ctypes.c_void_p, ctypes.c_int
        L.oracle_num_threads.restype = ci
        L.oracle_set_threads.argtypes = [ci]
        L.oracle_f32_to_bf16.argtypes = [vp, vp, i64]
        L.oracle_absmax.argtypes = [vp, i64, i64, i64, vp]
        L.oracle_normalise.argtypes = [vp, i64, i64, i64, vp]
        L.oracle_plan.argtypes = [vp, i64, i64, vp, vp, vp, vp, vp]
        L.oracle_plan.restype = ci
        L.oracle_encode.argtypes = [vp, i64, i64, i64, vp, vp, vp, vp, vp]
        L.oracle_encode.restype = ci
        L.oracle_decode.argtypes = [vp, vp, vp, vp, i64, i64, i64, vp]
        L.oracle_decode.restype = ci
        L.oracle_initial_tables.argtypes = [ci, vp, vp]
        L.oracle_lloyd_max_row.argtypes = [vp, vp, i64, ci, ci, vp, vp, vp]
        L.oracle_lloyd_max.argtypes = [vp, i64, i64, i64, vp, ci, vp, vp, vp]
        L.oracle_lloyd_max.restype = ci
        L.oracle_matmul_naive.argtypes = [vp, vp, vp, i64, i64, i64]
        _lib = L
    return _lib


def _p(a: np.ndarray):
    return a.ctypes.data_as(ctypes.c_void_p)


def _c(a, dtype) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=dtype)


def num_threads() -> int:
    return int(_load().oracle_num_threads())


def set_threads(n: int) -> None:
    _load().oracle_set_threads(int(n))


# ---------------------------------------------------------------------------------------------
def f32_to_bf16(x: np.ndarray) -> np.ndarray:
    """fp32 -> bf16 bit patterns (uint16), round to nearest even."""
    x = _c(x, np.float32)
    out = np.empty(x.shape, dtype=np.uint16)
    _load().oracle_f32_to_bf16(_p(x), _p(out), x.size)
    return out


def bf16_to_f64(b: np.ndarray) -> np.ndarray:
    """bf16 bit patterns -> float64 (exact)."""
    return (np.asarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)


def absmax(W: np.ndarray, G: int = 64) -> np.ndarray:
    """Block maximum magnitude, natural row order, [N, K/G] fp32."""
    W = _c(W, np.float32)
    N, K = W.shape
    a = np.empty((N, K // G), dtype=np.float32)
    _load().oracle_absmax(_p(W), N, K, G, _p(a))
    return a


def normalise(W: np.ndarray, G: int = 64) -> np.ndarray:
    """x * fl(1/absmax) in fp32 (0 where the block is all zero), [N, K]."""
    W = _c(W, np.float32)
    N, K = W.shape
    out = np.empty((N, K), dtype=np.float32)
    _load().oracle_normalise(_p(W), N, K, G, _p(out))
    return out


def plan(precs: np.ndarray, K: int) -> dict:
    """Precision-grouped storage order: classes 1, 2, 4 bits, stable inside a class."""
    precs = _c(precs, np.uint8)
    N = precs.shape[0]
    perm = np.empty(N, dtype=np.int32)
    inv = np.empty(N, dtype=np.int32)
    counts = np.zeros(3, dtype=np.int32)
    seg = np.zeros(3, dtype=np.uint64)
    total = np.zeros(1, dtype=np.uint64)
    rc = _load().oracle_plan(_p(precs), N, K, _p(perm), _p(inv), _p(counts), _p(seg), _p(total))
    if rc != 0:
        raise ValueError("precisions must be 1, 2 or 4")
    return dict(perm=perm, inv_perm=inv, counts=counts, seg_off=seg, packed_bytes=int(total[0]))


def encode(W: np.ndarray, precs: np.ndarray, thresholds: np.ndarray, G: int = 64,
           return_codes: bool = False):
    """-> packed uint8 [packed_bytes], absmax fp32 [N, K/G] in stored row order (, codes [N,K])."""
    W = _c(W, np.float32)
    precs = _c(precs, np.uint8)
    thresholds = _c(thresholds, np.float32)
    N, K = W.shape
    assert thresholds.shape == (N, TABLE_STRIDE)
    pl = plan(precs, K)
    packed = np.empty(pl["packed_bytes"], dtype=np.uint8)
    a = np.empty((N, K // G), dtype=np.float32)
    codes = np.empty((N, K), dtype=np.uint8) if return_codes else None
    rc = _load().oracle_encode(_p(W), N, K, G, _p(precs), _p(thresholds), _p(packed), _p(a),
                               _p(codes) if return_codes else None)
    if rc != 0:
        raise ValueError(f"oracle_encode failed ({rc})")
    return (packed, a, codes) if return_codes else (packed, a)


def decode(packed: np.ndarray, absmax_stored: np.ndarray, maps: np.ndarray, precs: np.ndarray,
           K: int, G: int = 64) -> np.ndarray:
    """-> bf16 bit patterns uint16 [N, K], natural row order."""
    packed = _c(packed, np.uint8)
    a = _c(absmax_stored, np.float32)
    maps = _c(maps, np.float32)
    precs = _c(precs, np.uint8)
    N = precs.shape[0]
    assert maps.shape == (N, TABLE_STRIDE) and a.shape == (N, K // G)
    out = np.empty((N, K), dtype=np.uint16)
    rc = _load().oracle_decode(_p(packed), _p(a), _p(maps), _p(precs), N, K, G, _p(out))
    if rc != 0:
        raise ValueError(f"oracle_decode failed ({rc})")
    return out


def natural_layout(codes: np.ndarray, precs: np.ndarray):
    """The paper's own buffer layout (Appendix A.2: a thread finds its offset into the quantised buffer from the
    channels' bit precisions): rows in their ORIGINAL order, row r at byte offset sum_{i<r} K*b_i/8, codes packed
    LSB-first at the row's precision.  codes uint8 [N,K] -> (buffer uint8, offsets uint64 [N+1]).
    Written with plain shifts on the code matrix, independent of the C packer of the grouped layout."""
    codes = np.asarray(codes, dtype=np.uint8)
    precs = np.asarray(precs, dtype=np.int64)
    N, K = codes.shape
    row_bytes = K * precs // 8
    offsets = np.zeros(N + 1, dtype=np.uint64)
    offsets[1:] = np.cumsum(row_bytes)
    buf = np.zeros(int(offsets[-1]), dtype=np.uint8)
    for r in range(N):
        b = int(precs[r])
        per = 8 // b                                   # codes per byte
        c = codes[r].reshape(K // per, per).astype(np.uint32)
        byte = np.zeros(K // per, dtype=np.uint32)
        for j in range(per):
            byte |= (c[:, j] & ((1 << b) - 1)) << (b * j)
        buf[int(offsets[r]):int(offsets[r + 1])] = byte.astype(np.uint8)
    return buf, offsets


def quant_error(W: np.ndarray, precs: np.ndarray, maps: np.ndarray, thresholds: np.ndarray, G: int = 64):
    """Summed square error per output channel, SSE_i = sum_k (W[i,k] - W_hat[i,k])^2 (the precision
    assigner's objective, Section 5 and its footnote; the per-channel errors under 1, 2 and 4 bits are
    what Section 5.1 clusters), and the residual W - W_hat that an iterative low-rank initialiser
    factorises next (Appendix: LoftQ quantises, then decomposes what is left).
    W_hat is what decode(encode(W)) gives: bf16(level * absmax) (Appendix A.1, A.2).
    -> sse float64 [N] (exact differences, squared and summed in float64),
       residual float32 [N, K] (one fp32 subtraction per element)."""
    W = _c(W, np.float32)
    N, K = W.shape
    packed, a = encode(W, precs, thresholds, G)
    w_hat = bf16_to_f64(decode(packed, a, maps, precs, K, G))
    d = W.astype(np.float64) - w_hat
    sse = np.array([float(np.sum(d[i] * d[i])) for i in range(N)], dtype=np.float64)
    residual = W - w_hat.astype(np.float32)          # w_hat is exact in fp32; one rounding, in the subtraction
    return sse, residual


def initial_tables(b: int) -> Tuple[np.ndarray, np.ndarray]:
    """Initial levels [2^b] and thresholds [2^b - 1] (float64) of the learner."""
    maps = np.zeros(1 << b, dtype=np.float64)
    thr = np.zeros((1 << b) - 1, dtype=np.float64)
    _load().oracle_initial_tables(b, _p(maps), _p(thr))
    return maps, thr


def lloyd_max_row(x: np.ndarray, w: np.ndarray, b: int, T: int,
                  maps0: Optional[np.ndarray] = None, thr0: Optional[np.ndarray] = None):
    """Weighted Lloyd-Max on one data vector. -> (levels, thresholds, trace[2T])."""
    x = _c(x, np.float64)
    w = _c(w, np.float64)
    y, t = initial_tables(b)
    if maps0 is not None:
        y = _c(maps0, np.float64).copy()
    if thr0 is not None:
        t = _c(thr0, np.float64).copy()
    trace = np.zeros(2 * T, dtype=np.float64)
    _load().oracle_lloyd_max_row(_p(x), _p(w), x.size, b, T, _p(y), _p(t), _p(trace))
    return y, t, trace


def lloyd_max(W: np.ndarray, precs: np.ndarray, T: int = 10, G: int = 64, return_trace: bool = False):
    """Per-row codebooks at the row's assigned precision. -> maps [N,16], thresholds [N,16] fp32."""
    W = _c(W, np.float32)
    precs = _c(precs, np.uint8)
    N, K = W.shape
    maps = np.empty((N, TABLE_STRIDE), dtype=np.float32)
    thr = np.empty((N, TABLE_STRIDE), dtype=np.float32)
    trace = np.zeros((N, 2 * T), dtype=np.float64) if return_trace else None
    rc = _load().oracle_lloyd_max(_p(W), N, K, G, _p(precs), T, _p(maps), _p(thr),
                                  _p(trace) if return_trace else None)
    if rc != 0:
        raise ValueError(f"oracle_lloyd_max failed ({rc})")
    return (maps, thr, trace) if return_trace else (maps, thr)


def matmul_naive(A: np.ndarray, B: np.ndarray) -> np.ndarray:
    """Triple loop in long double; small sizes only."""
    A = _c(A, np.float64)
    B = _c(B, np.float64)
    M, Kd = A.shape
    Kd2, Nn = B.shape
    assert Kd == Kd2
    C = np.empty((M, Nn), dtype=np.float64)
    _load().oracle_matmul_naive(_p(A), _p(B), _p(C), M, Kd, Nn)
    return C


# ---------------------------------------------------------------------------------------------
def lora_forward(W_hat_bf16: np.ndarray, X_bf16: np.ndarray, A_bf16: np.ndarray, B_bf16: np.ndarray,
                 s: float) -> np.ndarray:
    """Y = X . W_hat^T + s * ((X . A) . B), float64 [M, N]."""
    W = bf16_to_f64(W_hat_bf16)   # [N, K]
    X = bf16_to_f64(X_bf16)       # [M, K]
    A = bf16_to_f64(A_bf16)       # [K, r]
    B = bf16_to_f64(B_bf16)       # [r, N]
    return X @ W.T + float(s) * ((X @ A) @ B)


def lora_backward_input(W_hat_bf16: np.ndarray, dY_bf16: np.ndarray, A_bf16: np.ndarray,
                        B_bf16: np.ndarray, s: float) -> np.ndarray:
    """dX = dY . W_hat + s * ((dY . B^T) . A^T), float64 [M, K]."""
    W = bf16_to_f64(W_hat_bf16)   # [N, K]
    dY = bf16_to_f64(dY_bf16)     # [M, N]
    A = bf16_to_f64(A_bf16)
    B = bf16_to_f64(B_bf16)
    return dY @ W + float(s) * ((dY @ B.T) @ A.T)


def lora_backward_adapters(X_bf16: np.ndarray, dY_bf16: np.ndarray, A_bf16: np.ndarray, B_bf16: np.ndarray,
                           s: float):
    """Gradients of the trainable low-rank factors (Section 3: only they are trained) of
    Y = X . W_hat^T + s * (X . A) . B for the output gradient dY:
        dA = s * X^T . (dY . B^T)  [K, r],      dB = s * (X . A)^T . dY  [r, N],   float64."""
    X = bf16_to_f64(X_bf16)       # [M, K]
    dY = bf16_to_f64(dY_bf16)     # [M, N]
    A = bf16_to_f64(A_bf16)       # [K, r]
    B = bf16_to_f64(B_bf16)       # [r, N]
    return float(s) * (X.T @ (dY @ B.T)), float(s) * ((X @ A).T @ dY)
