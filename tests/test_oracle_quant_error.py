"""Pins of the oracle's per-channel quantisation error (SSE) and residual, against things that do not
come from the oracle: closed forms for special codebooks, a nearest-level brute force, exact scaling."""
import numpy as np
import pytest

import oracle

T = oracle.TABLE_STRIDE


def tables(N, levels):
    """Row tables [N,16] for one sorted level set: thresholds are the midpoints."""
    levels = np.asarray(levels, dtype=np.float64)
    maps = np.zeros((N, T), dtype=np.float32)
    thr = np.zeros((N, T), dtype=np.float32)
    maps[:, :levels.size] = levels
    thr[:, :levels.size - 1] = 0.5 * (levels[:-1] + levels[1:])
    return maps, thr


def blocks_with_power_of_two_absmax(rng, N, K, G=64):
    """fp32 matrix whose 64-blocks have maximum magnitude exactly 2^e: normalisation is then exact."""
    W = rng.uniform(-1.0, 1.0, size=(N, K)).astype(np.float32)
    W = W.reshape(N, K // G, G)
    W *= 0.999
    e = rng.integers(-6, 3, size=(N, K // G))
    pos = rng.integers(0, G, size=(N, K // G))
    sign = rng.choice([-1.0, 1.0], size=(N, K // G))
    for i in range(N):
        for j in range(K // G):
            W[i, j, pos[i, j]] = sign[i, j]
    W = (W * np.exp2(e)[:, :, None]).astype(np.float32)
    return W.reshape(N, K), np.exp2(e).astype(np.float64)


def test_one_bit_sign_codebook_closed_form():
    """Levels -1, +1 and threshold 0: every value becomes +-absmax of its block, so
    SSE = sum (|x| - absmax)^2, with a value of exactly 0 going to the upper level."""
    rng = np.random.default_rng(1)
    N, K = 5, 256
    W, a = blocks_with_power_of_two_absmax(rng, N, K)
    W[0, 3] = 0.0
    maps, thr = tables(N, [-1.0, 1.0])
    precs = np.full(N, 1, dtype=np.uint8)
    sse, res = oracle.quant_error(W, precs, maps, thr)
    a_elem = np.repeat(a, 64, axis=1)
    want = ((np.abs(W.astype(np.float64)) - a_elem) ** 2).sum(axis=1)
    np.testing.assert_allclose(sse, want, rtol=1e-13)
    assert res[0, 3] == -a_elem[0, 3]                       # 0 -> +absmax, residual 0 - absmax
    np.testing.assert_array_equal(res, (W.astype(np.float64) - np.where(W >= 0, 1.0, -1.0) * a_elem).astype(np.float32))


@pytest.mark.parametrize("b", [1, 2, 4])
def test_values_on_the_levels_have_no_error(b):
    rng = np.random.default_rng(2 + b)
    N, K = 4, 192
    levels = np.linspace(-1.0, 1.0, 2 ** b) if b < 4 else (np.arange(16) - 7.5) / 7.5
    levels = np.round(levels * 64) / 64                      # few mantissa bits: level * 2^e is exact in bf16
    levels[0], levels[-1] = -1.0, 1.0
    e = np.exp2(rng.integers(-5, 2, size=(N, K // 64)))
    idx = rng.integers(0, levels.size, size=(N, K))
    idx.reshape(N, K // 64, 64)[:, :, 0] = levels.size - 1    # every block holds a full-scale value
    W = (levels[idx] * np.repeat(e, 64, axis=1)).astype(np.float32)
    maps, thr = tables(N, levels)
    sse, res = oracle.quant_error(W, np.full(N, b, dtype=np.uint8), maps, thr)
    assert (sse == 0).all() and (res == 0).all()


@pytest.mark.parametrize("b", [2, 4])
def test_against_nearest_level_brute_force(b):
    """With midpoint thresholds and exact normalisation the chosen level is the nearest one, so
    SSE = sum_k min_j (x_k - level_j * absmax)^2 (levels with few mantissa bits: no bf16 rounding)."""
    rng = np.random.default_rng(10 + b)
    N, K = 3, 128
    W, a = blocks_with_power_of_two_absmax(rng, N, K)
    levels = np.sort(np.round(rng.uniform(-1, 1, size=2 ** b) * 32) / 32)
    levels[0], levels[-1] = -1.0, 1.0
    levels = np.unique(levels)
    while levels.size < 2 ** b:                               # keep 2^b distinct levels
        levels = np.unique(np.append(levels, np.round(rng.uniform(-1, 1) * 32) / 32))
    maps, thr = tables(N, levels)
    sse, _ = oracle.quant_error(W, np.full(N, b, dtype=np.uint8), maps, thr)
    a_elem = np.repeat(a, 64, axis=1)
    cand = levels[None, None, :] * a_elem[:, :, None]
    want = ((W.astype(np.float64)[:, :, None] - cand) ** 2).min(axis=2).sum(axis=1)
    np.testing.assert_allclose(sse, want, rtol=1e-12)


def test_scaling_by_a_power_of_two_scales_the_error_exactly():
    rng = np.random.default_rng(20)
    N, K = 6, 256
    W = (rng.standard_normal((N, K)) * 0.02).astype(np.float32)
    precs = np.array([1, 2, 4, 4, 2, 1], dtype=np.uint8)
    maps = np.zeros((N, T), dtype=np.float32); thr = np.zeros((N, T), dtype=np.float32)
    for i, b in enumerate(precs):
        lv = np.sort(rng.uniform(-1, 1, size=2 ** b)); lv[0], lv[-1] = -1.0, 1.0
        maps[i, :lv.size] = lv
        thr[i, :lv.size - 1] = 0.5 * (lv[:-1] + lv[1:])
    sse1, res1 = oracle.quant_error(W, precs, maps, thr)
    sse2, res2 = oracle.quant_error(W * np.float32(8.0), precs, maps, thr)
    np.testing.assert_array_equal(sse2, sse1 * 64.0)
    np.testing.assert_array_equal(res2, res1 * np.float32(8.0))


def test_nested_codebooks_more_bits_never_worse():
    """A 4-bit codebook that contains the 2-bit levels, which contain the 1-bit levels (all with few mantissa
    bits, block maxima powers of two, midpoint thresholds): the error cannot grow with the precision."""
    rng = np.random.default_rng(30)
    N, K = 4, 512
    W, _ = blocks_with_power_of_two_absmax(rng, N, K)
    l1 = np.array([-1.0, 1.0])
    l2 = np.array([-1.0, -0.25, 0.25, 1.0])
    l4 = np.unique(np.concatenate([l2, np.arange(-7, 8, 2) / 8.0, [-0.5, 0.5, -0.0625, 0.0625]]))
    assert l4.size == 16
    out = []
    for b, lv in ((1, l1), (2, l2), (4, l4)):
        maps, thr = tables(N, lv)
        out.append(oracle.quant_error(W, np.full(N, b, dtype=np.uint8), maps, thr)[0])
    assert (out[1] <= out[0]).all() and (out[2] <= out[1]).all()
    assert (out[2] < out[0]).all()


def test_residual_and_error_agree():
    rng = np.random.default_rng(40)
    N, K = 8, 384
    W = (rng.standard_normal((N, K)) * 0.05).astype(np.float32)
    precs = rng.choice([1, 2, 4], size=N).astype(np.uint8)
    maps, thr = oracle.lloyd_max(W, precs, T=3)
    sse, res = oracle.quant_error(W, precs, maps, thr)
    np.testing.assert_allclose((res.astype(np.float64) ** 2).sum(axis=1), sse, rtol=1e-6)
    packed, a = oracle.encode(W, precs, thr)
    w_hat = oracle.bf16_to_f64(oracle.decode(packed, a, maps, precs, K))
    assert np.abs(W.astype(np.float64) - w_hat - res).max() <= 2.0 ** -24 * np.abs(W).max()
