"""Pins for the oracle's codebook learner (weighted Lloyd-Max) and its two LoRA products."""
import os

import numpy as np
import pytest

import oracle
import synth_inputs as si

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "appendix_f_initial_tables.txt")


def _golden():
    out = {}
    with open(GOLDEN) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            name, *vals = line.split()
            out[name] = np.array([float(v) for v in vals])
    return out


def test_initial_tables_are_the_printed_ones():
    g = _golden()
    m4, t4 = oracle.initial_tables(4)
    m2, t2 = oracle.initial_tables(2)
    m1, t1 = oracle.initial_tables(1)
    assert np.array_equal(m4, g["mappings_4bit"]) and m4.size == 16
    assert np.array_equal(m2, g["mappings_2bit"]) and np.array_equal(t2, g["thresholds_2bit"])
    assert np.array_equal(m1, g["mappings_1bit"]) and np.array_equal(t1, g["thresholds_1bit"])
    # the printed 2-bit thresholds are the midpoints of the 4-bit list's entries -1, 0, 0.33791524, 1:
    # this is what fixes "thresholds = midpoints of consecutive levels" for the 4-bit case too
    lv = np.array([-1.0, 0.0, g["mappings_4bit"][11], 1.0])
    assert np.allclose(t2, (lv[:-1] + lv[1:]) / 2, atol=1e-8)
    assert np.allclose(t4, (m4[:-1] + m4[1:]) / 2, atol=0) and np.all(np.diff(t4) > 0)


@pytest.mark.parametrize("b", [1, 2, 4])
def test_distortion_never_increases(b):
    W = si.weights(8, 1024, matrix_id=20 + b)
    n = oracle.normalise(W, 64).astype(np.float64)
    w = np.repeat(oracle.absmax(W, 64), 64, axis=1).astype(np.float64)
    for r in range(8):
        y, t, trace = oracle.lloyd_max_row(n[r], w[r], b, 10)
        assert trace.size == 20
        assert np.all(np.diff(trace) <= 1e-12 * trace[0])
        assert trace[-1] < trace[0]
        assert np.all(np.diff(y) >= 0) and np.all(np.diff(t) >= 0)
        assert np.allclose(t, (y[:-1] + y[1:]) / 2, rtol=0, atol=0)
        # final distortion recomputed independently: nearest-level assignment of the last E step
        c = np.searchsorted((lambda yy: (yy[:-1] + yy[1:]) / 2)(y), n[r], side="right")
        d_after = np.sum(w[r] * (n[r] - y[c]) ** 2)
        assert d_after <= trace[-1] * (1 + 1e-12)


@pytest.mark.parametrize("b", [1, 2, 4])
def test_exactly_2b_separated_values_are_recovered(b):
    L = 1 << b
    rng = np.random.default_rng(b)
    init, _ = oracle.initial_tables(b)
    # separated points, one next to each initial level so that every bucket is hit
    pts = init + rng.uniform(-0.02, 0.02, size=L)
    x = np.repeat(pts, 50)
    rng.shuffle(x)
    w = rng.uniform(0.5, 2.0, size=x.size)
    y, t, trace = oracle.lloyd_max_row(x, w, b, 10)
    assert np.allclose(y, np.sort(pts), atol=1e-15)
    assert trace[-1] <= 1e-28


def test_symmetric_two_point_data_one_bit():
    x = np.array([-0.37, 0.37] * 64)
    w = np.ones_like(x)
    y, t, _ = oracle.lloyd_max_row(x, w, 1, 3)
    assert np.allclose(y, [-0.37, 0.37], atol=1e-16) and t[0] == 0.0


def test_weighted_centroid_closed_form_one_iteration():
    # one iteration, b = 1, threshold 0: levels are the weighted means of the two sides
    rng = np.random.default_rng(3)
    x = rng.uniform(-1, 1, 500)
    w = rng.uniform(0.1, 3.0, 500)
    y, t, _ = oracle.lloyd_max_row(x, w, 1, 1)
    neg, pos = x < 0, x >= 0
    assert np.isclose(y[0], np.sum(w[neg] * x[neg]) / np.sum(w[neg]), rtol=1e-13)
    assert np.isclose(y[1], np.sum(w[pos] * x[pos]) / np.sum(w[pos]), rtol=1e-13)
    assert np.isclose(t[0], (y[0] + y[1]) / 2, rtol=1e-15)
    # weights matter: scaling the weights of the positive side's largest point pulls y[1] up
    w2 = w.copy(); w2[np.argmax(x)] *= 100
    y2, _, _ = oracle.lloyd_max_row(x, w2, 1, 1)
    assert y2[1] > y[1] and y2[0] == y[0]


def test_empty_bucket_keeps_its_level():
    x = np.full(64, 0.9)          # everything lands in the top bucket of a 2-bit table
    y, t, _ = oracle.lloyd_max_row(x, np.ones(64), 2, 2)
    init, _ = oracle.initial_tables(2)
    assert np.array_equal(y[:3], init[:3]) and np.isclose(y[3], 0.9)


def test_matrix_learner_tables_layout():
    N, K = 48, 512
    W = si.weights(N, K, matrix_id=30)
    precs = si.precisions(N, {1: 0.3, 2: 0.4, 4: 0.3}, matrix_id=30)
    maps, thr, trace = oracle.lloyd_max(W, precs, T=10, return_trace=True)
    assert maps.shape == thr.shape == (N, 16) and maps.dtype == thr.dtype == np.float32
    n = oracle.normalise(W, 64).astype(np.float64)
    w = np.repeat(oracle.absmax(W, 64), 64, axis=1).astype(np.float64)
    for r in range(N):
        L = 1 << int(precs[r])
        assert np.all(maps[r, L:] == 0) and np.all(np.isinf(thr[r, L - 1:]))
        assert np.all(np.diff(maps[r, :L]) >= 0)
        mid = ((maps[r, :L - 1].astype(np.float64) + maps[r, 1:L].astype(np.float64)) / 2).astype(np.float32)
        assert np.array_equal(thr[r, :L - 1], mid)
        y, _, tr = oracle.lloyd_max_row(n[r], w[r], int(precs[r]), 10)
        assert np.array_equal(maps[r, :L], y.astype(np.float32))
        assert np.all(np.diff(trace[r]) <= 1e-12 * trace[r, 0])
    # the learnt tables beat the initial ones on the reconstruction error they are trained for
    _, a, codes = oracle.encode(W, precs, thr, return_codes=True)
    rec = np.take_along_axis(maps, codes.astype(np.int64), axis=1)
    err_learnt = np.sum(w * (n - rec) ** 2)
    maps0 = np.zeros_like(maps); thr0 = np.full_like(thr, np.inf)
    for r in range(N):
        y0, t0 = oracle.initial_tables(int(precs[r]))
        maps0[r, :y0.size] = y0; thr0[r, :t0.size] = t0
    _, _, codes0 = oracle.encode(W, precs, thr0, return_codes=True)
    err_init = np.sum(w * (n - np.take_along_axis(maps0, codes0.astype(np.int64), axis=1)) ** 2)
    assert err_learnt < err_init


# ------------------------------------------------------------------------------------------
def _case(M, N, K, r, seed):
    rng = np.random.default_rng(seed)
    bf = lambda a: si.f32_to_bf16_bits(a.astype(np.float32))
    W = bf(rng.standard_normal((N, K)) * 0.05)
    X = bf(rng.standard_normal((M, K)))
    dY = bf(rng.standard_normal((M, N)))
    A = bf(rng.standard_normal((K, r)) * 0.1)
    B = bf(rng.standard_normal((r, N)) * 0.1)
    return W, X, dY, A, B


@pytest.mark.parametrize("M,N,K,r", [(8, 8, 8, 2), (16, 24, 32, 4), (64, 64, 64, 16)])
def test_products_against_long_double_triple_loop(M, N, K, r):
    W, X, dY, A, B = _case(M, N, K, r, 1)
    f = oracle.bf16_to_f64
    s = 2.0
    Y = oracle.lora_forward(W, X, A, B, s)
    want = oracle.matmul_naive(f(X), f(W).T.copy()) + s * oracle.matmul_naive(oracle.matmul_naive(f(X), f(A)), f(B))
    assert np.allclose(Y, want, rtol=1e-12, atol=1e-13)
    dX = oracle.lora_backward_input(W, dY, A, B, s)
    want = oracle.matmul_naive(f(dY), f(W)) + s * oracle.matmul_naive(
        oracle.matmul_naive(f(dY), f(B).T.copy()), f(A).T.copy())
    assert np.allclose(dX, want, rtol=1e-12, atol=1e-13)


def test_product_identities():
    M, N, K, r = 32, 48, 40, 8
    W, X, dY, A, B = _case(M, N, K, r, 2)
    f = oracle.bf16_to_f64
    zero_A, zero_B = np.zeros_like(A), np.zeros_like(B)
    base = f(X) @ f(W).T
    assert np.allclose(oracle.lora_forward(W, X, A, B, 0.0), base, atol=1e-14)
    assert np.allclose(oracle.lora_forward(W, X, zero_A, B, 2.0), base, atol=1e-14)
    assert np.allclose(oracle.lora_forward(W, X, A, zero_B, 2.0), base, atol=1e-14)
    # X = identity  =>  Y = W_hat^T + s A B
    eye = si.f32_to_bf16_bits(np.eye(K, dtype=np.float32))
    assert np.allclose(oracle.lora_forward(W, eye, A, B, 2.0), f(W).T + 2.0 * f(A) @ f(B), atol=1e-14)
    # dY = identity =>  dX = W_hat + s B^T A^T
    eyeN = si.f32_to_bf16_bits(np.eye(N, dtype=np.float32))
    assert np.allclose(oracle.lora_backward_input(W, eyeN, A, B, 2.0), f(W) + 2.0 * (f(A) @ f(B)).T, atol=1e-14)
    # linear in s
    y1 = oracle.lora_forward(W, X, A, B, 1.0); y3 = oracle.lora_forward(W, X, A, B, 3.0)
    assert np.allclose(y3 - y1, 2.0 * (f(X) @ f(A)) @ f(B), atol=1e-13)


def test_backward_is_the_adjoint_of_forward():
    """<dY, forward(X)> == <backward(dY), X> for every X, dY: pins dX against Y."""
    M, N, K, r = 40, 56, 72, 8
    W, X, dY, A, B = _case(M, N, K, r, 3)
    f = oracle.bf16_to_f64
    lhs = np.sum(f(dY) * oracle.lora_forward(W, X, A, B, 2.0))
    rhs = np.sum(oracle.lora_backward_input(W, dY, A, B, 2.0) * f(X))
    assert abs(lhs - rhs) <= 1e-10 * abs(lhs)


def test_adapter_gradients_are_the_derivatives_of_the_forward():
    """Y is linear in A for fixed B (and in B for fixed A), so for any direction D:
    <dY, forward(A + D) - forward(A)> = <dA, D> exactly (up to fp64 rounding); same for B.
    Also a brute-force triple loop on a tiny case, and the trivial cases s = 0, dY = 0."""
    rng = np.random.default_rng(5)
    M, K, N, r, s = 12, 16, 10, 4, 1.5
    bf = lambda a: oracle.f32_to_bf16(a.astype(np.float32))
    f = oracle.bf16_to_f64
    X, dY = bf(rng.standard_normal((M, K))), bf(rng.standard_normal((M, N)))
    A, B = bf(rng.standard_normal((K, r))), bf(rng.standard_normal((r, N)))
    W = bf(rng.standard_normal((N, K)))
    dA, dB = oracle.lora_backward_adapters(X, dY, A, B, s)
    assert dA.shape == (K, r) and dB.shape == (r, N)
    DA, DB = bf(rng.standard_normal((K, r))), bf(rng.standard_normal((r, N)))
    # directional derivatives through the forward oracle (exactly representable perturbed factors)
    A2, B2 = bf(f(A) + f(DA)), bf(f(B) + f(DB))
    dirA, dirB = f(A2) - f(A), f(B2) - f(B)
    y0 = oracle.lora_forward(W, X, A, B, s)
    lhsA = np.sum(f(dY) * (oracle.lora_forward(W, X, A2, B, s) - y0))
    lhsB = np.sum(f(dY) * (oracle.lora_forward(W, X, A, B2, s) - y0))
    assert abs(lhsA - np.sum(dA * dirA)) <= 1e-10 * abs(lhsA)
    assert abs(lhsB - np.sum(dB * dirB)) <= 1e-10 * abs(lhsB)
    # definition written out with loops
    Xf, dYf, Af, Bf = f(X), f(dY), f(A), f(B)
    dA_loop = np.zeros((K, r)); dB_loop = np.zeros((r, N))
    for k in range(K):
        for j in range(r):
            dA_loop[k, j] = s * sum(Xf[m, k] * sum(dYf[m, n] * Bf[j, n] for n in range(N)) for m in range(M))
    for j in range(r):
        for n in range(N):
            dB_loop[j, n] = s * sum(sum(Xf[m, k] * Af[k, j] for k in range(K)) * dYf[m, n] for m in range(M))
    assert np.allclose(dA, dA_loop, rtol=1e-12, atol=1e-12) and np.allclose(dB, dB_loop, rtol=1e-12, atol=1e-12)
    z = oracle.lora_backward_adapters(X, dY, A, B, 0.0)
    assert not z[0].any() and not z[1].any()
    z = oracle.lora_backward_adapters(X, bf(np.zeros((M, N))), A, B, s)
    assert not z[0].any() and not z[1].any()
