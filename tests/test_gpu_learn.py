"""GPU parity of the codebook learner (weighted Lloyd-Max per output channel) against the oracle.

The learner works in fp64 on both sides, but the GPU adds its per-bucket sums up in a fixed parallel tree and
the oracle in index order, so levels agree to fp64 rounding; after the final rounding to fp32 they are either
equal or (rarely) one fp32 ulp apart.  Tolerance: 2 ulp of fp32 at the level's magnitude (levels live in
[-1, 1]: 2.4e-7), and at least 99 % of the entries bit-identical.  The thresholds are a function of the fp32
levels alone and must reproduce that function exactly.
"""
import numpy as np
import pytest
import torch

import oracle
import synth_inputs as si

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def lw():
    import paper_2502_08141_b200 as lw
    return lw


def _init_tables():
    y0 = np.zeros((3, 16), dtype=np.float64)
    t0 = np.zeros((3, 16), dtype=np.float64)
    for c, b in enumerate((1, 2, 4)):
        y, t = oracle.initial_tables(b)
        y0[c, :y.size] = y
        t0[c, :t.size] = t
    return y0, t0


def _run(lw, W, precs, T):
    N, K = W.shape
    layout = lw.Layout(precs, K)
    y0, t0 = _init_tables()
    maps, thr = lw.lowra_learn_codebooks(layout, torch.from_numpy(W).cuda(), y0, t0, T)
    torch.cuda.synchronize()
    return maps.cpu().numpy(), thr.cpu().numpy()


def _check(maps, thr, precs, maps_ref, thr_ref):
    assert maps.shape == maps_ref.shape and thr.shape == thr_ref.shape
    tol = 2.4e-7 * np.maximum(1.0, np.abs(maps_ref))
    assert np.all(np.abs(maps.astype(np.float64) - maps_ref) <= tol), float(np.abs(maps - maps_ref).max())
    assert (maps == maps_ref).mean() >= 0.99
    finite = np.isfinite(thr_ref)
    assert np.array_equal(np.isfinite(thr), finite)               # unused thresholds are +inf on both sides
    assert np.all(thr[~finite] > 0)
    assert np.all(np.abs(thr[finite].astype(np.float64) - thr_ref[finite]) <= 2.4e-7)
    # what holds exactly, whatever the sums: thresholds are the rounded midpoints of the fp32 levels, levels are
    # sorted, unused levels are zero
    for r in range(maps.shape[0]):
        L = 1 << int(precs[r])
        m = maps[r, :L].astype(np.float64)
        assert np.all(np.diff(m) >= 0)
        assert np.array_equal(thr[r, :L - 1], ((m[:-1] + m[1:]) * 0.5).astype(np.float32))
        assert np.all(maps[r, L:] == 0)


CASES = [
    # N, K, mix, kind, T
    (96, 512, {1: 0.34, 2: 0.33, 4: 0.33}, "llama", 10),
    (333, 1408, {1: 0.6, 2: 0.35, 4: 0.05}, "llama", 10),     # ragged everything
    (64, 4096, {1: 0.3, 2: 0.5, 4: 0.2}, "llama", 2),         # the paper's iteration count
    (128, 256, {1: 0.5, 2: 0.5}, "tiny", 10),
    (40, 11008, {2: 0.75, 4: 0.25}, "llama", 10),             # the longest rows of the 7B shapes
]


@pytest.mark.parametrize("N,K,mix,kind,T", CASES)
def test_learner_matches_oracle(lw, N, K, mix, kind, T):
    W = si.weights(N, K, matrix_id=(N + K) % 61, kind=kind)
    precs = si.precisions(N, mix, matrix_id=(N + K) % 61)
    maps_ref, thr_ref = oracle.lloyd_max(W, precs, T=T)
    maps, thr = _run(lw, W, precs, T)
    _check(maps, thr, precs, maps_ref, thr_ref)


def test_zero_iterations_return_the_initial_tables(lw):
    W = si.weights(32, 256, matrix_id=5, kind="llama")
    precs = si.precisions(32, {1: 0.34, 2: 0.33, 4: 0.33}, matrix_id=5)
    maps, thr = _run(lw, W, precs, 0)
    y0, _ = _init_tables()
    for r in range(32):
        c = {1: 0, 2: 1, 4: 2}[int(precs[r])]
        L = 1 << int(precs[r])
        assert np.array_equal(maps[r, :L], y0[c, :L].astype(np.float32))


def test_degenerate_rows(lw):
    """An all-zero row (every weight 0: all sums empty, levels stay) and a constant row."""
    W = si.weights(16, 256, matrix_id=9, kind="llama").copy()
    W[3, :] = 0.0
    W[7, :] = 0.125
    W[8, :128] = -2.0
    W[8, 128:] = 0.0
    precs = np.array([1, 2, 4, 1, 2, 4, 1, 2, 4, 1, 2, 4, 1, 2, 4, 1], dtype=np.uint8)
    maps_ref, thr_ref = oracle.lloyd_max(W, precs, T=10)
    maps, thr = _run(lw, W, precs, 10)
    _check(maps, thr, precs, maps_ref, thr_ref)


def test_learned_tables_feed_the_encoder(lw):
    """encode with GPU-learned thresholds, decode with GPU-learned levels: the reconstruction error is the one
    the oracle's codebooks give, to the same precision as the codebooks agree."""
    N, K = 128, 1024
    W = si.weights(N, K, matrix_id=11, kind="llama")
    precs = si.precisions(N, {1: 0.3, 2: 0.5, 4: 0.2}, matrix_id=11)
    layout = lw.Layout(precs, K)
    y0, t0 = _init_tables()
    Wd = torch.from_numpy(W).cuda()
    maps, thr = lw.lowra_learn_codebooks(layout, Wd, y0, t0, 10)
    packed, absmax = lw.lowra_encode(layout, Wd, thr)
    W_hat = lw.lowra_decode(layout, packed, absmax, maps).float().cpu().numpy()
    maps_ref, thr_ref = oracle.lloyd_max(W, precs, T=10)
    p_ref, a_ref = oracle.encode(W, precs, thr_ref)
    W_ref = si.bf16_bits_to_f32(oracle.decode(p_ref, a_ref, maps_ref, precs, K))
    err_gpu = float(((W_hat - W) ** 2).sum())
    err_ref = float(((W_ref - W) ** 2).sum())
    assert abs(err_gpu - err_ref) <= 1e-4 * err_ref


@pytest.mark.parametrize("N,K,T", [(96, 512, 10), (333, 1408, 2), (40, 11008, 3)])
def test_all_three_precisions_in_one_pass(lw, N, K, T):
    """lowra_learn_codebooks_all: every row at 1, 2 and 4 bits from one read of W.  Plane c is bit for bit what the
    per-layout learner gives when every row has 2^c bits (same arithmetic on the same normalised row), and agrees
    with the oracle like that one; its output feeds lowra_channel_errors as it stands."""
    W = si.weights(N, K, matrix_id=(N + K) % 53, kind="llama")
    Wd = torch.from_numpy(W).cuda()
    y0, t0 = _init_tables()
    maps3, thr3 = lw.lowra_learn_codebooks_all(Wd, y0, t0, T)
    torch.cuda.synchronize()
    sse_ref = np.zeros((N, 3))
    for c, b in enumerate((1, 2, 4)):
        precs = np.full(N, b, dtype=np.uint8)
        m1, h1 = lw.lowra_learn_codebooks(lw.Layout(precs, K), Wd, y0, t0, T)
        assert torch.equal(maps3[c].view(torch.int32), m1.view(torch.int32)), b
        assert torch.equal(thr3[c].view(torch.int32), h1.view(torch.int32)), b
        maps_ref, thr_ref = oracle.lloyd_max(W, precs, T=T)
        _check(maps3[c].cpu().numpy(), thr3[c].cpu().numpy(), precs, maps_ref, thr_ref)
        sse_ref[:, c], _ = oracle.quant_error(W, precs, maps3[c].cpu().numpy(), thr3[c].cpu().numpy())
    # the two calls that give the precision assigner its input: tables for all precisions, then the errors
    sse3 = lw.lowra_channel_errors(Wd, maps3, thr3).cpu().numpy()
    assert np.all(np.abs(sse3 - sse_ref) <= 2.0 ** -21 * sse_ref)
    assert (sse3[:, 1] < sse3[:, 0]).all() and (sse3[:, 2] < sse3[:, 1]).all()
