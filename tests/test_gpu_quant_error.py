"""GPU parity of the per-channel quantisation error and the residual against the oracle, through the C ABI.

The residual fl32(W - W_hat) is one IEEE subtraction per element on both sides: bit-exact.  The error is, on the
GPU, the sum of the squared fp32 residuals, four neighbouring squares added in fp32 and those partial sums in fp64
(fixed tree); in the oracle, the sum of the squared exact differences in fp64.  Every term carries (1 + 2^-24)^2
from the residual's rounding and every group of four at most three more fp32 roundings (square, two additions), so
the sums agree to 2^-23 + 3 * 2^-24 < 2^-21 relative plus fp64 summation noise; the test allows 2^-21.
"""
import numpy as np
import pytest
import torch

import oracle
import synth_inputs as si
from helpers import make_case

pytestmark = pytest.mark.gpu
RTOL = 2.0 ** -21


@pytest.fixture(scope="module")
def lw():
    import paper_2502_08141_b200 as lw
    return lw


CASES = [
    # N, K, mix, kind
    (16, 128, {1: 0.5, 2: 0.5}, "llama"),                          # one 128-element row piece per thread group
    (96, 1152, {1: 0.3, 2: 0.4, 4: 0.3}, "llama"),                 # K not a multiple of 1024: ragged last batch
    (33, 4096, {4: 1.0}, "llama"),
    (50, 11008, {1: 0.6, 2: 0.35, 4: 0.05}, "llama"),              # row longer than one batch of loads
    (2000, 256, {1: 0.34, 2: 0.33, 4: 0.33}, "tiny"),              # more rows than CTAs in the grid
]


@pytest.mark.parametrize("N,K,mix,kind", CASES)
def test_error_and_residual(lw, N, K, mix, kind):
    case = make_case(N, K, mix, matrix_id=(N * 7 + K) % 61, kind=kind)
    layout = lw.Layout(case.precs, K)
    W = torch.from_numpy(case.W).cuda()
    maps, thr = torch.from_numpy(case.maps).cuda(), torch.from_numpy(case.thr).cuda()
    sse, res = lw.lowra_quant_error(layout, W, maps, thr, want_residual=True)
    sse_only, none = lw.lowra_quant_error(layout, W, maps, thr)
    torch.cuda.synchronize()
    assert none is None
    sse_ref, res_ref = oracle.quant_error(case.W, case.precs, case.maps, case.thr)
    assert np.array_equal(res.cpu().numpy().view(np.uint32), res_ref.view(np.uint32))
    got = sse.cpu().numpy()
    assert np.all(np.abs(got - sse_ref) <= RTOL * sse_ref), float(np.max(np.abs(got - sse_ref) / np.maximum(sse_ref, 1e-300)))
    assert np.array_equal(got, sse_only.cpu().numpy())            # reproducible, with or without the residual


def test_zero_rows_and_exact_levels(lw):
    """All-zero blocks quantise to zero exactly; values on the levels leave no residual."""
    N, K = 8, 256
    precs = np.array([1, 2, 4, 1, 2, 4, 1, 2], dtype=np.uint8)
    maps, thr = si.standin_codebooks(precs)
    W = np.zeros((N, K), dtype=np.float32)
    W[3:, :] = (np.arange(K, dtype=np.float32) % 7 - 3.0) * 0.01
    W[5, 64:128] = 0.0
    layout = lw.Layout(precs, K)
    sse, res = lw.lowra_quant_error(layout, torch.from_numpy(W).cuda(), torch.from_numpy(maps).cuda(),
                                    torch.from_numpy(thr).cuda(), want_residual=True)
    sse_ref, res_ref = oracle.quant_error(W, precs, maps, thr)
    got, res = sse.cpu().numpy(), res.cpu().numpy()
    assert (got[:3] == 0).all() and (res[:3] == 0).all() and (res[5, 64:128] == 0).all()
    assert np.array_equal(res.view(np.uint32), res_ref.view(np.uint32))
    assert np.all(np.abs(got - sse_ref) <= RTOL * sse_ref)


def test_error_of_the_learned_codebooks_falls_with_the_precision(lw):
    """The use the paper makes of it: every channel's error under 1, 2 and 4 bits, codebooks from the learner."""
    N, K = 64, 1024
    W_np = si.weights(N, K, matrix_id=9)
    W = torch.from_numpy(np.ascontiguousarray(W_np)).cuda()
    y0 = np.zeros((3, 16)); t0 = np.zeros((3, 16))
    for c, b in enumerate((1, 2, 4)):
        y, t = oracle.initial_tables(b)
        y0[c, :y.size] = y; t0[c, :t.size] = t
    errs = []
    for b in (1, 2, 4):
        precs = np.full(N, b, dtype=np.uint8)
        layout = lw.Layout(precs, K)
        maps, thr = lw.lowra_learn_codebooks(layout, W, y0, t0, 4)
        sse, _ = lw.lowra_quant_error(layout, W, maps, thr)
        ref, _ = oracle.quant_error(W_np, precs, maps.cpu().numpy(), thr.cpu().numpy())
        assert np.all(np.abs(sse.cpu().numpy() - ref) <= RTOL * ref)
        errs.append(sse.cpu().numpy())
    assert (errs[1] < errs[0]).all() and (errs[2] < errs[1]).all()


@pytest.mark.parametrize("N,K", [(24, 128), (100, 1152), (300, 4096), (40, 11008)])
def test_three_precisions_in_one_pass(lw, N, K):
    """Every row under 1, 2 and 4 bits with its own three codebooks: equal to three calls of the oracle with uniform
    precisions, and bit-identical to three calls of lowra_quant_error (same arithmetic, same order)."""
    W_np = si.weights(N, K, matrix_id=(N + K) % 50)
    W = torch.from_numpy(np.ascontiguousarray(W_np)).cuda()
    maps3 = np.zeros((3, N, 16), dtype=np.float32)
    thr3 = np.zeros((3, N, 16), dtype=np.float32)
    ref = np.zeros((N, 3))
    single = np.zeros((N, 3))
    for c, b in enumerate((1, 2, 4)):
        precs = np.full(N, b, dtype=np.uint8)
        maps3[c], thr3[c] = oracle.lloyd_max(W_np, precs, T=2)
        ref[:, c], _ = oracle.quant_error(W_np, precs, maps3[c], thr3[c])
        sse, _ = lw.lowra_quant_error(lw.Layout(precs, K), W, torch.from_numpy(maps3[c]).cuda(), torch.from_numpy(thr3[c]).cuda())
        single[:, c] = sse.cpu().numpy()
    got = lw.lowra_channel_errors(W, torch.from_numpy(maps3).cuda(), torch.from_numpy(thr3).cuda()).cpu().numpy()
    assert np.all(np.abs(got - ref) <= RTOL * ref)
    assert np.array_equal(got, single)
