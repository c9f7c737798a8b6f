"""Seeded random shapes through the codec, every tensor-core entry point and the error kernel, against the oracle.

Shapes the hand-picked cases do not hit: channel counts that are any multiple of 8, contraction lengths that are
any multiple of 128, token counts from 1 upwards, every rank from 16 to 128, eight precision mixes (three of them
single-class), six many-tile / short-contraction problems that run the stream-K schedule with preloaded partial tiles
in one or both passes, and six with one to seven rows of pieces per cluster (partial tiles added in the epilogue).
"""
import numpy as np
import pytest
import torch

import oracle
import synth_inputs as si
from helpers import FRO_TOL, MAX_TOL, gemm_errors, make_case

pytestmark = pytest.mark.gpu

MIXES = [{1: 1.0}, {2: 1.0}, {4: 1.0}, {1: 0.6, 2: 0.35, 4: 0.05}, {1: 0.3, 2: 0.5, 4: 0.2}, {1: 0.85, 2: 0.15},
         {2: 0.75, 4: 0.25}, {1: 0.02, 2: 0.02, 4: 0.96}]


def _cases():
    rng = np.random.default_rng(20250208)
    out = []
    for i in range(14):
        N = int(rng.integers(1, 60)) * 8 * int(rng.choice([1, 1, 4, 8]))
        K = int(rng.integers(1, 12)) * 128
        out.append((N, K, int(rng.integers(1, 1500)), int(rng.integers(1, 9)) * 16, int(rng.integers(0, len(MIXES))), 100 + i))
    for i, (N, K, M, r) in enumerate([(2304, 256, 6000, 16), (2312, 384, 5900, 48), (1160, 512, 12000, 128),
                                      (3072, 256, 4100, 96), (256, 2304, 6100, 32), (384, 2432, 5800, 64)]):
        out.append((N, K, M, r, (3 + i) % len(MIXES), 200 + i))
    # between one and seven rows of pieces per cluster: whole rows first, then ranges over the last one or two
    # (partial tiles added in the epilogue, one to three slices per tile)
    for i, (N, K, M, r) in enumerate([(2680, 512, 8603, 16), (512, 2176, 3387, 64), (1536, 768, 6550, 96),
                                      (1408, 256, 8137, 64), (3264, 256, 8757, 80), (2040, 384, 6829, 80)]):
        out.append((N, K, M, r, (1 + i) % len(MIXES), 300 + i))
    return out


@pytest.mark.parametrize("N,K,M,r,mix_id,mid", _cases())
def test_random_shape(N, K, M, r, mix_id, mid):
    import paper_2502_08141_b200 as lw

    dev = lambda a: torch.from_numpy(np.ascontiguousarray(a)).cuda()
    bf = lambda b: dev(b.view(np.int16)).view(torch.bfloat16)
    bits = lambda t: t.view(torch.int16).cpu().numpy().view(np.uint16)
    case = make_case(N, K, MIXES[mix_id], matrix_id=mid, lloyd_iters=1)
    layout = lw.Layout(case.precs, K)
    X, dY = si.activations(M, K, matrix_id=mid), si.out_grads(M, N, matrix_id=mid)
    A = si.bf16_normal((K, r), 0.02, stream=300 + mid)
    B = si.bf16_normal((r, N), 0.02, stream=600 + mid)
    s = (0.5, 1.0, 2.0)[mid % 3]
    packed, absmax, maps = dev(case.packed), dev(case.absmax), dev(case.maps)
    ws = torch.empty(lw.lowra_workspace_bytes(layout, M, r), dtype=torch.uint8, device="cuda")

    # codec and row reordering: bit-exact
    p_gpu, a_gpu = lw.lowra_encode(layout, dev(case.W), dev(case.thr))
    assert np.array_equal(p_gpu.cpu().numpy()[:layout.packed_bytes], case.packed)
    assert np.array_equal(a_gpu.cpu().numpy().view(np.uint32), case.absmax.view(np.uint32))
    assert np.array_equal(bits(lw.lowra_decode(layout, packed, absmax, maps)), case.W_hat)
    off = torch.from_numpy(lw.lowra_natural_offsets(case.precs, K).view(np.int64)).cuda()
    nat, a_nat = lw.lowra_reorder_rows(layout, True, off, packed, absmax)
    back, a_back = lw.lowra_reorder_rows(layout, False, off, nat, a_nat)
    assert torch.equal(back, packed) and torch.equal(a_back, absmax)

    Y = torch.full((M, N), float("nan"), dtype=torch.bfloat16, device="cuda")
    lw.lowra_lora_forward(layout, packed, absmax, maps, bf(X), bf(A), bf(B), s, Y=Y, workspace=ws)
    assert lw.lowra_device_status(ws) == lw.LOWRA_OK
    emax, efro = gemm_errors(si.bf16_bits_to_f32(bits(Y)), oracle.lora_forward(case.W_hat, X, A, B, s))
    assert emax <= MAX_TOL and efro <= FRO_TOL, ("forward", emax, efro)

    dX = torch.full((M, K), float("nan"), dtype=torch.bfloat16, device="cuda")
    lw.lowra_lora_backward_input(layout, packed, absmax, maps, bf(dY), bf(A), bf(B), s, dX=dX, workspace=ws)
    assert lw.lowra_device_status(ws) == lw.LOWRA_OK
    emax, efro = gemm_errors(si.bf16_bits_to_f32(bits(dX)), oracle.lora_backward_input(case.W_hat, dY, A, B, s))
    assert emax <= MAX_TOL and efro <= FRO_TOL, ("backward", emax, efro)

    dA, dB = lw.lowra_lora_backward_adapters(bf(X), bf(dY), bf(A), bf(B), s)
    dA_ref, dB_ref = oracle.lora_backward_adapters(X, dY, A, B, s)
    for name, got, ref in (("dA", dA, dA_ref), ("dB", dB, dB_ref)):
        emax, efro = gemm_errors(si.bf16_bits_to_f32(bits(got)), ref)
        assert emax <= MAX_TOL and efro <= FRO_TOL, (name, emax, efro)

    sse, res = lw.lowra_quant_error(layout, dev(case.W), maps, dev(case.thr), want_residual=True)
    sse_ref, res_ref = oracle.quant_error(case.W, case.precs, case.maps, case.thr)
    assert np.array_equal(res.cpu().numpy().view(np.uint32), res_ref.view(np.uint32))
    assert np.all(np.abs(sse.cpu().numpy() - sse_ref) <= 2.0 ** -21 * sse_ref)
