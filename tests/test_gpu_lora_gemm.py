"""GPU parity of the fused dequant + LoRA products against the fp64 oracle, through the C ABI.

Acceptance (both must hold, for Y and for dX):
    max |Y - Y_ref|  <= 1e-2 * max |Y_ref|
    ||Y - Y_ref||_F  <= 5e-3 * ||Y_ref||_F
"""
import numpy as np
import pytest
import torch

import oracle
import synth_inputs as si
from helpers import FRO_TOL, MAX_TOL, gemm_errors, make_case

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def lw():
    import paper_2502_08141_b200 as lw
    return lw


def _dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def _bf(a_bits):
    return _dev(a_bits.view(np.int16)).view(torch.bfloat16)


def _bits(t):
    return t.view(torch.int16).cpu().numpy().view(np.uint16)


def test_dense_pipeline_matches_fp64(lw):
    """The tensor-core pipeline alone (TMA -> smem -> tcgen05 -> TMEM -> epilogue), no dequant."""
    for M, N, K in ((256, 128, 64), (300, 200, 256), (1024, 640, 1024)):
        P = si.bf16_normal((M, K), 1.0, stream=40)
        Q = si.bf16_normal((N, K), 1.0, stream=41)
        C = lw.lowra_dense_nt(_bf(P), _bf(Q))
        ws = torch.zeros(256, dtype=torch.uint8, device="cuda")
        C = lw.lowra_dense_nt(_bf(P), _bf(Q), workspace=ws)
        assert lw.lowra_device_status(ws) == lw.LOWRA_OK
        ref = oracle.bf16_to_f64(P) @ oracle.bf16_to_f64(Q).T
        emax, efro = gemm_errors(si.bf16_bits_to_f32(_bits(C)), ref)
        assert emax <= MAX_TOL and efro <= FRO_TOL, (M, N, K, emax, efro)


GEMM_CASES = [
    # N, K, M, r, mix, kind
    (512, 512, 16, 16, {1: 0.5, 2: 0.5}, "tiny"),                  # config 1
    (256, 384, 300, 32, {1: 0.3, 2: 0.5, 4: 0.2}, "llama"),         # ragged tokens, K = 3 * 128
    (200, 256, 64, 16, {1: 0.34, 2: 0.33, 4: 0.33}, "llama"),       # N not a multiple of 64
    (640, 1152, 515, 96, {1: 0.6, 2: 0.35, 4: 0.05}, "llama"),      # rank above 64, several tiles each way
    (384, 256, 257, 128, {4: 1.0}, "llama"),                        # 4-bit only, maximum rank
    (320, 640, 770, 48, {1: 0.5, 2: 0.3, 4: 0.2}, "llama"),         # odd number of 64-channel groups (the CTAs of a
                                                                    # cluster take them in turn), four token tiles
    (4096, 4096, 2048, 64, {1: 0.3, 2: 0.5, 4: 0.2}, "llama"),      # config 2
    (1800, 2304, 7500, 80, {1: 0.4, 2: 0.4, 4: 0.2}, "llama"),      # 240 / 285 tiles on 74 clusters: both passes cut the
                                                                    # contraction of some tiles between clusters; ragged
                                                                    # channels and tokens, two LoRA blocks
]


@pytest.mark.parametrize("N,K,M,r,mix,kind", GEMM_CASES)
def test_forward_and_backward_input(lw, N, K, M, r, mix, kind):
    case = make_case(N, K, mix, matrix_id=(N + K) % 89, kind=kind)
    layout = lw.Layout(case.precs, K)
    X = si.activations(M, K, matrix_id=3)
    dY = si.out_grads(M, N, matrix_id=3)
    A, B = si.lora_factors(K, N, r, matrix_id=3)
    s = 2.0
    packed, absmax, maps = _dev(case.packed), _dev(case.absmax), _dev(case.maps)
    ws = torch.empty(lw.lowra_workspace_bytes(layout, M, r), dtype=torch.uint8, device="cuda")

    Y = torch.full((M, N), float("nan"), dtype=torch.bfloat16, device="cuda")
    lw.lowra_lora_forward(layout, packed, absmax, maps, _bf(X), _bf(A), _bf(B), s, Y=Y, workspace=ws)
    assert lw.lowra_device_status(ws) == lw.LOWRA_OK
    Y_ref = oracle.lora_forward(case.W_hat, X, A, B, s)
    emax, efro = gemm_errors(si.bf16_bits_to_f32(_bits(Y)), Y_ref)
    assert emax <= MAX_TOL and efro <= FRO_TOL, ("forward", emax, efro)

    dX = torch.full((M, K), float("nan"), dtype=torch.bfloat16, device="cuda")
    lw.lowra_lora_backward_input(layout, packed, absmax, maps, _bf(dY), _bf(A), _bf(B), s, dX=dX, workspace=ws)
    assert lw.lowra_device_status(ws) == lw.LOWRA_OK
    dX_ref = oracle.lora_backward_input(case.W_hat, dY, A, B, s)
    emax, efro = gemm_errors(si.bf16_bits_to_f32(_bits(dX)), dX_ref)
    assert emax <= MAX_TOL and efro <= FRO_TOL, ("backward", emax, efro)


@pytest.mark.parametrize("N,K,M,r", [(256, 256, 128, 64), (640, 1152, 515, 96), (128, 1152, 256, 128),
                                     (1024, 2048, 700, 64)])
def test_lora_term_is_really_there(lw, N, K, M, r):
    """With large LoRA factors the low-rank term dominates: a path that dropped it, applied the wrong
    scale, or picked up a stale operand tile (long contractions, several LoRA blocks, several tiles per
    CTA) would fail by far.  Both directions."""
    case = make_case(N, K, {1: 0.5, 2: 0.3, 4: 0.2}, matrix_id=5)
    layout = lw.Layout(case.precs, K)
    X = si.activations(M, K, matrix_id=9)
    dY = si.out_grads(M, N, matrix_id=9)
    A = si.bf16_normal((K, r), 0.5, stream=50)
    B = si.bf16_normal((r, N), 0.5, stream=51)
    packed, absmax, maps = _dev(case.packed), _dev(case.absmax), _dev(case.maps)
    for s in (0.0, 0.25, -3.0):
        Y = lw.lowra_lora_forward(layout, packed, absmax, maps, _bf(X), _bf(A), _bf(B), s)
        dX = lw.lowra_lora_backward_input(layout, packed, absmax, maps, _bf(dY), _bf(A), _bf(B), s)
        torch.cuda.synchronize()
        ref = oracle.lora_forward(case.W_hat, X, A, B, s)
        emax, efro = gemm_errors(si.bf16_bits_to_f32(_bits(Y)), ref)
        assert emax <= MAX_TOL and efro <= FRO_TOL, ("forward", s, emax, efro)
        ref = oracle.lora_backward_input(case.W_hat, dY, A, B, s)
        emax, efro = gemm_errors(si.bf16_bits_to_f32(_bits(dX)), ref)
        assert emax <= MAX_TOL and efro <= FRO_TOL, ("backward", s, emax, efro)


def test_fused_weights_equal_decoded_weights(lw):
    """X = identity, s = 0: the forward output is deq(Wq)^T itself, so every element must be the
    bf16 value that lowra_decode produces (exact: one product term, fp32 accumulate, bf16 store)."""
    N, K = 384, 256
    case = make_case(N, K, {1: 0.3, 2: 0.4, 4: 0.3}, matrix_id=6)
    layout = lw.Layout(case.precs, K)
    eye = si.f32_to_bf16_bits(np.eye(K, dtype=np.float32))
    A = np.zeros((K, 16), np.uint16)
    B = np.zeros((16, N), np.uint16)
    Y = lw.lowra_lora_forward(layout, _dev(case.packed), _dev(case.absmax), _dev(case.maps),
                              _bf(eye), _bf(A), _bf(B), 0.0)
    torch.cuda.synchronize()
    assert np.array_equal(_bits(Y), case.W_hat.T)
    eyeN = si.f32_to_bf16_bits(np.eye(N, dtype=np.float32))
    dX = lw.lowra_lora_backward_input(layout, _dev(case.packed), _dev(case.absmax), _dev(case.maps),
                                      _bf(eyeN), _bf(A), _bf(B), 0.0)
    torch.cuda.synchronize()
    assert np.array_equal(_bits(dX), case.W_hat)
