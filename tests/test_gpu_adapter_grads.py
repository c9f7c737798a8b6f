"""GPU parity of the gradients of the low-rank factors against the fp64 oracle, through the C ABI.

Acceptance, the same as for the other products (both must hold, for dA and for dB):
    max |G - G_ref|  <= 1e-2 * max |G_ref|
    ||G - G_ref||_F  <= 5e-3 * ||G_ref||_F
"""
import numpy as np
import pytest
import torch

import oracle
import synth_inputs as si
from helpers import FRO_TOL, MAX_TOL, gemm_errors

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def lw():
    import paper_2502_08141_b200 as lw
    return lw


def _bf(a_bits):
    return torch.from_numpy(np.ascontiguousarray(a_bits).view(np.int16)).cuda().view(torch.bfloat16)


def _bits(t):
    return t.view(torch.int16).cpu().numpy().view(np.uint16)


CASES = [
    # N, K, M, r
    (512, 512, 16, 16),        # fewer tokens than one pipeline stage
    (256, 384, 300, 32),       # ragged tokens
    (200, 264, 64, 16),        # N and K not multiples of 64
    (640, 1152, 515, 96),      # rank between 64 and 128
    (384, 256, 257, 128),      # maximum rank
    (320, 640, 770, 48),       # rank not a multiple of 32
    (4096, 4096, 2048, 64),    # config 2
]


@pytest.mark.parametrize("N,K,M,r", CASES)
def test_adapter_gradients(lw, N, K, M, r):
    X = si.activations(M, K, matrix_id=5)
    dY = si.out_grads(M, N, matrix_id=5)
    A, B = si.lora_factors(K, N, r, matrix_id=5)
    # the paper's initialisation leaves B at zero, which would make dA vanish: give B the spread of A
    B = si.bf16_normal((r, N), 0.02, stream=77)
    s = 2.0
    ws = torch.empty(lw.lowra_adapter_workspace_bytes(M, r), dtype=torch.uint8, device="cuda")
    dA = torch.full((K, r), float("nan"), dtype=torch.bfloat16, device="cuda")
    dB = torch.full((r, N), float("nan"), dtype=torch.bfloat16, device="cuda")
    lw.lowra_lora_backward_adapters(_bf(X), _bf(dY), _bf(A), _bf(B), s, dA=dA, dB=dB, workspace=ws)
    assert lw.lowra_device_status(ws) == lw.LOWRA_OK
    dA_ref, dB_ref = oracle.lora_backward_adapters(X, dY, A, B, s)
    for name, got, ref in (("dA", dA, dA_ref), ("dB", dB, dB_ref)):
        g = si.bf16_bits_to_f32(_bits(got))
        assert np.isfinite(g).all(), name
        emax, efro = gemm_errors(g, ref)
        assert emax <= MAX_TOL and efro <= FRO_TOL, (name, emax, efro)


def test_zero_upper_factor_gives_zero_dA(lw):
    """With B = 0 (the usual starting point) the gradient of A vanishes exactly; dB does not."""
    N, K, M, r = 256, 256, 128, 16
    X = si.activations(M, K, matrix_id=6)
    dY = si.out_grads(M, N, matrix_id=6)
    A = si.bf16_normal((K, r), 0.05, stream=78)
    B = np.zeros((r, N), dtype=np.uint16)
    dA, dB = lw.lowra_lora_backward_adapters(_bf(X), _bf(dY), _bf(A), _bf(B), 1.5)
    assert (_bits(dA) & 0x7FFF == 0).all()
    _, dB_ref = oracle.lora_backward_adapters(X, dY, A, B, 1.5)
    emax, efro = gemm_errors(si.bf16_bits_to_f32(_bits(dB)), dB_ref)
    assert emax <= MAX_TOL and efro <= FRO_TOL


def test_repeated_calls_are_bit_identical(lw):
    N, K, M, r = 384, 512, 700, 64
    X = _bf(si.activations(M, K, matrix_id=7))
    dY = _bf(si.out_grads(M, N, matrix_id=7))
    A = _bf(si.bf16_normal((K, r), 0.05, stream=79))
    B = _bf(si.bf16_normal((r, N), 0.05, stream=80))
    a1, b1 = lw.lowra_lora_backward_adapters(X, dY, A, B, 0.5)
    a2, b2 = lw.lowra_lora_backward_adapters(X, dY, A, B, 0.5)
    assert torch.equal(a1.view(torch.int16), a2.view(torch.int16))
    assert torch.equal(b1.view(torch.int16), b2.view(torch.int16))


@pytest.mark.parametrize("N,K,M,r", [(256, 384, 300, 32), (640, 1152, 515, 96), (4096, 4096, 2048, 64)])
def test_gradients_from_the_projections_the_fused_calls_left_behind(lw, N, K, M, r):
    """A training step runs forward and backward-input first; their workspaces then hold s X A and s dY B^T, and the
    factors' gradients need X and dY only once more (lowra_lora_backward_adapters_reuse).  Against the fp64 oracle
    (same bounds) and against the call that forms the projections itself (same values up to the order of fp32 sums
    inside the projections: a bf16 rounding step apart at most, almost all equal)."""
    from helpers import make_case

    s = 2.0
    case = make_case(N, K, {1: 0.5, 2: 0.3, 4: 0.2}, matrix_id=21, lloyd_iters=2)
    layout = lw.Layout(case.precs, K).build_deal()
    packed, absmax, maps = (torch.from_numpy(a).cuda() for a in (case.packed, case.absmax, case.maps))
    X, dY = si.activations(M, K, matrix_id=22), si.out_grads(M, N, matrix_id=22)
    A = si.bf16_normal((K, r), 0.01, stream=23)
    B = si.bf16_normal((r, N), 0.01, stream=24)      # as spread out as A, so that dA is not zero
    ws_f, ws_b = (lw.lowra_workspace_init(torch.empty(lw.lowra_workspace_bytes(layout, M, r), dtype=torch.uint8, device="cuda"))
                  for _ in range(2))
    lw.lowra_lora_forward(layout, packed, absmax, maps, _bf(X), _bf(A), _bf(B), s, workspace=ws_f)
    lw.lowra_lora_backward_input(layout, packed, absmax, maps, _bf(dY), _bf(A), _bf(B), s, workspace=ws_b)
    assert lw.lowra_device_status(ws_f) == lw.LOWRA_OK and lw.lowra_device_status(ws_b) == lw.LOWRA_OK
    T = lw.lowra_workspace_projection(ws_f, M, r)
    U = lw.lowra_workspace_projection(ws_b, M, r)
    # the projections themselves: s X A and s dY B^T, rounded to bf16 once; columns past the rank are zero
    Xd, dYd, Ad, Bd = (oracle.bf16_to_f64(a) for a in (X, dY, A, B))
    for got, ref in ((T, s * (Xd @ Ad)), (U, s * (dYd @ Bd.T))):
        g = si.bf16_bits_to_f32(_bits(got)).astype(np.float64)
        assert np.all(g[:, r:] == 0)
        assert np.abs(g[:, :r] - ref).max() <= 2.0 ** -8 * np.abs(ref).max() + 1e-30
    wsa = torch.empty(256, dtype=torch.uint8, device="cuda")
    dA, dB = lw.lowra_lora_backward_adapters_reuse(_bf(X), _bf(dY), T, U, r, workspace=wsa)
    assert lw.lowra_device_status(wsa) == lw.LOWRA_OK
    dA_ref, dB_ref = oracle.lora_backward_adapters(X, dY, A, B, s)
    dA2, dB2 = lw.lowra_lora_backward_adapters(_bf(X), _bf(dY), _bf(A), _bf(B), s)
    for name, got, ref, other in (("dA", dA, dA_ref, dA2), ("dB", dB, dB_ref, dB2)):
        emax, efro = gemm_errors(si.bf16_bits_to_f32(_bits(got)), ref)
        assert emax <= MAX_TOL and efro <= FRO_TOL, (name, emax, efro)
        a, b = got.float(), other.float()
        assert (a - b).abs().max().item() <= 2.0 ** -6 * b.abs().max().item(), name
