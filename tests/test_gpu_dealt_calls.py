"""Fused calls on a layout that carries its row deal (lowra_deal_build) and a workspace that numbers its calls
(lowra_workspace_init): no prologue launch, no clearing of flags between calls.

The deal and the schedule are the same as in a call that works the deal out itself, so the results must be
bit-identical to such a call; one case per test is also held against the fp64 oracle.  The sequences below
leave flags of earlier calls behind on purpose (larger token counts first, other weights, the other
direction) - a flag that still read as "up" would let a tile run ahead of the data it waits for.
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


class _Weight:
    def __init__(self, lw, N, K, r, mix, mid):
        self.case = make_case(N, K, mix, matrix_id=mid, lloyd_iters=1)
        self.N, self.K, self.r = N, K, r
        self.plain = lw.Layout(self.case.precs, K)
        self.dealt = lw.Layout(self.case.precs, K).build_deal()
        self.packed, self.absmax, self.maps = _dev(self.case.packed), _dev(self.case.absmax), _dev(self.case.maps)
        self.A_bits = si.bf16_normal((K, r), 0.02, stream=300 + mid)
        self.B_bits = si.bf16_normal((r, N), 0.02, stream=400 + mid)
        self.A, self.B = _bf(self.A_bits), _bf(self.B_bits)

    def forward(self, lw, layout, X, ws):
        Y = torch.full((X.shape[0], self.N), float("nan"), dtype=torch.bfloat16, device="cuda")
        lw.lowra_lora_forward(layout, self.packed, self.absmax, self.maps, X, self.A, self.B, 1.5, Y=Y, workspace=ws)
        return Y

    def backward(self, lw, layout, dY, ws):
        dX = torch.full((dY.shape[0], self.K), float("nan"), dtype=torch.bfloat16, device="cuda")
        lw.lowra_lora_backward_input(layout, self.packed, self.absmax, self.maps, dY, self.A, self.B, 1.5, dX=dX, workspace=ws)
        return dX


SHAPES = [
    # N, K, M, r, mix
    (512, 512, 16, 16, {1: 0.5, 2: 0.5}),
    (200, 256, 300, 32, {1: 0.34, 2: 0.33, 4: 0.33}),               # ragged channels and tokens
    (1800, 2304, 7500, 80, {1: 0.4, 2: 0.4, 4: 0.2}),               # tiles cut between clusters in both directions
    (4096, 4096, 2048, 64, {1: 0.6, 2: 0.35, 4: 0.05}),             # partial tiles preloaded into the accumulator
]


@pytest.mark.parametrize("N,K,M,r,mix", SHAPES)
def test_dealt_call_equals_call_with_prologue(lw, N, K, M, r, mix):
    w = _Weight(lw, N, K, r, mix, mid=(N + K + M) % 97)
    X_bits, dY_bits = si.activations(M, K, matrix_id=5), si.out_grads(M, N, matrix_id=6)
    X, dY = _bf(X_bits), _bf(dY_bits)
    ws_plain = torch.empty(lw.lowra_workspace_bytes(w.plain, M, r), dtype=torch.uint8, device="cuda")
    ws = lw.lowra_workspace_init(torch.empty_like(ws_plain).fill_(0xA5))
    Y_ref, dX_ref = w.forward(lw, w.plain, X, ws_plain), w.backward(lw, w.plain, dY, ws_plain)
    assert lw.lowra_device_status(ws_plain) == lw.LOWRA_OK
    for rep in range(3):   # call numbers 1, 2, ... on the same workspace
        Y = w.forward(lw, w.dealt, X, ws)
        dX = w.backward(lw, w.dealt, dY, ws)
        assert torch.equal(Y.view(torch.int16), Y_ref.view(torch.int16)), rep
        assert torch.equal(dX.view(torch.int16), dX_ref.view(torch.int16)), rep
    assert lw.lowra_device_status(ws) == lw.LOWRA_OK
    if M * N <= 1 << 22:
        e = gemm_errors(si.bf16_bits_to_f32(_bits(Y)), oracle.lora_forward(w.case.W_hat, X_bits, w.A_bits, w.B_bits, 1.5))
        assert e[0] <= MAX_TOL and e[1] <= FRO_TOL, e
        e = gemm_errors(si.bf16_bits_to_f32(_bits(dX)), oracle.lora_backward_input(w.case.W_hat, dY_bits, w.A_bits, w.B_bits, 1.5))
        assert e[0] <= MAX_TOL and e[1] <= FRO_TOL, e


def test_one_workspace_serves_many_weights_and_token_counts(lw):
    """Two weights, three token counts (the largest first), both directions and both kinds of call in turn on one
    workspace: every result equals the one of a call with a prologue on a workspace of its own."""
    weights = [_Weight(lw, 1152, 1024, 64, {1: 0.6, 2: 0.35, 4: 0.05}, mid=11),
               _Weight(lw, 2304, 1792, 48, {2: 0.75, 4: 0.25}, mid=12)]
    tokens = [6000, 700, 2500]
    need = max(lw.lowra_workspace_bytes(w.plain, m, w.r) for w in weights for m in tokens)
    ws = lw.lowra_workspace_init(torch.empty(need, dtype=torch.uint8, device="cuda"))
    ws_plain = torch.empty(need, dtype=torch.uint8, device="cuda")
    acts = {(i, m): (_bf(si.activations(m, w.K, matrix_id=20 + i)), _bf(si.out_grads(m, w.N, matrix_id=30 + i)))
            for i, w in enumerate(weights) for m in tokens}
    ref = {}
    for (i, m), (X, dY) in acts.items():
        ref[(i, m)] = (weights[i].forward(lw, weights[i].plain, X, ws_plain),
                       weights[i].backward(lw, weights[i].plain, dY, ws_plain))
    step = 0
    for rnd in range(2):
        for m in tokens:
            for i, w in enumerate(weights):
                X, dY = acts[(i, m)]
                # every third call works its deal out itself, on the same workspace
                lay_f = w.plain if step % 3 == 2 else w.dealt
                lay_b = w.plain if step % 3 == 1 else w.dealt
                Y = w.forward(lw, lay_f, X, ws)
                dX = w.backward(lw, lay_b, dY, ws)
                assert torch.equal(Y.view(torch.int16), ref[(i, m)][0].view(torch.int16)), (rnd, m, i)
                assert torch.equal(dX.view(torch.int16), ref[(i, m)][1].view(torch.int16)), (rnd, m, i)
                step += 1
    assert lw.lowra_device_status(ws) == lw.LOWRA_OK


def test_deal_buffer_is_what_the_prologue_writes(lw):
    """The deal in the caller's buffer is byte for byte what a call's prologue leaves in the workspace (same kernel,
    same arguments): checked through the results of a call whose layout is switched between the two on a weight
    with every kind of ragged edge, and through the buffer being untouched by the calls."""
    w = _Weight(lw, 1000, 640, 16, {1: 0.5, 2: 0.3, 4: 0.2}, mid=3)
    before = w.dealt.deal.clone()
    M = 515
    X, dY = _bf(si.activations(M, w.K, matrix_id=1)), _bf(si.out_grads(M, w.N, matrix_id=2))
    ws = lw.lowra_workspace_init(torch.empty(lw.lowra_workspace_bytes(w.plain, M, w.r), dtype=torch.uint8, device="cuda"))
    a = (w.forward(lw, w.dealt, X, ws), w.backward(lw, w.dealt, dY, ws))
    b = (w.forward(lw, w.plain, X, ws), w.backward(lw, w.plain, dY, ws))
    assert torch.equal(a[0].view(torch.int16), b[0].view(torch.int16))
    assert torch.equal(a[1].view(torch.int16), b[1].view(torch.int16))
    assert torch.equal(before, w.dealt.deal)
    assert lw.lowra_device_status(ws) == lw.LOWRA_OK


def test_call_numbering_wraps(lw):
    """The number of the last call sits at byte 64 of the workspace.  Started three calls before the 32-bit wrap, the
    calls that cross it (the call with the last number clears the flags on its way out and the count restarts) give
    the same results as ever."""
    w = _Weight(lw, 1800, 2304, 80, {1: 0.4, 2: 0.4, 4: 0.2}, mid=9)
    M = 7500
    X, dY = _bf(si.activations(M, w.K, matrix_id=5)), _bf(si.out_grads(M, w.N, matrix_id=6))
    ws_plain = torch.empty(lw.lowra_workspace_bytes(w.plain, M, w.r), dtype=torch.uint8, device="cuda")
    Y_ref, dX_ref = w.forward(lw, w.plain, X, ws_plain), w.backward(lw, w.plain, dY, ws_plain)
    ws = lw.lowra_workspace_init(torch.empty_like(ws_plain))
    ws[64:68].view(torch.int32)[0] = -4          # 0xFFFFFFFC: the next calls are numbered ...FD, ...FE, ...FF, 1, 2, 3
    seen = []
    for rep in range(3):
        Y = w.forward(lw, w.dealt, X, ws)
        seen.append(int(ws[64:68].view(torch.int32)[0].item()) & 0xFFFFFFFF)
        dX = w.backward(lw, w.dealt, dY, ws)
        seen.append(int(ws[64:68].view(torch.int32)[0].item()) & 0xFFFFFFFF)
        assert torch.equal(Y.view(torch.int16), Y_ref.view(torch.int16)), rep
        assert torch.equal(dX.view(torch.int16), dX_ref.view(torch.int16)), rep
    assert seen == [0xFFFFFFFD, 0xFFFFFFFE, 0, 1, 2, 3], seen
    assert int(ws[128:132].view(torch.int32)[0].item()) == 0    # the count of CTAs that have left is back at zero
    assert lw.lowra_device_status(ws) == lw.LOWRA_OK
