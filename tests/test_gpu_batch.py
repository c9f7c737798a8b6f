"""Several weights of one shape in one launch (lowra_lora_forward_batch / lowra_lora_backward_input_batch): every member is
held against the fp64 oracle and against a single call on that weight - bit for bit where no tile is cut between SMs
(the same products added up in the same order); where tiles are cut, the batch cuts them elsewhere than a single call
does, fp32 partial sums are added in another order, and a few outputs may differ by one rounding of bf16."""
import numpy as np
import pytest
import torch

import oracle
import synth_inputs as si
from helpers import FRO_TOL, MAX_TOL, gemm_errors, make_case

pytestmark = pytest.mark.gpu


def _dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def _bf(bits):
    return _dev(bits.view(np.int16)).view(torch.bfloat16)


def _bits(t):
    return t.view(torch.int16).cpu().numpy().view(np.uint16)


@pytest.mark.parametrize("N,K,M,r,count,mixes,shared_x,cut", [
    (256, 384, 300, 32, 3, [{1: 0.3, 2: 0.5, 4: 0.2}] * 3, True, False),                   # q, k, v: one input, three weights
    (640, 1152, 515, 96, 2, [{1: 0.6, 2: 0.35, 4: 0.05}, {1: 0.85, 2: 0.15}], False, False),   # one member without 4-bit rows
    (320, 640, 770, 48, 4, [{1: 1.0}, {2: 1.0}, {1: 0.5, 2: 0.5}, {1: 0.9, 2: 0.1}], False, False),   # none has 4-bit rows: six weight slots
    (1800, 2304, 4300, 80, 3, [{1: 0.4, 2: 0.4, 4: 0.2}] * 3, True, True),                 # tiles cut between SMs, ranges across members
    (4096, 4096, 2048, 64, 3, [{1: 0.6, 2: 0.35, 4: 0.05}] * 3, True, True),               # q, k, v of a 7B layer
])
def test_batch_members_equal_single_calls_and_the_oracle(N, K, M, r, count, mixes, shared_x, cut):
    import paper_2502_08141_b200 as lw

    s = 2.0
    cases = [make_case(N, K, mixes[i], matrix_id=90 + i, lloyd_iters=2) for i in range(count)]
    layouts = [lw.Layout(c.precs, K).build_deal() for c in cases]
    Xs = [si.activations(M, K, matrix_id=95 + (0 if shared_x else i)) for i in range(count)]
    dYs = [si.out_grads(M, N, matrix_id=95 + i) for i in range(count)]
    ABs = [si.lora_factors(K, N, r, matrix_id=90 + i) for i in range(count)]
    X_d = [_bf(Xs[0])] * count if shared_x else [_bf(x) for x in Xs]
    ws = lw.lowra_workspace_init(torch.empty(lw.lowra_batch_workspace_bytes(layouts[0], count, M, r), dtype=torch.uint8, device="cuda"))
    ws1 = lw.lowra_workspace_init(torch.empty(lw.lowra_workspace_bytes(layouts[0], M, r), dtype=torch.uint8, device="cuda"))
    rows = np.unique(np.linspace(0, M - 1, min(M, 64)).astype(np.int64))
    idx = torch.from_numpy(rows).cuda()
    for backward in (False, True):
        members = []
        for i, c in enumerate(cases):
            members.append(dict(layout=layouts[i], packed=_dev(c.packed), absmax=_dev(c.absmax), maps=_dev(c.maps),
                                act=_bf(dYs[i]) if backward else X_d[i], A=_bf(ABs[i][0]), B=_bf(ABs[i][1]),
                                out=torch.full((M, K if backward else N), float("nan"), dtype=torch.bfloat16, device="cuda")))
        fn = lw.lowra_lora_backward_input_batch if backward else lw.lowra_lora_forward_batch
        for rep in range(2):                                    # twice: the workspace numbers its calls
            outs = fn(members, s, ws)
            assert lw.lowra_device_status(ws) == lw.LOWRA_OK
        for i, (c, m) in enumerate(zip(cases, members)):
            if backward:
                one = lw.lowra_lora_backward_input(layouts[i], m["packed"], m["absmax"], m["maps"], m["act"], m["A"], m["B"], s, workspace=ws1)
                ref = oracle.lora_backward_input(c.W_hat, dYs[i][rows], ABs[i][0], ABs[i][1], s)
            else:
                one = lw.lowra_lora_forward(layouts[i], m["packed"], m["absmax"], m["maps"], m["act"], m["A"], m["B"], s, workspace=ws1)
                ref = oracle.lora_forward(c.W_hat, Xs[i][rows], ABs[i][0], ABs[i][1], s)
            assert lw.lowra_device_status(ws1) == lw.LOWRA_OK
            if cut:
                a, b = outs[i].float(), one.float()
                assert (a - b).abs().max().item() <= 2.0 ** -7 * b.abs().max().item(), (backward, i)     # a bf16 rounding step at most
                assert (outs[i].view(torch.int16) != one.view(torch.int16)).float().mean().item() < 0.05, (backward, i)
            else:
                assert torch.equal(outs[i].view(torch.int16), one.view(torch.int16)), (backward, i)
            emax, efro = gemm_errors(si.bf16_bits_to_f32(_bits(outs[i][idx])), ref)
            assert emax <= MAX_TOL and efro <= FRO_TOL, (backward, i, emax, efro)


def test_batch_arguments_are_validated():
    import paper_2502_08141_b200 as lw

    N, K, M, r = 128, 128, 40, 16
    z = lambda *shape, dt=torch.bfloat16: torch.zeros(shape, dtype=dt, device="cuda")
    def member(layout, n=N, k=K):
        return dict(layout=layout, packed=z(max(layout.packed_bytes, 16), dt=torch.uint8), absmax=z(n, k // 64, dt=torch.float32),
                    maps=z(n, 16, dt=torch.float32), act=z(M, k), A=z(k, r), B=z(r, n), out=z(M, n))
    dealt = lw.Layout(np.full(N, 2, np.uint8), K).build_deal()
    plain = lw.Layout(np.full(N, 2, np.uint8), K)
    other = lw.Layout(np.full(256, 2, np.uint8), K).build_deal()
    ws = lw.lowra_workspace_init(z(lw.lowra_batch_workspace_bytes(other, 4, M, r), dt=torch.uint8))
    with pytest.raises(lw.LowraError) as e:
        lw.lowra_lora_forward_batch([member(dealt), member(plain)], 1.0, ws)          # a member without a deal
    assert e.value.code == lw.LOWRA_ERR_NULL
    with pytest.raises(lw.LowraError) as e:
        lw.lowra_lora_forward_batch([member(dealt), member(other, n=256)], 1.0, ws)   # two shapes
    assert e.value.code == lw.LOWRA_ERR_SHAPE
    with pytest.raises(lw.LowraError) as e:
        lw.lowra_lora_forward_batch([member(dealt)] * 5, 1.0, ws)                     # more than LOWRA_MAX_BATCH
    assert e.value.code == lw.LOWRA_ERR_SHAPE
    with pytest.raises(lw.LowraError) as e:
        lw.lowra_lora_forward_batch([member(dealt)] * 2, 1.0, ws[:4096])              # workspace too small
    assert e.value.code == lw.LOWRA_ERR_WORKSPACE
