"""A whole layer step (encode, decode, forward, backward-input) captured into a CUDA graph and replayed.

Nothing in the calls depends on host state between launches: the tensor maps are kernel arguments, the row deal
and the numbering of the calls live in device memory.  So a captured step must replay with bit-identical results,
with and without a deal kept by the caller.
"""
import numpy as np
import pytest
import torch

import synth_inputs as si
from helpers import make_case

pytestmark = pytest.mark.gpu


def _dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def _bf(bits):
    return _dev(bits.view(np.int16)).view(torch.bfloat16)


@pytest.mark.parametrize("dealt", [False, True])
def test_layer_step_replays_from_a_graph(dealt):
    import paper_2502_08141_b200 as lw

    N, K, M, r = 1152, 1024, 700, 32
    case = make_case(N, K, {1: 0.5, 2: 0.3, 4: 0.2}, matrix_id=7, lloyd_iters=1)
    layout = lw.Layout(case.precs, K)
    if dealt:
        layout.build_deal()
    W, thr, maps = _dev(case.W), _dev(case.thr), _dev(case.maps)
    X, dY = _bf(si.activations(M, K, matrix_id=1)), _bf(si.out_grads(M, N, matrix_id=2))
    A, B = _bf(si.bf16_normal((K, r), 0.02, stream=5)), _bf(si.bf16_normal((r, N), 0.02, stream=6))
    ws = lw.lowra_workspace_init(torch.empty(lw.lowra_workspace_bytes(layout, M, r), dtype=torch.uint8, device="cuda"))
    packed = torch.empty(max(layout.packed_bytes, 16), dtype=torch.uint8, device="cuda")
    absmax = torch.empty((N, K // 64), dtype=torch.float32, device="cuda")
    What = torch.empty((N, K), dtype=torch.bfloat16, device="cuda")
    Y = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
    dX = torch.empty((M, K), dtype=torch.bfloat16, device="cuda")
    outs = (packed, absmax, What, Y, dX)

    def step():
        lw.lowra_encode(layout, W, thr, packed=packed, absmax=absmax)
        lw.lowra_decode(layout, packed, absmax, maps, out=What)
        lw.lowra_lora_forward(layout, packed, absmax, maps, X, A, B, 2.0, Y=Y, workspace=ws)
        lw.lowra_lora_backward_input(layout, packed, absmax, maps, dY, A, B, 2.0, dX=dX, workspace=ws)

    step()                                   # eager: the reference, and the one-time set-up of every kernel
    torch.cuda.synchronize()
    assert np.array_equal(packed.cpu().numpy()[:layout.packed_bytes], case.packed)
    ref = [t.clone() for t in outs]
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        step()
    torch.cuda.current_stream().wait_stream(side)
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        step()
    for rep in range(3):
        for t in outs:
            t.zero_()
        graph.replay()
        torch.cuda.synchronize()
        for a, b in zip(ref, outs):
            assert torch.equal(a.view(torch.uint8), b.view(torch.uint8)), rep
    assert lw.lowra_device_status(ws) == lw.LOWRA_OK
