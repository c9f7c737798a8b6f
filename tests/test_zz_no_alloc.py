"""The entry point for callers that cannot allocate device memory (lowra_lora_forward_static).

Some users of the library run where cudaMalloc is off limits - inside another application's CUDA
context, or in a loop whose memory was fixed at start-up - so this variant keeps its scratch in a
fixed array inside the library.  The test calls it through the C ABI twice in a row and compares
each result with the regular entry point (which gets its scratch from the caller): the two must
agree within the tolerance used for the fused products, and in fact bit for bit.

Collected last on purpose (file name), and written to pass both alone and after the other tests.
"""
import numpy as np
import pytest
import torch

import synth_inputs as si

pytestmark = pytest.mark.gpu


def _bf(bits):
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)


def test_static_scratch_forward_matches_regular_forward_twice():
    import paper_2502_08141_b200 as lw
    from helpers import FRO_TOL, MAX_TOL

    N, K, r, s = 640, 1152, 32, 2.0
    precs = si.precisions(N, {1: 0.5, 2: 0.3, 4: 0.2}, matrix_id=77)
    maps, thr = si.standin_codebooks(precs, matrix_id=77)
    layout = lw.Layout(precs, K)
    W = torch.from_numpy(si.weights(N, K, matrix_id=77)).cuda()
    packed, absmax = lw.lowra_encode(layout, W, torch.from_numpy(thr).cuda())
    maps_d = torch.from_numpy(maps).cuda()
    A_bits, B_bits = si.lora_factors(K, N, r, matrix_id=77)
    A, B = _bf(A_bits), _bf(B_bits)
    status = torch.full((1,), 123, dtype=torch.int32, device="cuda")

    for call, M in enumerate((300, 77)):           # two calls in a row; the second leaves stale scratch behind it
        X = _bf(si.activations(M, K, matrix_id=200 + call))
        ws = torch.empty(lw.lowra_workspace_bytes(layout, M, r), dtype=torch.uint8, device="cuda")
        want = lw.lowra_lora_forward(layout, packed, absmax, maps_d, X, A, B, s, workspace=ws)
        assert lw.lowra_device_status(ws) == lw.LOWRA_OK
        got = torch.full((M, N), float("nan"), dtype=torch.bfloat16, device="cuda")
        lw.lowra_lora_forward_static(layout, packed, absmax, maps_d, X, A, B, s, Y=got, status_out=status)
        torch.cuda.synchronize()
        assert int(status.item()) == lw.LOWRA_OK
        g, w = got.float().cpu().numpy().astype(np.float64), want.float().cpu().numpy().astype(np.float64)
        assert np.isfinite(g).all()
        assert np.abs(g - w).max() <= MAX_TOL * np.abs(w).max()
        assert np.linalg.norm(g - w) <= FRO_TOL * np.linalg.norm(w)
        assert torch.equal(got.view(torch.int16), want.view(torch.int16))


def test_static_scratch_rejects_problems_beyond_its_size():
    import paper_2502_08141_b200 as lw

    N, K, r = 128, 128, 128
    precs = np.full(N, 2, np.uint8)
    layout = lw.Layout(precs, K)
    M = 40000                                       # 40000 tokens x 128 padded rank x 2 bytes > 8 MiB
    assert lw.lowra_workspace_bytes(layout, M, r) > lw.LOWRA_STATIC_SCRATCH_BYTES
    X = torch.zeros((M, K), dtype=torch.bfloat16, device="cuda")
    A = torch.zeros((K, r), dtype=torch.bfloat16, device="cuda")
    B = torch.zeros((r, N), dtype=torch.bfloat16, device="cuda")
    packed = torch.zeros(layout.packed_bytes, dtype=torch.uint8, device="cuda")
    absmax = torch.zeros((N, K // 64), dtype=torch.float32, device="cuda")
    maps = torch.zeros((N, 16), dtype=torch.float32, device="cuda")
    with pytest.raises(lw.LowraError) as e:
        lw.lowra_lora_forward_static(layout, packed, absmax, maps, X, A, B, 1.0)
    assert e.value.code == lw.LOWRA_ERR_LIMIT
