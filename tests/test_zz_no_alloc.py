"""The entry point for callers that cannot allocate device memory (lowra_lora_forward_static).

Some users of the library run where cudaMalloc is off limits - inside another application's CUDA
context, or in a loop whose memory was fixed at start-up - so this variant keeps its scratch in a
fixed array inside the library.  The tests call it through the C ABI several times in a row and compare
each result with the regular entry point (which gets its scratch from the caller): the two must
agree within the tolerance used for the fused products, and in fact bit for bit; the result is also
held against the fp64 oracle, and the free device memory is read before and after the calls to see
that they really allocate nothing.

Collected last on purpose (file name), and written to pass both alone and after the other tests.
"""
import numpy as np
import pytest
import torch

import synth_inputs as si

pytestmark = pytest.mark.gpu


def _bf(bits):
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)


def _problem():
    import paper_2502_08141_b200 as lw

    N, K, r = 640, 1152, 32
    precs = si.precisions(N, {1: 0.5, 2: 0.3, 4: 0.2}, matrix_id=77)
    maps, thr = si.standin_codebooks(precs, matrix_id=77)
    layout = lw.Layout(precs, K)
    W = si.weights(N, K, matrix_id=77)
    packed, absmax = lw.lowra_encode(layout, torch.from_numpy(W).cuda(), torch.from_numpy(thr).cuda())
    A_bits, B_bits = si.lora_factors(K, N, r, matrix_id=77)
    return dict(N=N, K=K, r=r, s=2.0, precs=precs, maps=maps, thr=thr, W=W, layout=layout, packed=packed, absmax=absmax,
                maps_d=torch.from_numpy(maps).cuda(), A_bits=A_bits, B_bits=B_bits, A=_bf(A_bits), B=_bf(B_bits))


def _agree(got, want):
    from helpers import FRO_TOL, MAX_TOL
    g, w = got.float().cpu().numpy().astype(np.float64), want.float().cpu().numpy().astype(np.float64)
    assert np.isfinite(g).all()
    assert np.abs(g - w).max() <= MAX_TOL * np.abs(w).max()
    assert np.linalg.norm(g - w) <= FRO_TOL * np.linalg.norm(w)
    assert torch.equal(got.view(torch.int16), want.view(torch.int16))


def test_static_scratch_forward_matches_regular_forward_twice():
    import oracle
    import paper_2502_08141_b200 as lw
    from helpers import FRO_TOL, MAX_TOL, gemm_errors

    p = _problem()
    N, K, r, s, layout = p["N"], p["K"], p["r"], p["s"], p["layout"]
    status = torch.full((1,), 123, dtype=torch.int32, device="cuda")
    # the oracle's own encode -> decode of the same weight (the packed bytes are compared on the way)
    packed_ref, absmax_ref = oracle.encode(p["W"], p["precs"], p["thr"])
    assert np.array_equal(p["packed"].cpu().numpy()[:layout.packed_bytes], packed_ref)
    what_ref = oracle.decode(packed_ref, absmax_ref, p["maps"], p["precs"], K)

    for call, M in enumerate((300, 77)):           # two calls in a row; the second leaves stale scratch behind it
        X_bits = si.activations(M, K, matrix_id=200 + call)
        X = _bf(X_bits)
        ws = torch.empty(lw.lowra_workspace_bytes(layout, M, r), dtype=torch.uint8, device="cuda")
        want = lw.lowra_lora_forward(layout, p["packed"], p["absmax"], p["maps_d"], X, p["A"], p["B"], s, workspace=ws)
        assert lw.lowra_device_status(ws) == lw.LOWRA_OK
        got = torch.full((M, N), float("nan"), dtype=torch.bfloat16, device="cuda")
        lw.lowra_lora_forward_static(layout, p["packed"], p["absmax"], p["maps_d"], X, p["A"], p["B"], s, Y=got, status_out=status)
        torch.cuda.synchronize()
        assert int(status.item()) == lw.LOWRA_OK
        _agree(got, want)
        ref = oracle.lora_forward(what_ref, X_bits, p["A_bits"], p["B_bits"], s)
        emax, efro = gemm_errors(si.bf16_bits_to_f32(got.view(torch.int16).cpu().numpy().view(np.uint16)), ref)
        assert emax <= MAX_TOL and efro <= FRO_TOL, (M, emax, efro)


def test_static_scratch_calls_allocate_nothing():
    """Free device memory is the same before and after a run of calls (taken after a first call, which makes the
    driver load the kernels' code; outputs and the status word are the caller's and exist beforehand)."""
    import paper_2502_08141_b200 as lw

    p = _problem()
    N, K, s, layout = p["N"], p["K"], p["s"], p["layout"]
    dealt = lw.Layout(p["precs"], K).build_deal()
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    Xs = [_bf(si.activations(M, K, matrix_id=210 + i)) for i, M in enumerate((300, 77, 512))]
    Ys = [torch.empty((x.shape[0], N), dtype=torch.bfloat16, device="cuda") for x in Xs]
    for lay in (layout, dealt):                    # first calls: code loading, address look-up of the built-in array
        lw.lowra_lora_forward_static(lay, p["packed"], p["absmax"], p["maps_d"], Xs[0], p["A"], p["B"], s, Y=Ys[0], status_out=status)
    torch.cuda.synchronize()
    free_before, _ = torch.cuda.mem_get_info()
    for _ in range(3):
        for lay in (layout, dealt):
            for X, Y in zip(Xs, Ys):
                lw.lowra_lora_forward_static(lay, p["packed"], p["absmax"], p["maps_d"], X, p["A"], p["B"], s, Y=Y, status_out=status)
    torch.cuda.synchronize()
    free_after, _ = torch.cuda.mem_get_info()
    assert free_after == free_before
    assert int(status.item()) == lw.LOWRA_OK


def test_static_scratch_with_rows_dealt_once_per_weight():
    """The same two calls in a row on a layout that carries a deal (no prologue launch: the flags in the shared array
    are told apart by the calls' numbers), then dealt and undealt calls mixed: always bit-identical to the regular
    entry point, and the status word handed back is the call's own."""
    import paper_2502_08141_b200 as lw

    p = _problem()
    N, K, r, s, layout = p["N"], p["K"], p["r"], p["s"], p["layout"]
    dealt = lw.Layout(p["precs"], K).build_deal()
    status = torch.full((1,), 123, dtype=torch.int32, device="cuda")
    sequence = [(dealt, 300), (dealt, 77), (layout, 300), (dealt, 515), (layout, 77), (dealt, 300)]
    for call, (lay, M) in enumerate(sequence):
        X = _bf(si.activations(M, K, matrix_id=220 + call))
        ws = torch.empty(lw.lowra_workspace_bytes(layout, M, r), dtype=torch.uint8, device="cuda")
        want = lw.lowra_lora_forward(layout, p["packed"], p["absmax"], p["maps_d"], X, p["A"], p["B"], s, workspace=ws)
        assert lw.lowra_device_status(ws) == lw.LOWRA_OK
        got = torch.full((M, N), float("nan"), dtype=torch.bfloat16, device="cuda")
        status.fill_(123)
        lw.lowra_lora_forward_static(lay, p["packed"], p["absmax"], p["maps_d"], X, p["A"], p["B"], s, Y=got, status_out=status)
        torch.cuda.synchronize()
        assert int(status.item()) == lw.LOWRA_OK, call
        _agree(got, want)


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
