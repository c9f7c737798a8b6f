"""GPU parity of the paper's natural row order: the conversion between it and the grouped order, and the kernels working
on a natural-order buffer directly - all bit-exact against the oracle's natural layout."""
import numpy as np
import pytest
import torch

import oracle
from helpers import make_case

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def lw():
    import paper_2502_08141_b200 as lw
    return lw


@pytest.mark.parametrize("N,K,mix", [
    (16, 128, {1: 0.5, 2: 0.25, 4: 0.25}),          # the smallest rows: 16 bytes at 1 bit
    (333, 1408, {1: 0.3, 2: 0.5, 4: 0.2}),
    (77, 256, {4: 1.0}),                             # one class: the permutation is the identity
    (3000, 512, {1: 0.6, 2: 0.35, 4: 0.05}),         # more rows than warps in the grid
])
def test_to_natural_and_back(lw, N, K, mix):
    case = make_case(N, K, mix, matrix_id=(3 * N + K) % 71)
    layout = lw.Layout(case.precs, K)
    _, _, codes = oracle.encode(case.W, case.precs, case.thr, return_codes=True)
    nat_ref, off_ref = oracle.natural_layout(codes, case.precs)
    off = lw.lowra_natural_offsets(case.precs, K)
    assert np.array_equal(off, off_ref)
    off_d = torch.from_numpy(off.view(np.int64)).cuda()
    packed = torch.from_numpy(case.packed).cuda()
    absmax = torch.from_numpy(case.absmax).cuda()                       # stored (grouped) order
    nat = torch.full((case.packed.size + 32,), 0x5A, dtype=torch.uint8, device="cuda")
    am_nat = torch.full((N * (K // 64) + 8,), -3.0, dtype=torch.float32, device="cuda")
    lw.lowra_reorder_rows(layout, True, off_d, packed, absmax, nat[:case.packed.size], am_nat[:N * (K // 64)].view(N, K // 64))
    torch.cuda.synchronize()
    got = nat.cpu().numpy()
    assert np.array_equal(got[:case.packed.size], nat_ref) and (got[case.packed.size:] == 0x5A).all()
    am = am_nat.cpu().numpy()
    pl = oracle.plan(case.precs, K)
    assert np.array_equal(am[:N * (K // 64)].reshape(N, K // 64), case.absmax[pl["inv_perm"]])   # original row order
    assert (am[N * (K // 64):] == -3.0).all()
    # and back: what the decoder of this library reads
    back, am_back = lw.lowra_reorder_rows(layout, False, off_d, nat[:case.packed.size].clone(),
                                          am_nat[:N * (K // 64)].view(N, K // 64).clone())
    assert np.array_equal(back.cpu().numpy(), case.packed)
    assert np.array_equal(am_back.cpu().numpy(), case.absmax)
    out = lw.lowra_decode(layout, back, am_back, torch.from_numpy(case.maps).cuda())
    assert np.array_equal(out.view(torch.int16).cpu().numpy().view(np.uint16), case.W_hat)


def _bf(bits):
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)


def _bits(t):
    return t.view(torch.int16).cpu().numpy().view(np.uint16)


@pytest.mark.parametrize("N,K,M,r,mix", [
    (16, 128, 40, 16, {1: 0.5, 2: 0.25, 4: 0.25}),
    (336, 1408, 300, 32, {1: 0.3, 2: 0.5, 4: 0.2}),          # several tiles, ragged tokens
    (1800, 2304, 7500, 80, {1: 0.4, 2: 0.4, 4: 0.2}),        # tiles cut between SMs in both directions
    (4096, 4096, 2048, 64, {1: 0.3, 2: 0.5, 4: 0.2}),        # config 2
])
def test_kernels_work_on_the_natural_order_buffer_directly(lw, N, K, M, r, mix):
    """A layout that carries the natural offsets: encode writes the paper's buffer (bit for bit the oracle's natural
    layout of the oracle's codes, absmax rows in original order), decode reads it (bit for bit the oracle's decode),
    and the fused products on it are bit-identical to the products on the grouped buffer (same arithmetic, rows found
    at other addresses) and within the product tolerances of the fp64 oracle.  No conversion pass anywhere."""
    import synth_inputs as si
    from helpers import FRO_TOL, MAX_TOL, gemm_errors

    s = 2.0
    case = make_case(N, K, mix, matrix_id=(5 * N + K) % 83, lloyd_iters=2)
    _, _, codes = oracle.encode(case.W, case.precs, case.thr, return_codes=True)
    nat_ref, _ = oracle.natural_layout(codes, case.precs)
    absmax_nat_ref = oracle.absmax(case.W)                                  # original row order
    nat = lw.Layout(case.precs, K, natural=True)
    W_d, thr_d, maps_d = (torch.from_numpy(a).cuda() for a in (case.W, case.thr, case.maps))
    packed = torch.full((nat.packed_bytes + 64,), 0xA5, dtype=torch.uint8, device="cuda")
    absmax = torch.full((N * (K // 64) + 16,), -7.0, dtype=torch.float32, device="cuda")
    lw.lowra_encode(nat, W_d, thr_d, packed=packed[:nat.packed_bytes], absmax=absmax[:N * (K // 64)].view(N, K // 64))
    torch.cuda.synchronize()
    got = packed.cpu().numpy()
    assert np.array_equal(got[:nat.packed_bytes], nat_ref) and (got[nat.packed_bytes:] == 0xA5).all()
    am = absmax.cpu().numpy()
    assert np.array_equal(am[:N * (K // 64)].reshape(N, K // 64).view(np.uint32), absmax_nat_ref.view(np.uint32))
    assert (am[N * (K // 64):] == -7.0).all()
    pk, am_d = packed[:nat.packed_bytes], absmax[:N * (K // 64)].view(N, K // 64)
    what = lw.lowra_decode(nat, pk, am_d, maps_d)
    assert np.array_equal(_bits(what), case.W_hat)

    # the two products: natural against grouped (bit-identical) and against the oracle
    grouped = lw.Layout(case.precs, K)
    pk_g, am_g = torch.from_numpy(case.packed).cuda(), torch.from_numpy(case.absmax).cuda()
    X, dY = si.activations(M, K, matrix_id=41), si.out_grads(M, N, matrix_id=41)
    A, B = si.lora_factors(K, N, r, matrix_id=41)
    ws = torch.empty(lw.lowra_workspace_bytes(grouped, M, r), dtype=torch.uint8, device="cuda")
    for dealt in (False, True):
        if dealt:
            nat.build_deal()
            lw.lowra_workspace_init(ws)
        Y = lw.lowra_lora_forward(nat, pk, am_d, maps_d, _bf(X), _bf(A), _bf(B), s, workspace=ws)
        dX = lw.lowra_lora_backward_input(nat, pk, am_d, maps_d, _bf(dY), _bf(A), _bf(B), s, workspace=ws)
        assert lw.lowra_device_status(ws) == lw.LOWRA_OK
        Yg = lw.lowra_lora_forward(grouped, pk_g, am_g, maps_d, _bf(X), _bf(A), _bf(B), s)
        dXg = lw.lowra_lora_backward_input(grouped, pk_g, am_g, maps_d, _bf(dY), _bf(A), _bf(B), s)
        assert torch.equal(Y.view(torch.int16), Yg.view(torch.int16))
        assert torch.equal(dX.view(torch.int16), dXg.view(torch.int16))
    rows = np.unique(np.linspace(0, M - 1, min(M, 96)).astype(np.int64))
    idx = torch.from_numpy(rows).cuda()
    emax, efro = gemm_errors(si.bf16_bits_to_f32(_bits(Y[idx])), oracle.lora_forward(case.W_hat, X[rows], A, B, s))
    assert emax <= MAX_TOL and efro <= FRO_TOL, ("forward", emax, efro)
    emax, efro = gemm_errors(si.bf16_bits_to_f32(_bits(dX[idx])), oracle.lora_backward_input(case.W_hat, dY[rows], A, B, s))
    assert emax <= MAX_TOL and efro <= FRO_TOL, ("backward", emax, efro)
