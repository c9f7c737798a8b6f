"""GPU parity of the conversion between the grouped and the paper's natural row order: bit-exact."""
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
