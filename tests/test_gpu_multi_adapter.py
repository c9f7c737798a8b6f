"""Several adapters on one quantised base weight (the paper's production use case: shared thresholds, hence one packed
buffer; one mapping table and one pair of low-rank factors per adapter): one call routes the token groups of a batch
to their adapters.  Every group is held against the fp64 oracle run with that adapter's tables, and against the
single-adapter entry point, with which it must agree bit for bit (up to one bf16 rounding where the tiles of a large
call are cut between SMs, which a call for all groups does elsewhere than a call for one)."""
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


@pytest.mark.parametrize("N,K,r,groups,dealt,big_ws", [
    (256, 384, 16, [5, 300, 0, 77], False, False),            # an empty group, groups smaller and larger than a token tile
    (640, 1152, 64, [515, 1, 260], True, False),              # a launch per group (workspace of a single call)
    (640, 1152, 64, [515, 1, 260, 0, 33, 700], True, True),   # five groups in two launches (four and one)
    (4096, 4096, 64, [1024, 512, 512], True, True),           # config-2 shape, 2048 tokens, three groups in one launch
    (1800, 2304, 80, [2000, 1500, 2500, 1300], True, True),   # tiles cut between SMs, ranges across groups
])
def test_token_groups_are_routed_to_their_adapters(N, K, r, groups, dealt, big_ws):
    import paper_2502_08141_b200 as lw

    s, n = 2.0, len(groups)
    case = make_case(N, K, {1: 0.3, 2: 0.5, 4: 0.2}, matrix_id=61, lloyd_iters=2)
    layout = lw.Layout(case.precs, K)
    if dealt:
        layout.build_deal()
    packed, absmax = _dev(case.packed), _dev(case.absmax)
    # adapter 0 decodes with the learnt levels, the others with tables of their own (same thresholds, so same codes)
    maps = np.stack([case.maps] + [si.standin_codebooks(case.precs, matrix_id=70 + a)[0] for a in range(1, n)])
    A = np.stack([si.lora_factors(K, N, r, matrix_id=80 + a)[0] for a in range(n)])
    B = np.stack([si.lora_factors(K, N, r, matrix_id=80 + a)[1] for a in range(n)])
    start = np.concatenate([[0], np.cumsum(groups)]).astype(np.int32)
    M = int(start[-1])
    X = si.activations(M, K, matrix_id=62)
    nbytes = lw.lowra_batch_workspace_bytes(layout, 4, M, r) if big_ws else lw.lowra_workspace_bytes(layout, M, r)
    ws = lw.lowra_workspace_init(torch.empty(nbytes, dtype=torch.uint8, device="cuda"))
    Y = torch.full((M, N), float("nan"), dtype=torch.bfloat16, device="cuda")
    lw.lowra_lora_forward_adapters(layout, packed, absmax, _dev(maps), _bf(X), start, _bf(A.reshape(n * K, r)).view(n, K, r),
                                   _bf(B.reshape(n * r, N)).view(n, r, N), s, Y=Y, workspace=ws)
    assert lw.lowra_device_status(ws) == lw.LOWRA_OK
    got = _bits(Y)
    for a in range(n):
        m0, m1 = int(start[a]), int(start[a + 1])
        if m1 == m0:
            continue
        what = oracle.decode(case.packed, case.absmax, maps[a], case.precs, K)
        ref = oracle.lora_forward(what, X[m0:m1], A[a], B[a], s)
        emax, efro = gemm_errors(si.bf16_bits_to_f32(got[m0:m1]), ref)
        assert emax <= MAX_TOL and efro <= FRO_TOL, (a, emax, efro)
        one = lw.lowra_lora_forward(layout, packed, absmax, _dev(maps[a]), _bf(X[m0:m1]), _bf(A[a]), _bf(B[a]), s, workspace=ws)
        if N >= 1800 and big_ws:      # tiles are cut elsewhere than in a single call: a bf16 rounding step at most
            o, g = si.bf16_bits_to_f32(_bits(one)), si.bf16_bits_to_f32(got[m0:m1])
            assert np.abs(o - g).max() <= 2.0 ** -7 * np.abs(o).max(), a
        else:
            assert np.array_equal(_bits(one), got[m0:m1]), a


def test_group_boundaries_are_validated():
    import paper_2502_08141_b200 as lw

    N, K, r = 128, 128, 16
    layout = lw.Layout(np.full(N, 2, np.uint8), K)
    z = lambda *shape, dt=torch.bfloat16: torch.zeros(shape, dtype=dt, device="cuda")
    args = (layout, z(layout.packed_bytes, dt=torch.uint8), z(N, K // 64, dt=torch.float32), z(2, N, 16, dt=torch.float32), z(10, K))
    for bad in ([0, 4, 9], [1, 4, 10], [0, 11, 10]):
        with pytest.raises(lw.LowraError) as e:
            lw.lowra_lora_forward_adapters(*args, np.array(bad, np.int32), z(2, K, r), z(2, r, N), 1.0)
        assert e.value.code == lw.LOWRA_ERR_SHAPE
