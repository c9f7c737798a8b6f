"""Failure detection on the device without faulting anything: every wait in the tensor-core kernels has a limit,
and when one runs out the kernel records LOWRA_ERR_TIMEOUT, lets what it has in flight land, frees its tensor
memory and returns.  The tests make waits run out in two ways - a one-warp kernel that waits for a barrier and a
flag nobody will ever signal, and fused calls whose "down-projection ready" flags are withheld (switched off on
the host) - and check the status word, that the GPU is healthy afterwards, and that the next ordinary call on the
same workspace gives the right answer.  Nothing here traps, faults or waits without a limit.
"""
import numpy as np
import pytest
import torch

import oracle
import synth_inputs as si
from helpers import FRO_TOL, MAX_TOL, gemm_errors

pytestmark = pytest.mark.gpu


def _dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def _bf(bits):
    return _dev(bits.view(np.int16)).view(torch.bfloat16)


def _bits(t):
    return t.view(torch.int16).cpu().numpy().view(np.uint16)


@pytest.fixture
def short_waits():
    import paper_2502_08141_b200 as lw
    lw.lowra_set_wait_limit(2_000_000)      # 2 ms
    yield lw
    lw.lowra_diag_drop_t_flags(0)
    lw.lowra_set_wait_limit(0)              # back to the default


def test_waits_that_nobody_answers_run_out():
    import paper_2502_08141_b200 as lw

    ws = torch.zeros(256, dtype=torch.uint8, device="cuda")
    lw.lowra_diag_wait_expiry(ws, 1_000_000)                     # 1 ms per wait
    assert lw.lowra_device_status(ws) == lw.LOWRA_ERR_TIMEOUT
    report = ws.view(torch.int32)[8:11].cpu().numpy()
    assert report[0] == 7                                        # barrier wait, flag wait and the whole-warp form
    assert 900 <= report[1] <= 50_000 and 900 <= report[2] <= 50_000, report   # microseconds: the limit, not much more
    # the context is intact: an ordinary product right afterwards
    P, Q = si.bf16_normal((128, 128), 1.0, stream=50), si.bf16_normal((128, 128), 1.0, stream=51)
    ws2 = torch.zeros(256, dtype=torch.uint8, device="cuda")
    C = lw.lowra_dense_nt(_bf(P), _bf(Q), workspace=ws2)
    assert lw.lowra_device_status(ws2) == lw.LOWRA_OK
    emax, efro = gemm_errors(si.bf16_bits_to_f32(_bits(C)), oracle.bf16_to_f64(P) @ oracle.bf16_to_f64(Q).T)
    assert emax <= MAX_TOL and efro <= FRO_TOL


def test_wait_limit_argument_range():
    import paper_2502_08141_b200 as lw

    with pytest.raises(lw.LowraError):
        lw.lowra_set_wait_limit(10)                              # below a microsecond
    with pytest.raises(lw.LowraError):
        lw.lowra_set_wait_limit(10 ** 11)
    lw.lowra_set_wait_limit(0)


def _timeout_then_recover(lw, N, K, M, r, mix, mid, dealt):
    from helpers import make_case

    s = 2.0
    case = make_case(N, K, mix, matrix_id=mid, lloyd_iters=2)
    layout = lw.Layout(case.precs, K)
    if dealt:
        layout.build_deal()
    packed, absmax, maps = _dev(case.packed), _dev(case.absmax), _dev(case.maps)
    X, dY = si.activations(M, K, matrix_id=600 + mid), si.out_grads(M, N, matrix_id=600 + mid)
    A, B = si.lora_factors(K, N, r, matrix_id=mid)
    ws = lw.lowra_workspace_init(torch.empty(lw.lowra_workspace_bytes(layout, M, r), dtype=torch.uint8, device="cuda"))
    refs = {"forward": oracle.lora_forward(case.W_hat, X, A, B, s), "backward": oracle.lora_backward_input(case.W_hat, dY, A, B, s)}

    def call(which):
        if which == "forward":
            return lw.lowra_lora_forward(layout, packed, absmax, maps, _bf(X), _bf(A), _bf(B), s, workspace=ws)
        return lw.lowra_lora_backward_input(layout, packed, absmax, maps, _bf(dY), _bf(A), _bf(B), s, workspace=ws)

    for which in ("forward", "backward"):
        good = call(which)
        assert lw.lowra_device_status(ws) == lw.LOWRA_OK
        lw.lowra_diag_drop_t_flags(1)                            # the next fused call never sees its down-projection
        call(which)
        assert lw.lowra_device_status(ws) == lw.LOWRA_ERR_TIMEOUT, which
        if dealt:                                                # no prologue clears the word: it is sticky until re-initialised
            lw.lowra_workspace_init(ws)
        again = call(which)                                      # the workspace and the GPU are as good as before
        assert lw.lowra_device_status(ws) == lw.LOWRA_OK, which
        assert torch.equal(again.view(torch.int16), good.view(torch.int16)), which
        emax, efro = gemm_errors(si.bf16_bits_to_f32(_bits(again)), refs[which])
        assert emax <= MAX_TOL and efro <= FRO_TOL, (which, emax, efro)


@pytest.mark.parametrize("dealt", [False, True])
def test_fused_call_times_out_and_the_next_one_is_right_small(short_waits, dealt):
    _timeout_then_recover(short_waits, 256, 256, 64, 16, {1: 0.4, 2: 0.4, 4: 0.2}, 31, dealt)


def test_fused_call_times_out_and_the_next_one_is_right_several_tiles(short_waits):
    _timeout_then_recover(short_waits, 640, 1152, 515, 96, {1: 0.6, 2: 0.35, 4: 0.05}, 32, False)


def test_fused_call_times_out_and_the_next_one_is_right_cut_tiles(short_waits):
    """Enough tiles for the schedule that cuts the contraction of the last tiles between SMs: the SMs that would
    collect partial tiles wait for slices that were given up, and give up in turn."""
    _timeout_then_recover(short_waits, 1800, 2304, 7500, 80, {1: 0.4, 2: 0.4, 4: 0.2}, 33, True)
