"""GPU parity of lowra_encode / lowra_decode against the CPU oracle: bit-exact, through the C ABI."""
import numpy as np
import pytest
import torch

import oracle
import synth_inputs as si
from helpers import make_case

pytestmark = pytest.mark.gpu

CASES = [
    # N, K, mix, kind
    (512, 512, {1: 0.5, 2: 0.5}, "tiny"),                 # config 1
    (333, 1408, {1: 0.3, 2: 0.5, 4: 0.2}, "llama"),        # ragged: K = 11 * 128, odd N
    (77, 128, {4: 1.0}, "llama"),                          # a single class, the smallest K
    (130, 5120, {1: 0.85, 2: 0.15}, "llama"),              # no 4-bit rows, K not a multiple of 4096
    (9, 11008, {1: 0.34, 2: 0.33, 4: 0.33}, "llama"),      # very few rows, long ragged rows
    (1, 256, {2: 1.0}, "llama"),
    (4096, 4096, {1: 0.3, 2: 0.5, 4: 0.2}, "llama"),       # config 2
]


@pytest.fixture(scope="module")
def lw():
    import paper_2502_08141_b200 as lw
    return lw


def _dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


@pytest.mark.parametrize("N,K,mix,kind", CASES)
def test_encode_decode_bit_exact(lw, N, K, mix, kind):
    case = make_case(N, K, mix, matrix_id=N % 97, kind=kind)
    layout = lw.Layout(case.precs, K)
    assert layout.packed_bytes == case.packed.size

    # canary-padded outputs: the kernels must write exactly their extent
    packed = torch.full((layout.packed_bytes + 64,), 0xA5, dtype=torch.uint8, device="cuda")
    absmax = torch.full((N * (K // 64) + 16,), -7.0, dtype=torch.float32, device="cuda")
    lw.lowra_encode(layout, _dev(case.W), _dev(case.thr), packed[:layout.packed_bytes],
                    absmax[:N * (K // 64)].view(N, K // 64))
    torch.cuda.synchronize()
    got_packed = packed.cpu().numpy()
    got_absmax = absmax.cpu().numpy()
    assert np.array_equal(got_packed[:layout.packed_bytes], case.packed)
    assert np.all(got_packed[layout.packed_bytes:] == 0xA5)
    assert np.array_equal(got_absmax[:N * (K // 64)].view(np.uint32), case.absmax.reshape(-1).view(np.uint32))
    assert np.all(got_absmax[N * (K // 64):] == -7.0)

    out = torch.full((N * K + 64,), 0x7FC0, dtype=torch.int16, device="cuda")
    lw.lowra_decode(layout, _dev(case.packed), _dev(case.absmax), _dev(case.maps),
                    out[:N * K].view(N, K).view(torch.bfloat16))
    torch.cuda.synchronize()
    got = out.cpu().numpy().view(np.uint16)
    assert np.array_equal(got[:N * K].reshape(N, K), case.W_hat)
    assert np.all(got[N * K:] == 0x7FC0)


def test_special_values(lw):
    """Zero blocks, values exactly on a threshold (ties go up) and repeated thresholds."""
    N, K = 12, 256
    rng = np.random.default_rng(4)
    W = (rng.integers(-8, 9, size=(N, K)) / 8.0).astype(np.float32)   # exact dyadic values, many ties
    W[:, 0] = 1.0                                                      # absmax 1 in the first block
    W[3, 64:128] = 0.0                                                 # an all-zero block
    W[5, 128:192] = -0.0
    precs = np.array([1, 2, 4] * 4, np.uint8)
    maps = np.zeros((N, 16), np.float32)
    thr = np.full((N, 16), np.inf, np.float32)
    for r in range(N):
        L = 1 << int(precs[r])
        maps[r, :L] = np.linspace(-1, 1, L)
        t = np.round(np.linspace(-1, 1, L + 1)[1:-1] * 8) / 8          # thresholds on the value grid
        if L == 16:
            t[5] = t[4]                                                # a repeated threshold
        thr[r, :L - 1] = np.sort(t)
    packed_ref, a_ref = oracle.encode(W, precs, thr)
    what_ref = oracle.decode(packed_ref, a_ref, maps, precs, K)
    layout = lw.Layout(precs, K)
    packed, absmax = lw.lowra_encode(layout, _dev(W), _dev(thr))
    out = lw.lowra_decode(layout, packed, absmax, _dev(maps))
    torch.cuda.synchronize()
    assert np.array_equal(packed.cpu().numpy()[:layout.packed_bytes], packed_ref)
    assert np.array_equal(absmax.cpu().numpy().view(np.uint32), a_ref.view(np.uint32))
    assert np.array_equal(out.view(torch.int16).cpu().numpy().view(np.uint16), what_ref)


def test_roundtrip_on_device_matches_oracle_chain(lw):
    """decode(encode(W)) computed entirely on the GPU equals the oracle's chain."""
    case = make_case(256, 1024, {1: 0.6, 2: 0.35, 4: 0.05}, matrix_id=41)
    layout = lw.Layout(case.precs, case.K)
    packed, absmax = lw.lowra_encode(layout, _dev(case.W), _dev(case.thr))
    out = lw.lowra_decode(layout, packed, absmax, _dev(case.maps))
    torch.cuda.synchronize()
    assert np.array_equal(out.view(torch.int16).cpu().numpy().view(np.uint16), case.W_hat)


def test_runs_on_a_side_stream(lw):
    case = make_case(64, 512, {1: 0.5, 2: 0.25, 4: 0.25}, matrix_id=42)
    layout = lw.Layout(case.precs, case.K)
    s = torch.cuda.Stream()
    W, thr, maps = _dev(case.W), _dev(case.thr), _dev(case.maps)
    torch.cuda.synchronize()
    with torch.cuda.stream(s):
        packed, absmax = lw.lowra_encode(layout, W, thr, stream=s)
        out = lw.lowra_decode(layout, packed, absmax, maps, stream=s)
    s.synchronize()
    assert np.array_equal(out.view(torch.int16).cpu().numpy().view(np.uint16), case.W_hat)


def test_one_packed_buffer_many_decode_tables(lw):
    """The production variant of Section 4.1: one set of thresholds (one packed buffer, shared by every
    adapter), a different decode mapping per adapter.  Decode and the fused forward take the mapping as an
    argument of its own, so each adapter's table gives that adapter's weights from the same codes."""
    N, K, M, r = 256, 512, 96, 16
    case = make_case(N, K, {1: 0.4, 2: 0.4, 4: 0.2}, matrix_id=43)
    layout = lw.Layout(case.precs, K)
    packed, absmax = lw.lowra_encode(layout, _dev(case.W), _dev(case.thr))
    X = si.activations(M, K, matrix_id=43)
    A, B = si.lora_factors(K, N, r, matrix_id=43)
    bf = lambda bits: _dev(bits.view(np.int16)).view(torch.bfloat16)
    rng = np.random.default_rng(43)
    for adapter in range(3):
        maps = case.maps.copy()
        if adapter > 0:   # this adapter's levels: the shared ones moved a little, still sorted
            for i in range(N):
                L = 1 << int(case.precs[i])
                gap = np.diff(maps[i, :L]).min() if L > 1 else 0.0
                maps[i, :L] += (rng.uniform(-0.3, 0.3, size=L) * gap).astype(np.float32)
        ref = oracle.decode(case.packed, case.absmax, maps, case.precs, K)
        out = lw.lowra_decode(layout, packed, absmax, _dev(maps))
        assert np.array_equal(out.view(torch.int16).cpu().numpy().view(np.uint16), ref)
        Y = lw.lowra_lora_forward(layout, packed, absmax, _dev(maps), bf(X), bf(A), bf(B), 2.0)
        Y_ref = oracle.lora_forward(ref, X, A, B, 2.0)
        got = si.bf16_bits_to_f32(Y.view(torch.int16).cpu().numpy().view(np.uint16))
        assert np.abs(got - Y_ref).max() <= 1e-2 * np.abs(Y_ref).max()
        assert np.linalg.norm(got - Y_ref) <= 5e-3 * np.linalg.norm(Y_ref)
