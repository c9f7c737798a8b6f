"""Pins of the oracle's natural-row-order buffer (the paper's own layout of the packed codes)."""
import numpy as np

import oracle


def _case(N=12, K=128, seed=3):
    rng = np.random.default_rng(seed)
    precs = rng.choice([1, 2, 4], size=N).astype(np.uint8)
    W = (rng.standard_normal((N, K)) * 0.05).astype(np.float32)
    maps, thr = oracle.lloyd_max(W, precs, T=2)
    packed, a, codes = oracle.encode(W, precs, thr, return_codes=True)
    return precs, W, maps, thr, packed, a, codes


def test_offsets_are_the_prefix_sums_of_the_row_sizes():
    precs, _, _, _, packed, _, codes = _case()
    buf, off = oracle.natural_layout(codes, precs)
    K = codes.shape[1]
    assert off[0] == 0 and buf.size == off[-1] == packed.size
    for r in range(len(precs)):
        assert off[r + 1] - off[r] == K * int(precs[r]) // 8


def test_bit_by_bit_read_back():
    """Code k of row r sits at bit offset 8*off[r] + b*k of the buffer, least significant bit first."""
    precs, _, _, _, _, _, codes = _case(N=7, K=128, seed=5)
    buf, off = oracle.natural_layout(codes, precs)
    bits = np.unpackbits(buf, bitorder="little")
    for r in range(len(precs)):
        b = int(precs[r])
        for k in range(codes.shape[1]):
            start = 8 * int(off[r]) + b * k
            val = sum(int(bits[start + j]) << j for j in range(b))
            assert val == codes[r, k], (r, k)


def test_same_rows_as_the_grouped_buffer():
    """The grouped buffer (C packer, pinned on its own) holds the same row images, at the plan's offsets."""
    precs, _, _, _, packed, _, codes = _case(N=20, K=256, seed=7)
    buf, off = oracle.natural_layout(codes, precs)
    K = codes.shape[1]
    pl = oracle.plan(precs, K)
    starts = [0, pl["counts"][0], pl["counts"][0] + pl["counts"][1]]
    for r in range(len(precs)):
        c = {1: 0, 2: 1, 4: 2}[int(precs[r])]
        nbytes = K * int(precs[r]) // 8
        p = int(pl["inv_perm"][r])
        g0 = int(pl["seg_off"][c]) + (p - starts[c]) * nbytes
        assert np.array_equal(buf[int(off[r]):int(off[r + 1])], packed[g0:g0 + nbytes])
