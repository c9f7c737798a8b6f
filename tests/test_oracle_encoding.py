"""Pins for the encoding half of the CPU oracle (absmax, normalise, bucket, pack, decode).

Nothing here needs a GPU.  Each test compares the oracle with something other than itself:
a brute-force restatement on tiny matrices, a library routine (numpy searchsorted / packbits,
torch's bf16 cast), a closed form, or an invariant that the method fixes.
"""
import numpy as np
import pytest
import torch

import oracle
import synth_inputs as si

BITS = (1, 2, 4)


def _tables_from_levels(levels_per_row, precs):
    """[N,16] maps / thresholds from per-row sorted level lists; thresholds at midpoints."""
    N = len(precs)
    maps = np.zeros((N, 16), np.float32)
    thr = np.full((N, 16), np.inf, np.float32)
    for r in range(N):
        lv = np.asarray(levels_per_row[r], np.float32)
        maps[r, :lv.size] = lv
        thr[r, :lv.size - 1] = ((lv[:-1].astype(np.float64) + lv[1:].astype(np.float64)) / 2).astype(np.float32)
    return maps, thr


def _random_tables(rng, precs):
    levels = []
    for b in precs:
        lv = np.sort(rng.uniform(-1, 1, size=1 << int(b)))
        levels.append(lv)
    return _tables_from_levels(levels, precs)


def _unpack_row(row_bytes, K, b):
    """Independent unpacker: numpy bit expansion, little-endian bit order."""
    bits = np.unpackbits(row_bytes, bitorder="little")[: K * b].reshape(K, b)
    return (bits.astype(np.int64) << np.arange(b)).sum(axis=1)


# ------------------------------------------------------------------------------------------
def test_bf16_rounding_matches_torch():
    rng = np.random.default_rng(0)
    x = np.concatenate([
        rng.standard_normal(20000).astype(np.float32),
        (rng.standard_normal(2000) * 1e-30).astype(np.float32),
        np.array([0.0, -0.0, 1.0, -1.0, 3.3895314e38, 1e-45, np.inf, -np.inf], np.float32),
        # exact ties: low 16 bits = 0x8000 with even and odd upper halves
        np.array([0x3F808000, 0x3F818000, 0xBF808000, 0xBF818000], np.uint32).view(np.float32),
    ])
    got = oracle.f32_to_bf16(x)
    want = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(got, want)


def test_absmax_matches_numpy_and_blocks_run_along_k():
    W = si.weights(24, 256, matrix_id=3)
    a = oracle.absmax(W, 64)
    want = np.abs(W).reshape(24, 4, 64).max(axis=2)
    assert a.dtype == np.float32 and np.array_equal(a, want)
    # every block holds an element of exactly that magnitude
    assert np.all((np.abs(W).reshape(24, 4, 64) == a[:, :, None]).any(axis=2))


def test_normalise_is_two_rounded_fp32_operations():
    W = si.weights(16, 128, matrix_id=4)
    W[3, 64:128] = 0.0  # a zero block
    n = oracle.normalise(W, 64)
    a = np.repeat(oracle.absmax(W, 64), 64, axis=1)
    with np.errstate(divide="ignore", invalid="ignore"):
        inv = (np.float32(1.0) / a).astype(np.float32)
        want = np.where(a == 0, np.float32(0), (W * inv).astype(np.float32))
    assert np.array_equal(n, want)
    assert np.all(n[3, 64:128] == 0)
    assert np.abs(n).max() <= 1.0 + 2 ** -23
    # the element attaining the maximum normalises to +-1 within one rounding
    assert np.all(np.abs(np.abs(n).reshape(16, 2, 64).max(axis=2)[a.reshape(16, 2, 64)[:, :, 0] > 0] - 1) <= 2 ** -23)


@pytest.mark.parametrize("G", [4, 8])
def test_bucket_brute_force_8x8(G):
    rng = np.random.default_rng(10 + G)
    for trial in range(20):
        precs = rng.choice(BITS, size=8).astype(np.uint8)
        W = rng.standard_normal((8, 8)).astype(np.float32)
        maps, thr = _random_tables(rng, precs)
        _, _, codes = oracle.encode(W, precs, thr, G=G, return_codes=True)
        n = oracle.normalise(W, G)
        for r in range(8):
            b = int(precs[r])
            t = thr[r, :(1 << b) - 1]
            for k in range(8):
                c = int(codes[r, k])
                # interval test t_{c-1} <= n < t_c
                lo = -np.inf if c == 0 else t[c - 1]
                hi = np.inf if c == t.size else t[c]
                assert lo <= n[r, k] < hi
            # library binary search, ties to the right
            assert np.array_equal(codes[r], np.searchsorted(t, n[r], side="right"))
            # thresholds at midpoints => nearest level (away from exact ties)
            d = np.abs(n[r][:, None].astype(np.float64) - maps[r, :1 << b][None, :].astype(np.float64))
            near = d.argmin(axis=1)
            margin = np.sort(d, axis=1)
            clear = (margin[:, 1] - margin[:, 0]) > 1e-6
            assert np.array_equal(codes[r][clear], near[clear])


def test_tie_goes_to_upper_bucket():
    # one block of 8 with absmax 1 so that normalised values equal the weights
    W = np.array([[1.0, -0.5, 0.25, 0.75, 0.0, -1.0, 0.5, 0.125]], np.float32)
    for b, t in ((1, [0.0]), (2, [-0.5, 0.25, 0.75]), (4, list(np.linspace(-0.875, 0.875, 15)))):
        thr = np.full((1, 16), np.inf, np.float32)
        thr[0, :len(t)] = t
        _, _, codes = oracle.encode(W, np.array([b], np.uint8), thr, G=8, return_codes=True)
        for k in range(8):
            want = sum(1 for tj in np.asarray(t, np.float32) if tj <= W[0, k])
            assert codes[0, k] == want
        if b == 2:
            assert list(codes[0]) == [3, 1, 2, 3, 1, 0, 2, 1]
        if b == 1:
            assert list(codes[0]) == [1, 0, 1, 1, 1, 0, 1, 1]  # 0.0 sits on the threshold -> upper


def test_plan_is_stable_class_sorted_permutation():
    precs = si.precisions(1000, {1: 0.3, 2: 0.5, 4: 0.2}, matrix_id=7)
    K = 256
    pl = oracle.plan(precs, K)
    perm, inv = pl["perm"], pl["inv_perm"]
    assert np.array_equal(np.sort(perm), np.arange(1000))
    assert np.array_equal(inv[perm], np.arange(1000)) and np.array_equal(perm[inv], np.arange(1000))
    stored = precs[perm]
    assert np.all(np.diff(stored.astype(int)) >= 0)              # classes in order 1,2,4
    for b in BITS:
        rows = perm[stored == b]
        assert np.all(np.diff(rows) > 0)                         # stable
        assert np.array_equal(rows, np.nonzero(precs == b)[0])
    counts = [int((precs == b).sum()) for b in BITS]
    assert list(pl["counts"]) == counts
    assert pl["packed_bytes"] == sum(K * int(b) // 8 for b in precs)   # sum of per-row bits
    assert list(pl["seg_off"]) == [0, counts[0] * K // 8, counts[0] * K // 8 + counts[1] * K // 4]


@pytest.mark.parametrize("N,K,G", [(8, 8, 4), (8, 8, 8), (128, 128, 64), (37, 192, 64)])
def test_pack_against_independent_packer(N, K, G):
    rng = np.random.default_rng(N * 1000 + K)
    precs = rng.choice(BITS, size=N).astype(np.uint8)
    W = rng.standard_normal((N, K)).astype(np.float32)
    maps, thr = _random_tables(rng, precs)
    packed, a, codes = oracle.encode(W, precs, thr, G=G, return_codes=True)
    pl = oracle.plan(precs, K)
    assert packed.size == pl["packed_bytes"] == sum(K * int(b) // 8 for b in precs)
    # word-wise writer: element e of a little-endian 32-bit word sits at bits [e*b, e*b+b)
    want = np.zeros_like(packed)
    off = 0
    for p in range(N):
        r = int(pl["perm"][p]); b = int(precs[r])
        nbytes = K * b // 8
        vals = codes[r].astype(np.uint64)
        if K * b % 32 == 0:
            per = 32 // b
            words = (vals.reshape(-1, per) << (np.arange(per, dtype=np.uint64) * np.uint64(b))).sum(axis=1)
            row = words.astype("<u4").view(np.uint8)
        else:
            bits = ((vals[:, None] >> np.arange(b, dtype=np.uint64)) & np.uint64(1)).astype(np.uint8).reshape(-1)
            row = np.packbits(bits, bitorder="little")
        want[off:off + nbytes] = row
        # round trip through an independent unpacker
        assert np.array_equal(_unpack_row(packed[off:off + nbytes], K, b), codes[r])
        off += nbytes
    assert off == packed.size
    assert np.array_equal(packed, want)
    # absmax is stored in stored-row order
    assert np.array_equal(a, oracle.absmax(W, G)[pl["perm"]])


def test_decode_one_bit_sign_quantiser_closed_form():
    # b = 1, threshold 0, levels -1 / +1  =>  decode = sign(x) * absmax (zero counts as +)
    N, K = 16, 256
    W = si.weights(N, K, matrix_id=11)
    W[0, :5] = 0.0
    precs = np.ones(N, np.uint8)
    maps = np.zeros((N, 16), np.float32); maps[:, 0] = -1; maps[:, 1] = 1
    thr = np.full((N, 16), np.inf, np.float32); thr[:, 0] = 0
    packed, a = oracle.encode(W, precs, thr)
    out = oracle.decode(packed, a, maps, precs, K)
    sign = np.where(W >= 0, 1.0, -1.0).astype(np.float32)
    want = torch.from_numpy(sign * np.repeat(a, 64, axis=1)).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(out, want)


def test_decode_level_is_bucket_of_normalised_value():
    """decode(encode(W)) equals bf16(map[bucket(n)] * absmax), with the bucket found by a
    library search and the bf16 cast done by torch."""
    N, K = 96, 512
    W = si.weights(N, K, matrix_id=12)
    precs = si.precisions(N, {1: 0.3, 2: 0.5, 4: 0.2}, matrix_id=12)
    rng = np.random.default_rng(5)
    maps, thr = _random_tables(rng, precs)
    packed, a = oracle.encode(W, precs, thr)
    out = oracle.decode(packed, a, maps, precs, K)
    n = oracle.normalise(W, 64)
    a_nat = np.abs(W).reshape(N, K // 64, 64).max(axis=2)
    want = np.empty((N, K), np.float32)
    for r in range(N):
        b = int(precs[r])
        code = np.searchsorted(thr[r, :(1 << b) - 1], n[r], side="right")
        want[r] = (maps[r, code] * np.repeat(a_nat[r], 64)).astype(np.float32)
    want16 = torch.from_numpy(want).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(out, want16)
    # magnitude bound and the absmax element with top level 1
    dec = si.bf16_bits_to_f32(out).astype(np.float64)
    bound = np.repeat(a_nat, 64, axis=1) * np.abs(maps).max(axis=1, keepdims=True)
    assert np.all(np.abs(dec) <= bound * (1 + 2 ** -8))


def test_block_maximum_decodes_to_absmax_when_outer_levels_are_unit():
    N, K = 32, 256
    W = si.weights(N, K, matrix_id=13)
    precs = si.precisions(N, {1: 0.25, 2: 0.5, 4: 0.25}, matrix_id=13)
    levels = []
    rng = np.random.default_rng(9)
    for b in precs:
        lv = np.sort(rng.uniform(-0.9, 0.9, size=1 << int(b)))
        lv[0], lv[-1] = -1.0, 1.0
        levels.append(lv)
    maps, thr = _tables_from_levels(levels, precs)
    packed, a = oracle.encode(W, precs, thr)
    dec = si.bf16_bits_to_f32(oracle.decode(packed, a, maps, precs, K))
    a_nat = oracle.absmax(W, 64)
    a16 = si.bf16_bits_to_f32(oracle.f32_to_bf16(a_nat))
    blocks = np.abs(dec).reshape(N, K // 64, 64)
    arg = np.abs(W).reshape(N, K // 64, 64).argmax(axis=2)
    got = np.take_along_axis(blocks, arg[:, :, None], axis=2)[:, :, 0]
    assert np.array_equal(got, a16)


def test_reencoding_the_reconstruction_is_idempotent():
    """With thresholds at midpoints, quantising the (unrounded) reconstruction map*absmax again
    returns the same codes whenever the block maximum is reproduced (outer levels +-1)."""
    N, K = 24, 128
    W = si.weights(N, K, matrix_id=14)
    precs = si.precisions(N, {1: 0.3, 2: 0.4, 4: 0.3}, matrix_id=14)
    levels = []
    rng = np.random.default_rng(2)
    for b in precs:
        lv = np.sort(rng.uniform(-0.9, 0.9, size=1 << int(b)))
        lv[0], lv[-1] = -1.0, 1.0
        levels.append(lv)
    maps, thr = _tables_from_levels(levels, precs)
    _, a, codes = oracle.encode(W, precs, thr, return_codes=True)
    a_nat = oracle.absmax(W, 64)
    recon = np.take_along_axis(maps, codes.astype(np.int64), axis=1) * np.repeat(a_nat, 64, axis=1)
    _, a2, codes2 = oracle.encode(recon.astype(np.float32), precs, thr, return_codes=True)
    assert np.array_equal(a2, a)
    assert np.array_equal(codes2, codes)


def test_rejects_bad_precision():
    with pytest.raises(ValueError):
        oracle.plan(np.array([1, 3, 2], np.uint8), 64)
