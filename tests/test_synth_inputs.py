"""The seeded generators: deterministic, chunk-independent, and shaped as the recipe says."""
import numpy as np

import synth_inputs as si


def test_weights_are_deterministic_and_chunk_independent():
    a = si.weights(96, 256, matrix_id=5, row_chunk=512)
    b = si.weights(96, 256, matrix_id=5, row_chunk=7)
    assert a.dtype == np.float32 and np.array_equal(a, b)
    assert not np.array_equal(a, si.weights(96, 256, matrix_id=6))


def test_weight_distribution():
    W = si.weights(512, 1024, matrix_id=1).astype(np.float64)
    sig = np.median(np.abs(W), axis=1) / 0.6745
    assert 0.004 < sig.min() and sig.max() < 0.06
    assert sig.max() / sig.min() > 5          # log-uniform spread over a decade
    z = W / sig[:, None]
    frac_big = np.mean(np.abs(z) > 6)
    assert 3e-4 < frac_big < 2e-3             # ~0.1 % outliers, x10
    T = si.weights(64, 512, kind="tiny").astype(np.float64)
    assert abs(T.std() - 0.02) < 1e-3 and np.abs(T).max() < 0.12


def test_precision_mix_counts_are_exact():
    p = si.precisions(4096, {1: 0.3, 2: 0.5, 4: 0.2})
    assert [(p == b).sum() for b in (1, 2, 4)] == [1229, 2048, 819]
    p = si.precisions(5120, {1: 0.85, 2: 0.15})
    assert [(p == b).sum() for b in (1, 2, 4)] == [4352, 768, 0]
    # positions are mixed, not sorted
    assert np.count_nonzero(np.diff(p.astype(int))) > 1000


def test_bf16_inputs():
    X = si.activations(64, 256)
    x = si.bf16_bits_to_f32(X).astype(np.float64)
    assert X.dtype == np.uint16 and abs(x.std() - 1) < 0.05 and abs(x.mean()) < 0.05
    A, B = si.lora_factors(256, 128, 16)
    assert A.shape == (256, 16) and B.shape == (16, 128)
    assert abs(si.bf16_bits_to_f32(A).std() - 0.01) < 2e-3


def test_standin_codebooks_are_sorted_with_midpoint_thresholds():
    p = si.precisions(300, {1: 0.3, 2: 0.4, 4: 0.3})
    maps, thr = si.standin_codebooks(p)
    for r in range(300):
        L = 1 << int(p[r])
        assert np.all(np.diff(maps[r, :L]) > 0) and np.all(maps[r, L:] == 0)
        assert np.all(np.isinf(thr[r, L - 1:]))
        assert np.all((thr[r, :L - 1] > maps[r, :L - 1]) & (thr[r, :L - 1] < maps[r, 1:L]))


def test_configs():
    c3 = si.config(3)
    assert [(m.N, m.K) for m in c3.matrices] == [(4096, 4096)] * 4 + [(11008, 4096)] * 2 + [(4096, 11008)]
    assert abs(si.avg_bits(c3.mix) - 1.5) < 1e-9
    assert abs(si.avg_bits(si.config(4).mix) - 1.15) < 1e-9
    assert abs(si.avg_bits(si.config(5).mix) - 2.5) < 1e-9 and len(si.config(5).matrices) == 224
    assert sum(m.N * m.K for m in si.config(5).matrices) == 6_476_005_376


def test_initial_codebooks_are_the_printed_tables():
    """The starting tables handed to the GPU learner by the benchmark are the ones the oracle starts from."""
    import oracle
    y0, t0 = si.initial_codebooks()
    for c, b in enumerate((1, 2, 4)):
        y, t = oracle.initial_tables(b)
        assert np.array_equal(y0[c, :y.size], y) and np.all(y0[c, y.size:] == 0)
        assert np.array_equal(t0[c, :t.size], t) and np.all(t0[c, t.size:] == 0)
