"""lowra_encode_group / lowra_decode_group: the chunks of several matrices - any shapes, any layouts - handed to the warps
of one launch.  Every member's packed bytes, absmax values and decoded weights must be bit for bit what the single calls
give, and (one member per precision mix) what the oracle gives."""
import numpy as np
import pytest
import torch

import oracle
import synth_inputs as si

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def lw():
    import paper_2502_08141_b200 as lw
    return lw


SHAPES = [
    # N, K, mix, natural order
    (640, 1152, {1: 0.6, 2: 0.35, 4: 0.05}, False),
    (96, 4096, {1: 0.34, 2: 0.33, 4: 0.33}, False),
    (1024, 128, {2: 0.75, 4: 0.25}, True),
    (333, 1408, {1: 0.85, 2: 0.15}, False),
    (8, 11008, {4: 1.0}, False),
    (2048, 2048, {1: 1.0}, True),
    (130, 256, {2: 1.0}, False),
    (512, 5120, {1: 0.5, 4: 0.5}, False),
]


def _members(lw, shapes):
    ms = []
    for i, (N, K, mix, natural) in enumerate(shapes):
        precs = si.precisions(N, mix, matrix_id=40 + i)
        maps, thr = si.standin_codebooks(precs, matrix_id=40 + i)
        W = si.weights(N, K, matrix_id=40 + i)
        ms.append(dict(layout=lw.Layout(precs, K, natural=natural), precs=precs, W_host=W, maps_host=maps, thr_host=thr,
                       W=torch.from_numpy(W).cuda(), thresholds=torch.from_numpy(thr).cuda(), maps=torch.from_numpy(maps).cuda()))
    return ms


@pytest.mark.parametrize("count", [1, 3, 8])
def test_group_calls_equal_the_single_calls(lw, count):
    ms = _members(lw, SHAPES[:count])
    singles = [lw.lowra_encode(m["layout"], m["W"], m["thresholds"]) for m in ms]
    group = lw.lowra_encode_group([dict(layout=m["layout"], W=m["W"], thresholds=m["thresholds"]) for m in ms])
    for m, (p1, a1), (p2, a2) in zip(ms, singles, group):
        nbytes = m["layout"].packed_bytes
        assert torch.equal(p1[:nbytes], p2[:nbytes])
        assert torch.equal(a1.view(torch.int32), a2.view(torch.int32))
    outs1 = [lw.lowra_decode(m["layout"], p, a, m["maps"]) for m, (p, a) in zip(ms, singles)]
    canary = [torch.full((m["layout"].N * m["layout"].K + 64,), -1, dtype=torch.int16, device="cuda") for m in ms]
    outs2 = lw.lowra_decode_group([dict(layout=m["layout"], packed=p, absmax=a, maps=m["maps"],
                                        out=c[16:16 + m["layout"].N * m["layout"].K].view(torch.bfloat16).view(m["layout"].N, m["layout"].K))
                                   for m, (p, a), c in zip(ms, group, canary)])
    for m, o1, o2, c in zip(ms, outs1, outs2, canary):
        assert torch.equal(o1.view(torch.int16), o2.view(torch.int16))
        assert bool((c[:16] == -1).all()) and bool((c[-48:] == -1).all())   # nothing written outside a member's output


def test_group_members_against_the_oracle(lw):
    ms = _members(lw, [s for s in SHAPES if not s[3]][:5])   # the natural-order members are covered by the test above
    group = lw.lowra_encode_group([dict(layout=m["layout"], W=m["W"], thresholds=m["thresholds"]) for m in ms])
    outs = lw.lowra_decode_group([dict(layout=m["layout"], packed=p, absmax=a, maps=m["maps"]) for m, (p, a) in zip(ms, group)])
    for m, (p, a), o in zip(ms, group, outs):
        K = m["layout"].K
        p_ref, a_ref = oracle.encode(m["W_host"], m["precs"], m["thr_host"])
        w_ref = oracle.decode(p_ref, a_ref, m["maps_host"], m["precs"], K)
        assert np.array_equal(p.cpu().numpy()[:m["layout"].packed_bytes], p_ref)
        assert np.array_equal(a.cpu().numpy().view(np.uint32), np.asarray(a_ref, dtype=np.float32).view(np.uint32))
        assert np.array_equal(o.view(torch.int16).cpu().numpy().view(np.uint16), w_ref)


def test_group_argument_checks(lw):
    ms = _members(lw, SHAPES[:1])
    with pytest.raises(lw.LowraError) as e:
        lw.lowra_encode_group([])
    assert e.value.code == lw.LOWRA_ERR_SHAPE
    nine = [dict(layout=ms[0]["layout"], W=ms[0]["W"], thresholds=ms[0]["thresholds"])] * 9
    with pytest.raises(lw.LowraError) as e:
        lw.lowra_encode_group(nine)
    assert e.value.code == lw.LOWRA_ERR_SHAPE


@pytest.mark.parametrize("config", [3, 4])
def test_a_whole_layer_in_one_launch_equals_the_single_calls(lw, config):
    """The launch configuration bench.py times: the seven matrices of a layer (full size, the config's precision mix,
    largest first) through one lowra_encode_group and one lowra_decode_group launch; bit for bit the single calls, which
    tests/test_gpu_full_size.py holds against the oracle on the same shapes."""
    cfg = si.config(config)
    mats = sorted(cfg.matrices, key=lambda m: -m.N * m.K)
    gen = torch.Generator(device="cuda").manual_seed(config)
    ms = []
    for m in mats:
        precs = si.precisions(m.N, cfg.mix, matrix_id=m.matrix_id)
        maps, thr = si.standin_codebooks(precs, matrix_id=m.matrix_id)
        W = torch.randn(m.N, m.K, device="cuda", generator=gen) * 0.02
        W[::97, ::61] *= 10.0                                   # a few outliers, as in the weight recipe
        ms.append(dict(layout=lw.Layout(precs, m.K), W=W, thresholds=torch.from_numpy(thr).cuda(), maps=torch.from_numpy(maps).cuda()))
    group = lw.lowra_encode_group([dict(layout=m["layout"], W=m["W"], thresholds=m["thresholds"]) for m in ms])
    outs = lw.lowra_decode_group([dict(layout=m["layout"], packed=p, absmax=a, maps=m["maps"]) for m, (p, a) in zip(ms, group)])
    for m, (p, a), o in zip(ms, group, outs):
        p1, a1 = lw.lowra_encode(m["layout"], m["W"], m["thresholds"])
        assert torch.equal(p1[:m["layout"].packed_bytes], p[:m["layout"].packed_bytes])
        assert torch.equal(a1.view(torch.int32), a.view(torch.int32))
        o1 = lw.lowra_decode(m["layout"], p1, a1, m["maps"])
        assert torch.equal(o1.view(torch.int16), o.view(torch.int16))
        del p1, a1, o1
