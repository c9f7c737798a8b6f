"""The N > 1 path of bench.py on CPU: two gloo ranks (no GPU).

Ranks run independent layers (no data-path collective); what they share is the timing protocol:
max over ranks of the device time, whole-job value = world x per-rank work / that time, and
disjoint seeded inputs per rank.
"""
import os
import socket
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        import bench
        import synth_inputs as si
        my_ms = 10.0 + 5.0 * rank                      # rank 1 is the slow one
        ms = bench.max_over_ranks(my_ms, world, device="cpu")
        value = bench.aggregate_tflops(1e12, world, ms)
        mid = bench.rank_matrix_id(3, rank)
        w = si.weights(8, 128, matrix_id=mid, kind="normal")
        gathered = [None] * world
        dist.all_gather_object(gathered, (ms, value, mid, float(np.abs(w).sum())))
        if rank == 0:
            out.put(gathered)
    finally:
        dist.destroy_process_group()


@pytest.mark.timeout(120)
def test_two_ranks_agree_on_the_slowest_time_and_hold_different_layers():
    world = 2
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    res = out.get(timeout=100)
    for p in procs:
        p.join(timeout=30)
        assert p.exitcode == 0
    (ms0, v0, mid0, s0), (ms1, v1, mid1, s1) = res
    assert ms0 == ms1 == 15.0                          # the maximum, on every rank
    assert v0 == v1 == pytest.approx(2 * 1e12 / 15e-3 / 1e12)
    assert (mid0, mid1) == (3, 10)                     # 7 matrices per layer
    assert s0 != s1                                    # different seeded weights


def test_single_rank_needs_no_process_group():
    import bench
    assert bench.max_over_ranks(3.5, 1) == 3.5
    assert bench.aggregate_tflops(2e12, 1, 1000.0) == pytest.approx(2.0)
