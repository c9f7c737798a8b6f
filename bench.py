#!/usr/bin/env python
"""Benchmark of the LowRA quantized-LoRA hot path on B200.

A *step* is one pass of the whole hot path over one workload, through the C ABI: for every weight matrix
lowra_encode, lowra_decode, lowra_lora_forward and (where the workload has it) lowra_lora_backward_input.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload {2,3,4,5}] [--impl reference]
    python bench.py --case NAME        # one small launch of one kernel family, sized for a profiler capture

Workloads (the configurations of the benchmark spec; 3 is the default and the headline):
    2  one 4096 x 4096 matrix at 2048 tokens, 2.1 bits on average (run on 8 seeded matrices of that shape per
       step, so that a step's inputs exceed the L2 cache)
    3  one Llama-7B-shaped decoder layer (7 matrices), 4096 tokens, 1.5 bits
    4  one Llama-13B-shaped decoder layer, 4096 tokens, 1.15 bits
    5  a whole 32-layer Llama-7B-shaped model (224 matrices, 6.5 G parameters), 2.5 bits: encode + decode sweep
       over every matrix, forward at 1024 / 4096 / 8192 tokens per matrix (no backward)
Codebooks are learnt on the GPU before the timed region (lowra_learn_codebooks: 10 rounds of weighted Lloyd-Max
per row from the paper's Appendix-F starting tables), as the configurations say.

Prints ONE JSON line.  `value` is the fused dequant+LoRA product throughput of the step (algorithmic FLOPs of
the products divided by the time of the WHOLE step, encode and decode included), measured with CUDA events and
inputs resident in HBM; `phases` breaks the step down; `per_matrix` gives every (matrix, operation) its own
figure; `e2e` repeats the step with host buffers and the host<->device copies inside the timed region;
`roofline` is for the dominant kernel (the fused tensor-core kernel) and carries, under `secondary`, the HBM
figures of decode and encode taken over several GB of distinct buffers (so that what is still in L2 when the
clock stops is a few per cent); `cpu_baseline` times the CPU oracle on a bounded sample of the same workload and
holds the GPU's results of that sample against the oracle's.

With N > 1 (torchrun) every rank runs the same shapes on its own seeded weights (independent problems, no
data-path collective; weak scaling) and rank 0 reports the aggregate.

`--impl reference` times the CPU oracle alone (there is no reference code for this paper).
"""
from __future__ import annotations

import argparse
import json
import math
import os
import statistics
import subprocess
import sys
import threading
import time
from concurrent.futures import ThreadPoolExecutor

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import synth_inputs as si  # noqa: E402

METRIC = "fused dequant+LoRA product throughput over one step (encode + decode + forward + backward-input of every matrix)"
UNIT = "TFLOP/s"
LLOYD_ITERS = 10
SWEEP_BYTES = 3.2e9          # decode / encode HBM figures are taken over at least this much output (input)
L2_BYTES = 126e6


def gemm_flops(M, N, K, r):
    """Algorithmic FLOPs of one forward (or one backward-input) call."""
    return 2.0 * M * N * K + 2.0 * M * r * (K + N)


def decode_bytes(N, K, bits):
    return N * K * (bits / 8.0 + 4.0 / 64.0 + 2.0)   # packed codes + absmax in, bf16 out (tables: < 0.1 %, not counted)


def encode_bytes(N, K, bits):
    return N * K * (4.0 + bits / 8.0 + 4.0 / 64.0)


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return dict(hbm=float(p["hbm_gbs"]), tensor_burst=float(p["bf16_tflops"]),
                    tensor_sustained=float(p.get("bf16_tflops_sustained", p["bf16_tflops"])), source="measured")
    return dict(hbm=6650.0, tensor_burst=1590.0, tensor_sustained=1400.0, source="fallback")


# --------------------------------------------------------------------------------------------------
# clocks sampling
# --------------------------------------------------------------------------------------------------
class ClockSampler:
    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu_index = gpu_index
        self.proc = None
        self.lines = []
        self.thread = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.gpu_index}", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits",
                 "-lms", "20"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._read, daemon=True)
        self.thread.start()

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append((time.time(), line.strip()))

    def stop(self, t0: float, t1: float) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=2)
        except Exception:
            self.proc.kill()
        sm, smax, reasons = [], [], set()
        # samples taken while the GPU was working: a line arrives a few milliseconds after it was sampled; when the
        # region is shorter than that allows, the window is widened by one sampling period on either side
        for lo, hi in ((t0 + 0.004, t1 + 0.004), (t0 - 0.02, t1 + 0.03)):
            for ts, line in self.lines:
                parts = [p.strip() for p in line.split(",")]
                if len(parts) < 9:
                    continue
                try:
                    clk, mx = float(parts[1]), float(parts[2])
                except ValueError:
                    continue
                if lo <= ts <= hi:
                    sm.append(clk)
                    smax.append(mx)
                    for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"),
                                         parts[5:9]):
                        if val.lower().startswith("active"):
                            reasons.add(name)
            if len(sm) >= 2:
                break
        if not sm:  # region shorter than the sampling period: take everything seen
            for ts, line in self.lines:
                parts = [p.strip() for p in line.split(",")]
                try:
                    sm.append(float(parts[1])); smax.append(float(parts[2]))
                except Exception:
                    pass
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(smax) if smax else None,
                "sm_min_mhz": min(sm) if sm else None, "reasons": sorted(reasons), "samples": len(sm)}


# --------------------------------------------------------------------------------------------------
# workload
# --------------------------------------------------------------------------------------------------
def workload_matrices(workload: int):
    """(config, list of matrices of one step).  Workload 2 runs its one shape on 8 seeded matrices per step so
    that the step's inputs exceed L2 between timed iterations."""
    cfg = si.config(workload)
    mats = list(cfg.matrices)
    if workload == 2:
        mats = [si.Matrix(f"{mats[0].name}#{i}", mats[0].N, mats[0].K, i) for i in range(8)]
    return cfg, mats


def rank_matrix_id(matrix_id: int, rank: int, per_rank: int = 7) -> int:
    """Ranks hold different weights: the seed stream of matrix j on rank q is that of matrix j + per_rank * q."""
    return matrix_id + per_rank * rank


def host_matrix(cfg, mat, rank: int, per_rank: int):
    mid = rank_matrix_id(mat.matrix_id, rank, per_rank)
    W = si.weights(mat.N, mat.K, matrix_id=mid, kind=cfg.weight_kind)
    precs = si.precisions(mat.N, cfg.mix, matrix_id=mid)
    A, B = si.lora_factors(mat.K, mat.N, cfg.rank, matrix_id=mid % 7)      # factors repeat from layer to layer
    return dict(name=mat.name, N=mat.N, K=mat.K, W=W, precs=precs, A=A, B=B, matrix_id=mid)


# DRAM traffic of one fused_kernel launch measured with ncu (dram__bytes_read.sum + dram__bytes_write.sum) on a
# launch of workload 3: the backward-input pass of gate_proj (dX [4096, 4096] from dY [4096, 11008];
# profiles/fused_backward_input_11008x4096_m4096_streamk.md): 169.0 MB read + 26.9 MB written.  The bytes the call
# has to read and write once are 137 MB (the output is partly still in L2 when the kernel ends; the stream-K partial
# tiles add 19 MB each way).  Scaled to the step's average launch in proportion to those input + output bytes.
NCU_CASE = dict(N=4096, K=11008, M=4096, r=64, bits=1.5, dram_bytes=169.0e6 + 26.9e6)


def fused_io_bytes(N, K, M, r, bits):
    """Bytes a fused call has to read and write once: activations, packed codes, absmax, tables, factors; output."""
    return 2.0 * M * K + N * K * (bits / 8 + 4 / 64) + 64.0 * N + 2.0 * (K + N) * r + 2.0 * M * N


def fused_traffic_per_launch(calls, r, bits):
    """calls: (N, K, M) of every fused launch of a step, with N = rows of the operand that is dequantised."""
    case = fused_io_bytes(NCU_CASE["N"], NCU_CASE["K"], NCU_CASE["M"], NCU_CASE["r"], NCU_CASE["bits"])
    per = [fused_io_bytes(N, K, M, r, bits) for N, K, M in calls]
    return NCU_CASE["dram_bytes"] / case * sum(per) / len(per)


def max_over_ranks(ms: float, world: int, device="cuda") -> float:
    """Slowest rank's time: the job is done when its last rank is (all-reduce MAX over the process group)."""
    if world <= 1:
        return float(ms)
    import torch
    import torch.distributed as dist
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_tflops(flops_per_rank_step: float, world: int, ms_per_step: float) -> float:
    """Whole-job throughput: every rank does one step's work per step (weak scaling)."""
    return world * flops_per_rank_step / (ms_per_step * 1e-3) / 1e12


def run_gpu(args):
    import torch
    import torch.distributed as dist

    import paper_2502_08141_b200 as lw

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    lw.lib()

    cfg, mat_list = workload_matrices(args.workload)
    token_counts = list(cfg.tokens)
    with_backward = "backward" in cfg.ops
    r, s = cfg.rank, cfg.s
    bits = si.avg_bits(cfg.mix)
    per_rank = len(mat_list)
    y0, t0 = si.initial_codebooks()

    bfv = lambda t: t.view(torch.bfloat16)
    stream = torch.cuda.current_stream()
    # ---- device-resident problem: weights are drawn on the host (seeded, one matrix after the other, a few threads
    # ahead of the uploads) and stay in HBM; codebooks are learnt here, on the GPU, from the Appendix-F tables
    dev = []
    t_gen = time.time()
    with ThreadPoolExecutor(max_workers=min(os.cpu_count() or 8, 32, len(mat_list))) as ex:
        for m in ex.map(lambda mat: host_matrix(cfg, mat, rank, per_rank), mat_list):
            layout = lw.Layout(m["precs"], m["K"])
            if not args.deal_per_call:
                layout.build_deal()     # the deal of the rows depends on the precisions only: once per weight, like the plan
            N, K = m["N"], m["K"]
            d = dict(name=m["name"], N=N, K=K, layout=layout, matrix_id=m["matrix_id"],
                     W=torch.from_numpy(m["W"]).cuda(),
                     A=bfv(torch.from_numpy(m["A"].view(np.int16)).cuda()), B=bfv(torch.from_numpy(m["B"].view(np.int16)).cuda()),
                     maps=torch.empty((N, 16), dtype=torch.float32, device="cuda"),
                     thr=torch.empty((N, 16), dtype=torch.float32, device="cuda"),
                     packed=torch.empty(max(layout.packed_bytes, 16), dtype=torch.uint8, device="cuda"),
                     absmax=torch.empty((N, K // 64), dtype=torch.float32, device="cuda"),
                     What=torch.empty((N, K), dtype=torch.bfloat16, device="cuda"))
            lw.lowra_learn_codebooks(layout, d["W"], y0, t0, LLOYD_ITERS, maps=d["maps"], thresholds=d["thr"])
            if len(dev) < 7:
                d["host"] = m            # kept for the end-to-end leg and the check against the oracle
            dev.append(d)
    torch.cuda.synchronize()
    t_gen = time.time() - t_gen
    shapes = sorted({(d["N"], d["K"]) for d in dev})
    widths = sorted({w for N, K in shapes for w in (N, K)})
    # one activation / output-gradient buffer per (token count, width), shared by the matrices of that width; one
    # output buffer per (token count, width) when the workload has many matrices, one per matrix otherwise
    act_dev = {}
    for M in token_counts:
        for wdt in widths:
            act_dev[(M, wdt)] = bfv(torch.from_numpy(si.activations(M, wdt, matrix_id=100 + rank).view(np.int16)).cuda())
    # Inputs per matrix: the projections that read the same activations in a decoder layer share X (q, k, v; gate and
    # up), every other matrix has its own; every matrix has its own output gradient.  Distinct buffers are the width's
    # seeded buffer rotated by a few token rows (the first matrix of the workload keeps the unrotated one).
    GROUPS = {"q_proj": "qkv", "k_proj": "qkv", "v_proj": "qkv", "gate_proj": "gate_up", "up_proj": "gate_up"}
    x_groups, x_bufs, g_bufs = [], {}, {}
    for i, d in enumerate(dev):
        d["group"] = GROUPS.get(d["name"], d["name"])
        if d["group"] not in x_groups:
            x_groups.append(d["group"])
        gi, j = x_groups.index(d["group"]) % 7, i % 7
        d["X"], d["G"] = {}, {}
        for M in token_counts:
            kx, kg = (M, d["K"], gi), (M, d["N"], j)
            if kx not in x_bufs:
                x_bufs[kx] = act_dev[(M, d["K"])] if gi == 0 else torch.roll(act_dev[(M, d["K"])], 37 * gi, dims=0)
            if kg not in g_bufs and with_backward:
                g_bufs[kg] = act_dev[(M, d["N"])] if j == 0 else torch.roll(act_dev[(M, d["N"])], 53 * j, dims=0)
            d["X"][M] = x_bufs[kx]
            d["G"][M] = g_bufs.get(kg)
    shared_out = len(dev) > 8
    out_shared = {}

    def out_buf(d, M, cols, key):
        if shared_out:
            k = (M, cols, key)
            if k not in out_shared:
                out_shared[k] = torch.empty((M, cols), dtype=torch.bfloat16, device="cuda")
            return out_shared[k]
        return torch.empty((M, cols), dtype=torch.bfloat16, device="cuda")

    for d in dev:
        d["Y"] = {M: out_buf(d, M, d["N"], "Y") for M in token_counts}
        d["dX"] = {M: out_buf(d, M, d["K"], "dX") for M in token_counts} if with_backward else None
    ws_shared = {}
    for d in dev:
        d["ws"] = {}
        for M in token_counts:
            n = lw.lowra_workspace_bytes(d["layout"], M, r)
            if shared_out:      # calls on one stream never overlap: one workspace per token count, sized for the largest
                if M not in ws_shared or ws_shared[M].numel() < n:
                    ws_shared[M] = torch.empty(n, dtype=torch.uint8, device="cuda")
                d["ws"][M] = None
            else:
                d["ws"][M] = lw.lowra_workspace_init(torch.empty(n, dtype=torch.uint8, device="cuda"))
    if shared_out:
        for M in token_counts:
            lw.lowra_workspace_init(ws_shared[M])
        for d in dev:
            for M in token_counts:
                d["ws"][M] = ws_shared[M]
    all_ws = list({id(w): w for d in dev for w in d["ws"].values()}.values())

    def check_status(where):
        for w in all_ws:
            st = lw.lowra_device_status(w)
            if st != 0:
                raise SystemExit(f"device status {st} ({lw.status_string(st)}) {where}")

    f_encode = lambda d, M=None: lw.lowra_encode(d["layout"], d["W"], d["thr"], packed=d["packed"], absmax=d["absmax"])
    f_decode = lambda d, M=None: lw.lowra_decode(d["layout"], d["packed"], d["absmax"], d["maps"], out=d["What"])
    f_forward = lambda d, M: lw.lowra_lora_forward(d["layout"], d["packed"], d["absmax"], d["maps"], d["X"][M],
                                                   d["A"], d["B"], s, Y=d["Y"][M], workspace=d["ws"][M])
    f_backward = lambda d, M: lw.lowra_lora_backward_input(d["layout"], d["packed"], d["absmax"], d["maps"], d["G"][M],
                                                           d["A"], d["B"], s, dX=d["dX"][M], workspace=d["ws"][M])
    phase_list = [("encode", f_encode, [None]), ("decode", f_decode, [None]), ("forward", f_forward, token_counts)]
    if with_backward:
        phase_list.append(("backward", f_backward, token_counts))
    # The q, k and v projections of a layer (one shape, one input) go through the one-launch batch calls, as a layer
    # would issue them; everything else is a call per matrix.  units: lists of matrix indices, one list per launch.
    units, i = [], 0
    while i < len(dev):
        j = i + 1
        if dev[i]["group"] == "qkv" and not args.deal_per_call and not args.no_batch and not shared_out:
            while (j < len(dev) and j - i < 4 and dev[j]["group"] == "qkv" and (dev[j]["N"], dev[j]["K"]) == (dev[i]["N"], dev[i]["K"])):
                j += 1
        units.append(list(range(i, j)))
        i = j
    batch_ws, batch_members = {}, {}
    for u in units:
        if len(u) > 1:
            for M in token_counts:
                n = lw.lowra_batch_workspace_bytes(dev[u[0]]["layout"], len(u), M, r)
                batch_ws[(u[0], M)] = lw.lowra_workspace_init(torch.empty(n, dtype=torch.uint8, device="cuda"))
                common = lambda d: dict(layout=d["layout"], packed=d["packed"], absmax=d["absmax"], maps=d["maps"], A=d["A"], B=d["B"])
                batch_members[("forward", u[0], M)] = [dict(common(dev[k]), act=dev[k]["X"][M], out=dev[k]["Y"][M]) for k in u]
                if with_backward:
                    batch_members[("backward", u[0], M)] = [dict(common(dev[k]), act=dev[k]["G"][M], out=dev[k]["dX"][M]) for k in u]
            all_ws.extend(batch_ws[(u[0], M)] for M in token_counts)

    # encode and decode: the matrices of a layer in one launch each (lowra_encode_group / lowra_decode_group, up to eight
    # members, the largest first), as a layer or a model is quantised; --no-batch: a call per matrix
    codec_groups = []
    if not args.no_batch:
        gsz = 7 if len(dev) > lw.LOWRA_MAX_GROUP else lw.LOWRA_MAX_GROUP      # a model: layer by layer (seven matrices)
        for g0 in range(0, len(dev), gsz):
            idx = sorted(range(g0, min(g0 + gsz, len(dev))), key=lambda i: -dev[i]["N"] * dev[i]["K"])
            codec_groups.append((
                [dict(layout=dev[i]["layout"], W=dev[i]["W"], thresholds=dev[i]["thr"], packed=dev[i]["packed"], absmax=dev[i]["absmax"]) for i in idx],
                [dict(layout=dev[i]["layout"], packed=dev[i]["packed"], absmax=dev[i]["absmax"], maps=dev[i]["maps"], out=dev[i]["What"]) for i in idx]))

    def run_unit(name, fn, u, M):
        if len(u) == 1 or name in ("encode", "decode"):
            for k in u:
                fn(dev[k], M)
        elif name == "forward":
            lw.lowra_lora_forward_batch(batch_members[(name, u[0], M)], s, batch_ws[(u[0], M)])
        else:
            lw.lowra_lora_backward_input_batch(batch_members[(name, u[0], M)], s, batch_ws[(u[0], M)])

    def step(record=None, per_call=None):
        """One pass.  `record` (a list) receives (phase, event_start, event_end) per phase: the calls of a phase
        run back to back, as a user would issue them; `per_call` receives the same per call (diagnostic pass)."""
        for name, fn, Ms in phase_list:
            if record is not None:
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(stream)
            for M in Ms:
                if per_call is not None:          # diagnostic pass: a call per matrix, events around each
                    for i, d in enumerate(dev):
                        c0, c1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                        c0.record(stream); fn(d, M); c1.record(stream)
                        per_call.append((name, M, i, c0, c1))
                elif codec_groups and name == "encode":
                    for enc_members, _ in codec_groups:
                        lw.lowra_encode_group(enc_members)
                elif codec_groups and name == "decode":
                    for _, dec_members in codec_groups:
                        lw.lowra_decode_group(dec_members)
                else:
                    for u in units:
                        run_unit(name, fn, u, M)
            if record is not None:
                e1.record(stream)
                record.append((name, e0, e1))

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    n_warm = max(args.warmup, 3)
    for _ in range(n_warm):
        step()
    check_status("after warm-up")

    # ---- timed region: exactly K steps, device timing with CUDA events, max over ranks
    sampler = ClockSampler(local_rank)
    sampler.start()
    time.sleep(0.25)
    barrier()
    records = []
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0w = time.time()
    ev0.record(stream)
    for _ in range(args.steps):
        step(records)
    ev1.record(stream)
    barrier()
    t1w = time.time()
    clocks = sampler.stop(t0w, t1w)
    total_ms = ev0.elapsed_time(ev1)
    total_ms = max_over_ranks(total_ms, world)
    ms_per_step = total_ms / args.steps
    check_status("after the timed steps")

    dirs = 2 if with_backward else 1
    flops_dir = sum(gemm_flops(M, d["N"], d["K"], r) for M in token_counts for d in dev)
    flops_step = dirs * flops_dir
    value = aggregate_tflops(flops_step, world, ms_per_step)

    phase_ms = {}
    for phase, e0, e1 in records:
        phase_ms[phase] = phase_ms.get(phase, 0.0) + e0.elapsed_time(e1)
    for k in phase_ms:
        phase_ms[k] /= args.steps
    # the fused phases step by step: the power cap sets in some tens of milliseconds into a run of tensor-core calls
    n_ph = len(phase_list)
    fused_ms_by_step = [round(sum(e0.elapsed_time(e1) for ph, e0, e1 in records[i * n_ph:(i + 1) * n_ph] if ph in ("forward", "backward")), 3)
                        for i in range(args.steps)]
    # diagnostic pass outside the timed region: the same step with events around every call
    n_diag = 3 if len(dev) <= 8 else 1
    calls = []
    for _ in range(n_diag):
        step(per_call=calls)
    torch.cuda.synchronize()
    call_ms = {}
    for phase, M, i, c0, c1 in calls:
        call_ms[(phase, M, i)] = call_ms.get((phase, M, i), 0.0) + c0.elapsed_time(c1) / n_diag
    elems = sum(d["N"] * d["K"] for d in dev)
    P = peaks()
    dec_bytes = sum(decode_bytes(d["N"], d["K"], bits) for d in dev)
    enc_bytes = sum(encode_bytes(d["N"], d["K"], bits) for d in dev)
    dec_gbs = dec_bytes / (phase_ms["decode"] * 1e-3) / 1e9
    enc_gbs = enc_bytes / (phase_ms["encode"] * 1e-3) / 1e9
    fwd_tf = flops_dir / (phase_ms["forward"] * 1e-3) / 1e12
    tens = lambda tf: {"TFLOP/s": tf, "frac_tensor_burst": tf / P["tensor_burst"], "frac_tensor_sustained": tf / P["tensor_sustained"],
                       "frac_tensor_nominal_2250": tf / 2250.0}
    phases = {
        "encode": {"ms": phase_ms["encode"], "GB/s": enc_gbs, "frac_hbm": enc_gbs / P["hbm"], "frac_hbm_nominal_8TBs": enc_gbs / 8000.0},
        "decode": {"ms": phase_ms["decode"], "GB/s": dec_gbs, "frac_hbm": dec_gbs / P["hbm"], "frac_hbm_nominal_8TBs": dec_gbs / 8000.0},
        "forward": dict(ms=phase_ms["forward"], **tens(fwd_tf)),
    }
    if with_backward:
        bwd_tf = flops_dir / (phase_ms["backward"] * 1e-3) / 1e12
        phases["backward_input"] = dict(ms=phase_ms["backward"], **tens(bwd_tf))
    # every (matrix shape, token count, operation): mean over the matrices of that shape (separate pass, events around every call)
    per_matrix = []
    for N, K in shapes:
        idx = [i for i, d in enumerate(dev) if (d["N"], d["K"]) == (N, K)]
        names = sorted({dev[i]["name"].split("#")[0] for i in idx})
        row = {"shape": f"{N}x{K}", "matrices": "/".join(names), "count": len(idx)}
        mean = lambda phase, M: sum(call_ms[(phase, M, i)] for i in idx) / len(idx)
        row["encode_GB/s"] = round(encode_bytes(N, K, bits) / (mean("encode", None) * 1e-3) / 1e9, 1)
        row["decode_GB/s"] = round(decode_bytes(N, K, bits) / (mean("decode", None) * 1e-3) / 1e9, 1)
        for M in token_counts:
            row[f"forward_TFLOP/s@{M}"] = round(gemm_flops(M, N, K, r) / (mean("forward", M) * 1e-3) / 1e12, 1)
            if with_backward:
                row[f"backward_input_TFLOP/s@{M}"] = round(gemm_flops(M, N, K, r) / (mean("backward", M) * 1e-3) / 1e12, 1)
        per_matrix.append(row)

    # ---- decode and encode as HBM figures: several GB of distinct buffers inside one event pair, so that the part of
    # the output still dirty in L2 when the clock stops (at most one L2's worth) is a few per cent of the bytes
    out_layer = sum(d["N"] * d["K"] * 2.0 for d in dev)
    secondary = {}
    if out_layer >= SWEEP_BYTES:      # the step's own sweep is long enough (workload 5)
        for key, gbs, ms, by in (("decode", dec_gbs, phase_ms["decode"], dec_bytes), ("encode", enc_gbs, phase_ms["encode"], enc_bytes)):
            secondary[key] = {"bound": "hbm", "achieved": gbs, "peak": P["hbm"], "unit": "GB/s", "frac": gbs / P["hbm"],
                              "frac_nominal_8TBs": gbs / 8000.0, "bytes": by, "ms": ms, "launches": len(codec_groups) if codec_groups else len(dev),
                              "how": "the step's own sweep over every matrix of the model (one event pair per phase)"}
    else:
        n_sets = int(math.ceil(SWEEP_BYTES / out_layer))
        what_sets = [[torch.empty_like(d["What"]) for d in dev] for _ in range(n_sets)]
        in_layer = sum(d["N"] * d["K"] * 4.0 for d in dev)
        n_w = max(1, int(math.ceil(8 * L2_BYTES / in_layer)))           # copies of W so that re-reads never hit L2
        w_sets = [[d["W"] if j == 0 else d["W"].clone() for d in dev] for j in range(n_w)]
        pk_sets = [[(torch.empty_like(d["packed"]), torch.empty_like(d["absmax"])) for d in dev] for _ in range(min(n_sets, 4))]

        # largest matrices first in every pass: the host (a Python call per launch) is then ahead of the GPU when the
        # short launches come, so that the figure is the kernels' and not the interpreter's
        order = sorted(range(len(dev)), key=lambda i: -dev[i]["N"] * dev[i]["K"])

        def decode_sweep(grouped):
            for ws_ in what_sets:
                if grouped:
                    lw.lowra_decode_group([dict(layout=dev[i]["layout"], packed=dev[i]["packed"], absmax=dev[i]["absmax"],
                                                maps=dev[i]["maps"], out=ws_[i]) for i in order])
                else:
                    for i in order:
                        d = dev[i]
                        lw.lowra_decode(d["layout"], d["packed"], d["absmax"], d["maps"], out=ws_[i])

        def encode_sweep(grouped):
            for j in range(n_sets):
                if grouped:
                    lw.lowra_encode_group([dict(layout=dev[i]["layout"], W=w_sets[j % n_w][i], thresholds=dev[i]["thr"],
                                                packed=pk_sets[j % len(pk_sets)][i][0], absmax=pk_sets[j % len(pk_sets)][i][1])
                                           for i in order])
                else:
                    for i in order:
                        d = dev[i]
                        pk, am = pk_sets[j % len(pk_sets)][i]
                        lw.lowra_encode(d["layout"], w_sets[j % n_w][i], d["thr"], packed=pk, absmax=am)

        def best_of_three(fn, grouped):
            fn(grouped)
            torch.cuda.synchronize()
            best = None
            for _ in range(3):
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record(stream); fn(grouped); b.record(stream)
                torch.cuda.synchronize()
                ms = a.elapsed_time(b)
                best = ms if best is None else min(best, ms)
            return best

        grouped = bool(codec_groups) and len(dev) <= lw.LOWRA_MAX_GROUP
        for key, fn, by in (("decode", decode_sweep, dec_bytes), ("encode", encode_sweep, enc_bytes)):
            best = best_of_three(fn, grouped)
            gbs = n_sets * by / (best * 1e-3) / 1e9
            secondary[key] = {"bound": "hbm", "achieved": gbs, "peak": P["hbm"], "unit": "GB/s", "frac": gbs / P["hbm"],
                              "frac_nominal_8TBs": gbs / 8000.0, "bytes": n_sets * by, "ms": best,
                              "launches": n_sets * (1 if grouped else len(dev)),
                              "how": f"{n_sets} passes over the step's matrices back to back inside one event pair, every pass "
                                     f"into its own output buffers ({n_sets * out_layer / 1e9:.1f} GB of distinct decode output; "
                                     f"encode reads {n_w} cop{'y' if n_w == 1 else 'ies'} of the weights in turn); best of 3; " +
                                     ("the matrices of a pass in one launch (lowra_%s_group)" % key if grouped else "a launch per matrix")}
            if grouped:          # the same sweep with a launch per matrix, for comparison
                single = best_of_three(fn, False)
                secondary[key]["a_launch_per_matrix"] = {"achieved": n_sets * by / (single * 1e-3) / 1e9,
                                                         "frac": n_sets * by / (single * 1e-3) / 1e9 / P["hbm"], "ms": single}
        del what_sets, w_sets, pk_sets
        # the packed codes in d["packed"] were not touched by the sweeps (they wrote their own buffers)

    # dominant kernel: the fused tensor-core kernel (forward + backward launches), timed as whole calls
    fused_ms = phase_ms["forward"] + (phase_ms["backward"] if with_backward else 0.0)
    achieved = flops_step / (fused_ms * 1e-3) / 1e12
    # denominator: the cuBLAS bf16 figure of the clock regime this run was in - the burst figure while the SM clock
    # stayed at its maximum (a timed region of tens of milliseconds), the sustained one when the power cap held it
    # below (hundreds of steps); both fractions are reported either way
    sm_now, sm_max = clocks.get("sm_mhz"), clocks.get("sm_max_mhz")
    capped = bool(sm_now and sm_max and sm_now < 0.95 * sm_max)
    peak = P["tensor_sustained"] if capped else P["tensor_burst"]
    fused_calls = [(d["N"], d["K"], M) for M in token_counts for d in dev]
    if with_backward:
        fused_calls += [(d["K"], d["N"], M) for M in token_counts for d in dev]   # backward reads dY [M, N], writes dX [M, K]
    # the steps that ran before the power limiter set in (within 2 % of the fastest step): the same figure over those alone
    fastest = min(fused_ms_by_step)
    quick = [m for m in fused_ms_by_step if m <= 1.02 * fastest]
    tf_quick = flops_step / (sum(quick) / len(quick) * 1e-3) / 1e12
    before_limit = {"steps": len(quick), "of": args.steps, "achieved": tf_quick, "frac_burst": tf_quick / P["tensor_burst"],
                    "what": "fused phases of the steps within 2 % of the fastest one (the power limiter slows the later steps of a run, see ms_by_step)"}
    roofline = {"bound": "tensor", "kernel": "fused_kernel (forward" + (" + backward-input" if with_backward else "") + " calls" +
                                              (", prologue launch included)" if args.deal_per_call else ")"),
                "achieved": achieved, "peak": peak, "unit": "TFLOP/s", "frac": achieved / peak,
                "peak_burst": P["tensor_burst"], "frac_burst": achieved / P["tensor_burst"],
                "peak_sustained": P["tensor_sustained"], "frac_sustained": achieved / P["tensor_sustained"],
                "peak_source": P["source"] + (" (sustained figure: the SM clock was held below its maximum during the timed region)"
                                              if capped else " (burst figure: the SM clock stayed at its maximum during the timed region)"),
                "traffic": fused_traffic_per_launch(fused_calls, r, bits),
                "traffic_source": "ncu dram__bytes_read.sum + dram__bytes_write.sum of the gate_proj backward-input launch of "
                                  "workload 3 (profiles/fused_backward_input_11008x4096_m4096_streamk.md), scaled by the "
                                  "input + output bytes of this step's average launch",
                "ms_by_step": fused_ms_by_step if args.steps <= 64 else fused_ms_by_step[:32] + fused_ms_by_step[-32:],
                "before_power_limit": before_limit,
                "secondary": secondary}

    # ---- end to end: host buffers, pinned, copies inside the timed region (the first seven matrices of the workload)
    e2e = None
    if not args.no_e2e:
        e2e = run_e2e(args, lw, torch, dev[:7], token_counts[-1] if args.workload != 5 else 4096, act_dev, token_counts, r, s,
                      with_backward, stream, barrier, world, len(dev))
        check_status("after the end-to-end steps")

    # ---- outside the step: learner, adapter gradients, quantisation error on (at most) the first seven matrices
    extras = None
    if rank == 0 and not args.no_extras:
        extras = run_extras(lw, torch, dev[:7], token_counts[0] if args.workload != 5 else 4096, act_dev, r, s, stream, P, y0, t0)

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu:
        cpu = cpu_baseline_sample(args.workload, gpu=dict(lw=lw, torch=torch, d=dev[0], act=act_dev, M=token_counts[0], r=r, s=s,
                                                          with_backward=with_backward))

    if rank == 0:
        n_fused = len(units) * len(token_counts) * (2 if with_backward else 1)     # fused launches per step
        out = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": n_warm, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": f"config {args.workload}: {cfg.name}, {len(dev)} matrices, tokens {token_counts}, rank {r}, "
                                   f"mix {cfg.mix} (avg {bits:.2f} bits), codebooks learnt on the GPU "
                                   f"({LLOYD_ITERS} rounds of weighted Lloyd-Max per row from the Appendix-F tables)",
                       "elements": elems,
                       "l2": f"inputs larger than L2 ({(elems * 4 + out_layer) / 1e9:.1f} GB of weights read and written per step)",
                       "row_deal": "in every call (prologue launch)" if args.deal_per_call else
                                   "once per weight (lowra_deal_build), outside the step like the storage plan",
                       "launches": "one call per matrix" if all(len(u) == 1 for u in units) else
                                   "q, k and v projections (one shape, one input) through lowra_lora_forward_batch / "
                                   "lowra_lora_backward_input_batch, one launch per direction; every other matrix a call "
                                   "of its own; per_matrix figures are single calls",
                       "codec_launches": ("encode and decode: the matrices of a layer in one launch each (lowra_encode_group / "
                                          "lowra_decode_group); per_matrix figures are single calls") if codec_groups else "a launch per matrix",
                       "inputs": "q/k/v share X, gate/up share X, every other matrix its own; one output gradient per matrix",
                       "host_generation_s": round(t_gen, 1)},
            "phases": phases, "per_matrix": per_matrix, "roofline": roofline, "e2e": e2e, "cpu_baseline": cpu, "extras": extras,
            "gpu_launches": args.steps * ((2 * len(codec_groups) if codec_groups else 2 * len(dev)) + n_fused * (2 if args.deal_per_call else 1)), "clocks": clocks,
        }
        print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


def run_e2e(args, lw, torch, dev, M, act_dev, token_counts, r, s, with_backward, stream, barrier, world, n_all):
    """The same calls with HOST buffers: every step uploads the step's inputs from pinned memory and downloads its
    results.  Three streams: uploads, kernels, downloads - matrix i + 1 arrives while matrix i is computed and matrix
    i - 1 leaves; every buffer has its own events, so none is overwritten before its last reader is done."""
    pin = lambda a: torch.from_numpy(np.ascontiguousarray(a)).pin_memory()
    if M not in token_counts:
        M = token_counts[0]
    host = []
    for d in dev:
        m = d["host"]
        h = dict(W=pin(m["W"]), thr=d["thr"].cpu().pin_memory(), maps=d["maps"].cpu().pin_memory(),
                 A=pin(m["A"].view(np.int16)), B=pin(m["B"].view(np.int16)),
                 Y=torch.empty((M, d["N"]), dtype=torch.bfloat16).pin_memory())
        if with_backward:
            h["dX"] = torch.empty((M, d["K"]), dtype=torch.bfloat16).pin_memory()
        host.append(h)
    act_host = {k: act_dev[(M, k)].view(torch.int16).cpu().pin_memory() for k in sorted({w for d in dev for w in (d["N"], d["K"])})}
    nbytes = lambda t: t.numel() * t.element_size()
    h2d = sum(nbytes(h[k]) for h in host for k in ("W", "thr", "maps", "A", "B")) \
        + sum(nbytes(act_host[d["K"]]) + (nbytes(act_host[d["N"]]) if with_backward else 0) for d in dev)
    d2h = sum(nbytes(h[k]) for h in host for k in ("Y", "dX") if k in h)
    s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()
    xs = [torch.empty_like(act_dev[(M, d["K"])]) for d in dev]      # per-matrix activations / output gradients
    gs = [torch.empty_like(act_dev[(M, d["N"])]) for d in dev] if with_backward else None
    Ys = [torch.empty((M, d["N"]), dtype=torch.bfloat16, device="cuda") for d in dev]
    dXs = [torch.empty((M, d["K"]), dtype=torch.bfloat16, device="cuda") for d in dev] if with_backward else None
    ev_in = [torch.cuda.Event() for _ in dev]
    ev_done = [None] * len(dev)
    ev_out = [None] * len(dev)

    def e2e_step():
        for i, (d, h) in enumerate(zip(dev, host)):
            with torch.cuda.stream(s_in):
                if ev_done[i] is not None:
                    s_in.wait_event(ev_done[i])                      # the previous step's kernels have read them
                d["W"].copy_(h["W"], non_blocking=True); d["thr"].copy_(h["thr"], non_blocking=True)
                d["maps"].copy_(h["maps"], non_blocking=True)
                d["A"].view(torch.int16).copy_(h["A"], non_blocking=True)
                d["B"].view(torch.int16).copy_(h["B"], non_blocking=True)
                xs[i].view(torch.int16).copy_(act_host[d["K"]], non_blocking=True)
                if with_backward:
                    gs[i].view(torch.int16).copy_(act_host[d["N"]], non_blocking=True)
                ev_in[i].record(s_in)
            stream.wait_event(ev_in[i])
            if ev_out[i] is not None:
                stream.wait_event(ev_out[i])                         # the previous step's results have left
            lw.lowra_encode(d["layout"], d["W"], d["thr"], packed=d["packed"], absmax=d["absmax"])
            lw.lowra_decode(d["layout"], d["packed"], d["absmax"], d["maps"], out=d["What"])
            lw.lowra_lora_forward(d["layout"], d["packed"], d["absmax"], d["maps"], xs[i], d["A"], d["B"], s, Y=Ys[i], workspace=d["ws"][M])
            if with_backward:
                lw.lowra_lora_backward_input(d["layout"], d["packed"], d["absmax"], d["maps"], gs[i], d["A"], d["B"], s, dX=dXs[i],
                                             workspace=d["ws"][M])
            ev_done[i] = torch.cuda.Event(); ev_done[i].record(stream)
            with torch.cuda.stream(s_out):
                s_out.wait_event(ev_done[i])
                h["Y"].copy_(Ys[i], non_blocking=True)
                if with_backward:
                    h["dX"].copy_(dXs[i], non_blocking=True)
                ev_out[i] = torch.cuda.Event(); ev_out[i].record(s_out)

    def e2e_join():   # the step is over when its last download is
        for e in ev_out:
            if e is not None:
                stream.wait_event(e)

    e2e_step()
    e2e_join()
    barrier()
    n_e2e = max(1, args.steps)
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record(stream)
    for _ in range(n_e2e):
        e2e_step()
    e2e_join()
    b.record(stream)
    barrier()
    ms = a.elapsed_time(b) / n_e2e
    ms = max_over_ranks(ms, world)
    flops = (2 if with_backward else 1) * sum(gemm_flops(M, d["N"], d["K"], r) for d in dev)
    note = ("uploads, kernels and downloads on three streams: a matrix is computed while the next one arrives and the "
            "previous one leaves")
    if len(dev) < n_all or len(token_counts) > 1:
        note += f"; bounded sample of the workload: its first {len(dev)} matrices at {M} tokens"
    return {"value": aggregate_tflops(flops, world, ms), "unit": UNIT, "ms_per_step": ms,
            "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h), "steps": n_e2e, "note": note}


def run_extras(lw, torch, dev, M, act_dev, r, s, stream, P, y0, t0):
    """Kernels around the step, timed on the same matrices: the codebook learner (the stage before encode), the
    gradients of the low-rank factors, the per-channel quantisation error."""
    if (M, dev[0]["K"]) not in act_dev:
        M = sorted({k[0] for k in act_dev})[0]
    elems = sum(d["N"] * d["K"] for d in dev)

    def timed(fn):
        fn()
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream); fn(); b.record(stream)
        torch.cuda.synchronize()
        return a.elapsed_time(b)

    extras = {"matrices": len(dev), "tokens": M}
    tabs = [(torch.empty_like(d["maps"]), torch.empty_like(d["thr"])) for d in dev]
    ms = timed(lambda: [lw.lowra_learn_codebooks(d["layout"], d["W"], y0, t0, LLOYD_ITERS, maps=mp, thresholds=th)
                        for d, (mp, th) in zip(dev, tabs)])
    extras["learn_codebooks"] = {"ms": ms, "iterations": LLOYD_ITERS, "GB/s": 4.0 * elems / (ms * 1e-3) / 1e9,
                                 "frac_hbm": 4.0 * elems / (ms * 1e-3) / 1e9 / P["hbm"],
                                 "element_passes_per_s": elems * LLOYD_ITERS / (ms * 1e-3),
                                 "note": "not part of the step; from the Appendix-F starting tables; algorithmic bytes = one read of W (4 B per element)"}
    # the same for all three precisions of every row in one pass (what the precision assigner starts from)
    tabs3 = [(torch.empty((3, d["N"], 16), dtype=torch.float32, device="cuda"),
              torch.empty((3, d["N"], 16), dtype=torch.float32, device="cuda")) for d in dev]
    ms = timed(lambda: [lw.lowra_learn_codebooks_all(d["W"], y0, t0, LLOYD_ITERS, maps3=m3, thresholds3=h3)
                        for d, (m3, h3) in zip(dev, tabs3)])
    extras["learn_codebooks_all_precisions"] = {
        "ms": ms, "iterations": LLOYD_ITERS, "element_passes_per_s": 3 * elems * LLOYD_ITERS / (ms * 1e-3),
        "note": "not part of the step; every row at 1, 2 and 4 bits from one read of W"}

    # the gradients of the low-rank factors (the other half of a training step's backward pass)
    ws_ad = torch.empty(lw.lowra_adapter_workspace_bytes(M, r), dtype=torch.uint8, device="cuda")
    grads = [(torch.empty_like(d["A"]), torch.empty_like(d["B"])) for d in dev]
    ms = timed(lambda: [lw.lowra_lora_backward_adapters(act_dev[(M, d["K"])], act_dev[(M, d["N"])], d["A"], d["B"], s,
                                                        dA=gA, dB=gB, workspace=ws_ad) for d, (gA, gB) in zip(dev, grads)])
    if lw.lowra_device_status(ws_ad) != 0:
        raise SystemExit("device status after the adapter gradients")
    ad_bytes = sum(2.0 * M * (d["K"] + d["N"]) for d in dev)      # X and dY once, bf16
    ad_flops = sum(4.0 * M * r * (d["K"] + d["N"]) for d in dev)
    extras["adapter_gradients"] = {"ms": ms, "GB/s": ad_bytes / (ms * 1e-3) / 1e9, "frac_hbm": ad_bytes / (ms * 1e-3) / 1e9 / P["hbm"],
                                   "TFLOP/s": ad_flops / (ms * 1e-3) / 1e12,
                                   "note": "not part of the step; algorithmic bytes = X and dY read once"}

    # the same gradients from the down-projections that forward and backward-input leave in their workspaces: X and dY
    # are read once.  One workspace per direction, so that both projections survive; the fused calls run outside the timing.
    ws_f = [lw.lowra_workspace_init(torch.empty(lw.lowra_workspace_bytes(d["layout"], M, r), dtype=torch.uint8, device="cuda")) for d in dev]
    for d, w in zip(dev, ws_f):
        lw.lowra_lora_forward(d["layout"], d["packed"], d["absmax"], d["maps"], act_dev[(M, d["K"])], d["A"], d["B"], s,
                              Y=d["Y"][M], workspace=w)
        lw.lowra_lora_backward_input(d["layout"], d["packed"], d["absmax"], d["maps"], act_dev[(M, d["N"])], d["A"], d["B"], s,
                                     dX=d["dX"][M] if d["dX"] else None, workspace=d["ws"][M])
    proj = [(lw.lowra_workspace_projection(w, M, r), lw.lowra_workspace_projection(d["ws"][M], M, r)) for d, w in zip(dev, ws_f)]
    ms = timed(lambda: [lw.lowra_lora_backward_adapters_reuse(act_dev[(M, d["K"])], act_dev[(M, d["N"])], T, U, r,
                                                              dA=gA, dB=gB, workspace=ws_ad) for d, (T, U), (gA, gB) in zip(dev, proj, grads)])
    if lw.lowra_device_status(ws_ad) != 0:
        raise SystemExit("device status after the adapter gradients (reusing the projections)")
    extras["adapter_gradients_reusing_projections"] = {
        "ms": ms, "GB/s": ad_bytes / (ms * 1e-3) / 1e9, "frac_hbm": ad_bytes / (ms * 1e-3) / 1e9 / P["hbm"],
        "note": "not part of the step; dA and dB from the s X A and s dY B^T that lowra_lora_forward / lowra_lora_backward_input "
                "left in their workspaces: two products instead of four, X and dY read once"}
    del ws_f, proj

    # per-channel quantisation error (the precision assigner's input) and the residual W - W_hat
    sse = [torch.empty(d["N"], dtype=torch.float64, device="cuda") for d in dev]
    res = torch.empty(max(d["N"] * d["K"] for d in dev), dtype=torch.float32, device="cuda")
    qe = {}
    for key, with_res in (("sse_only", False), ("with_residual", True)):
        ms = timed(lambda: [lw.lowra_quant_error(d["layout"], d["W"], d["maps"], d["thr"], sse=e,
                                                 residual=res[:d["N"] * d["K"]].view(d["N"], d["K"]) if with_res else None)
                            for d, e in zip(dev, sse)])
        by = (8.0 if with_res else 4.0) * elems
        qe[key] = {"ms": ms, "GB/s": by / (ms * 1e-3) / 1e9, "frac_hbm": by / (ms * 1e-3) / 1e9 / P["hbm"]}
    # every channel under 1, 2 and 4 bits in one pass, with the tables learnt above
    out3 = [torch.empty((d["N"], 3), dtype=torch.float64, device="cuda") for d in dev]
    ms = timed(lambda: [lw.lowra_channel_errors(d["W"], m3, h3, sse3=o3) for d, (m3, h3), o3 in zip(dev, tabs3, out3)])
    qe["three_precisions_one_pass"] = {"ms": ms, "GB/s": 4.0 * elems / (ms * 1e-3) / 1e9,
                                       "frac_hbm": 4.0 * elems / (ms * 1e-3) / 1e9 / P["hbm"]}
    qe["note"] = "not part of the step; algorithmic bytes = W read once (4 B per element) + residual written (4 B)"
    extras["quant_error"] = qe
    return extras


# --------------------------------------------------------------------------------------------------
# CPU oracle arm
# --------------------------------------------------------------------------------------------------
SAMPLE_TOKENS = 512


def oracle_sample_step(problem, with_backward=True, keep=None):
    """The oracle on the bounded sample: one matrix of the workload, its own codebooks (the learner is input
    generation and is not timed), encode + decode in full, forward (+ backward-input) on SAMPLE_TOKENS token rows.
    Returns per-phase seconds; `keep` (a dict) receives the results."""
    import oracle
    W, precs, maps, thr, X, dY, A, B, s = problem
    K = W.shape[1]
    t = {}
    t0 = time.time(); packed, a = oracle.encode(W, precs, thr); t["encode"] = time.time() - t0
    t0 = time.time(); what = oracle.decode(packed, a, maps, precs, K); t["decode"] = time.time() - t0
    t0 = time.time(); Y = oracle.lora_forward(what, X, A, B, s); t["forward"] = time.time() - t0
    dX = None
    if with_backward:
        t0 = time.time(); dX = oracle.lora_backward_input(what, dY, A, B, s); t["backward"] = time.time() - t0
    if keep is not None:
        keep.update(packed=packed, absmax=a, what=what, Y=Y, dX=dX)
    return t


def sample_rows(M):
    """SAMPLE_TOKENS token rows spread over the M tokens of the step (every tile of 256 tokens is hit)."""
    return np.unique(np.linspace(0, M - 1, min(SAMPLE_TOKENS, M)).astype(np.int64))


def make_sample_problem(workload):
    import oracle
    cfg, mats = workload_matrices(workload)
    mat = mats[0]
    M = cfg.tokens[0]
    W = si.weights(mat.N, mat.K, matrix_id=mat.matrix_id, kind=cfg.weight_kind)
    precs = si.precisions(mat.N, cfg.mix, matrix_id=mat.matrix_id)
    maps, thr = oracle.lloyd_max(W, precs, T=LLOYD_ITERS)
    rows = sample_rows(M)
    X = si.activations(M, mat.K, matrix_id=100)[rows]
    dY = si.activations(M, mat.N, matrix_id=100)[rows]
    A, B = si.lora_factors(mat.K, mat.N, cfg.rank, matrix_id=mat.matrix_id % 7)
    return (W, precs, maps, thr, X, dY, A, B, cfg.s), mat, cfg, rows


def cpu_baseline_sample(workload, reps: int = 2, gpu=None):
    """Times the oracle, as it stands, on a bounded sample of the workload (its first matrix: encode + decode in
    full, the products on SAMPLE_TOKENS token rows), on all host cores and on one.  With `gpu` (the benchmark's
    device-resident first matrix) the oracle's results of the sample are also held against what the GPU path - its
    own learner, encode, decode and fused products, in the launch configuration that was timed - gives for the same
    matrix and token rows; a mismatch ends the run."""
    import oracle
    problem, mat, cfg, rows = make_sample_problem(workload)
    with_backward = "backward" in cfg.ops
    keep = {}
    oracle_sample_step(problem, with_backward, keep)  # warm; its results serve the check below
    ts = [oracle_sample_step(problem, with_backward) for _ in range(reps)]
    tot = min(sum(t.values()) for t in ts)
    best = min(ts, key=lambda t: sum(t.values()))
    n_rows = len(rows)
    flops = (2 if with_backward else 1) * gemm_flops(n_rows, mat.N, mat.K, cfg.rank)
    el = mat.N * mat.K
    gemm_s = best["forward"] + best.get("backward", 0.0)
    out = {"value": flops / tot / 1e12, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
           "sample": f"{mat.name} {mat.N}x{mat.K}: oracle encode + decode in full, forward" + (" + backward-input" if with_backward else "") +
                     f" on {n_rows} of {cfg.tokens[0]} token rows (fp64); same value definition as the GPU arm",
           "seconds_per_sample_step": tot,
           "encode_ns_per_element": best["encode"] / el * 1e9, "decode_ns_per_element": best["decode"] / el * 1e9,
           "gemm_fp64_gflops": flops / gemm_s / 1e9}
    # one thread: encode + decode on the first 512 rows of the matrix, the forward product on 32 token rows
    n_all = oracle.num_threads()
    oracle.set_threads(1)
    try:
        import threadpoolctl
        limiter = threadpoolctl.threadpool_limits(limits=1)
    except Exception:
        limiter = None
    try:
        W, precs, maps, thr, X, dY, A, B, s = problem
        sub = slice(0, min(512, mat.N))
        t0 = time.time(); pk, am = oracle.encode(W[sub], precs[sub], thr[sub]); t_e = time.time() - t0
        t0 = time.time(); wh = oracle.decode(pk, am, maps[sub], precs[sub], mat.K); t_d = time.time() - t0
        t0 = time.time(); oracle.lora_forward(keep["what"], X[:32], A, B, s); t_f = time.time() - t0
        el1 = W[sub].size
        out["one_thread"] = {"encode_ns_per_element": t_e / el1 * 1e9, "decode_ns_per_element": t_d / el1 * 1e9,
                             "gemm_fp64_gflops": gemm_flops(32, mat.N, mat.K, cfg.rank) / t_f / 1e9,
                             "sample": f"encode + decode of {sub.stop} rows, forward on 32 token rows"}
    finally:
        oracle.set_threads(n_all)
        if limiter is not None:
            limiter.restore_original_limits()

    if gpu is not None:
        lw, torch, d, M = gpu["lw"], gpu["torch"], gpu["d"], gpu["M"]
        bits16 = lambda t: t.view(torch.int16).cpu().numpy().view(np.uint16)
        idx = torch.from_numpy(rows).cuda()
        # the step's own calls, once more, on the step's own buffers (same layout, deal, workspace and token count)
        lw.lowra_encode(d["layout"], d["W"], d["thr"], packed=d["packed"], absmax=d["absmax"])
        lw.lowra_decode(d["layout"], d["packed"], d["absmax"], d["maps"], out=d["What"])
        Y = lw.lowra_lora_forward(d["layout"], d["packed"], d["absmax"], d["maps"], gpu["act"][(M, d["K"])], d["A"], d["B"],
                                  gpu["s"], Y=d["Y"][M], workspace=d["ws"][M])
        got = {"forward": si.bf16_bits_to_f32(bits16(Y[idx])).astype(np.float64)}
        ref = {"forward": keep["Y"]}
        if gpu["with_backward"]:
            dX = lw.lowra_lora_backward_input(d["layout"], d["packed"], d["absmax"], d["maps"], gpu["act"][(M, d["N"])], d["A"], d["B"],
                                              gpu["s"], dX=d["dX"][M], workspace=d["ws"][M])
            got["backward_input"] = si.bf16_bits_to_f32(bits16(dX[idx])).astype(np.float64)
            ref["backward_input"] = keep["dX"]
        if lw.lowra_device_status(d["ws"][M]) != 0:
            raise SystemExit("device status during the check against the oracle")
        chk = {}
        # tables: the GPU learner's levels against the oracle's (equal or one ulp apart); codes and decoded weights:
        # identical wherever the tables are
        maps_gpu = d["maps"].cpu().numpy()
        chk["codebook_entries_identical"] = float((maps_gpu == problem[2]).mean())
        chk["packed_bytes_identical"] = float((d["packed"].cpu().numpy()[:d["layout"].packed_bytes] == keep["packed"]).mean())
        chk["decoded_elements_identical"] = float((bits16(d["What"]) == keep["what"]).mean())
        ok = chk["codebook_entries_identical"] >= 0.99 and chk["packed_bytes_identical"] >= 0.999 and chk["decoded_elements_identical"] >= 0.999
        for k in got:
            dlt = got[k] - ref[k]
            emax = float(np.abs(dlt).max() / np.abs(ref[k]).max())
            efro = float(np.linalg.norm(dlt) / np.linalg.norm(ref[k]))
            chk[k] = {"max_rel": emax, "fro_rel": efro}
            ok = ok and emax <= 1e-2 and efro <= 5e-3
        chk["ok"] = bool(ok)
        chk["what"] = (f"GPU path of the timed configuration (own learner, encode, decode, fused products) against the oracle's own "
                       f"pipeline on {mat.name}, {n_rows} token rows; bounds: max 1e-2, Frobenius 5e-3")
        out["check_against_oracle"] = chk
        if not ok:
            raise SystemExit("the GPU results of the timed configuration disagree with the oracle: " + json.dumps(chk))
    return out


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    problem, mat, cfg, rows = make_sample_problem(args.workload)
    with_backward = "backward" in cfg.ops
    for _ in range(min(args.warmup, 1)):
        oracle_sample_step(problem, with_backward)
    t0 = time.time()
    for _ in range(args.steps):
        oracle_sample_step(problem, with_backward)
    dt = (time.time() - t0) / args.steps
    flops = (2 if with_backward else 1) * gemm_flops(len(rows), mat.N, mat.K, cfg.rank)
    value = flops / dt / 1e12
    sample = (f"each step = the CPU oracle on {mat.name} {mat.N}x{mat.K}: encode + decode in full, forward" +
              (" + backward-input" if with_backward else "") + f" on {len(rows)} of {cfg.tokens[0]} token rows (fp64)")
    out = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT,
           "n_gpus": int(os.environ.get("WORLD_SIZE", "1")), "steps": args.steps, "warmup": min(args.warmup, 1),
           "ms_per_step": dt * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
           "dtype": "f64", "data": "synthetic",
           "config": {"workload": f"config {args.workload}: {cfg.name} (bounded sample: {sample})"},
           "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle", "sample": sample},
           "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(out))


# --------------------------------------------------------------------------------------------------
# small single-kernel cases for profiler captures (a few hundred MB on the device, three launches each)
# --------------------------------------------------------------------------------------------------
CASES = ("forward", "backward", "forward4096", "backward_gate", "forward_4bit", "backward_4bit", "forward_1bit", "backward_1bit",
         "codec", "decode_layer", "learn", "adapters", "adapters_reuse", "errors")


def run_case(case: str) -> None:
    """forward / backward: fused calls, N = K = 4096, 2048 tokens, rank 64 (config-3 mix; *_4bit, *_1bit: every row
    at that precision); forward4096: 4096 tokens (264 pieces: tiles cut between SMs, partial tiles preloaded);
    backward_gate: 11008 x 4096 at 4096 tokens (last row of tiles cut); codec: decode + encode of an 11008 x 4096
    matrix; decode_layer: the seven decodes of a Llama-7B layer back to back; learn: codebook learner, 4096 x 4096,
    10 rounds; adapters: gradients of the low-rank factors, 4096 x 11008, 4096 tokens (adapters_reuse: from given projections); errors: per-channel
    quantisation error with and without the residual, 11008 x 4096."""
    import torch

    import paper_2502_08141_b200 as lw

    cfg = si.config(3)
    r, s = cfg.rank, cfg.s
    gen = torch.Generator(device="cuda").manual_seed(1)
    if case in ("adapters", "adapters_reuse"):
        N, K, M = 11008, 4096, 4096
        X = torch.randn(M, K, device="cuda", generator=gen).bfloat16()
        dY = torch.randn(M, N, device="cuda", generator=gen).bfloat16()
        A = (torch.randn(K, r, device="cuda", generator=gen) * 0.01).bfloat16()
        B = (torch.randn(r, N, device="cuda", generator=gen) * 0.01).bfloat16()
        ws = torch.empty(lw.lowra_adapter_workspace_bytes(M, r), dtype=torch.uint8, device="cuda")
        if case == "adapters_reuse":     # the projections as a forward / backward-input call leaves them: bf16 [M, 64]
            T = (s * (X.float() @ A.float())).bfloat16()
            U = (s * (dY.float() @ B.float().T)).bfloat16()
            for _ in range(3):
                lw.lowra_lora_backward_adapters_reuse(X, dY, T, U, r, workspace=ws)
        else:
            for _ in range(3):
                lw.lowra_lora_backward_adapters(X, dY, A, B, s, workspace=ws)
        status = lw.lowra_device_status(ws)
        print("adapters status", status)
        if status != 0:
            raise SystemExit(1)
        return
    if case == "decode_layer":
        mats = []
        for mat in cfg.matrices:
            precs = si.precisions(mat.N, cfg.mix, matrix_id=mat.matrix_id)
            maps, thr = si.standin_codebooks(precs, matrix_id=mat.matrix_id)
            layout = lw.Layout(precs, mat.K)
            W = torch.randn(mat.N, mat.K, device="cuda", generator=gen) * 0.02
            packed, absmax = lw.lowra_encode(layout, W, torch.from_numpy(thr).cuda())
            mats.append((layout, packed, absmax, torch.from_numpy(maps).cuda(),
                         torch.empty(mat.N, mat.K, dtype=torch.bfloat16, device="cuda")))
            del W
        for _ in range(2):
            for layout, packed, absmax, maps_d, out in mats:
                lw.lowra_decode(layout, packed, absmax, maps_d, out=out)
        torch.cuda.synchronize()
        print("decode_layer ok")
        return
    mix = {4: 1.0} if case.endswith("_4bit") else {1: 1.0} if case.endswith("_1bit") else cfg.mix
    base = case.split("_")[0] if case.endswith("bit") else case
    N, K = (11008, 4096) if base in ("codec", "errors", "backward_gate") else (4096, 4096)
    M = 4096 if base in ("forward4096", "backward_gate") else 2048
    precs = si.precisions(N, mix)
    maps, thr = si.standin_codebooks(precs)
    layout = lw.Layout(precs, K)
    W = torch.randn(N, K, device="cuda", generator=gen) * 0.02
    maps_d, thr_d = torch.from_numpy(maps).cuda(), torch.from_numpy(thr).cuda()
    if base == "learn":
        y0, t0 = si.initial_codebooks()
        for _ in range(3):
            lw.lowra_learn_codebooks(layout, W, y0, t0, LLOYD_ITERS)
        torch.cuda.synchronize()
        print("learn ok")
        return
    if base == "errors":
        sse = torch.empty(N, dtype=torch.float64, device="cuda")
        res = torch.empty(N, K, dtype=torch.float32, device="cuda")
        for _ in range(3):
            lw.lowra_quant_error(layout, W, maps_d, thr_d, sse=sse, residual=res)
            lw.lowra_quant_error(layout, W, maps_d, thr_d, sse=sse)
        torch.cuda.synchronize()
        print("errors ok")
        return
    packed, absmax = lw.lowra_encode(layout, W, thr_d)
    if base == "codec":
        out = torch.empty(N, K, dtype=torch.bfloat16, device="cuda")
        for _ in range(3):
            lw.lowra_decode(layout, packed, absmax, maps_d, out=out)
            lw.lowra_encode(layout, W, thr_d, packed=packed, absmax=absmax)
        torch.cuda.synchronize()
        print("codec ok")
        return
    fwd = base in ("forward", "forward4096")
    act = torch.randn(M, K if fwd else N, device="cuda", generator=gen).bfloat16()
    A = (torch.randn(K, r, device="cuda", generator=gen) * 0.01).bfloat16()
    B = (torch.randn(r, N, device="cuda", generator=gen) * 0.01).bfloat16()
    ws = torch.empty(lw.lowra_workspace_bytes(layout, M, r), dtype=torch.uint8, device="cuda")
    fn = lw.lowra_lora_forward if fwd else lw.lowra_lora_backward_input
    for _ in range(3):
        fn(layout, packed, absmax, maps_d, act, A, B, s, workspace=ws)
    status = lw.lowra_device_status(ws)
    print(case, "status", status)
    if status != 0:
        raise SystemExit(1)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", type=int, default=3, choices=[2, 3, 4, 5])
    ap.add_argument("--case", default=None, choices=CASES, help="run one small single-kernel case (for a profiler) and exit")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu", action="store_true")
    ap.add_argument("--no-extras", action="store_true")
    ap.add_argument("--no-batch", action="store_true", help="a fused call per matrix, also for the q, k and v projections")
    ap.add_argument("--deal-per-call", action="store_true",
                    help="fused calls work out the row deal in a prologue launch of their own (no lowra_deal_build)")
    args = ap.parse_args()
    if args.case is not None:
        run_case(args.case)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_gpu(args)


if __name__ == "__main__":
    main()
