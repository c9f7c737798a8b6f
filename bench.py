#!/usr/bin/env python
"""Benchmark of the LowRA quantized-LoRA hot path on B200.

A *step* is one pass of the whole hot path over one Llama-7B-shaped decoder layer (seven weight
matrices, 4096 tokens, LoRA rank 64, precision mix averaging 1.5 bits): for every matrix
lowra_encode, lowra_decode, lowra_lora_forward and lowra_lora_backward_input, through the C ABI.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]

Prints ONE JSON line.  `value` is the fused dequant+LoRA product throughput of the step (algorithmic
FLOPs of the 7 forward + 7 backward products divided by the time of the WHOLE step, encode and decode
included), measured with CUDA events and inputs resident in HBM; `phases` breaks the step down
(encode / decode in GB/s, forward / backward in TFLOP/s); `e2e` repeats the step with host buffers and
the host<->device copies inside the timed region; `roofline` is for the dominant kernel (the fused
tensor-core kernel); `cpu_baseline` times the CPU oracle on a bounded sample of the same workload.

With N > 1 (torchrun) every rank runs the same layer shapes on its own seeded weights (independent
problems, no data-path collective; weak scaling) and rank 0 reports the aggregate.

`--impl reference` times the CPU oracle alone (there is no reference code for this paper).
"""
from __future__ import annotations

import argparse
import json
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

WORKLOAD = 3  # Llama-7B decoder layer, 4096 tokens, avg 1.5 bits
METRIC = "fused dequant+LoRA fwd+bwd throughput over one Llama-7B layer step (encode+decode+fwd+bwd)"
UNIT = "TFLOP/s"


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
        for ts, line in self.lines:
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 9:
                continue
            try:
                clk, mx = float(parts[1]), float(parts[2])
            except ValueError:
                continue
            if t0 - 0.05 <= ts <= t1 + 0.15:
                sm.append(clk)
                smax.append(mx)
                for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"),
                                     parts[5:9]):
                    if val.lower().startswith("active"):
                        reasons.add(name)
        if not sm:  # region shorter than the sampling period: take everything seen
            for ts, line in self.lines:
                parts = [p.strip() for p in line.split(",")]
                try:
                    sm.append(float(parts[1])); smax.append(float(parts[2]))
                except Exception:
                    pass
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(smax) if smax else None,
                "reasons": sorted(reasons), "samples": len(sm)}


# --------------------------------------------------------------------------------------------------
# workload
# --------------------------------------------------------------------------------------------------
def make_host_inputs(cfg, rank: int):
    """Seeded host inputs of one layer (matrix ids offset by the rank, so ranks hold different layers)."""
    M, r = cfg.tokens[0], cfg.rank

    def one(mat):
        mid = rank_matrix_id(mat.matrix_id, rank)
        W = si.weights(mat.N, mat.K, matrix_id=mid, kind=cfg.weight_kind)
        precs = si.precisions(mat.N, cfg.mix, matrix_id=mid)
        maps, thr = si.standin_codebooks(precs, matrix_id=mid)
        A, B = si.lora_factors(mat.K, mat.N, r, matrix_id=mid)
        return dict(name=mat.name, N=mat.N, K=mat.K, W=W, precs=precs, maps=maps, thr=thr, A=A, B=B)

    with ThreadPoolExecutor(max_workers=min(8, len(cfg.matrices))) as ex:
        mats = list(ex.map(one, cfg.matrices))
    # one activation / gradient buffer per distinct width, shared by the matrices of that width
    acts = {}
    for m in mats:
        if m["K"] not in acts:
            acts[m["K"]] = si.activations(M, m["K"], matrix_id=100 + rank)
        if m["N"] not in acts:
            acts[m["N"]] = si.activations(M, m["N"], matrix_id=100 + rank)
    return mats, acts


# DRAM traffic of one fused_kernel launch measured with ncu (dram__bytes_read.sum + dram__bytes_write.sum) on a
# launch of this very workload: the backward-input pass of gate_proj (dX [4096, 4096] from dY [4096, 11008];
# profiles/fused_backward_input_11008x4096_m4096_streamk.md): 167.9 MB read + 29.7 MB written.  The bytes the call
# has to read and write once are 137 MB (the output is partly still in L2 when the kernel ends; the stream-K partial
# tiles add 19 MB each way).  Scaled to the step's average launch in proportion to those input + output bytes.
NCU_CASE = dict(N=4096, K=11008, M=4096, r=64, bits=1.5, dram_bytes=167.9e6 + 29.7e6)


def fused_io_bytes(N, K, M, r, bits):
    """Bytes a fused call has to read and write once: activations, packed codes, absmax, tables, factors; output."""
    return 2.0 * M * K + N * K * (bits / 8 + 4 / 64) + 64.0 * N + 2.0 * (K + N) * r + 2.0 * M * N


def fused_traffic_per_launch(dev, M, r, bits):
    case = fused_io_bytes(NCU_CASE["N"], NCU_CASE["K"], NCU_CASE["M"], NCU_CASE["r"], NCU_CASE["bits"])
    per = [fused_io_bytes(d["m"]["N"], d["m"]["K"], M, r, bits) for d in dev] + \
          [fused_io_bytes(d["m"]["K"], d["m"]["N"], M, r, bits) for d in dev]   # backward reads dY [M, N], writes dX [M, K]
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
    """Whole-job throughput: every rank does one layer step per step (weak scaling)."""
    return world * flops_per_rank_step / (ms_per_step * 1e-3) / 1e12


def rank_matrix_id(matrix_id: int, rank: int, per_layer: int = 7) -> int:
    """Ranks hold different layers: the seed stream of matrix j on rank q is that of matrix j + 7 q."""
    return matrix_id + per_layer * rank


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

    cfg = si.config(WORKLOAD)
    M, r, s = cfg.tokens[0], cfg.rank, cfg.s
    bits = si.avg_bits(cfg.mix)
    mats, acts = make_host_inputs(cfg, rank)

    pin = lambda a: torch.from_numpy(np.ascontiguousarray(a)).pin_memory()
    bfv = lambda t: t.view(torch.bfloat16)
    # ---- device-resident problem
    dev = []
    for m in mats:
        # the deal of the rows to the dequant warps depends on the precisions only: built once per weight, like the
        # storage plan, unless --deal-per-call asks for the prologue launch in every call
        layout = lw.Layout(m["precs"], m["K"])
        if not args.deal_per_call:
            layout.build_deal()
        d = dict(m=m, layout=layout,
                 W=torch.from_numpy(m["W"]).cuda(), thr=torch.from_numpy(m["thr"]).cuda(),
                 maps=torch.from_numpy(m["maps"]).cuda(),
                 A=bfv(torch.from_numpy(m["A"].view(np.int16)).cuda()), B=bfv(torch.from_numpy(m["B"].view(np.int16)).cuda()),
                 packed=torch.empty(max(layout.packed_bytes, 16), dtype=torch.uint8, device="cuda"),
                 absmax=torch.empty((m["N"], m["K"] // 64), dtype=torch.float32, device="cuda"),
                 What=torch.empty((m["N"], m["K"]), dtype=torch.bfloat16, device="cuda"),
                 Y=torch.empty((M, m["N"]), dtype=torch.bfloat16, device="cuda"),
                 dX=torch.empty((M, m["K"]), dtype=torch.bfloat16, device="cuda"),
                 ws=lw.lowra_workspace_init(torch.empty(lw.lowra_workspace_bytes(layout, M, r), dtype=torch.uint8, device="cuda")))
        dev.append(d)
    act_dev = {k: bfv(torch.from_numpy(v.view(np.int16)).cuda()) for k, v in acts.items()}
    stream = torch.cuda.current_stream()

    def step(record=None, per_call=None):
        """One pass.  `record` (a list) receives (phase, event_start, event_end) per phase: the calls of a phase
        run back to back, as a user would issue them; `per_call` receives the same per call (diagnostic pass)."""
        def phase(name, fn):
            if record is not None:
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(stream)
            for d in dev:
                if per_call is not None:
                    c0, c1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    c0.record(stream); fn(d); c1.record(stream)
                    per_call.append((name, c0, c1))
                else:
                    fn(d)
            if record is not None:
                e1.record(stream)
                record.append((name, e0, e1))
        phase("encode", lambda d: lw.lowra_encode(d["layout"], d["W"], d["thr"], packed=d["packed"], absmax=d["absmax"]))
        phase("decode", lambda d: lw.lowra_decode(d["layout"], d["packed"], d["absmax"], d["maps"], out=d["What"]))
        phase("forward", lambda d: lw.lowra_lora_forward(d["layout"], d["packed"], d["absmax"], d["maps"],
                                                         act_dev[d["m"]["K"]], d["A"], d["B"], s, Y=d["Y"], workspace=d["ws"]))
        phase("backward", lambda d: lw.lowra_lora_backward_input(d["layout"], d["packed"], d["absmax"], d["maps"],
                                                                 act_dev[d["m"]["N"]], d["A"], d["B"], s, dX=d["dX"],
                                                                 workspace=d["ws"]))

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    for _ in range(max(args.warmup, 3)):
        step()
    for d in dev:
        st = lw.lowra_device_status(d["ws"])
        if st != 0:
            raise SystemExit(f"device status {st} after warm-up")

    # ---- timed region: exactly K steps, device timing with CUDA events, max over ranks
    sampler = ClockSampler(local_rank)
    sampler.start()
    time.sleep(0.25)
    barrier()
    records = []
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0 = time.time()
    ev0.record(stream)
    for _ in range(args.steps):
        step(records)
    ev1.record(stream)
    barrier()
    t1 = time.time()
    clocks = sampler.stop(t0, t1)
    total_ms = ev0.elapsed_time(ev1)
    total_ms = max_over_ranks(total_ms, world)
    ms_per_step = total_ms / args.steps

    flops_step = sum(2 * gemm_flops(M, d["m"]["N"], d["m"]["K"], r) for d in dev)
    value = aggregate_tflops(flops_step, world, ms_per_step)

    phase_ms, call_ms = {}, {}
    for phase, e0, e1 in records:
        phase_ms[phase] = phase_ms.get(phase, 0.0) + e0.elapsed_time(e1)
    for k in phase_ms:
        phase_ms[k] /= args.steps
    # diagnostic pass outside the timed region: the same step with events around every call
    n_diag = 3
    calls = []
    for _ in range(n_diag):
        step(per_call=calls)
    torch.cuda.synchronize()
    for idx, (phase, c0, c1) in enumerate(calls):
        per = call_ms.setdefault(phase, [0.0] * len(dev))
        per[idx % len(dev)] += c0.elapsed_time(c1) / n_diag      # the calls of a phase run in the order of the matrices
    elems = sum(d["m"]["N"] * d["m"]["K"] for d in dev)
    P = peaks()
    dec_gbs = sum(decode_bytes(d["m"]["N"], d["m"]["K"], bits) for d in dev) / (phase_ms["decode"] * 1e-3) / 1e9
    enc_gbs = sum(encode_bytes(d["m"]["N"], d["m"]["K"], bits) for d in dev) / (phase_ms["encode"] * 1e-3) / 1e9
    fwd_tf = flops_step / 2 / (phase_ms["forward"] * 1e-3) / 1e12
    bwd_tf = flops_step / 2 / (phase_ms["backward"] * 1e-3) / 1e12
    phases = {
        "encode": {"ms": phase_ms["encode"], "GB/s": enc_gbs, "frac_hbm": enc_gbs / P["hbm"], "frac_hbm_nominal_8TBs": enc_gbs / 8000.0},
        "decode": {"ms": phase_ms["decode"], "GB/s": dec_gbs, "frac_hbm": dec_gbs / P["hbm"], "frac_hbm_nominal_8TBs": dec_gbs / 8000.0},
        "forward": {"ms": phase_ms["forward"], "TFLOP/s": fwd_tf, "frac_tensor_burst": fwd_tf / P["tensor_burst"],
                    "frac_tensor_sustained": fwd_tf / P["tensor_sustained"], "frac_tensor_nominal_2250": fwd_tf / 2250.0},
        "backward_input": {"ms": phase_ms["backward"], "TFLOP/s": bwd_tf, "frac_tensor_burst": bwd_tf / P["tensor_burst"],
                           "frac_tensor_sustained": bwd_tf / P["tensor_sustained"], "frac_tensor_nominal_2250": bwd_tf / 2250.0},
    }
    names = [d["m"].get("name", f'{d["m"]["N"]}x{d["m"]["K"]}') for d in dev]
    for key, phase in (("forward", "forward"), ("backward_input", "backward")):
        phases[key]["TFLOP/s_per_matrix (separate pass, events around every call)"] = {
            f"{i}:{n}": round(gemm_flops(M, d["m"]["N"], d["m"]["K"], r) / (ms * 1e-3) / 1e12, 1)
            for i, (n, d, ms) in enumerate(zip(names, dev, call_ms[phase]))}

    # dominant kernel: the fused tensor-core kernel (forward + backward launches), timed as whole calls
    fused_ms = phase_ms["forward"] + phase_ms["backward"]
    achieved = flops_step / (fused_ms * 1e-3) / 1e12
    # denominator: the cuBLAS bf16 figure of the clock regime this run was in - the burst figure while the SM clock
    # stayed at its maximum (a timed region of tens of milliseconds), the sustained one when the power cap held it
    # below (hundreds of steps); both fractions are reported either way
    sm_now, sm_max = clocks.get("sm_mhz"), clocks.get("sm_max_mhz")
    capped = bool(sm_now and sm_max and sm_now < 0.95 * sm_max)
    peak = P["tensor_sustained"] if capped else P["tensor_burst"]
    roofline = {"bound": "tensor", "kernel": "fused_kernel (forward + backward-input calls" + (", prologue launch included)" if args.deal_per_call else ")"),
                "achieved": achieved, "peak": peak, "unit": "TFLOP/s", "frac": achieved / peak,
                "peak_burst": P["tensor_burst"], "frac_burst": achieved / P["tensor_burst"],
                "peak_sustained": P["tensor_sustained"], "frac_sustained": achieved / P["tensor_sustained"],
                "peak_source": P["source"] + (" (sustained figure: the SM clock was held below its maximum during the timed region)"
                                              if capped else " (burst figure: the SM clock stayed at its maximum during the timed region)"),
                "traffic": fused_traffic_per_launch(dev, M, r, bits),
                "traffic_source": "ncu dram__bytes_read.sum + dram__bytes_write.sum of the gate_proj backward-input launch of "
                                  "this workload (profiles/fused_backward_input_11008x4096_m4096_streamk.md), scaled by the "
                                  "input + output bytes of the step's average launch"}

    # ---- end to end: host buffers, pinned, copies inside the timed region
    e2e = None
    if not args.no_e2e:
        host = []
        for m in mats:
            host.append(dict(W=pin(m["W"]), thr=pin(m["thr"]), maps=pin(m["maps"]), A=pin(m["A"].view(np.int16)),
                             B=pin(m["B"].view(np.int16)),
                             Y=torch.empty((M, m["N"]), dtype=torch.bfloat16).pin_memory(),
                             dX=torch.empty((M, m["K"]), dtype=torch.bfloat16).pin_memory()))
        act_host = {k: pin(v.view(np.int16)) for k, v in acts.items()}
        h2d = sum(h[k].numel() * h[k].element_size() for h in host for k in ("W", "thr", "maps", "A", "B")) \
            + sum(2 * act_host[d["m"]["K"]].numel() + 2 * act_host[d["m"]["N"]].numel() for d in dev)
        d2h = sum(h[k].numel() * h[k].element_size() for h in host for k in ("Y", "dX"))

        # Three streams: uploads, kernels, downloads.  Matrix i + 1 is uploaded while matrix i is computed and
        # matrix i - 1 is downloaded (the copies of one step are PCIe-bound: 2.1 GB); every buffer has its own
        # events, so a buffer is never overwritten before its last reader is done, across steps too.
        s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()
        xs = [torch.empty_like(act_dev[d["m"]["K"]]) for d in dev]      # per-matrix activations / output gradients
        gs = [torch.empty_like(act_dev[d["m"]["N"]]) for d in dev]
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
                    xs[i].view(torch.int16).copy_(act_host[d["m"]["K"]], non_blocking=True)
                    gs[i].view(torch.int16).copy_(act_host[d["m"]["N"]], non_blocking=True)
                    ev_in[i].record(s_in)
                stream.wait_event(ev_in[i])
                if ev_out[i] is not None:
                    stream.wait_event(ev_out[i])                         # the previous step's results have left
                lw.lowra_encode(d["layout"], d["W"], d["thr"], packed=d["packed"], absmax=d["absmax"])
                lw.lowra_decode(d["layout"], d["packed"], d["absmax"], d["maps"], out=d["What"])
                lw.lowra_lora_forward(d["layout"], d["packed"], d["absmax"], d["maps"], xs[i], d["A"], d["B"], s, Y=d["Y"], workspace=d["ws"])
                lw.lowra_lora_backward_input(d["layout"], d["packed"], d["absmax"], d["maps"], gs[i], d["A"], d["B"], s, dX=d["dX"], workspace=d["ws"])
                ev_done[i] = torch.cuda.Event(); ev_done[i].record(stream)
                with torch.cuda.stream(s_out):
                    s_out.wait_event(ev_done[i])
                    h["Y"].copy_(d["Y"], non_blocking=True); h["dX"].copy_(d["dX"], non_blocking=True)
                    ev_out[i] = torch.cuda.Event(); ev_out[i].record(s_out)

        def e2e_join():   # the step is over when its last download is
            for e in ev_out:
                if e is not None:
                    stream.wait_event(e)

        e2e_step()
        e2e_join()
        barrier()
        n_e2e = max(1, min(args.steps, 3))
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        for _ in range(n_e2e):
            e2e_step()
        e2e_join()
        b.record(stream)
        barrier()
        for d in dev:
            if lw.lowra_device_status(d["ws"]) != 0:
                raise SystemExit("device status after the end-to-end steps")
        ms = a.elapsed_time(b) / n_e2e
        ms = max_over_ranks(ms, world)
        e2e = {"value": aggregate_tflops(flops_step, world, ms), "unit": UNIT, "ms_per_step": ms,
               "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h), "steps": n_e2e,
               "note": "uploads, kernels and downloads on three streams: a matrix is computed while the next one "
                       "arrives and the previous one leaves"}

    # ---- outside the step: the codebook learner (the stage before encode), timed on the layer's seven matrices
    extras = None
    if rank == 0:
        y0 = np.zeros((3, 16)); t0 = np.zeros((3, 16))        # stand-in starting tables: equally spaced levels
        for c, b in enumerate((1, 2, 4)):
            lv = np.linspace(-1.0, 1.0, 1 << b)
            y0[c, :lv.size] = lv
            t0[c, :lv.size - 1] = 0.5 * (lv[:-1] + lv[1:])
        T_learn = 10
        torch.cuda.synchronize()
        for d in dev:   # warm-up
            lw.lowra_learn_codebooks(d["layout"], d["W"], y0, t0, T_learn, maps=d["maps"], thresholds=d["thr"])
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        for d in dev:
            lw.lowra_learn_codebooks(d["layout"], d["W"], y0, t0, T_learn, maps=d["maps"], thresholds=d["thr"])
        b.record(stream)
        torch.cuda.synchronize()
        ms_learn = a.elapsed_time(b)
        extras = {"learn_codebooks": {"ms": ms_learn, "iterations": T_learn, "GB/s": 4.0 * elems / (ms_learn * 1e-3) / 1e9,
                                      "frac_hbm": 4.0 * elems / (ms_learn * 1e-3) / 1e9 / P["hbm"],
                                      "element_passes_per_s": elems * T_learn / (ms_learn * 1e-3),
                                      "note": "not part of the step; algorithmic bytes = one read of W (4 B per element)"}}
        # the same for all three precisions of every row in one pass (what the precision assigner starts from)
        tabs3 = [(torch.empty((3, d["m"]["N"], 16), dtype=torch.float32, device="cuda"),
                  torch.empty((3, d["m"]["N"], 16), dtype=torch.float32, device="cuda")) for d in dev]
        for d, (m3, h3) in zip(dev, tabs3):
            lw.lowra_learn_codebooks_all(d["W"], y0, t0, T_learn, maps3=m3, thresholds3=h3)
        a.record(stream)
        for d, (m3, h3) in zip(dev, tabs3):
            lw.lowra_learn_codebooks_all(d["W"], y0, t0, T_learn, maps3=m3, thresholds3=h3)
        b.record(stream)
        torch.cuda.synchronize()
        ms_learn3 = a.elapsed_time(b)
        extras["learn_codebooks_all_precisions"] = {
            "ms": ms_learn3, "iterations": T_learn, "element_passes_per_s": 3 * elems * T_learn / (ms_learn3 * 1e-3),
            "note": "not part of the step; every row at 1, 2 and 4 bits from one read of W"}
        del tabs3

        # the gradients of the low-rank factors (the other half of a training step's backward pass)
        ws_ad = torch.empty(lw.lowra_adapter_workspace_bytes(M, r), dtype=torch.uint8, device="cuda")
        grads = [(torch.empty_like(d["A"]), torch.empty_like(d["B"])) for d in dev]

        def adapters():
            for d, (gA, gB) in zip(dev, grads):
                lw.lowra_lora_backward_adapters(act_dev[d["m"]["K"]], act_dev[d["m"]["N"]], d["A"], d["B"], s,
                                                dA=gA, dB=gB, workspace=ws_ad)
        adapters()
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        adapters()
        b.record(stream)
        torch.cuda.synchronize()
        if lw.lowra_device_status(ws_ad) != 0:
            raise SystemExit("device status after the adapter gradients")
        ms_ad = a.elapsed_time(b)
        ad_bytes = sum(2.0 * M * (d["m"]["K"] + d["m"]["N"]) for d in dev)      # X and dY once, bf16
        ad_flops = sum(4.0 * M * r * (d["m"]["K"] + d["m"]["N"]) for d in dev)
        extras["adapter_gradients"] = {"ms": ms_ad, "GB/s": ad_bytes / (ms_ad * 1e-3) / 1e9,
                                       "frac_hbm": ad_bytes / (ms_ad * 1e-3) / 1e9 / P["hbm"],
                                       "TFLOP/s": ad_flops / (ms_ad * 1e-3) / 1e12, "launches": 5 * len(dev),
                                       "note": "not part of the step; algorithmic bytes = X and dY read once"}

        # per-channel quantisation error (the precision assigner's input) and the residual W - W_hat
        sse = [torch.empty(d["m"]["N"], dtype=torch.float64, device="cuda") for d in dev]
        res = torch.empty(max(d["m"]["N"] * d["m"]["K"] for d in dev), dtype=torch.float32, device="cuda")
        qe = {}
        for key, with_res in (("sse_only", False), ("with_residual", True)):
            def errors():
                for d, e in zip(dev, sse):
                    lw.lowra_quant_error(d["layout"], d["W"], d["maps"], d["thr"], sse=e,
                                         residual=res[:d["m"]["N"] * d["m"]["K"]].view(d["m"]["N"], d["m"]["K"]) if with_res else None)
            errors()
            torch.cuda.synchronize()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            errors()
            b.record(stream)
            torch.cuda.synchronize()
            ms_q = a.elapsed_time(b)
            by = (8.0 if with_res else 4.0) * elems
            qe[key] = {"ms": ms_q, "GB/s": by / (ms_q * 1e-3) / 1e9, "frac_hbm": by / (ms_q * 1e-3) / 1e9 / P["hbm"]}
        # every channel under 1, 2 and 4 bits in one pass (stand-in tables for all three precisions)
        t3 = []
        for d in dev:
            m3 = np.zeros((3, d["m"]["N"], 16), dtype=np.float32); h3 = np.zeros_like(m3)
            for c, b in enumerate((1, 2, 4)):
                m3[c], h3[c] = si.standin_codebooks(np.full(d["m"]["N"], b, dtype=np.uint8))
            t3.append((torch.from_numpy(m3).cuda(), torch.from_numpy(h3).cuda(),
                       torch.empty((d["m"]["N"], 3), dtype=torch.float64, device="cuda")))

        def errors3():
            for d, (m3, h3, o3) in zip(dev, t3):
                lw.lowra_channel_errors(d["W"], m3, h3, sse3=o3)
        errors3()
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        errors3()
        b.record(stream)
        torch.cuda.synchronize()
        ms_q = a.elapsed_time(b)
        qe["three_precisions_one_pass"] = {"ms": ms_q, "GB/s": 4.0 * elems / (ms_q * 1e-3) / 1e9,
                                           "frac_hbm": 4.0 * elems / (ms_q * 1e-3) / 1e9 / P["hbm"]}
        qe["note"] = "not part of the step; algorithmic bytes = W read once (4 B per element) + residual written (4 B)"
        extras["quant_error"] = qe

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu:
        cpu = cpu_baseline_sample()

    if rank == 0:
        out = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": f"config {WORKLOAD}: {cfg.name}, 7 matrices, {M} tokens, rank {r}, "
                                   f"mix {cfg.mix} (avg {bits:.2f} bits), stand-in codebooks",
                       "elements": elems, "l2": "inputs larger than L2 (about 2.7 GB touched per step)",
                       "row_deal": "in every call (prologue launch)" if args.deal_per_call else
                                   "once per weight (lowra_deal_build), outside the step like the storage plan"},
            "phases": phases, "roofline": roofline, "e2e": e2e, "cpu_baseline": cpu, "extras": extras,
            "gpu_launches": args.steps * len(dev) * (6 if args.deal_per_call else 4), "clocks": clocks,
        }
        print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


# --------------------------------------------------------------------------------------------------
# CPU oracle arm
# --------------------------------------------------------------------------------------------------
SAMPLE_TOKENS = 512


def oracle_sample_step(problem):
    """The oracle on the bounded sample: q_proj-shaped matrix, encode + decode in full, forward +
    backward-input on SAMPLE_TOKENS token rows.  Returns per-phase seconds."""
    import oracle
    W, precs, maps, thr, X, dY, A, B, s = problem
    K = W.shape[1]
    t = {}
    t0 = time.time(); packed, a = oracle.encode(W, precs, thr); t["encode"] = time.time() - t0
    t0 = time.time(); what = oracle.decode(packed, a, maps, precs, K); t["decode"] = time.time() - t0
    t0 = time.time(); oracle.lora_forward(what, X, A, B, s); t["forward"] = time.time() - t0
    t0 = time.time(); oracle.lora_backward_input(what, dY, A, B, s); t["backward"] = time.time() - t0
    return t


def make_sample_problem():
    cfg = si.config(WORKLOAD)
    mat = cfg.matrices[0]
    W = si.weights(mat.N, mat.K, matrix_id=mat.matrix_id)
    precs = si.precisions(mat.N, cfg.mix, matrix_id=mat.matrix_id)
    maps, thr = si.standin_codebooks(precs, matrix_id=mat.matrix_id)
    X = si.activations(SAMPLE_TOKENS, mat.K, matrix_id=100)
    dY = si.activations(SAMPLE_TOKENS, mat.N, matrix_id=101)
    A, B = si.lora_factors(mat.K, mat.N, cfg.rank, matrix_id=mat.matrix_id)
    return (W, precs, maps, thr, X, dY, A, B, cfg.s), mat, cfg


def cpu_baseline_sample(reps: int = 3):
    import oracle
    problem, mat, cfg = make_sample_problem()
    oracle_sample_step(problem)  # warm
    ts = [oracle_sample_step(problem) for _ in range(reps)]
    tot = min(sum(t.values()) for t in ts)
    best = min(ts, key=lambda t: sum(t.values()))
    flops = 2 * gemm_flops(SAMPLE_TOKENS, mat.N, mat.K, cfg.rank)
    el = mat.N * mat.K
    return {"value": flops / tot / 1e12, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
            "sample": f"{mat.name} {mat.N}x{mat.K}: oracle encode + decode in full, forward + backward-input on "
                      f"{SAMPLE_TOKENS} of {cfg.tokens[0]} token rows (fp64); same value definition as the GPU arm",
            "seconds_per_sample_step": tot,
            "encode_ns_per_element": best["encode"] / el * 1e9, "decode_ns_per_element": best["decode"] / el * 1e9,
            "gemm_fp64_gflops": flops / (best["forward"] + best["backward"]) / 1e9}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    problem, mat, cfg = make_sample_problem()
    for _ in range(min(args.warmup, 1)):
        oracle_sample_step(problem)
    t0 = time.time()
    for _ in range(args.steps):
        oracle_sample_step(problem)
    dt = (time.time() - t0) / args.steps
    flops = 2 * gemm_flops(SAMPLE_TOKENS, mat.N, mat.K, cfg.rank)
    value = flops / dt / 1e12
    sample = (f"each step = the CPU oracle on {mat.name} {mat.N}x{mat.K}: encode + decode in full, forward + "
              f"backward-input on {SAMPLE_TOKENS} of {cfg.tokens[0]} token rows (fp64)")
    out = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT,
           "n_gpus": int(os.environ.get("WORLD_SIZE", "1")), "steps": args.steps, "warmup": min(args.warmup, 1),
           "ms_per_step": dt * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
           "dtype": "f64", "data": "synthetic",
           "config": {"workload": f"config {WORKLOAD}: {cfg.name} (bounded sample: {sample})"},
           "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle", "sample": sample},
           "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(out))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu", action="store_true")
    ap.add_argument("--deal-per-call", action="store_true",
                    help="fused calls work out the row deal in a prologue launch of their own (no lowra_deal_build)")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_gpu(args)


if __name__ == "__main__":
    main()
