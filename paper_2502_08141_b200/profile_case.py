"""Small, self-contained launches of one kernel family, sized for an `ncu --set full` capture.

    python -m paper_2502_08141_b200.profile_case forward     # fused forward,  N = K = 4096, 2048 tokens, rank 64
    python -m paper_2502_08141_b200.profile_case backward    # fused backward-input, same shapes
    python -m paper_2502_08141_b200.profile_case forward4096 # fused forward at 4096 tokens (264 pieces: stream-K, preloaded partial tiles)
    python -m paper_2502_08141_b200.profile_case backward_gate # fused backward-input, 11008 x 4096, 4096 tokens (stream-K on the last row)
    python -m paper_2502_08141_b200.profile_case codec       # decode + encode of an 11008 x 4096 matrix
    python -m paper_2502_08141_b200.profile_case learn       # codebook learner, 4096 x 4096, 10 iterations
    python -m paper_2502_08141_b200.profile_case adapters    # gradients of the low-rank factors, 4096 x 11008, 4096 tokens
    python -m paper_2502_08141_b200.profile_case errors      # per-channel quantisation error + residual, 11008 x 4096

Each case runs its call three times on seeded synthetic inputs (config-3 precision mix) and checks the
device status word; a few hundred MB on the device at most.
"""
from __future__ import annotations

import sys

import torch

import synth_inputs as si

from . import (Layout, lowra_adapter_workspace_bytes, lowra_decode, lowra_device_status, lowra_encode, lowra_learn_codebooks,
               lowra_lora_backward_adapters, lowra_lora_backward_input, lowra_lora_forward, lowra_quant_error,
               lowra_workspace_bytes)


def adapters() -> None:
    cfg = si.config(3)
    N, K, M, r = 11008, 4096, 4096, cfg.rank
    gen = torch.Generator(device="cuda").manual_seed(1)
    X = torch.randn(M, K, device="cuda", generator=gen).bfloat16()
    dY = torch.randn(M, N, device="cuda", generator=gen).bfloat16()
    A = (torch.randn(K, r, device="cuda", generator=gen) * 0.01).bfloat16()
    B = (torch.randn(r, N, device="cuda", generator=gen) * 0.01).bfloat16()
    ws = torch.empty(lowra_adapter_workspace_bytes(M, r), dtype=torch.uint8, device="cuda")
    for _ in range(3):
        lowra_lora_backward_adapters(X, dY, A, B, cfg.s, workspace=ws)
    status = lowra_device_status(ws)
    print("adapters status", status)
    if status != 0:
        raise SystemExit(1)


def main(case: str) -> None:
    if case == "adapters":
        adapters()
        return
    cfg = si.config(3)
    N, K = (11008, 4096) if case in ("codec", "errors", "backward_gate") else (4096, 4096)
    M, r, s = (4096 if case in ("forward4096", "backward_gate") else 2048), cfg.rank, cfg.s
    precs = si.precisions(N, cfg.mix)
    maps, thr = si.standin_codebooks(precs)
    layout = Layout(precs, K)
    gen = torch.Generator(device="cuda").manual_seed(1)
    W = torch.randn(N, K, device="cuda", generator=gen) * 0.02
    maps_d, thr_d = torch.from_numpy(maps).cuda(), torch.from_numpy(thr).cuda()
    if case == "learn":
        import numpy as np
        y0 = np.zeros((3, 16)); t0 = np.zeros((3, 16))   # equally spaced starting levels
        for c, b in enumerate((1, 2, 4)):
            lv = np.linspace(-1.0, 1.0, 1 << b)
            y0[c, :lv.size] = lv
            t0[c, :lv.size - 1] = 0.5 * (lv[:-1] + lv[1:])
        for _ in range(3):
            lowra_learn_codebooks(layout, W, y0, t0, 10)
        torch.cuda.synchronize()
        print("learn ok")
        return
    if case == "errors":
        sse = torch.empty(N, dtype=torch.float64, device="cuda")
        res = torch.empty(N, K, dtype=torch.float32, device="cuda")
        for _ in range(3):
            lowra_quant_error(layout, W, maps_d, thr_d, sse=sse, residual=res)
            lowra_quant_error(layout, W, maps_d, thr_d, sse=sse)
        torch.cuda.synchronize()
        print("errors ok")
        return
    packed, absmax = lowra_encode(layout, W, thr_d)
    if case == "codec":
        out = torch.empty(N, K, dtype=torch.bfloat16, device="cuda")
        for _ in range(3):
            lowra_decode(layout, packed, absmax, maps_d, out=out)
            lowra_encode(layout, W, thr_d, packed=packed, absmax=absmax)
        torch.cuda.synchronize()
        print("codec ok")
        return
    act_cols = K if case in ("forward", "forward4096") else N
    act = torch.randn(M, act_cols, device="cuda", generator=gen).bfloat16()
    A = (torch.randn(K, r, device="cuda", generator=gen) * 0.01).bfloat16()
    B = (torch.randn(r, N, device="cuda", generator=gen) * 0.01).bfloat16()
    ws = torch.empty(lowra_workspace_bytes(layout, M, r), dtype=torch.uint8, device="cuda")
    fn = lowra_lora_forward if case in ("forward", "forward4096") else lowra_lora_backward_input
    for _ in range(3):
        fn(layout, packed, absmax, maps_d, act, A, B, s, workspace=ws)
    status = lowra_device_status(ws)
    print(case, "status", status)
    if status != 0:
        raise SystemExit(1)


if __name__ == "__main__":
    main(sys.argv[1] if len(sys.argv) > 1 else "forward")
