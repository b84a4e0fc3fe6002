#!/usr/bin/env python
"""Times gq_cd_cycles (cyclic coordinate descent with fixed codebooks, Algorithm 4) and, optionally, the LNQ loop
(Algorithm 2: gq_codebook_update + gq_cd_cycles) on a synthetic layer.

    python bench_lnq.py [--d-in 4096] [--d-out 4096] [--g 4] [--levels 16] [--cycles 2]
                        [--tokens 8192] [--lnq-rounds 0]

The layer's guided Hessians come from the library's own path (gq_saliency, gq_hessian_accumulate,
gq_hessian_finalize on seeded synthetic activations and gradients), the codebooks are per-channel grids
between the smallest and largest weight, and the starting point is nearest-level rounding.  Prints one JSON
line: milliseconds per cycle, per-kernel device time, and the objective before and after (gq_objective).
"""
from __future__ import annotations

import argparse
import json
import os
import sys

import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2505_07004_b200 import api as libgq, synth


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--d-in", type=int, default=4096)
    ap.add_argument("--d-out", type=int, default=4096)
    ap.add_argument("--g", type=int, default=4)
    ap.add_argument("--levels", type=int, default=16)
    ap.add_argument("--cycles", type=int, default=2)
    ap.add_argument("--tokens", type=int, default=8192)
    ap.add_argument("--lnq-rounds", type=int, default=0,
                    help="also time Algorithm 2: this many rounds of (codebook step, --cycles CD cycles) + a final codebook step")
    args = ap.parse_args()
    if not torch.cuda.is_available():
        raise RuntimeError("bench_lnq.py needs a CUDA device: libgq has no CPU path")
    dev = torch.device("cuda:0")
    torch.cuda.set_device(dev)
    cfg = synth.LayerConfig("cd", args.tokens, min(args.tokens, 8192), args.d_in, args.d_out, (args.g,), "lognormal",
                            0.01, 20.0)
    syn = synth.LayerSynth(cfg, dev, seed=0)
    g = args.g
    H = torch.zeros((g, cfg.d_in, cfg.d_in), dtype=torch.float32, device=dev)
    hws = libgq.alloc_workspace(libgq.gq_hessian_workspace_bytes(cfg.chunk, cfg.d_in, g), dev)
    for c in range(cfg.n_chunks):
        s = libgq.gq_saliency(syn.grad_chunk(c), g, 1e3)
        libgq.gq_hessian_accumulate(syn.x_chunk(c), s, H, hws)
    libgq.gq_hessian_finalize(H)
    W, _ = syn.weights()
    lo, hi = W.min(1, keepdim=True).values, W.max(1, keepdim=True).values
    m = args.levels
    cb = (lo + (hi - lo) * (torch.arange(m, device=dev)[None, :] + 0.5) / m).contiguous()
    W0 = torch.gather(cb, 1, (W[:, :, None] - cb[:, None, :]).abs().argmin(-1)).contiguous()
    ws = libgq.alloc_workspace(libgq.gq_cd_workspace_bytes(cfg.d_in, cfg.d_out, g), dev)
    ows = libgq.alloc_workspace(libgq.gq_objective_workspace_bytes(cfg.d_in, cfg.d_out, g), dev)
    f0 = float(libgq.gq_objective(W, W0, H, ows).cpu()[-1])
    Wh = W0.clone()
    libgq.gq_cd_cycles(W, Wh, cb, H, 1, ws)          # warm-up
    libgq.gq_check()
    Wh = W0.clone()
    libgq.gq_kernel_timing_enable(True)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    libgq.gq_cd_cycles(W, Wh, cb, H, args.cycles, ws)
    e1.record()
    e1.synchronize()
    kern = libgq.gq_kernel_timing_read()
    libgq.gq_kernel_timing_enable(False)
    libgq.gq_check()
    f1 = float(libgq.gq_objective(W, Wh, H, ows).cpu()[-1])
    ms = e0.elapsed_time(e1)
    out = {
        "op": "gq_cd_cycles", "d_in": cfg.d_in, "d_out": cfg.d_out, "g": g, "levels": m, "cycles": args.cycles,
        "ms_total": ms, "ms_per_cycle": ms / max(1, args.cycles),
        "tflops_2_din2_dout_per_cycle": 2.0 * cfg.d_in ** 2 * cfg.d_out * args.cycles / (ms * 1e-3) / 1e12,
        "kernels_ms": {k: {"ms": round(v[0], 4), "launches": v[1]} for k, v in kern.items() if v[1]},
        "objective_start": f0, "objective_end": f1,
    }
    if args.lnq_rounds > 0:
        cbw = libgq.alloc_workspace(libgq.gq_codebook_workspace_bytes(cfg.d_in, cfg.d_out, g, m), dev)
        Q = (W[:, :, None] - cb[:, None, :]).abs().argmin(-1).to(torch.uint8).contiguous()
        Wh = W0.clone()
        cbl, _ = libgq.gq_codebook_update(W, Q, m, H, cbw, W_hat=Wh)      # warm-up
        libgq.gq_check()
        Wh = W0.clone()
        traj = [f0]
        libgq.gq_kernel_timing_enable(True)
        e0.record()
        for _ in range(args.lnq_rounds):
            cbl, Wh = libgq.gq_codebook_update(W, Q, m, H, cbw, W_hat=Wh)
            Wh, Q = libgq.gq_cd_cycles(W, Wh, cbl, H, args.cycles, ws, Q=Q)
        cbl, Wh = libgq.gq_codebook_update(W, Q, m, H, cbw, W_hat=Wh)
        e1.record()
        e1.synchronize()
        kern = libgq.gq_kernel_timing_read()
        libgq.gq_kernel_timing_enable(False)
        libgq.gq_check()
        traj.append(float(libgq.gq_objective(W, Wh, H, ows).cpu()[-1]))
        out["lnq"] = {"rounds": args.lnq_rounds, "cd_cycles_per_round": args.cycles, "ms_total": e0.elapsed_time(e1),
                      "kernels_ms": {k: {"ms": round(v[0], 4), "launches": v[1]} for k, v in kern.items() if v[1]},
                      "objective_start": traj[0], "objective_end": traj[1]}
    print(json.dumps(out), flush=True)


if __name__ == "__main__":
    main()
