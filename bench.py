#!/usr/bin/env python
"""Benchmark of the guided-objective hot path (saliency -> guided Hessians -> objective).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload NAME]

One "step" is one pass of the whole path over one synthetic layer: gq_saliency_prepared for the first token
chunk, then one gq_hessian_accumulate_ahead per chunk (the Hessian step of that chunk and, on the warps it leaves
idle, the saliency step of the next one), then gq_hessian_finalize and gq_objective (H is zeroed at the start of
the step).  `--two-launch-chunks` runs gq_saliency_prepared + gq_hessian_accumulate per chunk instead.  The default workload is the Llama-2-7B attention-projection shape
(131072 tokens in 16 chunks of 8192, d_in = d_out = 4096, g = 4).  All inputs are seeded and
synthetic and stay resident in HBM for the device-timed number; the `e2e` number goes through
gq_layer_objective_host with pinned host buffers (host->device copies inside the timed region).

With N > 1 (launched by torch.distributed.run, one rank per GPU) every rank processes its own layer
(different seed): the path shards over layers with no data-path collective, so scaling is weak and the
only communication is the barrier / max-reduction of the timing.

`--impl reference` times the CPU fp64 oracle on the host cores on a bounded sample of the same
workload (rank 0 only).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np
import torch

from paper_2505_07004_b200 import shard, synth

METRIC = "guided_hessian_tokens_per_s"
UNIT = "tokens/s"
KERNEL_TIMING_EVERY = 8      # steps between two steps whose launches are timed one by one
NOMINAL_BF16_TFLOPS = 2250.0     # B200 dense bf16 / fp16 tensor peak (vendor figure), for context beside the measured peaks
# DRAM bytes (read + write) per launch of the dominant kernel, from an ncu capture of one launch of that
# workload; None where no capture of the current kernel exists.
# Keyed by (workload, chunk loop): a launch of the look-ahead loop also reads the next chunk's gradients.
NCU_TRAFFIC_BYTES = {("c1_7b_attn", "ahead"): 415.59e6, ("c1_7b_attn", "two_launch"): 347.50e6}
# The oracle sample both the cpu_baseline leg and --impl reference time (one size, so that the oracle's
# throughput is one number): tokens of chunk 0 for saliency + Hessian, channels per group for the objective.
ORACLE_SAMPLE_TOKENS, ORACLE_SAMPLE_CHANNELS = 1024, 64
OBJ_B2B_CALLS = 10           # calls of gq_objective inside one event pair
SAL_B2B_PASSES = 5           # passes over all chunks in the back-to-back saliency measurement
OBJECTIVE_KERNELS = ("split_delta", "gram_dot", "reduce")     # the kernels one gq_objective call launches
CPU_BASELINE_PASSES = 4      # passes of that sample in the cpu_baseline leg (about 10-15 s of host time)


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": float(p["hbm_gbs"]), "bf16_tflops": float(p["bf16_tflops"]),
                "bf16_tflops_sustained": float(p.get("bf16_tflops_sustained", p["bf16_tflops"])),
                "source": "of measured (MEASURED_PEAKS.json)"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0,
            "source": "of fallback (earlier measurement on this pool)"}


class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons of one GPU through NVML while the timed region runs."""
    REASONS = {0x4: "sw_power_cap", 0x8: "hw_slowdown", 0x20: "sw_thermal_slowdown",
               0x40: "hw_thermal_slowdown", 0x80: "hw_power_brake_slowdown", 0x2: "applications_clocks_setting"}

    def __init__(self, device):
        super().__init__(daemon=True)
        self.samples, self.reasons, self.max_mhz, self.ok = [], set(), None, False
        self._stop_evt = threading.Event()
        try:
            import pynvml
            pynvml.nvmlInit()
            uuid = str(torch.cuda.get_device_properties(device).uuid)
            if not uuid.startswith("GPU-"):
                uuid = "GPU-" + uuid
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByUUID(uuid.encode() if hasattr(uuid, "encode") else uuid)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
            self.ok = True
        except Exception as e:  # NVML missing: clocks are reported as unknown
            self.err = repr(e)

    def run(self):
        if not self.ok:
            return
        while not self._stop_evt.is_set():
            try:
                self.samples.append(int(self.nv.nvmlDeviceGetClockInfo(self.h, self.nv.NVML_CLOCK_SM)))
                try:
                    mask = int(self.nv.nvmlDeviceGetCurrentClocksEventReasons(self.h))
                except Exception:
                    mask = int(self.nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h))
                for bit, name in self.REASONS.items():
                    if mask & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            self._stop_evt.wait(0.02)

    def finish(self):
        self._stop_evt.set()
        self.join(timeout=2.0)
        if not self.ok or not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": ["nvml_unavailable"]}
        return {"sm_mhz": statistics.median(self.samples), "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(self.samples)}


def config_dict(cfg, g):
    """The workload description both arms print (identical keys and values)."""
    return {"workload": cfg.name, "n": cfg.n, "chunk": cfg.chunk, "d_in": cfg.d_in, "d_out": cfg.d_out, "g": g,
            "l2": "inputs (%.2f GB of X and grad per step, streamed once) are larger than L2; no flush"
                  % ((cfg.n * (cfg.d_in + cfg.d_out) * 2) / 1e9),
            "parallelism": "one layer per GPU, no collective"}


def hessian_issued_flops(d_in, g, tokens):
    """Flops the tensor cores are asked to do by one gq_hessian_accumulate launch: whole 256 x 256 tiles on the
    upper triangle (the half of every diagonal tile below the diagonal is computed and discarded), tokens
    rounded up to the 64-token step.  Pairs of groups share a tile pass; an odd last group runs on (row block,
    two column tiles) units."""
    nj = (d_in + 255) // 256
    tiles = nj * (nj + 1) // 2
    tok = (tokens + 63) // 64 * 64
    return 2.0 * 256 * 256 * tok * tiles * g


def dist_env():
    return int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")), int(os.environ.get("WORLD_SIZE", "1"))


def oracle_sample(cfg, g, tokens, channels_per_group, seed=0):
    """One bounded pass of the oracle: saliency + Hessian on `tokens` tokens of chunk 0 and the objective
    on `channels_per_group` channels of every group.  Returns (tokens/s equivalent, seconds, description)."""
    from oracle import gq_oracle as orc
    syn = synth.LayerSynth(cfg, "cpu", seed=seed)
    xb = synth.bf16_bits(syn.x_chunk(0, tokens))
    gb = synth.bf16_bits(syn.grad_chunk(0, tokens))
    m = cfg.d_out // g
    cpg = min(channels_per_group, m)
    W, What = syn.weights()
    rows = torch.cat([torch.arange(k * m, k * m + cpg) for k in range(g)])
    Wn, Whn = W[rows].contiguous().numpy(), What[rows].contiguous().numpy()
    t0 = time.perf_counter()
    s = orc.saliency(gb, g, 1.0)
    t1 = time.perf_counter()
    H = orc.hessian(xb, s)
    t2 = time.perf_counter()
    orc.objective(Wn, Whn, H)
    t3 = time.perf_counter()
    # the objective is paid once per layer: amortise its full-layer cost over the layer's n tokens
    t_obj_per_token = (t3 - t2) * (m / cpg) / cfg.n
    seconds = (t1 - t0) + (t2 - t1) + t_obj_per_token * tokens
    desc = ("fp64 oracle as is: saliency+Hessian on the first %d tokens of chunk 0 (%.2f s + %.2f s), objective on %d of "
            "%d channels per group (%.2f s) scaled to all channels and amortised over n=%d tokens"
            % (tokens, t1 - t0, t2 - t1, cpg, m, t3 - t2, cfg.n))
    return tokens / seconds, (t3 - t0), desc


def run_reference(args, cfg, g):
    rank, _, world = dist_env()
    if rank != 0:
        return
    from oracle import gq_oracle as orc
    orc.build()
    tokens, cpg = args.ref_tokens, args.ref_channels
    for _ in range(args.warmup):
        oracle_sample(cfg, g, tokens, cpg)
    t0 = time.perf_counter()
    vals = []
    desc = ""
    for _ in range(args.steps):
        v, _, desc = oracle_sample(cfg, g, tokens, cpg)
        vals.append(v)
    wall = time.perf_counter() - t0
    value = len(vals) / sum(1.0 / v for v in vals)          # harmonic mean = total tokens / total time
    out = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * wall / max(1, args.steps),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": config_dict(cfg, g),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": orc.threads(), "kind": "oracle", "sample": desc},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(out), flush=True)


def run_token_sharded(libgq, cfg, g, dev, rank, world):
    """One token-sharded layer on `world` GPUs: rank r accumulates chunks r, r + world, ... of the SAME synthetic layer
    into its own H (allocated in memory every rank can address), then the partial matrices are added by
    gq_hessian_reduce_share / gq_hessian_gather_shares with host barriers in between (plain peer loads; no kernel
    waits for another GPU).  Not part of the timed region of the headline number.  Returns the record for the JSON
    line (identical on every rank), or {"error": ...} if peer memory could not be set up."""
    import torch.distributed as dist

    def all_ok(ok):
        flag = torch.tensor([1 if ok else 0], dtype=torch.int32, device=dev)
        dist.all_reduce(flag, op=dist.ReduceOp.MIN)
        return bool(flag.item())

    try:
        H, ptrs, err = None, None, None
        try:
            H, ptrs = shard.allocate_symmetric_hessian(g, cfg.d_in, dev)
        except Exception as exc:
            err = repr(exc)[:300]
        if not all_ok(err is None):                             # every rank takes the same way out
            return {"error": err or "peer memory could not be set up on another rank"}
        syn = synth.LayerSynth(cfg, dev, seed=0)
        ws = libgq.alloc_workspace(libgq.gq_hessian_workspace_bytes(cfg.chunk, cfg.d_in, g), dev)
        mine = shard.chunks_for_rank(cfg.n_chunks, rank, world)
        xs = [syn.x_chunk(c) for c in mine]
        gs = [syn.grad_chunk(c) for c in mine]
        rank_ptrs = [H if r == rank else ptrs[r] for r in range(world)]

        def accumulate(Hbuf, xs_, gs_):
            for x, gr in zip(xs_, gs_):
                sb = libgq.gq_saliency_prepared(gr, g, ws, 1.0)
                libgq.gq_hessian_accumulate(x, sb, Hbuf, ws, flags=libgq.GQ_HESSIAN_S_PREPARED)

        accumulate(H, xs, gs)                                   # warm-up of kernels and peer mappings
        shard.exchange_hessian(H, rank_ptrs, rank)
        torch.cuda.synchronize()
        dist.barrier()
        H.zero_()
        torch.cuda.synchronize()
        dist.barrier()
        e = [torch.cuda.Event(enable_timing=True) for _ in range(3)]
        e[0].record()
        accumulate(H, xs, gs)
        e[1].record()
        shard.exchange_hessian(H, rank_ptrs, rank)
        e[2].record()
        torch.cuda.synchronize()
        libgq.gq_check()
        ms_acc, ms_ex = e[0].elapsed_time(e[1]), e[1].elapsed_time(e[2])
        # every rank must hold the same bits: compare a checksum of the bit patterns
        bits = H.view(torch.int32).to(torch.int64)
        checksum = torch.stack([bits.sum(), (bits * (torch.arange(bits.numel(), device=dev).view_as(bits) % 1021)).sum()])
        sums = [torch.zeros_like(checksum) for _ in range(world)]
        dist.all_gather(sums, checksum)
        bit_equal = all(bool(torch.equal(t, sums[0])) for t in sums)
        # rank 0 also builds the layer unsharded and compares (summation order differs)
        rel = torch.zeros(1, dtype=torch.float64, device=dev)
        if rank == 0:
            H1 = torch.zeros_like(H)
            accumulate(H1, [syn.x_chunk(c) for c in range(cfg.n_chunks)], [syn.grad_chunk(c) for c in range(cfg.n_chunks)])
            libgq.gq_hessian_finalize(H1)
            libgq.gq_check()
            rel[0] = ((H.double() - H1.double()).norm() / H1.double().norm()).item()
            del H1
        dist.broadcast(rel, 0)
        ms_acc, ms_ex = shard.max_over_ranks([ms_acc, ms_ex], device=dev)
        nvl = shard.exchange_bytes_per_rank(cfg.d_in, g, world)
        return {"ms_accumulate": ms_acc, "ms_exchange": ms_ex, "bytes_over_nvlink": nvl,
                "exchange_gbs_per_rank": nvl / (ms_ex * 1e-3) / 1e9 if ms_ex > 0 else None,
                "all_ranks_bit_equal": bit_equal, "max_rel_vs_rank0_unsharded": float(rel.item()),
                "chunks_per_rank": len(mine), "note": "exchange time includes its three host barriers and the mirror step"}
    except Exception as exc:      # peer memory unavailable etc.: the headline numbers stand, the leg reports why it did not run
        return {"error": repr(exc)[:300]}


def run_ours(args, cfg, g):
    from paper_2505_07004_b200 import api as libgq
    rank, local_rank, world = dist_env()
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: libgq has no CPU path")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
    libgq.lib()
    peaks = load_peaks()

    # ---- resident synthetic layer (one per rank: the path shards over layers)
    syn = synth.LayerSynth(cfg, dev, seed=shard.layer_seed_for_rank(0, rank))
    n_chunks = cfg.n_chunks
    xs = [syn.x_chunk(c) for c in range(n_chunks)]
    gs = [syn.grad_chunk(c) for c in range(n_chunks)]
    W, What = syn.weights()
    H = torch.empty((g, cfg.d_in, cfg.d_in), dtype=torch.float32, device=dev)
    s_buf = torch.empty((g, cfg.chunk), dtype=torch.float32, device=dev)
    s_alt = torch.empty((g, cfg.chunk), dtype=torch.float32, device=dev)
    ws = libgq.alloc_workspace(libgq.gq_hessian_workspace_bytes(cfg.chunk, cfg.d_in, g), dev)
    ws_alt = libgq.alloc_workspace(libgq.gq_hessian_workspace_bytes(cfg.chunk, cfg.d_in, g), dev)
    ows = libgq.alloc_workspace(libgq.gq_objective_workspace_bytes(cfg.d_in, cfg.d_out, g), dev)
    loss = torch.empty(g + 1, dtype=torch.float64, device=dev)

    def step_two_launch_chunks():
        H.zero_()
        for c in range(n_chunks):
            nt = xs[c].shape[0]
            libgq.gq_saliency_prepared(gs[c], g, ws, 1.0, s=s_buf[:, :nt])
            libgq.gq_hessian_accumulate(xs[c], s_buf[:, :nt], H, ws, flags=libgq.GQ_HESSIAN_S_PREPARED)
        libgq.gq_hessian_finalize(H)
        libgq.gq_objective(W, What, H, ows, loss=loss)

    def step_ahead():
        # two saliency buffers / scratch blocks in turn: chunk c reads one pair while chunk c + 1's is written
        sb, wb = (s_buf, s_alt), (ws, ws_alt)
        H.zero_()
        libgq.gq_saliency_prepared(gs[0], g, wb[0], 1.0, s=sb[0][:, :gs[0].shape[0]])
        for c in range(n_chunks):
            nt = xs[c].shape[0]
            if c + 1 < n_chunks:
                libgq.gq_hessian_accumulate_ahead(xs[c], sb[c & 1][:, :nt], H, wb[c & 1], gs[c + 1], wb[(c + 1) & 1], 1.0,
                                                  sb[(c + 1) & 1][:, :gs[c + 1].shape[0]], flags=libgq.GQ_HESSIAN_S_PREPARED)
            else:
                libgq.gq_hessian_accumulate(xs[c], sb[c & 1][:, :nt], H, wb[c & 1], flags=libgq.GQ_HESSIAN_S_PREPARED)
        libgq.gq_hessian_finalize(H)
        libgq.gq_objective(W, What, H, ows, loss=loss)

    step = step_two_launch_chunks if args.two_launch_chunks else step_ahead

    def barrier():
        if world > 1:
            import torch.distributed as dist
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(args.warmup):
        step()
    libgq.gq_check()

    sampler = ClockSampler(dev)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    launches0 = libgq.gq_launch_count()
    # Per-kernel durations come from CUDA-event pairs around every launch (gq_kernel_timing_*).  The pairs
    # themselves cost about 4 % of a step (52 launches), so they are recorded in every KERNEL_TIMING_EVERY-th
    # step of the timed region only, which keeps their cost in the whole-job number below 1 %.
    libgq.gq_kernel_timing_enable(False)
    libgq.gq_kernel_timing_read()
    sampler.start()
    e0.record()
    for i in range(args.steps):
        sampled = (i % KERNEL_TIMING_EVERY == 0)
        if sampled:
            libgq.gq_kernel_timing_enable(True)
        step()
        if sampled:
            libgq.gq_kernel_timing_enable(False)
    e1.record()
    barrier()
    clocks = sampler.finish()
    ms_total = e0.elapsed_time(e1)
    kern = libgq.gq_kernel_timing_read()
    launches = libgq.gq_launch_count() - launches0
    libgq.gq_check()
    loss_host = loss.cpu().numpy()
    if not np.all(np.isfinite(loss_host)) or loss_host[g] <= 0:
        raise RuntimeError("objective is not finite/positive: %s" % loss_host)

    # ---- the Hessian kernel without the look-ahead work: two passes of the two-launch chunk loop right after the
    # timed region (same clocks, same cache state), an event pair around every launch
    plain_hessian = None
    if not args.two_launch_chunks:
        step_two_launch_chunks()
        libgq.gq_kernel_timing_read()
        libgq.gq_kernel_timing_enable(True)
        for _ in range(2):
            step_two_launch_chunks()
        libgq.gq_kernel_timing_enable(False)
        torch.cuda.synchronize()
        k2 = libgq.gq_kernel_timing_read()
        if k2["hessian"][1]:
            plain_hessian = k2["hessian"][0] / k2["hessian"][1]
        libgq.gq_check()

    # ---- saliency alone: all chunks' launches captured into one CUDA graph (no host time between launches, no
    # per-launch event pair), replayed SAL_B2B_PASSES times inside one event pair
    sal_b2b_gbs = None
    if n_chunks * cfg.chunk * cfg.d_out * 2 > 200e6:                    # only meaningful when a pass exceeds L2
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            for c in range(n_chunks):
                libgq.gq_saliency_prepared(gs[c], g, ws, 1.0, s=s_buf[:, :gs[c].shape[0]])
        side.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            for c in range(n_chunks):
                libgq.gq_saliency_prepared(gs[c], g, ws, 1.0, s=s_buf[:, :gs[c].shape[0]])
        graph.replay()
        torch.cuda.synchronize()
        b0, b1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        b0.record()
        for _ in range(SAL_B2B_PASSES):
            graph.replay()
        b1.record()
        torch.cuda.synchronize()
        sal_b2b_gbs = SAL_B2B_PASSES * sum(x.shape[0] * (2 * cfg.d_out + 4 * g) for x in gs) / (b0.elapsed_time(b1) * 1e-3) / 1e9
        del graph

    # ---- the objective alone: OBJ_B2B_CALLS calls inside one event pair (its inputs, W, W_hat and H, exceed L2)
    libgq.gq_objective(W, What, H, ows, loss=loss)
    torch.cuda.synchronize()
    o0, o1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    o0.record()
    for _ in range(OBJ_B2B_CALLS):
        libgq.gq_objective(W, What, H, ows, loss=loss)
    o1.record()
    torch.cuda.synchronize()
    obj_b2b_ms = o0.elapsed_time(o1) / OBJ_B2B_CALLS
    libgq.gq_check()

    # ---- end to end from pinned host memory through the host-buffer entry point
    e2e_s, e2e_steps, h2d, d2h = float('nan'), 0, 0, 0
    if not args.no_e2e:
        e2e_steps = max(1, min(args.steps, args.e2e_steps))
        Xh = torch.empty((cfg.n, cfg.d_in), dtype=torch.bfloat16).pin_memory()
        Gh = torch.empty((cfg.n, cfg.d_out), dtype=torch.bfloat16).pin_memory()
        off = 0
        for c in range(n_chunks):
            nt = xs[c].shape[0]
            Xh[off:off + nt].copy_(xs[c])
            Gh[off:off + nt].copy_(gs[c])
            off += nt
        Wh, Whh = W.cpu().pin_memory(), What.cpu().pin_memory()
        loss_h = torch.empty(g + 1, dtype=torch.float64).pin_memory()
        del xs, gs
        torch.cuda.empty_cache()
        arena = libgq.alloc_workspace(libgq.gq_layer_host_arena_bytes(cfg.chunk, cfg.d_in, cfg.d_out, g), dev)
        libgq.gq_layer_objective_host(Xh, Gh, cfg.chunk, g, 1.0, Wh, Whh, arena, loss_host=loss_h)   # warm-up
        barrier()
        t0 = time.perf_counter()
        for _ in range(e2e_steps):
            libgq.gq_layer_objective_host(Xh, Gh, cfg.chunk, g, 1.0, Wh, Whh, arena, loss_host=loss_h)
        torch.cuda.synchronize()
        e2e_s = time.perf_counter() - t0
        # same arithmetic on both paths; the units that were cut along the token axis are added to H in an
        # order that varies from launch to launch, hence agreement to fp32 summation order only
        if abs(loss_h[g].item() - loss_host[g]) > 1e-6 * abs(loss_host[g]):
            raise RuntimeError("host-buffer path and device path disagree: %r vs %r" % (loss_h[g].item(), loss_host[g]))
        h2d = Xh.numel() * 2 + Gh.numel() * 2 + Wh.numel() * 4 + Whh.numel() * 4
        d2h = (g + 1) * 8

    # ---- N > 1 only: ONE layer (seed of rank 0) with its token chunks dealt to the ranks, partial matrices added
    # by the library's exchange kernels over peer memory (Algorithm 1, Hessian step: H is a sum over tokens)
    token_sharded = None
    if world > 1 and not args.no_token_sharded:
        token_sharded = run_token_sharded(libgq, cfg, g, dev, rank, world)

    # ---- max over ranks
    ms_total, e2e_ms = shard.max_over_ranks([ms_total, e2e_s * 1e3], device=dev)

    if rank == 0:
        value = shard.whole_job_throughput(cfg.n, args.steps, ms_total * 1e-3, world)
        e2e_value = shard.whole_job_throughput(cfg.n, e2e_steps, e2e_ms * 1e-3, world) if e2e_steps else None
        # dominant kernel: the tensor-core kernel of gq_hessian_accumulate
        ga_ms, ga_n = kern["hessian"]
        flops_per_launch = float(g) * cfg.chunk * cfg.d_in * (cfg.d_in + 1)      # upper triangle, mul + add
        issued_per_launch = hessian_issued_flops(cfg.d_in, g, cfg.chunk)
        ms_per_launch = ga_ms / max(1, ga_n)
        achieved = flops_per_launch / (ms_per_launch * 1e-3) / 1e12 if ga_n else None
        issued = issued_per_launch / (ms_per_launch * 1e-3) / 1e12 if ga_n else None
        # Which measured tensor peak applies: the burst figure when the sampled SM clock stayed near its maximum (the
        # kernel ran as in a burst), the sustained one when the run sat at the power cap with the clock pulled
        # down.  Both fractions are printed either way.
        sm, sm_max = clocks.get("sm_mhz"), clocks.get("sm_max_mhz")
        near_max = bool(sm and sm_max and sm >= 0.9 * sm_max)
        burst = near_max if (sm and sm_max) else ms_total < 1000.0          # no clock samples: go by the duration
        peak = peaks["bf16_tflops"] if burst else peaks["bf16_tflops_sustained"]
        kernel_ms = sum(v[0] for v in kern.values())
        kernels = {k: {"launches": v[1], "ms_total": round(v[0], 4), "share": round(v[0] / kernel_ms, 4) if kernel_ms else None}
                   for k, v in kern.items()}
        sal_ms, sal_n = kern["saliency"]
        sal_bytes = cfg.chunk * (2 * cfg.d_out + 4 * g)
        frac = lambda a, p: (a / p) if (a is not None and p) else None
        roofline = {
            "kernel": "hessian_kernel (gq_hessian_accumulate)" if args.two_launch_chunks else
                      "hessian_kernel (gq_hessian_accumulate_ahead: the launch also computes the next chunk's saliency; "
                      "only the Hessian flops are counted)", "bound": "tensor",
            "achieved": achieved, "peak": peak, "unit": "TFLOP/s", "frac": frac(achieved, peak),
            "traffic": NCU_TRAFFIC_BYTES.get((cfg.name, "two_launch" if args.two_launch_chunks else "ahead")),
            "peak_source": ("bf16_tflops (burst), " if burst else "bf16_tflops_sustained, ") + peaks["source"],
            "peak_regime": ("burst: %s" % ("median SM clock %.0f of %.0f MHz" % (sm, sm_max) if near_max
                                           else "no clock samples, timed region of %.2f s" % (ms_total * 1e-3))) if burst
                           else "sustained: timed region of %.2f s at a median SM clock of %s of %s MHz" % (ms_total * 1e-3, sm, sm_max),
            "frac_of_burst_peak": frac(achieved, peaks["bf16_tflops"]),
            "frac_of_sustained_peak": frac(achieved, peaks["bf16_tflops_sustained"]),
            "frac_of_nominal_peak": frac(achieved, NOMINAL_BF16_TFLOPS),
            "peaks_tflops": {"burst": peaks["bf16_tflops"], "sustained": peaks["bf16_tflops_sustained"],
                             "nominal": NOMINAL_BF16_TFLOPS},
            "flops_per_launch": flops_per_launch, "ms_per_launch": ms_per_launch,
            "issued_flops_per_launch": issued_per_launch, "issued_tflops": issued,
            "issued_frac_of_nominal_peak": frac(issued, NOMINAL_BF16_TFLOPS),
            "target": "60 %% of the nominal peak: %s" % ("met" if (achieved or 0) >= 0.6 * NOMINAL_BF16_TFLOPS else "not met"),
        }
        if plain_hessian:
            tf = flops_per_launch / (plain_hessian * 1e-3) / 1e12
            roofline["without_look_ahead"] = {
                "ms_per_launch": plain_hessian, "achieved": tf, "frac_of_burst_peak": frac(tf, peaks["bf16_tflops"]),
                "frac_of_sustained_peak": frac(tf, peaks["bf16_tflops_sustained"]), "frac_of_nominal_peak": frac(tf, NOMINAL_BF16_TFLOPS),
                "timing": "event pairs around the gq_hessian_accumulate launches of two passes of the two-launch chunk loop, "
                          "run directly after the timed region (the launches of the timed region also compute the next "
                          "chunk's saliency)"}
        sal_gbs = (sal_bytes / (sal_ms / max(1, sal_n) * 1e-3) / 1e9) if sal_n else None
        saliency_roofline = {
            "kernel": "saliency_kernel (gq_saliency_prepared) as a launch of its own" +
                      ("" if args.two_launch_chunks else "; in the step only the first chunk's saliency is such a launch, "
                       "the others run inside the Hessian launches"),
            "bound": "hbm", "unit": "GB/s", "peak": peaks["hbm_gbs"],
            "bytes_per_launch": sal_bytes,
            "achieved": sal_b2b_gbs, "frac": frac(sal_b2b_gbs, peaks["hbm_gbs"]),
            "timing": "one event pair around %d replays of a CUDA graph holding the launches of all %d chunks "
                      "(%.2f GB per replay, larger than L2)" % (SAL_B2B_PASSES, n_chunks, n_chunks * sal_bytes / 1e9),
            "achieved_per_launch_events": sal_gbs, "frac_per_launch_events": frac(sal_gbs, peaks["hbm_gbs"]),
            "timing_per_launch_events": "event pair around each launch inside the step (a %d MB launch lasts ~12 us: the "
                                        "pair's own cost is part of this figure)" % (sal_bytes // 1000000),
        }
        objective_roofline = None
        if kern["gram_dot"][1]:
            calls = kern["gram_dot"][1]
            obj_events_ms = sum(kern[k][0] for k in OBJECTIVE_KERNELS) / calls
            obj_ms = obj_b2b_ms
            obj_bytes = 2.0 * g * cfg.d_in * (cfg.d_in + 1) + 8.0 * cfg.d_in * cfg.d_out     # upper triangle of H (fp32) + W, W_hat
            obj_flops_sym = float(cfg.d_in) * cfg.d_in * cfg.d_out                           # 2 d_in^2 d_out, halved by symmetry
            t_bytes = obj_bytes / (peaks["hbm_gbs"] * 1e9) * 1e3
            t_flops = obj_flops_sym / (peaks["bf16_tflops"] * 1e12) * 1e3
            objective_roofline = {
                "kernel": "gq_objective (all of its kernels)", "ms_per_call": obj_ms,
                "timing": "one event pair around %d back-to-back calls" % OBJ_B2B_CALLS,
                "ms_per_call_kernel_events": obj_events_ms,
                "bound": "tensor" if t_flops >= t_bytes else "hbm",
                "algorithmic_bytes": obj_bytes, "symmetric_flops": obj_flops_sym,
                "ms_at_hbm_peak": t_bytes, "ms_at_tensor_burst_peak": t_flops,
                "frac": max(t_bytes, t_flops) / obj_ms,
                "gbs_algorithmic": obj_bytes / (obj_ms * 1e-3) / 1e9,
                "frac_of_hbm_peak": obj_bytes / (obj_ms * 1e-3) / 1e9 / peaks["hbm_gbs"],
                "tflops_symmetric": obj_flops_sym / (obj_ms * 1e-3) / 1e12,
                "tflops_dense_equivalent": 2.0 * obj_flops_sym / (obj_ms * 1e-3) / 1e12,
                "note": "frac = the slower of (bytes at the measured copy bandwidth, symmetric flops at the measured burst "
                        "16-bit tensor peak) divided by the measured time of the whole call",
            }
        out = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": ms_total / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16", "data": "synthetic",
            "config": config_dict(cfg, g),
            "hessian_tflops_useful": (float(g) * cfg.n * cfg.d_in * (cfg.d_in + 1)) * world * args.steps / (ms_total * 1e-3) / 1e12,
            "roofline": roofline,
            "saliency_hbm": saliency_roofline,
            "objective": objective_roofline,
            "kernels": kernels,
            "kernel_timing": "CUDA-event pairs around every launch of every %d-th timed step" % KERNEL_TIMING_EVERY,
            "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                    "steps": e2e_steps, "api": "gq_layer_objective_host (pinned host buffers)"},
            "gpu_launches": int(launches),
            "chunk_loop": ("gq_saliency_prepared + gq_hessian_accumulate per chunk" if args.two_launch_chunks else
                           "gq_hessian_accumulate_ahead: the saliency step of chunk c + 1 runs inside the Hessian launch of chunk c"),
            "clocks": clocks,
            "loss_total": float(loss_host[g]),
        }
        if token_sharded is not None:
            out["token_sharded"] = token_sharded
        if world == 1 and not args.no_cpu_baseline:
            from oracle import gq_oracle as orc
            orc.build()
            vals, secs, desc = [], 0.0, ""
            for _ in range(CPU_BASELINE_PASSES):
                v, sec, desc = oracle_sample(cfg, g, args.cpu_tokens, args.cpu_channels)
                vals.append(v)
                secs += sec
            out["cpu_baseline"] = {"value": len(vals) / sum(1.0 / v for v in vals), "unit": UNIT, "cores": orc.threads(),
                                   "kind": "oracle", "sample": "%d passes of: %s" % (CPU_BASELINE_PASSES, desc),
                                   "seconds": secs}
        print(json.dumps(out), flush=True)
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c1_7b_attn", choices=sorted(synth.CONFIGS))
    ap.add_argument("--g", type=int, default=0, help="override the number of groups (sweep config)")
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--cpu-tokens", type=int, default=ORACLE_SAMPLE_TOKENS)
    ap.add_argument("--cpu-channels", type=int, default=ORACLE_SAMPLE_CHANNELS)
    ap.add_argument("--ref-tokens", type=int, default=ORACLE_SAMPLE_TOKENS,
                    help="tokens per step of the reference arm (the same sample as the cpu_baseline leg)")
    ap.add_argument("--ref-channels", type=int, default=ORACLE_SAMPLE_CHANNELS)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer leg (profiling runs)")
    ap.add_argument("--no-token-sharded", action="store_true", help="N > 1: skip the token-sharded layer with the peer-memory exchange")
    ap.add_argument("--two-launch-chunks", action="store_true",
                    help="per chunk gq_saliency_prepared + gq_hessian_accumulate instead of gq_hessian_accumulate_ahead")
    ap.add_argument("--tokens", type=int, default=0, help="use only the first TOKENS tokens (profiling runs)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    cfg = synth.CONFIGS[args.workload]
    if args.tokens:
        import dataclasses
        cfg = dataclasses.replace(cfg, n=min(cfg.n, args.tokens))
    g = args.g if args.g else cfg.g
    if args.impl == "reference":
        run_reference(args, cfg, g)
    else:
        run_ours(args, cfg, g)


if __name__ == "__main__":
    main()
