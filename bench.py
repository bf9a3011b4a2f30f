#!/usr/bin/env python
"""Benchmark of the GKA hot path on B200.

One "step" is one pass of the chunk-wise forward (gate prep, state scan, chunk-wise Frobenius
norms, Chebyshev iterations, output, state carry) over one batch of configuration 1
(B=4, heads=16, T=4096, d=128, chunk=64, n_iter=10, bf16 I/O).  The recurrent decode step
(configuration 2: 256 sequences x 32 heads, fp32 state) is timed in the same run and reported
in the "decode" object of the same JSON line, next to "fwd_r30" (the same shapes at the paper's
setting: 30 iterations, lambda_t = 0.02 ||H_t||_F), "fwd_d64" (the same shapes at head dimension 64) and "fwd_long"
(configuration 3, T = 131072).

    python bench.py --gpus N --steps K --warmup W            # this library
    python bench.py --impl reference --steps K --warmup W    # the fp64 CPU oracle, bounded sample
    python bench.py --case fwd 2 16 4096 10 3                # one small case a few times (profiling captures)

Under torchrun every rank runs its own seeded batch of the same shape (weak scaling; (batch, head)
pairs are independent, so there is no data-path collective); times are the max over ranks.
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

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

from paper_2511_21016_b200 import shard, synth  # noqa: E402

METRIC = "gka_layer_fwd_tokens_per_s"
UNIT = "tokens/s"
KERNEL_PASS_LAUNCHES = 20  # launches of the separate pass that times the dominant kernel alone
SAMPLING_PASS_S = 0.4      # length of the back-to-back pass during which the clocks are sampled
L2_FLUSH_BYTES = 256 << 20

# DRAM traffic per launch of the dominant kernels (dram__bytes_read.sum + dram__bytes_write.sum from the
# ncu captures summarised under profiles/).  Both captures ran a half / quarter-size case of the same kernel
# (solve kernel: 1024 of 2048 tiles; decode: 2048 of 8192 (sequence, head) pairs) and are scaled by the
# units per launch; traffic is proportional to the units in both kernels.
NCU_TRAFFIC_BYTES = {"fwd_solve_per_tile": (169_212_672 + 16_138_240) / 1024, "decode": 4 * 482_096_896}


def fwd_flops(n_chunks: int, n_iter: int, C: int = 64, D: int = 128, part: str = "all") -> float:
    """Algorithmic flops of the chunk-wise forward (masked triangles and symmetric halves counted
    once, no credit for padding, split operands or the segment-summary pass).  part = "solve": the
    share of the solve kernel (everything but the state update, which the state kernel does)."""
    it = 2 * C * D * D + 2 * D * C * (C + 1)
    s5 = it
    s1 = C * D * (D + 1) + 2 * C * D * D
    s2 = 2 * C * D * D + D * C * (C + 1) + C * C * (C + 1)
    return float(n_chunks) * (n_iter * it + s5 + s2 + (0 if part == "solve" else s1))


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return dict(hbm_gbs=p["hbm_gbs"], bf16_tflops=p["bf16_tflops"],
                    bf16_tflops_sustained=p.get("bf16_tflops_sustained"), source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, source="fallback")


class ClockSampler:
    """nvidia-smi clock / throttle-reason samples taken while the timed region runs."""

    FIELDS = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu_index = gpu_index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "20", "-i", str(self.gpu_index)],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons, power = [], [], set(), []
        for ln in self.lines:
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1])); mx.append(float(f[2])); power.append(float(f[3]))
            except ValueError:
                continue
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown",
                                  "sw_power_cap"), f[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        top = sorted(sm)[len(sm) // 2:]          # samples under load are the upper half
        return {"sm_mhz": statistics.median(top), "sm_max_mhz": max(mx), "reasons": sorted(reasons),
                "samples": len(sm), "power_w_max": max(power)}


# ------------------------------------------------------------------------------------ reference arm
def run_reference(args):
    """The fp64 CPU oracle as it stands, timed on the host cores on a bounded sample of cfg 1."""
    rank, _, world = shard.env_rank_world()
    if rank != 0:
        return 0
    import oracle
    cfg = synth.CONFIGS[1]
    cores = oracle.max_threads()
    T_s = 256
    pairs = [(i // cfg.heads % cfg.B, i % cfg.heads) for i in range(cores)]
    sample_cfg = synth.shrink(cfg, T=T_s)
    heads_in = []
    for (b, h) in pairs:
        heads_in.append(synth.draw_head(sample_cfg, b, h, T_s))
    q = np.stack([x[0] for x in heads_in], 1)[None]      # [1, T, pairs, d]
    k = np.stack([x[1] for x in heads_in], 1)[None]
    v = np.stack([x[2] for x in heads_in], 1)[None]
    g = np.stack([x[3] for x in heads_in], 1)[None]
    lam = np.stack([x[4] for x in heads_in], 1)[None]
    q, k, v = (synth.round_bf16(a.astype(np.float32)) for a in (q, k, v))
    for _ in range(args.warmup):
        oracle.fwd(q, k, v, g, lam, cfg.n_iter)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle.fwd(q, k, v, g, lam, cfg.n_iter)
    dt = (time.perf_counter() - t0) / args.steps
    head_tokens = len(pairs) * T_s
    value = head_tokens / cfg.heads / dt                  # layer tokens/s (all heads of the layer)
    sample = (f"{len(pairs)} (batch, head) pairs x {T_s} tokens of cfg1 per step, fp64 token-by-token "
              f"oracle, OpenMP over pairs")
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic",
        "config": {"workload": cfg.name, "B": cfg.B, "heads": cfg.heads, "T": cfg.T, "d": cfg.d,
                   "chunk": cfg.chunk, "n_iter": cfg.n_iter, "io_dtype": cfg.io_dtype},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))
    return 0


# ------------------------------------------------------------------------------------------ our arm
def make_decode_inputs_device(cfg, device, seed):
    """Configuration 2 inputs drawn on the device with torch's seeded generator (the host recipe of
    synth.py at this size would take minutes): same distributions, bf16 q/k/v, fp32 gate / lam."""
    import torch
    gen = torch.Generator(device=device)
    gen.manual_seed(seed)
    N, Hh, d, Tp = cfg.B, cfg.heads, cfg.d, cfg.prefix_T

    def unit(shape):
        x = torch.randn(shape, generator=gen, device=device, dtype=torch.float32)
        return (x / x.norm(dim=-1, keepdim=True)).to(torch.bfloat16)

    def gates(shape):
        return torch.sigmoid(torch.randn(shape, generator=gen, device=device) + cfg.gate_mean)

    def lams(shape):
        return torch.nn.functional.softplus(torch.randn(shape, generator=gen, device=device) + cfg.lam_mean) \
            * cfg.lam_scale + cfg.lam_eps

    pre = dict(q=unit((N, Tp, Hh, d)), k=unit((N, Tp, Hh, d)),
               v=torch.randn((N, Tp, Hh, d), generator=gen, device=device).to(torch.bfloat16),
               gate=gates((N, Tp, Hh)), lam=lams((N, Tp, Hh)))
    step = dict(q=unit((N, Hh, d)), k=unit((N, Hh, d)),
                v=torch.randn((N, Hh, d), generator=gen, device=device).to(torch.bfloat16),
                gate=gates((N, Hh)), lam=lams((N, Hh)))
    return pre, step


def make_fwd_inputs_device(cfg, device, seed):
    """Forward inputs of a configuration drawn on the device with torch's seeded generator (for the sizes whose
    host recipe would take minutes): same distributions as synth.py, bf16 q/k/v, fp32 gate / lam."""
    import torch
    gen = torch.Generator(device=device)
    gen.manual_seed(seed)
    shape = (cfg.B, cfg.T, cfg.heads, cfg.d)

    def unit():
        x = torch.randn(shape, generator=gen, device=device, dtype=torch.float32)
        return (x / x.norm(dim=-1, keepdim=True)).to(torch.bfloat16)

    q, k = unit(), unit()
    v = torch.randn(shape, generator=gen, device=device).to(torch.bfloat16)
    gate = torch.sigmoid(torch.randn(shape[:-1], generator=gen, device=device) + cfg.gate_mean)
    lam = torch.nn.functional.softplus(torch.randn(shape[:-1], generator=gen, device=device) + cfg.lam_mean) \
        * cfg.lam_scale + cfg.lam_eps
    return dict(q=q, k=k, v=v, gate=gate, lam=lam)


def time_forward(gka, dev, cfg, n_iter, flags, steps, warmup, peaks, stream, new_event, flush, world, device):
    """K timed calls of the chunk-wise forward (L2 flushed between calls, CUDA events on the launch stream, every
    call exactly as a user's), then a separate pass of bracketed launches that times the dominant kernel alone."""
    import torch
    out = torch.empty_like(dev["v"])
    state_out = torch.empty(cfg.B, cfg.heads, 2 * cfg.d * cfg.d, dtype=torch.float32, device=device)
    ws = gka.alloc_workspace(cfg.B, cfg.T, cfg.heads, cfg.d, device)
    status = torch.zeros(1, dtype=torch.int32, device=device)

    def fwd(profile=None):
        gka.gka_fwd_chunked(dev["q"], dev["k"], dev["v"], dev["gate"], dev["lam"], n_iter, cfg.chunk, out=out,
                            state_out=state_out, workspace=ws, device_status=status, flags=flags,
                            profile_events=profile)

    for _ in range(warmup):
        flush.zero_()
        fwd()
    torch.cuda.synchronize()
    ev = [(new_event(), new_event()) for _ in range(steps)]
    torch.cuda.synchronize()
    shard.barrier()
    torch.cuda.synchronize()
    wall0 = time.perf_counter()
    for i in range(steps):
        flush.zero_()
        ev[i][0].record(stream)
        fwd()
        ev[i][1].record(stream)
    torch.cuda.synchronize()
    shard.barrier()
    wall = time.perf_counter() - wall0
    total_ms = shard.max_over_ranks(sum(a.elapsed_time(b) for a, b in ev), device)
    ms_per_step = total_ms / steps
    # the dominant kernel alone: the library records the two events right around its launch
    kev = [(new_event(), new_event()) for _ in range(KERNEL_PASS_LAUNCHES)]
    torch.cuda.synchronize()
    for i in range(KERNEL_PASS_LAUNCHES):
        flush.zero_()
        fwd(profile=(kev[i][0].cuda_event, kev[i][1].cuda_event))
    torch.cuda.synchronize()
    assert int(status.item()) == 0, "a device-side bounded wait timed out"
    kernel_ms = statistics.mean(a.elapsed_time(b) for a, b in kev)
    n_chunks = cfg.B * cfg.heads * ((cfg.T + cfg.chunk - 1) // cfg.chunk)
    n_tiles = cfg.B * cfg.heads * ((cfg.T + 127) // 128)
    flops_solve = fwd_flops(n_chunks, n_iter, cfg.chunk, cfg.d, part="solve")
    flops_all = fwd_flops(n_chunks, n_iter, cfg.chunk, cfg.d)
    achieved_tf = flops_solve / (kernel_ms * 1e-3) / 1e12
    tokens_per_step = cfg.B * cfg.T * world
    roofline = {"bound": "tensor", "kernel": "fwd_tc_solve_kernel (Frobenius norms, Chebyshev iterations, read)",
                "achieved": achieved_tf, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
                "frac": achieved_tf / peaks["bf16_tflops"], "peak_source": peaks["source"] + " (burst cuBLAS bf16)",
                "traffic": int(NCU_TRAFFIC_BYTES["fwd_solve_per_tile"] * n_tiles), "flops_per_launch": flops_solve,
                "kernel_ms": kernel_ms, "kernel_launches_timed": KERNEL_PASS_LAUNCHES,
                "whole_call_flops": flops_all,
                "whole_call_frac": flops_all / (ms_per_step * 1e-3) / 1e12 / peaks["bf16_tflops"],
                "frac_of_nominal_2250": achieved_tf / 2250.0}
    return dict(ms_per_step=ms_per_step, value=tokens_per_step / (ms_per_step * 1e-3), roofline=roofline, wall=wall,
                fwd=fwd, ws=ws, status=status)


def run_ours(args):
    import torch
    from paper_2511_21016_b200 import gka

    rank, local_rank, world = shard.env_rank_world()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the product path has no CPU fallback")
    torch.cuda.set_device(local_rank)
    device = f"cuda:{local_rank}"
    if world > 1:
        shard.init_process_group("nccl")
    peaks = load_peaks()
    gka.load_library()

    cfg = synth.CONFIGS[args.config]
    assert cfg.kind == "fwd"
    cfg = synth.shrink(cfg, seed=shard.shard_seed(cfg.seed, rank))
    t_gen = time.perf_counter()
    host = synth.make_inputs(cfg)
    t_gen = time.perf_counter() - t_gen
    bf16 = cfg.io_dtype == "bf16"
    io_t = torch.bfloat16 if bf16 else torch.float32

    # pinned host buffers (the end-to-end arm copies from / to these every step)
    pin = {}
    for n in ("q", "k", "v"):
        pin[n] = torch.from_numpy(host[n]).to(io_t).pin_memory()
    for n in ("gate", "lam"):
        pin[n] = torch.from_numpy(host[n]).pin_memory()
    dev = {n: torch.empty_like(t, device=device) for n, t in pin.items()}
    for n in pin:
        dev[n].copy_(pin[n])
    out_pin = torch.empty_like(pin["v"]).pin_memory()
    flush = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device=device)
    stream = torch.cuda.current_stream()

    def new_event():
        e = torch.cuda.Event(enable_timing=True)
        e.record(stream)          # creates the underlying cudaEvent_t so that its handle can be passed
        return e

    K, W = args.steps, args.warmup
    sampler = ClockSampler(local_rank)
    sampler.start()
    # ---- device-resident timing of the headline workload
    head = time_forward(gka, dev, cfg, cfg.n_iter, 0, K, W, peaks, stream, new_event, flush, world, device)
    ms_per_step, value, roofline, wall = head["ms_per_step"], head["value"], head["roofline"], head["wall"]
    tokens_per_step = cfg.B * cfg.T * world
    ws, status = head["ws"], head["status"]
    # ---- the same call back to back for a few hundred milliseconds, so that the clock samples (one per 20 ms) fall
    # inside a region that runs nothing else
    n_back = max(8, int(SAMPLING_PASS_S / (ms_per_step * 1e-3)))
    b0, b1 = new_event(), new_event()
    torch.cuda.synchronize()
    b0.record(stream)
    for _ in range(n_back):
        head["fwd"]()
    b1.record(stream)
    torch.cuda.synchronize()
    back_ms = b0.elapsed_time(b1) / n_back

    # ---- end to end: pinned host -> device copies, forward, device -> host read of the result
    h2d = sum(pin[n].numel() * pin[n].element_size() for n in pin)
    d2h = out_pin.numel() * out_pin.element_size()

    staging = torch.empty(gka.gka_fwd_host_staging_bytes(cfg.B, cfg.T, cfg.heads, cfg.d,
                                                         gka.GKA_BF16 if bf16 else gka.GKA_F32),
                          dtype=torch.uint8, device=device)

    def e2e_step():   # the C-ABI call with host buffers: H2D copies, kernels, D2H copy of the result
        gka.gka_fwd_chunked_host(pin["q"], pin["k"], pin["v"], pin["gate"], pin["lam"], cfg.n_iter, cfg.chunk,
                                 out_pin, None, staging=staging, workspace=ws, device_status=status)

    for _ in range(min(W, 3)):
        e2e_step()
    torch.cuda.synchronize()
    shard.barrier()
    e0, e1 = new_event(), new_event()
    torch.cuda.synchronize()
    e0.record(stream)
    for _ in range(K):
        e2e_step()
    e1.record(stream)
    torch.cuda.synchronize()
    shard.barrier()
    clocks = sampler.stop()
    clocks["sampled_over"] = "the timed steps, a %.1f s back-to-back pass of the same call (%.4f ms per call) and the end-to-end steps" % (SAMPLING_PASS_S, back_ms)
    if clocks.get("sm_mhz"):
        roofline["kernel_ms_x_sm_mhz"] = roofline["kernel_ms"] * clocks["sm_mhz"]
    e2e_ms = shard.max_over_ranks(e0.elapsed_time(e1), device) / K
    e2e_value = tokens_per_step / (e2e_ms * 1e-3)

    work_items = gka.gka_fwd_num_work_items(cfg.B, cfg.T, cfg.heads, cfg.d)
    any_cut = any(gka.gka_fwd_work_range(cfg.B, cfg.T, cfg.heads, cfg.d, work_items, i)[3]
                  for i in range(work_items))
    launches_per_step = 3 if any_cut else 2     # (segment summaries,) state kernel, solve kernel

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": W,
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16" if bf16 else "f32", "data": "synthetic",
        "config": {"workload": cfg.name, "B": cfg.B, "heads": cfg.heads, "T": cfg.T, "d": cfg.d,
                   "chunk": cfg.chunk, "n_iter": cfg.n_iter, "io_dtype": cfg.io_dtype,
                   "l2": "flushed between timed steps (256 MiB write)", "work_items": work_items,
                   "batch_per_gpu": cfg.B},
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "ms_per_step": e2e_ms},
        "gpu_launches": launches_per_step * K,
        "roofline": roofline,
        "clocks": clocks,
        "wall_s_timed_region": wall,
        "input_generation_s": t_gen,
    }
    del staging
    torch.cuda.empty_cache()

    # ---- the paper's setting on the same shapes: 30 iterations, lambda_t = 0.02 ||H_t||_F (Section 4.1 eq. (4))
    if not args.no_extra:
        K2 = min(K, 50)
        dev30 = dict(dev)
        dev30["lam"] = torch.full_like(dev["lam"], 0.02)
        r30 = time_forward(gka, dev30, cfg, 30, gka.GKA_FLAG_ADAPTIVE_LAMBDA, K2, W, peaks, stream, new_event, flush, world, device)
        line["fwd_r30"] = {"metric": METRIC, "value": r30["value"], "unit": UNIT, "ms_per_step": r30["ms_per_step"],
                           "steps": K2, "config": {"workload": "cfg1 shapes at the paper's setting", "B": cfg.B,
                                                   "heads": cfg.heads, "T": cfg.T, "d": cfg.d, "n_iter": 30,
                                                   "lam": "adaptive, a = 0.02", "io_dtype": cfg.io_dtype},
                           "roofline": r30["roofline"], "gpu_launches": launches_per_step * K2}
        del r30, dev30
        # ---- head dimension 64 on configuration 1's shapes (the tensor path's four-k-step instantiation), inputs drawn
        # on the device; no ncu capture of this instantiation exists, so its traffic is not reported
        if world == 1:
            import dataclasses
            cfg64 = dataclasses.replace(cfg, d=64)
            K4 = min(K, 50)
            dev64 = make_fwd_inputs_device(cfg64, device, cfg64.seed)
            r64 = time_forward(gka, dev64, cfg64, cfg64.n_iter, 0, K4, W, peaks, stream, new_event, flush, 1, device)
            r64["roofline"]["traffic"] = None
            line["fwd_d64"] = {"metric": METRIC, "value": r64["value"], "unit": UNIT, "ms_per_step": r64["ms_per_step"],
                               "steps": K4, "config": {"workload": "cfg1 shapes at head dimension 64", "B": cfg64.B,
                                                       "heads": cfg64.heads, "T": cfg64.T, "d": 64, "n_iter": cfg64.n_iter,
                                                       "io_dtype": cfg64.io_dtype, "inputs": "drawn on the device"},
                               "roofline": r64["roofline"], "gpu_launches": launches_per_step * K4}
            del r64, dev64
            torch.cuda.empty_cache()
        # ---- long context (configuration 3), inputs drawn on the device
        if world == 1:
            cfg3 = synth.CONFIGS[3]
            K3 = min(K, 10)
            dev3 = make_fwd_inputs_device(cfg3, device, cfg3.seed)
            r3 = time_forward(gka, dev3, cfg3, cfg3.n_iter, 0, K3, W, peaks, stream, new_event, flush, 1, device)
            line["fwd_long"] = {"metric": METRIC, "value": r3["value"], "unit": UNIT, "ms_per_step": r3["ms_per_step"],
                                "steps": K3, "config": {"workload": cfg3.name, "B": cfg3.B, "heads": cfg3.heads,
                                                        "T": cfg3.T, "d": cfg3.d, "n_iter": cfg3.n_iter,
                                                        "io_dtype": cfg3.io_dtype, "inputs": "drawn on the device"},
                                "roofline": r3["roofline"], "gpu_launches": 3 * K3}
            del r3, dev3
            torch.cuda.empty_cache()

    # ---- decode step (configuration 2), rank-local, reported alongside
    if not args.no_decode:
        line["decode"] = bench_decode(args, device, peaks, stream, new_event, rank, world == 1 and not args.no_cpu_baseline)

    # ---- CPU baseline: the oracle on a bounded sample, rank 0 at N = 1 only
    if world == 1 and not args.no_cpu_baseline:
        line["cpu_baseline"] = cpu_baseline(cfg, host)

    if rank == 0:
        print(json.dumps(line))
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()
    return 0


def bench_decode(args, device, peaks, stream, new_event, rank, with_cpu):
    import torch
    from paper_2511_21016_b200 import gka
    cfg = synth.CONFIGS[2]
    pre, step = make_decode_inputs_device(cfg, device, shard.shard_seed(cfg.seed, rank))
    # the prefix state comes from the product path itself: prefill, then decode
    _, state = gka.gka_fwd_chunked(pre["q"], pre["k"], pre["v"], pre["gate"], pre["lam"], 0, cfg.chunk)
    torch.cuda.synchronize()
    del pre
    torch.cuda.empty_cache()
    out = torch.empty_like(step["v"])
    status = torch.zeros(1, dtype=torch.int32, device=device)
    K, W = args.steps, args.warmup

    def dec(profile=None):
        gka.gka_decode_step(state, step["q"], step["k"], step["v"], step["gate"], step["lam"], cfg.n_iter,
                            out=out, device_status=status, profile_events=profile)

    for _ in range(W):
        dec()
    torch.cuda.synchronize()
    ev = [(new_event(), new_event()) for _ in range(K)]
    torch.cuda.synchronize()
    for i in range(K):
        dec(profile=(ev[i][0].cuda_event, ev[i][1].cuda_event))
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    ms = statistics.mean(a.elapsed_time(b) for a, b in ev)
    st_bytes = cfg.B * cfg.heads * 2 * (2 * cfg.d * cfg.d) * 4          # state read + written
    gbs = st_bytes / (ms * 1e-3) / 1e9
    cpu = None
    if with_cpu:
        # the oracle's decode step on the host cores, on a bounded sample: the first sequences of the same batch
        import oracle
        n_s = 8
        st_host = state[:n_s].cpu().numpy()
        hs = {n: step[n][:n_s].float().cpu().numpy() for n in ("q", "k", "v")}
        g_h, l_h = step["gate"][:n_s].cpu().numpy(), step["lam"][:n_s].cpu().numpy()
        t0 = time.perf_counter()
        oracle.decode(st_host, hs["q"], hs["k"], hs["v"], g_h, l_h, cfg.n_iter)
        dt = time.perf_counter() - t0
        cpu = {"value": n_s / dt, "unit": UNIT, "cores": oracle.max_threads(), "kind": "oracle", "seconds": dt,
               "sample": f"one decode step of {n_s} of the {cfg.B} sequences ({n_s * cfg.heads} (sequence, head) pairs), fp64 oracle"}
    return {
        "metric": "gka_decode_tokens_per_s", "value": cfg.B / (ms * 1e-3), "unit": UNIT,
        "ms_per_step": ms, "head_steps_per_s": cfg.B * cfg.heads / (ms * 1e-3),
        "config": {"workload": cfg.name, "sequences": cfg.B, "heads": cfg.heads, "d": cfg.d,
                   "n_iter": cfg.n_iter, "state": "fp32, 1 GiB, larger than L2; updated in place",
                   "prefix_T": cfg.prefix_T},
        "roofline": {"bound": "hbm", "kernel": "gka decode kernel", "achieved": gbs,
                     "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": gbs / peaks["hbm_gbs"],
                     "peak_source": peaks["source"] + " (copy bandwidth)",
                     "traffic": NCU_TRAFFIC_BYTES["decode"], "bytes_per_launch": st_bytes,
                     # the state is updated in place with no flush between steps, so part of it is served by the L2:
                     # the DRAM-side figure uses the measured traffic instead of the algorithmic bytes
                     "dram_gbs": NCU_TRAFFIC_BYTES["decode"] / (ms * 1e-3) / 1e9,
                     "dram_frac": NCU_TRAFFIC_BYTES["decode"] / (ms * 1e-3) / 1e9 / peaks["hbm_gbs"]},
        "gpu_launches": K,
        **({"cpu_baseline": cpu} if cpu else {}),
    }


def cpu_baseline(cfg, host):
    """The oracle as it stands on the host cores: the whole workload once (tens of core-seconds)."""
    import oracle
    cores = oracle.max_threads()
    t0 = time.perf_counter()
    oracle.fwd(host["q"], host["k"], host["v"], host["gate"], host["lam"], cfg.n_iter)
    dt = time.perf_counter() - t0
    value = cfg.B * cfg.T / dt
    return {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "seconds": dt,
            "sample": f"the whole {cfg.name} workload once ({cfg.B * cfg.heads} (batch, head) pairs x {cfg.T} "
                      f"tokens), fp64 token-by-token oracle, OpenMP over pairs"}


def run_case(argv) -> int:
    """One small case of the hot path a few times (seeded, device-generated inputs, the benchmark's distributions):
    `--case fwd B heads T n_iter reps [flags]`, `--case decode N heads reps`, `--case tokens N heads T reps`.
    For profiling captures: a case of a few hundred MB that ends by itself."""
    import torch
    from paper_2511_21016_b200 import gka
    dev, d = "cuda:0", 128
    gen = torch.Generator(device=dev)
    gen.manual_seed(0)

    def unit(shape):
        x = torch.randn(shape, device=dev, generator=gen)
        return (x / x.norm(dim=-1, keepdim=True)).bfloat16()

    def scalars(shape):
        gate = torch.sigmoid(torch.randn(shape, device=dev, generator=gen) + 2)
        lam = torch.nn.functional.softplus(torch.randn(shape, device=dev, generator=gen)) + 1e-2
        return gate, lam

    kind, n = argv[0], [int(x) for x in argv[1:]]
    if kind == "fwd" and len(n) >= 5:
        B, heads, T, n_iter, reps = n[:5]
        flags = n[5] if len(n) > 5 else 0
        q, k = unit((B, T, heads, d)), unit((B, T, heads, d))
        v = torch.randn(B, T, heads, d, device=dev, generator=gen).bfloat16()
        gate, lam = scalars((B, T, heads))
        if flags & gka.GKA_FLAG_ADAPTIVE_LAMBDA:
            lam = torch.full_like(lam, 0.02)
        ws = gka.alloc_workspace(B, T, heads, d, dev)
        out, state = torch.empty_like(v), torch.empty(B, heads, 2 * d * d, device=dev)
        for _ in range(reps):
            gka.gka_fwd_chunked(q, k, v, gate, lam, n_iter, 64, out=out, state_out=state, workspace=ws, flags=flags)
    elif kind in ("decode", "tokens") and len(n) >= 3:
        N, heads = n[:2]
        T, reps = (n[2], n[3]) if kind == "tokens" else (None, n[2])
        state = torch.randn(N, heads, 2 * d * d, device=dev, generator=gen) * 0.05
        shape = (N, heads) if T is None else (N, T, heads)
        q, k = unit(shape + (d,)), unit(shape + (d,))
        v = torch.randn(shape + (d,), device=dev, generator=gen).bfloat16()
        gate, lam = scalars(shape)
        out = torch.empty_like(v)
        for _ in range(reps):
            if T is None:
                gka.gka_decode_step(state, q, k, v, gate, lam, 10, out=out)
            else:
                gka.gka_decode_tokens(state, q, k, v, gate, lam, 10, out=out)
    else:
        print(run_case.__doc__)
        return 2
    torch.cuda.synchronize()
    print("ok", float(out.float().abs().mean()))
    return 0


def launch_local_ranks(n: int, argv) -> int:
    """`--gpus N` without torchrun: start N local ranks of this script (one per GPU) with the torchrun environment;
    rank 0 prints the line.  No collective on the data path: NCCL serves the barrier and the max over ranks only."""
    port = shard.free_port()
    procs = [subprocess.Popen([sys.executable, os.path.abspath(__file__), *argv], env=shard.rank_env(r, n, port))
             for r in range(n)]
    return max(p.wait() for p in procs)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", type=int, default=1, help="forward configuration to time (1 or 3, 4)")
    ap.add_argument("--no-decode", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-extra", action="store_true", help="skip the fwd_r30, fwd_d64 and fwd_long objects")
    ap.add_argument("--case", nargs="+", help="run one small case a few times instead of the benchmark (see run_case)")
    args = ap.parse_args()
    if args.case:
        return run_case(args.case)
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        return launch_local_ranks(args.gpus, sys.argv[1:])
    if args.warmup < 3 and args.impl == "ours":
        args.warmup = 3
    if args.impl == "reference":
        return run_reference(args)
    return run_ours(args)


if __name__ == "__main__":
    sys.exit(main())
