#!/usr/bin/env python
"""Benchmark of the GKA hot path on B200.

One "step" is one pass of the chunk-wise forward (gate prep, state scan, chunk-wise Frobenius
norms, Chebyshev iterations, output, state carry) over one batch of configuration 1
(B=4, heads=16, T=4096, d=128, chunk=64, n_iter=10, bf16 I/O).  The recurrent decode step
(configuration 2: 256 sequences x 32 heads, fp32 state) is timed in the same run and reported
in the "decode" object of the same JSON line.

    python bench.py --gpus N --steps K --warmup W            # this library
    python bench.py --impl reference --steps K --warmup W    # the fp64 CPU oracle, bounded sample

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
PROFILE_EVERY = 8          # one timed step in this many also times the main kernel alone
L2_FLUSH_BYTES = 256 << 20

# DRAM traffic per launch of the dominant kernels (dram__bytes_read.sum + dram__bytes_write.sum from the
# ncu captures summarised under profiles/).  Both captures ran a quarter/half-size case of the same kernel
# (forward: 2048 of 4096 chunks, 133.71 MB; decode: 2048 of 8192 (sequence, head) pairs, 480.67 MB) and
# are scaled by the units per launch; traffic is proportional to the units in both kernels.
NCU_TRAFFIC_BYTES = {"fwd_main": 2 * 133_384_960, "decode": 4 * 481_565_440}


def fwd_flops(n_chunks: int, n_iter: int, C: int = 64, D: int = 128) -> float:
    """Algorithmic flops of the chunk-wise forward (masked triangles and symmetric halves counted
    once, no credit for padding, split precision or the segment-summary pass)."""
    it = 2 * C * D * D + 2 * D * C * (C + 1)
    s5 = it
    s1 = C * D * (D + 1) + 2 * C * D * D
    s2 = 2 * C * D * D + D * C * (C + 1) + C * C * (C + 1)
    return float(n_chunks) * (n_iter * it + s5 + s1 + s2)


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
    out = torch.empty_like(dev["v"])
    out_pin = torch.empty_like(pin["v"]).pin_memory()
    state_out = torch.empty(cfg.B, cfg.heads, 2 * cfg.d * cfg.d, dtype=torch.float32, device=device)
    ws = gka.alloc_workspace(cfg.B, cfg.T, cfg.heads, cfg.d, device)
    status = torch.zeros(1, dtype=torch.int32, device=device)
    flush = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device=device)
    stream = torch.cuda.current_stream()

    def new_event():
        e = torch.cuda.Event(enable_timing=True)
        e.record(stream)          # creates the underlying cudaEvent_t so that its handle can be passed
        return e

    def fwd(profile=None):
        gka.gka_fwd_chunked(dev["q"], dev["k"], dev["v"], dev["gate"], dev["lam"], cfg.n_iter, cfg.chunk,
                            out=out, state_out=state_out, workspace=ws, device_status=status,
                            profile_events=profile)

    K, W = args.steps, args.warmup
    sampler = ClockSampler(local_rank)
    sampler.start()
    for _ in range(W):
        flush.zero_()
        fwd()
    torch.cuda.synchronize()

    # ---- device-resident timing: K steps, L2 flushed between steps, CUDA events on the launch stream
    ev = [(new_event(), new_event(), new_event(), new_event()) for _ in range(K)]
    torch.cuda.synchronize()
    shard.barrier()
    torch.cuda.synchronize()
    wall0 = time.perf_counter()
    # Every PROFILE_EVERY-th step also brackets the main kernel alone with the library's profile events (the roofline's
    # duration).  Those events sit between the summary kernel and the main kernel and so keep the main kernel from
    # starting its prologue under the summary kernel's tail; the other steps run exactly as a user's call does.
    for i in range(K):
        flush.zero_()
        ev[i][0].record(stream)
        fwd(profile=(ev[i][2].cuda_event, ev[i][3].cuda_event) if i % PROFILE_EVERY == 0 else None)
        ev[i][1].record(stream)
    torch.cuda.synchronize()
    shard.barrier()
    wall = time.perf_counter() - wall0
    step_ms = [a.elapsed_time(b) for a, b, _, _ in ev]
    main_ms = [c.elapsed_time(d) for i, (_, _, c, d) in enumerate(ev) if i % PROFILE_EVERY == 0]
    total_ms = shard.max_over_ranks(sum(step_ms), device)
    ms_per_step = total_ms / K
    tokens_per_step = cfg.B * cfg.T * world
    value = tokens_per_step / (ms_per_step * 1e-3)
    assert int(status.item()) == 0, "a device-side bounded wait timed out"

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
    e2e_ms = shard.max_over_ranks(e0.elapsed_time(e1), device) / K
    e2e_value = tokens_per_step / (e2e_ms * 1e-3)

    # ---- roofline of the dominant kernel (main forward kernel, timed alone by the library's events)
    n_chunks = cfg.B * cfg.heads * (cfg.T // cfg.chunk)
    flops = fwd_flops(n_chunks, cfg.n_iter, cfg.chunk, cfg.d)
    main_avg_ms = statistics.mean(main_ms)
    achieved_tf = flops / (main_avg_ms * 1e-3) / 1e12
    roofline = {"bound": "tensor", "kernel": "gka_fwd main kernel", "achieved": achieved_tf,
                "peak": peaks["bf16_tflops"], "unit": "TFLOP/s", "frac": achieved_tf / peaks["bf16_tflops"],
                "peak_source": peaks["source"] + " (burst cuBLAS bf16)",
                "traffic": NCU_TRAFFIC_BYTES["fwd_main"], "flops_per_launch": flops,
                "kernel_ms": main_avg_ms, "kernel_launches_timed": len(main_ms), "whole_call_frac": flops / (ms_per_step * 1e-3) / 1e12 / peaks["bf16_tflops"],
                "frac_of_nominal_2250": achieved_tf / 2250.0}

    work_items = gka.gka_fwd_num_work_items(cfg.B, cfg.T, cfg.heads, cfg.d)
    any_cut = any(gka.gka_fwd_work_range(cfg.B, cfg.T, cfg.heads, cfg.d, work_items, i)[3]
                  for i in range(work_items))
    launches_per_step = 2 if any_cut else 1     # segment summaries + main kernel, or the main kernel alone

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

    # ---- decode step (configuration 2), rank-local, reported alongside
    if not args.no_decode:
        line["decode"] = bench_decode(args, device, peaks, stream, new_event, rank)

    # ---- CPU baseline: the oracle on a bounded sample, rank 0 at N = 1 only
    if world == 1 and not args.no_cpu_baseline:
        line["cpu_baseline"] = cpu_baseline(cfg, host)

    if rank == 0:
        print(json.dumps(line))
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()
    return 0


def bench_decode(args, device, peaks, stream, new_event, rank):
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
    return {
        "metric": "gka_decode_tokens_per_s", "value": cfg.B / (ms * 1e-3), "unit": UNIT,
        "ms_per_step": ms, "head_steps_per_s": cfg.B * cfg.heads / (ms * 1e-3),
        "config": {"workload": cfg.name, "sequences": cfg.B, "heads": cfg.heads, "d": cfg.d,
                   "n_iter": cfg.n_iter, "state": "fp32, 1 GiB, larger than L2; updated in place",
                   "prefix_T": cfg.prefix_T},
        "roofline": {"bound": "hbm", "kernel": "gka decode kernel", "achieved": gbs,
                     "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": gbs / peaks["hbm_gbs"],
                     "peak_source": peaks["source"] + " (copy bandwidth)",
                     "traffic": NCU_TRAFFIC_BYTES["decode"], "bytes_per_launch": st_bytes},
        "gpu_launches": K,
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


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", type=int, default=1, help="forward configuration to time (1 or 3, 4)")
    ap.add_argument("--no-decode", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    if args.warmup < 3 and args.impl == "ours":
        args.warmup = 3
    if args.impl == "reference":
        return run_reference(args)
    return run_ours(args)


if __name__ == "__main__":
    sys.exit(main())
