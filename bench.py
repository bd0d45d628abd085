#!/usr/bin/env python
"""Benchmark of the zero-expert MoE layer forward (one step = one zeda_moe_forward call over one
batch of synthetic tokens: router, top-K, compaction, grouped SwiGLU experts, combine).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload prefill|decode|net|glm|sweep25|stack|...]
    python bench.py --impl reference ...      # the CPU oracle, timed on the host cores

Prints ONE JSON line.  The default workload is the prefill batch (T = 8192) of the Qwen3-30B-A3B-shaped
layer; its line also carries, as nested objects, the decode batch (T = 64) on the same layer, the
static top-K layer (Z = 0) and the NET layer (Z = 0, K/2) run through the same kernels.  With N > 1 (launched by torch.distributed.run) every rank is a data-parallel
replica of the layer with its own token batch; there is no collective on the data path.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np
import torch

from paper_2605_18643_b200 import flops, inputs

METRIC = "MoE-layer tokens/s"
UNIT = "tokens/s"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
L2_NOTE = "256 MiB written, then 256 MiB read, between timed steps (outside the event pairs)"
# sources of the dominant kernel (expert GEMM1 + SwiGLU): the ncu traffic figures are only valid for
# the build they were captured on
GEMM_SOURCES = ("expert_pair.cu", "tc_common.cuh")


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            d = json.load(f)
        return d, "measured"
    return dict(FALLBACK_PEAKS), "fallback"


def kernel_source_id():
    """Short hash of the expert kernels' sources: ties an ncu traffic figure to the build it was taken on."""
    import hashlib
    h = hashlib.sha256()
    for f in GEMM_SOURCES:
        with open(os.path.join(ROOT, "paper_2605_18643_b200", "csrc", f), "rb") as fh:
            h.update(fh.read())
    return h.hexdigest()[:12]


def ncu_traffic_bytes(workload: str):
    """dram__bytes_read.sum + dram__bytes_write.sum of one launch of the dominant kernel, from the
    line `<workload> <bytes> <source id>` of profiles/gemm1_dram_traffic.txt (written beside the
    ncu summary it comes from).  None when there is no line for this workload or the kernel's
    sources have changed since the capture."""
    p = os.path.join(ROOT, "profiles", "gemm1_dram_traffic.txt")
    if not os.path.exists(p):
        return None
    sid = kernel_source_id()
    for line in open(p):
        f = line.split()
        if len(f) >= 3 and not line.startswith("#") and f[0] == workload and f[2] == sid:
            return float(f[1])
    return None


GLM_SHAPE = dict(d=2048, He=1536, E=64, Z=32, K=4)   # N, K, N_Z from the paper's table of adapted models; d, H_e free


def make_workload(name: str):
    if name == "decode":
        return inputs.decode()
    if name == "prefill":
        return inputs.prefill()
    if name == "tiny":
        return inputs.tiny()
    if name == "hot4":     # 32,768 pairs on four experts: full tiles only, weights resident in L2 (kernel ceiling)
        return inputs.make_layer("hot4", T=8192, d=2048, He=768, E=4, Z=0, K=4, zero_fraction=None)
    if name == "net":      # the paper's iso-FLOP static baseline: no zero experts, K/2 slots
        return net_reference(inputs.prefill())
    if name == "glm":      # second adapted model's expert counts at the prefill size
        return inputs.make_layer("glm", T=8192, zero_fraction=0.5, zipf_s=1.1, **GLM_SHAPE)
    if name.startswith("sweep"):
        return inputs.sweep_point(int(name[5:]) / 100.0)
    if name.startswith("prefill_f"):   # zero-fraction sweep at the prefill size
        f = int(name[9:]) / 100.0
        return inputs.prefill(Z=0, zero_fraction=None) if f == 0 else inputs.prefill(zero_fraction=f)
    raise SystemExit("unknown workload " + name)


def net_reference(wl):
    """NET (Section 3.1): the static layer with half the slots, K/2, and no zero experts, on the same
    x, expert weights, normal router rows and normal-expert bias."""
    import dataclasses
    st = inputs.static_reference(wl)
    return dataclasses.replace(st, name=wl.name + "_net", K=max(1, wl.K // 2))


def workload_config(wl, name, P, U, world):
    """The `config` object of the JSON line; identical for both arms (P and U follow from the routing)."""
    return {"workload": name, "T": wl.T, "d": wl.d, "d_expert": wl.He, "n_real": wl.E, "n_zero": wl.Z,
            "top_k": wl.K, "zero_slot_fraction": round(wl.zero_fraction, 4), "seed": 0, "P": int(P), "U": int(U),
            "l2": L2_NOTE, "parallelism": "dp%d replicas, no collective" % world}


class ClockSampler:
    """nvidia-smi clock / throttle-reason samples taken while the timed region runs."""

    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.path = None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(
                ["nvidia-smi", "--id=%d" % self.index, "--query-gpu=" + self.Q, "--format=csv,noheader,nounits",
                 "-lms", "20"], stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        try:
            for line in open(self.path):
                f = [v.strip() for v in line.split(",")]
                if len(f) < 7:
                    continue
                try:
                    sm.append(float(f[0]))
                    mx.append(float(f[1]))
                except ValueError:
                    continue
                for n, v in zip(names, f[3:7]):
                    if v.lower().startswith("active"):
                        reasons.add(n)
            os.unlink(self.path)
        except Exception:
            pass
        if sm:
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(mx), samples=len(sm))
        out["reasons"] = sorted(reasons)
        return out


def oracle_tokens_per_s(wl, sample_tokens: int, seed: int = 0, min_seconds: float = 0.0, max_passes: int = 1):
    """Times the CPU oracle, as it stands, on a bounded token sample of the workload."""
    import oracle
    n = min(sample_tokens, wl.T)
    ids = None if n == wl.T else np.sort(np.random.default_rng(seed).choice(wl.T, n, replace=False)).astype(np.int32)
    bias = None if wl.router_bias is None else wl.router_bias.numpy()
    args = (inputs.bits(wl.x), wl.router_w.numpy(), bias, inputs.bits(wl.w_gate_up), inputs.bits(wl.w_down),
            wl.E, wl.Z, wl.K)
    passes, dt = 0, 0.0
    while passes < max_passes and (passes == 0 or dt < min_seconds):
        t0 = time.perf_counter()
        oracle.forward(*args, token_ids=ids)
        dt += time.perf_counter() - t0
        passes += 1
    what = "%d of %d tokens, seeded sample" % (n, wl.T) if ids is not None else "all %d tokens" % wl.T
    return n * passes / dt, dt, oracle.num_threads(), "%s, %d passes" % (what, passes)


def oracle_pairs(wl):
    """P and U of the workload from the oracle's routing of every token (no expert math)."""
    import oracle
    bias = None if wl.router_bias is None else wl.router_bias.numpy()
    _, idx, _ = oracle.forward(inputs.bits(wl.x), wl.router_w.numpy(), bias, inputs.bits(wl.w_gate_up),
                               inputs.bits(wl.w_down), wl.E, wl.Z, wl.K, want_y=False)
    counts, _, _, P = oracle.compact(idx, wl.E)
    return P, int((counts > 0).sum())


def run_reference(args):
    """--impl reference: the CPU oracle on the host cores, same metric, workload and config.  Each
    step is the oracle, as it stands, on a bounded seeded sample of the workload's tokens."""
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if rank != 0:
        return
    wl = make_workload(args.workload)
    P, U = oracle_pairs(wl)
    sample = 64 if wl.T > 64 else wl.T
    for _ in range(args.warmup):
        oracle_tokens_per_s(wl, sample)
    total, info = 0.0, None
    for _ in range(args.steps):
        v, dt, cores, desc = oracle_tokens_per_s(wl, sample)
        total += dt
        info = (cores, desc)
    value = sample * args.steps / total
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 * total / args.steps, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": workload_config(wl, args.workload, P, U, world),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": info[0], "kind": "oracle",
                         "sample": "each step = the oracle on %s" % info[1]},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def max_over_ranks(values, dist, device):
    """Element-wise maximum of per-rank timings over all ranks (every rank gets the result); the
    identity without a process group.  The only collective of a multi-GPU run: replicas exchange
    no data."""
    if dist is None:
        return [float(v) for v in values]
    t = torch.tensor([float(v) for v in values], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t]


def job_tokens_per_s(world: int, tokens_per_rank: int, ms_per_step: float) -> float:
    """Whole-job throughput of `world` replicas that each push tokens_per_rank tokens per step."""
    return world * tokens_per_rank / (ms_per_step * 1e-3)


def rank_tokens(wl, rank: int):
    """Token batch of data-parallel replica `rank`: the workload's own batch on rank 0, a fresh
    seeded batch (same layer, same tie margin) on every other rank."""
    return wl.x if rank == 0 else inputs.replica_tokens(wl, rank)


class L2Flush:
    """Evicts the layer's data from L2 between timed steps: writes a 256 MiB buffer (twice the
    126 MB L2), then reads a second one so that the lines left behind are clean.  (Dirty lines of
    the written buffer would otherwise be written back during the timed step, which charges the
    step with about 126 MB of DRAM writes that belong to the flush.)"""

    def __init__(self, dev, nbytes=256 << 20):
        self.w = torch.empty(nbytes, dtype=torch.uint8, device=dev)
        self.r = torch.zeros(nbytes // 4, dtype=torch.float32, device=dev)
        self.sink = None

    def zero_(self):
        self.w.zero_()
        self.sink = self.r.sum()


def time_forward(m, x, y, steps, warmup, flush, dist_barrier):
    """Per-step CUDA-event timing with an L2 flush (outside the event pairs) between steps."""
    for _ in range(warmup):
        flush.zero_()
        m.forward(x, y)
    starts = [torch.cuda.Event(enable_timing=True) for _ in range(steps)]
    ends = [torch.cuda.Event(enable_timing=True) for _ in range(steps)]
    dist_barrier()
    torch.cuda.synchronize()
    for i in range(steps):
        flush.zero_()
        starts[i].record()
        m.forward(x, y)
        ends[i].record()
    torch.cuda.synchronize()
    dist_barrier()
    per = [s.elapsed_time(e) for s, e in zip(starts, ends)]
    return sum(per), per


def run_stack(args, peaks, peaks_kind, dev, world, rank, barrier, dist):
    """--workload stack: a pass through --layers stacked MoE blocks (attention excluded) with the
    residual + RMSNorm glue between them.  One step = one pass of T tokens through every layer."""
    from paper_2605_18643_b200 import zeda
    layers, r0 = inputs.stack_layers(args.layers, T=args.stack_tokens)
    T, d, He, E, Z, K = (layers[0].T, layers[0].d, layers[0].He, layers[0].E, layers[0].Z, layers[0].K)
    mods = []
    for l, wl in enumerate(layers):
        wgu, wd = inputs.device_expert_weights(E, He, d, 100 + l, dev)
        bias = None if wl.router_bias is None else wl.router_bias.to(dev)
        mods.append(zeda.ZedaMoE(wl.router_w.to(dev), bias, wgu, wd, E, Z, K, T))
    if rank > 0:
        r0 = inputs.replica_tokens(layers[0], rank)
    r_init = r0.to(dev)
    r = r_init.clone()
    hs = [torch.empty_like(r), torch.empty_like(r)]
    y_last = torch.empty_like(r)
    fused = args.stack_glue == "fused"

    def one_pass():
        r.copy_(r_init)
        if fused:
            # the glue of layers 1.. rides in the last pass of the layer before it
            zeda.residual_rmsnorm(r, None, hs[0])
            for l, m in enumerate(mods[:-1]):
                m.forward_residual(hs[l & 1], r, hs[(l + 1) & 1])
            return mods[-1].forward(hs[(len(mods) - 1) & 1], y_last)
        y = None
        for l, m in enumerate(mods):
            zeda.residual_rmsnorm(r, y, hs[0])
            y = m.forward(hs[0], y_last if l & 1 else hs[1])
        return y

    clocks = ClockSampler(dev.index or 0)
    clocks.start()
    for _ in range(args.warmup):
        one_pass()
    starts = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps)]
    ends = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps)]
    barrier()
    torch.cuda.synchronize()
    for i in range(args.steps):
        starts[i].record()
        one_pass()
        ends[i].record()
    torch.cuda.synchronize()
    barrier()
    total_ms = sum(a.elapsed_time(b) for a, b in zip(starts, ends))
    counters = [m.last_counters() for m in mods]
    # stage events, one more pass
    for m in mods:
        m.set_profiling(True)
    one_pass()
    torch.cuda.synchronize()
    stage = np.zeros(5)
    for m in mods:
        stage += np.array(m.stage_ms())
        m.set_profiling(False)
    # end to end: host residual in, host result out
    r_pin = r0.pin_memory()
    out_pin = torch.empty_like(r_pin).pin_memory()
    e2e_s = 0.0
    for i in range(args.warmup + args.steps):
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        r_init.copy_(r_pin, non_blocking=True)
        y = one_pass()
        out_pin.copy_(y, non_blocking=True)
        torch.cuda.synchronize()
        if i >= args.warmup:
            e2e_s += time.perf_counter() - t0
    barrier()
    clock_info = clocks.stop()
    total_ms, e2e_s = max_over_ranks([total_ms, e2e_s], dist, dev)
    if rank == 0:
        ms_per_step = total_ms / args.steps
        hbm = peaks["hbm_gbs"] * 1e9
        burst = peaks["bf16_tflops"]
        sustained = peaks.get("bf16_tflops_sustained", burst)
        t_roof = t_roof_s = 0.0
        g1_bytes = g1_flops = 0
        for (P, U, _, _) in counters:
            t_roof += flops.layer_roofline_seconds(T, d, He, E + Z, P, U, burst * 1e12, hbm)[0]
            t_roof_s += flops.layer_roofline_seconds(T, d, He, E + Z, P, U, sustained * 1e12, hbm)[0]
            g1_bytes += U * 2 * He * d * 2 + T * d * 2 + P * He * 2
            g1_flops += 4 * P * d * He
        g1_s = stage[2] * 1e-3
        if g1_bytes / hbm >= g1_flops / (sustained * 1e12):
            roof = {"bound": "hbm", "achieved": g1_bytes / g1_s / 1e9, "peak": peaks["hbm_gbs"], "unit": "GB/s"}
        else:
            roof = {"bound": "tensor", "achieved": g1_flops / g1_s / 1e12, "peak": sustained, "unit": "TFLOP/s",
                    "peak_kind": "sustained (kernel timed inside the step)", "peak_burst": burst}
        roof["frac"] = roof["achieved"] / roof["peak"]
        roof.update(traffic=None, kernel="expert GEMM1 + SwiGLU, summed over the layers", peak_source=peaks_kind,
                    algorithmic_bytes=g1_bytes, algorithmic_flops=g1_flops, kernel_ms=stage[2])
        Ps = [c[0] for c in counters]
        line = {
            "metric": METRIC, "value": job_tokens_per_s(world, T, ms_per_step), "unit": UNIT, "n_gpus": world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": "stack", "layers": len(mods), "glue": args.stack_glue, "T": T, "d": d, "d_expert": He, "n_real": E,
                       "n_zero": Z, "top_k": K, "seed": 0, "pairs_per_layer_min_max": [min(Ps), max(Ps)],
                       "zero_slot_fraction_mean": round(1.0 - sum(Ps) / (len(Ps) * T * K), 4),
                       "weights_gb": round(len(mods) * E * 3 * d * He * 2 / 1e9, 2),
                       "l2": "inputs larger than L2: every layer streams its own 1.2 GB of expert weights",
                       "parallelism": "dp%d replicas, no collective" % world},
            "clocks": clock_info,
            "e2e": {"value": world * T * args.steps / e2e_s, "unit": UNIT, "h2d_bytes_per_step": T * d * 2,
                    "d2h_bytes_per_step": T * d * 2, "ms_per_step": 1e3 * e2e_s / args.steps},
            "gpu_launches": (sum(c[3] for c in counters) + (1 if fused else len(mods))) * args.steps,
            "roofline": roof,
            "layer_roofline": {"t_roof_us": t_roof * 1e6, "frac": t_roof / (ms_per_step * 1e-3),
                               "t_roof_us_sustained": t_roof_s * 1e6,
                               "frac_sustained": t_roof_s / (ms_per_step * 1e-3), "peak_source": peaks_kind},
            "stage_ms": {n: float(v) for n, v in zip(["router", "sort", "gemm1", "gemm2", "combine"], stage)},
        }
        print(json.dumps(line))
    for m in mods:
        m.close()


def run_ep(args, peaks, peaks_kind, dev, world, rank, barrier, dist):
    """--workload ep: the prefill layer with its experts partitioned over the N ranks (expert parallel)
    and the tokens data-parallel, T tokens per rank.  One step = dispatch (route, drop zero slots, pack),
    all-to-all of the surviving rows, local experts, all-to-all back, combine.  With N = 1 the exchange
    is a loopback."""
    from paper_2605_18643_b200 import ep, zeda
    wl = inputs.prefill()
    G = world
    if wl.E % G:
        raise SystemExit("--workload ep needs a rank count that divides %d experts" % wl.E)
    n_local = wl.E // G
    x_cpu = rank_tokens(wl, rank)
    wgu = wl.w_gate_up[rank * n_local:(rank + 1) * n_local].contiguous().to(dev)
    wd = wl.w_down[rank * n_local:(rank + 1) * n_local].contiguous().to(dev)
    m = zeda.ZedaMoE(wl.router_w.to(dev), wl.router_bias.to(dev), wgu, wd, wl.E, wl.Z, wl.K, wl.T, ep_size=G,
                     ep_rank=rank, max_recv_pairs=G * wl.T * wl.K)
    layer = ep.ExpertParallelMoE(m, ep.TorchDistExchange() if dist is not None else ep.LoopbackExchange())
    x = x_cpu.to(dev)
    y = torch.empty_like(x)
    flush = L2Flush(dev)
    clocks = ClockSampler(dev.index or 0)
    clocks.start()
    for _ in range(args.warmup):
        flush.zero_()
        layer.forward(x, y)
    starts = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps)]
    ends = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps)]
    barrier()
    torch.cuda.synchronize()
    for i in range(args.steps):
        flush.zero_()
        starts[i].record()
        layer.forward(x, y)
        ends[i].record()
    torch.cuda.synchronize()
    barrier()
    total_ms = sum(a.elapsed_time(b) for a, b in zip(starts, ends))
    per_phase = []
    layer.forward(x, y, launches=per_phase)            # one more step, untimed: kernels per phase
    launches = sum(per_phase)
    R, U_local, _, _ = m.last_counters()               # pair rows this rank's experts processed, its active experts
    x_pin = x_cpu.pin_memory()
    y_pin = torch.empty_like(x_pin).pin_memory()
    e2e_s = 0.0
    for i in range(args.warmup + args.steps):
        flush.zero_()
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        x.copy_(x_pin, non_blocking=True)
        layer.forward(x, y)
        y_pin.copy_(y, non_blocking=True)
        torch.cuda.synchronize()
        if i >= args.warmup:
            e2e_s += time.perf_counter() - t0
    barrier()
    clock_info = clocks.stop()
    total_ms, e2e_s, rows_max = max_over_ranks([total_ms, e2e_s, float(R)], dist, dev)
    if rank == 0:
        ms = total_ms / args.steps
        line = {
            "metric": METRIC, "value": job_tokens_per_s(world, wl.T, ms), "unit": UNIT, "n_gpus": world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": "ep", "T_per_rank": wl.T, "d": wl.d, "d_expert": wl.He, "n_real": wl.E, "n_zero": wl.Z,
                       "top_k": wl.K, "zero_slot_fraction": round(wl.zero_fraction, 4), "seed": 0,
                       "pair_rows_rank0": int(R), "pair_rows_max_over_ranks": int(rows_max), "active_experts_rank0": int(U_local),
                       "l2": L2_NOTE, "parallelism": "ep%d: experts over %d ranks, tokens data-parallel, zero slots dropped "
                                                     "before the all-to-all" % (G, G)},
            "clocks": clock_info,
            "e2e": {"value": world * wl.T * args.steps / e2e_s, "unit": UNIT, "h2d_bytes_per_step": wl.T * wl.d * 2,
                    "d2h_bytes_per_step": wl.T * wl.d * 2, "ms_per_step": 1e3 * e2e_s / args.steps},
            "gpu_launches": launches * args.steps,
            "roofline": None,
        }
        print(json.dumps(line))
    m.close()


class DeviceWeights:
    """Device copies of expert weights, shared between the handles of one run (the zero-expert layer,
    its static reference, the decode batch on the same layer): 1.2 GB is copied once."""

    def __init__(self, dev):
        self.dev = dev
        self.cache = {}

    def handle(self, zeda, wl, max_tokens=None):
        key = (wl.w_gate_up.data_ptr(), wl.w_down.data_ptr())
        if key not in self.cache:
            self.cache[key] = (wl.w_gate_up.to(self.dev).contiguous(), wl.w_down.to(self.dev).contiguous())
        wgu, wd = self.cache[key]
        bias = None if wl.router_bias is None else wl.router_bias.to(self.dev).contiguous()
        return zeda.ZedaMoE(wl.router_w.to(self.dev).contiguous(), bias, wgu, wd, wl.E, wl.Z, wl.K, max_tokens or wl.T)


def gemm1_roofline(wl, P, U, kernel_ms, peaks, peaks_kind, workload):
    """Roofline object of the dominant kernel (expert GEMM1 + SwiGLU).  Algorithmic bytes: gate and up
    weights of the U active experts + the x rows read + the intermediate written; algorithmic FLOPs:
    4 d H_e per pair.  The kernel is timed by stage events inside the step, back to back with the other
    kernels, so the tensor peak it is held against is the sustained one (burst beside it)."""
    hbm = peaks["hbm_gbs"] * 1e9
    burst = peaks["bf16_tflops"]
    sustained = peaks.get("bf16_tflops_sustained", burst)
    g1_bytes = U * 2 * wl.He * wl.d * 2 + wl.T * wl.d * 2 + P * wl.He * 2
    g1_flops = 4 * P * wl.d * wl.He
    g1_s = kernel_ms * 1e-3
    if g1_bytes / hbm >= g1_flops / (sustained * 1e12):
        roof = {"bound": "hbm", "achieved": g1_bytes / g1_s / 1e9, "peak": peaks["hbm_gbs"], "unit": "GB/s"}
    else:
        roof = {"bound": "tensor", "achieved": g1_flops / g1_s / 1e12, "peak": sustained, "unit": "TFLOP/s",
                "peak_kind": "sustained (kernel timed inside the step)", "peak_burst": burst,
                "frac_of_burst": g1_flops / g1_s / 1e12 / burst}
    roof["frac"] = roof["achieved"] / roof["peak"]
    roof.update(traffic=ncu_traffic_bytes(workload), kernel="expert GEMM1 + SwiGLU (expert_gemm_pair_kernel<1,..>)",
                peak_source=peaks_kind, algorithmic_bytes=g1_bytes, algorithmic_flops=g1_flops, kernel_ms=kernel_ms)
    return roof


def layer_roofline(wl, P, U, ms_per_step, peaks, peaks_kind):
    hbm = peaks["hbm_gbs"] * 1e9
    burst = peaks["bf16_tflops"]
    sustained = peaks.get("bf16_tflops_sustained", burst)
    n_cand = wl.E + wl.Z
    t_roof, t_flop, t_mem = flops.layer_roofline_seconds(wl.T, wl.d, wl.He, n_cand, P, U, burst * 1e12, hbm)
    t_roof_s, t_flop_s, _ = flops.layer_roofline_seconds(wl.T, wl.d, wl.He, n_cand, P, U, sustained * 1e12, hbm)
    return {"t_roof_us": t_roof * 1e6, "t_flop_us": t_flop * 1e6, "t_hbm_us": t_mem * 1e6,
            "frac": t_roof / (ms_per_step * 1e-3), "peak_source": peaks_kind,
            "t_flop_us_sustained": t_flop_s * 1e6, "t_roof_us_sustained": t_roof_s * 1e6,
            "frac_sustained": t_roof_s / (ms_per_step * 1e-3)}


def measure_layer(zeda, weights, wl, x_cpu, args, flush, barrier, dist, dev, e2e=True, static=True, net=False):
    """Times one workload: the step itself, its stages, the host-buffer entry point, and the same
    kernels on the static (Z = 0) and NET (Z = 0, K/2) reference layers.  Every rank runs this; the
    timings returned are maxima over the ranks."""
    m = weights.handle(zeda, wl)
    x = x_cpu.to(dev)
    y = torch.empty_like(x)
    total_ms, _ = time_forward(m, x, y, args.steps, args.warmup, flush, barrier)
    P, U, zero_slots, launches = m.last_counters()
    # the same steps again with stage events on the stream: duration of every stage
    m.set_profiling(True)
    stage = np.zeros(5)
    for i in range(args.steps):
        flush.zero_()
        m.forward(x, y)
        stage += np.array(m.stage_ms())
    stage /= args.steps
    m.set_profiling(False)
    e2e_s = 0.0
    if e2e:
        # end to end through the host-buffer entry point: H2D of x and D2H of y inside the timed region
        x_pin = x_cpu.pin_memory()
        y_pin = torch.empty_like(x_pin).pin_memory()
        for _ in range(args.warmup):
            flush.zero_()
            m.forward_host(x_pin, y_pin)
        barrier()
        torch.cuda.synchronize()
        for i in range(args.steps):
            flush.zero_()
            torch.cuda.synchronize()
            t0 = time.perf_counter()
            m.forward_host(x_pin, y_pin)
            e2e_s += time.perf_counter() - t0
        barrier()
    m.close()
    refs = {}
    if static and wl.Z > 0:
        todo = [("static_reference", inputs.static_reference(wl))]
        if net:
            todo.append(("net_reference", net_reference(wl)))
        for key, ws in todo:
            ms_ = weights.handle(zeda, ws)
            st_total, _ = time_forward(ms_, x, y, args.steps, args.warmup, flush, barrier)
            Ps, Us, _, _ = ms_.last_counters()
            ms_.close()
            refs[key] = {"ms_per_step": st_total / args.steps, "P": Ps, "U": Us, "top_k": ws.K}
    keys = sorted(refs)
    red = max_over_ranks([total_ms, e2e_s] + [refs[k]["ms_per_step"] for k in keys], dist, dev)
    for k, v in zip(keys, red[2:]):
        refs[k]["ms_per_step"] = v
    return {"ms_per_step": red[0] / args.steps, "e2e_s": red[1], "P": P, "U": U, "launches": launches,
            "stage": stage, "refs": refs}


def layer_report(wl, name, r, world, steps, peaks, peaks_kind):
    """The per-workload part of the JSON line from measure_layer's result."""
    ms = r["ms_per_step"]
    out = {
        "value": job_tokens_per_s(world, wl.T, ms), "ms_per_step": ms,
        "roofline": gemm1_roofline(wl, r["P"], r["U"], float(r["stage"][2]), peaks, peaks_kind, name),
        "layer_roofline": layer_roofline(wl, r["P"], r["U"], ms, peaks, peaks_kind),
        "stage_ms": {n: float(v) for n, v in zip(["router", "sort", "gemm1", "gemm2", "combine"], r["stage"])},
    }
    for key, ref in r["refs"].items():
        out[key] = dict(ref, value=world * wl.T / (ref["ms_per_step"] * 1e-3),
                        speedup_vs_this_reference=ref["ms_per_step"] / ms)
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="prefill",
                    help="prefill (default; carries the decode batch on the same layer as a nested object), decode, "
                         "tiny, net, glm, hot4, sweepNN, prefill_fNN, stack, ep (experts over the ranks)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-static", action="store_true")
    ap.add_argument("--no-decode", action="store_true", help="prefill only: skip the nested decode measurement")
    ap.add_argument("--no-sweep", action="store_true", help="prefill only: skip the nested zero-fraction sweep")
    ap.add_argument("--layers", type=int, default=48, help="layers of --workload stack")
    ap.add_argument("--stack-tokens", type=int, default=4096, help="tokens per pass of --workload stack")
    ap.add_argument("--stack-glue", choices=["fused", "separate"], default="fused",
                    help="--workload stack: residual + RMSNorm fused into each layer's combine pass, or its own kernel")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
        return
    args.warmup = max(args.warmup, 3)

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the layer has no CPU path")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group(backend="nccl", device_id=dev)

    def barrier():
        if dist is not None:
            dist.barrier()

    from paper_2605_18643_b200 import zeda  # raises if libzeda.so is missing

    peaks, peaks_kind = load_peaks()
    if args.workload in ("stack", "ep"):
        (run_stack if args.workload == "stack" else run_ep)(args, peaks, peaks_kind, dev, world, rank, barrier, dist)
        if dist is not None:
            dist.destroy_process_group()
        return
    wl = make_workload(args.workload)
    weights = DeviceWeights(dev)
    flush = L2Flush(dev)
    clocks = ClockSampler(local_rank)
    clocks.start()
    headline = args.workload == "prefill"
    r = measure_layer(zeda, weights, wl, rank_tokens(wl, rank), args, flush, barrier, dist, dev,
                      static=not args.no_static, net=headline)
    clock_info = clocks.stop()
    nested = None
    if headline and not args.no_decode:
        # the decode batch on the same layer shape (same expert weights), timed in the same run
        wd_ = inputs.decode()
        clocks_d = ClockSampler(local_rank)
        clocks_d.start()
        rd = measure_layer(zeda, weights, wd_, rank_tokens(wd_, rank), args, flush, barrier, dist, dev,
                           e2e=False, static=not args.no_static)
        nested = (wd_, rd, clocks_d.stop())

    sweep = None
    if headline and not args.no_sweep and not args.no_static:
        # layer time against the zero-routed share at the prefill size: 0 (the static layer) and the
        # headline's own share are measured above; two more points with the same x and expert weights
        sweep = {}
        for f in (0.25, 0.75):
            wf = inputs.prefill(zero_fraction=f)
            rf = measure_layer(zeda, weights, wf, rank_tokens(wf, rank), args, flush, barrier, dist, dev, e2e=False, static=False)
            sweep[f] = (wf, rf)

    if rank == 0:
        rep = layer_report(wl, args.workload, r, world, args.steps, peaks, peaks_kind)
        line = {
            "metric": METRIC, "value": rep.pop("value"), "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": rep.pop("ms_per_step"), "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": workload_config(wl, args.workload, r["P"], r["U"], world),
            "clocks": clock_info,
            "e2e": {"value": world * wl.T * args.steps / r["e2e_s"], "unit": UNIT,
                    "h2d_bytes_per_step": wl.T * wl.d * 2, "d2h_bytes_per_step": wl.T * wl.d * 2,
                    "ms_per_step": 1e3 * r["e2e_s"] / args.steps},
            "gpu_launches": r["launches"] * args.steps,
        }
        line.update(rep)
        if nested:
            wd_, rd, clk = nested
            dec = layer_report(wd_, "decode", rd, world, args.steps, peaks, peaks_kind)
            dec["config"] = workload_config(wd_, "decode", rd["P"], rd["U"], world)
            dec["clocks"] = clk
            dec["gpu_launches"] = rd["launches"] * args.steps
            line["decode"] = dec
        if sweep:
            # time relative to the static layer next to the share of slots that still reach an expert
            t0 = line["static_reference"]["ms_per_step"]
            pts = [{"zero_slot_fraction": 0.0, "P": line["static_reference"]["P"], "ms_per_step": t0}]
            for f, (wf, rf) in sorted(list(sweep.items()) + [(wl.zero_fraction, (wl, r))], key=lambda kv: kv[0]):
                pts.append({"zero_slot_fraction": round(wf.zero_fraction, 4), "P": rf["P"], "U": rf["U"],
                            "ms_per_step": rf["ms_per_step"]})
            for p_ in pts:
                p_["time_vs_static"] = p_["ms_per_step"] / t0
                p_["real_slot_share"] = 1.0 - p_["zero_slot_fraction"]
            line["zero_fraction_sweep"] = pts
        if not args.no_cpu_baseline:
            v, dt, cores, desc = oracle_tokens_per_s(wl, 64, min_seconds=10.0, max_passes=400)
            line["cpu_baseline"] = {"value": v, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": desc,
                                    "seconds": dt}
        print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
