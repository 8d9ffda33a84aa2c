#!/usr/bin/env python
"""Benchmark of the RAPID verify step on B200.

One step = one pass of the whole hot path over one batch of synthetic input:
`layers` verify-attention calls (independently seeded K/V caches, all resident in
HBM) followed by one accept call.  Metric: KV-read GB/s of the step (all KV bytes
of the step / step time).  Prints ONE JSON line.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl reference]

`--impl reference` times the fp64 CPU oracle (as it stands) on a bounded sample of
the same workload on the host cores.
"""
from __future__ import annotations

import argparse
import ctypes
import json
import os
import statistics
import sys
import threading
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import workloads as wl  # noqa: E402


def _peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return float(p["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


def ncu_traffic(workload, kernel="verify_attn_splitkv_tc_kernel"):
    """DRAM bytes per split-kernel launch from the committed ncu capture, or None if the kernel
    sources have changed since the counters were taken (or the capture is of the other kernel)."""
    import hashlib
    try:
        rec = json.load(open(os.path.join(ROOT, "profiles", "traffic.json")))
        h = hashlib.sha256()
        for f in ("attention.cu", "attention_kt.cuh", "tcgen05.cuh", "common.cuh"):
            h.update(open(os.path.join(ROOT, "paper_2502_20330_b200", "csrc", f), "rb").read())
        if h.hexdigest() != rec["kernel_sha256"] or workload not in rec or rec.get("kernel") != kernel:
            return None
        return int(rec[workload]["dram_bytes_read"] + rec[workload]["dram_bytes_write"])
    except Exception:
        return None


def rank_seed(seed: int, rank: int) -> int:
    """Every rank verifies its own requests (weak scaling, no exchange on the data path)."""
    return int(seed) + 1000 * int(rank)


def max_over_ranks(value: float, device="cpu") -> float:
    """MAX all-reduce of a scalar over the default process group (identity without one)."""
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_throughput_gbs(bytes_per_rank_step: int, world: int, ms_per_step: float) -> float:
    """Whole-job KV-read GB/s: all ranks' bytes over the slowest rank's step time."""
    return bytes_per_rank_step * world / (ms_per_step * 1e-3) / 1e9


def kv_bytes_per_layer(cfg, ctx) -> int:
    return int(4 * cfg.Hkv * cfg.D * int(ctx.sum()))


# ------------------------------------------------------------------------------------------------
# CPU oracle leg (bounded sample)
# ------------------------------------------------------------------------------------------------
class OracleSample:
    """The oracle, as it stands, on a bounded sample of one step: a subset of one layer's
    (sequence, head, row) units plus one full accept call, extrapolated to the whole step."""

    def __init__(self, cfg, seed):
        import oracle
        self.oracle = oracle
        self.cfg = cfg
        self.ctx = wl.context_lengths(cfg, seed)
        q, k, v, ctx_t = wl.attention_inputs(cfg, seed, device="cpu", layer=0)
        self.bits = (wl.bf16_bits(q), wl.bf16_bits(k), wl.bf16_bits(v))
        self.ctx_np = ctx_t.numpy()
        self.acc = [t.numpy() for t in wl.accept_inputs(cfg, seed, device="cpu")]
        self.total_units = cfg.B * cfg.Hq * cfg.R
        self.cores = oracle.num_threads()
        self.rng = np.random.default_rng(seed)
        # calibrate the cost of one unit with one unit per core
        t = self._attention(self.cores)[0]
        self.unit_s = t / 1.0   # seconds per batch of `cores` units
        t0 = time.perf_counter()
        self._accept()
        self.accept_s = time.perf_counter() - t0

    def _attention(self, n_units):
        n_units = int(min(self.total_units, max(1, n_units)))
        units = np.sort(self.rng.choice(self.total_units, size=n_units, replace=False)).astype(np.int64)
        t0 = time.perf_counter()
        self.oracle.verify_attention(*self.bits, self.ctx_np, self.cfg.gamma, units=units)
        return time.perf_counter() - t0, n_units

    def _accept(self):
        z, d, tok, u = self.acc
        self.oracle.accept(z, d, tok, u, eta=self.cfg.eta, T=self.cfg.temperature,
                           tail_alpha=self.cfg.tail_alpha, want_ratios=False)

    def step(self, budget_s):
        """Returns (GB/s of the extrapolated step, description, seconds spent)."""
        cfg = self.cfg
        attn_budget = max(0.0, budget_s - self.accept_s)
        n = max(self.cores, int(self.cores * attn_budget / max(self.unit_s, 1e-6)))
        t_attn, n = self._attention(n)
        t0 = time.perf_counter()
        self._accept()
        t_acc = time.perf_counter() - t0
        step_s = t_attn * (self.total_units / n) * cfg.layers + t_acc
        gbs = kv_bytes_per_layer(cfg, self.ctx) * cfg.layers / step_s / 1e9
        sample = (f"{n} of {self.total_units} (sequence, head, row) units of one layer ({t_attn:.2f} s) "
                  f"+ one full accept call ({t_acc:.2f} s), extrapolated to {cfg.layers} layer(s)")
        return gbs, sample, t_attn + t_acc


def run_reference(args, cfg):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    smp = OracleSample(cfg, args.seed)
    per_step_budget = max(0.2, min(20.0, 150.0 / max(1, args.steps + args.warmup)))
    vals, sample = [], ""
    for i in range(args.warmup + args.steps):
        gbs, sample, _ = smp.step(per_step_budget)
        if i >= args.warmup:
            vals.append(gbs)
    value = float(np.mean(vals))
    ctx = smp.ctx
    ms = kv_bytes_per_layer(cfg, ctx) * cfg.layers / value / 1e6
    line = {
        "impl": "reference", "metric": "verify_step_kv_read_gbs", "value": value, "unit": "GB/s",
        "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": cfg.name, "B": cfg.B, "Hq": cfg.Hq, "Hkv": cfg.Hkv, "D": cfg.D,
                   "ctx": [int(x) for x in ctx], "gamma": cfg.gamma, "V": cfg.V, "layers": cfg.layers},
        "cpu_baseline": {"value": value, "unit": "GB/s", "cores": smp.cores, "kind": "oracle",
                         "sample": sample + f"; mean of {args.steps} such samples"},
        "e2e": {"value": value, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# ------------------------------------------------------------------------------------------------
# clocks sampling (NVML, read only)
# ------------------------------------------------------------------------------------------------
class ClockSampler:
    REASONS = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown",
               0x4: "sw_power_cap", 0x80: "hw_power_brake_slowdown"}

    def __init__(self, index):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self.nv = None

    def _loop(self):
        while not self._stop.is_set():
            try:
                self.samples.append(int(self.nv.nvmlDeviceGetClockInfo(self.h, self.nv.NVML_CLOCK_SM)))
                bits = int(self.nv.nvmlDeviceGetCurrentClocksEventReasons(self.h))
                for bit, name in self.REASONS.items():
                    if bits & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            self._stop.wait(0.01)

    def start(self):
        if self.nv is not None:
            self._thread = threading.Thread(target=self._loop, daemon=True)
            self._thread.start()

    def stop(self):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()
        return {"sm_mhz": int(statistics.median(self.samples)) if self.samples else None,
                "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": len(self.samples)}


# ------------------------------------------------------------------------------------------------
# CUDA runtime events by handle (the library records one between its two attention kernels)
# ------------------------------------------------------------------------------------------------
class RawEvents:
    def __init__(self):
        self.rt = None
        for name in ("libcudart.so.12", "libcudart.so"):
            try:
                self.rt = ctypes.CDLL(name)
                break
            except OSError:
                continue
        if self.rt is None:
            import glob
            cands = glob.glob(os.path.join(os.path.dirname(torch.__file__), "..", "nvidia", "cuda_runtime", "lib",
                                           "libcudart.so*"))
            self.rt = ctypes.CDLL(cands[0])
        self.rt.cudaEventCreate.argtypes = [ctypes.POINTER(ctypes.c_void_p)]
        self.rt.cudaEventRecord.argtypes = [ctypes.c_void_p, ctypes.c_void_p]
        self.rt.cudaEventElapsedTime.argtypes = [ctypes.POINTER(ctypes.c_float), ctypes.c_void_p, ctypes.c_void_p]
        self.rt.cudaEventDestroy.argtypes = [ctypes.c_void_p]

    def create(self):
        e = ctypes.c_void_p()
        assert self.rt.cudaEventCreate(ctypes.byref(e)) == 0
        return e.value

    def record(self, e, stream):
        assert self.rt.cudaEventRecord(e, stream) == 0

    def elapsed_ms(self, a, b):
        ms = ctypes.c_float()
        rc = self.rt.cudaEventElapsedTime(ctypes.byref(ms), a, b)
        assert rc == 0, rc
        return ms.value


# ------------------------------------------------------------------------------------------------
def run_ours(args, cfg):
    import paper_2502_20330_b200 as R

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)

    R.load_library()
    seed = rank_seed(args.seed, rank)
    ctx_cpu = wl.context_lengths(cfg, seed)
    Lmax = wl.cache_capacity(cfg, ctx_cpu)
    layers = []
    for layer in range(cfg.layers):
        q, k, v, ctx = wl.attention_inputs(cfg, seed, device=dev, layer=layer)
        layers.append((q, k, v, torch.empty_like(q)))
    z, d, tok, u = wl.accept_inputs(cfg, seed, device=dev)
    alen = torch.zeros(cfg.B, dtype=torch.int32, device=dev)
    ntok = torch.zeros_like(alen)
    aws = R.new_workspace(R.attention_workspace_bytes(cfg.B, cfg.Hq, cfg.Hkv, cfg.D, Lmax, cfg.gamma), device=dev)
    cws = R.new_workspace(R.accept_workspace_bytes(cfg.B, cfg.gamma, cfg.V), device=dev)
    acc_params = R.AcceptParams(temperature=cfg.temperature, tail_alpha=cfg.tail_alpha)
    attn_params = R.AttnParams(kernel=args.kernel)
    keys_on_m = args.kernel == 2 or (args.kernel == 0 and cfg.D == 128 and cfg.G * cfg.R <= 64)
    split_kernel = "verify_attn_splitkv_kt_kernel" if keys_on_m else "verify_attn_splitkv_tc_kernel"
    stream = torch.cuda.current_stream()
    sptr = int(stream.cuda_stream)
    ev = RawEvents()

    kv_layer = kv_bytes_per_layer(cfg, ctx_cpu)
    kv_step = kv_layer * cfg.layers

    def step(split_events=None):
        for li, (q, k, v, out) in enumerate(layers):
            if split_events is not None:
                e0, e1 = split_events[li]
                ev.record(e0, sptr)
                R.rapid_verify_attention(q, k, v, ctx, cfg.gamma, out, aws,
                                         R.AttnParams(split_done_event=e1, kernel=args.kernel))
            else:
                R.rapid_verify_attention(q, k, v, ctx, cfg.gamma, out, aws, attn_params)
        R.rapid_accept(z, d, tok, u, cfg.eta, alen, ntok, cws, acc_params)

    def barrier():
        if world > 1:
            import torch.distributed as dist
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(max(3, args.warmup)):
        step()
    barrier()

    # The step is captured once in a CUDA graph (every call of the path is asynchronous and
    # allocation-free, so the whole step is capturable) and the timed region replays it: K graph
    # launches between two events on the launching stream, nothing else on it.  The same K steps
    # issued call by call from Python are timed right after, as `step_stream_launches`.
    side = torch.cuda.Stream(device=dev)
    side.wait_stream(stream)
    graph = torch.cuda.CUDAGraph()
    R.kernel_launch_count_reset()
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            for (q, k, v, out) in layers:
                R.rapid_verify_attention(q, k, v, ctx, cfg.gamma, out, aws, attn_params, stream=side)
            R.rapid_accept(z, d, tok, u, cfg.eta, alen, ntok, cws, acc_params, stream=side)
    launches_per_step = R.kernel_launch_count()
    torch.cuda.synchronize()
    for _ in range(3):
        graph.replay()
    barrier()

    e_begin, e_end = ev.create(), ev.create()
    sampler = ClockSampler(local_rank)
    sampler.start()
    barrier()
    ev.record(e_begin, sptr)
    for s in range(args.steps):
        graph.replay()
    ev.record(e_end, sptr)
    barrier()
    launches = launches_per_step * args.steps
    total_ms = ev.elapsed_ms(e_begin, e_end)

    s_begin, s_end = ev.create(), ev.create()
    ev.record(s_begin, sptr)
    for s in range(args.steps):
        step()
    ev.record(s_end, sptr)
    barrier()
    stream_us = 1e3 * ev.elapsed_ms(s_begin, s_end) / args.steps
    # second live pass for the roofline of the dominant kernel: the same steps with an event pair
    # around every split kernel (the event between split and merge costs the pair their
    # programmatic overlap, which is why this pass is not the one that gives `value`)
    k_steps = min(args.steps, 20)
    timed_pairs = [[(ev.create(), ev.create()) for _ in range(cfg.layers)] for _ in range(k_steps)]
    for s in range(k_steps):
        step(timed_pairs[s])
    barrier()
    clocks = sampler.stop()
    split_ms = [ev.elapsed_ms(a, b) for pairs in timed_pairs for (a, b) in pairs]
    status = R.workspace_status(aws) | R.workspace_status(cws)

    total_ms = max_over_ranks(total_ms, dev)
    ms_per_step = total_ms / args.steps
    value = job_throughput_gbs(kv_step, world, ms_per_step)
    peak, peak_kind = _peaks()
    split_avg_ms = float(np.mean(split_ms))
    achieved = kv_layer / (split_avg_ms * 1e-3) / 1e9

    del graph

    # accept latency alone (events around the call, L2-warm rows by nature of the step)
    a0, a1 = ev.create(), ev.create()
    acc_ms = []
    for _ in range(20):
        ev.record(a0, sptr)
        R.rapid_accept(z, d, tok, u, cfg.eta, alen, ntok, cws, acc_params)
        ev.record(a1, sptr)
        torch.cuda.synchronize()
        acc_ms.append(ev.elapsed_ms(a0, a1))

    line = {
        "metric": "verify_step_kv_read_gbs", "value": value, "unit": "GB/s", "n_gpus": world, "steps": args.steps,
        "warmup": max(3, args.warmup), "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": cfg.name, "B": cfg.B, "Hq": cfg.Hq, "Hkv": cfg.Hkv, "D": cfg.D,
                   "ctx": [int(x) for x in ctx_cpu], "gamma": cfg.gamma, "V": cfg.V, "layers": cfg.layers,
                   "eta": cfg.eta, "kv_bytes_per_step": kv_step,
                   "l2": f"inputs larger than L2: {cfg.layers} distinct caches of {kv_layer / 2**20:.0f} MiB per step",
                   "launch": "the step captured in one CUDA graph, replayed per step",
                   "parallelism": f"replicas x{world}" if world > 1 else "single GPU"},
        "verify_latency_us": {"attention_per_layer": 1e3 * (ms_per_step - float(np.median(acc_ms))) / cfg.layers,
                              "split_kernel_per_layer": 1e3 * split_avg_ms,
                              "accept": 1e3 * float(np.median(acc_ms)), "step": 1e3 * ms_per_step,
                              "step_stream_launches": stream_us},
        "frac_of_hbm_peak": {"measured": value / world / peak, "nominal_8TBs": value / world / 8000.0},
        "roofline": {"bound": "hbm", "kernel": split_kernel, "achieved": achieved, "peak": peak,
                     "peak_kind": peak_kind, "unit": "GB/s", "frac": achieved / peak, "traffic": ncu_traffic(cfg.name, split_kernel),
                     "algorithmic_bytes": kv_layer,
                     "timed": f"CUDA events around each of {len(split_ms)} launches in a second pass of {k_steps} steps"},
        "clocks": clocks, "gpu_launches": int(launches), "device_status": int(status),
    }

    if rank == 0 and world == 1 and not args.no_e2e:
        line["e2e"] = run_e2e(R, cfg, seed, Lmax, kv_layer, dev)
    elif rank == 0:
        line["e2e"] = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        del layers
        smp = OracleSample(cfg, seed)
        gbs, sample, _ = smp.step(12.0)
        line["cpu_baseline"] = {"value": gbs, "unit": "GB/s", "cores": smp.cores, "kind": "oracle", "sample": sample}
    if rank == 0:
        print(json.dumps(line))
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


def run_e2e(R, cfg, seed, Lmax, kv_layer, dev, steps=5):
    """The step through rapid_verify_step_host: pinned host tensors in, host results out; one layer
    per step (every layer would move its own 2*Hkv*L*D*2 bytes over PCIe the same way)."""
    q, k, v, ctx = [t.pin_memory() for t in wl.attention_inputs(cfg, seed, device="cpu", layer=0)]
    z, d, tok, u = [t.pin_memory() for t in wl.accept_inputs(cfg, seed, device="cpu")]
    out = torch.empty_like(q).pin_memory()
    alen = torch.zeros(cfg.B, dtype=torch.int32).pin_memory()
    ntok = torch.zeros(cfg.B, dtype=torch.int32).pin_memory()
    arena = torch.empty(R.verify_step_host_arena_bytes(cfg.B, cfg.Hq, cfg.Hkv, cfg.D, Lmax, cfg.gamma, cfg.V),
                        dtype=torch.uint8, device=dev)
    params = R.AcceptParams(temperature=cfg.temperature, tail_alpha=cfg.tail_alpha)
    times = []
    for i in range(steps + 2):
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        R.rapid_verify_step_host(q, k, v, ctx, cfg.gamma, out, z, d, tok, u, cfg.eta, alen, ntok, arena,
                                 accept_params=params)
        if i >= 2:
            times.append(time.perf_counter() - t0)
    nb = lambda t: t.numel() * t.element_size()  # noqa: E731
    h2d = sum(nb(t) for t in (q, k, v, ctx, z, d, tok, u))
    d2h = sum(nb(t) for t in (out, alen, ntok)) + 8
    t = float(np.median(times))
    return {"value": kv_layer / t / 1e9, "unit": "GB/s", "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h),
            "ms_per_step": 1e3 * t, "layers_per_step": 1,
            "note": "rapid_verify_step_host on pinned host tensors; copies inside the timed region"}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="llama8b_128k", choices=sorted(wl.CONFIGS))
    ap.add_argument("--layers", type=int, default=0, help="override the number of resident layers")
    ap.add_argument("--seed", type=int, default=2025)
    ap.add_argument("--kernel", type=int, default=0, choices=[0, 1, 2],
                    help="split kernel: 0 the library's choice, 1 rows on the MMA's M axis, 2 keys on the M axis")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    cfg = wl.CONFIGS[args.workload]
    if args.layers:
        cfg = wl.with_overrides(cfg, layers=args.layers)
    if args.impl == "reference":
        run_reference(args, cfg)
    else:
        run_ours(args, cfg)


if __name__ == "__main__":
    main()
