#!/usr/bin/env python
"""Benchmark of the RAPID verify step on B200.

One step = one pass of the whole hot path over one batch of synthetic input:
one plan of the work split, `layers` verify-attention calls (independently
seeded K/V caches, all resident in HBM) and one accept call.  Metric: KV-read
GB/s of the step (all KV bytes of the step / step time).  Prints ONE JSON line.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl reference] [--sharded]

With --gpus N > 1 and no launcher (no WORLD_SIZE in the environment) the script
starts N ranks itself, one per GPU.  `--impl reference` times the fp64 CPU oracle
(as it stands) on a bounded sample of the same workload on the host cores.
`--sharded` times the context-sharded form of the attention: one sequence's keys
spread over the N ranks, one all-gather of partial results per layer.
"""
from __future__ import annotations

import argparse
import ctypes
import json
import os
import socket
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


TRAFFIC_SOURCES = ("attention.cu", "attention_kt.cuh", "attention_kt8.cuh", "tcgen05.cuh", "common.cuh")


def kernel_sources_sha256() -> str:
    import hashlib
    h = hashlib.sha256()
    for f in TRAFFIC_SOURCES:
        h.update(open(os.path.join(ROOT, "paper_2502_20330_b200", "csrc", f), "rb").read())
    return h.hexdigest()


def ncu_traffic(workload, kernel):
    """DRAM bytes per launch of the dominant kernel from the committed ncu capture, or None if the
    kernel sources have changed since the counters were taken (or no capture covers this kernel on this
    workload, cache type and mask)."""
    try:
        rec = json.load(open(os.path.join(ROOT, "profiles", "traffic.json")))
        key = f"{kernel}:{workload}" + (":fp8" if KV_ELEMENT_BYTES == 1 else "") + (":window" if MASK[1] > 0 else "")
        ent = rec["captures"].get(key)
        if kernel_sources_sha256() != rec["sources_sha256"] or not ent:
            return None
        return int(ent["dram_bytes_read"] + ent["dram_bytes_write"])
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


KV_ELEMENT_BYTES = 2   # set to 1 by --kv fp8: the algorithmic bytes are those of the cache as it is stored


MASK = (0, 0)          # set by --sink / --window: (sink_keys, window_keys); (0, 0) is the full causal mask


def visible_keys(cfg, ctx) -> int:
    """Keys some row of a sequence can see, summed over the sequences: all of them under the full mask,
    the sinks and the union of the rows' windows otherwise.  These are the keys the method has to read."""
    sink, window = MASK
    total = 0
    for L in (int(x) for x in ctx):
        if window <= 0:
            total += L
        else:
            lo = max(0, L - cfg.R - window + 1)      # first key of the oldest row's window
            total += (L - lo) + min(sink, lo)
    return total


def kv_bytes_per_layer(cfg, ctx) -> int:
    return int(2 * KV_ELEMENT_BYTES * cfg.Hkv * cfg.D * visible_keys(cfg, ctx))


L2_BYTES = 126 * 2**20


def with_layer_chain(cfg, ctx):
    """A workload that names ONE layer is timed as a chain of independently seeded layers of that shape
    (at least 8, and enough of them to hold three times the L2): every layer then finds its cache cold,
    and the step's one accept call does not drown the attention it follows.  Both arms apply this."""
    if cfg.layers > 1:
        return cfg
    kv_layer = kv_bytes_per_layer(cfg, ctx)
    n = max(8, -(-3 * L2_BYTES // kv_layer))
    return wl.with_overrides(cfg, layers=int(min(64, n)))


def config_dict(cfg, ctx, world, sharded=False):
    """What both arms print as `config`: the workload, nothing of how an arm runs it."""
    kv_layer = kv_bytes_per_layer(cfg, ctx)
    return {"workload": cfg.name, "kv_cache": "fp8 e4m3 + fp32 scale per (sequence, KV head)" if KV_ELEMENT_BYTES == 1 else "bf16",
            "mask": "causal" if MASK[1] <= 0 else f"{MASK[0]} sink keys + a window of {MASK[1]} keys per row",
            "B": cfg.B, "Hq": cfg.Hq, "Hkv": cfg.Hkv, "D": cfg.D,
            "ctx": [int(x) for x in ctx], "gamma": cfg.gamma, "V": cfg.V, "layers": cfg.layers, "eta": cfg.eta,
            "kv_bytes_per_step": kv_layer * cfg.layers,
            "l2": f"inputs larger than L2: {cfg.layers} distinct cache(s) of {kv_layer / 2**20:.0f} MiB per step"
                  + ("" if kv_layer * cfg.layers > 2 * L2_BYTES else ", and a buffer larger than L2 rewritten "
                     "between steps"),
            "parallelism": ("context sharded x%d" % world if sharded else f"replicas x{world}") if world > 1
                           else "single GPU"}


def find_free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _spawn_entry(rank, world, port, fn, args):
    os.environ["RANK"] = str(rank)
    os.environ["LOCAL_RANK"] = str(rank)
    os.environ["WORLD_SIZE"] = str(world)
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    fn(*args)


def spawn_ranks(world: int, fn, args=()):
    """Starts `world` processes on this node, each with the launcher's environment (RANK, LOCAL_RANK,
    WORLD_SIZE, MASTER_ADDR = 127.0.0.1, MASTER_PORT), and runs fn(*args) in every one."""
    import torch.multiprocessing as mp
    mp.spawn(_spawn_entry, args=(world, find_free_port(), fn, args), nprocs=world, join=True)


# ------------------------------------------------------------------------------------------------
# CPU oracle leg (bounded sample); with device results at hand it also judges them
# ------------------------------------------------------------------------------------------------
class OracleSample:
    """The oracle, as it stands, on a bounded sample of one step: (sequence, head, row) units of one
    layer plus one full accept call, extrapolated to the whole step.  The inputs are the bits it is
    given (the benchmark hands it the very tensors the library ran on)."""

    def __init__(self, cfg, seed, attn_inputs=None, accept_inputs=None):
        import oracle
        self.oracle = oracle
        self.cfg = cfg
        if attn_inputs is None:
            attn_inputs = wl.attention_inputs(cfg, seed, device="cpu", layer=0)
        if accept_inputs is None:
            accept_inputs = wl.accept_inputs(cfg, seed, device="cpu")
        self.fp8 = KV_ELEMENT_BYTES == 1
        if self.fp8:
            if len(attn_inputs) == 4:      # the reference arm generates its own inputs
                attn_inputs = wl.attention_inputs_fp8(cfg, seed, device="cpu", layer=0)
            q, k, v, ks, vs, ctx_t = attn_inputs
            self.bits = (wl.bf16_bits(q), k.cpu().numpy(), v.cpu().numpy(), ks.cpu().numpy(), vs.cpu().numpy())
        else:
            q, k, v, ctx_t = attn_inputs
            self.bits = (wl.bf16_bits(q), wl.bf16_bits(k), wl.bf16_bits(v))
        self.ctx = ctx_t.cpu()
        self.ctx_np = self.ctx.numpy()
        self.acc = [t.cpu().numpy() for t in accept_inputs]
        self.total_units = cfg.B * cfg.Hq * cfg.R
        self.cores = oracle.num_threads()
        self.rng = np.random.default_rng(seed)
        # calibrate the cost of one unit with one unit per core
        t = self._attention(self.cores)[0]
        self.unit_s = t / 1.0   # seconds per batch of `cores` units
        t0 = time.perf_counter()
        self.accept_ref = self._accept()
        self.accept_s = time.perf_counter() - t0
        self.attn_ref = None

    def _attention(self, n_units):
        n_units = int(min(self.total_units, max(1, n_units)))
        units = None
        if n_units < self.total_units:
            units = np.sort(self.rng.choice(self.total_units, size=n_units, replace=False)).astype(np.int64)
        t0 = time.perf_counter()
        fn = self.oracle.verify_attention_fp8 if self.fp8 else self.oracle.verify_attention
        kw = {} if self.fp8 else {"sink": MASK[0], "window": MASK[1]}
        out, lse = fn(*self.bits, self.ctx_np, self.cfg.gamma, units=units, **kw)
        dt = time.perf_counter() - t0
        self.attn_ref = (out, lse)
        return dt, n_units

    def _accept(self):
        z, d, tok, u = self.acc
        return self.oracle.accept(z, d, tok, u, eta=self.cfg.eta, T=self.cfg.temperature,
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

    def judge(self, dev_out, dev_alen, dev_ntok, extra_accept=()):
        """Compares the library's results on the same bits with what the last step() computed, under
        the parity rules of the tests.  extra_accept: more (inputs, device results) pairs of the accept
        step on other seeds, for the histogram of accepted lengths."""
        from oracle import parity
        cfg = self.cfg
        ref, ref_lse = self.attn_ref
        rows = ~np.isnan(ref_lse)
        rep = parity.check_attention(dev_out, ref, rows)
        z, d, tok, u = self.acc
        acc = parity.check_accept(z, d, tok, u, cfg.eta, cfg.temperature, cfg.tail_alpha, 0, dev_alen, dev_ntok)
        hist = [0] * (cfg.gamma + 1)
        ties = list(acc["near_ties"])
        alts = len(acc["token_alternatives"])
        for n in dev_alen:
            hist[int(n)] += 1
        for (zz, dd, tt, uu), (al, nt) in extra_accept:
            r = parity.check_accept(zz, dd, tt, uu, cfg.eta, cfg.temperature, cfg.tail_alpha, 0, al, nt)
            ties += r["near_ties"]
            alts += len(r["token_alternatives"])
            for n in al:
                hist[int(n)] += 1
        return {"max_abs": rep["max_abs"], "max_row_rel_l2": rep["max_row_rel_l2"], "rows": rep["rows"],
                "rows_total": int(rows.size), "tolerance": {"max_abs": parity.ATTN_MAX_ABS,
                                                            "row_rel_l2": parity.ATTN_ROW_REL_L2},
                "accept_len": [int(x) for x in dev_alen], "accept_len_oracle": acc["accept_len_ref"],
                "near_ties": [[int(b), int(k), float(g)] for b, k, g in ties], "token_alternatives": alts,
                "accept_len_histogram": hist, "accept_calls_checked": 1 + len(extra_accept)}


def run_reference(args, cfg):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    cfg = with_layer_chain(cfg, wl.context_lengths(cfg, args.seed))
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
        "config": config_dict(cfg, ctx, args.gpus),
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
        self.samples, self.times, self.reasons, self.max_mhz = [], [], set(), None
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
                mhz = int(self.nv.nvmlDeviceGetClockInfo(self.h, self.nv.NVML_CLOCK_SM))
                self.samples.append(mhz)
                self.times.append(time.perf_counter())
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

    def mark(self):
        """Index of the next sample: lets a caller cut the record into regions."""
        return len(self.samples)

    def summary(self, lo=0, hi=None):
        s = self.samples[lo:hi]
        return {"sm_mhz": int(statistics.median(s)) if s else None, "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(s)}

    def stop(self):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()
        return self.summary()


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
    if not args.layers:
        cfg = with_layer_chain(cfg, ctx_cpu)
    Lmax = wl.cache_capacity(cfg, ctx_cpu)
    fp8 = KV_ELEMENT_BYTES == 1
    layers = []
    for layer in range(cfg.layers):
        if fp8:
            q, k, v, ks, vs, ctx = wl.attention_inputs_fp8(cfg, seed, device=dev, layer=layer)
            layers.append((q, k, v, torch.empty_like(q), ks, vs))
        else:
            q, k, v, ctx = wl.attention_inputs(cfg, seed, device=dev, layer=layer)
            layers.append((q, k, v, torch.empty_like(q)))

    def attention(layer, params, st=None):
        if fp8:
            q_, k_, v_, out_, ks_, vs_ = layer
            R.rapid_verify_attention_fp8(q_, k_, v_, ks_, vs_, ctx, cfg.gamma, out_, aws, params, stream=st)
        else:
            q_, k_, v_, out_ = layer
            R.rapid_verify_attention(q_, k_, v_, ctx, cfg.gamma, out_, aws, params, stream=st)
    z, d, tok, u = wl.accept_inputs(cfg, seed, device=dev)
    alen = torch.zeros(cfg.B, dtype=torch.int32, device=dev)
    ntok = torch.zeros_like(alen)
    aws = R.new_workspace(R.attention_workspace_bytes(cfg.B, cfg.Hq, cfg.Hkv, cfg.D, Lmax, cfg.gamma), device=dev)
    cws = R.new_workspace(R.accept_workspace_bytes(cfg.B, cfg.gamma, cfg.V), device=dev)
    acc_params = R.AcceptParams(temperature=cfg.temperature, tail_alpha=cfg.tail_alpha)
    plan_params = R.AttnParams(kernel=args.kernel, kv_fp8=fp8, sink_keys=MASK[0], window_keys=MASK[1])
    stream = torch.cuda.current_stream()
    sptr = int(stream.cuda_stream)
    ev = RawEvents()

    kv_layer = kv_bytes_per_layer(cfg, ctx_cpu)
    kv_step = kv_layer * cfg.layers
    # one cache per step that fits in L2 would be served from it on the next step: such workloads
    # get a buffer larger than L2 rewritten between steps (outside the kernels that are timed one by one)
    flush = None
    if kv_step <= 2 * L2_BYTES:
        flush = torch.empty(192 * 2**20, dtype=torch.uint8, device=dev)

    def attn_params(li, split_event=None):
        # the plan of a step is made right before its first layer: that layer reads it after its
        # grid-dependency wait, the later ones (other kernels lie in between) before it
        mode = R.PLAN_NONE if args.no_plan else (R.PLAN_READY if li == 0 else R.PLAN_SETTLED)
        # every cache of the step was written long before the step: all but a layer's newest rows may be
        # copied while the preceding kernel still runs (what a decode loop can state as well)
        return R.AttnParams(kernel=args.kernel, plan=mode, split_done_event=split_event, sink_keys=MASK[0],
                            window_keys=MASK[1], kv_settled=not args.no_early_kv)

    def step(split_events=None, call_events=None, st=None):
        if flush is not None:
            flush.fill_(1)
        if not args.no_plan:
            R.rapid_attention_plan(ctx, cfg.gamma, cfg.B, cfg.Hq, cfg.Hkv, cfg.D, Lmax, aws, plan_params, stream=st)
        for li, layer in enumerate(layers):
            if call_events is not None:
                ev.record(call_events[li][0], sptr)
            e1 = split_events[li] if split_events is not None else None
            attention(layer, attn_params(li, e1), st)
            if call_events is not None:
                ev.record(call_events[li][1], sptr)
        R.rapid_accept(z, d, tok, u, cfg.eta, alen, ntok, cws, acc_params, stream=st)

    def barrier():
        if world > 1:
            import torch.distributed as dist
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(max(3, args.warmup)):
        step()
    barrier()
    # which kernels serve an attention call of this workload
    info = R.rapid_attention_describe(cfg.B, cfg.Hq, cfg.Hkv, cfg.D, Lmax, cfg.gamma, plan_params)
    launches_per_call = info["kernels_per_call"]
    if fp8:
        dominant = "verify_attn_splitkv_kt8_kernel"
    elif info["kernel"] == R.ATTN_KERNEL_CLUSTER_MERGE:
        dominant = f"verify_attn_splitkv_kt_kernel (clusters of {info['cluster_size']} CTAs, merged on chip)"
    else:
        dominant = "verify_attn_splitkv_kt_kernel" if info["kernel"] == R.ATTN_KERNEL_KEYS_ON_M \
            else "verify_attn_splitkv_tc_kernel"

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
            step(st=side)
    launches_per_step = R.kernel_launch_count()
    torch.cuda.synchronize()
    for _ in range(3):
        graph.replay()
    barrier()

    e_begin, e_end = ev.create(), ev.create()
    sampler = ClockSampler(local_rank)
    sampler.start()
    barrier()
    m0 = sampler.mark()
    ev.record(e_begin, sptr)
    for s in range(args.steps):
        graph.replay()
    ev.record(e_end, sptr)
    barrier()
    m1 = sampler.mark()
    launches = launches_per_step * args.steps
    total_ms = ev.elapsed_ms(e_begin, e_end)
    flush_ms = 0.0
    if flush is not None:   # the rewrite of the L2-sized buffer is not part of the step: timed alone, taken off
        f0, f1 = ev.create(), ev.create()
        ev.record(f0, sptr)
        for s in range(args.steps):
            flush.fill_(1)
        ev.record(f1, sptr)
        torch.cuda.synchronize()
        flush_ms = ev.elapsed_ms(f0, f1)
        total_ms -= flush_ms

    s_begin, s_end = ev.create(), ev.create()
    ev.record(s_begin, sptr)
    for s in range(args.steps):
        step()
    ev.record(s_end, sptr)
    barrier()
    stream_us = 1e3 * (ev.elapsed_ms(s_begin, s_end) - flush_ms) / args.steps
    # second live pass for the roofline of the dominant kernel: the same steps with an event pair
    # around every launch of it (the event between split and merge costs the pair their programmatic
    # overlap, which is why this pass is not the one that gives `value`).  A call that is one kernel
    # is timed as the call.
    k_steps = min(args.steps, 20)
    pairs = [[(ev.create(), ev.create()) for _ in range(cfg.layers)] for _ in range(k_steps)]
    for s in range(k_steps):
        if launches_per_call == 1:
            step(call_events=pairs[s])
        else:
            step(split_events=[p[1] for p in pairs[s]], call_events=[(p[0], ev.create()) for p in pairs[s]])
    barrier()
    kernel_ms = [ev.elapsed_ms(a, b) for ps in pairs for (a, b) in ps]
    m2 = sampler.mark()

    # sustained: the same graph replayed for about two seconds, an event after every step; the step
    # times are binned by the SM clock NVML reported at that moment
    sustained = None
    if rank == 0 and world == 1 and not args.no_sustained:
        est_ms = total_ms / args.steps + flush_ms / args.steps
        n_sus = int(min(20000, max(50, 2000.0 / max(est_ms, 1e-3))))
        marks = [ev.create() for _ in range(n_sus + 1)]
        torch.cuda.synchronize()
        t_host0 = time.perf_counter()
        ev.record(marks[0], sptr)
        for s in range(n_sus):
            graph.replay()
            ev.record(marks[s + 1], sptr)
        torch.cuda.synchronize()
        t_host1 = time.perf_counter()
        m3 = sampler.mark()
        ends = np.array([ev.elapsed_ms(marks[0], marks[s + 1]) for s in range(n_sus)])
        per_step = np.diff(np.concatenate([[0.0], ends])) - flush_ms / args.steps
        # device time 0 = t_host0 (the stream was idle), so sample i falls into the step running then
        scale = (t_host1 - t_host0) * 1e3 / max(ends[-1], 1e-6)
        bins = {}
        series = []
        for i in range(m2, m3):
            t_ms = (sampler.times[i] - t_host0) * 1e3 / scale
            if 0 <= t_ms <= ends[-1]:
                sidx = int(np.searchsorted(ends, t_ms))
                mhz = sampler.samples[i]
                series.append([round(t_ms, 1), mhz])
                bins.setdefault(mhz // 50 * 50, []).append(float(per_step[min(sidx, n_sus - 1)]))
        second_half = per_step[n_sus // 2:]
        sus_ms = float(np.mean(second_half))
        sustained = {"seconds": round(float(ends[-1]) / 1e3, 2), "steps": n_sus,
                     "ms_per_step_second_half": sus_ms,
                     "value_second_half": job_throughput_gbs(kv_step, 1, sus_ms),
                     "ms_per_step_first_20": float(np.mean(per_step[:20])),
                     "by_sm_mhz": {str(kk): {"steps": len(vv), "ms_per_step": float(np.mean(vv))}
                                   for kk, vv in sorted(bins.items())},
                     "clock_samples_ms_mhz": series[:: max(1, len(series) // 40)],
                     "clocks": sampler.summary(m2, m3)}
    clocks = sampler.stop()
    clocks.update(sampler.summary(m0, m1))
    status = R.workspace_status(aws) | R.workspace_status(cws)

    total_ms = max_over_ranks(total_ms, dev)
    ms_per_step = total_ms / args.steps
    value = job_throughput_gbs(kv_step, world, ms_per_step)
    peak, peak_kind = _peaks()
    kernel_avg_ms = float(np.mean(kernel_ms))
    achieved = kv_layer / (kernel_avg_ms * 1e-3) / 1e9

    del graph

    # accept latency alone: 20 calls back to back in a CUDA graph (issued from the host one by one they
    # would be timed together with the host's launch overhead); the rows are L2-warm, as in the step
    a0, a1 = ev.create(), ev.create()
    agraph = torch.cuda.CUDAGraph()
    side.wait_stream(stream)
    with torch.cuda.stream(side):
        with torch.cuda.graph(agraph, stream=side):
            for _ in range(20):
                R.rapid_accept(z, d, tok, u, cfg.eta, alen, ntok, cws, acc_params, stream=side)
    torch.cuda.synchronize()
    acc_ms = []
    for _ in range(5):
        ev.record(a0, sptr)
        agraph.replay()
        ev.record(a1, sptr)
        torch.cuda.synchronize()
        acc_ms.append(ev.elapsed_ms(a0, a1) / 20)
    del agraph

    # (the shortest of the accept timings is taken off: the smaller that figure, the longer the layers read)
    attn_layer_us = 1e3 * (ms_per_step - float(np.min(acc_ms))) / cfg.layers
    chain_gbs = kv_layer / (attn_layer_us * 1e-6) / 1e9
    line = {
        "metric": "verify_step_kv_read_gbs", "value": value, "unit": "GB/s", "n_gpus": world, "steps": args.steps,
        "warmup": max(3, args.warmup), "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "fp8 e4m3 cache, bf16 q/out, fp32 accumulate" if fp8 else "bf16", "data": "synthetic",
        "config": config_dict(cfg, ctx_cpu, world),
        "run": {"launch": "the step captured in one CUDA graph, replayed per step",
                "plan": "none" if args.no_plan else "one rapid_attention_plan per step, shared by its layers",
                "early_kv": "off" if (args.no_early_kv or args.no_plan) else
                            "kv_settled: a layer's first tiles below its newest rows are copied before its stream-order wait",
                "kernels_per_attention_call": int(launches_per_call), "attention_launch": info,
                "l2_flush_ms_per_step_not_counted": flush_ms / args.steps},
        "verify_latency_us": {"attention_per_layer": attn_layer_us,
                              "dominant_kernel_per_layer": 1e3 * kernel_avg_ms,
                              "accept": 1e3 * float(np.median(acc_ms)), "step": 1e3 * ms_per_step,
                              "step_stream_launches": stream_us},
        "frac_of_hbm_peak": {"measured": value / world / peak, "nominal_8TBs": value / world / 8000.0},
        # The dominant kernel's time per launch, from the CUDA events of the timed steps themselves: the
        # step minus its one accept call (timed beside it), over the layers.  That is one split AND one
        # merge launch per layer, the layers overlapping as programmatic dependents the way they do in
        # use, so it bounds the split kernel's own share from above.  Timed alone between two events
        # (second pass) a launch loses that overlap and takes its launch latency and prologue along.
        "roofline": {"bound": "hbm", "kernel": dominant, "achieved": chain_gbs, "peak": peak,
                     "peak_kind": peak_kind, "unit": "GB/s", "frac": chain_gbs / peak,
                     "traffic": ncu_traffic(cfg.name, dominant.split(" ")[0]),
                     "algorithmic_bytes": kv_layer,
                     "us_per_launch": attn_layer_us,
                     "timed": f"CUDA events around the {args.steps} timed steps: (step - accept call) / {cfg.layers} layers = "
                              "one split + one merge launch per layer, layers overlapping as programmatic dependents",
                     "kernel_alone": {"us_per_launch": 1e3 * kernel_avg_ms, "achieved": achieved, "frac": achieved / peak,
                                      "timed": f"CUDA events around each of {len(kernel_ms)} launches in a second pass of "
                                               f"{k_steps} steps; an event between two launches costs them their "
                                               "overlap: launch latency and prologue are inside"}},
        "clocks": clocks, "gpu_launches": int(launches), "device_status": int(status),
    }
    if sustained is not None:
        line["sustained"] = sustained

    if rank == 0 and world == 1 and not args.no_e2e and not fp8 and MASK[1] <= 0:
        line["e2e"] = run_e2e(R, cfg, seed, Lmax, kv_layer, dev)
    elif rank == 0:
        line["e2e"] = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        # The CPU leg runs on the very bits the library ran on (layer 0 and the logits, copied back
        # from the device), and what it computes is also what the library's results are judged by.
        out0 = layers[0][3]
        attention(layers[0], R.AttnParams(kernel=args.kernel, sink_keys=MASK[0], window_keys=MASK[1]))
        R.rapid_accept(z, d, tok, u, cfg.eta, alen, ntok, cws, acc_params)
        torch.cuda.synchronize()
        dev_out = out0.float().cpu().numpy()
        dev_alen, dev_ntok = alen.cpu().numpy().copy(), ntok.cpu().numpy().copy()
        extra = []
        n_extra = 0 if args.no_hist else max(0, min(15, 128 // max(1, cfg.B) - 1))
        for i in range(n_extra):
            zz, dd, tt, uu = wl.accept_inputs(cfg, seed + 7919 * (i + 1), device=dev)
            R.rapid_accept(zz, dd, tt, uu, cfg.eta, alen, ntok, cws, acc_params)
            torch.cuda.synchronize()
            extra.append(([t.cpu().numpy() for t in (zz, dd, tt, uu)], (alen.cpu().numpy().copy(), ntok.cpu().numpy().copy())))
        l0 = layers[0]
        host_attn = tuple(t.cpu() for t in ((l0[0], l0[1], l0[2], l0[4], l0[5], ctx) if fp8 else (l0[0], l0[1], l0[2], ctx)))
        host_acc = tuple(t.cpu() for t in (z, d, tok, u))
        del layers, l0
        smp = OracleSample(cfg, seed, host_attn, host_acc)
        gbs, sample, _ = smp.step(12.0)
        line["cpu_baseline"] = {"value": gbs, "unit": "GB/s", "cores": smp.cores, "kind": "oracle", "sample": sample}
        line["parity"] = smp.judge(dev_out, dev_alen, dev_ntok, extra)
    if rank == 0:
        print(json.dumps(line))
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


def run_e2e(R, cfg, seed, Lmax, kv_layer, dev, steps=5):
    """The step through rapid_verify_step_host: pinned host tensors in, host results out.  The entry
    point takes one layer (cache, rows, logits); a step of `layers` layers is that call `layers`
    times, every layer moving its own 2*Hkv*L*D*2 bytes over PCIe.  The layers of the long step are
    copied from one pinned cache (the same number of bytes crosses the bus as from `layers` caches)."""
    q, k, v, ctx = [t.pin_memory() for t in wl.attention_inputs(cfg, seed, device="cpu", layer=0)]
    z, d, tok, u = [t.pin_memory() for t in wl.accept_inputs(cfg, seed, device="cpu")]
    out = torch.empty_like(q).pin_memory()
    alen = torch.zeros(cfg.B, dtype=torch.int32).pin_memory()
    ntok = torch.zeros(cfg.B, dtype=torch.int32).pin_memory()
    arena = torch.empty(R.verify_step_host_arena_bytes(cfg.B, cfg.Hq, cfg.Hkv, cfg.D, Lmax, cfg.gamma, cfg.V),
                        dtype=torch.uint8, device=dev)
    params = R.AcceptParams(temperature=cfg.temperature, tail_alpha=cfg.tail_alpha)

    def one():
        R.rapid_verify_step_host(q, k, v, ctx, cfg.gamma, out, z, d, tok, u, cfg.eta, alen, ntok, arena,
                                 accept_params=params)

    times = []
    for i in range(steps + 2):
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        one()
        if i >= 2:
            times.append(time.perf_counter() - t0)
    nb = lambda t: t.numel() * t.element_size()  # noqa: E731
    h2d = sum(nb(t) for t in (q, k, v, ctx, z, d, tok, u))
    d2h = sum(nb(t) for t in (out, alen, ntok)) + 8
    t = float(np.median(times))
    res = {"value": kv_layer / t / 1e9, "unit": "GB/s", "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h),
           "ms_per_step": 1e3 * t, "layers_per_step": 1,
           "note": "rapid_verify_step_host on pinned host tensors; copies inside the timed region"}
    if cfg.layers > 1:
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        for _ in range(cfg.layers):
            one()
        tl = time.perf_counter() - t0
        res["whole_step"] = {"value": kv_layer * cfg.layers / tl / 1e9, "unit": "GB/s", "ms_per_step": 1e3 * tl,
                             "layers_per_step": cfg.layers, "h2d_bytes_per_step": int(h2d) * cfg.layers,
                             "d2h_bytes_per_step": int(d2h) * cfg.layers,
                             "note": f"{cfg.layers} rapid_verify_step_host calls back to back, one per layer (each "
                                     "also runs the accept step on its 8.7 MB of logits); all copied from one "
                                     "pinned host cache"}
    return res


def run_sharded(args, cfg):
    """Context-sharded attention: the keys of every sequence spread over the ranks, one all-gather of
    (output, log-sum-exp) per layer, then the merge.  Strong scaling: the job's bytes are fixed.
    Not measured on several GPUs here (a call of this benchmark gets one); with one rank it runs as
    a check of the plumbing."""
    import torch.distributed as dist
    import paper_2502_20330_b200 as R
    from paper_2502_20330_b200 import sharded

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if not dist.is_initialized():
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        os.environ.setdefault("MASTER_PORT", str(find_free_port()))
        dist.init_process_group("nccl", rank=rank, world_size=world, device_id=dev)
    ctx_cpu = wl.context_lengths(cfg, args.seed)
    bounds = sharded.context_shard_bounds(ctx_cpu.tolist(), cfg.gamma, world)[rank]
    lens = torch.tensor([e - s for s, e in bounds], dtype=torch.int32, device=dev)
    Lloc = int(lens.max())
    shard_cfg = wl.with_overrides(cfg, ctx_lens=tuple(int(x) for x in lens), ctx_range=None, Lmax=Lloc)
    layers = []
    for layer in range(cfg.layers):
        q, _, _, _ = wl.attention_inputs(wl.with_overrides(cfg, ctx_lens=(cfg.R,) * cfg.B, ctx_range=None, Lmax=cfg.R),
                                         args.seed, device=dev, layer=layer)      # the same rows on every rank
        _, k, v, _ = wl.attention_inputs(shard_cfg, rank_seed(args.seed, rank), device=dev, layer=layer)
        layers.append((q, k, v, torch.empty_like(q)))
    ws = R.new_workspace(R.attention_workspace_bytes(cfg.B, cfg.Hq, cfg.Hkv, cfg.D, Lloc, cfg.gamma), device=dev)

    def step():
        for q, k, v, out in layers:
            sharded.sharded_verify_attention(q, k, v, lens, cfg.gamma, out, ws)

    for _ in range(max(3, args.warmup)):
        step()
    dist.barrier()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sampler = ClockSampler(local_rank)
    sampler.start()
    e0.record()
    for _ in range(args.steps):
        step()
    e1.record()
    dist.barrier()
    torch.cuda.synchronize()
    clocks = sampler.stop()
    ms = max_over_ranks(e0.elapsed_time(e1), dev) / args.steps
    kv_step = kv_bytes_per_layer(cfg, ctx_cpu) * cfg.layers
    if rank == 0:
        print(json.dumps({
            "metric": "verify_step_kv_read_gbs", "value": kv_step / (ms * 1e-3) / 1e9, "unit": "GB/s", "n_gpus": world,
            "steps": args.steps, "warmup": max(3, args.warmup), "ms_per_step": ms, "higher_is_better": True,
            "scaling": "strong", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": config_dict(cfg, ctx_cpu, world, sharded=True),
            "run": {"exchange": "one NCCL all-gather of (fp32 output, log-sum-exp) per layer, then rapid_merge_partials",
                    "accept": "not part of this mode"},
            "clocks": clocks, "e2e": None, "gpu_launches": int(3 * cfg.layers * args.steps)}))
    dist.destroy_process_group()


def _rank_main(args):
    global KV_ELEMENT_BYTES, MASK
    KV_ELEMENT_BYTES = 1 if args.kv == "fp8" else 2
    if args.window > 0:
        if args.kv == "fp8" or args.sharded:
            raise SystemExit("--window is for the bf16 cache on one rank's own context")
        MASK = (max(0, args.sink), args.window)
    cfg = wl.CONFIGS[args.workload]
    if args.layers:
        cfg = wl.with_overrides(cfg, layers=args.layers)
    if args.gamma >= 0:
        cfg = wl.with_overrides(cfg, gamma=args.gamma)
    if args.impl == "reference":
        run_reference(args, cfg)
    elif args.sharded:
        run_sharded(args, cfg)
    else:
        run_ours(args, cfg)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="llama8b_128k", choices=sorted(wl.CONFIGS))
    ap.add_argument("--layers", type=int, default=0, help="override the number of resident layers")
    ap.add_argument("--gamma", type=int, default=-1, help="override the workload's number of draft tokens")
    ap.add_argument("--seed", type=int, default=2025)
    ap.add_argument("--kernel", type=int, default=0, choices=[0, 1, 2, 3],
                    help="split kernel: 0 the library's choice, 1 rows on the MMA's M axis, 2 keys on the M axis, "
                         "3 keys on M with one cluster per KV head")
    ap.add_argument("--kv", default="bf16", choices=["bf16", "fp8"],
                    help="storage of the KV cache: bf16, or FP8 E4M3 codes with a scale per (sequence, KV head)")
    ap.add_argument("--sink", type=int, default=0, help="with --window: the first keys every row sees")
    ap.add_argument("--window", type=int, default=0,
                    help="every row sees the sinks and its own newest WINDOW keys only (0: the full causal mask)")
    ap.add_argument("--sharded", action="store_true", help="context-sharded attention over the ranks")
    ap.add_argument("--no-plan", action="store_true", help="every attention call works its split out itself")
    ap.add_argument("--no-early-kv", action="store_true",
                    help="do not let a layer copy its first (old) K/V tiles while the preceding kernel runs")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-sustained", action="store_true")
    ap.add_argument("--no-hist", action="store_true")
    args = ap.parse_args()
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ and args.impl != "reference":
        spawn_ranks(args.gpus, _rank_main, (args,))   # no launcher: start one rank per GPU here
    else:
        _rank_main(args)


if __name__ == "__main__":
    main()
