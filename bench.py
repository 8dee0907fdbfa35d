#!/usr/bin/env python
"""Benchmark of the vocabulary-mask path: one "step" = one decoding step of the whole batch
(row resets the stream asks for, fmt_state_advance with the chosen tokens, fmt_fill_and_apply on
that step's logits).  Metric: vocab-mask token-checks per second = batch * V * steps / time.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config C] [--impl ours|reference]

With --gpus N > 1 the script is launched by torch.distributed.run, one rank per GPU; every rank
runs the same workload on its own replica of the tables (sequences are independent, so the path
shards by sequence with no collective on the data path); time is the max over ranks.
--impl reference times the CPU oracle on the host cores instead (a deliberately slow baseline).
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

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import workloads  # noqa: E402

METRIC = "vocab-mask token-checks/s"
UNIT = "token-checks/s"
DEFAULT_CONFIG = 3
L2_BYTES = 126 * 1024 * 1024
# dram__bytes_read.sum + dram__bytes_write.sum per launch from the ncu captures summarised under
# profiles/ (config 3 only; taken on the kernels as committed with those summaries)
NCU_TRAFFIC_BYTES = {3: {"sweep_kernel": 3.6e6, "gather_apply_kernel": 7.9e6, "advance_kernel": 1.6e5}}


# --------------------------------------------------------------------------- small helpers


def measured_peaks():
    """HBM GB/s to divide by: the measured copy bandwidth if its file is there."""
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return 6650.0, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons while the timed region runs: through NVML every few
    milliseconds when the nvidia_ml_py module can be loaded, else by calling nvidia-smi."""

    QUERY = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")
    REASON_BITS = {"sw_power_cap": 0x4, "hw_slowdown": 0x8, "sw_thermal_slowdown": 0x20, "hw_thermal_slowdown": 0x40}

    def __init__(self, index: int):
        self.index = index
        self.sm, self.mx, self.reasons = [], [], set()
        self._stop = threading.Event()
        self._thread = None
        self._nvml = None
        try:
            import pynvml

            pynvml.nvmlInit()
            uuid = None
            try:
                import torch

                uuid = str(torch.cuda.get_device_properties(index).uuid)
            except Exception:
                pass
            h = None
            if uuid:
                for i in range(pynvml.nvmlDeviceGetCount()):
                    hi = pynvml.nvmlDeviceGetHandleByIndex(i)
                    u = pynvml.nvmlDeviceGetUUID(hi)
                    u = u.decode() if isinstance(u, bytes) else u
                    if uuid in u:
                        h = hi
            if h is None:
                h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self._nvml, self._h = pynvml, h
            self.source = "nvml"
        except Exception:
            self.source = "nvidia-smi"

    def _sample_nvml(self):
        n, h = self._nvml, self._h
        self.sm.append(float(n.nvmlDeviceGetClockInfo(h, n.NVML_CLOCK_SM)))
        self.mx.append(float(n.nvmlDeviceGetMaxClockInfo(h, n.NVML_CLOCK_SM)))
        bits = int(n.nvmlDeviceGetCurrentClocksThrottleReasons(h))
        for name, bit in self.REASON_BITS.items():
            if bits & bit:
                self.reasons.add(name)

    def _sample_smi(self):
        out = subprocess.run(
            ["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.QUERY, "--format=csv,noheader,nounits"],
            capture_output=True, text=True, timeout=5).stdout.strip()
        s = [x.strip() for x in out.split(",")]
        self.sm.append(float(s[0]))
        self.mx.append(float(s[1]))
        for n, v in zip(["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"], s[2:6]):
            if v.lower().startswith("active"):
                self.reasons.add(n)

    def _run(self):
        while not self._stop.is_set():
            try:
                if self._nvml is not None:
                    self._sample_nvml()
                else:
                    self._sample_smi()
            except Exception:
                pass
            self._stop.wait(0.004 if self._nvml is not None else 0.2)

    def start(self):
        self._thread = threading.Thread(target=self._run, daemon=True)
        self._thread.start()

    def stop(self) -> dict:
        self._stop.set()
        if self._thread:
            self._thread.join(timeout=6)
        return {"sm_mhz": statistics.median(self.sm) if self.sm else None, "sm_max_mhz": max(self.mx) if self.mx else None,
                "reasons": sorted(self.reasons), "samples": len(self.sm), "source": self.source}


def aggregate_over_ranks(elapsed_ms: float, units: float, dist=None):
    """Whole-job throughput: all ranks' units divided by the slowest rank's time.
    `dist` is torch.distributed (initialised) or None for a single process."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return elapsed_ms, units
    import torch

    dev = torch.device("cuda", torch.cuda.current_device()) if dist.get_backend() == "nccl" else torch.device("cpu")
    t = torch.tensor([elapsed_ms], dtype=torch.float64, device=dev)
    u = torch.tensor([units], dtype=torch.float64, device=dev)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(t.item()), float(u.item())


# --------------------------------------------------------------------------- the GPU arm


class Driver:
    """Owns the library objects and the device buffers of one replica and runs steps."""

    def __init__(self, w: workloads.Workload, device, ring_bytes: int = int(1.6 * L2_BYTES)):
        import torch

        import paper_2506_01151_b200 as fmt

        self.torch, self.fmt, self.w, self.device = torch, fmt, w, device
        self.grammar = fmt.Grammar(w.ebnf, w.start, w.vocab, w.eos)
        self.state = fmt.State(self.grammar, w.batch)
        self.stream = torch.cuda.current_stream(device)
        B, V = w.batch, w.V
        self.status = torch.zeros(B, dtype=torch.int32, device=device)
        self.tokens = torch.from_numpy(np.ascontiguousarray(w.tokens)).to(device)  # [steps, B]
        self.prefix = torch.from_numpy(np.ascontiguousarray(w.prefix)).to(device)
        self.resets = {}
        for i in range(w.steps):
            r = np.nonzero(w.reset_before[i])[0]
            if len(r):
                self.resets[i] = torch.from_numpy(r.astype(np.int32)).to(device)
        # logits: a ring of buffers larger than L2 so that no step finds its logits cached
        row_bytes = B * V * 2
        self.n_ring = max(2, -(-ring_bytes // row_bytes))
        g = torch.Generator(device=device)
        g.manual_seed(2506_01151)
        self.ring = (torch.randn((self.n_ring, B, V), generator=g, device=device, dtype=torch.float32) * 2.0).to(torch.bfloat16)
        self.launches = 0

    def feed_prefix(self):
        for p in range(self.prefix.shape[0]):
            self.state.advance(self.prefix[p], self.status, stream=self.stream.cuda_stream)
        self.torch.cuda.synchronize(self.device)

    def step(self, i: int, logits=None):
        s = self.stream.cuda_stream
        r = self.resets.get(i)
        if r is not None:
            self.state.reset(r, stream=s)
            self.launches += 1
        self.state.advance(self.tokens[i], self.status, stream=s)
        lg = self.ring[i % self.n_ring] if logits is None else logits
        self.state.fill_and_apply(lg, self.fmt.BF16, stream=s)
        self.launches += 5  # advance; plan, sweep, publish, mask+apply


def run_ours(args):
    import torch
    import torch.distributed as dist

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the mask path has no CPU fallback")
    torch.cuda.set_device(local)
    device = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=device)
    K, W = args.steps, args.warmup
    w = workloads.build(args.config, steps=K + W, batch=args.batch)
    drv = Driver(w, device)
    drv.feed_prefix()
    for i in range(W):
        drv.step(i)
    torch.cuda.synchronize(device)
    stats0 = drv.state.stats()
    drv.launches = 0

    # ---- timed region: device-resident inputs
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize(device)
    sampler = ClockSampler(local)
    sampler.start()
    drv.state.set_profiling(True)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(drv.stream)
    for i in range(W, W + K):
        drv.step(i)
    e1.record(drv.stream)
    torch.cuda.synchronize(device)
    if world > 1:
        dist.barrier()
    elapsed_ms = e0.elapsed_time(e1)
    clocks = sampler.stop()
    prof = drv.state.read_profile()
    drv.state.set_profiling(False)
    launches = drv.launches
    stats1 = drv.state.stats()
    units = float(w.batch) * w.V * K
    t_ms, total_units = aggregate_over_ranks(elapsed_ms, units, dist if world > 1 else None)

    # ---- cold fills: the same steps with the state cache emptied before every fill
    cold = None
    e2e = None
    if rank == 0:
        cold = measure_cold(drv, w, W, min(K, 32))
        e2e = measure_e2e(drv, w, W, min(K, 64))
    if world > 1:
        dist.barrier()
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    info = drv.grammar.info()
    peak, peak_kind = measured_peaks()
    B, V, Wm = w.batch, w.V, info.mask_words
    # algorithmic bytes per launch of each kernel kind: what the method itself must move through HBM
    trie_bytes = info.trie_nodes * (1 + 4 + 1) + 4 * V  # node byte, parent, depth; token -> node
    jobs = stats1["fills_computed"] - stats0["fills_computed"]
    walk_bytes_per_launch = trie_bytes + (jobs / max(1, K)) * (4 * Wm + 2048)
    apply_bytes_per_launch = B * (4 * Wm + 2 * V)
    kinds = {
        "sweep_kernel": (prof["sweep_ms"], prof["sweep_launches"], walk_bytes_per_launch),
        "gather_apply_kernel": (prof["apply_ms"], prof["apply_launches"], apply_bytes_per_launch),
        "advance_kernel": (prof["advance_ms"], prof["advance_launches"], B * 2 * 4 * 256),
    }
    dom = max(kinds, key=lambda k: kinds[k][0])
    d_ms, d_n, d_bytes = kinds[dom]
    avg_ms = d_ms / max(1, d_n)
    achieved = d_bytes / (avg_ms * 1e-3) / 1e9 if avg_ms > 0 else 0.0
    roofline = {
        "bound": "hbm", "kernel": dom, "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
        "traffic": NCU_TRAFFIC_BYTES.get(args.config, {}).get(dom), "peak_source": peak_kind + " copy bandwidth", "avg_launch_us": avg_ms * 1e3,
        "bytes_per_launch": d_bytes,
        "per_kernel_ms": {k: v[0] for k, v in kinds.items()},
        "hbm_floor_us_per_step": (apply_bytes_per_launch + trie_bytes) / (peak * 1e9) * 1e6,
        "step_frac_of_hbm_floor": ((apply_bytes_per_launch + trie_bytes) / (peak * 1e9) * 1e3) / (t_ms / K),
    }
    fills = stats1["fills"] - stats0["fills"]
    out = {
        "metric": METRIC, "value": total_units / (t_ms * 1e-3), "unit": UNIT, "n_gpus": world, "steps": K, "warmup": W,
        "ms_per_step": t_ms / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "u32",
        "data": "synthetic",
        "config": {"workload": w.name, "config": args.config, "batch": B, "vocab": V, "logits": "bf16",
                   "l2": "logits cycle through a ring of %d buffers (%.0f MB) > 126 MB L2" % (drv.n_ring, drv.n_ring * B * V * 2 / 1e6),
                   "state_cache": "on (the paper's state cache; cold numbers under 'cold')",
                   "parallelism": "replicas" if world > 1 else "single"},
        "clocks": clocks, "e2e": e2e, "gpu_launches": launches, "roofline": roofline,
        "cache": {"fills": fills, "computed": jobs,
                  "from_cache": stats1["fills_from_cache"] - stats0["fills_from_cache"],
                  "shared": stats1["fills_shared"] - stats0["fills_shared"],
                  "hit_rate": 1.0 - jobs / max(1, fills), "states_cached": stats1["states_cached"],
                  "chart_items_max": stats1["chart_items_max"], "chart_sets_max": stats1["chart_sets_max"],
                  "capacity_errors": stats1["capacity_errors"],
                  "sweep_transitions": stats1["sweep_transitions"] - stats0["sweep_transitions"],
                  "sweep_states": stats1["sweep_states"] - stats0["sweep_states"],
                  "big_mode": stats1["big_mode_units"] - stats0["big_mode_units"],
                  "advances": stats1["steps_advanced"] - stats0["steps_advanced"],
                  "advances_from_cache": stats1["advances_cached"] - stats0["advances_cached"]},
        "cold": cold,
        "grammar": {"nonterminals": info.n_nonterminals, "rules": info.n_rules, "dotted": info.n_dotted,
                    "trie_nodes": info.trie_nodes, "byte_classes": info.n_byte_classes},
    }
    if not args.no_cpu_baseline and world == 1:
        out["cpu_baseline"] = cpu_baseline(w, W, budget_s=args.cpu_seconds)
    else:
        out["cpu_baseline"] = None
    print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


def measure_cold(drv: "Driver", w, start: int, n: int):
    """ms per fill when every row's mask is recomputed (state cache emptied before each fill)."""
    torch = drv.torch
    s = drv.stream.cuda_stream
    mask = torch.zeros((w.batch, drv.grammar.mask_words), dtype=torch.int32, device=drv.device)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    total = 0.0
    drv.state.read_profile()
    drv.state.set_profiling(True)
    for i in range(n):
        drv.state.cache_clear(stream=s)
        e0.record(drv.stream)
        drv.state.fill_mask(mask, stream=s)
        e1.record(drv.stream)
        torch.cuda.synchronize(drv.device)
        total += e0.elapsed_time(e1)
    prof = drv.state.read_profile()
    drv.state.set_profiling(False)
    return {"fills": n, "ms_per_fill": total / n, "sweep_ms_per_fill": prof["sweep_ms"] / max(1, prof["sweep_launches"]),
            "token_checks_per_s": w.batch * w.V / (total / n * 1e-3),
            "what": "fmt_fill_mask with the state cache emptied before each call: every distinct row state walks the trie"}


def measure_e2e(drv: "Driver", w, start: int, n: int):
    """The same step driven from HOST buffers: token ids and logits are copied host->device from
    pinned memory, mask and status are copied back, all inside the timed region.  The mask does
    not depend on the logits, so the step is issued the way a serving loop would: the logits
    travel on a copy stream while fmt_state_advance and fmt_fill_mask run, and fmt_apply_mask
    waits for them."""
    torch = drv.torch
    B, V = w.batch, w.V
    s = drv.stream.cuda_stream
    h_logits = torch.empty((B, V), dtype=torch.bfloat16).pin_memory()
    h_logits.copy_(drv.ring[0].cpu())
    h_tokens = torch.from_numpy(np.ascontiguousarray(w.tokens)).pin_memory()
    d_logits = torch.empty((B, V), dtype=torch.bfloat16, device=drv.device)
    d_tokens = torch.empty(B, dtype=torch.int32, device=drv.device)
    d_mask = torch.zeros((B, drv.grammar.mask_words), dtype=torch.int32, device=drv.device)
    h_mask = torch.empty((B, drv.grammar.mask_words), dtype=torch.int32).pin_memory()
    h_status = torch.empty(B, dtype=torch.int32).pin_memory()
    # replay from a fresh state so that the token stream is valid again
    drv.state.reset(stream=s)
    drv.feed_prefix()
    for i in range(start):
        drv.step(i)
    copy_stream = torch.cuda.Stream(device=drv.device)
    arrived = torch.cuda.Event()
    torch.cuda.synchronize(drv.device)
    t0 = time.perf_counter()
    for i in range(start, start + n):
        r = drv.resets.get(i)
        if r is not None:
            drv.state.reset(r, stream=s)
        with torch.cuda.stream(copy_stream):
            d_logits.copy_(h_logits, non_blocking=True)
            arrived.record(copy_stream)
        d_tokens.copy_(h_tokens[i], non_blocking=True)
        drv.state.advance(d_tokens, drv.status, stream=s)
        drv.state.fill_mask(d_mask, stream=s)
        drv.stream.wait_event(arrived)
        drv.fmt.apply_mask(d_mask, d_logits, drv.fmt.BF16, B, V, stream=s)
        h_mask.copy_(d_mask, non_blocking=True)
        h_status.copy_(drv.status, non_blocking=True)
        torch.cuda.synchronize(drv.device)
    dt = time.perf_counter() - t0
    return {"value": B * V * n / dt, "unit": UNIT, "ms_per_step": dt / n * 1e3,
            "h2d_bytes_per_step": B * 4 + B * V * 2, "d2h_bytes_per_step": B * drv.grammar.mask_words * 4 + B * 4,
            "steps": n}


# --------------------------------------------------------------------------- the CPU oracle arm


def oracle_sample(w, start: int, rows: int):
    """Oracle sequences for the first `rows` rows, advanced to step `start`."""
    import oracle

    g = oracle.Grammar(w.ebnf, w.start)
    vocab = oracle.Vocab(w.vocab, w.eos)
    seqs = []
    for b in range(rows):
        s = oracle.Sequence_(g)
        s.advance(w.prefix_bytes[b])
        seqs.append(s)

    def advance(i):
        for b in range(rows):
            if w.reset_before[i, b]:
                seqs[b] = oracle.Sequence_(g)
            t = int(w.tokens[i, b])
            if t != w.eos and t >= 0:
                seqs[b].advance(w.vocab[t])

    for i in range(start):
        advance(i)
    return g, vocab, seqs, advance


def cpu_baseline(w, start: int, budget_s: float = 15.0):
    import oracle

    rows = min(w.batch, 16)
    g, vocab, seqs, advance = oracle_sample(w, start, rows)
    t0 = time.perf_counter()
    masks = 0
    i = start
    while time.perf_counter() - t0 < budget_s and i < w.steps:
        advance(i)
        for b in range(rows):
            seqs[b].mask(vocab)
            masks += 1
        i += 1
    dt = time.perf_counter() - t0
    return {"value": masks * w.V / dt, "unit": UNIT, "cores": oracle.max_threads(), "kind": "oracle",
            "ms_per_row_mask": dt / max(1, masks) * 1e3,
            "sample": "%d rows x %d steps of %s: advance + full-vocabulary mask per row, OpenMP over tokens" % (rows, i - start, w.name)}


def run_reference(args):
    import oracle

    if int(os.environ.get("RANK", "0")) != 0:
        return
    K, W = args.steps, args.warmup
    w = workloads.build(args.config, steps=K + W, batch=args.batch)
    rows = min(w.batch, 4)
    g, vocab, seqs, advance = oracle_sample(w, 0, rows)
    for i in range(W):
        advance(i)
        for b in range(rows):
            seqs[b].mask(vocab)
    t0 = time.perf_counter()
    for i in range(W, W + K):
        advance(i)
        for b in range(rows):
            seqs[b].mask(vocab)
    dt = time.perf_counter() - t0
    value = rows * w.V * K / dt
    cores = oracle.max_threads()
    sample = "each step: %d of the %d rows of %s, advance + full-vocabulary mask per row (CPU oracle)" % (rows, w.batch, w.name)
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": int(os.environ.get("WORLD_SIZE", "1")),
        "steps": K, "warmup": W, "ms_per_step": dt / K * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "u32", "data": "synthetic",
        "config": {"workload": w.name, "config": args.config, "batch": w.batch, "vocab": w.V, "logits": "bf16",
                   "l2": "not applicable (CPU oracle)", "state_cache": "none (every mask recomputed)",
                   "parallelism": "OpenMP over tokens"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=256)
    ap.add_argument("--warmup", type=int, default=16)
    ap.add_argument("--config", type=int, default=DEFAULT_CONFIG)
    ap.add_argument("--batch", type=int, default=None, help="override the config's batch size (not the headline workload)")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--cpu-seconds", type=float, default=15.0)
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
