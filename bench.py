#!/usr/bin/env python
"""Benchmark of the vocabulary-mask path: one "step" = one decoding step of the whole batch
(row resets the stream asks for, fmt_state_advance with the chosen tokens, fmt_fill_and_apply on
that step's logits).  Metric: vocab-mask token-checks per second = batch * V * steps / time.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config C] [--repeats R] [--passes P] [--impl ours|reference]

The K timed steps are repeated R times, every repeat from empty caches and a fresh replay of the
prefixes and the W warm-up steps; the line's value is the median repeat, with CUDA events around
every step (latency_ms).  After that the same token stream is run P - 1 more times with the caches
kept (passes).  With --gpus N > 1 the script is launched by torch.distributed.run, one rank per GPU; every rank
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
DEFAULT_CONFIG = 5
L2_BYTES = 126 * 1024 * 1024


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
        self._stop.clear()
        self._thread = threading.Thread(target=self._run, daemon=True)
        self._thread.start()

    def pause(self):
        self._stop.set()
        if self._thread:
            self._thread.join(timeout=6)
            self._thread = None

    def stop(self) -> dict:
        self.pause()
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

    def __init__(self, w: workloads.Workload, device, roots: bool = False, cache: bool = True, ring_bytes: int = int(1.6 * L2_BYTES)):
        import torch

        import paper_2506_01151_b200 as fmt

        self.torch, self.fmt, self.w, self.device = torch, fmt, w, device
        self.grammar = fmt.Grammar(w.ebnf, w.start, w.vocab, w.eos)
        self.state = fmt.State(self.grammar, w.batch, roots=roots, cache=cache)
        self.roots = roots
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
        self.events = []

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
        # advance; plan, [entry look-up (2), sweep of new entries, its collection, job set-up], trie sweep, publish, mask+apply
        self.launches += 10 if self.roots else 5

    def restart(self, warmup: int, clear_caches: bool):
        """Back to the start of the token stream: all rows reset, prefixes fed, `warmup` untimed steps."""
        s = self.stream.cuda_stream
        if clear_caches:
            self.state.cache_clear(stream=s)
            self.state.ci_cache_clear(stream=s)
        self.state.reset(stream=s)
        self.feed_prefix()
        for i in range(warmup):
            self.step(i)
        self.torch.cuda.synchronize(self.device)

    def timed(self, start: int, n: int):
        """Steps start .. start+n-1 with an event after every step, on the stream the kernels run on:
        total milliseconds and the n per-step durations."""
        torch = self.torch
        while len(self.events) < n + 1:
            self.events.append(torch.cuda.Event(enable_timing=True))
        ev = self.events
        ev[0].record(self.stream)
        for k in range(n):
            self.step(start + k)
            ev[k + 1].record(self.stream)
        torch.cuda.synchronize(self.device)
        return ev[0].elapsed_time(ev[n]), [ev[k].elapsed_time(ev[k + 1]) for k in range(n)]


def percentile(xs, q):
    s = sorted(xs)
    return s[min(len(s) - 1, int(q * len(s)))]


def stat_delta(a, b, keys):
    return {k: b[k] - a[k] for k in keys}


STAT_KEYS = ["fills", "fills_computed", "fills_from_cache", "fills_shared", "rows_mask_only", "rows_from_root", "rows_plain",
             "root_sweeps", "sweep_transitions", "sweep_states", "walk_transitions", "walk_states", "walk_frames",
             "big_mode_units", "steps_advanced", "advances_cached", "earley_step_cycles", "capacity_errors", "fills_aborted"]


def read_traffic(config: int, kernel: str):
    """dram__bytes_read.sum + dram__bytes_write.sum per launch of `kernel` on workload `config`, from the
    table of ncu captures kept under profiles/ (None if there is no line for it)."""
    try:
        with open(os.path.join(ROOT, "profiles", "dram_traffic.txt")) as f:
            for line in f:
                p = line.split("#")[0].split()
                if len(p) >= 3 and p[0] == str(config) and p[1] == kernel:
                    return float(p[2])
    except OSError:
        pass
    return None


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
    K, W, R = args.steps, args.warmup, max(1, args.repeats)
    w = workloads.build(args.config, steps=K + W, batch=args.batch)
    drv = Driver(w, device, roots=args.roots)
    units = float(w.batch) * w.V * K
    sampler = ClockSampler(local)

    # ---- R repeats of the same work: empty caches, prefixes, W untimed steps, then EXACTLY K timed steps
    reps = []
    for r in range(R):
        drv.restart(W, clear_caches=r > 0)  # (the first repeat starts from a new state: its caches are empty)
        stats0 = drv.state.stats()
        drv.launches = 0
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize(device)
        sampler.start()
        drv.state.read_profile()
        drv.state.set_profiling(True)
        total_ms, per_step = drv.timed(W, K)
        if world > 1:
            dist.barrier()
        sampler.pause()
        series = {name: [float(x) for x in drv.state.read_profile_series(kind)]
                  for kind, name in ((0, "advance"), (1, "sweep"), (2, "masking"))}
        prof = drv.state.read_profile()
        drv.state.set_profiling(False)
        t_ms, total_units = aggregate_over_ranks(total_ms, units, dist if world > 1 else None)
        reps.append({"t_ms": t_ms, "units": total_units, "per_step": per_step, "prof": prof, "launches": drv.launches, "series": series,
                     "stats": stat_delta(stats0, drv.state.stats(), STAT_KEYS)})
    clocks = sampler.stop()
    # ---- once more, untimed, with the cycle counter read around every Earley step (it slows the sweeps a little)
    drv.restart(W, clear_caches=True)
    stats0 = drv.state.stats()
    drv.state.set_profiling(True, step_cycles=True)
    drv.timed(W, K)
    prof_cyc = drv.state.read_profile()
    drv.state.set_profiling(False)
    st_cyc = stat_delta(stats0, drv.state.stats(), STAT_KEYS)
    order = sorted(range(R), key=lambda r: reps[r]["t_ms"])
    med = reps[order[(R - 1) // 2]]  # the median repeat (the lower one of two) is the one reported in full
    t_ms, total_units, prof, st = med["t_ms"], med["units"], med["prof"], med["stats"]

    cold = cold_all = e2e = passes = cache_off = None
    stats_end = drv.state.stats()
    if rank == 0:
        if world == 1 and args.passes > 1:
            passes = measure_passes(drv, W, K, args.passes, med)
        stats_end = drv.state.stats()
        cold = measure_cold(drv, w, W, min(K, 16), clear_ci=False)
        cold_all = measure_cold(drv, w, W, min(K, 16), clear_ci=True)
        e2e = measure_e2e(drv, w, W, min(K, 64))
        if world == 1:
            cache_off = measure_cache_off(w, device, W, min(K, 32))
    if world > 1:
        dist.barrier()
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    info = drv.grammar.info()
    peak, peak_kind = measured_peaks()
    B, V, Wm = w.batch, w.V, info.mask_words
    sm_mhz = clocks["sm_mhz"] or 1900.0
    # ---- algorithmic bytes per launch of each kind of kernel: what the method itself must move through HBM
    trie_bytes = info.trie_nodes * (1 + 4 + 1) + 4 * V  # node byte, parent, depth; token -> node
    jobs = st["fills_computed"]
    sweep_jobs = st["rows_from_root"] + st["rows_plain"]
    sweep_bytes = trie_bytes + (sweep_jobs / max(1, K)) * (4 * Wm + 2048)  # + per job: its mask row and its chart
    apply_rw = B * (4 * Wm + 2 * 2 * V)   # mask words read, logits read and written
    apply_wo = B * (4 * Wm + 2 * V)       # if the logits only had to be written
    kinds = {
        ("fill_kernel" if drv.roots else "sweep_kernel"): (prof["sweep_ms"], prof["sweep_launches"], sweep_bytes),
        "sweep_kernel (new entries)": (prof["roots_ms"], prof["roots_launches"], trie_bytes),
        "gather_apply_kernel": (prof["apply_ms"], prof["apply_launches"], apply_rw),
        "advance_kernel": (prof["advance_ms"], prof["advance_launches"], B * 2 * 4 * 256),
    }
    dom = max(kinds, key=lambda k: kinds[k][0])
    d_ms, d_n, d_bytes = kinds[dom]
    avg_ms = d_ms / max(1, d_n)
    achieved = d_bytes / (avg_ms * 1e-3) / 1e9 if avg_ms > 0 else 0.0
    # ---- the other bound of the trie sweep: Earley steps.  Each step is one warp's work; the sweep kernels keep
    # `resident_warps` warps on the GPU, so steps * cycles per step / (resident warps * SM clock) is the time the
    # sweeps would take if every warp did nothing but Earley steps from start to end.
    steps_earley = st_cyc["sweep_transitions"] + st_cyc["walk_transitions"]
    resident_warps = 148 * 24
    earley_ms = st_cyc["earley_step_cycles"] / (resident_warps * sm_mhz * 1e3) if steps_earley else 0.0
    sweeps_ms = prof_cyc["sweep_ms"] + prof_cyc["roots_ms"]
    second = {
        "bound": "latency (Earley steps)", "earley_steps_per_step": steps_earley / K,
        "earley_steps_per_computed_row": steps_earley / max(1, st_cyc["fills_computed"]),
        "cycles_per_earley_step": st_cyc["earley_step_cycles"] / max(1, steps_earley), "resident_warps": resident_warps,
        "sm_mhz": sm_mhz, "all_warps_busy_ms_per_step": earley_ms / K, "sweeps_ms_per_step": sweeps_ms / K,
        "frac": earley_ms / sweeps_ms if sweeps_ms > 0 else None,
        "what": "measured in a run of its own (reading the cycle counter around every step slows the sweeps): warp-cycles "
                "spent inside Earley steps / (resident warps x SM clock) = the sweeps' time if no warp ever waited for a "
                "trie level, a queue or a barrier; frac = that time / the sweeps' time in the same run",
    }
    floor_rw = (apply_rw + trie_bytes) / (peak * 1e9) * 1e3
    floor_wo = (apply_wo + trie_bytes) / (peak * 1e9) * 1e3
    ms_step = t_ms / K
    roofline = {
        "bound": "hbm", "kernel": dom, "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
        "traffic": read_traffic(args.config, dom.split()[0]), "peak_source": peak_kind + " copy bandwidth",
        "avg_launch_us": avg_ms * 1e3, "bytes_per_launch": d_bytes,
        "per_kernel_ms": {k: v[0] for k, v in kinds.items()},
        "per_kernel_ms_per_step": {k: v[0] / K for k, v in kinds.items()},
        "hbm_floor_ms_per_step": {"read_write": floor_rw, "write_only": floor_wo,
                                  "what": "trie once + mask words + logits (read and written | written only) at the peak"},
        "step_frac_of_hbm_floor": {"read_write": floor_rw / ms_step, "write_only": floor_wo / ms_step},
        "gather_apply_gbs": apply_rw / (prof["apply_ms"] / max(1, prof["apply_launches"]) * 1e-3) / 1e9 if prof["apply_ms"] > 0 else None,
        "second_bound": second,
    }
    ms_list = [r["t_ms"] / K for r in reps]
    fills = max(1, st["fills"])
    states = max(1, stats_end["states_cached"])
    out = {
        "metric": METRIC, "value": total_units / (t_ms * 1e-3), "unit": UNIT, "n_gpus": world, "steps": K, "warmup": W,
        "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "u32",
        "data": "synthetic",
        "config": {"workload": w.name, "config": args.config, "batch": B, "vocab": V, "logits": "bf16",
                   "l2": "logits cycle through a ring of %d buffers (%.0f MB) > 126 MB L2" % (drv.n_ring, drv.n_ring * B * V * 2 / 1e6),
                   "state_cache": "on, empty at the start of every repeat (the paper's state cache; per-pass numbers under 'passes')",
                   "context_independent_cache": "on" if drv.roots else "off",
                   "parallelism": "replicas" if world > 1 else "single"},
        "repeats": {"n": R, "ms_per_step": ms_list, "median": statistics.median(ms_list), "min": min(ms_list), "max": max(ms_list),
                    "what": "each repeat: caches emptied, prefixes fed, W untimed steps, K timed steps; value = the median repeat"},
        "latency_ms": {"p50": percentile(med["per_step"], 0.50), "p90": percentile(med["per_step"], 0.90),
                       "p99": percentile(med["per_step"], 0.99), "max": max(med["per_step"]), "min": min(med["per_step"]),
                       "what": "per decoding step (advance + fill + masking of B rows), CUDA events around every step of the median repeat"},
        "kernel_latency_ms": {name: ({"p50": percentile(xs, 0.5), "p99": percentile(xs, 0.99), "max": max(xs), "launches": len(xs)} if xs else None)
                              for name, xs in med["series"].items()},
        "clocks": clocks, "e2e": e2e, "gpu_launches": med["launches"], "roofline": roofline,
        "cache": {"fills": st["fills"], "computed": jobs, "from_state_cache": st["fills_from_cache"], "shared_within_fill": st["fills_shared"],
                  "hit_rate": 1.0 - jobs / fills,
                  "computed_by": {"context_independent_row_only": st["rows_mask_only"], "sweep_in_frames": st["rows_from_root"],
                                  "sweep_from_chart": st["rows_plain"]},
                  "new_entries_swept": st["root_sweeps"], "entries": stats_end["roots"],
                  "earley_steps": {"rows": st["walk_transitions"], "new_entries": st["sweep_transitions"]},
                  "states_cached": stats_end["states_cached"], "chart_items_max": stats_end["chart_items_max"],
                  "chart_sets_max": stats_end["chart_sets_max"], "capacity_errors": stats_end["capacity_errors"],
                  "fills_aborted": stats_end["fills_aborted"], "big_mode": st["big_mode_units"],
                  "advances": st["steps_advanced"], "advances_from_cache": st["advances_cached"]},
        "memory": {"device_bytes": stats_end["device_bytes"], "states_cached": stats_end["states_cached"],
                   "state_pool_bytes_used": 4 * stats_end["pool_words_used"], "mask_rows_cached": stats_end["mask_rows_cached"],
                   "bytes_per_cached_state": (4 * stats_end["pool_words_used"] + 4 * Wm * stats_end["mask_rows_cached"]) / states},
        "passes": passes, "cold": cold, "cold_all": cold_all, "cache_off": cache_off,
        "grammar": {"nonterminals": info.n_nonterminals, "rules": info.n_rules, "dotted": info.n_dotted,
                    "trie_nodes": info.trie_nodes, "trie_depth": info.trie_depth, "byte_classes": info.n_byte_classes,
                    "automata": info.n_automata, "automaton_states": info.n_automaton_states},
    }
    if not args.no_cpu_baseline and world == 1:
        out["cpu_baseline"] = cpu_baseline(w, W, budget_s=args.cpu_seconds)
    else:
        out["cpu_baseline"] = None
    print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


def measure_passes(drv: "Driver", W: int, K: int, n_passes: int, first):
    """The same token stream again and again with the caches kept: pass 1 is a repeat from empty caches, pass p
    finds what passes 1..p-1 left."""
    out = [{"pass": 1, "ms_per_step": first["t_ms"] / K, "hit_rate": 1.0 - first["stats"]["fills_computed"] / max(1, first["stats"]["fills"]),
            "computed": first["stats"]["fills_computed"], "new_entries_swept": first["stats"]["root_sweeps"],
            "earley_steps": first["stats"]["walk_transitions"] + first["stats"]["sweep_transitions"],
            "p50_ms": percentile(first["per_step"], 0.5), "p99_ms": percentile(first["per_step"], 0.99)}]
    # the last repeat has left the caches as one pass leaves them
    for p in range(2, n_passes + 1):
        drv.restart(W, clear_caches=False)
        s0 = drv.state.stats()
        total_ms, per_step = drv.timed(W, K)
        d = stat_delta(s0, drv.state.stats(), STAT_KEYS)
        out.append({"pass": p, "ms_per_step": total_ms / K, "hit_rate": 1.0 - d["fills_computed"] / max(1, d["fills"]),
                    "computed": d["fills_computed"], "new_entries_swept": d["root_sweeps"],
                    "earley_steps": d["walk_transitions"] + d["sweep_transitions"],
                    "p50_ms": percentile(per_step, 0.5), "p99_ms": percentile(per_step, 0.99)})
    return out


def measure_cache_off(w, device, W: int, n: int):
    """The same steps on a state created without the state cache (Section 5.2 switched off): every fill
    computes every row that is not finished."""
    import torch

    drv = Driver(w, device, cache=False)
    drv.restart(W, clear_caches=False)
    total_ms, per_step = drv.timed(W, n)
    st = drv.state.stats()
    out = {"steps": n, "ms_per_step": total_ms / n, "p50_ms": percentile(per_step, 0.5), "p99_ms": percentile(per_step, 0.99),
           "token_checks_per_s": w.batch * w.V * n / (total_ms * 1e-3), "fills_from_cache": st["fills_from_cache"],
           "what": "advance + fill + masking per step with fmt_state_options.cache_disable = 1"}
    drv.state.close()
    del drv
    torch.cuda.empty_cache()
    return out


def measure_cold(drv: "Driver", w, start: int, n: int, clear_ci: bool):
    """ms per fill when every row's mask is recomputed: the state cache is emptied before each fill, and with
    `clear_ci` the cache of context-independent entries too."""
    torch = drv.torch
    s = drv.stream.cuda_stream
    mask = torch.zeros((w.batch, drv.grammar.mask_words), dtype=torch.int32, device=drv.device)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    times = []
    s0 = drv.state.stats()
    for i in range(n):
        drv.state.cache_clear(stream=s)
        if clear_ci:
            drv.state.ci_cache_clear(stream=s)
        e0.record(drv.stream)
        drv.state.fill_mask(mask, stream=s)
        e1.record(drv.stream)
        torch.cuda.synchronize(drv.device)
        times.append(e0.elapsed_time(e1))
    d = stat_delta(s0, drv.state.stats(), STAT_KEYS)
    return {"fills": n, "ms_per_fill": statistics.median(times), "min": min(times), "max": max(times),
            "rows_computed_per_fill": d["fills_computed"] / n,
            "earley_steps_per_computed_row": (d["walk_transitions"] + d["sweep_transitions"]) / max(1, d["fills_computed"]),
            "token_checks_per_s": w.batch * w.V / (statistics.median(times) * 1e-3),
            "what": "fmt_fill_mask with the state cache emptied before each call%s: every distinct row state is computed"
                    % (" and the context-independent entries too" if clear_ci else ", context-independent entries kept")}


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
    # the same rows with the oracle's CPU Compact (Section 4.2.3), for the sizes of pruned against full charts
    n_pruned = min(rows, 4)
    pruned = []
    for b in range(n_pruned):
        s = oracle.Sequence_(g, pruned=True)
        s.advance(w.prefix_bytes[b])
        pruned.append(s)
    for i in range(start):
        for b in range(n_pruned):
            if w.reset_before[i, b]:
                pruned[b] = oracle.Sequence_(g, pruned=True)
            t = int(w.tokens[i, b])
            if t != w.eos and t >= 0:
                pruned[b].advance(w.vocab[t])
    sizes = {"full_items_max": 0, "full_sets_max": 0, "pruned_items_max": 0, "pruned_sets_max": 0}

    def note_sizes():
        for b in range(n_pruned):
            sizes["full_items_max"] = max(sizes["full_items_max"], seqs[b].total_items)
            sizes["full_sets_max"] = max(sizes["full_sets_max"], seqs[b].num_sets)
            sizes["pruned_items_max"] = max(sizes["pruned_items_max"], pruned[b].total_items)
            sizes["pruned_sets_max"] = max(sizes["pruned_sets_max"], pruned[b].num_sets)

    note_sizes()
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
    for k in range(start, i):  # (outside the timed part) the pruned copies follow, then both are measured
        for b in range(n_pruned):
            if w.reset_before[k, b]:
                pruned[b] = oracle.Sequence_(g, pruned=True)
            t = int(w.tokens[k, b])
            if t != w.eos and t >= 0:
                pruned[b].advance(w.vocab[t])
    note_sizes()
    t1 = time.perf_counter()
    seqs[0].mask(vocab, threads=1)
    single = w.V / (time.perf_counter() - t1)
    sizes["what"] = ("items and Earley sets of the oracle's charts for %d of the sampled rows, full chart against the chart "
                     "after the oracle's Compact (the paper's maximum-memory comparison)" % n_pruned)
    return {"value": masks * w.V / dt, "unit": UNIT, "cores": oracle.max_threads(), "kind": "oracle",
            "ms_per_row_mask": dt / max(1, masks) * 1e3, "single_thread_value": single, "chart_sizes": sizes,
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
    ap.add_argument("--repeats", type=int, default=5, help="repeats of the timed K steps, each from empty caches (value = the median)")
    ap.add_argument("--passes", type=int, default=10, help="passes over the token stream with the caches kept (1 GPU only; 0 or 1: none)")
    ap.add_argument("--roots", action="store_true", help="switch the cache of context-independent entries on (off by default)")
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
