#!/usr/bin/env python
"""Benchmark of the fused KVCache retrieval step (select + resolve + gather + attention) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl swarm|reference] [--workload c2_128k]

A step is one swarm_step over one batch of synthetic input (one layer).  The workload is the 128K
Llama-3-8B-shaped configuration.  Because one step touches less data than the L2 holds, the run
rotates over several independent data sets (pool, summaries, query) so consecutive steps never
re-read cached data.  Each step is replayed from a CUDA graph captured from the library call.

Prints ONE JSON line (rank 0).  N > 1 (torchrun) runs N independent replicas -- the path is
single-GPU by definition, so there is no data-path collective; only the timing barrier and the
max-over-ranks reduction use torch.distributed.

--impl reference times the CPU oracle (test infrastructure, plain C++) on the host cores instead.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "decode steps/sec of fused select+resolve+gather+attn; HBM GB/s (% of peak)"
UNIT = "steps/s"
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--impl", default="swarm", choices=["swarm", "reference"])
    ap.add_argument("--workload", default="c2_128k")
    ap.add_argument("--n-rot", type=int, default=0, help="independent data sets rotated through (0: enough to exceed 4x the L2)")
    ap.add_argument("--skip-per-workload", action="store_true", help="only the headline workload")
    ap.add_argument("--no-graph", action="store_true", help="call the library directly instead of replaying graphs")
    ap.add_argument("--skip-cpu-baseline", action="store_true")
    ap.add_argument("--attn-splits", type=int, default=0, help="key-range splits of the attention kernel (0: chosen from the shape)")
    ap.add_argument("--shard", default="none", choices=["none", "heads"],
                    help="heads: ONE step stream whose KV heads are spread over the ranks (strong scaling; the ranks "
                         "exchange the cluster flags once per step); default: independent replicas")
    return ap.parse_args()


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


# ------------------------------------------------------------------------------------------- clocks

class ClockSampler:
    """Samples SM clock and throttle reasons through NVML (read-only) while the timed regions run."""

    def __init__(self, index: int, period_s: float = 0.02):
        self.samples = []   # (t, sm_mhz, reasons_bitmask)
        self.max_mhz = None
        self._stop = threading.Event()
        self._thread = None
        self.ok = False
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
            self.ok = True
        except Exception:
            self.ok = False
        self.period = period_s

    def _read(self):
        nv = self.nv
        mhz = int(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
        try:
            reasons = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self.h))
        except Exception:
            reasons = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h))
        return mhz, reasons

    def _run(self):
        while not self._stop.is_set():
            try:
                mhz, reasons = self._read()
                self.samples.append((time.perf_counter(), mhz, reasons))
            except Exception:
                pass
            self._stop.wait(self.period)

    def start(self):
        if self.ok:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()

    def stop(self):
        if self._thread is not None:
            self._stop.set()
            self._thread.join()

    def summary(self, windows):
        if not self.ok or not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": ["unavailable"]}
        inside = [s for s in self.samples if any(a <= s[0] <= b for a, b in windows)] or self.samples
        mhz = sorted(s[1] for s in inside)
        bits = 0
        for s in inside:
            bits |= s[2]
        names = {0x1: "gpu_idle", 0x2: "applications_clocks_setting", 0x4: "sw_power_cap", 0x8: "hw_slowdown",
                 0x10: "sync_boost", 0x20: "sw_thermal_slowdown", 0x40: "hw_thermal_slowdown",
                 0x80: "hw_power_brake_slowdown", 0x100: "display_clock_setting"}
        reasons = [n for b, n in names.items() if bits & b and n != "gpu_idle"]
        return {"sm_mhz": mhz[len(mhz) // 2], "sm_max_mhz": self.max_mhz, "reasons": reasons,
                "samples_in_timed_region": len(inside)}


# ----------------------------------------------------------------------------------- byte accounting

def step_bytes(w, sel, n_sel):
    """Algorithmic bytes of one step (what the method must move), from the executed selection.
    summaries: every existing page's 512 B row per KV head, read once.
    kv (compulsory): K and V blocks of the distinct (request, kv head, page) triples selected by any head
    of the group; kv (nominal): one K and V block per selected (head, page) slot."""
    import numpy as np
    cfg = w.cfg
    S, d, Hkv, g = cfg.page_size, cfg.head_dim, cfg.n_kv_heads, cfg.group
    pages = -(-w.ctx_len.cpu().numpy().astype(np.int64) // S)
    summaries = int(pages.sum()) * Hkv * 2 * d * 2
    sel = sel.cpu().numpy()
    n_sel = n_sel.cpu().numpy()
    blk = S * d * 2 * 2
    distinct = 0
    for b in range(cfg.batch):
        for kv in range(Hkv):
            ids = [sel[b, h, : n_sel[b, h]] for h in range(kv * g, (kv + 1) * g)]
            distinct += len(np.unique(np.concatenate(ids)))
    nominal = int(n_sel.sum())
    small = cfg.batch * cfg.n_q_heads * (d * 2 + d * 4 + 4 + cfg.top_k * 4)
    return dict(summaries=summaries, kv_compulsory=distinct * blk, kv_nominal=nominal * blk, small=small)


# ------------------------------------------------------------------------------------------ swarm arm

WORKLOADS = ("c1_tiny", "c2_128k", "c3_batched", "c4_long", "c5_skewed")
# most data sets kept resident per workload (device memory: c5 is 33 GiB of pool per data set)
MAX_DATA_SETS = {"c1_tiny": 48, "c2_128k": 8, "c3_batched": 2, "c4_long": 2, "c5_skewed": 1}


def l2_bytes(dev) -> int:
    import torch
    return int(torch.cuda.get_device_properties(dev).L2_cache_size)


def build_signature() -> str:
    """Identifies the library that is running: version and a hash of its kernel sources."""
    import hashlib
    h = hashlib.sha256()
    csrc = os.path.join(ROOT, "paper_2603_17803_b200", "csrc")
    for name in sorted(os.listdir(csrc)):
        with open(os.path.join(csrc, name), "rb") as f:
            h.update(name.encode() + b"\0" + f.read())
    return h.hexdigest()[:16]


def captured_traffic(workload: str):
    """dram read + write bytes of one attention launch from the ncu capture summarised under profiles/ (a text
    file of `key: value` lines), if that capture was made from the kernel sources that are running now;
    (None, why) otherwise."""
    path = os.path.join(ROOT, "profiles", f"attn_kernel_{workload}_traffic.txt")
    try:
        with open(path) as f:
            ent = dict(line.split(":", 1) for line in f if ":" in line and not line.startswith("#"))
        ent = {k.strip(): v.strip() for k, v in ent.items()}
        total = int(ent["dram_bytes_read"]) + int(ent["dram_bytes_write"])
    except Exception:
        return None, "no capture on record for this workload"
    if ent.get("kernel_sources") != build_signature():
        return None, f"the capture of {ent.get('date')} belongs to other kernel sources ({ent.get('kernel_sources')})"
    return total, f"ncu capture of {ent.get('date')}, same kernel sources"


class Bench:
    """The data sets, sessions and graphs of one workload, and the timed loops over them."""

    def __init__(self, name, n_rot, rank, dev, stream, tail_stream, attn_splits=0, no_graph=False):
        import torch
        from paper_2603_17803_b200 import binding as B
        from paper_2603_17803_b200 import replicas
        from paper_2603_17803_b200 import workloads as W
        from paper_2603_17803_b200.session import Session
        self.torch, self.B = torch, B
        self.cfg = W.CONFIGS[name]
        self.n_rot, self.stream, self.tail_stream, self.no_graph = n_rot, stream, tail_stream, no_graph
        self.workloads, self.serial, self.tail = [], [], []
        for r in range(n_rot):      # every rank draws its own data sets (weak scaling: fixed work per GPU)
            w = W.generate(self.cfg, seed=replicas.replica_seed(rank, r), device=dev, step=r)
            self.workloads.append(w)
            a = Session(w)
            b = Session(w, ksum=a.ksum, tail_stream=tail_stream)
            for s_ in (a, b):
                if attn_splits > 0:
                    B.swarm_set_attn_splits(s_.ctx, attn_splits)
            self.serial.append(a)
            self.tail.append(b)
        torch.cuda.synchronize()

    def close(self):
        for s in self.serial + self.tail:
            s.close()

    def _graph(self, sessions, fn, n_calls, join):
        """A CUDA graph of n_calls consecutive calls, data sets in rotation (None with --no-graph or n_calls 0)."""
        torch = self.torch
        if self.no_graph or n_calls == 0:
            return None
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=self.stream):
            for i in range(n_calls):
                fn(sessions[i % self.n_rot])
            if join:
                for s in sessions:
                    s.tail_join(self.stream)
        return g

    def time_calls(self, sessions, fn, n_calls, *, join=False, warmup=0, min_ms=50.0, max_repeats=200, barrier=None):
        """Device time of exactly n_calls consecutive calls (CUDA events on the launching stream), repeated
        until min_ms of timed work has accumulated; returns (median, min, max) microseconds per call and the
        number of repeats.  Whole rotations go out as one graph launch each, the remainder as one more."""
        torch, stream, n_rot = self.torch, self.stream, self.n_rot
        with torch.cuda.stream(stream):
            for s in sessions:
                fn(s)
            if join:
                for s in sessions:
                    s.tail_join(stream)
            stream.synchronize()
            # up to 512 calls: the whole region is one graph; beyond that, graphs of 8 rotations and a remainder
            per_graph = n_calls if n_calls <= 512 else n_rot * 8
            g_full = self._graph(sessions, fn, per_graph, join)
            g_rem = self._graph(sessions, fn, n_calls % per_graph, join)

            def run():
                if self.no_graph:
                    for i in range(n_calls):
                        fn(sessions[i % n_rot])
                    if join:
                        for s in sessions:
                            s.tail_join(stream)
                    return
                for _ in range(n_calls // per_graph):
                    g_full.replay()
                if g_rem is not None:
                    g_rem.replay()

            for _ in range(max(1, -(-warmup // max(1, n_calls)))):
                run()
            times, total = [], 0.0
            while True:
                if barrier is not None:
                    barrier()
                stream.synchronize()
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(stream)
                run()
                e1.record(stream)
                if barrier is not None:
                    barrier()
                stream.synchronize()
                ms = e0.elapsed_time(e1)
                times.append(ms)
                total += ms
                if total >= min_ms or len(times) >= max_repeats:
                    break
        times.sort()
        per = [t * 1e3 / n_calls for t in times]
        return per[len(per) // 2], per[0], per[-1], len(per)


def measure_workload(name, args, rank, dev, stream, tail_stream, peak, *, steps, warmup, barrier=None, extras=False):
    """Everything reported for one workload: step time (strictly serial and with the overlapped tail), the stages
    alone, bytes and roofline fractions.  `extras`: also the step variants and the medoid-index step."""
    import torch
    from paper_2603_17803_b200 import binding as B
    cfg_probe = __import__("paper_2603_17803_b200.workloads", fromlist=["CONFIGS"]).CONFIGS[name]
    l2 = l2_bytes(dev)
    n_rot = args.n_rot if (args.n_rot and name == args.workload) else None
    # first guess of the bytes a step touches: summaries + half of the nominal K/V
    S, d, Hkv = cfg_probe.page_size, cfg_probe.head_dim, cfg_probe.n_kv_heads
    pages = cfg_probe.batch * (cfg_probe.max_pages() if not cfg_probe.ctx_range else (cfg_probe.ctx_range[0] + cfg_probe.ctx_range[1]) // (2 * S))
    guess = pages * Hkv * 2 * d * 2 + cfg_probe.batch * cfg_probe.n_q_heads * cfg_probe.top_k * S * d * 2
    if n_rot is None:
        n_rot = max(2 if guess < 4 * l2 else 1, min(MAX_DATA_SETS[name], -(-4 * l2 // max(1, guess))))
    bench = Bench(name, n_rot, rank, dev, stream, tail_stream, args.attn_splits, args.no_graph)
    cfg = bench.cfg
    step = lambda s: s.step(stream=stream)
    kw = dict(warmup=warmup, barrier=barrier)
    t_a = time.perf_counter()
    tail_us, tail_min, tail_max, tail_reps = bench.time_calls(bench.tail, step, steps, join=True, **kw)
    serial_us, serial_min, serial_max, serial_reps = bench.time_calls(bench.serial, step, steps, **kw)
    # the same overlapped-tail steps with the scorer's index prefetch switched on (swarm_set_index_prefetch): reported
    # beside the headline, never as it
    for s_ in bench.tail:
        bench.B.swarm_set_index_prefetch(s_.ctx, True)
    pre_us, pre_min, pre_max, _ = bench.time_calls(bench.tail, step, steps, join=True, **kw)
    for s_ in bench.tail:
        bench.B.swarm_set_index_prefetch(s_.ctx, False)
    t_b = time.perf_counter()
    n_loop = max(3 * n_rot, min(steps, 2000))
    attn_us = bench.time_calls(bench.serial, lambda s: s.sparse_attn_paged(stream=stream, reuse_last_selection=True), n_loop)[0]
    select_us = bench.time_calls(bench.serial, lambda s: s.select(stream=stream), n_loop)[0]
    resolve_us = bench.time_calls(bench.serial, lambda s: s.resolve(stream=stream), n_loop)[0]
    for s_ in bench.serial:
        s_.step(stream=stream)                            # leave a whole step's outputs in place
    torch.cuda.synchronize()
    status = max(s.status() for s in bench.serial + bench.tail)
    by = step_bytes(bench.workloads[0], bench.serial[0].o.sel, bench.serial[0].o.n_sel)
    alg = by["summaries"] + by["kv_compulsory"] + by["small"]
    nominal = by["summaries"] + by["kv_nominal"] + by["small"]
    attn_gbs = by["kv_compulsory"] / (attn_us * 1e-6) / 1e9
    out = {
        "workload": cfg.name, "us_per_step": tail_us, "us_per_step_min_max": [tail_min, tail_max], "repeats": tail_reps,
        "us_per_step_serial": serial_us, "us_per_step_serial_min_max": [serial_min, serial_max],
        "us_per_step_index_prefetch": pre_us, "us_per_step_index_prefetch_min_max": [pre_min, pre_max],
        "best_mode": "overlapped tail" if tail_us <= serial_us else "serial",
        "steps_timed": steps, "data_sets": n_rot,
        "bytes_per_step": {"algorithmic": alg, "nominal": nominal, **by},
        "hbm_gbs": alg / (tail_us * 1e-6) / 1e9,
        "hbm_frac_of_measured_copy": alg / (tail_us * 1e-6) / 1e9 / peak,
        "hbm_frac_of_nominal_8tbs": alg / (tail_us * 1e-6) / 1e9 / NOMINAL_HBM_GBS,
        "nominal_bytes_frac_of_nominal_8tbs": nominal / (tail_us * 1e-6) / 1e9 / NOMINAL_HBM_GBS,
        "serial_hbm_frac_of_measured_copy": alg / (serial_us * 1e-6) / 1e9 / peak,
        "stage_us_alone": {"select(score+topk)": select_us, "resolve": resolve_us, "attention_paged(+combine)": attn_us},
        "attention_alone": {"gbs_of_compulsory_kv": attn_gbs, "frac_of_measured_copy": attn_gbs / peak, "us": attn_us},
        "l2_policy": f"rotating {n_rot} independent data sets ({n_rot * alg / 1e6:.0f} MB touched per rotation, "
                     f"L2 {l2 / 1e6:.0f} MB)" if n_rot > 1 else
                     f"one data set: a step touches {alg / 1e6:.0f} MB, {alg / l2:.0f}x the {l2 / 1e6:.0f} MB L2",
        "device_status": status, "n_uniq_clusters": int(bench.serial[0].o.n_uniq[0]),
        "_windows": [(t_a, t_b)],
    }
    if cfg.n_layers > 1:
        out["note"] = (f"one layer-step; the configuration's step is {cfg.n_layers} sequential layers = "
                       f"{tail_us * cfg.n_layers / 1e3:.3f} ms")
    if extras:
        # the same step with the paper's own selector (medoid index, whole clusters retrieved): k_c clusters of
        # ~8 pages stand for the page step's top_k pages
        k_c = max(1, cfg.top_k // 8)
        for s_ in bench.serial:
            s_.enable_medoid_index(k_c)
        medoid_us = bench.time_calls(bench.serial, lambda s: s.step_medoid(stream=stream), n_loop)[0]
        # the page step with the optional parts of cluster resolution switched on, one at a time
        keep = []
        for s_ in bench.serial:
            n_c = s_.w.n_clusters
            g_ = torch.Generator(device="cpu").manual_seed(7)
            keep.append(dict(resident=(torch.rand(n_c, generator=g_) < 0.25).to(torch.uint8).to(dev),
                             freq=torch.zeros(n_c, dtype=torch.int32, device=dev),
                             score=torch.zeros(n_c, dtype=torch.float32, device=dev),
                             n_hit=torch.zeros(4, dtype=torch.int32, device=dev)))
            B.swarm_set_cache(s_.ctx, t_base=80.0, t_transfer=2.5, **keep[-1])
        cached_us = bench.time_calls(bench.serial, step, n_loop)[0]
        for s_ in bench.serial:
            B.swarm_set_cache(s_.ctx)
            s_.enable_submit_order()
        submit_us = bench.time_calls(bench.serial, step, n_loop)[0]
        for s_ in bench.serial:
            B.swarm_set_submit_order(s_.ctx, None, None)
            s_.step(stream=stream)
        torch.cuda.synchronize()
        out["step_variants_us"] = {"with_cache_state(25% resident: Eq. 8 filter, counters, Eq. 6)": cached_us,
                                   "with_submission_order(Sec. 5.1 batches)": submit_us}
        out["medoid_step"] = {"us_per_step": medoid_us, "top_k_clusters": k_c,
                              "note": "swarm_step_medoid on the same data sets: clusters scored by their medoid page, whole clusters attended"}
    return out, bench


def run_swarm(args):
    import torch
    from paper_2603_17803_b200 import replicas

    world, rank, local_rank = replicas.env_world()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU fallback")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    replicas.init("nccl", dev)
    K = args.steps if args.steps is not None else 20000
    Wm = max(3, args.warmup if args.warmup is not None else 50)
    peak, peak_kind = measured_peak()

    sampler = ClockSampler(local_rank)
    sampler.start()
    stream, tail_stream = torch.cuda.Stream(), torch.cuda.Stream()

    def barrier():
        replicas.barrier()
        torch.cuda.synchronize()

    head, bench = measure_workload(args.workload, args, rank, dev, stream, tail_stream, peak, steps=K, warmup=Wm,
                                   barrier=barrier, extras=True)
    cfg = bench.cfg
    windows = head.pop("_windows")

    # end to end: per-step data in pinned host memory, copies inside the timed region
    Bq, Hq, d, D = cfg.batch, cfg.n_q_heads, cfg.head_dim, cfg.n_queues
    q_host = [w.q.cpu().pin_memory() for w in bench.workloads]
    out_host = torch.empty((Bq, Hq, d), dtype=torch.float32).pin_memory()
    lse_host = torch.empty((Bq, Hq), dtype=torch.float32).pin_memory()
    n_host = torch.zeros(1, dtype=torch.int32).pin_memory()
    load_host = torch.zeros(D, dtype=torch.int32).pin_memory()
    K_e2e = max(200, min(K, 5000))
    sessions, n_rot = bench.serial, bench.n_rot
    with torch.cuda.stream(stream):
        for i in range(20):
            sessions[i % n_rot].step_host(q_host[i % n_rot], out_host, lse_host, n_host, load_host, stream)
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t_e = time.perf_counter()
        e0.record(stream)
        for i in range(K_e2e):
            sessions[i % n_rot].step_host(q_host[i % n_rot], out_host, lse_host, n_host, load_host, stream)
        e1.record(stream)
        barrier()
        t_f = time.perf_counter()
        ms_e2e = e0.elapsed_time(e1)
    windows.append((t_e, t_f))

    us, us_serial, us_pre, ms_e2e = replicas.max_over_ranks(
        [head["us_per_step"], head["us_per_step_serial"], head["us_per_step_index_prefetch"], ms_e2e], device=dev)
    ms = us * K / 1e3
    by = head["bytes_per_step"]
    traffic, traffic_source = captured_traffic(cfg.name)
    attn = head["attention_alone"]
    result = {
        "metric": METRIC, "value": replicas.aggregate_steps_per_s(world, K, ms), "unit": UNIT, "n_gpus": world, "steps": K,
        "warmup": Wm, "ms_per_step": us / 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": {"workload": cfg.name, "batch": cfg.batch, "n_q_heads": cfg.n_q_heads, "n_kv_heads": cfg.n_kv_heads,
                   "head_dim": cfg.head_dim, "context": cfg.max_ctx(), "page_size": cfg.page_size,
                   "top_k": cfg.top_k, "n_queues": cfg.n_queues, "n_topics": cfg.n_topics,
                   "parallelism": f"replicas x{world} (no data-path collective)",
                   "l2_policy": head["l2_policy"],
                   "launch": "library calls, no graph" if args.no_graph else
                             "CUDA graph replay of consecutive swarm_step calls (whole rotations of the data sets per graph). "
                             "value: overlapped tail (swarm_set_tail_stream) -- scoring, selection and attention of a step "
                             "run strictly after the attention of the step before; only the cluster resolution of a step "
                             "(uniq / queue_of / loads: the I/O schedule) runs beside the next step's scoring and selection, "
                             "every output of every step is computed and the graph joins the tail stream. "
                             "serial: the same steps with the resolution inside the step (nothing overlaps)",
                   "timing": f"exactly {K} steps per timed region (CUDA events on the launching stream, max over ranks); the region "
                             f"is repeated until 50 ms have been timed and the median is reported ({head['repeats']} repeats here)"},
        "serial": {"value": replicas.aggregate_steps_per_s(world, K, us_serial * K / 1e3), "unit": UNIT, "us_per_step": us_serial,
                   "hbm_frac_of_measured_copy": head["serial_hbm_frac_of_measured_copy"]},
        "index_prefetch": {"value": replicas.aggregate_steps_per_s(world, K, us_pre * K / 1e3), "unit": UNIT, "us_per_step": us_pre,
                           "note": "not the headline: the overlapped-tail steps with swarm_set_index_prefetch on -- the scorer's "
                                   "CTAs become resident while the previous step's attention kernel merges its partial results "
                                   "and ask for their first blocks of the page index (which does not depend on the queries) "
                                   "before they wait for that kernel; everything that reads q starts after it, as in `value`"},
        "us_per_step_min_max": head["us_per_step_min_max"],
        "hbm_gbs": head["hbm_gbs"], "hbm_frac_of_measured_copy": head["hbm_frac_of_measured_copy"],
        "hbm_frac_of_nominal_8tbs": head["hbm_frac_of_nominal_8tbs"],
        "nominal_bytes_frac_of_nominal_8tbs": head["nominal_bytes_frac_of_nominal_8tbs"],
        "bytes_per_step": by,
        "stage_us_alone": head["stage_us_alone"],
        "step_variants_us": head.get("step_variants_us"), "medoid_step": head.get("medoid_step"),
        "roofline": {"kernel": "attn_kernel<paged> (tensor-core split-K attention over the union of selected pages, merge included)",
                     "bound": "hbm", "achieved": attn["gbs_of_compulsory_kv"], "peak": peak,
                     "peak_kind": f"of {peak_kind} copy bandwidth", "unit": "GB/s", "frac": attn["frac_of_measured_copy"],
                     "traffic": traffic, "traffic_source": traffic_source,
                     "algorithmic_bytes_per_launch": by["kv_compulsory"], "avg_launch_us": attn["us"],
                     "nominal_bytes_per_launch": by["kv_nominal"], "nominal_gbs": by["kv_nominal"] / (attn["us"] * 1e-6) / 1e9},
        "e2e": {"value": replicas.aggregate_steps_per_s(world, K_e2e, ms_e2e), "unit": UNIT, "steps": K_e2e,
                "h2d_bytes_per_step": Bq * Hq * d * 2, "d2h_bytes_per_step": Bq * Hq * d * 4 + Bq * Hq * 4 + 4 + D * 4,
                "note": "swarm_step_host: q from pinned host memory, out/lse/n_uniq/queue_load read back; "
                        "the KV pool and its summaries are resident state, like weights"},
        "gpu_launches": K * 4,   # scorer, selection, cluster resolution (tail stream), attention
        "gpu_launches_per_step": 4,
        "device_status": head["device_status"],
        "n_uniq_clusters": head["n_uniq_clusters"],
        "kernel_sources": build_signature(),
    }
    cpu = None
    if rank == 0 and not args.skip_cpu_baseline and world == 1:
        cpu = cpu_baselines(bench.workloads[0], budget_s=6.0)
        result["cpu_baseline"] = cpu["all_cores"]
        result["cpu_baseline_one_thread"] = cpu["one_thread"]
    bench.close()
    del bench
    torch.cuda.empty_cache()

    # the other workloads, shorter runs (one GPU, rank 0's numbers; every rank runs them so the ranks stay in step)
    if not args.skip_per_workload:
        per = {}
        for name in WORKLOADS:
            if name == cfg.name:
                ent = {k: v for k, v in head.items() if not k.startswith("_")}
                if cpu is not None:
                    ent["cpu_baseline"] = cpu
            else:
                short = {"c1_tiny": 2000, "c3_batched": 400, "c4_long": 200, "c5_skewed": 60}.get(name, 400)
                ent, b2 = measure_workload(name, args, rank, dev, stream, tail_stream, peak, steps=short, warmup=max(3, short // 20))
                windows += ent.pop("_windows")
                if rank == 0 and not args.skip_cpu_baseline and world == 1:
                    ent["cpu_baseline"] = cpu_baselines(b2.workloads[0], budget_s=4.0)
                b2.close()
                del b2
                torch.cuda.empty_cache()
            per[name] = ent
        result["per_workload"] = per
    sampler.stop()
    result["clocks"] = sampler.summary(windows)
    if rank == 0:
        print(json.dumps(result))
    replicas.shutdown()


# ------------------------------------------------------------------------------------------ CPU oracle

def oracle_inputs(w):
    import numpy as np
    from paper_2603_17803_b200.workloads import bits_u16
    return dict(q=bits_u16(w.q), kv_pool=bits_u16(w.kv_pool), page_base=w.page_base.cpu().numpy(),
                ctx_len=w.ctx_len.cpu().numpy(), page2cluster=w.page2cluster.cpu().numpy(),
                cluster_base=w.cluster_base.cpu().numpy(),
                replica_mask=w.cluster_replica_mask.cpu().numpy().view(np.uint32),
                cluster_size=w.cluster_size.cpu().numpy().view(np.uint16))


def oracle_step_fn(w):
    import oracle
    cfg = w.cfg
    x = oracle_inputs(w)
    ksum = oracle.build_summaries(x["kv_pool"], x["page_base"], x["ctx_len"], cfg.n_kv_heads, cfg.head_dim,
                                  cfg.page_size)   # index build: outside the timed step, as on the GPU
    Pmax = int((-(-x["ctx_len"].astype("int64") // cfg.page_size)).max())

    def fn():
        return oracle.step(x["q"], ksum, x["kv_pool"], x["page_base"], x["ctx_len"], x["page2cluster"],
                           x["cluster_base"], x["replica_mask"], x["cluster_size"], Hkv=cfg.n_kv_heads,
                           S=cfg.page_size, k=cfg.top_k, D=cfg.n_queues, Pmax=Pmax)
    return fn


def oracle_sample(w, max_bytes=3 << 30):
    """(sample workload on the host, scale, description): the whole batch when its pool fits max_bytes, else
    requests picked evenly over the batch sorted by length -- a step of the whole batch costs `scale` times the
    sample's step (the oracle's stages are per request, except the cluster assignment, which is a small part)."""
    import numpy as np
    from paper_2603_17803_b200 import workloads as W
    cfg = w.cfg
    pages = (w.page_base[1:] - w.page_base[:-1]).cpu().numpy()
    per_page = cfg.n_kv_heads * 2 * cfg.page_size * cfg.head_dim * 2
    order = np.argsort(pages, kind="stable")
    n = cfg.batch
    while n > 1 and pages[order[np.linspace(0, cfg.batch - 1, n).round().astype(int)]].sum() * per_page > max_bytes:
        n -= 1
    pick = sorted(set(int(order[i]) for i in np.linspace(0, cfg.batch - 1, n).round().astype(int)))
    if len(pick) == cfg.batch:
        return W.subset_requests(w, range(cfg.batch)), 1.0, f"all {cfg.batch} requests"
    scale = float(pages.sum()) / float(pages[pick].sum())
    return (W.subset_requests(w, pick), scale,
            f"requests {pick} of {cfg.batch} (evenly spaced by length), time scaled by pages {scale:.2f}x")


def cpu_baselines(w, budget_s: float):
    """The oracle as it stands on this host's cores, on (a sample of) the same workload: whole steps at one
    thread and at all cores."""
    import oracle
    sample, scale, what = oracle_sample(w)
    fn = oracle_step_fn(sample)
    out = {}
    n_cores = len(os.sched_getaffinity(0))
    for key, threads in (("all_cores", n_cores), ("one_thread", 1)):
        cores = oracle.set_threads(threads)
        fn()
        n, t0 = 0, time.perf_counter()
        while True:
            fn()
            n += 1
            el = time.perf_counter() - t0
            if el >= budget_s or n >= 1000:
                break
        out[key] = {"value": n / (el * scale), "unit": UNIT, "cores": cores, "kind": "oracle",
                    "sample": f"{n} oracle steps over {what} of {w.cfg.name} (all {w.cfg.n_q_heads} heads), "
                              f"OpenMP over (request, head) units, {el:.1f} s"}
    oracle.set_threads(n_cores)
    return out


def run_sharded(args):
    """--shard heads: every rank holds the K/V of its own KV heads of the SAME workload; a step is selection,
    all-reduce(max) of the cluster flags, attention + resolution (paper_2603_17803_b200.sharding).  Plain launches,
    no graph (the collective sits between the two halves)."""
    import torch
    from paper_2603_17803_b200 import replicas, sharding
    from paper_2603_17803_b200 import workloads as W
    from paper_2603_17803_b200.session import Session

    world, rank, local_rank = replicas.env_world()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU fallback")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    replicas.init("nccl", dev)
    K = args.steps if args.steps is not None else 5000
    Wm = max(3, args.warmup if args.warmup is not None else 50)
    cfg = W.CONFIGS[args.workload]
    n_rot = args.n_rot or 8
    sampler = ClockSampler(local_rank)
    sampler.start()
    sessions = []
    for r in range(n_rot):                             # the same data sets on every rank, each keeps its heads
        w = W.generate(cfg, seed=r, device=dev, step=r)
        sessions.append(Session(sharding.shard_workload(w, rank, world)))
        del w
    torch.cuda.synchronize()
    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        for i in range(Wm):
            sharding.sharded_step(sessions[i % n_rot], stream)
        replicas.barrier()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t_a = time.perf_counter()
        e0.record(stream)
        for i in range(K):
            sharding.sharded_step(sessions[i % n_rot], stream)
        e1.record(stream)
        replicas.barrier()
        torch.cuda.synchronize()
        t_b = time.perf_counter()
        ms = e0.elapsed_time(e1)
    sampler.stop()
    ms, = replicas.max_over_ranks([ms], device=dev)
    status = max(s.status() for s in sessions)
    n_flags = int(sessions[0].cluster_flags().numel())
    if rank == 0:
        print(json.dumps({
            "metric": METRIC, "value": K / (ms * 1e-3), "unit": UNIT, "n_gpus": world, "steps": K, "warmup": Wm,
            "ms_per_step": ms / K, "higher_is_better": True, "scaling": "strong", "vs_baseline": None, "dtype": "bf16",
            "data": "synthetic",
            "config": {"workload": cfg.name, "parallelism": f"kv-head shards x{world}: one all-reduce(max) of {n_flags} "
                                                             "cluster-flag bytes per step, every rank schedules the union",
                       "l2_policy": f"rotating {n_rot} independent data sets", "launch": "plain launches, no graph"},
            "gpu_launches": K * 3, "device_status": status, "clocks": sampler.summary([(t_a, t_b)])}))
    replicas.shutdown()


def run_reference(args):
    """--impl reference: the CPU oracle on the host cores, same config / metric / unit."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    from paper_2603_17803_b200 import workloads as W
    cfg = W.CONFIGS[args.workload]
    K = args.steps if args.steps is not None else 5
    Wm = args.warmup if args.warmup is not None else 1
    w = W.generate(cfg, seed=0, device="cpu")
    cores = oracle.set_threads(len(os.sched_getaffinity(0)))
    fn = oracle_step_fn(w)
    t0 = time.perf_counter()
    fn()
    t_step = time.perf_counter() - t0
    # bounded run: if K whole steps would exceed the budget, a step is a sample of the query heads
    budget = 150.0
    frac = min(1.0, budget / max(1e-9, (K + Wm) * t_step))
    heads = max(1, int(cfg.n_q_heads * frac))
    if heads < cfg.n_q_heads:
        import dataclasses
        g = cfg.group
        heads = max(g, heads // g * g)                # whole KV groups
        cfg_s = dataclasses.replace(cfg, n_q_heads=heads, n_kv_heads=heads // g)
        w_s = dataclasses.replace(w, cfg=cfg_s, q=w.q[:, :heads].contiguous(),
                                  kv_pool=w.kv_pool[:, : heads // g].contiguous())
        fn = oracle_step_fn(w_s)
    scale = cfg.n_q_heads / heads
    for _ in range(Wm):
        fn()
    t0 = time.perf_counter()
    for _ in range(K):
        fn()
    el = (time.perf_counter() - t0) * scale
    value = K / el
    sample = (f"each step = {heads} of {cfg.n_q_heads} query heads of {cfg.name} "
              f"(time scaled by {scale:.2f}), {K} steps")
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": int(os.environ.get("WORLD_SIZE", "1")),
        "steps": K, "warmup": Wm, "ms_per_step": el / K * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": cfg.name, "batch": cfg.batch, "n_q_heads": cfg.n_q_heads, "n_kv_heads": cfg.n_kv_heads,
                   "head_dim": cfg.head_dim, "context": cfg.max_ctx(), "page_size": cfg.page_size, "top_k": cfg.top_k,
                   "n_queues": cfg.n_queues, "n_topics": cfg.n_topics},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


if __name__ == "__main__":
    a = parse_args()
    if a.impl == "reference":
        run_reference(a)
    elif a.shard == "heads":
        run_sharded(a)
    else:
        run_swarm(a)
