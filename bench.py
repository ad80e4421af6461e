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
# dram__bytes_read.sum + dram__bytes_write.sum of one attn_kernel launch at the default workload (c2_128k),
# from the ncu capture summarised in profiles/; reported only for that workload.
ATTN_TRAFFIC_BYTES_NCU = 33_072_128 + 12_544   # profiles/launch_list_c2_128k.md: dram read + write of attn_kernel<16,paged>


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--impl", default="swarm", choices=["swarm", "reference"])
    ap.add_argument("--workload", default="c2_128k")
    ap.add_argument("--n-rot", type=int, default=8, help="independent data sets rotated through")
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

def run_swarm(args):
    import torch
    from paper_2603_17803_b200 import replicas
    from paper_2603_17803_b200 import workloads as W
    from paper_2603_17803_b200.session import Session
    from paper_2603_17803_b200 import binding as B

    world, rank, local_rank = replicas.env_world()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU fallback")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    replicas.init("nccl", dev)
    K = args.steps if args.steps is not None else 20000
    Wm = args.warmup if args.warmup is not None else 50
    cfg = W.CONFIGS[args.workload]

    sampler = ClockSampler(local_rank)
    sampler.start()

    # independent data sets; every rank draws its own (weak scaling: fixed work per GPU)
    sessions, workloads = [], []
    for r in range(args.n_rot):
        w = W.generate(cfg, seed=replicas.replica_seed(rank, r), device=dev, step=r)
        workloads.append(w)
        sessions.append(Session(w))
        if args.attn_splits > 0:
            B.swarm_set_attn_splits(sessions[-1].ctx, args.attn_splits)
    torch.cuda.synchronize()
    stream = torch.cuda.Stream()

    def barrier():
        replicas.barrier()
        torch.cuda.synchronize()

    graphs = []
    cycle_graph = None
    with torch.cuda.stream(stream):
        for s in sessions:
            s.step(stream=stream)
        stream.synchronize()
        if not args.no_graph:
            for s in sessions:
                g = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g, stream=stream):
                    s.step(stream=stream)
                graphs.append(g)
            # one graph holding a whole rotation (n_rot consecutive steps): one launch per n_rot steps
            cycle_graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(cycle_graph, stream=stream):
                for s in sessions:
                    s.step(stream=stream)

        def one_step(i):
            if graphs:
                graphs[i % args.n_rot].replay()
            else:
                sessions[i % args.n_rot].step(stream=stream)

        def run_steps(n):
            """Exactly n steps, rotating over the data sets; whole rotations go out as one graph launch."""
            i = 0
            if cycle_graph is not None:
                for _ in range(n // args.n_rot):
                    cycle_graph.replay()
                i = n - n % args.n_rot
            for j in range(i, n):
                one_step(j)

        run_steps(Wm)
        barrier()
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t_a = time.perf_counter()
        ev0.record(stream)
        run_steps(K)
        ev1.record(stream)
        barrier()
        t_b = time.perf_counter()
        ms = ev0.elapsed_time(ev1)

        # the dominant kernel (attention straight from the pool) and the other stages timed alone: one graph
        # holds one call per data set (so the host's launch cost is off the clock), replayed back to back
        def time_loop(fn, n):
            for s_ in sessions:
                fn(s_)
            stream.synchronize()
            if args.no_graph:
                def go():
                    for s_ in sessions:
                        fn(s_)
            else:
                g_ = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g_, stream=stream):
                    for s_ in sessions:
                        fn(s_)
                go = g_.replay
            reps = max(1, n // args.n_rot)
            go()
            stream.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            for _ in range(reps):
                go()
            e1.record(stream)
            stream.synchronize()
            return e0.elapsed_time(e1) / (reps * args.n_rot) * 1e3    # microseconds per call

        n_loop = max(3 * args.n_rot, min(K, 2000))
        t_c = time.perf_counter()
        attn_us = time_loop(lambda s: s.sparse_attn_paged(stream=stream, reuse_last_selection=True), n_loop)
        select_us = time_loop(lambda s: s.select(stream=stream), n_loop)
        resolve_us = time_loop(lambda s: s.resolve(stream=stream), n_loop)
        # the same step with the paper's own selector (medoid index, whole clusters retrieved): k_c clusters of
        # ~8 pages stand for the page step's top_k pages
        k_c = max(1, cfg.top_k // 8)
        for s_ in sessions:
            s_.enable_medoid_index(k_c)
        medoid_us = time_loop(lambda s: s.step_medoid(stream=stream), n_loop)
        # the page step with the optional parts of cluster resolution switched on, one at a time
        cache_state = []
        for s_ in sessions:
            n_c = s_.w.n_clusters
            g_ = torch.Generator(device="cpu").manual_seed(7)
            cache_state.append(dict(resident=(torch.rand(n_c, generator=g_) < 0.25).to(torch.uint8).to(dev),
                                    freq=torch.zeros(n_c, dtype=torch.int32, device=dev),
                                    score=torch.zeros(n_c, dtype=torch.float32, device=dev),
                                    n_hit=torch.zeros(4, dtype=torch.int32, device=dev)))
            B.swarm_set_cache(s_.ctx, t_base=80.0, t_transfer=2.5, **cache_state[-1])
        cached_us = time_loop(lambda s: s.step(stream=stream), n_loop)
        for s_ in sessions:
            B.swarm_set_cache(s_.ctx)
            s_.enable_submit_order()
        submit_us = time_loop(lambda s: s.step(stream=stream), n_loop)
        for s_ in sessions:
            B.swarm_set_submit_order(s_.ctx, None, None)
            s_.step(stream=stream)                       # leave the plain page step's outputs in place for the checks below
        stream.synchronize()
        t_d = time.perf_counter()

        # end to end: per-step data in pinned host memory, copies inside the timed region
        B, Hq, d, D = cfg.batch, cfg.n_q_heads, cfg.head_dim, cfg.n_queues
        q_host = [w.q.cpu().pin_memory() for w in workloads]
        out_host = torch.empty((B, Hq, d), dtype=torch.float32).pin_memory()
        lse_host = torch.empty((B, Hq), dtype=torch.float32).pin_memory()
        n_host = torch.zeros(1, dtype=torch.int32).pin_memory()
        load_host = torch.zeros(D, dtype=torch.int32).pin_memory()
        K_e2e = min(K, 5000)
        for i in range(min(Wm, 20)):
            sessions[i % args.n_rot].step_host(q_host[i % args.n_rot], out_host, lse_host, n_host, load_host, stream)
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t_e = time.perf_counter()
        e0.record(stream)
        for i in range(K_e2e):
            sessions[i % args.n_rot].step_host(q_host[i % args.n_rot], out_host, lse_host, n_host, load_host, stream)
        e1.record(stream)
        barrier()
        t_f = time.perf_counter()
        ms_e2e = e0.elapsed_time(e1)
    sampler.stop()

    ms, ms_e2e = replicas.max_over_ranks([ms, ms_e2e], device=dev)

    status = max(s.status() for s in sessions)
    by = step_bytes(workloads[0], sessions[0].o.sel, sessions[0].o.n_sel)
    peak, peak_kind = measured_peak()
    step_s = ms / 1e3 / K
    alg = by["summaries"] + by["kv_compulsory"] + by["small"]
    nominal = by["summaries"] + by["kv_nominal"] + by["small"]
    hbm_gbs = alg / step_s / 1e9
    attn_alg = by["kv_compulsory"]
    attn_gbs = attn_alg / (attn_us * 1e-6) / 1e9

    result = {
        "metric": METRIC, "value": replicas.aggregate_steps_per_s(world, K, ms), "unit": UNIT, "n_gpus": world, "steps": K, "warmup": Wm,
        "ms_per_step": ms / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
        "data": "synthetic",
        "config": {"workload": cfg.name, "batch": cfg.batch, "n_q_heads": cfg.n_q_heads, "n_kv_heads": cfg.n_kv_heads,
                   "head_dim": cfg.head_dim, "context": cfg.max_ctx(), "page_size": cfg.page_size,
                   "top_k": cfg.top_k, "n_queues": cfg.n_queues, "n_topics": cfg.n_topics,
                   "parallelism": f"replicas x{world} (no data-path collective)",
                   "l2_policy": f"rotating {args.n_rot} independent data sets "
                                f"({args.n_rot * alg / 1e6:.0f} MB touched per rotation > 126 MB L2)",
                   "launch": "library call" if args.no_graph else
                             f"CUDA graph replay: {args.n_rot} consecutive swarm_step calls per graph, executed one after another"},
        "hbm_gbs": hbm_gbs, "hbm_frac_of_measured_copy": hbm_gbs / peak, "hbm_frac_of_nominal_8tbs": hbm_gbs / NOMINAL_HBM_GBS,
        "bytes_per_step": {"algorithmic": alg, "nominal": nominal, **by},
        "stage_us_alone": {"select(score+topk)": select_us, "resolve": resolve_us, "attention_paged(+combine)": attn_us},
        "step_variants_us": {"with_cache_state(25% resident: Eq. 8 filter, counters, Eq. 6)": cached_us,
                             "with_submission_order(Sec. 5.1 batches)": submit_us},
        "medoid_step": {"us_per_step": medoid_us, "top_k_clusters": k_c,
                        "note": "swarm_step_medoid on the same data sets: clusters scored by their medoid page, whole clusters attended"},
        "roofline": {"kernel": "attn_kernel<paged> (tensor-core split-K attention over the union of selected pages, merge included)", "bound": "hbm", "achieved": attn_gbs,
                     "peak": peak, "peak_kind": f"of {peak_kind} copy bandwidth", "unit": "GB/s",
                     "frac": attn_gbs / peak, "traffic": ATTN_TRAFFIC_BYTES_NCU if cfg.name == "c2_128k" else None,
                     "algorithmic_bytes_per_launch": attn_alg, "avg_launch_us": attn_us,
                     "nominal_bytes_per_launch": by["kv_nominal"], "nominal_gbs": by["kv_nominal"] / (attn_us * 1e-6) / 1e9},
        "e2e": {"value": replicas.aggregate_steps_per_s(world, K_e2e, ms_e2e), "unit": UNIT, "steps": K_e2e,
                "h2d_bytes_per_step": B * Hq * d * 2, "d2h_bytes_per_step": B * Hq * d * 4 + B * Hq * 4 + 4 + D * 4,
                "note": "swarm_step_host: q from pinned host memory, out/lse/n_uniq/queue_load read back; "
                        "the KV pool and its summaries are resident state, like weights"},
        "gpu_launches": K * 3,   # scorer, selection, attention + cluster resolution
        "gpu_launches_per_step": 3,
        "device_status": status,
        "n_uniq_clusters": int(sessions[0].o.n_uniq[0]),
        "clocks": sampler.summary([(t_a, t_b), (t_e, t_f)]),
    }
    if rank == 0 and not args.skip_cpu_baseline and world == 1:
        result["cpu_baseline"] = cpu_baseline(workloads[0], budget_s=12.0)
    for s in sessions:
        s.close()
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

    def fn():
        return oracle.step(x["q"], ksum, x["kv_pool"], x["page_base"], x["ctx_len"], x["page2cluster"],
                           x["cluster_base"], x["replica_mask"], x["cluster_size"], Hkv=cfg.n_kv_heads,
                           S=cfg.page_size, k=cfg.top_k, D=cfg.n_queues, Pmax=cfg.max_pages())
    return fn


def cpu_baseline(w, budget_s: float):
    """The oracle as it stands, on this host's cores, on whole steps of the same workload."""
    import oracle
    cores = oracle.set_threads(0)
    fn = oracle_step_fn(w)
    fn()
    n, t0 = 0, time.perf_counter()
    while True:
        fn()
        n += 1
        el = time.perf_counter() - t0
        if el >= budget_s or n >= 1000:
            break
    return {"value": n / el, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": f"{n} whole steps of {w.cfg.name} (all {w.cfg.batch * w.cfg.n_q_heads} heads), "
                      f"OpenMP over (request, head) units, {el:.1f} s"}


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
    sampler = ClockSampler(local_rank)
    sampler.start()
    sessions = []
    for r in range(args.n_rot):                             # the same data sets on every rank, each keeps its heads
        w = W.generate(cfg, seed=r, device=dev, step=r)
        sessions.append(Session(sharding.shard_workload(w, rank, world)))
        del w
    torch.cuda.synchronize()
    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        for i in range(Wm):
            sharding.sharded_step(sessions[i % args.n_rot], stream)
        replicas.barrier()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t_a = time.perf_counter()
        e0.record(stream)
        for i in range(K):
            sharding.sharded_step(sessions[i % args.n_rot], stream)
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
                       "l2_policy": f"rotating {args.n_rot} independent data sets", "launch": "plain launches, no graph"},
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
    cores = oracle.set_threads(0)
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
