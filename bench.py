#!/usr/bin/env python
"""Benchmark of the retrieve + Chunked-RoPE-inject hot path on the Llama-3.1-8B KV shape at k=50.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--k 50] [--config llama8b]

A step is one request through the whole path: memstore_retrieve (score 2000 fp16 1024-d embeddings, top-k)
followed by memstore_inject (gather k facts' pre-RoPE K and V, rotate K at the assembled positions,
scatter both into the paged cache) on one stream, ids flowing device to device.  Requests rotate over a
pool of queries and block tables; one request moves 2 x m x 128 KiB (about 520 MB at k=50), more than the
126 MB L2, so every step is cold by construction.

One JSON line is printed by rank 0.  `value` is microseconds per request (whole job: the K steps of all
ranks divided into the max-over-ranks device time), lower is better.  With N > 1 every rank serves its own
replica of the store (the path has no exchange step: requests are independent).
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "retrieve+inject us per request at k=50 (Llama-3.1-8B KV shape)"
NOMINAL_HBM_GBS = 8000.0  # the benchmark spec quotes fractions of ~8 TB/s as well
COPY_REPEATS = 8  # consecutive launches of the copy kernel per timed event pair (see the per-part timing pass)


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", default="llama8b")
    ap.add_argument("--k", type=int, default=50)
    ap.add_argument("--seed", type=int, default=0)
    ap.add_argument("--cpu-baseline-seconds", type=float, default=15.0)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--scale-facts", type=float, default=1.0, help="shrink the store (profiling captures); the request keeps its shape")
    ap.add_argument("--pool-blocks", type=int, default=0, help="cache pool size in blocks (default: at least 4096)")
    ap.add_argument("--query-pool", type=int, default=16)
    ap.add_argument("--ordered", action="store_true", help="time the requests without MS_INPUTS_STABLE (each call ordered after all preceding work)")
    ap.add_argument("--no-configs", action="store_true", help="skip the extra keys: k = 5, 10, 20 and the batched configurations")
    ap.add_argument("--configs-budget-seconds", type=float, default=90.0, help="time budget of the batched configurations")
    return ap.parse_args()


# ---------------------------------------------------------------------------------------------- peaks / clocks
def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


class ClockSampler:
    """Polls SM clock and throttle reasons through NVML (read-only).  One sampler thread lives for the whole run and
    keeps a sample only while a GPU pass is marked with ``under_load()``: the timed region, the per-kernel and
    end-to-end passes, a sustained run of the same step, and the batched configurations - so that a short timed
    region (a few milliseconds at 20 steps) still comes with a clock record of the same work."""

    def __init__(self, index: int, period_s: float = 0.005):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self.timed_samples, self.timed_reasons = 0, set()
        self._load = self._timed = False
        self._stop = threading.Event()
        self._thr = None
        self.period = period_s
        try:
            import pynvml

            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None

    def _loop(self):
        nv = self.nv
        names = {
            "hw_slowdown": 0x8, "sw_power_cap": 0x4, "hw_thermal_slowdown": 0x40, "sw_thermal_slowdown": 0x20,
            "hw_power_brake": 0x80, "sync_boost": 0x10, "applications_clocks": 0x2,
        }  # fmt: skip
        while not self._stop.is_set():
            if self._load:
                try:
                    mhz = nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)
                    r = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                    if self._load:  # still inside the pass when the readings came back
                        self.samples.append(mhz)
                        self.timed_samples += self._timed
                        for n, bit in names.items():
                            if r & bit:
                                self.reasons.add(n)
                                if self._timed:
                                    self.timed_reasons.add(n)
                except Exception:
                    pass
            time.sleep(self.period)

    def under_load(self, timed: bool = False):
        sampler = self

        class _Pass:
            def __enter__(self):
                sampler._timed, sampler._load = timed, True

            def __exit__(self, *a):
                sampler._load = sampler._timed = False

        return _Pass()

    def __enter__(self):
        if self.nv is not None:
            self._thr = threading.Thread(target=self._loop, daemon=True)
            self._thr.start()
        return self

    def __exit__(self, *a):
        self._stop.set()
        if self._thr:
            self._thr.join()

    def summary(self):
        s = sorted(self.samples)
        return {"sm_mhz": s[len(s) // 2] if s else None, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(s), "samples_in_timed_region": self.timed_samples,
                "note": "samples are taken only while GPU passes run: the timed region, the per-kernel / end-to-end / latency "
                        "passes, a sustained run of the same step and the batched configurations"}  # fmt: skip


def max_over_ranks(value: float, world: int, device=None) -> float:
    """The slowest rank's figure (every multi-GPU time is the max over ranks).  Works on any initialised backend."""
    if world <= 1:
        return float(value)
    import torch
    import torch.distributed as dist

    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t[0])


def workload_string(name: str, shape, n_facts: int, k: int) -> str:
    """The one description of the benchmarked workload, printed by both arms."""
    return (f"{name}: {n_facts} facts of {shape.len_lo}-{shape.len_hi} tokens, L={shape.n_layers} h={shape.n_kv_heads} "
            f"d={shape.head_dim}, {shape.emb_dim}-d {shape.emb_dtype} embeddings, k={k}, start {shape.start_pos}, "
            f"block {shape.block_size}")  # fmt: skip


def captured_traffic(config: str, k: int):
    """DRAM bytes (read + write) per launch of the copy kernel from the committed ncu capture of that kernel: the data
    file next to the summary in profiles/ (one 'key = value' pair per line).  None when there is no capture of this
    workload."""
    path = os.path.join(ROOT, "profiles", f"inject_copy_kernel_{config}_k{k}.traffic.txt")
    if not os.path.exists(path):
        return None, None
    kv = {}
    with open(path) as f:
        for ln in f:
            if "=" in ln and not ln.lstrip().startswith("#"):
                a, b = ln.split("=", 1)
                kv[a.strip()] = b.strip()
    try:
        return float(kv["dram_bytes_per_launch"]), kv.get("captured_at_commit")
    except (KeyError, ValueError):
        return None, None


THERMAL_REASONS = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown")


# ---------------------------------------------------------------------------------------------- CPU oracle arm
class OracleArm:
    """Times the CPU oracle, as it stands, on a bounded sample of one request of the workload and scales the
    result to a whole request.  Sample: the full retrieval (all facts) plus the injection, over all layers, of
    the first facts of the oracle's own top-k list (placement order), as many tokens as fit the time budget."""

    def __init__(self, shape, k, seed, n_threads=0):
        import numpy as np

        import oracle
        from paper_2607_27090_b200 import synth

        oracle.build()
        self.np, self.oracle, self.synth = np, oracle, synth
        self.shape, self.k, self.seed, self.n_threads = shape, k, seed, n_threads
        self.cores = oracle.max_threads() if n_threads <= 0 else n_threads
        self.emb = synth.embeddings(seed, shape.n_facts, shape.emb_dim, shape.emb_dtype)
        self.q = synth.queries(seed, 1, shape.emb_dim, shape.emb_dtype)
        self.lens = synth.fact_lengths(seed, shape.n_facts, shape.len_lo, shape.len_hi)
        ids, _ = oracle.retrieve(self.emb, self.q, k, n_threads=n_threads)
        self.ids = ids[0][::-1].copy()  # the paper's placement: best fact last
        self.m_full = int(self.lens[self.ids].sum())
        self.table = np.arange((shape.start_pos + self.m_full) // shape.block_size + 2, dtype=np.int32)
        self._packed = {}
        t, m = self._inject(1)
        self.per_token_s = t / max(m, 1)

    def _pack(self, n_take):
        if n_take not in self._packed:
            np, s = self.np, self.shape
            offs = np.zeros(s.n_facts, np.int64)
            ln = np.zeros(s.n_facts, np.int32)
            ks, vs, t = [], [], 0
            for f in dict.fromkeys(int(i) for i in self.ids[:n_take]):
                kf, vf = self.synth.kv_fact(self.seed, f, s.n_layers, int(self.lens[f]), s.n_kv_heads, s.head_dim)
                ks.append(kf)
                vs.append(vf)
                offs[f], ln[f] = t, self.lens[f]
                t += int(self.lens[f])
            self._packed = {n_take: (offs, ln, np.concatenate(ks, axis=1), np.concatenate(vs, axis=1))}
        return self._packed[n_take]

    def _inject(self, n_take):
        s = self.shape
        offs, ln, kk, vv = self._pack(n_take)
        t0 = time.perf_counter()
        res = self.oracle.inject(self.ids[:n_take], offs, ln, kk, vv, s.rope_theta, s.start_pos, self.table, s.block_size,
                                 self.table.size, want_ref=False, n_threads=self.n_threads)  # fmt: skip
        return time.perf_counter() - t0, res.m

    def facts_for_budget(self, budget_s):
        n_take, tok = 1, int(self.lens[self.ids[0]])
        while n_take < len(self.ids) and (tok + self.lens[self.ids[n_take]]) * self.per_token_s < budget_s:
            tok += int(self.lens[self.ids[n_take]])
            n_take += 1
        return n_take

    def time_step(self, n_take):
        """One sampled request -> (microseconds scaled to the whole request, description of the sample)."""
        t0 = time.perf_counter()
        self.oracle.retrieve(self.emb, self.q, self.k, n_threads=self.n_threads)
        t_retrieve = time.perf_counter() - t0
        t_inj, m_s = self._inject(n_take)
        t_req = t_retrieve + t_inj * (self.m_full / m_s)
        sample = (f"retrieval over all {self.shape.n_facts} facts ({t_retrieve * 1e3:.1f} ms) + injection of the first "
                  f"{n_take} of {len(self.ids)} facts ({m_s} of {self.m_full} tokens, all {self.shape.n_layers} layers, "
                  f"{t_inj:.2f} s), injection time scaled by tokens")  # fmt: skip
        return t_req * 1e6, sample


def run_reference(args):
    """The reference arm: the CPU oracle timed on the host cores (rank 0 only)."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from paper_2607_27090_b200 import synth

    shape = synth.CONFIGS[args.config]
    arm = OracleArm(shape, args.k, args.seed)
    n_take = arm.facts_for_budget(max(0.02, 100.0 / max(1, args.steps + args.warmup)))
    vals, sample = [], ""
    for i in range(args.warmup + args.steps):
        v, sample = arm.time_step(n_take)
        if i >= args.warmup:
            vals.append(v)
    v = sum(vals) / len(vals)
    line = {
        "metric": METRIC, "value": v, "unit": "us", "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": v / 1e3, "higher_is_better": False, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic", "impl": "reference",
        "config": {"workload": workload_string(args.config, shape, shape.n_facts, args.k)},
        "cpu_baseline": {"value": v, "unit": "us", "cores": arm.cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": v, "unit": "us", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }  # fmt: skip
    print(json.dumps(line))


# ---------------------------------------------------------------------------------------------- CUDA arm
def run_ours(args):
    import numpy as np
    import torch
    import torch.distributed as dist

    from paper_2607_27090_b200 import memstore as M
    from paper_2607_27090_b200 import synth, workload

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the path has no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    shape = synth.CONFIGS[args.config]
    k = args.k
    n_pool = args.query_pool
    per_req_blocks = workload.blocks_per_request(shape, k)
    wl = workload.build(args.config, seed=args.seed + rank, device=dev, n_query_pool=n_pool, scale_facts=args.scale_facts,
                        num_blocks=args.pool_blocks or max(4096, per_req_blocks * n_pool))  # fmt: skip
    store, cache = wl.store, wl.cache
    tables = torch.from_numpy(synth.block_tables(args.seed + rank, cache.num_blocks, per_req_blocks, n_pool)).to(dev)
    queries = torch.from_numpy(wl.queries).to(dev)
    start = torch.full((1,), shape.start_pos, dtype=torch.int32, device=dev)
    ids = torch.empty((1, k), dtype=torch.int32, device=dev)
    n_tok = torch.zeros(n_pool, dtype=torch.int32, device=dev)
    status = torch.zeros(n_pool, dtype=torch.int32, device=dev)
    stream = torch.cuda.current_stream()

    # The queries and block tables of the pool are resident before the run starts, which is what MS_INPUTS_STABLE asks
    # of a caller: the scoring of a request may then start while the previous request's copy kernel drains.
    step_flags = M.INJECT_REVERSE | (0 if args.ordered else M.INPUTS_STABLE)

    # (views of the pool made once: slicing four tensors per step costs the Python loop several microseconds, which shows
    # at the small k, where a request takes the GPU less time than the binding's call)
    q_v = [queries[j : j + 1] for j in range(n_pool)]
    t_v = [tables[j : j + 1] for j in range(n_pool)]
    n_v = [n_tok[j : j + 1] for j in range(n_pool)]
    s_v = [status[j : j + 1] for j in range(n_pool)]

    def step(i, flags=step_flags):
        # one request through the whole path: the library's retrieve+inject call (two kernel launches)
        j = i % n_pool
        store.retrieve_inject(q_v[j], k, start, t_v[j], cache, out_ids=ids, out_n_tokens=n_v[j], out_status=s_v[j], flags=flags,
                              stream=stream)  # fmt: skip

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for i in range(max(args.warmup, 3)):
        step(i)
    barrier()
    assert int(status.abs().sum()) == 0, "a request reported a data error"
    m_pool = n_tok.cpu().numpy().astype(np.int64)
    if args.warmup < n_pool:  # make sure every pool entry has been seen once for the byte accounting
        for i in range(n_pool):
            step(i)
        barrier()
        m_pool = n_tok.cpu().numpy().astype(np.int64)

    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    remeasured = False
    clk = ClockSampler(local)
    clk.__enter__()
    while True:
        # the warm-up steps run once more right here: the set-up above (clock sampler, counters, copies to the host) leaves
        # the GPU idle for milliseconds, and a GPU that has been idle takes its first steps slowly
        for i in range(max(args.warmup, 3)):
            step(i)
        barrier()
        launches0 = store.stats()["kernels_launched"]
        barrier()
        with clk.under_load(timed=True):
            e0.record(stream)
            for i in range(args.steps):
                step(i)
            e1.record(stream)
            barrier()
        ms_total = e0.elapsed_time(e1)
        launches = store.stats()["kernels_launched"] - launches0
        # the same step, sustained for about 0.4 s: the clock record of this work under load (not part of `value`)
        with clk.under_load():
            for i in range(max(200, int(0.4e3 / max(ms_total / args.steps, 1e-3)))):
                step(i)
            torch.cuda.synchronize()
        throttled = max_over_ranks(float(any(r in clk.reasons for r in THERMAL_REASONS)), world, dev) > 0
        if throttled and not remeasured:  # a thermally throttled run is rejected and measured once more
            remeasured = True
            clk.samples.clear()
            clk.reasons.clear()
            clk.timed_reasons.clear()
            clk.timed_samples = 0
            time.sleep(2.0)
            continue
        break
    ms_total = max_over_ranks(ms_total, world, dev)
    us_per_request = ms_total * 1e3 / (args.steps * world)
    # the same steps with every call ordered after all preceding work (no MS_INPUTS_STABLE): reported beside `value`
    n_ord = max(args.steps, 200)
    for i in range(10):
        step(i, M.INJECT_REVERSE)
    barrier()
    with clk.under_load():
        e0.record(stream)
        for i in range(n_ord):
            step(i, M.INJECT_REVERSE)
        e1.record(stream)
        barrier()
    ordered_us = max_over_ranks(e0.elapsed_time(e1), world, dev) * 1e3 / (n_ord * world)

    # ---- per-part timing and the roofline of the dominant kernel (the copy kernel of inject) --------------
    # The copy kernel is timed by a CUDA-event pair that the library records around it.  An event record lets nothing of
    # a kernel launch overlap it, so a pair around ONE launch also measures a few microseconds of launch latency; the
    # kernel's own duration is taken from COPY_REPEATS consecutive launches on the same plan between the two records
    # (ordinary launches, each after the one before it has ended; every launch moves more bytes than the L2 holds).
    n_prof = min(args.steps, 400)
    r0 = [torch.cuda.Event(enable_timing=True) for _ in range(n_prof)]
    r1 = [torch.cuda.Event(enable_timing=True) for _ in range(n_prof)]

    def copy_kernel_pass(repeats):
        evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n_prof)]
        for a, b in evs:
            a.record(stream)
            b.record(stream)
        torch.cuda.synchronize()
        store.set_profile_repeats(repeats)
        with clk.under_load():
            for i in range(n_prof):
                j = i % n_pool
                r0[i].record(stream)
                store.retrieve(queries[j : j + 1], k, out_ids=ids, want_scores=False, stream=stream)
                r1[i].record(stream)
                store.set_profile_events(*evs[i])
                store.inject(ids, start, tables[j : j + 1], cache, out_n_tokens=n_tok[j : j + 1], out_status=status[j : j + 1],
                             flags=M.INJECT_REVERSE, stream=stream)  # fmt: skip
            store.set_profile_events(None, None)
            torch.cuda.synchronize()
        store.set_profile_repeats(1)
        return np.array([a.elapsed_time(b) * 1e3 / repeats for a, b in evs])

    pair_us = copy_kernel_pass(1)
    copy_us = copy_kernel_pass(COPY_REPEATS)
    retr_us = np.array([a.elapsed_time(b) * 1e3 for a, b in zip(r0, r1)])
    bytes_prof = np.array([workload.kv_bytes_moved(shape, int(m_pool[i % n_pool])) for i in range(n_prof)], dtype=np.float64)
    copy_gbs = float(bytes_prof.sum() / (copy_us.sum() * 1e-6) / 1e9)
    peak, peak_kind = measured_peaks()
    mean_m = float(np.mean([m_pool[i % n_pool] for i in range(args.steps)]))
    bytes_step = workload.kv_bytes_moved(shape, 1) * mean_m + workload.emb_bytes_scanned(shape, int(wl.lens.size))

    # ---- end to end through the binding with HOST buffers ------------------------------------------------
    n_e2e = min(args.steps, 500)
    q_host = torch.from_numpy(wl.queries).pin_memory()
    t_host = torch.from_numpy(synth.block_tables(args.seed + rank, cache.num_blocks, per_req_blocks, n_pool)).pin_memory()
    out_host = torch.empty((k + 2,), dtype=torch.int32).pin_memory()

    def e2e_step(i, flags=M.INJECT_REVERSE):
        # the public host-buffer call: one H2D transfer (query, start position, block table), retrieve, inject,
        # ids, token count and status written into pinned host memory and a stream synchronise, all inside the library
        j = i % n_pool
        store.serve_host(q_host[j], k, shape.start_pos, t_host[j], cache, out_host, flags=flags, stream=stream)

    def e2e_pass(flags):
        for i in range(5):
            e2e_step(i, flags)
        barrier()
        with clk.under_load():
            e0.record(stream)
            for i in range(n_e2e):
                e2e_step(i, flags)
            e1.record(stream)
            barrier()
        return max_over_ranks(e0.elapsed_time(e1), world, dev) * 1e3 / (n_e2e * world)

    e2e_us = e2e_pass(M.INJECT_REVERSE)
    # the same call returning as soon as ids, token count and status are on the host (MS_SERVE_EARLY_RETURN): the copy into
    # the cache of request i runs while the host prepares request i + 1; the last event still waits for all of it
    e2e_early_us = e2e_pass(M.INJECT_REVERSE | M.SERVE_EARLY_RETURN)
    h2d = ((q_host[0].numel() * q_host.element_size() + 15) // 16) * 16 + 16 + ((t_host[0].numel() * 4 + 15) // 16) * 16
    d2h = (k + 2) * 4

    traffic, traffic_commit = captured_traffic(args.config, k)
    line = {
        "metric": METRIC, "value": us_per_request, "unit": "us", "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": ms_total / args.steps, "higher_is_better": False,
        "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {
            "workload": workload_string(args.config, shape, int(wl.lens.size), k),
            "mean_tokens_per_request": mean_m, "bytes_per_request": bytes_step,
            "l2_policy": "inputs larger than L2: each request moves ~%.0f MB and rotates over %d queries / block tables"
                         % (bytes_step / 1e6, n_pool),
            "replicas": world, "storage_dtype": "bf16 K/V, fp16 embeddings", "remeasured_after_throttle": remeasured,
            "call": "memstore_retrieve_inject, flags MS_INJECT_REVERSE" + ("" if args.ordered else " | MS_INPUTS_STABLE (the query pool is resident before the run)"),
        },
        "ordered_us": ordered_us,
        "retrieve_us": float(np.median(retr_us)), "inject_copy_kernel_us": float(np.median(copy_us)),
        "path_gbs": bytes_step / (us_per_request * world * 1e-6) / 1e9,
        "roofline": {
            "bound": "hbm", "kernel": "inject_copy_kernel", "achieved": copy_gbs, "peak": peak, "unit": "GB/s",
            "frac": copy_gbs / peak, "peak_kind": f"of {peak_kind}", "frac_of_nominal_8TBs": copy_gbs / NOMINAL_HBM_GBS,
            "traffic": traffic, "traffic_captured_at_commit": traffic_commit,
            "algorithmic_bytes_per_launch": float(bytes_prof.mean()),
            "timing": "CUDA-event pair recorded by the library around %d consecutive launches of the kernel on one plan, "
                      "divided by %d (mean over %d requests)" % (COPY_REPEATS, COPY_REPEATS, n_prof),
            "event_pair_around_one_launch_us": float(np.median(pair_us)),
        },
        "e2e": {"value": e2e_early_us, "unit": "us", "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "call": "memstore_serve_host with MS_SERVE_EARLY_RETURN, host buffers in and out: every call copies its query, "
                        "start position and block table up from pinned memory and returns when the request's ids, token count "
                        "and status are on the host; the copy into the cache completes in stream order while the host prepares "
                        "the next request, and the timed region ends after the last request's copy (requests back to back, as "
                        "in `value`)",
                "waited_value": e2e_us,
                "waited_call": "the same call without the flag: it synchronises the stream before it returns, so no two "
                               "requests overlap"},
        "gpu_launches": int(launches),
    }  # fmt: skip

    # ---- per-request latency distribution (separate pass: an event after every step) and CUDA-graph replay ---------
    n_lat = min(args.steps, 500)
    marks = [torch.cuda.Event(enable_timing=True) for _ in range(n_lat + 1)]
    torch.cuda.synchronize()
    with clk.under_load():
        marks[0].record(stream)
        for i in range(n_lat):
            step(i)
            marks[i + 1].record(stream)
        torch.cuda.synchronize()
    lat = np.sort(np.array([marks[i].elapsed_time(marks[i + 1]) * 1e3 for i in range(n_lat)]))
    line["latency_us"] = {"p10": float(lat[n_lat // 10]), "p50": float(lat[n_lat // 2]), "p90": float(lat[(n_lat * 9) // 10]),
                          "n": n_lat, "note": "one CUDA event per step on the stream, steady state"}  # fmt: skip
    def graph_replay_us(kk, ids_buf, flags):
        """The n_pool requests captured once into a CUDA graph and replayed: the host issues one launch per n_pool
        requests, so the figure is free of the per-call cost of the Python binding (17 - 24 us per call, which bounds
        what a Python loop can show for the small k)."""
        side = torch.cuda.Stream()
        side.wait_stream(stream)
        graph = torch.cuda.CUDAGraph()

        def one(j):
            store.retrieve_inject(queries[j : j + 1], kk, start, tables[j : j + 1], cache, out_ids=ids_buf, out_n_tokens=n_tok[j : j + 1],
                                  out_status=status[j : j + 1], flags=flags, stream=side)  # fmt: skip

        with torch.cuda.stream(side):
            for j in range(2):  # make sure nothing is allocated lazily on this stream inside the capture
                one(j)
            side.synchronize()
            with torch.cuda.graph(graph, stream=side):
                for j in range(n_pool):
                    one(j)
        torch.cuda.synchronize()
        reps = max(1, min(max(args.steps, 200), 800) // n_pool)
        for _ in range(2):
            graph.replay()
        torch.cuda.synchronize()
        with clk.under_load():
            e0.record(stream)
            for _ in range(reps):
                graph.replay()
            e1.record(stream)
            torch.cuda.synchronize()
        return e0.elapsed_time(e1) * 1e3 / (reps * n_pool)

    try:
        line["graph_replay_us"] = graph_replay_us(k, ids, step_flags)
        line["graph_replay_ordered_us"] = graph_replay_us(k, ids, M.INJECT_REVERSE)
    except Exception as ex:  # graph capture is optional evidence, never a reason to lose the bench line
        line["graph_replay_us"] = None
        line["graph_replay_error"] = str(ex)[:200]
        torch.cuda.synchronize()

    if not args.no_configs:
        # the other values of k of this configuration (extra keys; at least 200 steps each whatever --steps says)
        sweep, n_sweep = {}, max(args.steps, 200)
        for kk in (5, 10, 20):
            ids_k = torch.empty((1, kk), dtype=torch.int32, device=dev)

            def step_k(i, flags=step_flags):
                j = i % n_pool
                store.retrieve_inject(q_v[j], kk, start, t_v[j], cache, out_ids=ids_k, out_n_tokens=n_v[j], out_status=s_v[j],
                                      flags=flags, stream=stream)  # fmt: skip

            for i in range(n_pool):
                step_k(i)
            torch.cuda.synchronize()
            m_k = float(n_tok.cpu().numpy().astype(np.float64).mean())
            with clk.under_load():
                e0.record(stream)
                for i in range(n_sweep):
                    step_k(i)
                e1.record(stream)
                torch.cuda.synchronize()
            us_k = e0.elapsed_time(e1) * 1e3 / n_sweep
            # the same request every time: at k = 5 and 10 its source rows and cache blocks (52 / 105 MB) stay in the
            # 126 MB L2, the "warm" figure next to the rotating ("cold") one above
            for i in range(10):
                step_k(0)
            torch.cuda.synchronize()
            with clk.under_load():
                e0.record(stream)
                for i in range(n_sweep):
                    step_k(0)
                e1.record(stream)
                torch.cuda.synchronize()
            same_us = e0.elapsed_time(e1) * 1e3 / n_sweep
            with clk.under_load():
                e0.record(stream)
                for i in range(n_sweep):
                    step_k(i, M.INJECT_REVERSE)
                e1.record(stream)
                torch.cuda.synchronize()
            ordered_k = e0.elapsed_time(e1) * 1e3 / n_sweep
            try:
                graph_k = graph_replay_us(kk, ids_k, step_flags)
            except Exception:
                graph_k = None
                torch.cuda.synchronize()
            bytes_k = workload.kv_bytes_moved(shape, 1) * m_k + workload.emb_bytes_scanned(shape, int(wl.lens.size))
            sweep[f"k{kk}"] = {"us_per_request": us_k, "same_request_us": same_us, "ordered_us": ordered_k, "graph_replay_us": graph_k,
                               "tokens": m_k,
                               "path_gbs": bytes_k / (us_k * 1e-6) / 1e9, "frac_of_measured": bytes_k / (us_k * 1e-6) / 1e9 / peak,
                               "hbm_floor_us": bytes_k / (peak * 1e9) * 1e6}  # fmt: skip
        line["sweep"] = sweep

    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        arm = OracleArm(shape, k, args.seed)
        n_take = arm.facts_for_budget(args.cpu_baseline_seconds)
        vals, t_begin = [], time.perf_counter()
        while not vals or (time.perf_counter() - t_begin < args.cpu_baseline_seconds and len(vals) < 100):
            v, sample = arm.time_step(n_take)
            vals.append(v)
        one = OracleArm(shape, k, args.seed, n_threads=1)
        v1, _ = one.time_step(one.facts_for_budget(3.0))
        line["cpu_baseline"] = {"value": sum(vals) / len(vals), "unit": "us", "cores": arm.cores, "kind": "oracle",
                                "sample": f"mean of {len(vals)} repeats of: {sample}", "single_thread_value": v1}  # fmt: skip
    store.close()
    if rank == 0 and world == 1 and not args.no_configs:
        # the batched configurations of the workload list (100 users, the 14B-class shape, 1M facts), each with its own
        # store: the headline store and pool are released first
        from paper_2607_27090_b200 import measure_configs

        del wl, cache, tables, queries
        torch.cuda.empty_cache()
        with clk.under_load():
            line["configs"] = measure_configs.measure_all(peak, budget_s=args.configs_budget_seconds, seed=args.seed)
    clk.__exit__()
    line["clocks"] = clk.summary()
    if rank == 0:
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    a = parse_args()
    if a.impl == "reference":
        run_reference(a)
    else:
        run_ours(a)
