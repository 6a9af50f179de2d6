#!/usr/bin/env python
"""Benchmark of the SparK decode step (spark_decode_attn) on synthetic Llama-3.1-8B-shaped caches.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config I] [--impl ours|reference] [--no-sweep]

One "step" is one spark_decode_attn call over the whole packed cache of the workload (all sequences,
all heads; 28 calls, one per layer, for the Qwen-shaped configuration).  The cache is compressed once,
outside the timed region (prefill side); its time is reported under "compress".  Steps rotate over several
copies of the packed cache so that each launch reads cold data (copies * bytes >= 4 * L2).

Timing.  The steps are captured in CUDA graphs and timed with CUDA events on the launching stream:
  value          exactly K steps in one region bracketed by barrier + synchronize, ORDINARY launches;
  replays        the same graph replayed >= 50 times, each replay timed on its own: median and minimum;
  value_pdl      the same K steps launched with SPARK_FLAG_OVERLAP_PREVIOUS (programmatic dependent launch:
                 step i+1 may start its page stream while step i drains), a pipelined-throughput figure that
                 holds only when the kernel enqueued before the step does not write the cache.
With the default workload (the 32K headline configuration) the run also times the 4x128K, the evicted
32x2048 and the 28-layer Qwen-shape configurations and reports them under "sweep" in the same JSON line
(--no-sweep skips them).

With N > 1 (torchrun) every rank runs the same workload on its own GPU with no data-path collective (weak
scaling); the reported time is the max over ranks.  --impl reference times the CPU oracle on the host cores
instead (a deliberately plain program).  Prints ONE JSON line on rank 0.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "channel-sparse decode attn µs/step & HBM GB/s (% of peak), Llama-8B shape, 32K"
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0
# dram__bytes_read.sum + dram__bytes_write.sum per decode launch from the ncu captures summarised in
# profiles/decode_bf16_*.md (bytes)
NCU_TRAFFIC_BYTES = {"llama8b_32k": 109.6e6, "llama8b_4x128k": 1380.6e6}        # 4 x (342.0 + 3.16) MB from one 128K sequence
MIN_REPLAYS = 50


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """Samples SM clock and throttle reasons through NVML (read-only) while a region runs."""

    def __init__(self, index: int, period_s: float = 0.004):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        self.period = period_s
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self.nv = None

    def _names(self, bits: int):
        nv = self.nv
        table = [("sw_power_cap", "nvmlClocksEventReasonSwPowerCap", 0x4),
                 ("hw_slowdown", "nvmlClocksEventReasonHwSlowdown", 0x8),
                 ("sw_thermal_slowdown", "nvmlClocksEventReasonSwThermalSlowdown", 0x20),
                 ("hw_thermal_slowdown", "nvmlClocksEventReasonHwThermalSlowdown", 0x40),
                 ("hw_power_brake", "nvmlClocksEventReasonHwPowerBrakeSlowdown", 0x80)]
        return [n for n, attr, default in table if bits & int(getattr(nv, attr, default))]

    def _run(self):
        nv = self.nv
        while not self._stop.is_set():
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)))
                get = getattr(nv, "nvmlDeviceGetCurrentClocksEventReasons", None) or \
                    nv.nvmlDeviceGetCurrentClocksThrottleReasons
                self.reasons.update(self._names(int(get(self.h))))
            except Exception:
                pass
            self._stop.wait(self.period)

    def __enter__(self):
        self.samples, self.reasons = [], set()
        if self.nv is not None:
            self._stop.clear()
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()
        return self

    def __exit__(self, *exc):
        if self._thread is not None:
            self._stop.set()
            self._thread.join()
            self._thread = None

    def summary(self):
        return {"sm_mhz": statistics.median(self.samples) if self.samples else None,
                "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": len(self.samples)}


def workload_desc(cfg, keep, copies=None, keep_v=0):
    d = {"workload": cfg["name"], "batch": cfg["batch"], "n_q_heads": cfg["n_q_heads"],
         "n_kv_heads": cfg["n_kv_heads"], "head_dim": cfg["head_dim"], "cached_tokens": cfg["seq_lens"],
         "window": cfg["window"], "pruning_ratio": cfg["ratio"], "keep": keep, "page_tokens": 16}
    if "token_budget" in cfg:
        d["cached_tokens_after_eviction"] = cfg["token_budget"]
    if 0 < keep_v < 128:
        d["value_keep"] = keep_v                     # value-channel pruning on top of the named workload
    if copies is not None:
        d["cold_cache"] = f"rotation over {copies} packed-cache copies (copies*bytes >= 4*L2)"
    return d


# ----------------------------------------------------------------------------------------------------
# the oracle on the host cores
# ----------------------------------------------------------------------------------------------------
def oracle_prepare(q_win, k, v, lens, keep, keep_v=0, variant=None):
    """Untimed preparation of an oracle decode: window mean, key pruning (fixed T or a ratio-free variant),
    value masks.  `variant` = dict(top_p | group_prune, recovery, seed) or None."""
    import oracle
    variant = variant or {}
    _, a = oracle.window_mean(q_win, k.shape[1])
    if variant.get("top_p") is not None:
        c = oracle.select_variant(k, lens, a, top_p=variant["top_p"], cap=keep, want_stats=True)
    elif variant.get("group_prune") is not None:
        c = oracle.select_variant(k, lens, a, group_prune=variant["group_prune"], want_stats=True)
    else:
        c = oracle.compress(k, lens, keep, a, want_stats=bool(variant.get("recovery")))
    c["recovery"], c["seed"] = int(variant.get("recovery") or 0), int(variant.get("seed") or 0)
    vm = oracle.prune_values(v, lens, keep_v) if 0 < keep_v < 128 else None
    return a, c, vm


def oracle_decode(q, k, v, lens, a, c, vm):
    import oracle
    if c.get("recovery"):
        return oracle.decode_attn_sampled(q, k, v, lens, c["mask"], c["mu_all"], c["sigma_all"], a,
                                          mode=c["recovery"], seed=c["seed"])[0]
    return oracle.decode_attn(q, k, v, lens, c["mask"], c["mu"], a, vmask=vm)[0]


def oracle_decode_time(q, k, v, lens, a, c, vm, reps=3):
    """Median time of the oracle's decode step on the host cores -> (seconds, threads, output)."""
    import oracle
    oracle_decode(q, k, v, lens, a, c, vm)                                               # warm
    ts, out = [], None
    for _ in range(reps):
        t0 = time.perf_counter()
        out = oracle_decode(q, k, v, lens, a, c, vm)
        ts.append(time.perf_counter() - t0)
    return statistics.median(ts), oracle.threads(), out


def run_reference(args, cfg, keep):
    """The oracle as the reference arm: a bounded sample (one full decode step per timed step)."""
    from workloads import inputs
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    if "token_budget" in cfg or "n_layers" in cfg:
        print(json.dumps({"impl": "reference", "unavailable": "the oracle arm is timed on the single-layer "
                          "configurations (0, 1, 2); this one needs the GPU path to lay out its cache"}))
        return
    wl = inputs.config_workload(args.config, device="cpu")
    inputs.enforce_saliency_gap(wl, keep)
    a, c, vm = oracle_prepare(wl.q_win, wl.k, wl.v, wl.seq_lens, keep)
    steps, warm = max(1, min(args.steps, 20)), max(1, min(args.warmup, 3))
    for _ in range(warm):
        oracle.decode_attn(wl.q, wl.k, wl.v, wl.seq_lens, c["mask"], c["mu"], a)
    t0 = time.perf_counter()
    for _ in range(steps):
        oracle.decode_attn(wl.q, wl.k, wl.v, wl.seq_lens, c["mask"], c["mu"], a)
    dt = (time.perf_counter() - t0) / steps
    us = dt * 1e6
    sample = f"{steps} full decode steps of the workload (steps capped at 20 for the CPU arm)"
    line = {"impl": "reference", "metric": METRIC, "value": us, "unit": "us/step", "n_gpus": args.gpus,
            "steps": steps, "warmup": warm, "ms_per_step": dt * 1e3, "higher_is_better": False,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": workload_desc(cfg, keep),
            "cpu_baseline": {"value": us, "unit": "us/step", "cores": oracle.threads(), "kind": "oracle",
                             "sample": sample},
            "e2e": {"value": us, "unit": "us/step", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


# ----------------------------------------------------------------------------------------------------
# workloads: packed caches resident in HBM, ready to decode
# ----------------------------------------------------------------------------------------------------
class Work:
    """One benchmark configuration laid out on the GPU.  step_sets[i] is the list of (cache, q, out) decode
    launches of one step; consecutive steps use consecutive sets (cold copies)."""

    def __init__(self):
        self.step_sets, self.caches = [], []
        self.alg_bytes = 0
        self.copies = 1
        self.compress_us = self.compress_bytes = None
        self.compress_what = None
        self.oracle_inputs = None          # callable -> (q, k, v, lens, q_win) host tensors of set 0, or None
        self.oracle_sample = None
        self.oracle_scale = 1              # the timed oracle sample is 1 / oracle_scale of a step
        self.cfg, self.keep, self.keep_v = None, 0, 0
        self.variant = None                # dict(top_p | group_prune, recovery, seed) of a ratio-free / sampled run

    @property
    def launches_per_step(self):
        return len(self.step_sets[0])


def build_work(index, cfg, keep, keep_v, rank, torch, B, variant=None):
    from paper_2508_15212_b200 import dist_utils
    from paper_2508_15212_b200.cache import SparkCache
    from workloads import inputs
    from workloads.batches import build_evicted_batch, permuted_block_table
    w = Work()
    w.cfg, w.keep, w.keep_v, w.variant = cfg, keep, keep_v, variant
    vkw = {} if not variant else {k_: v_ for k_, v_ in variant.items() if v_ is not None}
    l2 = torch.cuda.get_device_properties(torch.cuda.current_device()).L2_cache_size
    D = cfg["head_dim"]
    esize = 2 if cfg["dtype"] == "bf16" else 4
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
    if "token_budget" in cfg:          # prompts evicted and pruned one at a time into one batch cache
        per_tok = B.spark_algorithmic_bytes_per_token(B.make_params(
            batch=1, n_q_heads=cfg["n_q_heads"], n_kv_heads=cfg["n_kv_heads"], window=cfg["window"], keep=keep,
            dtype=torch.bfloat16 if cfg["dtype"] == "bf16" else torch.float32, n_pool_pages=1, keep_v=keep_v))
        w.alg_bytes = per_tok * cfg["n_kv_heads"] * cfg["token_budget"] * cfg["batch"]
        w.copies = max(1, -(-4 * l2 // w.alg_bytes))
        prep = []
        for c in range(w.copies):
            cache, q, _, _ = build_evicted_batch(cfg, keep, seed_offset=dist_utils.rank_seed_offset(rank, c),
                                                 keep_v=keep_v, keep_gathered=(c == 0))
            out = torch.empty(cfg["batch"], cfg["n_q_heads"], D, dtype=torch.float32, device="cuda")
            w.step_sets.append([(cache, q, out)])
            w.caches.append(cache)
            prep += cache.prep_us
        prep.sort()
        w.compress_us, w.compress_bytes = prep[len(prep) // 2], 2 * cfg["n_kv_heads"] * int(cfg["seq_lens"]) * D * esize
        w.compress_what = "evict + prune one prompt (median over all prompts)"
        first, q0 = w.caches[0], w.step_sets[0][0][1]

        def oracle_inputs():
            q_win, kg, vg = first.gathered
            return q0.cpu(), kg.cpu(), vg.cpu(), first.packed_lens.cpu(), q_win.cpu()
        w.oracle_inputs = oracle_inputs
        w.oracle_sample = "one full decode step over the evicted caches of all prompts, median of 3"
    elif "n_layers" in cfg:            # paged pool, variable lengths, all layers per step
        layer_set, total_tokens = [], 0
        for layer in range(cfg["n_layers"]):
            wl_l = inputs.config_workload(index, device="cuda", seed_offset=dist_utils.rank_seed_offset(rank, layer))
            Bn, Hq, Hkv, W, _, S = wl_l.shape
            lens = wl_l.seq_lens.tolist()
            table, n_pages = permuted_block_table(Bn, Hkv, lens, "cuda", seed=977 * layer + rank)
            cache = SparkCache(batch=Bn, n_q_heads=Hq, n_kv_heads=Hkv, window=W, keep=keep, dtype=wl_l.dtype,
                               max_tokens=S, block_table=table, n_pool_pages=n_pages, keep_v=keep_v)
            cache.compress(wl_l.q_win, wl_l.k, wl_l.v, wl_l.seq_lens)
            w.alg_bytes += cache.algorithmic_bytes_per_token * Hkv * sum(lens)
            layer_set.append((cache, wl_l.q.clone(), torch.empty(Bn, Hq, D, dtype=torch.float32, device="cuda")))
            w.caches.append(cache)
            total_tokens += sum(lens)
            del wl_l
            torch.cuda.empty_cache()
        w.step_sets.append(layer_set)
        cfg["seq_lens"] = (f"uniform[8192,131072] per sequence, independent per layer; "
                           f"{total_tokens} tokens over {cfg['n_layers']} layers")

        def oracle_inputs():               # layer 0 again, from its seed (the layers' dense tensors are not kept)
            wl0 = inputs.config_workload(index, device="cuda", seed_offset=dist_utils.rank_seed_offset(rank, 0))
            return wl0.q.cpu(), wl0.k.cpu(), wl0.v.cpu(), wl0.seq_lens.cpu(), wl0.q_win.cpu()
        w.oracle_inputs = oracle_inputs
        w.oracle_scale = cfg["n_layers"]
        w.oracle_sample = (f"layer 0 of {cfg['n_layers']} in full (one decode launch), median of 3, "
                           f"times {cfg['n_layers']} for the step")
    else:
        wl = inputs.config_workload(index, device="cuda", seed_offset=dist_utils.rank_seed_offset(rank),
                                    batch=cfg["batch"])
        inputs.enforce_saliency_gap(wl, keep)
        Bn, Hq, Hkv, W, _, S = wl.shape
        lens = wl.seq_lens.tolist()
        mk = lambda: SparkCache(batch=Bn, n_q_heads=Hq, n_kv_heads=Hkv, window=W, keep=keep, dtype=wl.dtype,
                                max_tokens=S, keep_v=keep_v, **vkw)
        first = mk()
        w.alg_bytes = first.algorithmic_bytes_per_token * Hkv * sum(lens)
        w.copies = max(1, min(64, -(-4 * l2 // max(w.alg_bytes, 1))))
        w.caches = [first] + [mk() for _ in range(w.copies - 1)]
        for c in w.caches:               # compress (prefill side): timed for information
            c.compress(wl.q_win, wl.k, wl.v, wl.seq_lens)
        torch.cuda.synchronize()
        ev[0].record()
        for c in w.caches:
            c.compress(wl.q_win, wl.k, wl.v, wl.seq_lens)
        ev[1].record()
        torch.cuda.synchronize()
        w.compress_us = ev[0].elapsed_time(ev[1]) * 1e3 / len(w.caches)
        w.compress_bytes = Hkv * sum(lens) * (2 * D * esize + first.page_bytes // 16)
        w.compress_what = "prune the whole batch"
        out = torch.empty(Bn, Hq, D, dtype=torch.float32, device="cuda")
        w.step_sets = [[(c, wl.q, out)] for c in w.caches]
        w.oracle_inputs = lambda: (wl.q.cpu(), wl.k.cpu(), wl.v.cpu(), wl.seq_lens.cpu(), wl.q_win.cpu())
        w.oracle_sample = "one full decode step of the workload, median of 3"
    return w


def time_work(work, steps, warmup, flags, dist, torch, stream, sampler):
    """Times `steps` decode steps of `work` launched with `flags`.  Returns a dict: us_step (the single
    bracketed K-step region, max over ranks), median_us / min_us over >= MIN_REPLAYS individually timed graph
    replays, the clock record of the region, and the kernels launched in it."""
    from paper_2508_15212_b200 import dist_utils
    for c in work.caches:
        c.params.flags = flags
    n_sets, lps = len(work.step_sets), work.launches_per_step

    def launch(i):
        for cache, q, out in work.step_sets[i % n_sets]:
            cache.decode(q, out=out)

    def capture(n):
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=stream):
            for i in range(n):
                launch(i)
        return g

    with torch.cuda.stream(stream):
        for i in range(max(warmup, 3)):
            launch(i)
    stream.synchronize()
    spg = min(steps, max(1, (20 * n_sets) // lps))            # steps per graph: a whole number of rotations
    g_main = capture(spg)
    n_rep, rem = divmod(steps, spg)
    g_rem = capture(rem) if rem else None
    with torch.cuda.stream(stream):
        g_main.replay()
        if g_rem is not None:
            g_rem.replay()
    stream.synchronize()

    def timed_region():
        t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()
        with torch.cuda.stream(stream):
            g_main.replay()             # untimed: keeps the GPU busy while the timed launches are enqueued, so
            t0.record(stream)           # the region holds K steps and no host launch latency
            for _ in range(n_rep):
                g_main.replay()
            if g_rem is not None:
                g_rem.replay()
            t1.record(stream)
        stream.synchronize()
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
        return t0.elapsed_time(t1)

    with sampler:
        ms = timed_region()
        if len(sampler.samples) < 5:            # region shorter than the sampling period: sample under the same load
            t_end = time.time() + 0.25
            while time.time() < t_end:
                with torch.cuda.stream(stream):
                    g_main.replay()
                stream.synchronize()
    clocks = sampler.summary()
    ms = dist_utils.max_over_ranks(ms, dist, "cuda")
    # the same graph replayed on its own, each replay between its own pair of events
    n_stat = MIN_REPLAYS if lps > 1 else max(MIN_REPLAYS, min(200, n_rep))
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n_stat)]
    with torch.cuda.stream(stream):
        for a, b in evs:
            a.record(stream)
            g_main.replay()
            b.record(stream)
    stream.synchronize()
    per = sorted(a.elapsed_time(b) * 1e3 / spg for a, b in evs)
    return {"us_step": ms * 1e3 / steps, "median_us": statistics.median(per), "min_us": per[0],
            "replays": n_stat, "steps_per_replay": spg, "clocks": clocks, "launches": steps * lps}


def oracle_check(work):
    """Oracle on the host cores for set 0 of `work`: (cpu_baseline dict, max|delta| of the GPU output, inputs)."""
    if work.oracle_inputs is None:
        return None, None, None
    q, k, v, lens, q_win = work.oracle_inputs()
    a, c, vm = oracle_prepare(q_win, k, v, lens, work.keep, work.keep_v, work.variant)
    t_or, cores, o_ref = oracle_decode_time(q, k, v, lens, a, c, vm)
    cache, qd, _ = work.step_sets[0][0]
    for cch in work.caches:
        cch.params.flags = 0
    got = cache.decode(qd).cpu().numpy()
    err = float(abs(got - o_ref).max())
    return ({"value": t_or * 1e6 * work.oracle_scale, "unit": "us/step", "cores": cores, "kind": "oracle",
             "sample": work.oracle_sample},
            err, (q, k, v, lens, a, c, vm))


def oracle_single_thread(prepared, cores):
    """The oracle's decode step on one thread (the plain, slow reference point), one run."""
    import ctypes
    import oracle
    q, k, v, lens, a, c, vm = prepared
    try:
        omp = ctypes.CDLL("libgomp.so.1")
    except OSError:
        return None
    omp.omp_set_num_threads(1)
    try:
        t0 = time.perf_counter()
        oracle_decode(q, k, v, lens, a, c, vm)
        dt = time.perf_counter() - t0
    finally:
        omp.omp_set_num_threads(int(cores))
    return {"value": dt * 1e6, "unit": "us/step", "cores": 1, "kind": "oracle",
            "sample": "one full decode step of the workload on one thread, one run"}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--config", type=int, default=1, help="index into the benchmark configurations (0-based)")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--keep", type=int, default=0, help="override the kept-channel count T")
    ap.add_argument("--ratio", type=float, default=None, help="pruning ratio (configuration 5 sweeps 0.3/0.5/0.7/0.8)")
    ap.add_argument("--ratio-v", type=float, default=None,
                    help="also prune value channels with this ratio (default: values stay dense)")
    ap.add_argument("--top-p", type=float, default=None, help="SparK-p: keep the channels that reach this share of a "
                    "token's saliency (the page holds up to --keep, default 128, channels per token)")
    ap.add_argument("--groups", type=str, default=None, help="SparK-g: comma-separated pruning ratios of the rank "
                    "groups, most salient first (e.g. 0.25,0.5,0.75,1.0)")
    ap.add_argument("--recovery", default="degenerate", choices=["degenerate", "gaussian", "exponential"])
    ap.add_argument("--seed", type=int, default=1, help="seed of the sampled-recovery draws")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-sweep", action="store_true", help="time only the workload named by --config")
    ap.add_argument("--batch", type=int, default=0, help="override the batch size (smaller cases for profiling)")
    args = ap.parse_args()

    from workloads import inputs
    from paper_2508_15212_b200 import binding as B
    from paper_2508_15212_b200 import build as spark_build

    rank_env = int(os.environ.get("RANK", "0"))
    if args.impl == "reference":        # the oracle arm touches nothing of the CUDA library
        import math
        keep_count = lambda d, ratio: int(math.floor((1.0 - ratio) * d + 1e-9))      # T = floor((1 - ratio) D)
    else:
        if rank_env == 0:
            spark_build.build()
        keep_count = B.spark_keep_count

    def resolve(index, ratio_override=None, batch=0):
        cfg = dict(inputs.CONFIGS[index])
        ratio = cfg["ratio"] if not isinstance(cfg["ratio"], tuple) else cfg["ratio"][1]
        if ratio_override is not None:
            ratio = ratio_override
        if batch:
            cfg["batch"] = batch
        cfg["ratio"] = ratio
        if isinstance(cfg["seq_lens"], tuple):
            cfg["seq_lens"] = list(cfg["seq_lens"])
        return cfg, keep_count(cfg["head_dim"], ratio)

    if args.impl == "reference":
        if rank_env != 0:
            return
        cfg, keep = resolve(args.config, args.ratio, args.batch)
        run_reference(args, cfg, args.keep or keep)
        return

    import torch
    from paper_2508_15212_b200 import dist_utils
    rank, world, local = dist_utils.env_ranks()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
    torch.cuda.set_device(local)
    dist = dist_utils.init_process_group("nccl", torch.device("cuda", local))
    if dist is not None:
        dist.barrier()                  # rank 0 has built the library
    B.lib()
    cfg, keep = resolve(args.config, args.ratio, args.batch)
    keep = args.keep or keep
    keep_v = B.spark_keep_count(cfg["head_dim"], args.ratio_v) if args.ratio_v is not None else 0
    variant = None
    recovery = {"degenerate": 0, "gaussian": 1, "exponential": 2}[args.recovery]
    if args.top_p is not None or args.groups or recovery:
        groups = [float(x) for x in args.groups.split(",")] if args.groups else None
        variant = dict(top_p=args.top_p, group_prune=groups, recovery=recovery, seed=args.seed if recovery else 0)
        if groups:
            keep = B.spark_group_keep(cfg["head_dim"], groups)
        elif args.top_p is not None:
            keep = args.keep or cfg["head_dim"]
        if "token_budget" in cfg or "n_layers" in cfg:
            raise SystemExit("the variant flags are wired for the single-layer configurations (0, 1, 2)")
    stream = torch.cuda.Stream()
    sampler = ClockSampler(local)
    peak, peak_kind = measured_peak()

    # ---- the headline workload ----
    work = build_work(args.config, cfg, keep, keep_v, rank, torch, B, variant)
    first = work.caches[0]
    t_plain = time_work(work, args.steps, args.warmup, 0, dist, torch, stream, sampler)
    t_pdl = time_work(work, args.steps, args.warmup, B.SPARK_FLAG_OVERLAP_PREVIOUS, dist, torch, stream, sampler)
    status = first.status()
    us_step = t_plain["us_step"]

    # ---- end to end through the public call: pinned host q -> device, decode, out -> pinned host ----
    for c in work.caches:
        c.params.flags = 0
    cur = torch.cuda.current_stream()
    bound = []
    for st in work.step_sets:           # spark_decode_attn_host: copy-in, step and copy-out enqueued by one call
        bound.append([(cache.bind_decode_host(q.cpu().pin_memory(),
                                              torch.empty(out.shape, dtype=torch.float32).pin_memory(),
                                              stream=cur.cuda_stream), q, out) for cache, q, out in st])
    h2d = sum(q.numel() * q.element_size() for _, q, _ in bound[0])
    d2h = sum(out.numel() * 4 for _, _, out in bound[0])
    e2e_steps = max(200, min(args.steps, 500)) if work.launches_per_step == 1 else max(10, min(args.steps, 50))

    def e2e_step(i):
        for call, _, _ in bound[i % len(bound)]:
            call()
        cur.synchronize()
    for i in range(20):
        e2e_step(i)
    if dist is not None:
        dist.barrier()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(e2e_steps):
        e2e_step(i)
    e1.record()
    torch.cuda.synchronize()
    e2e_us = dist_utils.max_over_ranks(e0.elapsed_time(e1), dist, "cuda") * 1e3 / e2e_steps
    # the same call with SPARK_FLAG_HOST_MAPPED: the query travels inside the launch (or is read by the kernel)
    # and the kernel writes the result into the pinned host buffer itself, no staging copies; reported beside
    # the staged figure; the e2e value is the faster of the two
    for c in work.caches:
        c.params.flags = B.SPARK_FLAG_HOST_MAPPED
    for i in range(20):
        e2e_step(i)
    torch.cuda.synchronize()
    e0.record()
    for i in range(e2e_steps):
        e2e_step(i)
    e1.record()
    torch.cuda.synchronize()
    e2e_mapped_us = dist_utils.max_over_ranks(e0.elapsed_time(e1), dist, "cuda") * 1e3 / e2e_steps
    host_out = bound[0][0][0].out_host.clone()
    for c in work.caches:
        c.params.flags = 0
    del bound

    # ---- oracle on the host cores (rank 0, N = 1 only) ----
    cpu_baseline, max_err, cpu_single = None, None, None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        cpu_baseline, max_err, prepared = oracle_check(work)
        if prepared is not None and args.config == 1 and not args.batch:
            cpu_single = oracle_single_thread(prepared, cpu_baseline["cores"])
        del prepared

    # ---- the other workloads of the target range (N = 1, default configuration only) ----
    sweep = []
    if world == 1 and args.config == 1 and not args.no_sweep and not keep_v and not args.batch and not args.keep \
            and variant is None:
        for idx in (2, 3, 4):
            torch.cuda.empty_cache()
            cfg_s, keep_s = resolve(idx)
            work_s = build_work(idx, cfg_s, keep_s, 0, rank, torch, B)
            steps_s = max(20, min(args.steps, 400))
            ts = time_work(work_s, steps_s, args.warmup, 0, dist, torch, stream, sampler)
            tp = time_work(work_s, steps_s, args.warmup, B.SPARK_FLAG_OVERLAP_PREVIOUS, dist, torch, stream, sampler)
            cb, err = None, None
            if not args.no_cpu_baseline:
                cb, err, _ = oracle_check(work_s)
            gb = work_s.alg_bytes / (ts["us_step"] * 1e-6) / 1e9
            sweep.append({"workload": cfg_s["name"], "config": workload_desc(cfg_s, keep_s, work_s.copies),
                          "steps": steps_s, "us_per_step": ts["us_step"], "median_us": ts["median_us"],
                          "min_us": ts["min_us"], "replays": ts["replays"], "us_per_step_pdl": tp["us_step"],
                          "algorithmic_bytes_per_step": work_s.alg_bytes, "hbm_gbs": gb,
                          "frac_of_measured": gb / peak, "frac_of_nominal": gb / NOMINAL_HBM_GBS,
                          "clocks": ts["clocks"], "max_abs_err_vs_oracle": err, "cpu_baseline": cb,
                          "device_status": work_s.caches[0].status(),
                          "compress": {"us": work_s.compress_us, "what": work_s.compress_what}})
            del work_s

    if rank == 0:
        gbs = work.alg_bytes / (us_step * 1e-6) / 1e9
        name = cfg["name"]
        lps = work.launches_per_step
        line = {
            "metric": METRIC, "value": us_step, "unit": "us/step", "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": us_step / 1e3, "higher_is_better": False,
            "scaling": "weak", "vs_baseline": None, "dtype": "f32", "storage_dtype": cfg["dtype"], "data": "synthetic",
            "config": dict(workload_desc(cfg, keep, work.copies, keep_v),
                           launch="ordinary launches, K steps replayed from CUDA graphs",
                           **({"variant": {k_: v_ for k_, v_ in variant.items() if v_}} if variant else {})),
            "replays": {"n": t_plain["replays"], "steps_per_replay": t_plain["steps_per_replay"],
                        "median_us_per_step": t_plain["median_us"], "min_us_per_step": t_plain["min_us"]},
            "value_pdl": t_pdl["us_step"],
            "value_pdl_note": ("same steps with SPARK_FLAG_OVERLAP_PREVIOUS (programmatic dependent launch): step i+1 "
                               "starts its page stream while step i drains; valid only when the kernel enqueued before "
                               "the step does not write the cache, so it is not the headline"),
            "hbm_gbs": gbs, "hbm_gbs_all_gpus": dist_utils.aggregate_throughput(work.alg_bytes / 1e9, world, us_step * 1e-6),
            "frac_of_nominal_8tbs": gbs / NOMINAL_HBM_GBS,
            "algorithmic_bytes_per_step": work.alg_bytes,
            "clocks": t_plain["clocks"],
            "e2e": {"value": min(e2e_us, e2e_mapped_us), "unit": "us/step", "h2d_bytes_per_step": h2d,
                    "d2h_bytes_per_step": d2h, "steps": e2e_steps,
                    "transport": ("SPARK_FLAG_HOST_MAPPED" if e2e_mapped_us < e2e_us else "staged copies"),
                    "value_staged_copies": e2e_us, "value_host_mapped": e2e_mapped_us,
                    "note": ("packed cache resident; per step one spark_decode_attn_host call (query in pinned host "
                             "memory -> device, the decode step, result -> pinned host memory) and a stream "
                             "synchronize; timed with both transports of that call, the value is the faster one: "
                             "staged = cudaMemcpyAsync in, kernel, cudaMemcpyAsync out; SPARK_FLAG_HOST_MAPPED = the "
                             "query bytes travel inside the kernel launch (up to 24 KB, else the kernel reads them "
                             "from the host buffer) and the kernel writes the result into the host buffer; the same "
                             "bytes cross the bus either way")},
            "gpu_launches": t_plain["launches"] * B.spark_last_launch_count(),
            "launches_per_step": lps,
            "roofline": {"bound": "hbm", "achieved": gbs, "peak": peak, "unit": "GB/s", "frac": gbs / peak,
                         "peak_kind": f"of {peak_kind}", "traffic": NCU_TRAFFIC_BYTES.get(name) if not keep_v else None,
                         "kernel": ("spark::decode_bf16_kernel" if cfg["dtype"] == "bf16" and not recovery
                                    else "spark::decode_scalar_kernel"),
                         "algorithmic_bytes_per_launch": work.alg_bytes / lps,
                         "avg_launch_us": us_step / lps},
            "cpu_baseline": cpu_baseline,
            "cpu_baseline_single_thread": cpu_single,
            "compress": None if work.compress_us is None else {
                "us": work.compress_us, "gbs": work.compress_bytes / (work.compress_us * 1e-6) / 1e9,
                "bytes": work.compress_bytes, "what": work.compress_what},
            "max_abs_err_vs_oracle": max_err, "device_status": status,
            "sweep": sweep,
        }
        print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
