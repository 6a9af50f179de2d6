#!/usr/bin/env python
"""Benchmark of the SparK decode step (spark_decode_attn) on synthetic Llama-3.1-8B-shaped caches.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config I] [--impl ours|reference]

One "step" is one spark_decode_attn call over the whole packed cache of the workload (all sequences,
all heads).  The cache is compressed once, outside the timed region (prefill side); its time is reported
under "compress".  Steps rotate over several copies of the packed cache so that each launch reads cold
data (copies * bytes >= 4 * L2).  The timed region is K launches replayed from CUDA graphs, bracketed by
CUDA events on the launching stream.  With N > 1 (torchrun) every rank runs the same workload on its own
GPU with no data-path collective (weak scaling); the reported time is the max over ranks.

--impl reference times the CPU oracle on the host cores instead (it is a deliberately plain program).
Prints ONE JSON line on rank 0.
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
# dram__bytes_read.sum + dram__bytes_write.sum per decode launch from the ncu capture summarised in
# profiles/ (bytes); None until a capture exists for the workload.
NCU_TRAFFIC_BYTES = {"llama8b_32k": 109.3e6, "llama8b_4x128k": 1391.7e6}      # profiles/decode_bf16_llama8b_32k.md


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


def oracle_decode_time(wl_cpu, keep, reps=3, keep_v=0):
    """Times the CPU oracle's decode (window mean and compress are prepared, untimed)."""
    import oracle
    Hkv = wl_cpu.k.shape[1]
    _, a = oracle.window_mean(wl_cpu.q_win, Hkv)
    c = oracle.compress(wl_cpu.k, wl_cpu.seq_lens, keep, a)
    vm = oracle.prune_values(wl_cpu.v, wl_cpu.seq_lens, keep_v) if 0 < keep_v < 128 else None
    oracle.decode_attn(wl_cpu.q, wl_cpu.k, wl_cpu.v, wl_cpu.seq_lens, c["mask"], c["mu"], a, vmask=vm)   # warm
    ts = []
    for _ in range(reps):
        t0 = time.perf_counter()
        out, _ = oracle.decode_attn(wl_cpu.q, wl_cpu.k, wl_cpu.v, wl_cpu.seq_lens, c["mask"], c["mu"], a, vmask=vm)
        ts.append(time.perf_counter() - t0)
    return statistics.median(ts), oracle.threads(), out


def workload_desc(cfg, keep, copies=None, keep_v=0):
    d = {"workload": cfg["name"], "batch": cfg["batch"], "n_q_heads": cfg["n_q_heads"],
         "n_kv_heads": cfg["n_kv_heads"], "head_dim": cfg["head_dim"], "cached_tokens": cfg["seq_lens"],
         "window": cfg["window"], "pruning_ratio": cfg["ratio"], "keep": keep, "page_tokens": 16}
    if 0 < keep_v < 128:
        d["value_keep"] = keep_v                     # value-channel pruning on top of the named workload
    if copies is not None:
        d["cold_cache"] = f"rotation over {copies} packed-cache copies (copies*bytes >= 4*L2)"
    return d


def run_reference(args, cfg, keep):
    """The oracle as the reference arm: a bounded sample (one full decode step per timed step)."""
    import torch
    from workloads import inputs
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    wl = inputs.config_workload(args.config, device="cpu")
    inputs.enforce_saliency_gap(wl, keep)
    import oracle
    Hkv = wl.k.shape[1]
    _, a = oracle.window_mean(wl.q_win, Hkv)
    c = oracle.compress(wl.k, wl.seq_lens, keep, a)
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
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-overlap", action="store_true",
                    help="ordinary launches (default: each step may start its page stream while the previous drains)")
    ap.add_argument("--batch", type=int, default=0, help="override the batch size (smaller cases for profiling)")
    args = ap.parse_args()

    import torch
    from workloads import inputs
    from paper_2508_15212_b200 import binding as B
    cfg = dict(inputs.CONFIGS[args.config])
    ratio = cfg["ratio"] if not isinstance(cfg["ratio"], tuple) else cfg["ratio"][1]
    if args.ratio is not None:
        ratio = args.ratio
    if args.batch:
        cfg["batch"] = args.batch
    cfg["ratio"] = ratio
    keep = args.keep or B.spark_keep_count(cfg["head_dim"], ratio)
    keep_v = B.spark_keep_count(cfg["head_dim"], args.ratio_v) if args.ratio_v is not None else 0
    if isinstance(cfg["seq_lens"], tuple):
        cfg["seq_lens"] = list(cfg["seq_lens"])

    if args.impl == "reference":
        run_reference(args, cfg, keep)
        return

    from paper_2508_15212_b200 import build as spark_build
    from paper_2508_15212_b200.cache import SparkCache

    from paper_2508_15212_b200 import dist_utils
    rank, world, local = dist_utils.env_ranks()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
    torch.cuda.set_device(local)
    dist = dist_utils.init_process_group("nccl", torch.device("cuda", local))
    if rank == 0:
        spark_build.build()
    if dist is not None:
        dist.barrier()
    B.lib()

    # ---- workload (weak scaling: every rank holds its own copy of the configuration) ----
    # A step is a list of (cache, q, out) decode launches: one for the single-layer configurations
    # (rotating over cold copies), 28 (one per layer) for the Qwen-shaped configuration.
    from workloads.batches import build_evicted_batch, permuted_block_table
    l2 = torch.cuda.get_device_properties(local).L2_cache_size
    flags = 0 if args.no_overlap else B.SPARK_FLAG_OVERLAP_PREVIOUS
    D = cfg["head_dim"]
    esize = 2 if cfg["dtype"] == "bf16" else 4
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
    wl = None
    step_sets = []                     # step i uses step_sets[i % len(step_sets)]
    compress_us = compress_bytes = None
    if "token_budget" in cfg:          # prompts evicted and pruned one at a time into one batch cache
        per_tok = B.spark_algorithmic_bytes_per_token(B.make_params(
            batch=1, n_q_heads=cfg["n_q_heads"], n_kv_heads=cfg["n_kv_heads"], window=cfg["window"], keep=keep,
            dtype=torch.bfloat16 if cfg["dtype"] == "bf16" else torch.float32, n_pool_pages=1, keep_v=keep_v))
        alg_bytes = per_tok * cfg["n_kv_heads"] * cfg["token_budget"] * cfg["batch"]
        copies = max(1, -(-4 * l2 // alg_bytes))
        for c in range(copies):
            cache, q, _, _ = build_evicted_batch(cfg, keep, seed_offset=dist_utils.rank_seed_offset(rank, c), flags=flags,
                                                     keep_v=keep_v)
            out = torch.empty(cfg["batch"], cfg["n_q_heads"], D, dtype=torch.float32, device="cuda")
            step_sets.append([(cache, q, out)])
            prep = sorted(cache.prep_us)
        cfg["cached_tokens_after_eviction"] = cfg["token_budget"]
        compress_us, compress_bytes = prep[len(prep) // 2], 2 * cfg["n_kv_heads"] * int(cfg["seq_lens"]) * D * esize
    elif "n_layers" in cfg:            # paged pool, variable lengths, all layers per step
        copies, alg_bytes, layer_set = 1, 0, []
        for layer in range(cfg["n_layers"]):
            wl_l = inputs.config_workload(args.config, device="cuda", seed_offset=dist_utils.rank_seed_offset(rank, layer))
            Bn, Hq, Hkv, W, _, S = wl_l.shape
            lens = wl_l.seq_lens.tolist()
            table, n_pages = permuted_block_table(Bn, Hkv, lens, "cuda", seed=977 * layer + rank)
            cache = SparkCache(batch=Bn, n_q_heads=Hq, n_kv_heads=Hkv, window=W, keep=keep, dtype=wl_l.dtype,
                               max_tokens=S, block_table=table, n_pool_pages=n_pages, flags=flags, keep_v=keep_v)
            cache.compress(wl_l.q_win, wl_l.k, wl_l.v, wl_l.seq_lens)
            alg_bytes += cache.algorithmic_bytes_per_token * Hkv * sum(lens)
            layer_set.append((cache, wl_l.q.clone(), torch.empty(Bn, Hq, D, dtype=torch.float32, device="cuda")))
            total_tokens = locals().get("total_tokens", 0) + sum(lens)
            del wl_l
            torch.cuda.empty_cache()
        step_sets.append(layer_set)
        cfg["seq_lens"] = (f"uniform[8192,131072] per sequence, independent per layer; "
                           f"{total_tokens} tokens over {cfg['n_layers']} layers")
    else:
        wl = inputs.config_workload(args.config, device="cuda", seed_offset=dist_utils.rank_seed_offset(rank),
                                    batch=cfg["batch"])
        inputs.enforce_saliency_gap(wl, keep)
        Bn, Hq, Hkv, W, _, S = wl.shape
        lens = wl.seq_lens.tolist()
        mk = lambda: SparkCache(batch=Bn, n_q_heads=Hq, n_kv_heads=Hkv, window=W, keep=keep, dtype=wl.dtype,
                                max_tokens=S, flags=flags, keep_v=keep_v)
        first = mk()
        alg_bytes = first.algorithmic_bytes_per_token * Hkv * sum(lens)
        copies = max(1, min(64, -(-4 * l2 // max(alg_bytes, 1))))
        caches = [first] + [mk() for _ in range(copies - 1)]
        for c in caches:               # compress (prefill side): timed for information
            c.compress(wl.q_win, wl.k, wl.v, wl.seq_lens)
        torch.cuda.synchronize()
        ev[0].record()
        for c in caches:
            c.compress(wl.q_win, wl.k, wl.v, wl.seq_lens)
        ev[1].record()
        torch.cuda.synchronize()
        compress_us = ev[0].elapsed_time(ev[1]) * 1e3 / len(caches)
        compress_bytes = Hkv * sum(lens) * (2 * D * esize + first.page_bytes // 16)
        out = torch.empty(Bn, Hq, D, dtype=torch.float32, device="cuda")
        step_sets = [[(c, wl.q, out)] for c in caches]
    launches_per_step = len(step_sets[0])
    first = step_sets[0][0][0]
    stream = torch.cuda.Stream()

    def launch(i):
        for cache, q, out in step_sets[i % len(step_sets)]:
            cache.decode(q, out=out)

    # ---- graphs of decode launches ----
    def capture(n):
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=stream):
            for i in range(n):
                launch(i)
        return g

    with torch.cuda.stream(stream):
        for i in range(max(args.warmup, 3)):
            launch(i)
    stream.synchronize()
    spg = min(args.steps, max(1, (20 * len(step_sets)) // launches_per_step))
    g_main = capture(spg)
    n_rep, rem = divmod(args.steps, spg)
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
            t0.record(stream)
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

    sampler = ClockSampler(local)
    with sampler:
        ms = timed_region()
        if len(sampler.samples) < 5:            # region shorter than the sampling period: sample under the same load
            t_end = time.time() + 0.25
            while time.time() < t_end:
                with torch.cuda.stream(stream):
                    g_main.replay()
                stream.synchronize()
    ms = dist_utils.max_over_ranks(ms, dist, "cuda")
    us_step = ms * 1e3 / args.steps
    status = first.status()

    # ---- end to end through the public call: pinned host q -> device, decode, out -> pinned host ----
    host = [[(q.cpu().pin_memory(), torch.empty(out.shape, dtype=torch.float32).pin_memory(), torch.empty_like(q))
             for _, q, out in st] for st in step_sets]
    h2d = sum(qh.numel() * qh.element_size() for qh, _, _ in host[0])
    d2h = sum(oh.numel() * 4 for _, oh, _ in host[0])
    e2e_steps = min(args.steps, 500 if launches_per_step == 1 else 50)

    def e2e_step(i):
        k = i % len(step_sets)
        for (cache, _, out), (qh, oh, qd) in zip(step_sets[k], host[k]):
            qd.copy_(qh, non_blocking=True)
            cache.decode(qd, out=out)
            oh.copy_(out, non_blocking=True)
        torch.cuda.current_stream().synchronize()
    for i in range(5):
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
    e2e_ms = e0.elapsed_time(e1)
    e2e_ms = dist_utils.max_over_ranks(e2e_ms, dist, "cuda")
    e2e_us = e2e_ms * 1e3 / e2e_steps

    # ---- oracle on the host cores (rank 0, N = 1 only) ----
    cpu_baseline, max_err = None, None
    if rank == 0 and world == 1 and not args.no_cpu_baseline and wl is not None:
        wl_cpu = wl.to("cpu")
        t_or, cores, o_ref = oracle_decode_time(wl_cpu, keep, keep_v=keep_v)
        cpu_baseline = {"value": t_or * 1e6, "unit": "us/step", "cores": cores, "kind": "oracle",
                        "sample": "one full decode step of the workload, median of 3"}
        max_err = float((first.decode(wl.q).cpu().numpy() - o_ref).__abs__().max())

    if rank == 0:
        peak, peak_kind = measured_peak()
        gbs = alg_bytes / (us_step * 1e-6) / 1e9
        name = cfg["name"]
        line = {
            "metric": METRIC, "value": us_step, "unit": "us/step", "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": us_step / 1e3, "higher_is_better": False,
            "scaling": "weak", "vs_baseline": None, "dtype": "f32", "storage_dtype": cfg["dtype"], "data": "synthetic",
            "config": dict(workload_desc(cfg, keep, copies, keep_v),
                           launch=("programmatic dependent launch: the page stream of step i+1 may start while step i "
                                   "drains; q, out and workspace wait for step i" if flags else "ordinary launches")),
            "hbm_gbs": gbs, "hbm_gbs_all_gpus": dist_utils.aggregate_throughput(alg_bytes / 1e9, world, us_step * 1e-6),
            "frac_of_nominal_8tbs": gbs / NOMINAL_HBM_GBS,
            "algorithmic_bytes_per_step": alg_bytes,
            "clocks": sampler.summary(),
            "e2e": {"value": e2e_us, "unit": "us/step", "h2d_bytes_per_step": h2d,
                    "d2h_bytes_per_step": d2h, "steps": e2e_steps,
                    "note": "packed cache resident; per step: pinned q -> device, spark_decode_attn, out -> pinned host, sync"},
            "gpu_launches": args.steps * launches_per_step * B.spark_last_launch_count(),
            "launches_per_step": launches_per_step,
            "roofline": {"bound": "hbm", "achieved": gbs, "peak": peak, "unit": "GB/s", "frac": gbs / peak,
                         "peak_kind": f"of {peak_kind}", "traffic": NCU_TRAFFIC_BYTES.get(name) if not keep_v else None,
                         "kernel": "spark::decode_bf16_kernel" if cfg["dtype"] == "bf16" else "spark::decode_f32_kernel",
                         "algorithmic_bytes_per_launch": alg_bytes / launches_per_step,
                         "avg_launch_us": us_step / launches_per_step},
            "cpu_baseline": cpu_baseline,
            "compress": None if compress_us is None else {
                "us": compress_us, "gbs": compress_bytes / (compress_us * 1e-6) / 1e9, "bytes": compress_bytes,
                "what": ("evict + prune one prompt (median; first call includes one-time set-up)" if "token_budget" in cfg
                         else "prune the whole batch")},
            "max_abs_err_vs_oracle": max_err, "device_status": status,
        }
        print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
