"""Benchmark of the decode hot path: one step = append + tiered attention + mass update (decode_attn)
followed by one routing event (rebalance) over every (layer, sequence) unit of a synthetic workload.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config I] [--layers L] [--impl ours|reference]

Prints ONE JSON line.  `value` is whole-workload decode steps per second with all inputs resident in
HBM; `e2e` is the same loop through the host-buffer entry point (H2D of q/k_new/v_new and D2H of the
output inside the timed region); `roofline` is the attention kernel's algorithmic bytes per launch
over its CUDA-event duration, against the measured HBM copy bandwidth; `cpu_baseline` is the CPU
oracle timed on a bounded sample of the same workload on this host.
"""

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time
from dataclasses import replace

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import torch  # noqa: E402

from paper_2608_05326_b200 import sharding, workloads  # noqa: E402

METRIC = "decode_steps_per_sec"
UNIT = "steps/s"
HBM_FALLBACK_GBS = 6650.0
# dram__bytes_read.sum + dram__bytes_write.sum of one attention-kernel launch, from the ncu captures
# summarised under profiles/ (bytes per launch, keyed by workload name); None = not captured.
NCU_TRAFFIC_BYTES = {
    # profiles/decode_attn_c1x32.md: 440.83 MB read + 6.50 MB written per launch
    "c1-llama3-8b-32k": 446_080_000,
}


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=256)
    ap.add_argument("--warmup", type=int, default=8)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", type=int, default=1)
    ap.add_argument("--layers", type=int, default=None, help="stacked layers (config 1 defaults to 32)")
    ap.add_argument("--batch", type=int, default=None)
    ap.add_argument("--bits", type=int, default=None, help="config 4 sweep point")
    ap.add_argument("--fp-frac", type=float, default=None, help="config 4 sweep point")
    ap.add_argument("--rebalance-interval", type=int, default=1)
    ap.add_argument("--sink-windows", type=int, default=0, help="protected sink prefix, in windows (0 in every BASELINE config)")
    ap.add_argument("--recent-windows", type=int, default=0, help="filled windows kept in the protected recent region")
    ap.add_argument("--rank-mode", type=int, default=0, help="0 cumulative attention (Eq. 1), 1 decayed, 2 p-norm")
    ap.add_argument("--rank-param", type=float, default=0.0, help="lambda of the decayed score / p of the p-norm")
    ap.add_argument("--rope-base", type=float, default=0.0,
                    help="> 0: keys are stored pre-RoPE and rotated by the attention kernel (0 in every BASELINE config)")
    ap.add_argument("--prefill-score", type=int, default=0, metavar="N_OBS",
                    help="instead of the decode loop: time qevict_prefill_score (window scores of one layer's prompt from "
                         "N_OBS observation queries per head) and print its own JSON line")
    ap.add_argument("--timeline", action="store_true",
                    help="instead of the throughput run: load the tracing build of the library and print, per kernel, the "
                         "median start-to-end interval inside the pipelined step and the median gap to the kernel before "
                         "(device timer stamps; not a bench value)")
    ap.add_argument("--splits", type=int, default=0)
    ap.add_argument("--fixed-context", action="store_true", help="no appends (k_new = NULL)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--cpu-seconds", type=float, default=15.0)
    return ap.parse_args()


def make_workload(args, total_steps):
    kw = {}
    if args.config == 4:
        if args.bits is not None:
            kw["bits"] = args.bits
        if args.fp_frac is not None:
            kw["fp_frac"] = args.fp_frac
    wl = workloads.config(args.config, **kw)
    layers = args.layers if args.layers is not None else (32 if args.config == 1 else (8 if args.config == 3 else wl.n_layers))
    batch = args.batch if args.batch is not None else wl.batch
    return replace(wl, n_layers=layers, batch=batch, steps=total_steps, rebalance_interval=args.rebalance_interval,
                   sink_windows=args.sink_windows, recent_windows=args.recent_windows, rank_mode=args.rank_mode,
                   rank_param=args.rank_param, rope_base=args.rope_base)


def peak_hbm_gbs():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return HBM_FALLBACK_GBS, "fallback"


class ClockSampler:
    """Samples the SM clock and the throttle reasons through NVML (read-only queries) from a thread while
    the timed region runs."""

    REASONS = (("hw_slowdown", 0x8), ("hw_thermal_slowdown", 0x40), ("sw_thermal_slowdown", 0x20),
               ("sw_power_cap", 0x4))

    def __init__(self, index, period_s=0.002):
        self.index, self.period = index, period_s
        self.sm, self.power, self.reason_bits = [], [], 0
        self.max_mhz = None
        self._stop = threading.Event()
        self._thread = None
        self._nv = None

    def start(self):
        try:
            import pynvml
            pynvml.nvmlInit()
            visible = os.environ.get("CUDA_VISIBLE_DEVICES")
            phys = int(visible.split(",")[self.index]) if visible and visible.split(",")[self.index].isdigit() else self.index
            self._h = pynvml.nvmlDeviceGetHandleByIndex(phys)
            self._nv = pynvml
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self._h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self._nv = None
            return
        self._thread = threading.Thread(target=self._run, daemon=True)
        self._thread.start()

    def _run(self):
        nv = self._nv
        while not self._stop.is_set():
            try:
                self.sm.append(nv.nvmlDeviceGetClockInfo(self._h, nv.NVML_CLOCK_SM))
                self.power.append(nv.nvmlDeviceGetPowerUsage(self._h) / 1000.0)
                self.reason_bits |= int(nv.nvmlDeviceGetCurrentClocksEventReasons(self._h))
            except Exception:
                pass
            time.sleep(self.period)

    def stop(self):
        self._stop.set()
        if self._thread is not None:
            self._thread.join(timeout=2)
        reasons = [name for name, bit in self.REASONS if self.reason_bits & bit]
        return {"sm_mhz": statistics.median(self.sm) if self.sm else None, "sm_max_mhz": self.max_mhz,
                "reasons": reasons, "samples": len(self.sm),
                "power_w_max": max(self.power) if self.power else None}


# ------------------------------------------------------------------------------------------ ours
def build_inputs(wl, device):
    """All inputs of the run, resident on `device`: prompts are consumed by prefill layer by layer."""
    scores, queries, knew, vnew = [], [], [], []
    prompts = {}
    for u in range(wl.n_units):
        k, v = workloads.gen_prompt_kv(wl, u, device=device)
        s = workloads.place_planted(workloads.synthetic_window_scores(wl, u), workloads.planted_windows(wl, u),
                                    wl.fp_budget_windows, wl.q_budget_windows)
        scores.append(s)
        queries.append(workloads.gen_queries(wl, u, k, s, device=device))
        kn, vn = workloads.gen_new_kv(wl, u, device=device)
        knew.append(kn); vnew.append(vn)
        prompts[u] = (k, v)
        yield_layer = (u + 1) % wl.batch == 0
        if yield_layer:
            layer = u // wl.batch
            units = range(layer * wl.batch, (layer + 1) * wl.batch)
            yield ("layer", layer, torch.stack([prompts[x][0] for x in units]), torch.stack([prompts[x][1] for x in units]),
                   torch.stack([scores[x] for x in units]).to(device))
            for x in units:
                del prompts[x]
    shape_q = (wl.n_layers, wl.batch, wl.n_q_heads, wl.head_dim)
    shape_kv = (wl.n_layers, wl.batch, wl.n_kv_heads, wl.head_dim)
    q = torch.stack(queries, 1).reshape((wl.steps,) + shape_q).contiguous()
    kn = torch.stack(knew, 1).reshape((wl.steps,) + shape_kv).contiguous()
    vn = torch.stack(vnew, 1).reshape((wl.steps,) + shape_kv).contiguous()
    yield ("steps", q, kn, vn)


def attention_kernel_bytes(wl, stats, n_splits_hint=None):
    """Algorithmic bytes one attention-kernel launch must move: every live window once (Full and recent
    windows at 16 bit, Quantized windows as codes + parameters), the queries, the work list, and the
    partial results it writes."""
    m_f, m_q = wl.fp_window_bytes(), wl.q_window_bytes()
    n_fp = stats["n_full"] + stats["n_aged"] + stats.get("n_sink", 0)
    kv = n_fp * m_f + stats["n_quant"] * m_q + stats["n_open"] * m_f // 2
    live = n_fp + stats["n_quant"] + stats["n_open"]
    q_bytes = wl.n_units * wl.n_q_heads * wl.head_dim * 2
    lists = live * 8 + live * wl.n_q_heads * 8  # work list read, per-(head, window) records written
    return kv + q_bytes + lists


def run_ours(args, rank, world):
    if args.timeline:
        os.environ["QEVICT_TRACE_LIB"] = "1"  # read when the binding is first imported
    from paper_2608_05326_b200 import binding, build
    if rank == 0:
        build.build(trace=args.timeline)  # no-op when the in-tree library is newer than its sources
    if world > 1:
        torch.distributed.barrier()
    dev = torch.device("cuda", int(os.environ.get("LOCAL_RANK", 0)))
    torch.cuda.set_device(dev)
    K, W = args.steps, args.warmup
    phases = 2 + (0 if args.no_e2e else 1)
    total_steps = W + phases * K
    wl = make_workload(args, total_steps)
    wl = sharding.rank_workload(wl, rank)  # every rank owns its own sequences (weak scaling, no exchange)
    cfg = binding.make_config(wl.batch, wl.n_layers, wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.dtype, wl.window,
                              wl.quant_bits, wl.group_size, wl.fp_budget_windows, wl.q_budget_windows, wl.max_context,
                              rebalance_interval_hint=args.rebalance_interval, device=dev.index,
                              sink_windows=wl.sink_windows, recent_windows=wl.recent_windows, rank_mode=wl.rank_mode,
                              rank_param=wl.rank_param, rope_base=wl.rope_base)
    cache = binding.QEvictCache(cfg)
    if args.splits:
        cache.set_splits(args.splits)
    q = kn = vn = None
    for item in build_inputs(wl, dev):
        if item[0] == "layer":
            _, layer, k, v, s = item
            cache.prefill_assign(layer, k, v, s)
            torch.cuda.synchronize()
            del k, v
        else:
            _, q, kn, vn = item
    out = torch.empty_like(q[0])
    R = args.rebalance_interval
    append = not args.fixed_context

    def step(t):
        cache.decode_attn(-1, q[t], kn[t] if append else None, vn[t] if append else None, out)
        if (t + 1) % R == 0:
            cache.rebalance(-1)

    def barrier():
        if world > 1:
            torch.distributed.barrier()
        torch.cuda.synchronize()

    t = 0
    for _ in range(W):
        step(t); t += 1
    if args.timeline:
        cache.kernel_timeline()  # restart the record after the warm-up
        for _ in range(min(K, 250)):  # the library records 512 calls (two per step)
            step(t); t += 1
        line = timeline_summary(cache.kernel_timeline(), wl)
        cache.close()
        return line, wl
    # ---- timed region: device-resident inputs ----
    launches0 = cache.launch_count()
    sampler = ClockSampler(dev.index)
    sampler.start()
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    host_t0 = time.perf_counter()
    for _ in range(K):
        step(t); t += 1
    host_enqueue_s = time.perf_counter() - host_t0   # host time to enqueue the K steps (no synchronisation)
    e1.record()
    barrier()
    clocks = sampler.stop()
    ms = e0.elapsed_time(e1)
    launches = cache.launch_count() - launches0
    # ---- same loop with the attention kernel bracketed by events ----
    cache.set_kernel_timing(True)
    for _ in range(K):
        step(t); t += 1
    torch.cuda.synchronize()
    ktimes = cache.kernel_times()
    kernel_ms, kernel_n = ktimes["decode_attn"]
    cache.set_kernel_timing(False)
    stats = cache.stats()
    # ---- end to end: host buffers through the host entry point ----
    e2e = None
    if not args.no_e2e:
        qh = q[t:t + K].cpu().pin_memory(); knh = kn[t:t + K].cpu().pin_memory(); vnh = vn[t:t + K].cpu().pin_memory()
        outh = torch.empty_like(qh[0]).pin_memory()
        barrier()
        t0 = time.perf_counter()
        # every step: inputs leave pinned host memory, the step and its routing event are enqueued, and the host
        # waits until the result is in host memory before it sends the next step's inputs (the final barrier
        # waits for the last routing event)
        got = torch.cuda.Event()
        for i in range(K):
            cache.decode_attn_host_async(-1, qh[i], knh[i] if append else None, vnh[i] if append else None, outh)
            got.record()          # the result is in host memory once this event has passed
            if (t + i + 1) % R == 0:
                cache.rebalance(-1)
            got.synchronize()     # the routing event keeps running while the host turns around
        barrier()
        e2e_s = time.perf_counter() - t0
        h2d = qh[0].numel() * 2 + (2 * knh[0].numel() * 2 if append else 0)
        e2e = {"seconds": e2e_s, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": outh.numel() * 2}

    ms, e2e_s = sharding.max_over_ranks([ms, e2e["seconds"] if e2e else 0.0], device=dev)
    if e2e:
        e2e["seconds"] = e2e_s
    if rank != 0:
        cache.close()
        return None
    peak, peak_kind = peak_hbm_gbs()
    kbytes = attention_kernel_bytes(wl, stats)
    k_avg_ms = kernel_ms / max(kernel_n, 1)
    achieved = kbytes / (k_avg_ms * 1e-3) / 1e9 if k_avg_ms > 0 else 0.0
    line = {
        "metric": METRIC, "value": sharding.aggregate_steps_per_second(world, K, ms), "unit": UNIT, "n_gpus": world, "steps": K, "warmup": W,
        "ms_per_step": ms / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": wl.dtype,
        "data": "synthetic",
        "config": {
            "workload": "%s x %d layers x batch %d (layer-batched launches)" % (wl.name, wl.n_layers, wl.batch),
            "units_per_step": wl.n_units, "context": wl.context, "window": wl.window, "quant_bits": wl.quant_bits,
            "group_size": wl.group_size, "fp_budget_windows": wl.fp_budget_windows,
            "q_budget_windows": wl.q_budget_windows, "sink_windows": wl.sink_windows, "recent_windows": wl.recent_windows,
            "rebalance_interval": R, "append": append, "rope_base": wl.rope_base,
            "l2": "inputs larger than L2 (KV working set %.0f MB per step)" % (kbytes / 1e6),
        },
        "layer_steps_per_sec": world * K * wl.n_units / (ms * 1e-3),
        "clocks": clocks,
        "gpu_launches": int(launches),
        "roofline": {
            "bound": "hbm", "kernel": "decode_attn_kernel", "achieved": achieved, "peak": peak, "unit": "GB/s",
            "frac": achieved / peak, "peak_source": peak_kind + " copy bandwidth", "frac_of_8TBs": achieved / 8000.0,
            "bytes_per_launch": kbytes, "kernel_ms": k_avg_ms, "kernel_launches_timed": int(kernel_n),
            "kernel_share_of_step": k_avg_ms / (ms / K),
            "traffic": NCU_TRAFFIC_BYTES.get(wl.name),
        },
        "host_enqueue_us_per_step": round(host_enqueue_s * 1e6 / K, 2),
        "kernel_us_per_step": {k: round(v[0] * 1e3 / K, 2) for k, v in ktimes.items()},
        "tier_state": {k: stats[k] for k in ("n_full", "n_quant", "n_aged", "n_sink", "n_open", "n_evicted", "promotions",
                                             "quantizations", "reactivations", "deletions")},
    }
    if e2e:
        line["e2e"] = {"value": world * K / e2e["seconds"], "unit": UNIT, "h2d_bytes_per_step": e2e["h2d_bytes_per_step"],
                       "d2h_bytes_per_step": e2e["d2h_bytes_per_step"]}
    cache.close()
    return line, wl


# ------------------------------------------------------------------------------------- CPU oracle
def timeline_summary(records, wl):
    """Per kernel: median duration and median gap since the end of the launch before it, over the launches the
    tracing library recorded."""
    import statistics
    dur, gap, period = {}, {}, []
    last_append = None
    for i, (name, t0, t1) in enumerate(records):
        dur.setdefault(name, []).append(t1 - t0)
        if i:
            gap.setdefault(name, []).append(t0 - records[i - 1][2])
        if name == "append":
            if last_append is not None:
                period.append(t0 - last_append)
            last_append = t0
    med = statistics.median
    return {"metric": "kernel_timeline", "unit": "us", "data": "synthetic", "launches": len(records),
            "config": {"workload": wl.name},
            "median_us": {k: round(med(v), 2) for k, v in dur.items()},
            "median_gap_before_us": {k: round(med(v), 2) for k, v in gap.items()},
            "median_step_period_us": round(med(period), 2) if period else None,
            "last_step": [(n, round(a, 2), round(b, 2)) for n, a, b in records[-5:]]}


def oracle_threads():
    try:
        from threadpoolctl import threadpool_info
        n = [p.get("num_threads", 1) for p in threadpool_info()]
        return max(n) if n else 1
    except Exception:
        return 1


def time_oracle(wl, n_steps, warmup, budget_s):
    """Times the CPU oracle, as it stands, on unit 0 of the workload: `n_steps` decode + rebalance steps
    (at most `budget_s` seconds).  Returns (whole-workload steps/s, description)."""
    import numpy as np

    from oracle import OracleConfig, UnitOracle
    aged = (wl.rebalance_interval + wl.window - 1) // wl.window + 1
    ocfg = OracleConfig(wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.dtype, wl.window, wl.quant_bits, wl.group_size,
                        wl.fp_budget_windows, wl.q_budget_windows, wl.max_context, aged_windows=aged,
                        sink_windows=wl.sink_windows, recent_windows=wl.recent_windows, rank_mode=wl.rank_mode,
                        rank_param=wl.rank_param)
    k, v = workloads.gen_prompt_kv(wl, 0)
    s = workloads.place_planted(workloads.synthetic_window_scores(wl, 0), workloads.planted_windows(wl, 0),
                                wl.fp_budget_windows, wl.q_budget_windows)
    q = workloads.gen_queries(wl, 0, k, s).double().numpy()
    kn, vn = workloads.gen_new_kv(wl, 0)
    kn, vn = kn.double().numpy(), vn.double().numpy()
    orc = UnitOracle(ocfg)
    orc.prefill_assign(k.double().numpy(), v.double().numpy(), s.numpy())
    del k, v
    t = 0
    for _ in range(warmup):
        orc.decode_attn(q[t], kn[t], vn[t]); orc.rebalance(); t += 1
    done = 0
    t0 = time.perf_counter()
    while done < n_steps and t < q.shape[0] and time.perf_counter() - t0 < budget_s:
        orc.decode_attn(q[t], kn[t], vn[t])
        if (t + 1) % wl.rebalance_interval == 0:
            orc.rebalance()
        t += 1; done += 1
    dt = time.perf_counter() - t0
    unit_steps_per_s = done / dt
    value = unit_steps_per_s / wl.n_units
    sample = "unit 0 of %d, %d decode+rebalance steps in %.1f s" % (wl.n_units, done, dt)
    return value, sample, done, dt


def run_reference(args, rank):
    if rank != 0:
        return None
    K, W = args.steps, args.warmup
    wl = make_workload(args, max(W + K, 8))
    value, sample, done, dt = time_oracle(wl, K, W, budget_s=180.0)
    cores = oracle_threads()
    return {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": done,
        "warmup": W, "ms_per_step": 1e3 / value, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64", "data": "synthetic",
        "config": {"workload": "%s x %d layers x batch %d" % (wl.name, wl.n_layers, wl.batch), "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }


def run_prefill_score(args):
    """Prefill-side step of the path (not part of the decode metric): window scores of the prompt on the GPU."""
    from paper_2608_05326_b200 import binding, build
    build.build()
    dev = torch.device("cuda", int(os.environ.get("LOCAL_RANK", 0)))
    torch.cuda.set_device(dev)
    wl = replace(workloads.config(args.config), n_layers=1)
    cfg = binding.make_config(wl.batch, 1, wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.dtype, wl.window, wl.quant_bits,
                              wl.group_size, wl.fp_budget_windows, wl.q_budget_windows, wl.max_context, device=dev.index)
    cache = binding.QEvictCache(cfg)
    k = torch.stack([workloads.gen_prompt_kv(wl, u, device=dev)[0] for u in range(wl.batch)])
    g = torch.Generator(device=dev).manual_seed(wl.seed)
    q = torch.randn((wl.batch, args.prefill_score, wl.n_q_heads, wl.head_dim), generator=g, device=dev).to(wl.torch_dtype)
    for _ in range(max(3, args.warmup)):
        s = cache.prefill_score(k, q)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    n = max(1, min(args.steps, 50))
    e0.record()
    for _ in range(n):
        s = cache.prefill_score(k, q)
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / n
    line = {"metric": "prefill_score_ms", "value": ms, "unit": "ms", "higher_is_better": False, "n_gpus": 1, "steps": n,
            "dtype": wl.dtype, "data": "synthetic",
            "config": {"workload": "%s, one layer, %d observation queries per head" % (wl.name, args.prefill_score),
                       "key_bytes": k.numel() * 2},
            "mass_sum": float(s.sum()), "expected_mass_sum": float(wl.batch * args.prefill_score * wl.n_q_heads)}
    cache.close()
    return line


def main():
    args = parse_args()
    rank = int(os.environ.get("RANK", 0))
    world = int(os.environ.get("WORLD_SIZE", 1))
    if args.prefill_score > 0:
        if rank == 0:
            print(json.dumps(run_prefill_score(args)))
        return
    if args.impl == "reference":
        line = run_reference(args, rank)
        if line is not None:
            print(json.dumps(line))
        return
    if world > 1:
        torch.distributed.init_process_group("nccl")
    res = run_ours(args, rank, world)
    if rank == 0:
        line, wl = res
        if not args.timeline and not args.no_cpu_baseline and world >= 1:
            small = replace(wl, steps=256, seed=wl.seed)
            value, sample, _, _ = time_oracle(small, 1000, 1, budget_s=args.cpu_seconds)
            line["cpu_baseline"] = {"value": value, "unit": UNIT, "cores": oracle_threads(), "kind": "oracle", "sample": sample}
        print(json.dumps(line))
    if world > 1:
        torch.distributed.destroy_process_group()


if __name__ == "__main__":
    main()
