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

INPUT_POOL = 384        # distinct decode steps of inputs held on the device; longer runs go round the pool
SETTLE_STEPS = 256      # untimed steps right after prefill (state preparation, not warm-up).  A window is quantized
                        # once, at its first demotion; the windows that start in the full-precision tier go through that
                        # in the first couple of hundred steps after a prefill (at most K_f per sequence), a burst of
                        # page traffic that the steady state of a long generation does not see
IDLE_AFTER_SETTLE_S = 0.3
MIN_TIMED_SECONDS = 0.5 # a K-step loop shorter than this is repeated and the median repeat is reported
MAX_REPEATS = 9


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
    ap.add_argument("--settle-steps", type=int, default=SETTLE_STEPS,
                    help="untimed steps right after prefill, before the warm-up (state preparation)")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-also", action="store_true", help="default run only: skip the second target configuration (config 3 x 8 layers)")
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
def build_inputs(wl, n_input_steps, device):
    """All inputs of the run, resident on `device`: prompts are consumed by prefill layer by layer."""
    scores, queries, knew, vnew = [], [], [], []
    prompts = {}
    for u in range(wl.n_units):
        k, v = workloads.gen_prompt_kv(wl, u, device=device)
        s = workloads.place_planted(workloads.synthetic_window_scores(wl, u), workloads.planted_windows(wl, u),
                                    wl.fp_budget_windows, wl.q_budget_windows)
        scores.append(s)
        queries.append(workloads.gen_queries(wl, u, k, s, n_steps=n_input_steps, device=device))
        kn, vn = workloads.gen_new_kv(wl, u, n_steps=n_input_steps, device=device)
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
    q = torch.stack(queries, 1).reshape((n_input_steps,) + shape_q).contiguous()
    kn = torch.stack(knew, 1).reshape((n_input_steps,) + shape_kv).contiguous()
    vn = torch.stack(vnew, 1).reshape((n_input_steps,) + shape_kv).contiguous()
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


def dram_traffic_bytes(wl):
    """dram__bytes_read.sum + dram__bytes_write.sum of one attention-kernel launch on this workload, as recorded
    from an ncu capture in profiles/dram_traffic.txt (one line per workload: key, read bytes, write bytes, the
    summary the figures come from); None for a workload without a capture."""
    key = "%s/L%d/B%d/rope%d" % (wl.name, wl.n_layers, wl.batch, 1 if wl.rope_base > 0 else 0)
    try:
        with open(os.path.join(ROOT, "profiles", "dram_traffic.txt")) as f:
            for line in f:
                parts = line.split()
                if len(parts) >= 3 and parts[0] == key:
                    return int(parts[1]) + int(parts[2])
    except OSError:
        pass
    return None


def measure_workload(args, wl, rank, world, dev, K, W, with_e2e, timeline=False):
    """Builds the cache of `wl` on `dev`, runs the decode loop and returns the measurements of one workload."""
    from paper_2608_05326_b200 import binding
    Wwin = wl.window
    R = args.rebalance_interval
    append = not args.fixed_context
    # steps the run may take at most: settle + warm-up + the repeated timed loop + the event-bracketed loop + the
    # loop at the paper's interval (one routing event per filled window) + the end-to-end loop
    total_steps = args.settle_steps + W + (MAX_REPEATS + 1) * K + max(K, 4 * Wwin) + (5 * K if with_e2e else 0) + 2 * Wwin
    n_in = min(total_steps, INPUT_POOL)
    wl = replace(wl, steps=total_steps)  # sizes max_context for every token the run appends
    cfg = binding.make_config(wl.batch, wl.n_layers, wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.dtype, wl.window,
                              wl.quant_bits, wl.group_size, wl.fp_budget_windows, wl.q_budget_windows, wl.max_context,
                              rebalance_interval_hint=max(R, 1), device=dev.index,
                              sink_windows=wl.sink_windows, recent_windows=wl.recent_windows, rank_mode=wl.rank_mode,
                              rank_param=wl.rank_param, rope_base=wl.rope_base)
    cache = binding.QEvictCache(cfg)
    if args.splits:
        cache.set_splits(args.splits)
    q = kn = vn = None
    for item in build_inputs(wl, n_in, dev):
        if item[0] == "layer":
            _, layer, k, v, s = item
            cache.prefill_assign(layer, k, v, s)
            torch.cuda.synchronize()
            del k, v
        else:
            _, q, kn, vn = item
    out = torch.empty_like(q[0])
    state = {"t": 0}

    def step(interval=R):
        t = state["t"]
        i = t % n_in
        cache.decode_attn(-1, q[i], kn[i] if append else None, vn[i] if append else None, out)
        if (t + 1) % interval == 0:
            cache.rebalance(-1)
        state["t"] = t + 1

    def barrier():
        if world > 1:
            torch.distributed.barrier()
        torch.cuda.synchronize()

    def timed_loop(n, interval=R):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        e0.record()
        h0 = time.perf_counter()
        for _ in range(n):
            step(interval)
        host_s = time.perf_counter() - h0   # host time to enqueue the steps (no synchronisation)
        e1.record()
        barrier()
        return e0.elapsed_time(e1), host_s

    for _ in range(args.settle_steps):
        step()
    if args.settle_steps > 0:
        # the settle steps are state preparation; let the board's power window empty before the warm-up so that they
        # do not push the timed region under the software power cap (the long runs show the sustained figure)
        torch.cuda.synchronize()
        time.sleep(IDLE_AFTER_SETTLE_S)
    for _ in range(W):
        step()
    if timeline:
        cache.kernel_timeline()  # restart the record after the warm-up
        for _ in range(min(K, 250)):  # the library records 512 calls (two per step)
            step()
        line = timeline_summary(cache.kernel_timeline(), wl)
        cache.close()
        return line
    # ---- timed region: device-resident inputs; K steps, repeated while a loop is shorter than MIN_TIMED_SECONDS ----
    launches0 = cache.launch_count()
    sampler = ClockSampler(dev.index)
    sampler.start()
    loops = [timed_loop(K)]
    first_ms = sharding.max_over_ranks([loops[0][0]], device=dev)[0]
    repeats = 1 if first_ms * 1e-3 >= MIN_TIMED_SECONDS else MAX_REPEATS
    while len(loops) < repeats:
        loops.append(timed_loop(K))
    clocks = sampler.stop()
    launches = cache.launch_count() - launches0
    rep_order = sharding.max_over_ranks([ms for ms, _ in loops], device=dev) if world > 1 else [ms for ms, _ in loops]
    rep_ms = sorted(rep_order)
    ms = statistics.median(rep_ms)
    host_enqueue_s = statistics.median(h for _, h in loops)
    # ---- same loop with every kernel bracketed by events ----
    cache.set_kernel_timing(True)
    for _ in range(K):
        step()
    torch.cuda.synchronize()
    ktimes = cache.kernel_times()
    kernel_ms, kernel_n = ktimes["decode_attn"]
    cache.set_kernel_timing(False)
    stats = cache.stats()
    # ---- the paper's coupling of window and interval: one routing event per filled window (every W steps) ----
    interval_w = None
    if R != Wwin and not args.fixed_context:
        while state["t"] % Wwin:
            step()  # reach a window boundary with routing after every step, as before
        n_w = max(K, 4 * Wwin) // Wwin * Wwin
        ms_w, _ = timed_loop(n_w, interval=Wwin)
        ms_w = sharding.max_over_ranks([ms_w], device=dev)[0]
        interval_w = (ms_w, n_w)
    # ---- end to end: host buffers through the host entry point ----
    e2e = None
    if with_e2e:
        idx = [(state["t"] + i) % n_in for i in range(K)]
        qh = q[idx].cpu().pin_memory(); knh = kn[idx].cpu().pin_memory(); vnh = vn[idx].cpu().pin_memory()
        outh = torch.empty_like(qh[0]).pin_memory()
        # every step: inputs leave pinned host memory, the step and its routing event are enqueued, and the host
        # waits until the result is in host memory (qevict_wait_result: an event behind the write of `out`) before it
        # sends the next step's inputs (the final barrier waits for the last routing event).  A K-step loop shorter
        # than a quarter of a second is repeated (5 times) and the median repeat is reported: the host side of this
        # loop is noisier than the device side
        e2e_reps = []
        while True:
            barrier()
            t0 = time.perf_counter()
            for i in range(K):
                cache.decode_attn_host_async(-1, qh[i], knh[i] if append else None, vnh[i] if append else None, outh)
                if (state["t"] + i + 1) % R == 0:
                    cache.rebalance(-1)
                cache.wait_result()   # the result is in host memory; the routing event keeps running while the host turns around
            barrier()
            e2e_reps.append(sharding.max_over_ranks([time.perf_counter() - t0], device=dev)[0])
            state["t"] += K
            if e2e_reps[0] >= 0.25 or len(e2e_reps) >= 5:
                break
        e2e_s = statistics.median(e2e_reps)
        h2d = qh[0].numel() * 2 + (2 * knh[0].numel() * 2 if append else 0)
        e2e = {"seconds": e2e_s, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": outh.numel() * 2}
    cache.close()
    if rank != 0:
        return None
    peak, peak_kind = peak_hbm_gbs()
    kbytes = attention_kernel_bytes(wl, stats)
    k_avg_ms = kernel_ms / max(kernel_n, 1)
    achieved = kbytes / (k_avg_ms * 1e-3) / 1e9 if k_avg_ms > 0 else 0.0
    step_gbs = kbytes / (ms / K * 1e-3) / 1e9
    res = {
        "workload": "%s x %d layers x batch %d (layer-batched launches)" % (wl.name, wl.n_layers, wl.batch),
        "wl": wl, "K": K, "ms": ms, "rep_ms": rep_ms, "rep_order": rep_order, "repeats": len(rep_ms), "launches": int(launches), "clocks": clocks,
        "host_enqueue_us_per_step": round(host_enqueue_s * 1e6 / K, 2),
        "kernel_us_per_step": {k: round(v[0] * 1e3 / K, 2) for k, v in ktimes.items()},
        "stats": stats, "e2e": e2e, "kbytes": kbytes,
        "roofline": {
            "bound": "hbm", "kernel": "decode_attn_kernel", "achieved": achieved, "peak": peak, "unit": "GB/s",
            "frac": achieved / peak, "peak_source": peak_kind + " copy bandwidth", "frac_of_8TBs": achieved / 8000.0,
            "bytes_per_launch": kbytes, "kernel_ms": k_avg_ms, "kernel_launches_timed": int(kernel_n),
            "kernel_share_of_step": k_avg_ms / (ms / K),
            # the whole step (append + attention + combine + route + migrate) against the same algorithmic bytes
            "step_frac": step_gbs / peak, "step_frac_of_8TBs": step_gbs / 8000.0,
            "traffic": dram_traffic_bytes(wl),
        },
    }
    if interval_w:
        ms_w, n_w = interval_w
        gbs_w = kbytes / (ms_w / n_w * 1e-3) / 1e9
        res["interval_w"] = {"rebalance_interval": Wwin, "steps": n_w, "ms_per_step": ms_w / n_w,
                             "value": world * n_w / (ms_w * 1e-3), "step_frac": gbs_w / peak, "step_frac_of_8TBs": gbs_w / 8000.0}
    return res


def measure_two_streams(args, wl, dev, K, W, kbytes):
    """The same workload as two caches of half the layers each, stepped on two streams: the sequences of different
    caches are independent, so one cache's table kernels (append, combine, route, migrate) run under the other
    cache's attention kernel.  A pattern of the caller's, not of the library: reported beside the headline."""
    from paper_2608_05326_b200 import binding
    half = replace(wl, n_layers=wl.n_layers // 2)
    total_steps = args.settle_steps + W + (MAX_REPEATS + 1) * K + max(K, 4 * wl.window) + 3 * wl.window
    n_in = min(total_steps, INPUT_POOL)
    half = replace(half, steps=total_steps)
    groups = []
    for gidx in range(2):
        wl_g = replace(half, seed=half.seed + 101 * gidx)
        cfg = binding.make_config(wl_g.batch, wl_g.n_layers, wl_g.n_q_heads, wl_g.n_kv_heads, wl_g.head_dim, wl_g.dtype,
                                  wl_g.window, wl_g.quant_bits, wl_g.group_size, wl_g.fp_budget_windows,
                                  wl_g.q_budget_windows, wl_g.max_context, rebalance_interval_hint=1, device=dev.index)
        cache = binding.QEvictCache(cfg)
        q = kn = vn = None
        for item in build_inputs(wl_g, n_in, dev):
            if item[0] == "layer":
                _, layer, k, v, s = item
                cache.prefill_assign(layer, k, v, s)
                torch.cuda.synchronize()
                del k, v
            else:
                _, q, kn, vn = item
        groups.append((cache, q, kn, vn, torch.empty_like(q[0]), torch.cuda.Stream(device=dev)))
    state = {"t": 0}

    def step(interval=1):
        i = state["t"] % n_in
        for cache, q, kn, vn, out, stream in groups:
            cache.decode_attn(-1, q[i], kn[i], vn[i], out, stream=stream)
            if (state["t"] + 1) % interval == 0:
                cache.rebalance(-1, stream=stream)
        state["t"] += 1

    def timed(n, interval=1):
        torch.cuda.synchronize()
        starts = [torch.cuda.Event(enable_timing=True) for _ in groups]
        ends = [torch.cuda.Event(enable_timing=True) for _ in groups]
        for ev, g in zip(starts, groups):
            ev.record(g[5])
        for _ in range(n):
            step(interval)
        for ev, g in zip(ends, groups):
            ev.record(g[5])
        torch.cuda.synchronize()
        return max(starts[0].elapsed_time(e) for e in ends)  # from the first start to the last end

    for _ in range(args.settle_steps):
        step()
    torch.cuda.synchronize()
    time.sleep(IDLE_AFTER_SETTLE_S)
    for _ in range(W):
        step()
    reps = [timed(K) for _ in range(MAX_REPEATS)]
    while state["t"] % wl.window:
        step()
    n_w = max(K, 4 * wl.window) // wl.window * wl.window
    ms_w = timed(n_w, interval=wl.window)  # one routing event per filled window
    for g in groups:
        g[0].close()
    ms = statistics.median(reps)
    peak, _ = peak_hbm_gbs()
    gbs = kbytes / (ms / K * 1e-3) / 1e9
    gbs_w = kbytes / (ms_w / n_w * 1e-3) / 1e9
    return {"caches": 2, "layers_per_cache": half.n_layers, "streams": 2, "steps": K, "repeats": len(reps),
            "ms_per_step": ms / K, "value": K / (ms * 1e-3), "unit": UNIT, "step_frac": gbs / peak, "step_frac_of_8TBs": gbs / 8000.0,
            "rebalance_every_window": {"rebalance_interval": wl.window, "steps": n_w, "ms_per_step": ms_w / n_w,
                                       "value": n_w / (ms_w * 1e-3), "step_frac": gbs_w / peak, "step_frac_of_8TBs": gbs_w / 8000.0},
            "what": "two caches of half the layers each on two streams, a routing event after every step: one cache's table "
                    "kernels run under the other's attention kernel"}


def run_ours(args, rank, world):
    if args.timeline:
        os.environ["QEVICT_TRACE_LIB"] = "1"  # read when the binding is first imported
    from paper_2608_05326_b200 import build
    if rank == 0:
        build.build(trace=args.timeline)  # no-op when the in-tree library is newer than its sources
    if world > 1:
        torch.distributed.barrier()
    local = int(os.environ.get("LOCAL_RANK", 0))
    if os.environ.get("QEVICT_BENCH_SHARE_GPU"):  # test aid: several ranks on one device (the ranks never wait on one another on the GPU)
        local %= torch.cuda.device_count()
    dev = torch.device("cuda", local)
    torch.cuda.set_device(dev)
    K, W = args.steps, args.warmup
    wl = sharding.rank_workload(make_workload(args, K), rank)  # every rank owns its own sequences (weak scaling, no exchange)
    res = measure_workload(args, wl, rank, world, dev, K, W, with_e2e=not args.no_e2e, timeline=args.timeline)
    if args.timeline:
        return res, wl
    # the default run also carries the second target configuration (128k context, 8 layers in one launch)
    also = None
    default_run = (args.config == 1 and args.layers is None and args.batch is None and args.rope_base == 0.0 and
                   not args.fixed_context and args.rank_mode == 0 and not args.sink_windows and not args.recent_windows and
                   not args.no_also)
    if default_run:
        wl3 = sharding.rank_workload(replace(workloads.config(3), n_layers=8, rebalance_interval=args.rebalance_interval), rank)
        also = measure_workload(args, wl3, rank, world, dev, K, W, with_e2e=False)
    two = None
    if default_run and world == 1 and args.rebalance_interval == 1:
        two = measure_two_streams(args, wl, dev, K, W, res["kbytes"])
    if rank != 0:
        return None
    wl, ms, R = res["wl"], res["ms"], args.rebalance_interval
    line = {
        "metric": METRIC, "value": sharding.aggregate_steps_per_second(world, K, ms), "unit": UNIT, "n_gpus": world, "steps": K, "warmup": W,
        "ms_per_step": ms / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": wl.dtype,
        "data": "synthetic",
        "repeats": res["repeats"], "ms_per_step_min": res["rep_ms"][0] / K, "ms_per_step_max": res["rep_ms"][-1] / K,
        "ms_per_step_by_repeat": [round(x / K, 5) for x in res["rep_order"]],
        "config": {
            "workload": res["workload"],
            "units_per_step": wl.n_units, "context": wl.context, "window": wl.window, "quant_bits": wl.quant_bits,
            "group_size": wl.group_size, "fp_budget_windows": wl.fp_budget_windows,
            "q_budget_windows": wl.q_budget_windows, "sink_windows": wl.sink_windows, "recent_windows": wl.recent_windows,
            "rebalance_interval": R, "append": not args.fixed_context, "rope_base": wl.rope_base,
            "l2": "inputs larger than L2 (KV working set %.0f MB per step)" % (res["kbytes"] / 1e6),
            "settle_steps": args.settle_steps, "idle_after_settle_s": IDLE_AFTER_SETTLE_S, "input_pool_steps": min(INPUT_POOL, wl.steps),
            "timing": "median of %d repeats of the %d-step loop (a loop shorter than %.1f s is repeated)" % (res["repeats"], K, MIN_TIMED_SECONDS),
        },
        "layer_steps_per_sec": world * K * wl.n_units / (ms * 1e-3),
        "clocks": res["clocks"],
        "gpu_launches": res["launches"],
        "roofline": res["roofline"],
        "host_enqueue_us_per_step": res["host_enqueue_us_per_step"],
        "kernel_us_per_step": res["kernel_us_per_step"],
        "tier_state": {k: res["stats"][k] for k in ("n_full", "n_quant", "n_aged", "n_sink", "n_open", "n_evicted", "promotions",
                                                     "quantizations", "reactivations", "deletions")},
    }
    if "interval_w" in res:
        line["rebalance_every_window"] = res["interval_w"]
    if res["e2e"]:
        e2e = res["e2e"]
        line["e2e"] = {"value": world * K / e2e["seconds"], "unit": UNIT, "h2d_bytes_per_step": e2e["h2d_bytes_per_step"],
                       "d2h_bytes_per_step": e2e["d2h_bytes_per_step"]}
    if two:
        line["two_streams"] = two
    if also:
        line["also"] = {"workload": also["workload"], "value": sharding.aggregate_steps_per_second(world, K, also["ms"]),
                        "unit": UNIT, "ms_per_step": also["ms"] / K, "repeats": also["repeats"], "roofline": also["roofline"],
                        "kernel_us_per_step": also["kernel_us_per_step"], "gpu_launches": also["launches"],
                        "clocks": also["clocks"]}
        if "interval_w" in also:
            line["also"]["rebalance_every_window"] = also["interval_w"]
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
    """Size of the BLAS thread pool the oracle's matrix products may use (its element-wise numpy code is single-threaded)."""
    try:
        from threadpoolctl import threadpool_info
        n = [p.get("num_threads", 1) for p in threadpool_info()]
        return max(n) if n else 1
    except Exception:
        return 1


def _cpu_seconds():
    t = os.times()
    return t.user + t.system


def time_oracle(wl, n_steps, warmup, budget_s, one_thread_s=0.0):
    """Times the CPU oracle, as it stands, on unit 0 of the workload: `n_steps` decode + rebalance steps
    (at most `budget_s` seconds).  Returns (whole-workload steps/s, description, steps, seconds, cores kept busy,
    whole-workload steps/s with the BLAS pool limited to one thread over a further `one_thread_s` seconds or None)."""
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
    c0 = _cpu_seconds()
    t0 = time.perf_counter()
    while done < n_steps and t < q.shape[0] and time.perf_counter() - t0 < budget_s:
        orc.decode_attn(q[t], kn[t], vn[t])
        if (t + 1) % wl.rebalance_interval == 0:
            orc.rebalance()
        t += 1; done += 1
    dt = time.perf_counter() - t0
    busy = (_cpu_seconds() - c0) / dt if dt > 0 else 1.0   # cores kept busy on average (process CPU time / wall time)
    unit_steps_per_s = done / dt
    value = unit_steps_per_s / wl.n_units
    sample = "unit 0 of %d, %d decode+rebalance steps in %.1f s" % (wl.n_units, done, dt)
    one = None
    if one_thread_s > 0:
        try:
            from threadpoolctl import threadpool_limits
            with threadpool_limits(limits=1):
                n1, t1 = 0, time.perf_counter()
                while t < q.shape[0] and time.perf_counter() - t1 < one_thread_s:
                    orc.decode_attn(q[t], kn[t], vn[t])
                    if (t + 1) % wl.rebalance_interval == 0:
                        orc.rebalance()
                    t += 1; n1 += 1
                if n1:
                    one = n1 / (time.perf_counter() - t1) / wl.n_units
        except Exception:
            one = None
    return value, sample, done, dt, busy, one


def cpu_baseline_record(value, sample, busy, one_thread=None):
    rec = {"value": value, "unit": UNIT, "cores": max(1, round(busy)), "kind": "oracle", "sample": sample,
           "cores_busy_avg": round(busy, 2), "blas_threads": oracle_threads(), "host_cores": os.cpu_count()}
    if one_thread is not None:
        rec["value_one_thread"] = one_thread  # the same oracle with the BLAS pool limited to one thread
    return rec


def run_reference(args, rank):
    if rank != 0:
        return None
    K, W = args.steps, args.warmup
    wl = make_workload(args, max(W + K, 8))
    value, sample, done, dt, busy, _ = time_oracle(wl, K, W, budget_s=180.0)
    return {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": done,
        "warmup": W, "ms_per_step": 1e3 / value, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64", "data": "synthetic",
        "config": {"workload": "%s x %d layers x batch %d" % (wl.name, wl.n_layers, wl.batch), "sample": sample},
        "cpu_baseline": cpu_baseline_record(value, sample, busy),
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


def spawn_ranks(args):
    """`python bench.py --gpus N` outside a launcher: start N ranks of this script, one per GPU, under
    torch.distributed.run (rank 0 prints the one JSON line).  Returns the launcher's exit code."""
    import socket
    if args.impl == "ours":
        have = torch.cuda.device_count() if torch.cuda.is_available() else 0
        if have < args.gpus:
            sys.stderr.write("bench.py: --gpus %d asked for, %d CUDA device(s) visible; not running fewer ranks than asked\n" % (args.gpus, have))
            return 2
    with socket.socket() as sock:
        sock.bind(("127.0.0.1", 0))
        port = sock.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", str(args.gpus),
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.call(cmd)


def main():
    args = parse_args()
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        sys.exit(spawn_ranks(args))
    rank = int(os.environ.get("RANK", 0))
    world = int(os.environ.get("WORLD_SIZE", 1))
    if world != max(args.gpus, 1):
        sys.stderr.write("bench.py: --gpus %d does not match the launcher's WORLD_SIZE %d\n" % (args.gpus, world))
        sys.exit(2)
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
        os.environ.setdefault("NCCL_DEBUG", "WARN")
        # NCCL is used for the barrier and the max over ranks only; QEVICT_BENCH_BACKEND=gloo lets a test run two
        # ranks on one device (NCCL refuses two ranks per GPU)
        torch.distributed.init_process_group(os.environ.get("QEVICT_BENCH_BACKEND", "nccl"))
    res = run_ours(args, rank, world)
    if rank == 0:
        line, wl = res
        if not args.timeline and not args.no_cpu_baseline and world >= 1:
            small = replace(wl, steps=256, seed=wl.seed)
            value, sample, _, _, busy, one = time_oracle(small, 1000, 1, budget_s=args.cpu_seconds * 2 / 3,
                                                         one_thread_s=args.cpu_seconds / 3)
            line["cpu_baseline"] = cpu_baseline_record(value, sample, busy, one)
        print(json.dumps(line))
    if world > 1:
        torch.distributed.destroy_process_group()


if __name__ == "__main__":
    main()
