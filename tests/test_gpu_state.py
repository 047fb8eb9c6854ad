"""GPU tests of the boundary around the hot path: snapshot / restore of a cache, calls for single layers mixed
with calls for all layers on one handle, several caches of different shape in one process, and the refusal of
shapes the kernels cannot run."""

import pytest
import torch

from paper_2608_05326_b200 import binding, workloads

pytestmark = pytest.mark.gpu


def _lockstep():
    import lockstep  # tests/ is on sys.path (conftest)
    return lockstep


def _wl(name, **kw):
    base = dict(name=name, batch=2, n_layers=2, n_q_heads=8, n_kv_heads=2, head_dim=128, dtype="bf16", context=1536,
                window=32, quant_bits=4, group_size=32, fp_budget_windows=5, q_budget_windows=9, steps=48,
                rebalance_interval=1)
    base.update(kw)
    return workloads.Workload(**base)


@pytest.mark.parametrize("kw", [dict(), dict(quant_bits=2, window=64, group_size=64, rebalance_interval=3, dtype="fp16", head_dim=64),
                                dict(rank_mode=1, rank_param=0.9, sink_windows=1, recent_windows=2)],
                         ids=["bf16-4bit", "fp16-2bit-w64-R3", "decayed-sink-recent"])
def test_snapshot_restore_continues_bit_for_bit(kw):
    """export -> destroy -> create -> import, then 20 more lockstep steps: the restored cache must agree with the
    oracle (which never stopped) step by step, and with an uninterrupted GPU run bit for bit."""
    ls = _lockstep()
    wl = _wl("snapshot", **kw)
    run = ls.LockstepRun(wl, score_mode="synthetic")                   # interrupted at step 20
    twin = ls.LockstepRun(wl, oracle_units=[], score_mode="synthetic")  # never interrupted
    for _ in range(20):
        run.step(append=True)
        twin.step(append=True, check_mass=False)
    states = {u: run.cache.export_state(u // wl.batch, u % wl.batch) for u in range(wl.n_units)}
    before = run.cache.stats()
    run.cache.close()
    run.cache = binding.QEvictCache(ls.gpu_config(wl, rebalance_interval=run.R))
    for u, st in states.items():
        run.cache.import_state(u // wl.batch, u % wl.batch, st)
    after = run.cache.stats()
    for key in ("promotions", "quantizations", "reactivations", "deletions", "n_full", "n_quant", "n_aged", "n_open",
                "n_evicted", "n_sink", "decode_steps"):
        assert before[key] == after[key], key
    run.check_state("all", "after import")
    for _ in range(20):
        a = run.step(append=True)
        b = twin.step(append=True, check_mass=False)
        assert torch.equal(a, b)
    run.rebalance(full_check=True)
    twin.cache.rebalance(-1)
    for u in range(wl.n_units):
        x = run.cache.export_state(u // wl.batch, u % wl.batch)
        y = twin.cache.export_state(u // wl.batch, u % wl.batch)
        for key in ("tier", "ledger", "fp_page", "q_page", "importance", "event_mass", "fp_owner", "q_owner"):
            assert torch.equal(x[key], y[key]), (u, key)
        n = x["n_live"]
        assert n == y["n_live"] and torch.equal(x["entries"][:n], y["entries"][:n])
        # pages that a window holds must be the same bytes (free pages are whatever the buffer held before)
        for pool, owner in (("q_pool", "q_owner"), ("fp_pool", "fp_owner")):
            px, py = x[pool].reshape(len(x[owner]), -1), y[pool].reshape(len(y[owner]), -1)
            held = x[owner] >= 0
            if x["open_window"] >= 0:  # the open window's unfilled slots are not part of the state
                held &= x[owner] != x["open_window"]
            assert torch.equal(px[held], py[held]), (u, pool)
    run.close()
    twin.close()


def test_import_refuses_a_snapshot_that_does_not_fit():
    ls = _lockstep()
    wl = _wl("snapshot-bad", n_layers=1, steps=4)
    run = ls.LockstepRun(wl, oracle_units=[])
    run.step(append=True)
    st = run.cache.export_state(0, 0)
    other = binding.QEvictCache(ls.gpu_config(wl))
    bad = dict(st)
    bad["fp_page"] = st["fp_page"].clone()
    bad["fp_page"][3] = 10_000  # no such page
    with pytest.raises(binding.QEvictError) as e:
        other.import_state(0, 0, bad)
    assert e.value.status == 1 and "out of range" in str(e.value)
    bad = dict(st)
    bad["entries"] = st["entries"].clone()
    bad["entries"][0, 0] = (3 << 28) | 1  # no such entry kind
    with pytest.raises(binding.QEvictError):
        other.import_state(0, 0, bad)
    other.import_state(0, 0, st)  # the good one still goes in
    moved = dict(st)
    moved["open_fill"] = st["open_fill"] + 1
    moved["layer_open_fill"] = st["layer_open_fill"] + 1
    with pytest.raises(binding.QEvictError) as e:  # sequence 1 must stand where sequence 0 stands
        other.import_state(0, 1, moved)
    assert e.value.status == 2
    other.close()
    run.close()


def test_single_layer_and_all_layer_calls_mixed_on_one_handle():
    """Decode steps and routing events of one cache issued sometimes for all layers at once and sometimes layer by
    layer (the migration queue's alternating counters are kept per first layer of a call): every step is checked
    against the oracle."""
    ls = _lockstep()
    wl = _wl("mixed", batch=2, n_layers=3, steps=36, fp_budget_windows=4, q_budget_windows=7)
    run = ls.LockstepRun(wl)
    pattern = [False, True, True, False, True, False, False, True]
    for t in range(wl.steps):
        run.step(append=True, per_layer=pattern[t % len(pattern)])
    run.rebalance(full_check=True, per_layer=True)
    run.rebalance(full_check=True)
    st = run.cache.stats()
    assert st["decode_steps"] > 0 and st["promotions"] + st["quantizations"] > 0
    run.close()


def test_caches_of_different_shape_share_the_process():
    """A cache with large routing tables, then one with smaller ones (still beyond the default shared-memory
    limit), then routing events on the first: the kernels' shared-memory limit must not have been lowered."""
    ls = _lockstep()
    wl = _wl("tables", batch=1, n_layers=1, context=2048, steps=6)
    dev = torch.device("cuda")

    def make(max_context):
        cfg = binding.make_config(wl.batch, 1, wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.dtype, wl.window, wl.quant_bits,
                                  wl.group_size, wl.fp_budget_windows, wl.q_budget_windows, max_context,
                                  rebalance_interval_hint=1)
        cache = binding.QEvictCache(cfg)
        k, v = workloads.gen_prompt_kv(wl, 0)
        s = workloads.place_planted(workloads.synthetic_window_scores(wl, 0), workloads.planted_windows(wl, 0),
                                    wl.fp_budget_windows, wl.q_budget_windows)
        cache.prefill_assign(0, k[None].to(dev), v[None].to(dev), s[None].to(dev))
        return cache, k, s

    big, k, s = make(32 * 6000)     # routing tables of 8192 candidate slots: far beyond 48 KB
    small, _, _ = make(32 * 1800)   # 2048 slots: still beyond 48 KB, but less than the first cache asked for
    q = workloads.gen_queries(wl, 0, k, s)
    kn, vn = workloads.gen_new_kv(wl, 0)
    outs = []
    for cache in (big, small, big):
        o = cache.decode_attn(0, q[0][None].to(dev), kn[0][None].to(dev), vn[0][None].to(dev))
        cache.rebalance(0)
        torch.cuda.synchronize()
        outs.append(o.cpu())
        st = cache.stats()  # reports a failed launch or device check
        assert st["n_full"] == wl.fp_budget_windows
    assert torch.equal(outs[0], outs[1])  # same prompt, same query: the table size changes nothing
    big.close()
    small.close()


def test_device_is_left_as_the_caller_had_it():
    if torch.cuda.device_count() < 2:
        pytest.skip("needs two devices to observe a change of the current device")
    ls = _lockstep()
    wl = _wl("device", n_layers=1, steps=2)
    run = ls.LockstepRun(wl, oracle_units=[])
    torch.cuda.set_device(1)
    try:
        run.cache.stats()
        assert torch.cuda.current_device() == 1
    finally:
        torch.cuda.set_device(0)
    run.close()


def test_bench_under_a_launcher_with_two_ranks():
    """The N > 1 path of bench.py for real: two ranks under torch.distributed.run, each with its own sequences; both
    on this one device and over gloo (NCCL refuses two ranks per GPU; the ranks exchange nothing but a barrier and a
    max of their times, and never wait on one another on the GPU).  Rank 0 prints one line for two ranks."""
    import json
    import os
    import socket
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK")}
    env.update(QEVICT_BENCH_BACKEND="gloo", QEVICT_BENCH_SHARE_GPU="1")
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2", "--master-addr", "127.0.0.1",
           "--master-port", str(port), os.path.join(root, "bench.py"), "--gpus", "2", "--config", "0", "--steps", "8",
           "--warmup", "3", "--settle-steps", "8", "--no-cpu-baseline"]
    r = subprocess.run(cmd, capture_output=True, text=True, env=env, timeout=900)
    assert r.returncode == 0, r.stderr[-3000:]
    lines = [ln for ln in r.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1, r.stdout[-2000:]
    line = json.loads(lines[0])
    assert line["n_gpus"] == 2 and line["scaling"] == "weak" and line["value"] > 0 and line["gpu_launches"] > 0
    assert line["e2e"]["value"] > 0 and line["roofline"]["kernel_launches_timed"] == 8


def test_two_caches_on_two_streams_give_the_same_bits_as_one_after_the_other():
    """Independent caches stepped on different streams (so that one cache's table kernels run under the other's
    attention kernel) must not disturb each other: same outputs, same tables as the same caches stepped one after
    the other on one stream."""
    ls = _lockstep()
    wl_a = _wl("streams-a", n_layers=2, steps=24)
    wl_b = _wl("streams-b", n_layers=2, steps=24, quant_bits=2, fp_budget_windows=3, q_budget_windows=11)
    serial = [ls.LockstepRun(w, oracle_units=[], score_mode="synthetic") for w in (wl_a, wl_b)]
    overlapped = [ls.LockstepRun(w, oracle_units=[], score_mode="synthetic") for w in (wl_a, wl_b)]
    streams = [torch.cuda.Stream(), torch.cuda.Stream()]
    dev = serial[0].dev
    torch.cuda.synchronize()
    for t in range(24):
        outs_serial = [r.step(append=True, check_mass=False) for r in serial]
        outs = []
        for r, s in zip(overlapped, streams):
            wl = r.wl
            q = torch.stack([r.queries[u][t] for u in range(wl.n_units)]).reshape(wl.n_layers, wl.batch, wl.n_q_heads, wl.head_dim).to(dev)
            kn = torch.stack([r.new_kv[u][0][t] for u in range(wl.n_units)]).reshape(wl.n_layers, wl.batch, wl.n_kv_heads, wl.head_dim).to(dev)
            vn = torch.stack([r.new_kv[u][1][t] for u in range(wl.n_units)]).reshape(wl.n_layers, wl.batch, wl.n_kv_heads, wl.head_dim).to(dev)
            torch.cuda.current_stream().synchronize()  # the inputs were produced on the current stream
            with torch.cuda.stream(s):
                out = torch.empty_like(q)
            r.cache.decode_attn(-1, q, kn, vn, out, stream=s)
            r.cache.rebalance(-1, stream=s)
            outs.append((out, q, kn, vn))
        torch.cuda.synchronize()
        for (out, *_), ref, r in zip(outs, outs_serial, overlapped):
            assert torch.equal(out.cpu().reshape(r.wl.n_units, r.wl.n_q_heads, r.wl.head_dim), ref), t
    for a, b in zip(serial, overlapped):
        for u in range(a.wl.n_units):
            x = a.cache.export_tables(u // a.wl.batch, u % a.wl.batch)
            y = b.cache.export_tables(u // b.wl.batch, u % b.wl.batch)
            for key in x:
                assert torch.equal(x[key], y[key]), (u, key)
        a.close(); b.close()
