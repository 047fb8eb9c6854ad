"""The checking build of the library (-DQEVICT_DEBUG_BOUNDS): the same kernels with every page id, window index,
work-list entry and migration record range-checked before it is used, and both pools poisoned with NaN at
creation.  It stands in for a memory checker.  Two things are shown: the parity suite passes on it unchanged
(no check fires on good tables, no result depends on a page nobody wrote), and a table entry that is out of range
is refused by the kernel -- recorded, skipped, the context still usable.  The library is chosen when the binding
is imported, so each part runs in a process of its own."""

import os
import subprocess
import sys
import textwrap

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _run(code, extra_env=None, timeout=1500):
    env = dict(os.environ, QEVICT_CHECK_LIB="1", PYTHONPATH=os.pathsep.join([ROOT, os.path.join(ROOT, "tests")]))
    env.update(extra_env or {})
    return subprocess.run([sys.executable, "-c", textwrap.dedent(code)], capture_output=True, text=True, env=env,
                          cwd=ROOT, timeout=timeout)


def test_parity_suite_passes_on_the_checking_build():
    r = _run("""
        import sys, pytest
        from paper_2608_05326_b200 import binding, build
        build.build(variant="check")
        assert binding.lib().qevict_build_flavour() == 2
        sys.exit(pytest.main(["tests/test_gpu_parity.py", "-m", "gpu", "-x", "-q", "-p", "no:cacheprovider", "-k",
                              "config0 or shapes_lockstep or random_configurations or protected_sink or multiple_units"]))
    """)
    tail = r.stdout[-1500:] + r.stderr[-1500:]
    assert r.returncode == 0, tail
    assert " passed" in r.stdout and "failed" not in r.stdout, tail


_FIRE = """
    import torch
    from paper_2608_05326_b200 import binding, build, workloads
    build.build(variant="check")
    assert binding.lib().qevict_build_flavour() == 2
    dev = torch.device("cuda")
    # two sequences: an index one past the end of sequence 0's tables still points into the cache's own buffer
    wl = workloads.Workload(name="fire", batch=2, n_layers=1, n_q_heads=8, n_kv_heads=2, head_dim=128, dtype="bf16",
                            context=1024, window=32, quant_bits=4, group_size=32, fp_budget_windows=4, q_budget_windows=8,
                            steps=8, rebalance_interval=1)

    def fresh():
        cfg = binding.make_config(wl.batch, 1, wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.dtype, wl.window, wl.quant_bits,
                                  wl.group_size, wl.fp_budget_windows, wl.q_budget_windows, wl.max_context, rebalance_interval_hint=1)
        cache = binding.QEvictCache(cfg)
        ks, vs, ss = [], [], []
        for u in range(2):
            k, v = workloads.gen_prompt_kv(wl, u)
            ks.append(k); vs.append(v)
            ss.append(workloads.place_planted(workloads.synthetic_window_scores(wl, u), workloads.planted_windows(wl, u), 4, 8))
        cache.prefill_assign(0, torch.stack(ks).to(dev), torch.stack(vs).to(dev), torch.stack(ss).to(dev))
        q = torch.stack([workloads.gen_queries(wl, u, ks[u], ss[u]) for u in range(2)], 1).to(dev)
        kn = torch.stack([workloads.gen_new_kv(wl, u)[0] for u in range(2)], 1).to(dev)
        vn = torch.stack([workloads.gen_new_kv(wl, u)[1] for u in range(2)], 1).to(dev)
        cache.decode_attn(0, q[0], kn[0], vn[0])
        cache.rebalance(0)
        assert cache.stats()["n_full"] == 8 and cache.check_device() == 0  # no check has fired on good tables
        return cache, q, kn, vn

    def expect_check(cache, code):
        try:
            cache.check_device()
            cache.stats()
        except binding.QEvictError as e:
            assert e.status == 6 and ("check %d " % code) in str(e), str(e)
            return
        raise AssertionError("no device check was reported")

    lay = None
    # (a) a work-list entry whose page is one past the pool: the attention kernel ends that warp's run before it
    cache, q, kn, vn = fresh()
    lay = binding.qevict_state_layout_of(cache.handle)
    st = cache.export_state(0, 0)
    st["entries"][0, 1] = lay.n_fp_pages if (int(st["entries"][0, 0]) >> 28) != 1 else lay.n_q_pages
    cache.import_state(0, 0, st)
    out = cache.decode_attn(0, q[1], kn[1], vn[1])
    torch.cuda.synchronize()
    expect_check(cache, 6)
    assert torch.isfinite(out[1].float()).all()  # the other sequence is untouched
    cache.close()
    # (b) the open window's page id one past the pool: the append kernel refuses to write the token
    cache, q, kn, vn = fresh()
    st = cache.export_state(0, 0)
    st["fp_page"][st["open_window"]] = lay.n_fp_pages
    cache.import_state(0, 0, st)
    cache.decode_attn(0, q[1], kn[1], vn[1])
    torch.cuda.synchronize()
    expect_check(cache, 7)
    cache.close()
    # (c) a Quantized window's page id one past the pool: the routing kernel drops it when it gathers the tables
    cache, q, kn, vn = fresh()
    st = cache.export_state(0, 0)
    w = int((st["tier"] == 4).nonzero()[0])
    st["q_page"][w] = lay.n_q_pages
    cache.import_state(0, 0, st)
    cache.rebalance(0)
    torch.cuda.synchronize()
    expect_check(cache, 7)
    cache.close()
    # the context is still usable after all three
    cache, q, kn, vn = fresh()
    cache.close()
    print("checks fired")
"""


def test_out_of_range_table_entries_are_recorded_and_skipped():
    r = _run(_FIRE, {"QEVICT_IMPORT_UNCHECKED": "1"})
    assert r.returncode == 0 and "checks fired" in r.stdout, r.stdout[-1500:] + r.stderr[-3000:]
