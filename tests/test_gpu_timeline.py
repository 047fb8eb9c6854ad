"""The tracing build of the library: same kernels with device-timer stamps.  The normal library refuses the
timeline call; the tracing one returns the launches of the pipelined step in order, each kernel's body starting
only after the one before it has ended (programmatic dependent launch), and still matches the oracle."""

import json
import os
import subprocess
import sys

import pytest
import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
pytestmark = pytest.mark.gpu


def test_normal_build_refuses_the_timeline():
    from paper_2608_05326_b200 import binding, workloads

    wl = workloads.config(0)
    cfg = binding.make_config(wl.batch, wl.n_layers, wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.dtype, wl.window,
                              wl.quant_bits, wl.group_size, wl.fp_budget_windows, wl.q_budget_windows, wl.max_context)
    cache = binding.QEvictCache(cfg)
    with pytest.raises(binding.QEvictError) as err:
        cache.kernel_timeline()
    assert err.value.status == binding.STATUS_NAMES.index("UNSUPPORTED")
    cache.close()


def _run(code_or_args, env_extra):
    env = dict(os.environ, **env_extra)
    r = subprocess.run([sys.executable] + code_or_args, cwd=ROOT, env=env, capture_output=True, text=True, timeout=600)
    assert r.returncode == 0, r.stdout[-2000:] + r.stderr[-4000:]
    return r.stdout


def test_tracing_build_orders_the_kernels_of_a_step():
    out = _run(["bench.py", "--timeline", "--config", "0", "--steps", "12", "--warmup", "3"], {})
    line = json.loads(out.strip().splitlines()[-1])
    assert line["metric"] == "kernel_timeline" and line["launches"] >= 5 * 12
    names = [n for n, _, _ in line["last_step"]]
    assert names == ["append", "decode_attn", "combine", "route", "migrate"]
    prev_end = None
    for _, t0, t1 in line["last_step"]:
        assert t1 >= t0
        if prev_end is not None:
            assert t0 >= prev_end - 1.5, "a kernel body started before the one before it ended"
        prev_end = t1
    for name in names:
        assert 0.0 <= line["median_us"][name] < 5000.0


def test_tracing_build_matches_the_oracle():
    code = (
        "import sys; sys.path.insert(0, 'tests')\n"
        "from dataclasses import replace\n"
        "import lockstep\n"
        "from paper_2608_05326_b200 import binding, workloads\n"
        "assert binding.LIB_PATH.endswith('libqevict_trace.so')\n"
        "run = lockstep.LockstepRun(replace(workloads.config(0), steps=10))\n"
        "for _ in range(10):\n"
        "    run.step(append=True)\n"
        "run.rebalance(full_check=True)\n"
        "assert len(run.cache.kernel_timeline()) > 0\n"
        "run.close()\n"
    )
    from paper_2608_05326_b200 import build

    build.build(trace=True)
    _run(["-c", code], {"QEVICT_TRACE_LIB": "1"})
