"""Parity at the benchmark's full sizes, in the launch configuration bench.py times: the whole workload
runs on the GPU, the oracle follows a sample of its units step by step (outputs, per-window mass, tiers,
page tables, codes), and properties that hold at any size are checked on every unit."""

from dataclasses import replace

import numpy as np
import pytest
import torch

from paper_2608_05326_b200 import workloads

pytestmark = pytest.mark.gpu


def _run(wl, oracle_units, steps, rebalance_interval=1, check_all_units_mass=True):
    import lockstep
    wl = replace(wl, steps=steps)
    run = lockstep.LockstepRun(wl, oracle_units=oracle_units, score_mode="synthetic",
                               rebalance_interval=rebalance_interval, gen_device="cuda")
    run.check_state({u: list(range(0, wl.n_prompt_windows, max(1, wl.n_prompt_windows // 40))) for u in oracle_units},
                    "after prefill")
    for t in range(steps):
        run.step(append=True)
        if check_all_units_mass and t % 4 == 0:
            for u in range(wl.n_units):
                m = run.cache.export_last_mass(u // wl.batch, u % wl.batch).double().sum().item()
                assert abs(m - wl.n_q_heads) < 1e-4 * wl.n_q_heads, (u, m)
    run.rebalance(full_check=True)  # every live page, code and table of the followed units
    st = run.cache.stats()
    assert st["n_full"] <= wl.n_units * wl.fp_budget_windows and st["n_quant"] <= wl.n_units * wl.q_budget_windows
    for u in oracle_units:
        o = run.oracles[u]
        tab = run.cache.export_tables(u // wl.batch, u % wl.batch)
        assert np.array_equal(tab["tier"].numpy()[: o.n_windows], o.tier[: o.n_windows])
    run.close()
    return st


def test_config1_llama_32k_x32_layers_sampled_units():
    wl = workloads.config(1, n_layers=32)
    st = _run(wl, oracle_units=[0, 13, 31], steps=40)
    assert st["n_full"] == 32 * 64 and st["n_quant"] == 32 * 128


def test_config2_stacked_2bit_sampled_units():
    # 16 sequences x 8 of the 32 layers = 128 of the 512 units (the per-unit work and the split count are those
    # of the full configuration -- the launch fills the GPU several times over either way; 8 layers keep the
    # prompts of the test within a few GB and its run time short), 2-bit codes, rebalance every step
    wl = workloads.config(2, n_layers=8)
    _run(wl, oracle_units=[5, 37, 63, 127], steps=36)


def test_config3_long_context_window64_sampled_unit():
    wl = workloads.config(3)
    _run(wl, oracle_units=[2], steps=70, check_all_units_mass=True)


def test_config3_x8_layers_sampled_units():
    # the launch configuration the 128k roofline figure is quoted on: 8 layers x 4 sequences in one launch
    wl = workloads.config(3, n_layers=8)
    _run(wl, oracle_units=[3, 30], steps=40)


def test_config3_long_context_pre_rope_keys_sampled_unit():
    # the 128k configuration with the keys stored pre-RoPE: positions up to 131 072 go through the rotation table
    wl = replace(workloads.config(3), rope_base=500000.0)
    _run(wl, oracle_units=[1], steps=24, check_all_units_mass=True)


def test_config1_x32_layers_pre_rope_keys_sampled_unit():
    wl = replace(workloads.config(1, n_layers=32), rope_base=500000.0)
    _run(wl, oracle_units=[7], steps=34)


@pytest.mark.parametrize("bits,fp_frac", [(4, 0.05), (4, 0.10), (4, 0.20), (2, 0.05), (2, 0.10), (2, 0.20)])
def test_config4_qwen_gqa7_sampled_unit(bits, fp_frac):
    wl = workloads.config(4, bits=bits, fp_frac=fp_frac)
    _run(wl, oracle_units=[3], steps=34, rebalance_interval=2)


def test_config1_all_256_steps_two_units():
    # the whole run of the configuration (256 decode steps, routing event after every step), two units followed
    # step by step, every page, code and table compared at the end
    import lockstep
    wl = replace(workloads.config(1, n_layers=32), steps=256)
    run = lockstep.LockstepRun(wl, oracle_units=[0, 17], score_mode="synthetic", rebalance_interval=1, gen_device="cuda")
    for _ in range(256):
        run.step(append=True)
    run.rebalance(full_check=True)
    st = run.cache.stats()
    assert st["decode_steps"] == 256 and st["n_full"] == 32 * 64 and st["n_quant"] == 32 * 128
    for u, o in run.oracles.items():
        assert o.stats["promotions"] > 50 and o.stats["deletions"] > 832
    run.close()
