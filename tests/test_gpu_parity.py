"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle on the same seeded
inputs.  Integer results (codes, tiers, page tables, ledger flags) and everything derived exactly
from them (parameters, promoted page contents) are compared bit for bit; attention outputs within
max-abs 2e-3 + 1e-2 relative; window mass and scores within 1e-4 relative."""

from dataclasses import replace

import numpy as np
import pytest
import torch

from paper_2608_05326_b200 import binding, workloads

pytestmark = pytest.mark.gpu


def _lockstep():
    import lockstep  # tests/ is on sys.path (conftest)
    return lockstep


def _small(name, **kw):
    base = dict(name=name, batch=1, n_layers=1, n_q_heads=4, n_kv_heads=2, head_dim=64, dtype="fp16", context=1024,
                window=32, quant_bits=4, group_size=32, fp_budget_windows=4, q_budget_windows=8, steps=40,
                rebalance_interval=1)
    base.update(kw)
    return workloads.Workload(**base)


def test_config0_append_rebalance_every_step():
    ls = _lockstep()
    run = ls.LockstepRun(workloads.config(0))
    run.check_state("all", "after prefill")
    st = run.cache.stats()
    assert (st["n_full"], st["n_quant"], st["n_evicted"]) == (8, 16, 40)
    for _ in range(run.wl.steps):
        run.step(append=True)
    run.check_state("all", "end")
    st = run.cache.stats()
    o = run.oracles[0].stats
    assert st["promotions"] == o["promotions"] > 0
    assert st["quantizations"] == o["quantizations"] and st["reactivations"] == o["reactivations"]
    assert st["deletions"] == o["deletions"]
    run.close()


def test_config0_fixed_context_rebalance_every_window():
    ls = _lockstep()
    run = ls.LockstepRun(workloads.config(0), rebalance_interval=32)
    for _ in range(run.wl.steps):
        run.step(append=False)
    run.check_state("all", "end")
    assert run.cache.stats()["n_evicted"] == 40  # with a fixed context nothing is deleted after prefill
    run.close()


@pytest.mark.parametrize("kw", [
    dict(dtype="bf16", head_dim=128, n_q_heads=8, n_kv_heads=2),
    dict(dtype="bf16", head_dim=128, n_q_heads=8, n_kv_heads=2, quant_bits=2),
    dict(dtype="fp16", head_dim=64, quant_bits=2),
    dict(dtype="bf16", head_dim=64, n_q_heads=7, n_kv_heads=1),
    dict(dtype="bf16", head_dim=128, n_q_heads=8, n_kv_heads=1, window=64, group_size=64, context=2048),
    dict(dtype="bf16", head_dim=128, n_q_heads=4, n_kv_heads=2, window=64, group_size=32, context=2048, quant_bits=2),
    dict(dtype="fp16", head_dim=128, n_q_heads=2, n_kv_heads=2, window=64, group_size=64, context=2048, quant_bits=2),
    dict(dtype="fp16", head_dim=64, n_q_heads=3, n_kv_heads=1, window=64, group_size=32, context=2048),
    dict(dtype="bf16", head_dim=128, n_q_heads=8, n_kv_heads=2, outlier_channels=4, outlier_scale=8.0),
], ids=lambda kw: "-".join("%s%s" % (k[0], v) for k, v in kw.items()))
def test_shapes_lockstep(kw):
    ls = _lockstep()
    wl = _small("small", steps=2 * kw.get("window", 32) + 6, **kw)
    run = ls.LockstepRun(wl, rebalance_interval=3)
    run.check_state("all", "after prefill")
    for _ in range(wl.steps):
        run.step(append=True)
    run.rebalance(full_check=True)
    run.close()


@pytest.mark.parametrize("cfg", ["c0", "small-bf16"])
def test_free_running_routes_identically_or_flips_only_at_a_cut(cfg):
    # no score overwrite: the GPU routes on its float32 scores, the oracle on its float64 ones
    ls = _lockstep()
    wl = workloads.config(0) if cfg == "c0" else _small("free", dtype="bf16", head_dim=128, n_q_heads=8, n_kv_heads=2, steps=48)
    run = ls.LockstepRun(wl, rebalance_interval=1, free_running=True)
    for _ in range(wl.steps):
        if run.diverged:
            break
        run.step(append=True)
    # expected on the seeded inputs: no flip at all; a flip at a cut would be admissible and is reported
    print("free-running %s: %d steps compared, %d boundary flips" % (cfg, run.step_idx, run.boundary_flips))
    assert run.boundary_flips == 0 or run.diverged
    run.close()


@pytest.mark.parametrize("kw", [
    dict(sink_windows=2, recent_windows=3),
    dict(sink_windows=1, recent_windows=0, dtype="bf16", head_dim=128, n_q_heads=8, n_kv_heads=2, quant_bits=2),
    dict(sink_windows=0, recent_windows=2, window=64, group_size=64, context=2048, head_dim=128, n_q_heads=8, n_kv_heads=1,
         dtype="bf16"),
], ids=lambda kw: "-".join("%s%s" % (k[0], v) for k, v in kw.items()))
def test_protected_sink_and_recent_windows(kw):
    # the sink prefix and the recent region stay in full precision outside K_f and never become candidates;
    # filled windows turn into candidates only when newer windows have pushed them out of the recent region
    ls = _lockstep()
    w = kw.get("window", 32)
    wl = _small("protected", steps=4 * w + 7, **kw)
    for interval in (1, 5):
        run = ls.LockstepRun(wl, rebalance_interval=interval)
        run.check_state("all", "after prefill")
        st = run.cache.stats()
        assert st["n_sink"] == wl.sink_windows and st["n_aged"] == wl.recent_windows
        assert (st["n_full"], st["n_quant"]) == (wl.fp_budget_windows, wl.q_budget_windows)
        for _ in range(wl.steps):
            run.step(append=True)
        run.rebalance(full_check=True)
        st = run.cache.stats()
        assert st["n_sink"] == wl.sink_windows and st["n_aged"] == wl.recent_windows
        assert st["deletions"] == run.oracles[0].stats["deletions"] > 0
        run.close()


@pytest.mark.parametrize("mode,param", [(1, 0.9), (1, 0.5), (2, 3.0), (2, 2.0), (3, 0.0)])
def test_ranking_function_variants(mode, param):
    # decayed attention and attention p-norm: the mass is collected per routing event and folded into the score
    # in float32 by the routing kernel; key norm (mode 3): the score is minus the mean key norm of a complete
    # window; tiers, pages and codes must still match bit for bit
    ls = _lockstep()
    wl = _small("rank", steps=72, dtype="bf16", head_dim=128, n_q_heads=8, n_kv_heads=2, rank_mode=mode, rank_param=param)
    run = ls.LockstepRun(wl, rebalance_interval=3)
    run.check_state("all", "after prefill")
    for _ in range(wl.steps):
        run.step(append=True)
    run.rebalance(full_check=True)
    o = run.oracles[0]
    st = run.cache.stats()
    assert st["promotions"] == o.stats["promotions"] and st["deletions"] == o.stats["deletions"] > 0
    run.close()


def test_more_than_4096_windows():
    # the routing kernel reads window states 16 per thread up to 4096 windows and falls back to a block-wide
    # compaction above that; this prompt has 4200 windows
    ls = _lockstep()
    wl = _small("long", context=4200 * 32, n_q_heads=1, n_kv_heads=1, fp_budget_windows=6, q_budget_windows=10, steps=40,
                sink_windows=1, recent_windows=1)
    run = ls.LockstepRun(wl, rebalance_interval=1, score_mode="synthetic")
    run.check_state("all", "after prefill")
    st = run.cache.stats()
    assert (st["n_full"], st["n_quant"], st["n_sink"], st["n_aged"]) == (6, 10, 1, 1)
    assert st["n_evicted"] == 4200 - 18
    for _ in range(wl.steps):
        run.step(append=True)
    run.rebalance(full_check=True)
    run.close()


def test_routing_diagnostics_match_the_oracle():
    # tier-mass share and selection churn of the observation appendix, from the exported tables
    from oracle import retained_windows, selection_churn, tier_mass_share
    from paper_2608_05326_b200 import diagnostics
    ls = _lockstep()
    wl = _small("diag", steps=100, dtype="bf16", head_dim=128, n_q_heads=8, n_kv_heads=2, sink_windows=1)
    run = ls.LockstepRun(wl, rebalance_interval=4)
    prev_g = prev_o = None
    churns = []
    for t in range(wl.steps):
        run.step(append=True)
        if run.step_idx % 4 == 0:  # a routing event has just run
            tab = run.cache.export_tables(0, 0)
            orc = run.oracles[0]
            mu_g, mu_o = diagnostics.tier_mass_share(tab), tier_mass_share(orc)
            for k in mu_o:
                assert abs(mu_g[k] - mu_o[k]) <= 1e-4 * max(mu_o[k], 1e-6) + 1e-9, (k, mu_g[k], mu_o[k])
            assert abs(sum(mu_g.values()) - 1.0) < 1e-9
            rg, ro = diagnostics.retained_windows(tab), retained_windows(orc)
            assert rg == ro
            if prev_g is not None:
                cg, co = diagnostics.selection_churn(prev_g, rg), selection_churn(prev_o, ro)
                assert cg == co
                churns.append(cg)
            prev_g, prev_o = rg, ro
    assert len(churns) == wl.steps // 4 - 1 and all(0.0 <= c <= 1.0 for c in churns)
    run.close()


@pytest.mark.parametrize("kw", [dict(), dict(context=16384, n_q_heads=1, n_kv_heads=1, fp_budget_windows=120, q_budget_windows=260, steps=8)],
                         ids=["small", "380-candidates"])
def test_one_way_policy(kw):
    # no promotion: Quantized windows leave their tier only by eviction; tiers, pages and codes bit for bit
    ls = _lockstep()
    wl = _small("oneway", **{**dict(steps=72, dtype="bf16", head_dim=128, n_q_heads=8, n_kv_heads=2, one_way=True), **kw})
    run = ls.LockstepRun(wl, rebalance_interval=1, score_mode="synthetic")
    run.check_state("all", "after prefill")
    for _ in range(wl.steps):
        run.step(append=True)
    run.rebalance(full_check=True)
    st = run.cache.stats()
    assert st["promotions"] == 0 == run.oracles[0].stats["promotions"]
    assert st["deletions"] == run.oracles[0].stats["deletions"] and st["quantizations"] == run.oracles[0].stats["quantizations"]
    run.close()


def test_many_candidates_and_tied_scores():
    # more candidates than the counting rank handles (radix selection of the two cuts), with prefill scores
    # on 7 levels, so that both cuts fall inside large groups of equal scores and the window index decides
    ls = _lockstep()
    wl = _small("ties", context=16384, n_q_heads=1, n_kv_heads=1, fp_budget_windows=120, q_budget_windows=260, steps=10)
    run = ls.LockstepRun(wl, rebalance_interval=1, score_levels=7)
    run.check_state("all", "after prefill")
    st = run.cache.stats()
    assert (st["n_full"], st["n_quant"]) == (120, 260)
    for _ in range(wl.steps):
        run.step(append=True)
    run.rebalance(full_check=True)
    run.close()


def test_multiple_units_and_layers():
    ls = _lockstep()
    wl = _small("multi", batch=3, n_layers=2, dtype="bf16", head_dim=128, n_q_heads=8, n_kv_heads=2, steps=40)
    run = ls.LockstepRun(wl, rebalance_interval=2)
    run.check_state("all", "after prefill")
    for _ in range(wl.steps):
        run.step(append=True)
    run.rebalance(full_check=True)
    run.close()


def test_per_layer_calls_match_all_layer_call():
    """layer >= 0 calls on one layer give the same bits as the layer == -1 launch."""
    ls = _lockstep()
    wl = _small("perlayer", batch=2, n_layers=2, dtype="bf16", head_dim=128, n_q_heads=8, n_kv_heads=2, steps=8)
    run = ls.LockstepRun(wl, oracle_units=[])
    cache2 = binding.QEvictCache(ls.gpu_config(wl))
    dev = run.dev
    for layer in range(2):
        units = [layer * 2, layer * 2 + 1]
        k = torch.stack([workloads.gen_prompt_kv(wl, u)[0] for u in units]).to(dev)
        v = torch.stack([workloads.gen_prompt_kv(wl, u)[1] for u in units]).to(dev)
        s = torch.stack([run.scores[u] for u in units]).to(dev)
        cache2.prefill_assign(layer, k, v, s)
    for t in range(wl.steps):
        out_all = run.step(append=True, check_mass=False)
        for layer in range(2):
            units = [layer * 2, layer * 2 + 1]
            q = torch.stack([run.queries[u][t] for u in units]).to(dev)
            kn = torch.stack([run.new_kv[u][0][t] for u in units]).to(dev)
            vn = torch.stack([run.new_kv[u][1][t] for u in units]).to(dev)
            o = cache2.decode_attn(layer, q, kn, vn).cpu()
            assert torch.equal(o, out_all[units[0]:units[1] + 1])
            cache2.rebalance(layer)
    for u in range(4):
        a = run.cache.export_tables(u // 2, u % 2)
        b = cache2.export_tables(u // 2, u % 2)
        for key in a:
            assert torch.equal(a[key], b[key]), key
    cache2.close()
    run.close()


def test_split_count_changes_only_rounding_order():
    ls = _lockstep()
    wl = replace(workloads.config(0), steps=6)
    outs = []
    for splits in (1, 3, 16):
        run = ls.LockstepRun(wl, oracle_units=[])
        run.cache.set_splits(splits)
        o = [run.step(append=True, check_mass=False).double() for _ in range(wl.steps)]
        imp = run.cache.export_tables(0, 0)["importance"].double()
        outs.append((torch.stack(o), imp))
        run.close()
    for o, imp in outs[1:]:
        assert torch.allclose(o, outs[0][0], atol=2e-3, rtol=1e-2)
        assert torch.allclose(imp, outs[0][1], rtol=1e-5, atol=1e-7)


def test_runs_are_bit_reproducible():
    ls = _lockstep()
    wl = _small("repro", dtype="bf16", head_dim=128, n_q_heads=8, n_kv_heads=2, steps=20)
    res = []
    for _ in range(2):
        run = ls.LockstepRun(wl, oracle_units=[])
        o = torch.stack([run.step(append=True, check_mass=False) for _ in range(wl.steps)])
        tab = run.cache.export_tables(0, 0)
        res.append((o, tab))
        run.close()
    assert torch.equal(res[0][0], res[1][0])
    for key in res[0][1]:
        assert torch.equal(res[0][1][key], res[1][1][key]), key


def test_everything_full_precision_equals_plain_attention():
    """With the full-precision budget covering the whole context the output is ordinary attention."""
    wl = _small("allfp", dtype="bf16", head_dim=128, n_q_heads=8, n_kv_heads=2, context=512, fp_budget_windows=24,
                q_budget_windows=2, steps=10)
    ls = _lockstep()
    run = ls.LockstepRun(wl)
    k, v = workloads.gen_prompt_kv(wl, 0)
    ks, vs = [k.double()], [v.double()]
    for t in range(wl.steps):
        out = run.step(append=True)[0].double()
        ks.append(run.new_kv[0][0][t].double()[:, None]); vs.append(run.new_kv[0][1][t].double()[:, None])
        kk = torch.cat(ks, 1).repeat_interleave(4, 0); vv = torch.cat(vs, 1).repeat_interleave(4, 0)
        q = run.queries[0][t].double()
        p = torch.softmax(torch.einsum("hd,hnd->hn", q, kk) / np.sqrt(wl.head_dim), -1)
        ref = torch.einsum("hn,hnd->hd", p, vv)
        assert torch.all((out - ref).abs() <= 2e-3 + 1e-2 * ref.abs())
    assert run.cache.stats()["n_evicted"] == 0
    run.close()


def test_host_buffer_entry_point_matches_device_call():
    ls = _lockstep()
    wl = _small("host", dtype="bf16", head_dim=128, n_q_heads=8, n_kv_heads=2, steps=5, batch=2)
    a = ls.LockstepRun(wl, oracle_units=[])
    b = ls.LockstepRun(wl, oracle_units=[])
    for t in range(wl.steps):
        oa = a.step(append=True, check_mass=False)
        # page-locked buffers are read and written in place by the kernels; pageable ones take staged copies
        pin = (lambda x: x.pin_memory()) if t < 3 else (lambda x: x)
        q = pin(torch.stack([b.queries[u][t] for u in range(2)]).contiguous().cpu())
        kn = pin(torch.stack([b.new_kv[u][0][t] for u in range(2)]).contiguous().cpu())
        vn = pin(torch.stack([b.new_kv[u][1][t] for u in range(2)]).contiguous().cpu())
        out = pin(torch.empty_like(q))
        if t % 2 == 0:
            b.cache.decode_attn_host(-1, q, kn, vn, out)
            b.cache.rebalance(-1)
        else:  # the variant that only enqueues: the routing event goes in before the host waits for the result
            b.cache.decode_attn_host_async(-1, q, kn, vn, out)
            b.cache.rebalance(-1)
            if t == 1:
                b.cache.wait_result()  # waits for `out` only; the routing event may still be running
            else:
                torch.cuda.current_stream().synchronize()
        assert torch.equal(out, oa.cpu())
    a.close(); b.close()


def test_call_order_errors():
    wl = _small("errors", rebalance_interval=32, steps=200)
    ls = _lockstep()
    cache = binding.QEvictCache(ls.gpu_config(wl))
    q = torch.zeros((1, 1, wl.n_q_heads, wl.head_dim), dtype=torch.float16, device="cuda")
    with pytest.raises(binding.QEvictError) as e:
        cache.decode_attn(-1, q)
    assert e.value.status == 2
    with pytest.raises(binding.QEvictError) as e:
        cache.rebalance(0)
    assert e.value.status == 2
    k, v = workloads.gen_prompt_kv(wl, 0)
    s = workloads.synthetic_window_scores(wl, 0)
    cache.prefill_assign(0, k[None].cuda(), v[None].cuda(), s[None].cuda())
    with pytest.raises(binding.QEvictError) as e:
        cache.prefill_assign(0, k[None].cuda(), v[None].cuda(), s[None].cuda())
    assert e.value.status == 2
    # appending without ever rebalancing runs out of pages for aged windows: refused on the host
    kn = torch.zeros((1, 1, wl.n_kv_heads, wl.head_dim), dtype=torch.float16, device="cuda")
    with pytest.raises(binding.QEvictError) as e:
        for _ in range(10 * wl.window):
            cache.decode_attn(-1, q, kn, kn)
    assert e.value.status == 2
    cache.rebalance(-1)
    cache.decode_attn(-1, q, kn, kn)
    assert cache.stats()["n_aged"] == 0
    cache.close()


def test_config1_llama_shape_lockstep():
    ls = _lockstep()
    wl = replace(workloads.config(1), steps=40)
    run = ls.LockstepRun(wl)
    run.check_state("all", "after prefill")
    st = run.cache.stats()
    assert (st["n_full"], st["n_quant"], st["n_evicted"]) == (64, 128, 832)
    for _ in range(wl.steps):
        run.step(append=True)
    run.rebalance(full_check=True)
    assert run.cache.stats()["promotions"] == run.oracles[0].stats["promotions"]
    run.close()


@pytest.mark.parametrize("kw,n_obs", [
    (dict(dtype="bf16", head_dim=128, n_q_heads=8, n_kv_heads=2, batch=2, context=2048), 6),     # tensor-core path, N = 32
    (dict(dtype="fp16", head_dim=64, n_q_heads=3, n_kv_heads=1, window=64, group_size=32, context=1024), 6),
    (dict(dtype="bf16", head_dim=128, n_q_heads=8, n_kv_heads=1, context=1024), 12),              # 96 queries: N = 128
    (dict(dtype="bf16", head_dim=128, n_q_heads=8, n_kv_heads=2, context=1056), 5),               # not a multiple of 128: CUDA cores
    (dict(dtype="fp16", head_dim=128, n_q_heads=8, n_kv_heads=1, context=1024), 20),              # 160 queries: CUDA cores
    (dict(dtype="bf16", head_dim=128, n_q_heads=8, n_kv_heads=2, context=1024, rope_base=500000.0), 8),   # pre-RoPE keys
    (dict(dtype="fp16", head_dim=64, n_q_heads=4, n_kv_heads=2, context=1056, rope_base=10000.0), 5),     # same, CUDA cores
], ids=["bf16-d128-g4", "fp16-d64-w64", "bf16-96q", "bf16-ctx1056", "fp16-160q", "bf16-rope", "fp16-rope-ctx1056"])
def test_prefill_scores_on_the_gpu_match_the_oracle(kw, n_obs):
    """Window scores of the prompt from observation queries: the GPU routine against the oracle's attention
    (raw mass per window summed over observers and heads); then a prefill_assign on both sides from the
    oracle's scores."""
    from oracle import accessible_attention, apply_rope
    ls = _lockstep()
    wl = _small("pscore", steps=4, **kw)
    cache = binding.QEvictCache(ls.gpu_config(wl))
    orcs = []
    ks, vs, qs = [], [], []
    for u in range(wl.n_units):
        k, v = workloads.gen_prompt_kv(wl, u)
        g = torch.Generator().manual_seed(991 + u)
        q = torch.randn((n_obs, wl.n_q_heads, wl.head_dim), generator=g).to(wl.torch_dtype)
        ks.append(k); vs.append(v); qs.append(q)
    kd, vd, qd = torch.stack(ks).cuda(), torch.stack(vs).cuda(), torch.stack(qs).cuda()
    got = cache.prefill_score(kd, qd)
    torch.cuda.synchronize()
    scale = 1.0 / np.sqrt(wl.head_dim)
    ref_all = []
    for u in range(wl.n_units):
        k64 = ks[u].double().numpy()
        if wl.rope_base > 0:  # the prompt keys are pre-RoPE: attention sees them rotated for their positions
            k64 = apply_rope(k64, np.arange(k64.shape[1]), wl.rope_base, wl.dtype)
        ref = np.zeros(wl.n_prompt_windows)
        for o in range(n_obs):
            _, p = accessible_attention(qs[u][o].double().numpy(), k64, np.zeros_like(k64[:, :, :1]), scale)
            ref += p.sum(0).reshape(wl.n_prompt_windows, wl.window).sum(1)
        g_u = got[u].cpu().double().numpy()
        assert abs(g_u.sum() - n_obs * wl.n_q_heads) < 1e-3
        assert np.all(np.abs(g_u - ref) <= ls.MASS_RTOL * np.abs(ref) + 1e-7), np.abs(g_u - ref).max()
        ref_all.append(ref)
    # scores of this kind drive the first tier assignment: both sides are given the oracle's scores (as float32)
    refs = torch.from_numpy(np.stack(ref_all).astype(np.float32))
    cache.prefill_assign(0, kd, vd, refs.cuda())
    for u in range(wl.n_units):
        orc = ls.UnitOracle(ls.oracle_config(wl, ls.aged_capacity(wl)))
        orc.prefill_assign(ks[u].double().numpy(), vs[u].double().numpy(), refs[u].numpy())
        ls.compare_state(cache, 0, u, orc, wl, what="prefill from observation scores, unit %d" % u)
    cache.close()


def _random_workloads(n, seed=20260805):
    """Seeded draws over the supported configuration space (shapes, tiers, protected regions, ranking
    functions, routing intervals, pre-RoPE keys in two draws of five)."""
    rng = np.random.default_rng(seed)
    rope_rng = np.random.default_rng(seed + 1)  # its own stream: the other draws stay what they were
    out = []
    for i in range(n):
        window = int(rng.choice([32, 64]))
        group = int(rng.choice([32, 64])) if window == 64 else 32
        head_dim = int(rng.choice([64, 128]))
        if head_dim % group:
            group = 32
        n_kv = int(rng.choice([1, 2, 3]))
        gq = int(rng.choice([1, 2, 3, 4, 5, 7, 8]))
        n_win = int(rng.integers(10, 28))
        k_f = int(rng.integers(0, 6))
        k_q = int(rng.integers(0 if k_f else 1, 9))
        mode = int(rng.choice([0, 0, 1, 2, 3]))
        param = {0: 0.0, 1: float(rng.choice([0.5, 0.9, 0.99])), 2: float(rng.choice([2, 3])), 3: 0.0}[mode]
        interval = int(rng.choice([1, 2, 7, window, window + 5]))
        wl = _small("fuzz%d" % i, dtype=str(rng.choice(["fp16", "bf16"])), head_dim=head_dim, n_q_heads=gq * n_kv,
                    n_kv_heads=n_kv, window=window, group_size=group, quant_bits=int(rng.choice([2, 4])),
                    context=n_win * window, fp_budget_windows=k_f, q_budget_windows=k_q,
                    sink_windows=int(rng.integers(0, 3)), recent_windows=int(rng.integers(0, 3)),
                    rank_mode=mode, rank_param=param, steps=2 * window + int(rng.integers(3, 20)),
                    batch=int(rng.choice([1, 2])), rebalance_interval=interval,
                    rope_base=float(rope_rng.choice([0.0, 0.0, 0.0, 10000.0, 500000.0])))
        out.append(wl)
    return out


@pytest.mark.parametrize("wl", _random_workloads(24), ids=lambda wl: "%s-%s-d%d-h%d/%d-w%d-g%d-b%d-f%d-q%d-s%d-r%d-m%d-R%d" % (
    wl.name, wl.dtype, wl.head_dim, wl.n_q_heads, wl.n_kv_heads, wl.window, wl.group_size, wl.quant_bits,
    wl.fp_budget_windows, wl.q_budget_windows, wl.sink_windows, wl.recent_windows, wl.rank_mode, wl.rebalance_interval))
def test_random_configurations_lockstep(wl):
    ls = _lockstep()
    run = ls.LockstepRun(wl, rebalance_interval=wl.rebalance_interval, score_mode="synthetic")
    run.check_state("all", "after prefill")
    for _ in range(wl.steps):
        run.step(append=True)
    run.rebalance(full_check=True)
    for u, orc in run.oracles.items():
        layer, seq = run.unit_ls(u)
        st = run.cache.stats(layer)
        assert st["n_sink"] >= 0
    o = run.oracles[0]
    st = run.cache.stats()
    assert st["deletions"] == sum(x.stats["deletions"] for x in run.oracles.values())
    assert st["promotions"] == sum(x.stats["promotions"] for x in run.oracles.values())
    run.close()


@pytest.mark.parametrize("kw", [
    dict(dtype="bf16", head_dim=128, n_q_heads=8, n_kv_heads=2, rope_base=10000.0),
    dict(dtype="fp16", head_dim=64, n_q_heads=4, n_kv_heads=2, rope_base=500000.0),
    dict(dtype="bf16", head_dim=128, n_q_heads=8, n_kv_heads=1, quant_bits=2, rope_base=500000.0),
    dict(dtype="fp16", head_dim=128, n_q_heads=7, n_kv_heads=1, window=64, group_size=64, quant_bits=2, rope_base=10000.0),
    dict(dtype="bf16", head_dim=64, n_q_heads=3, n_kv_heads=1, window=64, quant_bits=4, rope_base=1000000.0,
         context=64 * 2040, fp_budget_windows=5, q_budget_windows=9),
])
def test_pre_rope_keys_rotated_at_attention_time(kw):
    # the cache holds pre-RoPE keys in every tier (they are quantized and promoted as such: codes and pages must
    # still match bit for bit) and the attention kernel rotates each key for its absolute position when it reads
    # it, after dequantization; the last case puts the positions near 130000
    ls = _lockstep()
    wl = _small("rope", steps=70, **kw)
    run = ls.LockstepRun(wl, rebalance_interval=2)
    run.check_state("all", "after prefill")
    for _ in range(wl.steps):
        run.step(append=True)
    run.rebalance(full_check=True)
    o = run.oracles[0]
    st = run.cache.stats()
    assert st["promotions"] == o.stats["promotions"] and st["quantizations"] == o.stats["quantizations"] > 0
    run.close()


def test_pre_rope_keys_change_the_result():
    # the same inputs with and without the rotation must not give the same output (a kernel that ignored the
    # rotation table would pass a comparison against itself, not this one)
    ls = _lockstep()
    a = ls.LockstepRun(_small("norope", steps=3), oracle_units=[])
    b = ls.LockstepRun(_small("norope", steps=3, rope_base=10000.0), oracle_units=[])
    oa = a.step(append=True, check_mass=False)
    ob = b.step(append=True, check_mass=False)
    assert (oa.float() - ob.float()).abs().max() > 1e-2
    a.close(); b.close()


@pytest.mark.parametrize("kw,gain", [
    (dict(dtype="bf16", head_dim=128, n_q_heads=8, n_kv_heads=2), 6.0),
    (dict(dtype="fp16", head_dim=64, n_q_heads=7, n_kv_heads=1, quant_bits=2), 8.0),
    (dict(dtype="bf16", head_dim=128, n_q_heads=4, n_kv_heads=1, window=64, group_size=64, quant_bits=2), 0.02),
], ids=["bf16-sharp", "fp16-gqa7-sharp", "w64-flat"])
def test_sharp_and_flat_attention_distributions(kw, gain):
    """Queries scaled up (logits spread over hundreds of log2 units: a few tokens take all the mass, and the running
    reference exponent of the online softmax is overtaken again and again) and down (every token matters
    equally): outputs, window mass and routing must stay within the same tolerances."""
    ls = _lockstep()
    wl = _small("sharp", steps=24, context=2048, fp_budget_windows=6, q_budget_windows=12, **kw)
    run = ls.LockstepRun(wl)
    for u in list(run.queries):
        run.queries[u] = (run.queries[u].float() * gain).to(run.queries[u].dtype)
    for _ in range(wl.steps):
        run.step(append=True)
    run.rebalance(full_check=True)
    run.close()
