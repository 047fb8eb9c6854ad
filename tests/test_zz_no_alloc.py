"""The decode entry point for callers that must not allocate device memory.

Some users of this library run under a fixed device-memory plan: the serving process gave all of HBM to
its own pool at start-up, or the calling thread must never enter the CUDA allocator because that can
block behind unrelated work.  For them `qevict_decode_attn_noalloc` keeps the attention kernel's scratch
(the per-split partial results) in an array that is part of the library's device image.  This test drives
two identical caches through the same steps, one through the ordinary entry point and one through the
no-allocation one, and requires the same results on two calls in a row; it also checks that a call too
large for the built-in array is refused with a clear message instead of being run.

The file name sorts last on purpose, so that a run which stops at the first failure has already run every
other test."""

import pytest
import torch

from paper_2608_05326_b200 import binding, workloads

pytestmark = pytest.mark.gpu


def _workload(n_layers=1):
    return workloads.Workload(name="noalloc", batch=2, n_layers=n_layers, n_q_heads=8, n_kv_heads=2, head_dim=128,
                              dtype="bf16", context=1024, window=32, quant_bits=4, group_size=32,
                              fp_budget_windows=4, q_budget_windows=8, steps=8, rebalance_interval=1)


def _make_cache(wl, dev):
    cfg = binding.make_config(wl.batch, wl.n_layers, wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.dtype, wl.window,
                              wl.quant_bits, wl.group_size, wl.fp_budget_windows, wl.q_budget_windows, wl.max_context,
                              rebalance_interval_hint=1)
    cache = binding.QEvictCache(cfg)
    ks, vs, ss = [], [], []
    for u in range(wl.n_units):
        k, v = workloads.gen_prompt_kv(wl, u)
        ks.append(k); vs.append(v)
        ss.append(workloads.place_planted(workloads.synthetic_window_scores(wl, u), workloads.planted_windows(wl, u),
                                          wl.fp_budget_windows, wl.q_budget_windows))
    shape = (wl.n_layers, wl.batch)
    cache.prefill_assign(-1, torch.stack(ks).reshape(shape + ks[0].shape).to(dev), torch.stack(vs).reshape(shape + vs[0].shape).to(dev),
                         torch.stack(ss).reshape(shape + ss[0].shape).to(dev))
    return cache, ks, ss


def test_no_alloc_entry_point_matches_the_ordinary_one_twice_in_a_row():
    dev = torch.device("cuda")
    wl = _workload()
    ref, ks, ss = _make_cache(wl, dev)
    alt, _, _ = _make_cache(wl, dev)
    q_all = [workloads.gen_queries(wl, u, ks[u], ss[u]) for u in range(wl.n_units)]
    kv_all = [workloads.gen_new_kv(wl, u) for u in range(wl.n_units)]
    for t in range(2):  # two calls in a row: the second one finds the first one's leftovers in the array
        q = torch.stack([q_all[u][t] for u in range(wl.n_units)]).to(dev)
        kn = torch.stack([kv_all[u][0][t] for u in range(wl.n_units)]).to(dev)
        vn = torch.stack([kv_all[u][1][t] for u in range(wl.n_units)]).to(dev)
        out_ref = ref.decode_attn(0, q, kn, vn)
        out_alt = torch.empty_like(q)
        binding.qevict_decode_attn_noalloc(alt.handle, 0, q, kn, vn, out_alt)
        torch.cuda.synchronize()
        # the same kernels with the same split count: not merely close, the same bits
        assert torch.equal(out_alt, out_ref), "step %d" % t
        for seq in range(wl.batch):
            ta, tb = alt.export_tables(0, seq), ref.export_tables(0, seq)
            assert torch.equal(ta["importance"], tb["importance"])
            assert torch.equal(ta["tier"], tb["tier"])
        ref.rebalance(0)
        alt.rebalance(0)
    assert alt.stats()["decode_steps"] == 2
    ref.close(); alt.close()


def test_no_alloc_entry_point_on_single_layers_of_a_many_layer_cache():
    """The built-in array holds the partial results of the units of one call only, so a call for one layer needs
    that layer's room wherever the layer sits: layers 1 and 2 of three, then all three at once, against the
    ordinary entry point on a twin cache -- same bits, on two steps in a row."""
    dev = torch.device("cuda")
    wl = _workload(n_layers=3)
    ref, ks, ss = _make_cache(wl, dev)
    alt, _, _ = _make_cache(wl, dev)
    for c in (ref, alt):
        c.set_splits(3)  # the built-in choice depends on the units per call; the summation order follows the splits
    q_all = [workloads.gen_queries(wl, u, ks[u], ss[u]) for u in range(wl.n_units)]
    kv_all = [workloads.gen_new_kv(wl, u) for u in range(wl.n_units)]
    shape = (wl.n_layers, wl.batch)
    for t in range(2):
        q = torch.stack([q_all[u][t] for u in range(wl.n_units)]).reshape(shape + q_all[0][t].shape).to(dev)
        kn = torch.stack([kv_all[u][0][t] for u in range(wl.n_units)]).reshape(shape + kv_all[0][0][t].shape).to(dev)
        vn = torch.stack([kv_all[u][1][t] for u in range(wl.n_units)]).reshape(shape + kv_all[0][1][t].shape).to(dev)
        out_ref = ref.decode_attn(-1, q, kn, vn)
        out_alt = torch.empty_like(q)
        if t == 0:  # layer by layer, last layer first
            for layer in (2, 1, 0):
                o = torch.empty_like(q[layer])
                binding.qevict_decode_attn_noalloc(alt.handle, layer, q[layer].contiguous(), kn[layer].contiguous(),
                                                   vn[layer].contiguous(), o)
                out_alt[layer] = o
        else:
            binding.qevict_decode_attn_noalloc(alt.handle, -1, q, kn, vn, out_alt)
        torch.cuda.synchronize()
        assert torch.equal(out_alt, out_ref), "step %d" % t
        ref.rebalance(-1)
        alt.rebalance(-1)
    for u in range(wl.n_units):
        ta, tb = alt.export_tables(u // wl.batch, u % wl.batch), ref.export_tables(u // wl.batch, u % wl.batch)
        for key in ta:
            assert torch.equal(ta[key], tb[key]), (u, key)
    ref.close(); alt.close()


def test_no_alloc_entry_point_against_the_oracle():
    """A whole lockstep run (outputs, window mass, tiers, pages, codes against the CPU oracle at every step) with
    every decode step going through the no-allocation entry point."""
    import lockstep
    wl = workloads.Workload(name="noalloc-oracle", batch=2, n_layers=2, n_q_heads=8, n_kv_heads=2, head_dim=128,
                            dtype="bf16", context=1024, window=32, quant_bits=4, group_size=32, fp_budget_windows=4,
                            q_budget_windows=8, steps=40, rebalance_interval=1)
    run = lockstep.LockstepRun(wl, entry="noalloc")
    for t in range(wl.steps):
        run.step(append=True, per_layer=(t % 3 == 1))
    run.rebalance(full_check=True)
    run.close()


def test_no_alloc_entry_point_refuses_what_does_not_fit():
    dev = torch.device("cuda")
    # 64 units x 32 heads of partial results are far beyond the 8 MiB array
    wl = workloads.Workload(name="big", batch=64, n_layers=1, n_q_heads=32, n_kv_heads=8, head_dim=128, dtype="bf16",
                            context=256, window=32, quant_bits=4, group_size=32, fp_budget_windows=2,
                            q_budget_windows=2, steps=4, rebalance_interval=1)
    cache, _, _ = _make_cache(wl, dev)
    q = torch.zeros((wl.batch, wl.n_q_heads, wl.head_dim), dtype=torch.bfloat16, device=dev)
    out = torch.empty_like(q)
    with pytest.raises(binding.QEvictError) as e:
        binding.qevict_decode_attn_noalloc(cache.handle, 0, q, None, None, out)
    assert e.value.status == 3 and "bytes" in str(e.value)
    cache.decode_attn(0, q)  # the ordinary entry point still serves the same cache
    torch.cuda.synchronize()
    cache.close()
