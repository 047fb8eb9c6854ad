"""Lockstep parity driver shared by the GPU tests: runs the CUDA cache and the CPU oracle side by side
on the same seeded inputs and compares them after every call.

Protocol: each decode step both sides start from identical state; outputs and per-window mass are
compared within the floating-point tolerances; then the oracle's scores are overwritten with the
GPU's float32 scores, so that the routing decision (an integer result decided by floating point)
is taken on identical numbers on both sides, and everything the routing event produces -- tiers,
page tables, ledger flags, codes, parameters, promoted page contents -- must match bit for bit."""

import numpy as np
import torch

from oracle import (LEDGER_NONE, TIER_AGED, TIER_FULL, TIER_OPEN, TIER_QUANT, TIER_SINK, OracleConfig, UnitOracle,
                    accessible_attention)
from paper_2608_05326_b200 import binding, workloads

OUT_ATOL, OUT_RTOL = 2e-3, 1e-2     # attention output, 16-bit inputs, fp32 accumulation
MASS_RTOL = 1e-4                    # window scores / per-step mass


def oracle_config(wl, aged_windows):
    return OracleConfig(wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.dtype, wl.window, wl.quant_bits, wl.group_size,
                        wl.fp_budget_windows, wl.q_budget_windows, wl.max_context, aged_windows=aged_windows,
                        sink_windows=wl.sink_windows, recent_windows=wl.recent_windows, rank_mode=wl.rank_mode,
                        rank_param=wl.rank_param, one_way=wl.one_way, rope_base=wl.rope_base)


def gpu_config(wl, batch=None, n_layers=None, rebalance_interval=None):
    r = wl.rebalance_interval if rebalance_interval is None else rebalance_interval
    return binding.make_config(wl.batch if batch is None else batch, wl.n_layers if n_layers is None else n_layers,
                               wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.dtype, wl.window, wl.quant_bits,
                               wl.group_size, wl.fp_budget_windows, wl.q_budget_windows, wl.max_context,
                               rebalance_interval_hint=r, sink_windows=wl.sink_windows, recent_windows=wl.recent_windows,
                               rank_mode=wl.rank_mode, rank_param=wl.rank_param, one_way=wl.one_way,
                               rope_base=wl.rope_base)


def aged_capacity(wl, rebalance_interval=None):
    r = wl.rebalance_interval if rebalance_interval is None else rebalance_interval
    return (r + wl.window - 1) // wl.window + 1


def observation_scores(wl, unit, k64, n_obs=8):
    """Prefill window scores: raw attention mass of n_obs N(0,1) observation queries per head under
    full-precision attention over the whole prompt (computed with the oracle's attention routine)."""
    g = torch.Generator().manual_seed(wl.seed * 31 + unit * 7 + 5)
    qs = torch.randn((n_obs, wl.n_q_heads, wl.head_dim), generator=g, dtype=torch.float64).numpy()
    scale = 1.0 / np.sqrt(wl.head_dim)
    mass = np.zeros(wl.n_prompt_windows)
    dummy_v = np.zeros_like(k64[:, :, :1])
    for i in range(n_obs):
        _, p = accessible_attention(qs[i], k64, dummy_v, scale)
        mass += p.sum(0).reshape(wl.n_prompt_windows, wl.window).sum(1)
    return torch.from_numpy(mass.astype(np.float32))


def assert_out_close(got, ref, what=""):
    got = np.asarray(got, dtype=np.float64)
    err = np.abs(got - ref)
    bound = OUT_ATOL + OUT_RTOL * np.abs(ref)
    assert np.all(err <= bound), "%s attention output off: max err %.3e (bound %.3e)" % (
        what, err.max(), bound.flat[err.argmax()])


def assert_mass_close(got, ref, n_q_heads, what=""):
    got = np.asarray(got, dtype=np.float64)
    err = np.abs(got - ref)
    bound = MASS_RTOL * np.abs(ref) + 1e-9 * n_q_heads
    assert np.all(err <= bound), "%s window mass off: max err %.3e at %d (ref %.6e)" % (
        what, err.max(), int(err.argmax()), ref.flat[err.argmax()])


def compare_state(cache, layer, seq, orc, wl, check_pages=None, what=""):
    """Bit-exact comparison of tables; `check_pages`: None = all live pages, else iterable of windows."""
    t = cache.export_tables(layer, seq)
    n = int(t["n_windows"][0])
    assert n == orc.n_windows, "%s n_windows %d != %d" % (what, n, orc.n_windows)
    for name, ref in (("tier", orc.tier), ("ledger", orc.ledger_flag), ("fp_page", orc.fp_page), ("q_page", orc.q_page)):
        got = t[name].numpy()[:n]
        bad = np.flatnonzero(got != ref[:n])
        assert bad.size == 0, "%s %s differs at windows %s: gpu %s oracle %s" % (
            what, name, bad[:8], got[bad[:8]], ref[:n][bad[:8]])
    windows = range(n) if check_pages is None else check_pages
    for w in windows:
        if orc.fp_page[w] >= 0 and orc.tier[w] in (TIER_FULL, TIER_AGED, TIER_OPEN, TIER_SINK):
            k, v = cache.export_fp_page(layer, seq, int(orc.fp_page[w]))
            rk, rv = orc.fp[w]
            if orc.tier[w] == TIER_OPEN:
                f = orc.open_fill
                assert np.array_equal(k.double().numpy()[:, :f], rk[:, :f]) and np.array_equal(v.double().numpy()[:, :f], rv[:, :f]), \
                    "%s open window %d contents differ" % (what, w)
            else:
                assert np.array_equal(k.double().numpy(), rk), "%s fp K of window %d differs" % (what, w)
                assert np.array_equal(v.double().numpy(), rv), "%s fp V of window %d differs" % (what, w)
        if orc.ledger_flag[w] != LEDGER_NONE:
            kc, kp, vc, vp = cache.export_q_page(layer, seq, int(orc.q_page[w]))
            e = orc.ledger[w]
            assert np.array_equal(kc.numpy(), e["k_codes"]), "%s K codes of window %d differ" % (what, w)
            assert np.array_equal(vc.numpy(), e["v_codes"]), "%s V codes of window %d differ" % (what, w)
            assert np.array_equal(kp[..., 0].double().numpy(), e["k_s"]) and np.array_equal(kp[..., 1].double().numpy(), e["k_z"]), \
                "%s K params of window %d differ" % (what, w)
            assert np.array_equal(vp[..., 0].double().numpy(), e["v_s"]) and np.array_equal(vp[..., 1].double().numpy(), e["v_z"]), \
                "%s V params of window %d differ" % (what, w)
    return t


class LockstepRun:
    """One workload instance on the GPU (all its units in one cache) and oracles for a subset of units."""

    def __init__(self, wl, oracle_units=None, score_mode="observation", rebalance_interval=None, device="cuda",
                 gen_device="cpu", score_levels=None, free_running=False, entry="decode_attn"):
        self.wl = wl
        self.entry = entry  # which decode entry point the steps go through: "decode_attn" or "noalloc"
        self.R = wl.rebalance_interval if rebalance_interval is None else rebalance_interval
        self.units = list(range(wl.n_units)) if oracle_units is None else list(oracle_units)
        self.cache = binding.QEvictCache(gpu_config(wl, rebalance_interval=self.R))
        self.dev = torch.device(device)
        ocfg = oracle_config(wl, aged_capacity(wl, self.R))
        self.oracles = {u: UnitOracle(ocfg) for u in self.units}
        self.k_prompt, self.scores, self.queries, self.new_kv = {}, {}, {}, {}
        # prompts are generated (on `gen_device`) and handed to the cache layer by layer; only the units
        # that have an oracle are copied to the host
        for layer in range(wl.n_layers):
            ks, vs, ss = [], [], []
            for u in range(layer * wl.batch, (layer + 1) * wl.batch):
                k, v = workloads.gen_prompt_kv(wl, u, device=gen_device)
                if u in self.oracles and score_mode == "observation":
                    s = observation_scores(wl, u, k.cpu().double().numpy())
                else:
                    s = workloads.synthetic_window_scores(wl, u)
                s = workloads.place_planted(s, workloads.planted_windows(wl, u), wl.fp_budget_windows,
                                            wl.q_budget_windows)
                if score_levels:  # few distinct prefill scores: the first routing event is decided by the tie-break
                    s = torch.round(s / s.max() * score_levels) * (s.max() / score_levels)
                ks.append(k); vs.append(v); ss.append(s)
                self.scores[u] = s
                self.queries[u] = workloads.gen_queries(wl, u, k, s)
                self.new_kv[u] = workloads.gen_new_kv(wl, u)
                if u in self.oracles:
                    self.oracles[u].prefill_assign(k.cpu().double().numpy(), v.cpu().double().numpy(), s.numpy())
            kd = torch.stack(ks).to(self.dev)
            vd = torch.stack(vs).to(self.dev)
            sd = torch.stack(ss).contiguous().to(self.dev)
            self.cache.prefill_assign(layer, kd, vd, sd)
            torch.cuda.synchronize()
            del ks, vs, kd, vd
        self.step_idx = 0
        # free-running: the oracle keeps its own float64 scores (no overwrite with the GPU's); a routing event
        # may then differ, but only by windows whose scores sit on a tier cut (see rebalance)
        self.free_running = free_running
        self.boundary_flips = 0
        self.diverged = False

    def unit_ls(self, u):
        return u // self.wl.batch, u % self.wl.batch

    def check_state(self, pages="all", what=""):
        for u, orc in self.oracles.items():
            layer, seq = self.unit_ls(u)
            compare_state(self.cache, layer, seq, orc, self.wl, None if pages == "all" else pages.get(u, []),
                          what="%s unit %d" % (what, u))

    def _decode(self, layer, q, kn, vn):
        if self.entry == "noalloc":
            out = torch.empty_like(q)
            binding.qevict_decode_attn_noalloc(self.cache.handle, layer, q, kn, vn, out)
            return out
        return self.cache.decode_attn(layer, q, kn, vn)

    def step(self, append=True, check_mass=True, per_layer=False):
        """One decode step of every unit; per_layer=True issues one call per layer instead of one for all."""
        wl, t = self.wl, self.step_idx
        shape_q = (wl.n_layers, wl.batch, wl.n_q_heads, wl.head_dim)
        shape_kv = (wl.n_layers, wl.batch, wl.n_kv_heads, wl.head_dim)
        q = torch.stack([self.queries[u][t] for u in range(wl.n_units)]).reshape(shape_q).to(self.dev)
        kn = vn = None
        if append:
            kn = torch.stack([self.new_kv[u][0][t] for u in range(wl.n_units)]).reshape(shape_kv).to(self.dev)
            vn = torch.stack([self.new_kv[u][1][t] for u in range(wl.n_units)]).reshape(shape_kv).to(self.dev)
        if per_layer:
            out = torch.stack([self._decode(l, q[l].contiguous(), None if kn is None else kn[l].contiguous(),
                                            None if vn is None else vn[l].contiguous()) for l in range(wl.n_layers)])
        else:
            out = self._decode(-1, q, kn, vn)
        out = out.cpu().reshape(wl.n_units, wl.n_q_heads, wl.head_dim)
        for u, orc in self.oracles.items():
            layer, seq = self.unit_ls(u)
            ref_out, ref_mass = orc.decode_attn(self.queries[u][t].double().numpy(),
                                                None if not append else self.new_kv[u][0][t].double().numpy(),
                                                None if not append else self.new_kv[u][1][t].double().numpy())
            what = "step %d unit %d" % (t, u)
            assert_out_close(out[u].double().numpy(), ref_out, what)
            tab = self.cache.export_tables(layer, seq)
            if check_mass:
                mass = self.cache.export_last_mass(layer, seq).double().numpy()
                assert_mass_close(mass, ref_mass, wl.n_q_heads, what)
                assert abs(mass.sum() - wl.n_q_heads) < 1e-4 * wl.n_q_heads, what
            imp = tab["importance"].double().numpy()
            assert np.all(np.abs(imp - orc.importance) <= MASS_RTOL * np.abs(orc.importance) + 1e-7), what + " scores"
            if wl.rank_mode != 0:  # the mass went to the event accumulator, the scores move at routing events only
                ev = self.cache.export_event_mass(layer, seq).double().numpy()
                assert np.all(np.abs(ev - orc.event_mass) <= MASS_RTOL * np.abs(orc.event_mass) + 1e-7), what + " event mass"
                if not self.free_running:
                    orc.event_mass[:] = ev
            if not self.free_running:
                orc.importance[:] = imp  # lockstep: route on the GPU's float32 scores
        self.step_idx += 1
        if self.step_idx % self.R == 0:
            self.rebalance(per_layer=per_layer)
        return out

    def rebalance(self, full_check=False, per_layer=False):
        if self.free_running:
            return self._rebalance_free()
        before = {u: (o.tier.copy(), o.ledger_flag.copy()) for u, o in self.oracles.items()}
        if per_layer:
            for l in range(self.wl.n_layers):
                self.cache.rebalance(l)
        else:
            self.cache.rebalance(-1)
        changed = {}
        for u, orc in self.oracles.items():
            orc.rebalance()
            t0, l0 = before[u]
            changed[u] = [int(w) for w in np.flatnonzero((t0 != orc.tier) | (l0 != orc.ledger_flag))
                          if orc.tier[w] in (TIER_FULL, TIER_QUANT, TIER_SINK)]
        self.check_state("all" if full_check else changed, what="after rebalance at step %d" % self.step_idx)

    def _rebalance_free(self):
        """Both sides route on their own scores.  Equal tiers -> everything must still match bit for bit.
        Different tiers are admissible only for windows whose oracle score lies within 1e-4 relative of the
        score at one of the two cuts (the K_f-th or the (K_f+K_q)-th candidate); the run then counts the flip
        and stops comparing states (pages are handed out differently from there on)."""
        wl = self.wl
        cuts = {}
        for u, orc in self.oracles.items():
            ranked = orc.ranked_candidates()
            sc = orc.importance.astype(np.float32)
            cuts[u] = [float(sc[ranked[k - 1]]) for k in (wl.fp_budget_windows, wl.fp_budget_windows + wl.q_budget_windows)
                       if 1 <= k <= len(ranked)]
            cuts[u] += [float(sc[ranked[k]]) for k in (wl.fp_budget_windows, wl.fp_budget_windows + wl.q_budget_windows)
                        if k < len(ranked)]
        self.cache.rebalance(-1)
        for u, orc in self.oracles.items():
            orc.rebalance()
            layer, seq = self.unit_ls(u)
            t = self.cache.export_tables(layer, seq)
            n = int(t["n_windows"][0])
            got = t["tier"].numpy()[:n]
            bad = np.flatnonzero(got != orc.tier[:n])
            if bad.size == 0:
                continue
            for w in bad:
                s = float(np.float32(orc.importance[w]))
                assert any(abs(s - c) <= MASS_RTOL * max(abs(c), 1e-30) for c in cuts[u]), \
                    "unit %d window %d: tiers differ (gpu %d oracle %d) away from a tier cut (score %.9g, cuts %s)" % (
                        u, w, got[w], orc.tier[w], s, cuts[u])
            self.boundary_flips += int(bad.size)
            self.diverged = True
        if not self.diverged:
            self.check_state("all", what="free-running, after rebalance at step %d" % self.step_idx)

    def close(self):
        self.cache.close()
