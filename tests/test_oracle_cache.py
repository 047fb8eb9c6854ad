"""Pins for the oracle's attention, score update, routing and ledger.

Each check is against something other than the oracle itself: a textbook softmax written with a library
routine, closed forms, a brute-force sort, and the invariants the paper states."""

import hashlib

import numpy as np
import pytest
import torch
from scipy.special import softmax

from oracle import (
    LEDGER_ACTIVE,
    LEDGER_DORMANT,
    LEDGER_NONE,
    TIER_AGED,
    TIER_EVICTED,
    TIER_FULL,
    TIER_OPEN,
    TIER_QUANT,
    TIER_SINK,
    OracleConfig,
    UnitOracle,
    accessible_attention,
    round_to_dtype,
    tier_capacities,
    window_bytes,
)
from paper_2608_05326_b200 import workloads as wlmod


def _full_attention_reference(q, k, v, scale):
    """Textbook GQA softmax attention with library routines (scipy softmax, einsum)."""
    hq, d = q.shape
    hkv = k.shape[0]
    kk = np.repeat(k, hq // hkv, axis=0)
    vv = np.repeat(v, hq // hkv, axis=0)
    p = softmax(np.einsum("hd,hnd->hn", q, kk) * scale, axis=-1)
    return np.einsum("hn,hnd->hd", p, vv), p


def _rand_T(rng, shape, dtype, scale=1.0):
    return round_to_dtype(rng.standard_normal(shape) * scale, dtype)


# ------------------------------------------------------------------------------ attention
def test_attention_matches_textbook_softmax():
    rng = np.random.default_rng(10)
    q = rng.standard_normal((8, 64))
    k = rng.standard_normal((2, 300, 64))
    v = rng.standard_normal((2, 300, 64))
    out, p = accessible_attention(q, k, v, 0.125)
    ref_out, ref_p = _full_attention_reference(q, k, v, 0.125)
    assert np.allclose(out, ref_out, rtol=1e-12, atol=1e-13)
    assert np.allclose(p, ref_p, rtol=1e-12, atol=1e-15)


def test_attention_closed_forms():
    rng = np.random.default_rng(11)
    q = rng.standard_normal((4, 32))
    key = rng.standard_normal((1, 1, 32))
    k = np.repeat(key, 50, axis=1)  # all keys equal -> uniform probabilities
    v = rng.standard_normal((1, 50, 32))
    out, p = accessible_attention(q, k, v, 0.3)
    assert np.allclose(p, 1.0 / 50)
    assert np.allclose(out, np.broadcast_to(v.mean(axis=1), (4, 32)))
    # one key aligned with the query and huge: the output is that token's value
    k2 = rng.standard_normal((1, 50, 32)) * 0.01
    k2[0, 17] = q[0] * 1000
    out2, p2 = accessible_attention(q[:1], k2, v, 1.0)
    assert p2[0, 17] > 1 - 1e-12 and np.allclose(out2[0], v[0, 17])
    # GQA: head h reads KV head h // (H_q / H_kv)
    k3 = rng.standard_normal((2, 20, 32))
    v3 = rng.standard_normal((2, 20, 32))
    out3, _ = accessible_attention(q, k3, v3, 0.2)
    for h in range(4):
        o1, _ = accessible_attention(q[h:h + 1], k3[h // 2:h // 2 + 1], v3[h // 2:h // 2 + 1], 0.2)
        assert np.allclose(out3[h], o1[0])


# -------------------------------------------------------------------------------- helpers
def _small_cfg(dtype="fp16", k_f=4, k_q=6, bits=4, hq=4, hkv=2, d=64, w=32, ctx_windows=16, extra=8):
    return OracleConfig(hq, hkv, d, dtype, w, bits, 32, k_f, k_q, (ctx_windows + extra) * w, aged_windows=2)


def _prefilled(cfg, rng, ctx_windows=16, scores=None):
    ctx = ctx_windows * cfg.window
    k = _rand_T(rng, (cfg.n_kv_heads, ctx, cfg.head_dim), cfg.dtype)
    v = _rand_T(rng, (cfg.n_kv_heads, ctx, cfg.head_dim), cfg.dtype)
    if scores is None:
        scores = rng.random(ctx_windows).astype(np.float32)
    u = UnitOracle(cfg)
    u.prefill_assign(k, v, scores)
    return u, k, v, scores


def _protected_cfg(dtype="fp16", k_f=3, k_q=4, sinks=2, recent=3, ctx_windows=16, extra=12):
    return OracleConfig(4, 2, 64, dtype, 32, 4, 32, k_f, k_q, (ctx_windows + extra) * 32, aged_windows=2,
                        sink_windows=sinks, recent_windows=recent)


# ------------------------------------------------------------- protected sink and recent regions
def test_sink_and_recent_windows_are_protected_and_outside_the_budget():
    """Cache partition (sink, recent, Full, Quantized, Evicted): the protected regions stay in full
    precision and never enter the candidate pool; candidates are the Full and Quantized windows plus the
    windows that have exited the recent region.  Checked against a model of the regions kept here: the
    sink prefix is windows 0..n_s-1; after every step the recent region is the n_r newest filled windows."""
    rng = np.random.default_rng(31)
    cfg = _protected_cfg()
    # lowest scores on the sink windows and on the newest prompt windows: unprotected they would be evicted
    scores = np.linspace(0.1, 1.0, 16).astype(np.float32)
    scores[:2] = 0.0
    scores[-3:] = 0.0
    u, k, v, _ = _prefilled(cfg, rng, scores=scores)
    c = u.tier_counts()
    assert c == {"open": 0, "aged": 3, "full": 3, "quant": 4, "evicted": 4, "sink": 2}
    assert list(np.flatnonzero(u.tier == TIER_SINK)) == [0, 1]
    assert list(np.flatnonzero(u.tier == TIER_AGED)) == [13, 14, 15]          # recent region of the prompt
    # the 11 unprotected windows were ranked on their own: 3 best Full, next 4 Quantized, 4 evicted
    assert list(np.flatnonzero(u.tier == TIER_FULL)) == [10, 11, 12]
    assert list(np.flatnonzero(u.tier == TIER_QUANT)) == [6, 7, 8, 9]
    assert list(np.flatnonzero(u.tier == TIER_EVICTED)) == [2, 3, 4, 5]
    # pages at prefill: ascending window index over everything that stays in full precision
    assert [int(u.fp_page[w]) for w in (0, 1, 10, 11, 12, 13, 14, 15)] == list(range(8))
    n_filled = 16
    for t in range(32 * 6):
        q = _rand_T(rng, (cfg.n_q_heads, cfg.head_dim), cfg.dtype)
        kn = _rand_T(rng, (cfg.n_kv_heads, cfg.head_dim), cfg.dtype)
        vn = _rand_T(rng, (cfg.n_kv_heads, cfg.head_dim), cfg.dtype)
        out, mass = u.decode_attn(q, kn, vn)
        assert abs(mass.sum() - cfg.n_q_heads) < 1e-9
        if (t + 1) % 32 == 0:
            n_filled += 1
        recent = set(range(n_filled - cfg.recent_windows, n_filled))
        cand = set(int(w) for w in u.ranked_candidates())
        assert cand.isdisjoint(recent) and cand.isdisjoint({0, 1})
        expect_cand = {w for w in range(n_filled) if u.tier[w] in (TIER_FULL, TIER_QUANT)} | \
                      {w for w in range(2, n_filled) if u.tier[w] == TIER_AGED and w not in recent}
        assert cand == expect_cand
        if t % 5 == 4:
            u.rebalance()
            c = u.tier_counts()
            assert c["sink"] == 2 and c["full"] <= cfg.fp_budget_windows and c["quant"] <= cfg.q_budget_windows
            assert all(u.tier[w] == TIER_AGED for w in recent)               # still protected
            assert c["aged"] == len(recent)                                   # everything that exited was routed
            fp_held = u.fp_page[u.fp_page >= 0]
            assert len(set(fp_held.tolist())) == len(fp_held) <= cfg.fp_pool_pages
            for w in range(u.n_windows):
                assert (u.fp_page[w] >= 0) == (u.tier[w] in (TIER_FULL, TIER_AGED, TIER_OPEN, TIER_SINK))
    assert u.stats["deletions"] > 4


def test_protected_regions_with_full_budget_equal_brute_force_attention():
    rng = np.random.default_rng(32)
    cfg = _protected_cfg("bf16", k_f=64, k_q=4, sinks=1, recent=2)
    u, k, v, _ = _prefilled(cfg, rng)
    assert u.tier_counts()["full"] == 13 and u.tier_counts()["sink"] == 1 and u.tier_counts()["aged"] == 2
    ks, vs = [k], [v]
    for t in range(70):
        q = _rand_T(rng, (cfg.n_q_heads, cfg.head_dim), "bf16")
        kn = _rand_T(rng, (cfg.n_kv_heads, cfg.head_dim), "bf16")
        vn = _rand_T(rng, (cfg.n_kv_heads, cfg.head_dim), "bf16")
        ks.append(kn[:, None]); vs.append(vn[:, None])
        out, mass = u.decode_attn(q, kn, vn)
        ref, p = _full_attention_reference(q, np.concatenate(ks, 1), np.concatenate(vs, 1), cfg.scale)
        assert np.array_equal(out, round_to_dtype(ref, "bf16"))
        if t % 7 == 6:
            u.rebalance()
            assert u.tier_counts()["evicted"] == 0 and u.tier_counts()["quant"] == 0


# ------------------------------------------------------------------- alternative ranking functions
def _rank_cfg(mode, param, k_f=3, k_q=4):
    return OracleConfig(4, 2, 64, "fp16", 32, 4, 32, k_f, k_q, 28 * 32, aged_windows=2, rank_mode=mode, rank_param=param)


@pytest.mark.parametrize("mode,param", [(1, 0.9), (2, 3.0)])
def test_ranking_variants_follow_their_recurrences(mode, param):
    """S_decay(t) = lambda S_decay(t - Omega) + u_t and S_p = (sum_r u_r^p)^(1/p): the oracle's scores are
    recomputed here in float64 from the per-step masses it returned, event by event."""
    rng = np.random.default_rng(41)
    cfg = _rank_cfg(mode, param, k_f=32, k_q=4)  # nothing is evicted: every window keeps a full history
    scores = rng.random(16).astype(np.float32)
    u, k, v, _ = _prefilled(cfg, rng, scores=scores)
    ref = np.zeros(cfg.max_windows)
    ref[:16] = scores
    acc = np.zeros(cfg.max_windows)
    for t in range(45):
        q = _rand_T(rng, (cfg.n_q_heads, cfg.head_dim), cfg.dtype)
        kn = _rand_T(rng, (cfg.n_kv_heads, cfg.head_dim), cfg.dtype)
        vn = _rand_T(rng, (cfg.n_kv_heads, cfg.head_dim), cfg.dtype)
        _, mass = u.decode_attn(q, kn, vn)
        acc += mass
        if t % 4 == 3:  # a routing event every 4 steps: u_t sums 4 steps
            u.rebalance()
            live = np.arange(u.n_windows)
            if mode == 1:
                ref[live] = param * ref[live] + acc[live]
            else:
                ref[live] = ref[live] + acc[live] ** param
            acc[:] = 0.0
            assert np.allclose(u.importance[: u.n_windows], ref[: u.n_windows], rtol=2e-6, atol=1e-12)
            assert np.all(u.event_mass == 0.0)
    if mode == 2:  # the stored quantity is S_p^p; S_p itself is its p-th root
        s_p = u.importance[: u.n_windows] ** (1.0 / param)
        assert np.allclose(s_p, ref[: u.n_windows] ** (1.0 / param), rtol=1e-6)


def test_decay_forgets_and_pnorm_prefers_peaks():
    """What distinguishes the variants: with equal total mass, the decayed score ranks the window attended
    recently above the one attended long ago, and the p-norm ranks a window attended in one burst above one
    attended evenly; the cumulative score cannot separate either pair."""
    for mode, param in ((0, 0.0), (1, 0.5), (2, 3.0)):
        cfg = _rank_cfg(mode, param, k_f=32, k_q=4)
        u = UnitOracle(cfg)
        u.n_windows = 4
        u.tier[:4] = TIER_FULL
        # per-event masses of windows 0..3 over 4 events: early, late, burst, even (total 4 each)
        events = np.array([[4, 0, 0, 0], [0, 0, 0, 4], [0, 4, 0, 0], [1, 1, 1, 1]], dtype=np.float64).T
        for e in events:
            if mode == 0:
                u.importance[:4] += e
            else:
                u.event_mass[:4] = e
                u.fold_event_mass()
        s = u.importance[:4]
        if mode == 0:
            assert s[0] == s[1] == s[2] == s[3] == 4.0
        elif mode == 1:
            assert s[1] > s[3] > s[0]            # late > even > early
            assert s[1] == 4.0 and s[0] == 4.0 * 0.5 ** 3
        else:
            assert s[0] == s[1] == s[2] == 64.0 and s[3] == 4.0   # one burst: 4^3; even: 4 x 1^3


def test_key_norm_ranking_keeps_the_windows_with_the_smallest_key_norms():
    """Key-norm equation: score = minus the mean L2 norm of the window's keys; lower norms are retained first.
    Checked against numpy.linalg.norm on the prompt and on the windows that fill during decoding."""
    rng = np.random.default_rng(43)
    cfg = _rank_cfg(3, 0.0, k_f=3, k_q=4)
    ctx = 16 * 32
    scale = np.repeat(np.linspace(0.5, 2.0, 16)[rng.permutation(16)], 32)  # every window its own key magnitude
    k = round_to_dtype(rng.standard_normal((2, ctx, 64)) * scale[None, :, None], "fp16")
    v = _rand_T(rng, (2, ctx, 64), "fp16")
    u = UnitOracle(cfg)
    u.prefill_assign(k, v, np.zeros(16, dtype=np.float32))            # the given scores are ignored
    norms = np.linalg.norm(k.reshape(2, 16, 32, 64), axis=-1).mean(axis=(0, 2))
    assert np.allclose(u.importance[:16], -norms, rtol=1e-12)
    order = np.argsort(norms, kind="stable")
    assert set(np.flatnonzero(u.tier[:16] == TIER_FULL)) == set(order[:3])
    assert set(np.flatnonzero(u.tier[:16] == TIER_QUANT)) == set(order[3:7])
    assert set(np.flatnonzero(u.tier[:16] == TIER_EVICTED)) == set(order[7:])
    new_k = []
    for t in range(64):
        kn = round_to_dtype(rng.standard_normal((2, 64)) * (0.1 if t < 32 else 5.0), "fp16")
        new_k.append(kn)
        u.decode_attn(_rand_T(rng, (4, 64), "fp16"), kn, _rand_T(rng, (2, 64), "fp16"))
    nk = np.stack(new_k, axis=1)                                       # [2, 64, 64]
    n16, n17 = (np.linalg.norm(nk[:, a:a + 32], axis=-1).mean() for a in (0, 32))
    assert np.isclose(u.importance[16], -n16, rtol=1e-12) and np.isclose(u.importance[17], -n17, rtol=1e-12)
    u.rebalance()
    assert u.tier[16] == TIER_FULL and u.tier[17] == TIER_EVICTED      # tiny keys are kept, huge keys go first
    assert np.isclose(u.importance[16], -n16, rtol=1e-12)             # attention mass never entered the score


def test_one_way_policy_never_promotes():
    """Promotion ablation: Full -> Quantized -> Evicted only.  Against a brute-force statement of the reading
    (Full tier = best K_f candidates that are not Quantized; Quantized tier = best K_q of the rest) on random
    scores, and against the bidirectional policy on the same scores."""
    rng = np.random.default_rng(44)
    cfg1 = OracleConfig(4, 2, 64, "fp16", 32, 4, 32, 3, 5, 40 * 32, aged_windows=2, one_way=True)
    cfg2 = OracleConfig(4, 2, 64, "fp16", 32, 4, 32, 3, 5, 40 * 32, aged_windows=2)
    a, k, v, s0 = _prefilled(cfg1, rng, ctx_windows=20)
    b = UnitOracle(cfg2)
    b.prefill_assign(k, v, s0)
    assert np.array_equal(a.tier, b.tier)                       # nothing is Quantized before the first event
    differed = False
    for it in range(30):
        scores = rng.random(a.n_windows)
        a.importance[: a.n_windows] = scores
        b.importance[: b.n_windows] = scores
        t0 = a.tier[: a.n_windows].copy()
        cand = [w for w in range(a.n_windows) if t0[w] in (TIER_FULL, TIER_QUANT, TIER_AGED)]
        order = sorted(cand, key=lambda w: (-np.float32(scores[w]), w))
        exp_f = [w for w in order if t0[w] != TIER_QUANT][:3]
        rest = [w for w in order if w not in exp_f]
        exp_q, exp_e = rest[:5], rest[5:]
        a.rebalance()
        b.rebalance()
        assert set(np.flatnonzero(a.tier[: a.n_windows] == TIER_FULL)) == set(exp_f)
        assert set(np.flatnonzero(a.tier[: a.n_windows] == TIER_QUANT)) == set(exp_q)
        assert all(a.tier[w] == TIER_EVICTED for w in exp_e)
        assert all(t0[w] != TIER_QUANT for w in exp_f)          # no window came back from the Quantized tier
        differed = differed or not np.array_equal(a.tier[: a.n_windows], b.tier[: b.n_windows])
        if not np.array_equal(a.tier[: a.n_windows], b.tier[: b.n_windows]):
            b.tier[:] = a.tier; b.ledger_flag[:] = a.ledger_flag      # keep the two comparable (states only)
            break
    assert a.stats["promotions"] == 0
    assert differed                                              # the bidirectional policy does promote here


# ------------------------------------------------------------------------------------ diagnostics
def test_tier_mass_share_and_selection_churn_on_a_hand_made_state():
    """Tier-mass equation and selection-churn equation of the observation appendix on a state small enough to
    do by hand: scores 1..8 on eight windows in tiers S F F Q Q E A(recent) O(pen)."""
    from oracle import retained_windows, selection_churn, tier_mass_share
    u = UnitOracle(_protected_cfg())
    u.n_windows = 8
    u.tier[:8] = [TIER_SINK, TIER_FULL, TIER_FULL, TIER_QUANT, TIER_QUANT, TIER_EVICTED, TIER_AGED, TIER_OPEN]
    u.importance[:8] = [1, 2, 3, 4, 5, 6, 7, 8]
    mu = tier_mass_share(u)
    assert mu == {"full": 5 / 36, "quant": 9 / 36, "evicted": 6 / 36, "local": 16 / 36}
    assert abs(sum(mu.values()) - 1.0) < 1e-15
    before = retained_windows(u)
    assert before == {1, 2, 3, 4}
    u.tier[:8] = [TIER_SINK, TIER_FULL, TIER_QUANT, TIER_EVICTED, TIER_QUANT, TIER_EVICTED, TIER_FULL, TIER_OPEN]
    after = retained_windows(u)
    assert after == {1, 2, 4, 6}
    assert selection_churn(before, after) == 1.0 - 3 / 5      # intersection {1,2,4}, union {1,2,3,4,6}
    assert selection_churn(before, before) == 0.0 and selection_churn(set(), set()) == 0.0
    assert selection_churn({1}, {2}) == 1.0


def test_no_protected_regions_is_the_default():
    rng = np.random.default_rng(33)
    a, k, v, s = _prefilled(_small_cfg(), rng)
    b = UnitOracle(_protected_cfg(k_f=4, k_q=6, sinks=0, recent=0, extra=8))
    b.prefill_assign(k, v, s)
    assert np.array_equal(a.tier, b.tier) and np.array_equal(a.fp_page, b.fp_page) and np.array_equal(a.q_page, b.q_page)


# ------------------------------------------------- (a) everything in full precision = full attention
@pytest.mark.parametrize("dtype", ["fp16", "bf16"])
def test_full_budget_equals_brute_force_attention(dtype):
    rng = np.random.default_rng(12)
    cfg = _small_cfg(dtype, k_f=64, k_q=4)
    u, k, v, _ = _prefilled(cfg, rng)
    assert u.tier_counts()["full"] == 16 and u.tier_counts()["quant"] == 0
    ks, vs = [k], [v]
    for t in range(40):
        q = _rand_T(rng, (cfg.n_q_heads, cfg.head_dim), dtype)
        kn = _rand_T(rng, (cfg.n_kv_heads, cfg.head_dim), dtype)
        vn = _rand_T(rng, (cfg.n_kv_heads, cfg.head_dim), dtype)
        ks.append(kn[:, None]); vs.append(vn[:, None])
        out, mass = u.decode_attn(q, kn, vn)
        ref, p = _full_attention_reference(q, np.concatenate(ks, 1), np.concatenate(vs, 1), cfg.scale)
        assert np.array_equal(out, round_to_dtype(ref, dtype))
        n_tok = p.shape[1]
        ref_mass = np.add.reduceat(p.sum(0), np.arange(0, n_tok, cfg.window))
        assert np.allclose(mass[: len(ref_mass)], ref_mass, rtol=1e-12, atol=1e-15)
        if t % 8 == 7:
            u.rebalance()
            assert u.tier_counts()["evicted"] == 0 and u.tier_counts()["quant"] == 0


# --------------------------------------------------------- (c) mass conservation, (d) budgets
def test_mass_sums_to_heads_times_steps_and_budgets_hold():
    wl = wlmod.config(0)
    k, v = wlmod.gen_prompt_kv(wl, 0)
    k = k.double().numpy(); v = v.double().numpy()
    cfg = OracleConfig(wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.dtype, wl.window, wl.quant_bits,
                       wl.group_size, wl.fp_budget_windows, wl.q_budget_windows, wl.max_context)
    scores = wlmod.place_planted(wlmod.synthetic_window_scores(wl, 0), wlmod.planted_windows(wl, 0),
                                 wl.fp_budget_windows, wl.q_budget_windows)
    u = UnitOracle(cfg)
    u.prefill_assign(k, v, scores.numpy())
    base = u.importance.sum()
    assert u.tier_counts() == {"open": 0, "aged": 0, "full": 8, "quant": 16, "evicted": 40, "sink": 0}
    q_all = wlmod.gen_queries(wl, 0, torch.from_numpy(k), scores).double().numpy()
    kn, vn = wlmod.gen_new_kv(wl, 0)
    evicted_before = set()
    for t in range(wl.steps):
        out, mass = u.decode_attn(q_all[t], kn[t].double().numpy(), vn[t].double().numpy())
        assert abs(mass.sum() - cfg.n_q_heads) < 1e-9
        assert abs(u.importance.sum() - base - cfg.n_q_heads * (t + 1)) < 1e-7
        u.rebalance()
        c = u.tier_counts()
        assert c["full"] <= cfg.fp_budget_windows and c["quant"] <= cfg.q_budget_windows
        assert c["aged"] == 0
        ev = set(np.flatnonzero(u.tier == TIER_EVICTED).tolist())
        assert evicted_before <= ev  # evicted windows never return
        evicted_before = ev
        # physical pools: no page held twice, occupancy within the pool
        fp_held = u.fp_page[u.fp_page >= 0]
        q_held = u.q_page[u.q_page >= 0]
        assert len(set(fp_held.tolist())) == len(fp_held) <= cfg.fp_pool_pages
        assert len(set(q_held.tolist())) == len(q_held) <= cfg.q_pool_pages
        for w in range(u.n_windows):
            assert (u.fp_page[w] >= 0) == (u.tier[w] in (TIER_FULL, TIER_AGED, TIER_OPEN))
            assert (u.q_page[w] >= 0) == (u.ledger_flag[w] != LEDGER_NONE)
            assert (u.tier[w] == TIER_QUANT) == (u.ledger_flag[w] == LEDGER_ACTIVE)
    # the drifting queries force recoveries from the quantized tier
    assert u.stats["promotions"] > 0 and u.stats["deletions"] > 40


# --------------------------------------------------------------------------------- routing
def test_routing_matches_brute_force_sort():
    rng = np.random.default_rng(13)
    for trial in range(20):
        cfg = _small_cfg(k_f=int(rng.integers(1, 6)), k_q=int(rng.integers(1, 8)))
        scores = rng.integers(0, 6, 16).astype(np.float32)  # many ties
        u, *_ = _prefilled(cfg, rng, scores=scores)
        ranked = sorted(range(16), key=lambda w: (-float(scores[w]), w))
        exp_f = set(ranked[: cfg.fp_budget_windows])
        exp_q = set(ranked[cfg.fp_budget_windows: cfg.fp_budget_windows + cfg.q_budget_windows])
        assert set(np.flatnonzero(u.tier == TIER_FULL).tolist()) == exp_f
        assert set(np.flatnonzero(u.tier == TIER_QUANT).tolist()) == exp_q
        assert set(np.flatnonzero(u.tier == TIER_EVICTED).tolist()) == set(range(16)) - exp_f - exp_q
        # prefill page order: ascending window index takes ascending page ids
        assert [int(u.fp_page[w]) for w in sorted(exp_f)] == list(range(len(exp_f)))
        assert [int(u.q_page[w]) for w in sorted(exp_q)] == list(range(len(exp_q)))


def test_rebalance_is_idempotent_and_small_pools_keep_everything_full():
    rng = np.random.default_rng(14)
    cfg = _small_cfg(k_f=3, k_q=5)
    u, *_ = _prefilled(cfg, rng)
    snap = (u.tier.copy(), u.fp_page.copy(), u.q_page.copy(), u.ledger_flag.copy(), dict(u.stats))
    u.rebalance()
    assert np.array_equal(snap[0], u.tier) and np.array_equal(snap[1], u.fp_page)
    assert np.array_equal(snap[2], u.q_page) and np.array_equal(snap[3], u.ledger_flag)
    assert snap[4] == u.stats
    cfg2 = _small_cfg(k_f=20, k_q=5)
    u2, *_ = _prefilled(cfg2, rng)
    assert u2.tier_counts()["full"] == 16


def test_scores_are_ranked_in_float32():
    """Two float64 scores that collapse to the same float32 are a tie: the lower index wins."""
    rng = np.random.default_rng(15)
    cfg = _small_cfg(k_f=1, k_q=1)
    u, *_ = _prefilled(cfg, rng, scores=np.zeros(16, np.float32))
    u.importance[:] = 0.0
    u.importance[5] = 1.0
    u.importance[9] = 1.0 + 1e-12
    # only windows 0 (F) and 1 (Q) are still candidates; give them the colliding scores instead
    u.importance[0] = 1.0
    u.importance[1] = 1.0 + 1e-12
    u.rebalance()
    assert u.tier[0] == TIER_FULL and u.tier[1] == TIER_QUANT


# ---------------------------------------------------------------------------------- ledger
def _ledger_hash(e):
    m = hashlib.sha256()
    for key in ("k_codes", "k_s", "k_z", "v_codes", "v_s", "v_z"):
        m.update(np.ascontiguousarray(e[key]).tobytes())
    return m.hexdigest()


def test_write_once_ledger_and_promotion_invariance():
    rng = np.random.default_rng(16)
    cfg = _small_cfg("bf16", k_f=2, k_q=3, bits=2)
    scores = np.arange(16, 0, -1).astype(np.float32)  # window 0 highest
    u, k, v, _ = _prefilled(cfg, rng, scores=scores)
    assert list(np.flatnonzero(u.tier == TIER_FULL)) == [0, 1]
    assert list(np.flatnonzero(u.tier == TIER_QUANT)) == [2, 3, 4]
    h2 = _ledger_hash(u.ledger[2])
    q = _rand_T(rng, (cfg.n_q_heads, cfg.head_dim), "bf16")
    u.decode_attn(q)  # fixed-context step, window 2 read from its codes
    u.importance[:16] = scores  # undo the score change, then lift window 2 to the top
    u.importance[2] = 100.0
    u.rebalance()
    assert u.tier[2] == TIER_FULL and u.ledger_flag[2] == LEDGER_DORMANT and u.q_page[2] >= 0
    assert u.tier[1] == TIER_QUANT and u.ledger_flag[1] == LEDGER_ACTIVE  # window 1 demoted, quantized now
    assert u.stats["promotions"] == 1 and u.stats["quantizations"] == 4
    # the promoted copy is the dequantized approximation, not the original values
    assert not np.array_equal(u.fp[2][0], k[:, 64:96])
    assert _ledger_hash(u.ledger[2]) == h2
    # demote window 2 again: reactivation, codes untouched, no new quantization
    u.importance[2] = 13.5  # between windows 1 and 3: back into the quantized tier
    u.importance[1] = 100.0
    u.rebalance()
    assert u.tier[2] == TIER_QUANT and u.ledger_flag[2] == LEDGER_ACTIVE
    assert u.stats["reactivations"] == 1 and u.stats["quantizations"] == 4
    assert _ledger_hash(u.ledger[2]) == h2
    assert u.tier[1] == TIER_FULL and u.ledger_flag[1] == LEDGER_DORMANT  # back as its own approximation
    # promotion invariance: swap windows 1 and 2 between the tiers once more.  Both already are
    # approximations, so no value changes and attention must be bit-identical.
    out_a, mass_a = u.decode_attn(q)
    u.importance -= mass_a
    u.importance[2] = 200.0
    u.importance[1] = 13.5
    u.rebalance()
    assert u.tier[2] == TIER_FULL and u.tier[1] == TIER_QUANT and u.tier[0] == TIER_FULL
    assert u.stats["quantizations"] == 4 and u.stats["reactivations"] == 2 and u.stats["promotions"] == 3
    out_b, mass_b = u.decode_attn(q)
    assert np.array_equal(out_a, out_b) and np.array_equal(mass_a, mass_b)


def test_eviction_deletes_ledger_and_is_permanent():
    rng = np.random.default_rng(17)
    cfg = _small_cfg(k_f=2, k_q=2)
    scores = np.arange(16, 0, -1).astype(np.float32)
    u, *_ = _prefilled(cfg, rng, scores=scores)
    assert u.tier_counts()["evicted"] == 12
    # fill one window by appending: it ages and must displace the weakest quantized window
    for t in range(cfg.window):
        u.decode_attn(_rand_T(rng, (cfg.n_q_heads, cfg.head_dim), cfg.dtype),
                      _rand_T(rng, (cfg.n_kv_heads, cfg.head_dim), cfg.dtype),
                      _rand_T(rng, (cfg.n_kv_heads, cfg.head_dim), cfg.dtype))
    assert u.tier[16] == TIER_AGED
    u.importance[16] = 1e6
    victim = 3  # lowest-ranked retained window
    page = u.q_page[victim]
    u.rebalance()
    assert u.tier[16] == TIER_FULL
    assert u.tier[victim] == TIER_EVICTED and u.ledger_flag[victim] == LEDGER_NONE
    assert victim not in u.ledger and u.q_owner[page] != victim
    u.importance[victim] = 1e9  # an evicted window is not a candidate any more, whatever its score
    u.rebalance()
    assert u.tier[victim] == TIER_EVICTED


def test_open_window_is_attended_and_ages():
    rng = np.random.default_rng(18)
    cfg = _small_cfg(k_f=2, k_q=2)
    u, *_ = _prefilled(cfg, rng)
    q = _rand_T(rng, (cfg.n_q_heads, cfg.head_dim), cfg.dtype)
    kn = _rand_T(rng, (cfg.n_kv_heads, cfg.head_dim), cfg.dtype)
    vn = _rand_T(rng, (cfg.n_kv_heads, cfg.head_dim), cfg.dtype)
    out, mass = u.decode_attn(q, kn, vn)
    assert u.tier[16] == TIER_OPEN and u.open_fill == 1 and mass[16] > 0
    assert u.fp_page[16] == 2  # lowest free full-precision page after pages 0 and 1
    assert sum(a[3] for a in u.accessible()) == 4 * cfg.window + 1


# ------------------------------------------------------------------------------ capacities
def test_tier_capacities_closed_form():
    cfg = OracleConfig(32, 8, 128, "bf16", 32, 4, 32, 1, 1, 4096)
    m_f, m_q = window_bytes(cfg)
    assert (m_f, m_q) == (131072, 40960)
    assert tier_capacities(100 * m_f, 0.0, m_f, m_q) == (100, 0)
    assert tier_capacities(100 * m_f, 1.0, m_f, m_q) == (0, 320)
    k_f, k_q = tier_capacities(10_000_000, 0.7, m_f, m_q)
    assert (k_f, k_q) == (22, 170)
    assert k_f * m_f <= 0.3 * 10_000_000 < (k_f + 1) * m_f
    assert k_q * m_q <= 0.7 * 10_000_000 < (k_q + 1) * m_q


# ------------------------------------------------------------------------------- pre-RoPE keys
def test_pre_rope_cache_with_full_budget_equals_attention_over_rotated_keys():
    """With every window in the Full tier the cache must give plain attention over the keys rotated for their
    absolute positions (complex multiplication of the half-split pairs, here in float64): the stored keys stay
    pre-RoPE, positions count from the start of the prompt through the appended tokens, values are untouched.
    The rounding of the rotated keys to the execution datatype bounds the difference."""
    from dataclasses import replace as dc_replace

    dtype = "fp16"
    rng = np.random.default_rng(21)
    cfg = dc_replace(_small_cfg(dtype, k_f=64, k_q=4), rope_base=10000.0)
    u, k, v, _ = _prefilled(cfg, rng)
    ks, vs = [k], [v]
    d = cfg.head_dim
    freq = 10000.0 ** (-2.0 * np.arange(d // 2) / d)
    for t in range(12):
        q = _rand_T(rng, (cfg.n_q_heads, d), dtype)
        kn = _rand_T(rng, (cfg.n_kv_heads, d), dtype)
        vn = _rand_T(rng, (cfg.n_kv_heads, d), dtype)
        ks.append(kn[:, None]); vs.append(vn[:, None])
        out, mass = u.decode_attn(q, kn, vn)
        kk = np.concatenate(ks, 1)
        z = (kk[..., : d // 2] + 1j * kk[..., d // 2 :]) * np.exp(1j * np.outer(np.arange(kk.shape[1]), freq))
        ref, p = _full_attention_reference(q, np.concatenate([z.real, z.imag], -1), np.concatenate(vs, 1), cfg.scale)
        assert np.abs(out - ref).max() < 2e-2 and np.abs(out - ref).mean() < 2e-3
        assert np.isclose(mass.sum(), cfg.n_q_heads, rtol=1e-12)
        # the stored keys are still the ones that were handed in
        assert np.array_equal(u.fp[0][0], k[:, : cfg.window])
    # and the rotation matters: without it the same cache state gives a different answer
    u2 = UnitOracle(dc_replace(cfg, rope_base=0.0))
    u2.prefill_assign(k, v, np.zeros(k.shape[1] // cfg.window))
    o2, _ = u2.decode_attn(q)
    o1, _ = u.decode_attn(q)
    assert np.abs(o1 - o2).max() > 1e-2


# ------------------------------------------------------------------------------ hand-worked pins
def test_page_ids_at_routing_events_follow_the_stated_rule_on_a_hand_worked_run():
    """Page hand-out rule of a routing event, worked by hand: all releases of the event first, then the windows
    that need a page take the free ids in ascending order, in ascending window index (full-precision pages for
    the windows entering the Full tier, quantized pages for first demotions); a promoted window keeps its
    quantized page (dormant ledger), a re-demoted window gets no new one."""
    rng = np.random.default_rng(41)
    cfg = _small_cfg(k_f=2, k_q=2, ctx_windows=6, extra=4)
    u, *_ = _prefilled(cfg, rng, ctx_windows=6, scores=np.array([6, 5, 4, 3, 2, 1], dtype=np.float32))
    # prefill: Full {0, 1} -> full-precision pages 0, 1; Quantized {2, 3} -> quantized pages 0, 1; 4, 5 evicted
    assert u.fp_page[:6].tolist() == [0, 1, -1, -1, -1, -1] and u.q_page[:6].tolist() == [-1, -1, 0, 1, -1, -1]
    # event 1: ranks 2, 3, 1, 0 -> Full {2, 3}, Quantized {0, 1}.  Releases: windows 0 and 1 give up full-precision
    # pages 0 and 1.  Then window 2 takes page 0 and window 3 page 1 (ascending window, ascending free id); the first
    # demotions 0 and 1 take the free quantized pages 2 and 3 (pages 0, 1 stay with the promoted windows' codes).
    u.importance[:4] = [1.0, 2.0, 10.0, 9.0]
    u.rebalance()
    assert u.tier[:4].tolist() == [TIER_QUANT, TIER_QUANT, TIER_FULL, TIER_FULL]
    assert u.fp_page[:4].tolist() == [-1, -1, 0, 1] and u.q_page[:4].tolist() == [2, 3, 0, 1]
    assert u.ledger_flag[:4].tolist() == [LEDGER_ACTIVE, LEDGER_ACTIVE, LEDGER_DORMANT, LEDGER_DORMANT]
    assert (u.stats["promotions"], u.stats["quantizations"], u.stats["reactivations"]) == (2, 4, 0)
    # event 2: ranks 1, 3, 0, 2 -> Full {1, 3}, Quantized {0, 2}.  Window 2 is demoted again: its codes are reused
    # (no new quantized page), its full-precision page 0 is released and goes to window 1, the only window that
    # needs one.
    u.importance[:4] = [8.0, 10.0, 1.0, 9.0]
    u.rebalance()
    assert u.tier[:4].tolist() == [TIER_QUANT, TIER_FULL, TIER_QUANT, TIER_FULL]
    assert u.fp_page[:4].tolist() == [-1, 0, -1, 1] and u.q_page[:4].tolist() == [2, 3, 0, 1]
    assert u.ledger_flag[:4].tolist() == [LEDGER_ACTIVE, LEDGER_DORMANT, LEDGER_ACTIVE, LEDGER_DORMANT]
    assert (u.stats["promotions"], u.stats["quantizations"], u.stats["reactivations"]) == (3, 4, 1)
    assert u.fp_owner[:2].tolist() == [1, 3] and u.q_owner[:4].tolist() == [2, 3, 0, 1]


def test_decayed_score_is_folded_with_each_float32_operation_rounded_on_its_own():
    """S <- lambda S + u in float32, product rounded, then sum rounded (worked by hand): lambda = 0.75,
    S = 1 + 3 ulp (ulp = 2^-23), u = 2^-26.  The exact product 0.75 + 4.5 * 2^-24 is a tie and rounds to the even
    0.75 + 4 * 2^-24; adding u gives 0.75 + 4.25 * 2^-24, which rounds to 0.75 + 4 * 2^-24.  A fused
    multiply-add would see 0.75 + 4.75 * 2^-24 and return 0.75 + 5 * 2^-24."""
    rng = np.random.default_rng(42)
    cfg = OracleConfig(4, 2, 64, "fp16", 32, 4, 32, 2, 2, 10 * 32, aged_windows=2, rank_mode=1, rank_param=0.75)
    u, *_ = _prefilled(cfg, rng, ctx_windows=6, scores=np.array([6, 5, 4, 3, 2, 1], dtype=np.float32))
    u.importance[0] = 1.0 + 3 * 2.0 ** -23
    u.event_mass[0] = 2.0 ** -26
    u.fold_event_mass()
    assert u.importance[0] == 0.75 + 4 * 2.0 ** -24
    assert u.importance[0] != 0.75 + 5 * 2.0 ** -24 and u.event_mass[0] == 0.0
