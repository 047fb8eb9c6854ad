"""Three-tier window cache of one (sequence, layer): state, decode step, routing (oracle, test infrastructure).

Paper basis:
  * cache partition (sink, recent, Full, Quantized, Evicted) and the three window
    states: Methodology, "Recoverable Cache Hierarchy" and Preliminaries;
  * cumulative window score: Eq. 1 (cumulative window scoring);
  * candidate pool, TopK_{K_f} / TopK_{K_q} partition, transitions
    Full <-> Quantized -> Evicted: "Dynamic Routing and Recovery" and Algorithm 1;
  * write-once ledger (quantize on the first demotion only, dormant on
    promotion, reactivated on a later demotion, deleted on eviction):
    "Migration-Stable Quantization" and Algorithm 1;
  * alternative ranking functions (exponentially decayed attention, attention
    p-norm): the ranking-function appendix, Eqs. for u_t(w), S_decay and S_p;
  * capacities K_f, K_q from a byte budget: the tier-capacity equation of
    "Byte-Constrained Tier Allocation"; per-window byte costs: the memory
    accounting appendix.

Readings taken where the paper is silent:
  * the window size W and the routing interval are separate parameters; routing
    happens when `rebalance()` is called;
  * the protected regions are window-granular: the sink prefix is the first
    `sink_windows` windows of the prompt, the recent region is the open window
    being filled plus the `recent_windows` most recently filled windows; both stay
    in full precision, are attended to, are never candidates and do not count
    against K_f (the budget constraint reserves B_sink and B_local separately);
    a filled window that is no longer among the `recent_windows` newest has exited
    the recent region and waits ("aged") for the next routing event;
  * the score is the raw sum over query heads (Eq. 1 without its constant
    1/H_q, which does not change any ranking) and is accumulated at every decode
    step, as the sum over tau in Eq. 1 states;
  * ranking compares scores as float32, higher first, lower window index first
    among equals;
  * K_q bounds the windows whose state is Quantized; the codes of a promoted
    window (dormant ledger entry) stay resident in additional physical pages;
  * physical pages are handed out deterministically: after all releases of a
    routing event, windows that need a page take the free page ids in ascending
    order, in ascending window index; a newly opened window takes the lowest
    free full-precision page.

Ranking variants (rank_mode 1, 2): the mass a window receives is collected in an
event accumulator u (raw sum over heads, like the score) and folded into the score at
every routing event after prefill, for every window that is still stored:
    decayed:  S <- RN32(RN32(lambda * S) + u)
    p-norm:   P <- RN32(P + u^p), u^p by p-1 float32 multiplications; windows are ranked
              by P, which orders them as S_p = P^(1/p) does
in float32 with every operation rounded separately, so that the ranking -- an integer
decision taken on floating point -- is taken on the same numbers by any implementation.
The prefill scores initialise S (or P) directly.

Key-norm ranking (rank_mode 3; ranking-function appendix, key-norm equation): the score of a window is
minus the mean L2 norm of its cached keys -- attention-free and fixed once the window is complete.  With several
KV heads the norm is taken per head and averaged over heads and tokens (the paper writes one key vector per
token and layer and does not say how heads combine).  Prefill scores are ignored; attention mass is still
collected in the event accumulator but never enters the score.

One-way policy (promotion ablation appendix: Full -> Quantized -> Evicted, "quantized windows may subsequently
be evicted but cannot return to the full tier", same capacities and ranking): the paper gives no algorithm for
it; the reading taken is Algorithm 1 with the Full tier drawn from the candidates that are not Quantized --
F' = TopK_{K_f} of the ranked candidates whose state is not Quantized, Q' = TopK_{K_q} of the ranked remainder,
E' = the rest.

Pre-RoPE keys (rope_base > 0): see rope.py.

Parity unpinned: the prefill window scores are an input here (the paper only says
that prompt attention initialises them), so their definition is pinned by nothing
beyond Eq. 1's form.  The page-id assignment order above is this build's own rule
(the paper never speaks of pages): the tests pin this file to the rule as stated, on
a run worked by hand, but nothing in the paper fixes the rule itself.
"""

from dataclasses import dataclass

import numpy as np

from .attention import accessible_attention
from .numerics import round_to_dtype
from .quantizer import dequantize_window, quantize_window
from .rope import apply_rope

TIER_NONE, TIER_OPEN, TIER_AGED, TIER_FULL, TIER_QUANT, TIER_EVICTED, TIER_SINK = 0, 1, 2, 3, 4, 5, 6
LEDGER_NONE, LEDGER_ACTIVE, LEDGER_DORMANT = 0, 1, 2

_ELEM_BYTES = {"fp16": 2, "bf16": 2}


@dataclass
class OracleConfig:
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    dtype: str  # "fp16" | "bf16"
    window: int  # W tokens
    quant_bits: int  # 2 | 4
    group_size: int  # g
    fp_budget_windows: int  # K_f
    q_budget_windows: int  # K_q
    max_context: int
    aged_windows: int = 2  # filled windows that may wait for the next routing event
    softmax_scale: float = 0.0  # 0 => 1/sqrt(head_dim)
    sink_windows: int = 0  # protected sink prefix, in windows
    rank_mode: int = 0  # 0 cumulative attention (Eq. 1), 1 exponentially decayed, 2 attention p-norm, 3 key norm
    rank_param: float = 0.0  # lambda of the decayed score, p of the p-norm (integer >= 2)
    one_way: bool = False  # no promotion: a Quantized window never returns to the Full tier
    recent_windows: int = 0  # filled windows kept in the protected recent region
    rope_base: float = 0.0  # > 0: stored keys are pre-RoPE and are rotated when attention reads them

    @property
    def scale(self):
        return self.softmax_scale if self.softmax_scale > 0 else 1.0 / np.sqrt(self.head_dim)

    @property
    def max_windows(self):
        return self.max_context // self.window

    @property
    def fp_pool_pages(self):
        return self.fp_budget_windows + self.sink_windows + self.recent_windows + self.aged_windows + 1

    @property
    def q_pool_pages(self):
        return self.q_budget_windows + self.fp_budget_windows


def window_bytes(cfg):
    """(M_f, M_q): bytes of one full-precision and one quantized window, all KV heads, K and V.

    Memory accounting appendix: M_Q holds the packed codes and M_quant-meta the
    scales and offsets; one (scale, zero) pair in the execution datatype per group.
    """
    c = _ELEM_BYTES[cfg.dtype]
    w, d, g, b, h = cfg.window, cfg.head_dim, cfg.group_size, cfg.quant_bits, cfg.n_kv_heads
    m_f = 2 * h * w * d * c
    codes = 2 * w * d * b // 8
    k_params = (w // g) * d * 2 * c
    v_params = w * (d // g) * 2 * c
    m_q = h * (codes + k_params + v_params)
    return m_f, m_q


def tier_capacities(hist_bytes, q_frac, m_f, m_q):
    """K_f = floor((1-q) B_hist / M_f), K_q = floor(q B_hist / M_q) (tier-capacity equation)."""
    k_f = int(np.floor((1.0 - q_frac) * hist_bytes / m_f))
    k_q = int(np.floor(q_frac * hist_bytes / m_q))
    return k_f, k_q


class UnitOracle:
    """The cache of one (sequence, layer)."""

    def __init__(self, cfg):
        self.cfg = cfg
        n = cfg.max_windows
        self.n_windows = 0  # windows created so far (chronological index)
        self.open_fill = 0  # tokens in the open window
        self.tier = np.zeros(n, dtype=np.uint8)
        self.ledger_flag = np.zeros(n, dtype=np.uint8)
        self.fp_page = np.full(n, -1, dtype=np.int32)
        self.q_page = np.full(n, -1, dtype=np.int32)
        self.importance = np.zeros(n, dtype=np.float64)
        self.event_mass = np.zeros(n, dtype=np.float64)  # u: mass since the last routing event (rank_mode 1, 2)
        self.fp = {}  # window -> (k, v) [H_kv, W, d] float64 in the execution datatype
        self.ledger = {}  # window -> dict of codes and params
        self.fp_owner = np.full(cfg.fp_pool_pages, -1, dtype=np.int32)
        self.q_owner = np.full(cfg.q_pool_pages, -1, dtype=np.int32)
        self.stats = {"promotions": 0, "quantizations": 0, "reactivations": 0, "deletions": 0, "steps": 0}

    # ---------------------------------------------------------------- pages
    @staticmethod
    def _take_lowest_free(owner, w):
        free = np.flatnonzero(owner < 0)
        if free.size == 0:
            raise RuntimeError("page pool exhausted")
        owner[free[0]] = w
        return int(free[0])

    # -------------------------------------------------------------- prefill
    def prefill_assign(self, k, v, window_scores):
        """Prefill initialisation (Methodology: prompt attention initialises the window scores and
        the first tier assignment).  k, v: [H_kv, ctx, d]; window_scores: [ctx / W], raw sums over
        heads.  Every prompt window becomes a routing candidate, then Algorithm 1 runs once."""
        cfg = self.cfg
        h, ctx, d = k.shape
        assert ctx % cfg.window == 0 and self.n_windows == 0
        n = ctx // cfg.window
        assert n <= cfg.max_windows
        for w in range(n):
            sl = slice(w * cfg.window, (w + 1) * cfg.window)
            self.fp[w] = (np.array(k[:, sl, :], dtype=np.float64), np.array(v[:, sl, :], dtype=np.float64))
            self.tier[w] = TIER_SINK if w < cfg.sink_windows else TIER_AGED
            self.importance[w] = self.key_norm_score(self.fp[w][0]) if cfg.rank_mode == 3 else float(window_scores[w])
        self.n_windows = n
        self.rebalance(prefill=True)

    @staticmethod
    def key_norm_score(k):
        """Key-norm equation: minus the mean over tokens (and KV heads) of the L2 norm of the keys; k [H_kv, W, d]."""
        return -float(np.sqrt((k * k).sum(axis=-1)).mean())

    # --------------------------------------------------------------- append
    def _append(self, k_new, v_new):
        """Newly generated states enter the protected recent region (Methodology, end of the scoring
        subsection): here the open window, which becomes an aged candidate once it holds W tokens."""
        cfg = self.cfg
        open_w = np.flatnonzero(self.tier[: self.n_windows] == TIER_OPEN)
        if open_w.size == 0:
            w = self.n_windows
            if w >= cfg.max_windows:
                raise RuntimeError("context exceeds max_context")
            self.n_windows += 1
            self.tier[w] = TIER_OPEN
            self.fp_page[w] = self._take_lowest_free(self.fp_owner, w)
            z = np.zeros((cfg.n_kv_heads, cfg.window, cfg.head_dim))
            self.fp[w] = (z.copy(), z.copy())
            self.open_fill = 0
        else:
            w = int(open_w[0])
        self.fp[w][0][:, self.open_fill, :] = k_new
        self.fp[w][1][:, self.open_fill, :] = v_new
        self.open_fill += 1
        if self.open_fill == cfg.window:
            self.tier[w] = TIER_AGED
            self.open_fill = 0
            if cfg.rank_mode == 3:
                self.importance[w] = self.key_norm_score(self.fp[w][0])

    # --------------------------------------------------------------- decode
    def accessible(self):
        """[(window, k, v, n_tokens)] of everything attention may read, ascending window index.

        Full, aged and open windows are read from their full-precision copy (for a promoted window
        that copy is the dequantized approximation); Quantized windows are dequantized from the
        ledger (Cache Execution: active low-bit windows are dequantized before attention);
        Evicted windows are absent."""
        cfg = self.cfg
        acc = []
        for w in range(self.n_windows):
            t = self.tier[w]
            if t in (TIER_FULL, TIER_AGED, TIER_SINK):
                k, v = self.fp[w]
                acc.append((w, k, v, cfg.window))
            elif t == TIER_OPEN:
                k, v = self.fp[w]
                if self.open_fill > 0:
                    acc.append((w, k[:, : self.open_fill], v[:, : self.open_fill], self.open_fill))
            elif t == TIER_QUANT:
                k, v = dequantize_window(self.ledger[w], cfg.group_size, cfg.dtype)
                acc.append((w, k, v, cfg.window))
        return acc

    def decode_attn(self, q, k_new=None, v_new=None):
        """One decode step: append (optional), attention over the accessible tokens, score update.

        Returns (out [H_q, d] rounded to the execution datatype, mass [max_windows] float64) where
        mass[w] = sum over query heads and over the tokens of w of the attention probability
        (the inner sums of Eq. 1 for this step)."""
        cfg = self.cfg
        if k_new is not None:
            self._append(np.asarray(k_new, dtype=np.float64), np.asarray(v_new, dtype=np.float64))
        acc = self.accessible()
        mass = np.zeros(cfg.max_windows, dtype=np.float64)
        if not acc:
            return np.zeros((cfg.n_q_heads, cfg.head_dim)), mass
        if cfg.rope_base > 0:
            # stored keys are pre-RoPE: the rotation for the key's absolute position is applied when it is read
            # (Migration-Stable Quantization: "RoPE is reapplied after dequantization")
            acc = [(w, apply_rope(k, w * cfg.window + np.arange(n), cfg.rope_base, cfg.dtype), v, n) for w, k, v, n in acc]
        k_acc = np.concatenate([a[1] for a in acc], axis=1)
        v_acc = np.concatenate([a[2] for a in acc], axis=1)
        out, probs = accessible_attention(q, k_acc, v_acc, cfg.scale)
        pos = 0
        for w, _, _, n in acc:
            mass[w] = probs[:, pos : pos + n].sum()
            pos += n
        if cfg.rank_mode == 0:
            self.importance += mass
        else:
            self.event_mass += mass
        self.stats["steps"] += 1
        return round_to_dtype(out, cfg.dtype), mass

    # -------------------------------------------------------------- routing
    def recent_lo(self):
        """First window index of the protected recent region: the `recent_windows` newest filled
        windows (the open window, if any, comes after them)."""
        t = self.tier[: self.n_windows]
        n_filled = self.n_windows - int((t == TIER_OPEN).sum())
        return n_filled - self.cfg.recent_windows

    def ranked_candidates(self):
        """Candidate pool F ∪ Q ∪ aged (filled windows that have exited the recent region), ranked by
        float32 score, higher first, lower index first.  Sink windows are never candidates."""
        t = self.tier[: self.n_windows]
        idx = np.arange(self.n_windows)
        cand = np.flatnonzero((t == TIER_FULL) | (t == TIER_QUANT) | ((t == TIER_AGED) & (idx < self.recent_lo())))
        s32 = self.importance[cand].astype(np.float32)
        order = np.lexsort((cand, -s32.astype(np.float64)))
        return cand[order]

    def fold_event_mass(self):
        """Ranking-function appendix: S_decay <- lambda S_decay + u and S_p^p <- S_p^p + u^p at a routing
        event, for every stored window; float32, each operation rounded on its own."""
        cfg = self.cfg
        t = self.tier[: self.n_windows]
        live = np.flatnonzero((t != TIER_NONE) & (t != TIER_EVICTED))
        s = self.importance[live].astype(np.float32)
        u = self.event_mass[live].astype(np.float32)
        if cfg.rank_mode == 1:
            s = np.float32(cfg.rank_param) * s + u  # numpy rounds the product, then the sum, to float32
        else:
            v = u.copy()
            for _ in range(int(cfg.rank_param) - 1):
                v = v * u
            s = s + v
        self.importance[live] = s.astype(np.float64)
        self.event_mass[live] = 0.0

    def rebalance(self, prefill=False):
        """Algorithm 1: TopK partition of the candidates, then promote / demote / evict with the ledger."""
        cfg = self.cfg
        if cfg.rank_mode in (1, 2) and not prefill:
            self.fold_event_mass()
        ranked = self.ranked_candidates()
        k_f, k_q = cfg.fp_budget_windows, cfg.q_budget_windows
        if cfg.one_way:
            new_f = np.array([w for w in ranked if self.tier[w] != TIER_QUANT][:k_f], dtype=ranked.dtype)
            in_f = set(int(w) for w in new_f)
            rest = np.array([w for w in ranked if int(w) not in in_f], dtype=ranked.dtype)
            new_q, new_e = rest[:k_q], rest[k_q:]
        else:
            new_f = ranked[:k_f]
            new_q = ranked[k_f : k_f + k_q]
            new_e = ranked[k_f + k_q :]

        promotions = sorted(int(w) for w in new_f if self.tier[w] == TIER_QUANT)
        demotions = sorted(int(w) for w in new_q if self.tier[w] != TIER_QUANT)
        first_demotions = [w for w in demotions if self.ledger_flag[w] == LEDGER_NONE]

        # first-time demotions read their full-precision data before any page changes hands
        new_entries = {}
        for w in first_demotions:
            k, v = self.fp[w]
            new_entries[w] = quantize_window(k, v, cfg.quant_bits, cfg.group_size, cfg.dtype)
        promoted_data = {w: dequantize_window(self.ledger[w], cfg.group_size, cfg.dtype) for w in promotions}

        # releases
        for w in demotions:
            if self.fp_page[w] >= 0:
                self.fp_owner[self.fp_page[w]] = -1
                self.fp_page[w] = -1
            self.fp.pop(w, None)
        for w in (int(x) for x in new_e):
            if self.fp_page[w] >= 0:
                self.fp_owner[self.fp_page[w]] = -1
                self.fp_page[w] = -1
            if self.q_page[w] >= 0:
                self.q_owner[self.q_page[w]] = -1
                self.q_page[w] = -1
            self.fp.pop(w, None)
            self.ledger.pop(w, None)
            self.ledger_flag[w] = LEDGER_NONE
            self.tier[w] = TIER_EVICTED
            self.stats["deletions"] += 1

        # allocations, ascending window index, ascending free page id.  A window of the new Full tier
        # that holds no full-precision page needs one: a promotion, or a prompt window at prefill.
        in_f = set(int(x) for x in new_f)
        pinned = [w for w in range(self.n_windows)
                  if self.tier[w] in (TIER_SINK, TIER_AGED) and w not in in_f and self.fp_page[w] < 0 and w in self.fp]
        for w in sorted(in_f | set(pinned)):
            if self.fp_page[w] < 0:
                self.fp_page[w] = self._take_lowest_free(self.fp_owner, w)
            if w not in in_f:
                continue  # sink or recent window of the prompt: gets its page, keeps its state
            if self.tier[w] == TIER_QUANT:
                self.fp[w] = promoted_data[w]
                self.ledger_flag[w] = LEDGER_DORMANT
                self.stats["promotions"] += 1
            self.tier[w] = TIER_FULL
        for w in demotions:
            if self.ledger_flag[w] == LEDGER_NONE:
                self.q_page[w] = self._take_lowest_free(self.q_owner, w)
                self.ledger[w] = new_entries[w]
                self.stats["quantizations"] += 1
            else:
                self.stats["reactivations"] += 1
            self.ledger_flag[w] = LEDGER_ACTIVE
        for w in (int(x) for x in new_q):
            self.tier[w] = TIER_QUANT

    # --------------------------------------------------------------- export
    def tier_counts(self):
        t = self.tier[: self.n_windows]
        return {name: int((t == val).sum()) for name, val in
                (("open", TIER_OPEN), ("aged", TIER_AGED), ("full", TIER_FULL),
                 ("quant", TIER_QUANT), ("evicted", TIER_EVICTED), ("sink", TIER_SINK))}
