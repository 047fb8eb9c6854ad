"""Seeded synthetic decode workloads (input generation only).

This module draws the inputs of the decode hot path -- prompt keys/values,
prefill window scores, decode queries, appended keys/values -- with the shapes
of the long-context models the paper evaluates.  It contains none of the
method's arithmetic (no attention, no quantizer, no routing): both the CUDA
path and the CPU oracle consume the tensors produced here, so they provably see
the same bytes.  Everything is drawn from `torch.Generator` streams keyed by
(seed, unit, stream); a "unit" is one (layer, sequence) pair, unit = layer * batch + seq.

Two helpers here restate a definition of the method because the workload DEFINITIONS need it, not because anything
is checked with them: `Workload.fp_window_bytes / q_window_bytes` (bytes of a window in either tier: configuration 4
sizes its quantized tier "to equal memory", and bench.py counts algorithmic bytes) and `initial_quantized_set` (which
windows a ranking puts in the quantized tier at prefill: configuration 3 steers a tenth of its queries at windows
"previously quantized").  Neither the CUDA path nor the oracle calls them.
"""

from dataclasses import dataclass, replace

import torch

_TORCH_DTYPE = {"fp16": torch.float16, "bf16": torch.bfloat16}

# stream ids
_S_K, _S_V, _S_QNOISE, _S_PLAN, _S_KNEW, _S_VNEW, _S_SCORES, _S_CHAN = 1, 2, 3, 4, 5, 6, 7, 8

BASE_SEED = 20260805


@dataclass(frozen=True)
class Workload:
    name: str
    batch: int
    n_layers: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    dtype: str
    context: int
    window: int
    quant_bits: int
    group_size: int
    fp_budget_windows: int
    q_budget_windows: int
    steps: int
    rebalance_interval: int
    drift: str = "planted"  # "planted" | "steered" | "random_walk"
    outlier_channels: int = 0
    outlier_scale: float = 1.0
    seed: int = BASE_SEED
    sink_windows: int = 0    # protected sink prefix (windows)
    recent_windows: int = 0  # filled windows kept in the protected recent region
    rank_mode: int = 0       # 0 cumulative attention, 1 exponentially decayed, 2 attention p-norm
    rank_param: float = 0.0  # lambda or p
    one_way: bool = False    # no promotion (promotion ablation)
    rope_base: float = 0.0   # > 0: keys are pre-RoPE and rotated at attention time

    @property
    def n_units(self):
        return self.batch * self.n_layers

    @property
    def n_prompt_windows(self):
        return self.context // self.window

    @property
    def max_context(self):
        return self.context + ((self.steps + self.window - 1) // self.window + 1) * self.window

    @property
    def torch_dtype(self):
        return _TORCH_DTYPE[self.dtype]

    def fp_window_bytes(self):
        return 2 * self.n_kv_heads * self.window * self.head_dim * 2

    def q_window_bytes(self):
        w, d, g, b = self.window, self.head_dim, self.group_size, self.quant_bits
        return self.n_kv_heads * (2 * w * d * b // 8 + (w // g) * d * 4 + w * (d // g) * 4)


def _equal_memory_kq(k_f, m_f, m_q, n_w):
    return min((k_f * m_f) // m_q, n_w - k_f)


def config(index, **overrides):
    """The five benchmark configurations (index 0..4).  Config 4 is a sweep; `bits` and `fp_frac`
    overrides pick the point (defaults: 4-bit, 10 %)."""
    if index == 0:
        wl = Workload("c0-tiny", 1, 1, 1, 1, 64, "fp16", 2048, 32, 4, 32, 8, 16, 64, 1)
    elif index == 1:
        wl = Workload("c1-llama3-8b-32k", 1, 1, 32, 8, 128, "bf16", 32768, 32, 4, 32, 64, 128, 256, 1,
                      outlier_channels=4, outlier_scale=8.0)
    elif index == 2:
        wl = Workload("c2-llama3-8b-stacked", 16, 32, 32, 8, 128, "bf16", 16384, 32, 2, 32, 32, 128, 128, 1)
    elif index == 3:
        wl = Workload("c3-llama31-8b-128k", 4, 1, 32, 8, 128, "bf16", 131072, 64, 4, 64, 64, 256, 512, 1,
                      drift="steered")
    elif index == 4:
        bits = overrides.pop("bits", 4)
        fp_frac = overrides.pop("fp_frac", 0.10)
        n_w = 65536 // 32
        k_f = int(fp_frac * n_w)
        base = Workload("c4-qwen25-7b-64k-b%d-f%02d" % (bits, round(fp_frac * 100)), 8, 1, 28, 4, 128, "bf16",
                        65536, 32, bits, 32, k_f, 0, 256, 1, drift="random_walk")
        k_q = _equal_memory_kq(k_f, base.fp_window_bytes(), base.q_window_bytes(), n_w)
        wl = replace(base, q_budget_windows=k_q)
    else:
        raise ValueError("config index must be 0..4")
    return replace(wl, **overrides) if overrides else wl


def _gen(wl, unit, stream, device, extra=0):
    g = torch.Generator(device=device)
    g.manual_seed((wl.seed * 1000003 + unit * 8191 + stream * 131 + extra * 7919) % (2**63 - 1))
    return g


def outlier_channel_ids(wl, unit):
    if wl.outlier_channels == 0:
        return []
    g = _gen(wl, unit, _S_CHAN, "cpu")
    return sorted(torch.randperm(wl.head_dim, generator=g)[: wl.outlier_channels].tolist())


def _apply_outliers(wl, unit, x):
    ch = outlier_channel_ids(wl, unit)
    if ch:
        x[..., ch] *= wl.outlier_scale
    return x


def gen_prompt_kv(wl, unit, device="cpu"):
    """Prompt keys and values of one unit: [H_kv, context, d] in the workload dtype, N(0,1) with the
    workload's outlier channels scaled (same channels for K and V)."""
    shape = (wl.n_kv_heads, wl.context, wl.head_dim)
    k = torch.randn(shape, generator=_gen(wl, unit, _S_K, device), device=device, dtype=torch.float32)
    v = torch.randn(shape, generator=_gen(wl, unit, _S_V, device), device=device, dtype=torch.float32)
    return (_apply_outliers(wl, unit, k).to(wl.torch_dtype), _apply_outliers(wl, unit, v).to(wl.torch_dtype))


def gen_new_kv(wl, unit, n_steps=None, device="cpu"):
    """Keys and values appended at each decode step: [steps, H_kv, d], same distribution as the prompt."""
    n = wl.steps if n_steps is None else n_steps
    shape = (n, wl.n_kv_heads, wl.head_dim)
    k = torch.randn(shape, generator=_gen(wl, unit, _S_KNEW, device), device=device, dtype=torch.float32)
    v = torch.randn(shape, generator=_gen(wl, unit, _S_VNEW, device), device=device, dtype=torch.float32)
    return (_apply_outliers(wl, unit, k).to(wl.torch_dtype), _apply_outliers(wl, unit, v).to(wl.torch_dtype))


def planted_windows(wl, unit, count=4):
    """Distinct prompt windows whose keys the drifting queries are aimed at."""
    g = _gen(wl, unit, _S_PLAN, "cpu")
    return torch.randperm(wl.n_prompt_windows, generator=g)[:count].tolist()


def synthetic_window_scores(wl, unit):
    """Heavy-tailed stand-in for prompt-attention window mass: float32 [prompt windows], positive,
    normalised to sum to H_q * 8 (eight observation queries per head)."""
    g = _gen(wl, unit, _S_SCORES, "cpu")
    s = torch.empty(wl.n_prompt_windows, dtype=torch.float64).exponential_(1.0, generator=g)
    s = s * s
    s = s / s.sum() * (wl.n_q_heads * 8.0)
    return s.to(torch.float32)


def place_planted(scores, planted, k_f, k_q):
    """Overwrite each planted window's score so that it ranks in the middle of the quantized tier:
    planted window j gets a value just below the score currently at rank k_f + k_q // 2 + j."""
    s = scores.clone()
    order = torch.argsort(s, descending=True, stable=True)
    for j, w in enumerate(planted):
        r = min(k_f + k_q // 2 + j, s.numel() - 1)
        target = scores[order[r]].item()
        s[w] = torch.nextafter(torch.tensor(target, dtype=s.dtype), torch.tensor(0.0, dtype=s.dtype)).item()
    return s


def initial_quantized_set(scores, k_f, k_q):
    """Windows at ranks k_f .. k_f+k_q-1 of a score vector (higher first, lower index first)."""
    order = torch.argsort(scores, descending=True, stable=True)
    return sorted(order[k_f:k_f + k_q].tolist())


def gen_queries(wl, unit, k_prompt, scores=None, n_steps=None, device="cpu"):
    """Decode queries [steps, H_q, d] in the workload dtype.

    planted:     q = eps + beta * ((1-lam) K[a_j0] + lam K[a_j1]) on a seeded half of the steps, pure
                 noise otherwise; the focus moves through the 4 planted windows over the run;
                 beta = 0.75 d / |K[a]|^2 so the anchor logit stays near 0.75 sqrt(d).
    steered:     as planted, and on a seeded 10 % of the steps the query is aimed (beta scaled to 1.0)
                 at the centre token of a window drawn from the set quantized at prefill (`scores`).
    random_walk: the focus window does a clipped Gaussian random walk (sigma 4 windows) over the
                 prompt; q = eps + beta * K[centre of the focus window].
    """
    n = wl.steps if n_steps is None else n_steps
    d, hq, hkv, w = wl.head_dim, wl.n_q_heads, wl.n_kv_heads, wl.window
    group = hq // hkv
    gq = _gen(wl, unit, _S_QNOISE, "cpu")
    eps = torch.randn((n, hq, d), generator=gq, dtype=torch.float32)
    focus_on = torch.rand(n, generator=gq) < 0.5
    steer = torch.rand(n, generator=gq) < 0.10
    walk = torch.randn(n, generator=gq) * 4.0
    cache = {}

    def anchor_keys(win):  # [H_q, d] key of the centre token of window `win`, expanded over the GQA group
        if win not in cache:
            a = win * w + w // 2
            ka = k_prompt[:, a, :].to(device="cpu", dtype=torch.float32)  # [H_kv, d]
            beta = 0.75 * d / (ka * ka).sum(-1, keepdim=True).clamp_min(1e-6)
            cache[win] = (beta * ka).repeat_interleave(group, dim=0)
        return cache[win]

    q = eps.clone()
    planted = planted_windows(wl, unit)
    if wl.drift in ("planted", "steered"):
        qset = initial_quantized_set(scores, wl.fp_budget_windows, wl.q_budget_windows) \
            if (wl.drift == "steered" and scores is not None) else None
        pick = torch.randint(0, 1 << 30, (n,), generator=gq)
        for t in range(n):
            if wl.drift == "steered" and qset and bool(steer[t]):
                q[t] += anchor_keys(qset[int(pick[t]) % len(qset)]) * (1.0 / 0.75)
            elif bool(focus_on[t]):
                phi = 4.0 * t / n
                j0 = int(phi) % 4
                j1 = (j0 + 1) % 4
                lam = phi - int(phi)
                q[t] += (1.0 - lam) * anchor_keys(planted[j0]) + lam * anchor_keys(planted[j1])
    elif wl.drift == "random_walk":
        c = float(planted[0])
        for t in range(n):
            c = min(max(c + float(walk[t]), 0.0), wl.n_prompt_windows - 1.0)
            q[t] += anchor_keys(int(round(c)))
    else:
        raise ValueError(wl.drift)
    return q.to(wl.torch_dtype).to(device)
