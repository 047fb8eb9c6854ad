"""Routing diagnostics of the paper's observation appendix, computed from exported window tables (host side).

`tables` is what QEvictCache.export_tables returns.  Tier-mass share: share of the cumulative window score
held by the Full tier, the Quantized tier, the Evicted set and the protected regions (Observation II).
Selection churn: Jaccard distance between the historical windows retained after two consecutive routing
events, protected regions excluded (Observation I)."""

import torch

from .binding import (QEVICT_TIER_AGED, QEVICT_TIER_EVICTED, QEVICT_TIER_FULL, QEVICT_TIER_OPEN, QEVICT_TIER_QUANT,
                      QEVICT_TIER_SINK)


def tier_mass_share(tables):
    n = int(tables["n_windows"][0])
    t = tables["tier"][:n]
    s = tables["importance"][:n].double()
    total = float(s.sum())
    local = (t == QEVICT_TIER_AGED) | (t == QEVICT_TIER_OPEN) | (t == QEVICT_TIER_SINK)
    groups = {"full": t == QEVICT_TIER_FULL, "quant": t == QEVICT_TIER_QUANT, "evicted": t == QEVICT_TIER_EVICTED,
              "local": local}
    return {k: (float(s[m].sum()) / total if total > 0 else 0.0) for k, m in groups.items()}


def retained_windows(tables):
    n = int(tables["n_windows"][0])
    t = tables["tier"][:n]
    return set(torch.nonzero((t == QEVICT_TIER_FULL) | (t == QEVICT_TIER_QUANT)).flatten().tolist())


def selection_churn(retained_before, retained_after):
    union = retained_before | retained_after
    if not union:
        return 0.0
    return 1.0 - len(retained_before & retained_after) / len(union)
