"""Routing diagnostics of the observation appendix, computed from the oracle's state (test infrastructure).

  * tier-mass share (Observation II, tier-mass equation): mu(z) = sum of the scores of the windows in tier z
    divided by the sum over all windows, z in {Full, Quantized, Evicted, Local}; Local = the protected
    regions (sink prefix, recent region, open window);
  * selection churn (Observation I, selection-churn equation): Jaccard distance between the sets of retained
    historical windows after two consecutive routing events; the protected recent region is excluded.
    Windows all have the same number of tokens, so the Jaccard distance over token positions equals the one
    over windows.
"""

import numpy as np

from .cache import TIER_AGED, TIER_EVICTED, TIER_FULL, TIER_OPEN, TIER_QUANT, TIER_SINK


def tier_mass_share(unit):
    """{"full", "quant", "evicted", "local"} -> share of the cumulative score held by that tier."""
    n = unit.n_windows
    t = unit.tier[:n]
    s = unit.importance[:n].astype(np.float64)
    total = s.sum()
    groups = {"full": t == TIER_FULL, "quant": t == TIER_QUANT, "evicted": t == TIER_EVICTED,
              "local": (t == TIER_AGED) | (t == TIER_OPEN) | (t == TIER_SINK)}
    return {k: (float(s[m].sum() / total) if total > 0 else 0.0) for k, m in groups.items()}


def retained_windows(unit):
    """Historical windows kept after a routing event: Full or Quantized (protected regions excluded)."""
    t = unit.tier[: unit.n_windows]
    return set(np.flatnonzero((t == TIER_FULL) | (t == TIER_QUANT)).tolist())


def selection_churn(retained_before, retained_after):
    union = retained_before | retained_after
    if not union:
        return 0.0
    return 1.0 - len(retained_before & retained_after) / len(union)
