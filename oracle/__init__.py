"""CPU oracle for the QEvict decode hot path (test infrastructure, not product code).

Everything under this package is a plain, slow, float64 restatement of what the
paper's method computes: the asymmetric low-bit window quantizer, attention over
the accessible tokens of a three-tier window cache, the cumulative window score,
the three-tier routing with its write-once ledger, and the byte-constrained tier
capacities.  It exists so that the CUDA path can be checked against it.

Rules this package keeps:
  * it imports nothing from the CUDA package and shares no code, table or
    constant with it;
  * only the tests, the smoke check and the benchmark's CPU-baseline leg may
    import it; the product path never routes through it;
  * every function cites the passage of the paper it restates.
"""

from .numerics import round_to_dtype, DTYPES  # noqa: F401
from .quantizer import (  # noqa: F401
    quantize_groups,
    dequantize_exact,
    dequantize,
    quantize_window,
    dequantize_window,
)
from .attention import accessible_attention  # noqa: F401
from .rope import apply_rope, rope_frequencies, rotate_exact  # noqa: F401
from .diagnostics import retained_windows, selection_churn, tier_mass_share  # noqa: F401
from .cache import (  # noqa: F401
    OracleConfig,
    UnitOracle,
    tier_capacities,
    window_bytes,
    TIER_NONE,
    TIER_OPEN,
    TIER_AGED,
    TIER_FULL,
    TIER_QUANT,
    TIER_EVICTED,
    TIER_SINK,
    LEDGER_NONE,
    LEDGER_ACTIVE,
    LEDGER_DORMANT,
)
