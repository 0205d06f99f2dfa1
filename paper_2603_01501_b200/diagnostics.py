"""Summaries of a logged alignment trace c_t, as the paper reports them:
the 90th percentile of |c_t|, its maximum and the fraction of updates with
|c_t| <= c_low, computed over the updates after an initial transient
(Table 3 uses the updates after step 50), plus the count of steps per regime
of Algorithm 1.  Host-side bookkeeping on numbers the library returns; no
gradient arithmetic happens here."""
from __future__ import annotations

import math
from dataclasses import dataclass
from typing import Dict, Iterable, List, Sequence, Tuple


@dataclass
class AlignmentSummary:
    updates: int
    q90_abs: float
    max_abs: float
    frac_within_c_low: float
    regimes: Dict[str, int]


def quantile(values: Sequence[float], q: float) -> float:
    """Linear-interpolation quantile (the common 'type 7' definition)."""
    xs = sorted(values)
    if not xs:
        return float("nan")
    pos = q * (len(xs) - 1)
    lo = int(math.floor(pos))
    hi = min(lo + 1, len(xs) - 1)
    return xs[lo] + (xs[hi] - xs[lo]) * (pos - lo)


def classify(c: float, c_low: float, c_high: float) -> str:
    """Regime of Algorithm 1 for one cosine (inclusive thresholds as printed)."""
    a = abs(c)
    if a <= c_low:
        return "safe"
    if a >= c_high:
        return "violation"
    return "project"


def summarize_alignment(cos_log: Iterable[float], c_low: float = 0.05, c_high: float = 0.3,
                        skip: int = 50) -> AlignmentSummary:
    cs = [abs(float(c)) for c in cos_log][skip:]
    regimes = {"safe": 0, "project": 0, "violation": 0}
    for c in cs:
        regimes[classify(c, c_low, c_high)] += 1
    n = len(cs)
    return AlignmentSummary(updates=n, q90_abs=quantile(cs, 0.9), max_abs=max(cs) if cs else float("nan"),
                            frac_within_c_low=(sum(c <= c_low for c in cs) / n) if n else float("nan"),
                            regimes=regimes)


def threshold_grid(cos_log: Sequence[float], c_lows=(0.03, 0.05, 0.07), c_highs=(0.2, 0.3, 0.4),
                   skip: int = 0) -> List[Tuple[float, float, Dict[str, int]]]:
    """Regime counts of one trace under every (c_low, c_high) pair of the paper's
    threshold sweep (App. C.3).  Valid because the trace does not depend on the
    thresholds: c_t is computed on raw gradients and the stored direction is raw."""
    return [(lo, hi, summarize_alignment(cos_log, lo, hi, skip).regimes)
            for lo in c_lows for hi in c_highs]
