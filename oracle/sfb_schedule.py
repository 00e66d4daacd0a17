"""Host-side schedules of SFB written from the paper's text.  TEST INFRASTRUCTURE ONLY (same rule as sfb_oracle).

* Halton-sequence broadcast (Section 4.3): with the sequence P/2, P/4, 3P/4, P/8, 3P/8, ... worker p sends its
  sufficient factors to the Q workers (p + floor(P * f)) mod P, f = 1/2, 1/4, 3/4, 1/8, 3/8, 5/8, 7/8, ...
  Pinned by the worked example printed in that section (tests/golden/halton_p6_q2.txt).
* SSP rule (Section 4.1, "SSP-SFB"): worker p, having computed t_p SF batches and received tau_p^q from worker q,
  pauses while some q has t_p - tau_p^q > s.  s = 0 is BSP, s = infinity is ASP.
"""
from __future__ import annotations

import math


def halton_fractions(q: int):
    """First q terms of 1/2, 1/4, 3/4, 1/8, 3/8, 5/8, 7/8, ... as (numerator, denominator)."""
    out, den = [], 2
    while len(out) < q:
        for num in range(1, den, 2):
            out.append((num, den))
            if len(out) == q:
                break
        den *= 2
    return out


def halton_offsets(P: int, Q: int):
    return [(num * P) // den for num, den in halton_fractions(Q)]


def halton_peers(p: int, P: int, Q: int):
    """Zero-based ids of the Q workers that worker p (zero-based) sends to, in sequence order."""
    return [(p + off) % P for off in halton_offsets(P, Q)]


def ssp_may_proceed(t_p: int, tau, s: float) -> bool:
    """True iff no worker q is more than s batches behind from p's point of view."""
    if math.isinf(s):
        return True
    return all(t_p - t_q <= s for t_q in tau)
