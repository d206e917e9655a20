"""Condition a seeded workload so that top-k routing has no near-ties.  TEST INFRASTRUCTURE ONLY.

For every token, each consecutive gap among its min(k+1, E) largest gate logits (fp64, computed by
the oracle from the dtype-rounded inputs) must be at least `margin`; token rows that fail are
redrawn from the generator's next stream until all pass.  This makes both the selected set and its
order robust to fp32 accumulation error, which is what lets routing tables be compared bit-exactly.
"""
from __future__ import annotations

import numpy as np

from . import gate_logits, gate_logits_low


def min_topk_gap(logits: np.ndarray, k: int) -> np.ndarray:
    """Per token: smallest gap between consecutive entries of its min(k+1, E) largest logits."""
    E = logits.shape[1]
    m = min(k + 1, E)
    if m < 2:
        return np.full(logits.shape[0], np.inf)
    top = -np.sort(-logits, axis=1)[:, :m]
    return np.min(top[:, :-1] - top[:, 1:], axis=1)


def enforce_margin(workload, inp, margin: float = 1e-3, max_attempts: int = 64, gate_low: bool = False,
                   round_x_lo_bf16: bool = False) -> int:
    """Redraw rows of inp["x"] in place until every token clears the margin; returns rows redrawn.
    gate_low: the logits are those of the gate that reads x' (w_gate [E,r])."""
    from paper_2502_16927_b200.workloads import redraw_rows

    x = inp["x"]
    bad = np.arange(x.shape[0])
    total = 0
    for attempt in range(1, max_attempts + 1):
        if gate_low:
            logits = gate_logits_low(x[bad], inp["w_down"], inp["w_gate"], inp.get("b_gate"), round_x_lo_bf16)
        else:
            logits = gate_logits(x[bad], inp["w_gate"], inp.get("b_gate"))
        bad = bad[min_topk_gap(logits, workload.k) < margin]
        if bad.size == 0:
            return total
        total += int(bad.size)
        redraw_rows(workload, x, bad, attempt)
    raise RuntimeError("could not reach the requested top-k margin")
