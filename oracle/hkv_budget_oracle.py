"""CPU oracle for the top-down budget allocation of HybridKV (paper Section 3.2).  TEST INFRASTRUCTURE ONLY.

Plain statement of the two allocation levels in the paper's notation, in float64 with the operations in
the order the equations print them; used by the tests only.  Pins (tests/test_budget_alloc.py): exact
rational arithmetic on small cases, B_dyna + B_stat = B_total, the sum of static budgets lies in
[B_stat, B_stat + N_stat), r = 1 splits the total in proportion to the head counts, alpha = 1 and equal
scores give every static head ceil(B_stat / N_stat).
"""
from __future__ import annotations

import math
from typing import Optional, Sequence

import numpy as np


def head_type_budgets(total_budget: int, n_stat: int, n_dyna: int, r: float):
    """Head-type level: B_bar = B_total / (N_stat + N_dyna); B_dyna = ceil(r * B_bar * N_dyna);
    B_stat = B_total - B_dyna.  r must not exceed B_total / (B_bar * N_dyna)."""
    b_total = float(total_budget)
    b_bar = b_total / float(n_stat + n_dyna)
    if n_dyna == 0:
        return int(total_budget), 0
    if r > b_total / (b_bar * float(n_dyna)):
        raise ValueError("share coefficient r exceeds its bound")
    b_dyna = min(int(math.ceil(r * b_bar * float(n_dyna))), int(total_budget))
    return int(total_budget) - b_dyna, b_dyna


def allocate_budgets(head_type: Sequence[int], scores: Optional[Sequence[float]], total_budget: int, r: float,
                     alpha: float, pad_pow2: bool = False) -> np.ndarray:
    """Per-head budgets.  Static head: ceil(alpha * B_stat / N_stat + (1 - alpha) * B_stat * S~) with S~ the
    score L1-normalised over all static heads; dynamic head: B_dyna split uniformly (rounded up), optionally
    padded up to a power of two."""
    ht = np.asarray(head_type).ravel()
    n = ht.size
    n_stat = int((ht == 0).sum())
    n_dyna = n - n_stat
    b_stat, b_dyna = head_type_budgets(total_budget, n_stat, n_dyna, r)
    out = np.zeros(n, dtype=np.int64)
    if n_dyna:
        each = max(1, -(-b_dyna // n_dyna))
        if pad_pow2:
            each = 1 << (each - 1).bit_length()
        out[ht == 1] = each
    if n_stat:
        ssum = 0.0
        if scores is not None:
            for i in range(n):
                if ht[i] == 0:
                    ssum += float(scores[i])
        for i in range(n):
            if ht[i] == 0:
                s_norm = float(scores[i]) / ssum if (scores is not None and ssum > 0.0) else 1.0 / float(n_stat)
                b = alpha * float(b_stat) / float(n_stat) + (1.0 - alpha) * float(b_stat) * s_norm
                out[i] = max(1, int(math.ceil(b)))
    return out
