"""Top-down budget allocation (Section 3.2): pins for the oracle, and the library's host routine against the
oracle.  CPU only (the routine does no device work)."""
import math
from fractions import Fraction

import numpy as np
import pytest

from oracle import hkv_budget_oracle as bo


@pytest.fixture(scope="module")
def hkv():
    from paper_2604_05887_b200.build import build_library
    build_library()
    from paper_2604_05887_b200 import binding
    return binding


def exact_reference(head_type, scores, total, r, alpha):
    """The same equations in exact rational arithmetic (inputs given as Fractions)."""
    ht = list(head_type)
    n_stat, n_dyna = ht.count(0), ht.count(1)
    b_bar = Fraction(total, n_stat + n_dyna)
    b_dyna = min(math.ceil(r * b_bar * n_dyna), total) if n_dyna else 0
    b_stat = total - b_dyna
    ssum = sum(s for s, t in zip(scores, ht) if t == 0)
    out = []
    for s, t in zip(scores, ht):
        if t == 1:
            out.append(max(1, math.ceil(Fraction(b_dyna, n_dyna))))
        else:
            sn = s / ssum if ssum else Fraction(1, n_stat)
            out.append(max(1, math.ceil(alpha * b_stat / n_stat + (1 - alpha) * b_stat * sn)))
    return b_stat, b_dyna, out


def test_oracle_matches_exact_rational_arithmetic_on_small_cases():
    rng = np.random.default_rng(0)
    for _ in range(300):
        n = int(rng.integers(2, 12))
        ht = rng.integers(0, 2, size=n).tolist()
        sc = [Fraction(int(rng.integers(1, 64)), 64) for _ in range(n)]          # exactly representable
        total = int(rng.integers(n * 40, n * 4000))
        r = Fraction(int(rng.integers(16, 64)), 64)
        alpha = Fraction(int(rng.integers(0, 65)), 64)
        b_stat, b_dyna, ref = exact_reference(ht, sc, total, r, alpha)
        if ht.count(0) and b_stat < ht.count(0):
            continue
        got = bo.allocate_budgets(ht, [float(s) for s in sc], total, float(r), float(alpha))
        diff = np.abs(np.array(ref) - got)
        # float64 may land on the other side of an exact integer only when the exact value IS an integer
        assert diff.max() <= 1
        for i in np.nonzero(diff)[0]:
            t = alpha * b_stat / ht.count(0) + (1 - alpha) * b_stat * (sc[i] / sum(s for s, tt in zip(sc, ht) if tt == 0))
            assert t.denominator == 1, "a difference away from an exact integer boundary"
        assert bo.head_type_budgets(total, ht.count(0), ht.count(1), float(r)) == (b_stat, b_dyna)


def test_oracle_invariants():
    rng = np.random.default_rng(1)
    for _ in range(200):
        n = int(rng.integers(4, 200))
        ht = rng.integers(0, 2, size=n)
        if ht.sum() in (0, n):
            ht[0], ht[1] = 0, 1
        sc = rng.random(n) * 0.5 + 0.5
        total = int(rng.integers(n * 100, n * 5000))
        r = float(rng.uniform(0.3, 1.0)); alpha = float(rng.uniform(0, 1))
        n_stat, n_dyna = int((ht == 0).sum()), int((ht == 1).sum())
        b_stat, b_dyna = bo.head_type_budgets(total, n_stat, n_dyna, r)
        assert b_stat + b_dyna == total
        b = bo.allocate_budgets(ht, sc, total, r, alpha)
        s_static = int(b[ht == 0].sum())
        assert b_stat <= s_static < b_stat + n_stat + 1          # each ceiling adds less than one token
        assert len(set(b[ht == 1].tolist())) == 1 and b[ht == 1][0] == -(-b_dyna // n_dyna)
        # a higher score never gets a smaller budget
        order = np.argsort(sc[ht == 0]); bs = b[ht == 0][order]
        assert np.all(np.diff(bs) >= 0)


def test_oracle_special_cases():
    # r = 1: the two head types share the total in proportion to their counts
    assert bo.head_type_budgets(12000, 9, 3, 1.0) == (9000, 3000)
    # r above its bound is refused
    with pytest.raises(ValueError):
        bo.head_type_budgets(12000, 9, 3, 4.01)
    # alpha = 1 or equal scores: every static head gets ceil(B_stat / N_stat)
    ht = [0, 0, 0, 1, 1]
    for alpha, sc in [(1.0, [0.9, 0.5, 0.7, 0, 0]), (0.3, [0.8] * 5), (0.3, None)]:
        b = bo.allocate_budgets(ht, sc, 10001, 0.75, alpha)
        b_stat, b_dyna = bo.head_type_budgets(10001, 3, 2, 0.75)
        assert b[:3].tolist() == [math.ceil(b_stat / 3)] * 3 and b[3:].tolist() == [math.ceil(b_dyna / 2)] * 2
    # power-of-two padding of the dynamic budget rounds up
    b = bo.allocate_budgets(ht, None, 10001, 0.75, 0.5, pad_pow2=True)
    assert b[3] == 2048 and b[4] == 2048 and bo.allocate_budgets(ht, None, 10001, 0.75, 0.5)[3] == 1501
    # alpha = 0: budgets proportional to the scores
    b = bo.allocate_budgets([0, 0, 1], [1.0, 3.0, 0.0], 9000, 1.0, 0.0)
    assert b.tolist() == [1500, 4500, 3000]


def test_library_matches_oracle(hkv):
    rng = np.random.default_rng(2)
    for it in range(500):
        n = int(rng.integers(2, 300))
        ht = rng.integers(0, 2, size=n).astype(np.uint8)
        sc = rng.random(n)
        total = int(rng.integers(n * 50, n * 6000))
        r = float(rng.uniform(0.2, 1.0)); alpha = float(rng.uniform(0, 1)); pad = bool(it & 1)
        n_stat = int((ht == 0).sum())
        b_stat, _ = bo.head_type_budgets(total, n_stat, n - n_stat, r)
        if n_stat and b_stat < n_stat:
            continue
        ref = bo.allocate_budgets(ht, sc, total, r, alpha, pad_pow2=pad)
        got = hkv.hkv_allocate_budgets(ht, sc, total, r, alpha, hkv.HKV_BUDGET_PAD_POW2 if pad else 0)
        assert np.array_equal(ref, got)
    # no scores, all static, all dynamic
    assert np.array_equal(hkv.hkv_allocate_budgets([0, 0, 0], None, 3001, 0.75, 0.5), bo.allocate_budgets([0, 0, 0], None, 3001, 0.75, 0.5))
    assert np.array_equal(hkv.hkv_allocate_budgets([1, 1, 1], None, 3001, 0.75, 0.5), bo.allocate_budgets([1, 1, 1], None, 3001, 0.75, 0.5))


def test_library_rejects_bad_arguments(hkv):
    for args, status in [(([0, 1], None, 1, 0.75, 0.5), 3),            # fewer tokens than heads
                         (([0, 1], None, 1000, 2.5, 0.5), 3),          # r above (N_stat + N_dyna) / N_dyna
                         (([0, 1], None, 1000, 0.75, 1.5), 3),         # alpha outside [0, 1]
                         (([0, 2], None, 1000, 0.75, 0.5), 1),         # head type not 0 / 1
                         (([0, 1], [-1.0, 0.0], 1000, 0.75, 0.5), 1)]: # negative score
        with pytest.raises(hkv.HkvError) as e:
            hkv.hkv_allocate_budgets(*args)
        assert e.value.status == status


def test_allocated_budgets_feed_the_planner(hkv):
    """The budgets of one layer's (b, h) units go straight into hkv_plan."""
    ht = np.array([[0, 1, 0, 1], [1, 0, 0, 1]], dtype=np.uint8)
    sc = np.array([[0.95, 0, 0.91, 0], [0, 0.99, 0.93, 0]])
    bud = hkv.hkv_allocate_budgets(ht, sc, 8 * 200, 0.75, 0.5).reshape(2, 4)
    cfg = hkv.make_config(2, 28, 4, 128, 2000, 32, 32)
    cache_bytes, ws = hkv.hkv_plan(cfg, [2000, 1800], ht, bud)
    assert cache_bytes > 0 and bud.min() >= 1
