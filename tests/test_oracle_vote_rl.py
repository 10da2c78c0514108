"""Pins for the checker's per-head vote selection (Sec. 3.2) and the (r, L) solver of problem P
(Sec. 3.4, Algorithm 1)."""
import math
import os
from fractions import Fraction

import numpy as np

from oracle import pdd_oracle as orc
from paper_2508_09035_b200 import workloads as wl

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _fields(path):
    out = {}
    for line in open(path):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        key, val = [x.strip() for x in line.split("=", 1)]
        out[key] = val
    return out


# ------------------------------------------------------------------ per-head vote

def test_golden_vote_example():
    f = _fields(os.path.join(GOLDEN, "vote_example.txt"))
    cs = np.array([[float(x) for x in f["colsum%d" % h].split()] for h in range(3)])
    kind = np.array([int(x) for x in f["kind"].split()], dtype=np.uint8)
    lo, hi = [int(x) for x in f["cand"].split()]
    ratio = float(Fraction(f["keep_ratio"]))
    keep, n_kept, votes, _ = orc.refine_vote(cs, kind, lo, hi, ratio)
    assert keep.tolist() == [int(x) for x in f["keep"].split()]
    assert votes.tolist() == [int(x) for x in f["votes"].split()]
    assert n_kept == int(f["n_kept"])
    # the example is built so that the two merge rules disagree
    keep_sum, _, _ = orc.refine_topk(orc.importance([cs]), kind, lo, hi, ratio)
    assert keep_sum.tolist() == [int(x) for x in f["keep_sum_first"].split()]


def test_vote_with_one_head_or_equal_heads_is_plain_topk():
    rng = wl.rng_for(500)
    for trial in range(20):
        n = int(rng.integers(4, 300))
        row = rng.random(n)
        if trial % 3 == 0:
            row = np.round(row * 5) / 5                       # ties
        kind = (rng.random(n) < 0.1).astype(np.uint8)
        lo, hi = int(rng.integers(0, n // 4 + 1)), n - int(rng.integers(0, n // 4 + 1))
        r = float(rng.random())
        want, want_n, _ = orc.refine_topk(row, kind, lo, hi, r)
        for heads in (1, 5):
            keep, n_kept, votes, _ = orc.refine_vote(np.tile(row, (heads, 1)), kind, lo, hi, r)
            np.testing.assert_array_equal(keep, want)
            assert n_kept == want_n
            cand = (kind == 0) & (np.arange(n) >= lo) & (np.arange(n) < hi)
            np.testing.assert_array_equal(votes[cand], heads * want[cand])


def test_vote_invariants_fix_the_set():
    """The order (votes desc, summed value desc, position asc) is total, so popcount plus
    "no dropped candidate beats a kept one" determines the mask uniquely."""
    rng = wl.rng_for(501)
    for trial in range(30):
        n, heads = int(rng.integers(6, 200)), int(rng.integers(2, 9))
        cs = rng.random((heads, n)) ** 3
        if trial % 2:
            cs = np.round(cs * 4) / 4
        kind = (rng.random(n) < 0.1).astype(np.uint8)
        lo, hi = int(rng.integers(0, 4)), n - int(rng.integers(0, 4))
        r = float(rng.choice([0.0, 0.2, 0.5, 0.8, 1.0]))
        pool = [("none", 1), ("avg", 3), ("max", 5)][trial % 3]
        keep, n_kept, votes, _ = orc.refine_vote(cs, kind, lo, hi, r, *pool)
        pos = np.arange(n)
        prompt = kind == 0
        cand = prompt & (pos >= lo) & (pos < hi)
        always = prompt & ~cand
        k = min(max(orc.keep_count(r, int(prompt.sum())) - int(always.sum()), 0), int(cand.sum()))
        assert keep[always].all() and not keep[~prompt].any()
        assert int(keep[cand].sum()) == k and n_kept == k + int(always.sum())
        assert int(votes.sum()) == heads * k and not votes[~cand].any()
        total = orc.pool1d(cs, *pool).sum(axis=0)
        rank = [(-int(votes[j]), -float(total[j]), int(j)) for j in pos[cand]]
        kept = [t for t in rank if keep[t[2]]]
        dropped = [t for t in rank if not keep[t[2]]]
        if kept and dropped:
            assert max(kept) < min(dropped)
        # each head's own choice contains its k largest pooled values
        pooled = orc.pool1d(cs, *pool)
        for h in range(heads):
            kh, _, _ = orc.refine_topk(pooled[h], kind, lo, hi, r)
            assert int((kh.astype(bool) & cand).sum()) == k


def test_vote_total_is_the_head_sum_of_pooled_values():
    rng = wl.rng_for(502)
    n, heads = 200, 6
    cs = rng.random((heads, n))
    for pool in (("none", 1), ("avg", 5), ("max", 3)):
        total = orc.refine_vote(cs, None, 3, n - 3, 0.35, *pool)[3]
        want = np.zeros(n)
        for h in range(heads):
            want += orc.pool1d(cs[h], *pool)
        np.testing.assert_allclose(total, want, rtol=1e-14)


# ------------------------------------------------------------------ (r, L) solver

def _feasible(p, r, L, tol=1e-9):
    """Eq. 5 and Eq. 6 written out for one (r, L)."""
    l, k_c, k_d, delta, delta_c, xi, tau, tpot_c, tpot_d = p
    ttft_c = k_c * l + delta_c
    ttft_d = k_c * l + delta + k_d * r * l
    if not (xi - tol <= r <= 1 - (k_c + delta / l) / k_d + tol and 0 < r <= 1 + tol):
        return False
    if tau <= tpot_d or L < 2:
        return False
    lower = (k_d * r * l - ttft_c) / (tau - tpot_d)
    upper = (ttft_d - ttft_c) / tpot_c
    return lower - tol <= L - 1 <= upper + tol


def test_golden_rl_examples():
    n = 0
    for line in open(os.path.join(GOLDEN, "rl_examples.txt")):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        lhs, rhs = line.split("|")
        p = [float(x) for x in lhs.split()]
        feas, r, L, ttft_c, ttft_d, smooth = rhs.split()
        got = orc.solve_rl(*p)
        assert got["feasible"] == bool(int(feas))
        assert math.isclose(got["ttft_c"], float(ttft_c), rel_tol=1e-12)
        if got["feasible"]:
            assert math.isclose(got["r"], float(r), rel_tol=1e-12)
            assert got["L"] == int(L)
            assert math.isclose(got["ttft_d"], float(ttft_d), rel_tol=1e-12)
            assert math.isclose(got["tpot_smooth"], float(smooth), rel_tol=1e-12)
        n += 1
    assert n == 4


def _random_problem(rng):
    l = float(rng.integers(64, 40000))
    k_d = float(rng.uniform(0.2, 3.0))
    k_c = k_d * float(rng.uniform(0.01, 0.5))
    delta = float(rng.uniform(0, 0.3)) * k_d * l * float(rng.random() < 0.8)
    delta_c = delta * float(rng.uniform(0.3, 1.0))
    xi = float(rng.uniform(0.05, 0.9))
    tpot_d = float(rng.uniform(20, 120))
    tau = tpot_d + float(rng.uniform(-10, 80))
    tpot_c = float(rng.uniform(5, 200))
    return (l, k_c, k_d, delta, delta_c, xi, tau, tpot_c, tpot_d)


def test_rl_solution_is_feasible_and_no_grid_point_is_better():
    """Brute force over a grid of r and every L up to 600: the solver's point satisfies Eq. 5
    and Eq. 6, no feasible grid point has a smaller r (TTFT_d grows with r), and where the
    solver finds nothing the grid finds nothing either."""
    rng = wl.rng_for(510)
    n_feas = 0
    grid = np.arange(1, 1001) / 1000.0
    for trial in range(120):
        p = _random_problem(rng)
        got = orc.solve_rl(*p)
        l, k_c, k_d, delta, delta_c, xi, tau, tpot_c, tpot_d = p
        best_r, best_L = None, None
        if tau > tpot_d:
            for r in grid:
                ttft_c = k_c * l + delta_c
                lo = max(1, math.ceil((k_d * r * l - ttft_c) / (tau - tpot_d) - 1e-12))
                for L1 in range(lo, min(lo + 2, 600)):
                    if _feasible(p, float(r), L1 + 1, tol=0.0):
                        best_r, best_L = float(r), L1 + 1
                        break
                if best_r is not None:
                    break
        if got["feasible"]:
            n_feas += 1
            assert _feasible(p, got["r"], got["L"])
            if best_r is not None:
                assert best_r >= got["r"] - 1e-12
            # Eq. 1, the amortisation identity: prefill_d + TPOT_d (L-1) = TTFT_c + TPOT_smooth (L-1)
            m = got["L"] - 1
            assert math.isclose(k_d * got["r"] * l + tpot_d * m,
                                got["ttft_c"] + got["tpot_smooth"] * m, rel_tol=1e-12)
            assert got["tpot_smooth"] <= tau * (1 + 1e-12)
            # Eq. 3 with the estimates of Sec. 3.4, and the gain condition TTFT_d <= prefill_d(l)
            assert math.isclose(got["ttft_d"], k_c * l + delta + k_d * got["r"] * l, rel_tol=1e-12)
            assert got["ttft_d"] <= k_d * l * (1 + 1e-12)
        else:
            assert best_r is None
    assert 20 < n_feas < 110


def test_rl_smallest_L_is_taken():
    """Among the L that fit Eq. 6 at the optimal r the smallest is returned: L - 2 must
    violate the lower bound (or L = 2)."""
    rng = wl.rng_for(511)
    for trial in range(200):
        p = _random_problem(rng)
        got = orc.solve_rl(*p)
        if not got["feasible"] or got["L"] == 2:
            continue
        l, k_c, k_d, delta, delta_c, xi, tau, tpot_c, tpot_d = p
        lower = (k_d * got["r"] * l - got["ttft_c"]) / (tau - tpot_d)
        assert got["L"] - 2 < lower + 1e-9


def test_rl_monotone_in_quality_floor():
    """Raising xi (a stricter quality floor) can only raise r and TTFT_d."""
    p = [8000, 0.05, 1.0, 300, 200, 0.1, 100, 30, 60]
    prev = None
    for xi in np.linspace(0.05, 0.9, 18):
        p[5] = float(xi)
        got = orc.solve_rl(*p)
        assert got["feasible"]
        assert got["r"] >= xi - 1e-15
        if prev is not None:
            assert got["r"] >= prev["r"] and got["ttft_d"] >= prev["ttft_d"]
        prev = got
