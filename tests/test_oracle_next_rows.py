"""Pins for the checker's sentence-level selection and mask bit stream (Sec. 3.2)."""
import os
from fractions import Fraction

import numpy as np

from oracle import pdd_oracle as orc
from paper_2508_09035_b200 import workloads as wl

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def test_unit_sentences_reduce_to_token_topk():
    """With one token per sentence and distinct scores, first-fit by decreasing value with
    unit sizes is exactly the token-level top-k, including prefix/suffix and received tokens."""
    rng = wl.rng_for(300)
    for trial in range(20):
        n = int(rng.integers(5, 200))
        score = rng.permutation(n).astype(np.float64) + 0.25
        kind = (rng.random(n) < 0.15).astype(np.uint8)
        lo = int(rng.integers(0, n // 3 + 1))
        hi = n - int(rng.integers(0, n // 3 + 1))
        r = float(rng.random())
        seg = np.arange(lo, hi + 1)
        keep_s, n_s, taken = orc.refine_sentences(score, kind, seg, r)
        keep_t, n_t, k = orc.refine_topk(score, kind, lo, hi, r)
        np.testing.assert_array_equal(keep_s, keep_t)
        assert n_s == n_t


def test_sentence_selection_invariants():
    rng = wl.rng_for(301)
    for trial in range(30):
        n = int(rng.integers(20, 400))
        score = rng.random(n)
        kind = (rng.random(n) < 0.1).astype(np.uint8)
        lo, hi = int(rng.integers(0, 5)), n - int(rng.integers(0, 5))
        cuts = np.unique(np.concatenate([[lo, hi], rng.integers(lo, hi + 1, size=int(rng.integers(1, 30)))]))
        r = float(rng.choice([0.0, 0.1, 0.3, 0.5, 0.9, 1.0]))
        keep, n_kept, taken = orc.refine_sentences(score, kind, cuts, r)
        value, count = orc.sentence_values(score, kind, cuts)
        prompt = kind == 0
        pos = np.arange(n)
        always = prompt & ((pos < lo) | (pos >= hi))
        k_total = orc.keep_count(r, int(prompt.sum()))
        budget = min(max(k_total - int(always.sum()), 0), int((prompt & ~always).sum()))
        assert keep[always].all() and not keep[~prompt].any()
        assert n_kept == int(keep.sum()) <= int(always.sum()) + budget
        used = int(count[taken].sum())
        assert used <= budget
        for s in range(len(value)):                       # whole sentences only
            sl = slice(cuts[s], cuts[s + 1])
            assert (keep[sl][prompt[sl]] == (1 if taken[s] else 0)).all()
        # every sentence left out either has no prompt token or did not fit when its turn came:
        # no left-out sentence fits in what is left over at the end
        rem = budget - used
        left = [s for s in range(len(value)) if not taken[s] and count[s] > 0]
        assert all(count[s] > rem for s in left)
        # the best sentence is taken whenever it fits the budget
        if len(value) and count.max() > 0:
            best = int(np.argsort(-value, kind="stable")[0])
            if 0 < count[best] <= budget:
                assert taken[best]
        if r == 1.0:
            assert taken[count > 0].all()
        if r == 0.0:
            assert not taken.any()


def test_sentence_value_is_the_mean_of_prompt_tokens():
    score = np.array([1.0, 2.0, 6.0, 10.0, 3.0, 5.0])
    kind = np.array([0, 0, 1, 0, 0, 0], np.uint8)
    v, c = orc.sentence_values(score, kind, [0, 3, 4, 6])
    np.testing.assert_allclose(v, [1.5, 10.0, 4.0])
    assert list(c) == [2, 1, 2]
    v, c = orc.sentence_values(score, np.array([1, 1, 1, 0, 0, 0], np.uint8), [0, 3, 6])
    assert v[0] == -np.inf and c[0] == 0 and abs(v[1] - 6.0) < 1e-15
    # fp32 inputs are widened before they are added (a single-precision sum would lose the ones)
    s32 = np.array([1e8, 1.0, 1.0, 1.0, 1.0], np.float32)
    v64, _ = orc.sentence_values(s32, None, [0, 5])
    assert v64[0] == (1e8 + 4) / 5


def test_select_sentences_is_first_fit_by_decreasing_value():
    value = np.array([0.5, 0.9, 0.9, -np.inf, 0.1])
    count = np.array([3, 4, 2, 0, 1])
    # order 1, 2, 0, 4: 4 tokens, then 2 (fits 6), then 3 does not fit the 1 left, then 1 fits
    assert list(orc.select_sentences(value, count, 7)) == [False, True, True, False, True]
    assert list(orc.select_sentences(value, count, 3)) == [False, False, True, False, True]
    assert not orc.select_sentences(value, count, 0).any()


def test_golden_sentence_example():
    """Hand-worked example in tests/golden/sentence_example.txt."""
    vals = {}
    for line in open(os.path.join(GOLDEN, "sentence_example.txt")):
        line = line.split("#")[0].strip()
        if line:
            name, rest = line.split("=")
            vals[name.strip()] = [float(Fraction(t)) for t in rest.split()]
    score = np.array(vals["score"])
    kind = np.array(vals["kind"], np.uint8)
    seg = np.array(vals["seg_start"], np.int64)
    keep, n_kept, taken = orc.refine_sentences(score, kind, seg, vals["keep_ratio"][0])
    v, c = orc.sentence_values(score, kind, seg)
    np.testing.assert_allclose(v, vals["value"], rtol=1e-15)
    assert list(taken.astype(int)) == [int(x) for x in vals["taken"]]
    assert list(keep) == [int(x) for x in vals["keep"]]
    assert n_kept == int(vals["n_kept"][0])


def test_mask_bit_stream_is_little_endian_within_bytes():
    rng = wl.rng_for(302)
    for n in (1, 7, 8, 9, 64, 100):
        keep = (rng.random(n) < 0.4).astype(np.uint8)
        got = orc.pack_mask_bits(keep)
        want = bytearray((n + 7) // 8)
        for i in range(n):
            if keep[i]:
                want[i // 8] |= 1 << (i % 8)
        assert bytes(got) == bytes(want)
    assert list(orc.pack_mask_bits([1, 0, 0, 0, 0, 0, 0, 0, 1])) == [1, 1]
    assert list(orc.pack_mask_bits([0, 1, 1])) == [6]
