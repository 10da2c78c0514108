"""GPU parity of the sliding-window variant (the device model's attention, Sec. 3.3): row p sees
keys max(0, p-w+1)..p in attention and in the observation window's column sums.  Same bars
as the plain causal path; windows below, at and above the tile and key-block sizes, windows
that cut through chunks, and a window longer than the sequence (which must equal the plain
path bit for bit)."""
import dataclasses
import os

import numpy as np
import pytest

from paper_2508_09035_b200 import workloads as wl
from tests import helpers as H

pytestmark = pytest.mark.gpu

PATHS = [int(x) for x in os.environ.get("PDD_TEST_PATHS", "0").split(",")]

CASES = [
    # name, seed, hq, hkv, d, n_prompt, chunk, n_received, page, obs. window, sliding window
    ("w1", 600, 2, 2, 128, 300, 128, 3, 64, "all", 1),
    ("w37_d64", 601, 4, 4, 64, 300, 77, 5, 64, "all", 37),
    ("w128_g4", 602, 8, 2, 128, 700, 256, 9, 64, "all", 128),
    ("w129_g4", 603, 8, 2, 128, 700, 256, 9, 64, "last", 129),
    ("w200_g6", 604, 12, 2, 128, 900, 400, 33, 128, "all", 200),
    ("w256_g1_rowpairs", 605, 3, 3, 128, 1100, 512, 7, 64, "all", 256),
    ("w500_multi_tile_chunk", 606, 4, 1, 128, 1500, 700, 17, 64, "last", 500),
    ("w1000_d64_page128", 607, 8, 8, 64, 1300, 650, 1, 128, "all", 1000),
]


def _with_window(w, sw):
    return dataclasses.replace(w, sliding_window=sw)


@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("case", CASES, ids=[c[0] for c in CASES])
def test_banded_cases_match_checker(case, path):
    name, seed, hq, hkv, d, n_prompt, chunk, n_recv, page, window, sw = case
    w = _with_window(wl.small_like(name, seed, hq, hkv, d, n_prompt, chunk, n_recv, keep_ratio=0.3,
                                   window=window, page_tokens=page), sw)
    got = H.run_library(w, kernel_path=path)
    H.compare_full(w, got, H.oracle_full(w))


@pytest.mark.parametrize("path", PATHS)
def test_ragged_batch_with_band(path):
    w = _with_window(wl.ragged_batch("ragged_band", 6, 8, 2, 128, 5, 40, 900, 128, 20, 0.4,
                                     window="all"), 150)
    got = H.run_library(w, kernel_path=path)
    H.compare_full(w, got, H.oracle_full(w))


def test_window_longer_than_sequence_is_the_plain_path():
    base = wl.small_like("band_off", 610, 8, 2, 128, 900, 300, 11, window="all")
    plain = H.run_library(base, kernel_path=0)
    wide = H.run_library(_with_window(base, 5000), kernel_path=0)
    np.testing.assert_array_equal(plain[0]["out"], wide[0]["out"])
    np.testing.assert_array_equal(plain[0]["colsum"], wide[0]["colsum"])
    np.testing.assert_array_equal(plain[0]["keep"], wide[0]["keep"])


def test_long_sequence_with_band_sampled():
    """8k-token prompt in 2048-row chunks (many CTAs share key ranges), w = 1024: sampled
    rows against the checker, column sums of sampled heads, and the mass identity
    sum_j colsum[h][j] = number of window rows."""
    from oracle import pdd_oracle as orc
    w = _with_window(wl.small_like("band_8k", 611, 8, 2, 128, 8192, 2048, 64, keep_ratio=0.25,
                                   window="last"), 1024)
    s = w.seqs[0]
    got = H.run_library(w, kernel_path=0)[0]
    rows = np.unique(np.concatenate([[0, 1, 127, 128, 1023, 1024, 1025, 2047, 2048, s.n_tokens - 1],
                                     wl.rng_for(612).integers(0, s.n_tokens, 40)]))
    q64, k64, v64 = (x.astype(np.float64) for x in (s.q, s.k, s.v))
    want, _ = orc.attention_rows(q64, k64, v64, w.softmax_scale, rows, 1024)
    H.check_out(got["out"][rows], want, "8k band sampled rows")
    win = H.window_mask(s)
    atol = H.imp_atol(int(win.sum()), w.n_q_heads, s.n_tokens) / w.n_q_heads
    for h in (0, 5):
        g = h // 4
        want_cs = orc.colsum(q64[:, h:h + 1], k64[:, g:g + 1], w.softmax_scale, win, 1024)[0]
        H.check_importance(got["colsum"][h], want_cs, atol, "8k band colsum head %d" % h)
        assert (got["colsum"][h][: int(np.flatnonzero(win)[0]) - 1023] == 0).all()
    np.testing.assert_allclose(got["colsum"].sum(axis=1), float(win.sum()), rtol=2e-3)
