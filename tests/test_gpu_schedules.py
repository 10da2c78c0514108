"""GPU parity of each way the attention kernel's work is cut among CTAs (whole tile pairs,
equal shares merged by a second kernel, one thread-block cluster per pair merged through
distributed shared memory, the pair-of-CTAs kernel where the shape allows it), forced one at
a time on workloads the cost model would send elsewhere: even and odd GQA group sizes, both head dims, ragged tails, pairs with fewer key
blocks than cluster CTAs, a batch of sequences, and the sliding window."""
import dataclasses

import numpy as np
import pytest

from paper_2508_09035_b200 import workloads as wl
from tests import helpers as H

pytestmark = pytest.mark.gpu

MODES = [1, 2, 3, 4]

CASES = [
    # name, seed, hq, hkv, d, n_prompt, chunk, n_received, page, obs. window, sliding window
    ("one_block", 700, 2, 2, 128, 100, 100, 0, 64, "all", 0),
    ("g4_d128", 701, 8, 2, 128, 1000, 384, 9, 64, "last", 0),
    ("g1_rowpairs_d64", 702, 3, 3, 64, 1100, 500, 7, 64, "all", 0),
    ("g3_rowpairs_d128", 703, 3, 1, 128, 900, 300, 5, 128, "all", 0),
    ("few_pairs_long", 704, 2, 1, 128, 2300, 256, 40, 64, "last", 0),
    ("band_g4", 705, 8, 2, 128, 1500, 512, 9, 64, "all", 300),
    ("band_rowpairs", 706, 3, 3, 128, 1400, 700, 3, 64, "all", 200),
    ("g8_long_d128", 707, 16, 2, 128, 3000, 1024, 40, 64, "last", 0),
    ("g4_ragged_tail", 708, 4, 1, 128, 1333, 777, 21, 128, "all", 0),
]


@pytest.mark.parametrize("mode", MODES)
@pytest.mark.parametrize("case", CASES, ids=[c[0] for c in CASES])
def test_forced_schedule_matches_checker(case, mode):
    name, seed, hq, hkv, d, n_prompt, chunk, n_recv, page, window, sw = case
    w = dataclasses.replace(wl.small_like(name, seed, hq, hkv, d, n_prompt, chunk, n_recv,
                                          keep_ratio=0.3, window=window, page_tokens=page),
                            sliding_window=sw)
    kv = H.make_cache(w, 0)
    kv.set_schedule(mode)
    got = H.run_library(w, cache=kv)
    kv.close()
    H.compare_full(w, got, H.oracle_full(w))


@pytest.mark.parametrize("mode", MODES)
def test_forced_schedule_ragged_batch(mode):
    w = wl.ragged_batch("ragged_sched", 7, 8, 2, 128, 4, 60, 700, 128, 12, 0.4, window="all")
    kv = H.make_cache(w, 0)
    kv.set_schedule(mode)
    got = H.run_library(w, cache=kv)
    kv.close()
    H.compare_full(w, got, H.oracle_full(w))


def test_schedules_agree_with_each_other():
    """Same inputs, four cuts: outputs differ only by the rounding order of the merge."""
    w = wl.small_like("sched_agree", 710, 8, 2, 128, 1200, 400, 16, window="all")
    res = []
    for mode in (1, 2, 3, 4):
        kv = H.make_cache(w, 0)
        kv.set_schedule(mode)
        res.append(H.run_library(w, cache=kv)[0])
        kv.close()
    for other in res[1:]:
        assert np.abs(other["out"] - res[0]["out"]).max() <= 2 ** -6      # a bf16 ulp near 2
        np.testing.assert_allclose(other["colsum"], res[0]["colsum"], rtol=1e-4, atol=1e-6)


def test_bad_schedule_mode_is_rejected():
    from paper_2508_09035_b200 import binding as B
    w = wl.small_like("sched_bad", 711, 2, 2, 64, 10, 10, 0)
    kv = H.make_cache(w, 0)
    with pytest.raises(B.PddError) as e:
        kv.set_schedule(5)
    assert e.value.status == B.PDD_ERR_INVALID
    kv.close()
