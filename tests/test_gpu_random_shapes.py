"""GPU parity on seeded random shapes: head counts and GQA group sizes (even and odd), both head
dims and page sizes, ragged prompt lengths and chunk sizes, received tokens at the end or after
every chunk, both observation windows, a sliding window now and then, every attention schedule.
Each case is compared element by element with the checker (outputs, column sums, scores, mask)."""
import dataclasses

import numpy as np
import pytest

from paper_2508_09035_b200 import workloads as wl
from tests import helpers as H

pytestmark = pytest.mark.gpu


def _case(i: int):
    rng = wl.rng_for(9000 + i)
    hkv = int(rng.choice([1, 2, 3, 4, 8]))
    G = int(rng.choice([1, 2, 3, 4, 6]))
    d = int(rng.choice([64, 128]))
    page = int(rng.choice([64, 128]))
    n_prompt = int(rng.integers(1, 1400))
    chunk = int(rng.integers(1, 700))
    n_recv = int(rng.integers(0, 70))
    window = str(rng.choice(["last", "all"]))
    sliding = int(rng.integers(16, 900)) if rng.random() < 0.3 else 0
    mode = int(rng.integers(0, 4))
    keep = float(rng.choice([0.1, 0.3, 0.5, 0.9]))
    return dict(hq=hkv * G, hkv=hkv, d=d, page=page, n_prompt=n_prompt, chunk=chunk, n_recv=n_recv,
                window=window, sliding=sliding, mode=mode, keep=keep)


@pytest.mark.parametrize("i", range(48))
def test_random_single_sequence(i):
    c = _case(i)
    w = wl.small_like("rand%d" % i, 9100 + i, c["hq"], c["hkv"], c["d"], c["n_prompt"], c["chunk"],
                      c["n_recv"], keep_ratio=c["keep"], window=c["window"], page_tokens=c["page"])
    w = dataclasses.replace(w, sliding_window=c["sliding"])
    kv = H.make_cache(w, 0)
    kv.set_schedule(c["mode"])
    got = H.run_library(w, cache=kv)
    kv.close()
    H.compare_full(w, got, H.oracle_full(w), what=str(c))


@pytest.mark.parametrize("i", range(16))
def test_random_ragged_batch(i):
    rng = wl.rng_for(9500 + i)
    hkv = int(rng.choice([1, 2, 4]))
    G = int(rng.choice([1, 2, 3, 4]))
    d = int(rng.choice([64, 128]))
    n_seqs = int(rng.integers(2, 12))
    len_hi = int(rng.integers(40, 900))
    chunk = int(rng.choice([64, 128, 192, 100]))
    w = wl.ragged_batch("randb%d" % i, 9600 + i, hkv * G, hkv, d, n_seqs, 1, len_hi, chunk,
                        int(rng.integers(0, 40)), float(rng.choice([0.2, 0.5])),
                        window=str(rng.choice(["last", "all"])), page_tokens=int(rng.choice([64, 128])))
    kv = H.make_cache(w, 0)
    kv.set_schedule(int(rng.integers(0, 4)))
    got = H.run_library(w, cache=kv)
    kv.close()
    H.compare_full(w, got, H.oracle_full(w), what="batch %d" % i)


@pytest.mark.parametrize("hq,hkv,d", [(11, 1, 128), (12, 1, 64), (16, 1, 128), (32, 2, 128), (40, 2, 64)])
def test_large_gqa_groups(hq, hkv, d):
    """Groups of more than eight query heads: the column-sum kernel keeps at most eight heads'
    partial sums per CTA and deals the rest out to further CTAs (a prime group size leaves one
    head per CTA)."""
    w = wl.small_like("gqa%d_%d" % (hq, hkv), 9900 + hq, hq, hkv, d, 520, 200, 24, keep_ratio=0.4,
                      window="all", page_tokens=64)
    kv = H.make_cache(w, 0)
    got = H.run_library(w, cache=kv)
    kv.close()
    H.compare_full(w, got, H.oracle_full(w), what="hq %d hkv %d d %d" % (hq, hkv, d))
