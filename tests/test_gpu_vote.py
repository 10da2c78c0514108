"""GPU parity of per-head selection with a vote (index work: the bar is bit-exact).  The
library pools and adds heads in fp32; the checker is the fp64 definition.  The inputs are
chosen so that every per-head decision is exact in fp32 (no pooling, max pooling, or
average pooling of multiples of 1/8), hence the vote counts must agree exactly; the head sum
that orders equal vote counts carries fp32 rounding, so the mask must agree outside the
near-tie band around the threshold's head sum and have the same popcount."""
import numpy as np
import pytest

from paper_2508_09035_b200 import workloads as wl
from tests import helpers as H

pytestmark = pytest.mark.gpu

POOLS = {"none": 0, "avg": 1, "max": 2}


def _run_vote(cs, kind, lo, hi, ratio, pool, width, ld_pad=0):
    import torch
    from paper_2508_09035_b200 import binding as B
    heads, n = cs.shape
    ld = n + ld_pad
    buf = np.full((heads, ld), 7.0, dtype=np.float32)
    buf[:, :n] = cs
    d_cs = torch.from_numpy(buf).cuda()
    d_kind = torch.from_numpy(kind).cuda() if kind is not None else None
    keep = torch.full((n,), 9, dtype=torch.uint8, device="cuda:0")
    n_kept = torch.full((1,), -1, dtype=torch.int32, device="cuda:0")
    votes = torch.full((n,), -1, dtype=torch.int32, device="cuda:0")
    nbytes = B.pdd_refine_vote_workspace(heads, n)
    work = torch.empty(nbytes + 256, dtype=torch.uint8, device="cuda:0")
    wptr = (work.data_ptr() + 255) & ~255
    B.pdd_refine_vote(d_cs.data_ptr(), ld, heads, d_kind.data_ptr() if kind is not None else None,
                      n, POOLS[pool], width, lo, hi, ratio, keep.data_ptr(), n_kept.data_ptr(),
                      votes.data_ptr(), wptr, nbytes, torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    return keep.cpu().numpy(), int(n_kept.item()), votes.cpu().numpy()


@pytest.mark.parametrize("n,heads", [(9, 3), (300, 8), (4160, 32), (33024, 32), (5000, 70)])
def test_vote_matches_fp64_checker(n, heads):
    from oracle import pdd_oracle as orc
    rng = wl.rng_for(600 + n + heads)
    cases = [(0.0, "none", 1), (0.3, "none", 1), (0.5, "max", 3), (1.0, "none", 1)]
    if n <= 5000:
        cases.append((0.4, "avg", 5))
    for ratio, pool, width in cases:
        # heavy-tailed column sums, heads that agree on some positions and differ on others
        shared = rng.random(n) ** 6
        cs = (0.5 * shared[None, :] + rng.random((heads, n)) ** 4).astype(np.float32)
        if ratio == 0.5 or pool == "avg":
            cs = (np.round(cs * 8) / 8).astype(np.float32)   # exact ties; exact fp32 window sums
        kind = (rng.random(n) < 0.05).astype(np.uint8)
        lo, hi = int(rng.integers(0, n // 10 + 1)), n - int(rng.integers(0, n // 10 + 1))
        keep, n_kept, votes = _run_vote(cs, kind, lo, hi, ratio, pool, width, ld_pad=int(n % 7))
        want, want_n, want_votes, total = orc.refine_vote(cs, kind, lo, hi, ratio, pool, width)
        band = H.check_vote_keep(keep, n_kept, votes, want, want_n, want_votes, total, kind, lo,
                                 hi, heads, "vote n=%d heads=%d r=%g %s" % (n, heads, ratio, pool))
        assert band <= max(8, n // 50), "near-tie band of %d positions: the check is vacuous" % band
        if pool != "avg":
            # multiples of 1/8 add exactly in fp32 too: there the mask is the checker's, bit for bit
            if ratio == 0.5:
                np.testing.assert_array_equal(keep, want)


def test_vote_on_library_column_sums():
    """End of the path: column sums from the attention pass, exported, then the vote."""
    import torch
    from oracle import pdd_oracle as orc
    w = wl.small_like("vote", 610, 8, 2, 128, 900, 256, 20, keep_ratio=0.3, window="last")
    s = w.seqs[0]
    kv = H.make_cache(w, 0)
    for c in s.calls:
        sl = slice(c.pos0, c.pos0 + c.length)
        fn = kv.prefill_chunk if c.kind == wl.PROMPT else kv.append_received
        fn(H.to_dev(s.q[sl]), H.to_dev(s.k[sl]), H.to_dev(s.v[sl]), window=c.window)
    cs = kv.export_colsum(0).cpu().numpy()
    keep, n_kept, votes = _run_vote(cs, s.kind, 16, 880, 0.3, "none", 1)
    want, want_n, want_votes, total = orc.refine_vote(cs, s.kind, 16, 880, 0.3)
    band = H.check_vote_keep(keep, n_kept, votes, want, want_n, want_votes, total, s.kind, 16,
                             880, 8, "vote on library column sums")
    assert band <= 8
    assert n_kept == orc.keep_count(0.3, s.n_prompt)
    assert not keep[s.kind == 1].any()
    kv.close()


def test_vote_argument_checks():
    import torch
    from paper_2508_09035_b200 import binding as B
    z = torch.zeros(64, dtype=torch.float32, device="cuda:0")
    k = torch.zeros(16, dtype=torch.uint8, device="cuda:0")
    nk = torch.zeros(1, dtype=torch.int32, device="cuda:0")
    work = torch.zeros(1 << 16, dtype=torch.uint8, device="cuda:0")
    wptr = (work.data_ptr() + 255) & ~255
    with pytest.raises(B.PddError) as e:      # workspace too small
        B.pdd_refine_vote(z.data_ptr(), 16, 4, None, 16, 0, 1, 0, 16, 0.5, k.data_ptr(),
                          nk.data_ptr(), None, wptr, 64, 0)
    assert e.value.status == B.PDD_ERR_CAPACITY
    with pytest.raises(B.PddError) as e:      # too many heads for the 8-bit vote field
        B.pdd_refine_vote_workspace(256, 16)
    assert e.value.status == B.PDD_ERR_INVALID
    with pytest.raises(B.PddError) as e:      # ld < n
        B.pdd_refine_vote(z.data_ptr(), 8, 4, None, 16, 0, 1, 0, 16, 0.5, k.data_ptr(),
                          nk.data_ptr(), None, wptr, 1 << 15, 0)
    assert e.value.status == B.PDD_ERR_INVALID
