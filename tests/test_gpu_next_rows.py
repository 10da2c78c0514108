"""GPU parity of sentence-level selection and the mask bit stream (byte/index work: the bar
is bit-exact).  The library forms the sentence means in fp32; the checker is the fp64
definition.  Where the checker's values separate every pair of sentences by more than the
fp32 evaluation error, both sides visit the sentences in the same order and the mask must be
equal bit for bit; where two means nearly tie, several visiting orders are correct, and the
test then checks the values (within tolerance) and that the mask is the exact first-fit
selection for the values the library reported."""
import numpy as np
import pytest

from paper_2508_09035_b200 import workloads as wl
from tests import helpers as H

pytestmark = pytest.mark.gpu


def _sentences(rng, lo, hi, mean_len):
    cuts = [lo]
    while cuts[-1] < hi:
        cuts.append(min(hi, cuts[-1] + 1 + int(rng.poisson(mean_len))))
    return np.asarray(cuts, dtype=np.int32)


def _run_sentences(score, kind, seg, ratio):
    import torch
    from paper_2508_09035_b200 import binding as B
    n = len(score)
    d_score = torch.from_numpy(score).cuda()
    d_kind = torch.from_numpy(kind).cuda() if kind is not None else None
    d_seg = torch.from_numpy(seg).cuda()
    keep = torch.full((n,), 9, dtype=torch.uint8, device="cuda:0")
    n_kept = torch.full((1,), -1, dtype=torch.int32, device="cuda:0")
    val = torch.zeros(len(seg) - 1, dtype=torch.float32, device="cuda:0")
    B.pdd_refine_sentences(d_score.data_ptr(), d_kind.data_ptr() if kind is not None else None, n,
                           d_seg.data_ptr(), len(seg) - 1, ratio, keep.data_ptr(),
                           n_kept.data_ptr(), val.data_ptr(),
                           torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    return keep.cpu().numpy(), int(n_kept.item()), val.cpu().numpy()


SENT_REL = 1e-5      # fp32 mean of up to ~100 terms against the fp64 mean


def _check_sentences(score, kind, seg, ratio, what):
    """Library against the fp64 checker; returns the number of near-tie pairs."""
    from oracle import pdd_oracle as orc
    keep, n_kept, val = _run_sentences(score, kind, seg, ratio)
    want, want_n, taken = orc.refine_sentences(score, kind, seg, ratio)
    v64, cnt = orc.sentence_values(score, kind, seg)
    np.testing.assert_allclose(val[cnt > 0], v64[cnt > 0], rtol=SENT_REL, err_msg=what)
    assert n_kept == int(keep.sum())
    ties = H.sentence_near_ties(v64, cnt, 4 * SENT_REL)
    if ties == 0:
        np.testing.assert_array_equal(keep, want, err_msg=what + " (no near-tie)")
        assert n_kept == want_n
    # the mask is the exact first-fit selection for the values the library formed
    own = orc.select_sentences(np.where(cnt > 0, val.astype(np.float64), -np.inf), cnt,
                               H.sentence_budget(kind, seg, ratio))
    own_keep = np.zeros(len(score), np.uint8)
    pos = np.arange(len(score))
    own_keep[(kind == 0) & ((pos < seg[0]) | (pos >= seg[-1]))] = 1
    for s in np.nonzero(own)[0]:
        sl = slice(int(seg[s]), int(seg[s + 1]))
        own_keep[sl] = kind[sl] == 0
    np.testing.assert_array_equal(keep, own_keep, err_msg=what + " (own values)")
    # secondary: the reported values are the sequential fp32 means, bit for bit
    v32, _ = H.replay_sentence_values_f32(score, kind, seg)
    np.testing.assert_array_equal(val[cnt > 0], v32[cnt > 0])
    return ties


@pytest.mark.parametrize("n,mean_len,n_levels", [(12, 2, 4), (300, 5, 40), (4160, 24, 4000),
                                                  (33024, 30, 8), (33024, 30, 4000)])
def test_sentence_selection_equals_fp64_checker_on_separated_values(n, mean_len, n_levels):
    """Sentence means that are exact in fp32 and in fp64 (tokens = level +- dyadic offsets that
    cancel, levels multiples of 2^-12): distinct levels differ by far more than any rounding and
    equal levels tie exactly on both sides, so the mask must equal the fp64 checker's."""
    rng = wl.rng_for(430 + n + mean_len + n_levels)
    for ratio in (0.0, 0.2, 0.5, 1.0):
        kind = (rng.random(n) < 0.05).astype(np.uint8)
        lo, hi = int(rng.integers(0, n // 10 + 1)), n - int(rng.integers(0, n // 10 + 1))
        seg = _sentences(rng, lo, hi, mean_len)
        score = rng.random(n).astype(np.float32)
        for s in range(len(seg) - 1):
            level = (64 + int(rng.integers(0, n_levels))) * 2.0 ** -12
            idx = [i for i in range(seg[s], seg[s + 1]) if kind[i] == 0]
            vals = np.full(len(idx), level)
            for a in range(0, len(idx) - 1, 2):          # offsets in cancelling pairs
                off = int(rng.integers(0, 8)) * 2.0 ** -12
                vals[a] += off
                vals[a + 1] -= off
            score[idx] = vals
        ties = _check_sentences(score, kind, seg, ratio, "separated n=%d r=%g" % (n, ratio))
        assert ties == 0


@pytest.mark.parametrize("n,mean_len", [(12, 2), (300, 5), (4160, 24), (33024, 30), (33024, 5)])
def test_sentence_selection_on_random_scores(n, mean_len):
    rng = wl.rng_for(400 + n + mean_len)
    for ratio in (0.0, 0.2, 0.5, 1.0):
        score = (rng.random(n) ** 4).astype(np.float32)
        if ratio == 0.5:
            score = (np.round(score * 4) / 4).astype(np.float32)       # many ties
        kind = (rng.random(n) < 0.05).astype(np.uint8)
        lo, hi = int(rng.integers(0, n // 10 + 1)), n - int(rng.integers(0, n // 10 + 1))
        seg = _sentences(rng, lo, hi, mean_len)
        if len(seg) - 1 > 8192:
            continue
        _check_sentences(score, kind, seg, ratio, "random n=%d r=%g" % (n, ratio))


def test_sentence_selection_on_library_scores():
    """End of the path: scores from the attention column sums, then whole sentences."""
    import torch
    from oracle import pdd_oracle as orc
    w = wl.small_like("sent", 410, 8, 2, 128, 900, 256, 20, keep_ratio=0.3, window="last")
    s = w.seqs[0]
    kv = H.make_cache(w, 0)
    for c in s.calls:
        sl = slice(c.pos0, c.pos0 + c.length)
        fn = kv.prefill_chunk if c.kind == wl.PROMPT else kv.append_received
        fn(H.to_dev(s.q[sl]), H.to_dev(s.k[sl]), H.to_dev(s.v[sl]), window=c.window)
    score = kv.token_importance(0).cpu().numpy()
    seg = _sentences(wl.rng_for(411), 64, 880, 20)
    _check_sentences(score, s.kind, seg, 0.3, "library scores")
    keep, n_kept, val = _run_sentences(score, s.kind, seg, 0.3)
    assert keep[:64][s.kind[:64] == 0].all() and not keep[s.kind == 1].any()
    kv.close()


def test_sentence_limits():
    import torch
    from paper_2508_09035_b200 import binding as B
    z = torch.zeros(16, dtype=torch.float32, device="cuda:0")
    seg = torch.zeros(8194, dtype=torch.int32, device="cuda:0")
    k = torch.zeros(16, dtype=torch.uint8, device="cuda:0")
    nk = torch.zeros(1, dtype=torch.int32, device="cuda:0")
    with pytest.raises(B.PddError) as e:
        B.pdd_refine_sentences(z.data_ptr(), None, 16, seg.data_ptr(), 8193, 0.5, k.data_ptr(),
                               nk.data_ptr(), None, 0)
    assert e.value.status == B.PDD_ERR_CAPACITY
    with pytest.raises(B.PddError) as e:
        B.pdd_refine_sentences(z.data_ptr(), None, 16, seg.data_ptr(), 0, 0.5, k.data_ptr(),
                               nk.data_ptr(), None, 0)
    assert e.value.status == B.PDD_ERR_INVALID


@pytest.mark.parametrize("n", [1, 7, 8, 9, 1000, 4160, 33025])
def test_pack_mask_bits(n):
    import torch
    from oracle import pdd_oracle as orc
    from paper_2508_09035_b200 import binding as B
    keep = (wl.rng_for(420 + n).random(n) < 0.3).astype(np.uint8)
    d_keep = torch.from_numpy(keep).cuda()
    bits = torch.full(((n + 7) // 8,), 0xAA, dtype=torch.uint8, device="cuda:0")
    B.pdd_pack_mask(d_keep.data_ptr(), n, bits.data_ptr(), torch.cuda.current_stream().cuda_stream)
    np.testing.assert_array_equal(bits.cpu().numpy(), orc.pack_mask_bits(keep))
