"""Error paths on the GPU, exercised without hanging or faulting anything: a bounded wait
that runs out (a short limit on a barrier nobody arrives at), the sticky status word and
what the hot kernels do once it is set, a failed enqueue step injected on the host, and
malformed sentence boundaries in device memory."""
import numpy as np
import pytest

from paper_2508_09035_b200 import workloads as wl
from tests import helpers as H

pytestmark = pytest.mark.gpu


def _small():
    return wl.small_like("err", 700, 8, 2, 128, 600, 200, 8, keep_ratio=0.3, window="last")


def _feed(kv, s, calls, out=None):
    outs = []
    for c in calls:
        sl = slice(c.pos0, c.pos0 + c.length)
        fn = kv.prefill_chunk if c.kind == wl.PROMPT else kv.append_received
        outs.append(fn(H.to_dev(s.q[sl]), H.to_dev(s.k[sl]), H.to_dev(s.v[sl]), window=c.window))
    return outs


def test_bounded_wait_expiry_sets_the_sticky_word_and_later_kernels_do_nothing():
    import torch
    from oracle import pdd_oracle as orc
    from paper_2508_09035_b200 import binding as B
    w = _small()
    s = w.seqs[0]
    kv = H.make_cache(w, 0)
    _feed(kv, s, s.calls[:1])
    assert kv.status() == B.PDD_OK
    # a wait that can never be satisfied gives up after one millisecond and reports it
    B.pdd_selftest_wait_timeout(kv.h, 1000, kv.stream)
    assert kv.status() == B.PDD_ERR_TIMEOUT
    assert B.lib().pdd_strerror(B.PDD_ERR_TIMEOUT).decode() == "a bounded device-side wait ran out"
    # the next hot call is accepted by the host but its kernels return at once
    c = s.calls[1]
    sl = slice(c.pos0, c.pos0 + c.length)
    out = torch.full((c.length, w.n_q_heads, w.head_dim), 7.0, dtype=torch.bfloat16, device="cuda:0")
    kv.prefill_chunk(H.to_dev(s.q[sl]), H.to_dev(s.k[sl]), H.to_dev(s.v[sl]), window=c.window, out=out)
    torch.cuda.synchronize()
    assert (out.float() == 7.0).all(), "a kernel wrote its output although the status word was set"
    assert kv.status() == B.PDD_ERR_TIMEOUT          # sticky
    # clearing the word and resetting the sequence makes the handle usable again
    B.pdd_clear_status(kv.h, kv.stream)
    kv.reset(0)
    assert kv.status() == B.PDD_OK
    outs = _feed(kv, s, s.calls)
    want, _ = orc.attention(s.q, s.k, s.v, w.softmax_scale)
    got = np.concatenate([H.from_dev_bf16(o) for o in outs])
    H.check_out(got, want, "after clear + reset")
    kv.close()
    # and a fresh handle is not affected at all
    kv2 = H.make_cache(w, 0)
    outs = _feed(kv2, s, s.calls)
    H.check_out(np.concatenate([H.from_dev_bf16(o) for o in outs]), want, "fresh handle")
    assert kv2.status() == B.PDD_OK
    kv2.close()


def test_selftest_argument_checks():
    from paper_2508_09035_b200 import binding as B
    w = _small()
    kv = H.make_cache(w, 0)
    for bad in (0, 100001):
        with pytest.raises(B.PddError) as e:
            B.pdd_selftest_wait_timeout(kv.h, bad, kv.stream)
        assert e.value.status == B.PDD_ERR_INVALID
    assert kv.status() == B.PDD_OK
    kv.close()


@pytest.mark.parametrize("nth", [1, 2, 3])
def test_failed_enqueue_step_leaves_the_host_state_unchanged(nth):
    """The nth enqueue step of a call (kv_append, attention, column sums) is made to fail on the
    host: the call returns PDD_ERR_CUDA, the sequence length and the page pool are as before,
    and repeating the same call gives the right result."""
    from oracle import pdd_oracle as orc
    from paper_2508_09035_b200 import binding as B
    w = _small()
    s = w.seqs[0]
    kv = H.make_cache(w, 0)
    n_before = len(s.calls) - 2          # fail the last prompt chunk (it is a window call)
    outs = _feed(kv, s, s.calls[:n_before])
    c = s.calls[n_before]
    assert c.window
    sl = slice(c.pos0, c.pos0 + c.length)
    B.pdd_debug_fail_launch(kv.h, nth)
    with pytest.raises(B.PddError) as e:
        kv.prefill_chunk(H.to_dev(s.q[sl]), H.to_dev(s.k[sl]), H.to_dev(s.v[sl]), window=True)
    assert e.value.status == B.PDD_ERR_CUDA
    assert kv.length(0) == c.pos0
    B.pdd_debug_fail_launch(kv.h, 0)
    if nth == 3:
        # attention ran and only the column sums were refused: they are still all zero
        assert float(kv.export_colsum(0).abs().sum().item()) == 0.0
    outs += _feed(kv, s, s.calls[n_before:])
    assert kv.length(0) == s.n_tokens
    want, _ = orc.attention(s.q, s.k, s.v, w.softmax_scale)
    H.check_out(np.concatenate([H.from_dev_bf16(o) for o in outs]), want, "after a failed call")
    cs = orc.colsum(s.q, s.k, w.softmax_scale, H.window_mask(s))
    atol = H.imp_atol(int(H.window_mask(s).sum()), w.n_q_heads, s.n_tokens)
    H.check_importance(kv.export_colsum(0).cpu().numpy().astype(np.float64), cs,
                       atol / w.n_q_heads, "column sums after a failed call")
    assert kv.status() == B.PDD_OK
    kv.close()


def test_malformed_sentence_boundaries_are_refused_in_the_kernel():
    import torch
    from paper_2508_09035_b200 import binding as B
    n = 1000
    score = torch.rand(n, dtype=torch.float32, device="cuda:0")
    guard = torch.full((n + 64,), 9, dtype=torch.uint8, device="cuda:0")
    keep = guard[:n]
    n_kept = torch.zeros(1, dtype=torch.int32, device="cuda:0")
    for seg in ([0, 100, 50, 1000],          # decreasing
                [0, 100, 2000],              # beyond n
                [-5, 100, 1000],             # negative
                [0, 100, 1000, 1 << 30]):    # far beyond n
        d_seg = torch.tensor(seg, dtype=torch.int32, device="cuda:0")
        guard.fill_(9)
        B.pdd_refine_sentences(score.data_ptr(), None, n, d_seg.data_ptr(), len(seg) - 1, 0.5,
                               keep.data_ptr(), n_kept.data_ptr(), None,
                               torch.cuda.current_stream().cuda_stream)
        torch.cuda.synchronize()
        assert int(n_kept.item()) == -1
        assert int(keep.sum().item()) == 0
        assert (guard[n:] == 9).all(), "wrote past the end of keep"
    # well-formed boundaries still work afterwards
    d_seg = torch.tensor([10, 100, 500, 990], dtype=torch.int32, device="cuda:0")
    B.pdd_refine_sentences(score.data_ptr(), None, n, d_seg.data_ptr(), 3, 0.5, keep.data_ptr(),
                           n_kept.data_ptr(), None, torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    assert int(n_kept.item()) == int(keep.sum().item()) > 0
