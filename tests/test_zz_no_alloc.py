"""pdd_refine_from_colsum_static: the allocation-free importance + top-k call.

Some users of this library run as a plug-in inside a serving engine that has handed out
all device memory at start-up: they own the column sums and the mask buffer, but they have
no allocator for the intermediate score vector and must not call cudaMalloc while a request
is being served.  For them the library keeps the score vector in a fixed buffer of its own.
This file checks, through the C ABI, that the call gives exactly the mask and count of the
two-step path (pdd_token_importance into a caller-owned vector, then pdd_refine_topk), on
two calls in a row that share the buffer (the second on a shorter sequence, so stale
contents of the first call sit right behind its data), and that it refuses sequences
longer than the buffer.  It is collected last on purpose.
"""
import numpy as np
import pytest

from paper_2508_09035_b200 import workloads as wl
from tests import helpers as H

pytestmark = pytest.mark.gpu


def _prefill(w, kernel_path=0):
    s = w.seqs[0]
    kv = H.make_cache(w, kernel_path)
    for c in s.calls:
        sl = slice(c.pos0, c.pos0 + c.length)
        fn = kv.prefill_chunk if c.kind == wl.PROMPT else kv.append_received
        fn(H.to_dev(s.q[sl]), H.to_dev(s.k[sl]), H.to_dev(s.v[sl]), window=c.window)
    return kv


def _both_paths(kv, n, keep_ratio, pool_kind, pool_k, lo, hi):
    import torch
    from paper_2508_09035_b200 import binding as B
    stream = kv.stream
    # existing path: caller-owned score vector
    score = kv.token_importance(0, pool_kind, pool_k)
    keep_ref, n_ref = kv.refine_topk(score, keep_ratio, 0, lo, hi)
    # new path: inputs and outputs from the caller, score vector inside the library
    colsum = kv.export_colsum(0)
    keep = torch.full((n,), 7, dtype=torch.uint8, device="cuda:0")
    n_kept = torch.full((1,), -1, dtype=torch.int32, device="cuda:0")
    B.pdd_refine_from_colsum_static(colsum.data_ptr(), colsum.shape[1], colsum.shape[0],
                                    kv.kinds_ptr(0), n, pool_kind, pool_k, lo, hi, keep_ratio,
                                    keep.data_ptr(), n_kept.data_ptr(), stream)
    torch.cuda.synchronize()
    return keep_ref.cpu().numpy(), int(n_ref.item()), keep.cpu().numpy(), int(n_kept.item())


def test_static_buffer_call_matches_two_step_path_twice_in_a_row():
    from paper_2508_09035_b200 import binding as B
    # first call: 1200 + 40 positions, average pooling, a candidate range with prefix/suffix
    w1 = wl.small_like("noalloc_a", 900, 8, 2, 128, 1200, 512, 40, keep_ratio=0.3, window="all")
    kv1 = _prefill(w1)
    n1 = w1.seqs[0].n_tokens
    ref, n_ref, got, n_got = _both_paths(kv1, n1, 0.3, B.PDD_POOL_AVG, 7, 100, 1100)
    np.testing.assert_array_equal(got, ref)
    assert n_got == n_ref == int(ref.sum()) and n_ref == 360
    # second call right after it, shorter sequence, no pooling: the buffer still holds the
    # first call's scores beyond position n2
    w2 = wl.small_like("noalloc_b", 901, 4, 4, 64, 300, 128, 5, keep_ratio=0.5, window="last")
    kv2 = _prefill(w2)
    n2 = w2.seqs[0].n_tokens
    ref, n_ref, got, n_got = _both_paths(kv2, n2, 0.5, B.PDD_POOL_NONE, 1, 0, n2)
    np.testing.assert_array_equal(got, ref)
    assert n_got == n_ref == 150
    # the same answer straight from the CPU checker: its importance (fp64 column sums of the
    # library's own fp32 column sums, no pooling) and its stable-sort top-k; heads are added in
    # fp32 on the GPU, so positions within that rounding of the threshold may differ
    from oracle import pdd_oracle as orc
    cs = kv2.export_colsum(0).cpu().numpy().astype(np.float64)
    score64 = orc.importance([cs])
    s2 = w2.seqs[0]
    want, want_n, k = orc.refine_topk(score64, s2.kind, 0, n2, 0.5)
    assert n_got == want_n
    theta = np.sort(score64[s2.kind == 0])[::-1][k - 1]
    near = np.abs(score64 - theta) <= 1e-6 * abs(theta)
    np.testing.assert_array_equal(got[~near], want[~near])
    assert int(near.sum()) <= 4
    # and the first problem again gives the same answer as before
    ref1, n_ref1, got1, n_got1 = _both_paths(kv1, n1, 0.3, B.PDD_POOL_AVG, 7, 100, 1100)
    np.testing.assert_array_equal(got1, ref1)
    assert n_got1 == n_ref1 == 360
    kv1.close()
    kv2.close()


def test_static_buffer_call_rejects_sizes_beyond_its_buffer():
    import torch
    from paper_2508_09035_b200 import binding as B
    n = B.PDD_STATIC_SCORE_MAX + 1
    colsum = torch.zeros((1, n), dtype=torch.float32, device="cuda:0")
    keep = torch.full((n,), 7, dtype=torch.uint8, device="cuda:0")
    n_kept = torch.full((1,), -1, dtype=torch.int32, device="cuda:0")
    with pytest.raises(B.PddError) as e:
        B.pdd_refine_from_colsum_static(colsum.data_ptr(), n, 1, None, n, 0, 1, 0, n, 0.5,
                                        keep.data_ptr(), n_kept.data_ptr(),
                                        torch.cuda.current_stream().cuda_stream)
    assert e.value.status == B.PDD_ERR_CAPACITY and "at most 65536" in str(e.value)
    torch.cuda.synchronize()
    assert int(n_kept.item()) == -1 and int(keep.min().item()) == 7      # nothing was launched
    # the largest allowed size works
    n = B.PDD_STATIC_SCORE_MAX
    score = torch.rand(n, device="cuda:0")
    colsum = score.view(1, n).contiguous()
    keep = torch.empty(n, dtype=torch.uint8, device="cuda:0")
    B.pdd_refine_from_colsum_static(colsum.data_ptr(), n, 1, None, n, 0, 1, 0, n, 0.25,
                                    keep.data_ptr(), n_kept.data_ptr(),
                                    torch.cuda.current_stream().cuda_stream)
    keep_ref = torch.empty(n, dtype=torch.uint8, device="cuda:0")
    n_ref = torch.zeros(1, dtype=torch.int32, device="cuda:0")
    B.pdd_refine_topk(score.data_ptr(), None, n, 0, n, 0.25, keep_ref.data_ptr(), n_ref.data_ptr(),
                      torch.cuda.current_stream().cuda_stream)
    assert torch.equal(keep, keep_ref) and int(n_kept.item()) == int(n_ref.item()) == 16384
