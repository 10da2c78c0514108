"""GPU parity: every step of the path through the C ABI against the CPU checker, element by
element on small and mid-size seeded workloads (several tiles, ragged tails, both head
dims, GQA ratios 1/4/6, both page sizes), plus API state/edge cases."""
import numpy as np
import pytest

from paper_2508_09035_b200 import workloads as wl
from tests import helpers as H

pytestmark = pytest.mark.gpu

import os
PATHS = [int(x) for x in os.environ.get("PDD_TEST_PATHS", "0").split(",")]   # 0 tensor-core (default), 1 SIMT, 2 simple tensor-core


def _orc():
    from oracle import pdd_oracle as orc
    return orc


SMALL = [
    # name, seed, hq, hkv, d, n_prompt, chunk, n_received, page, window
    ("one_tile", 100, 2, 2, 128, 128, 128, 0, 64, "all"),
    ("tiny", 101, 2, 1, 64, 5, 3, 2, 64, "all"),
    ("single_token", 102, 4, 4, 128, 1, 1, 0, 64, "all"),
    ("ragged_d128_g4", 103, 8, 2, 128, 333, 100, 9, 64, "last"),
    ("ragged_d64_g1", 104, 4, 4, 64, 300, 77, 5, 64, "all"),
    ("g6_page128", 105, 12, 2, 128, 450, 200, 33, 128, "all"),
    ("multi_tile_chunk", 106, 4, 1, 128, 700, 350, 17, 64, "last"),
    ("d64_page128", 107, 8, 8, 64, 260, 130, 1, 128, "last"),
]


@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("case", SMALL, ids=[c[0] for c in SMALL])
def test_small_cases_match_checker(case, path):
    name, seed, hq, hkv, d, n_prompt, chunk, n_recv, page, window = case
    w = wl.small_like(name, seed, hq, hkv, d, n_prompt, chunk, n_recv, keep_ratio=0.3,
                      window=window, page_tokens=page)
    got = H.run_library(w, kernel_path=path)
    want = H.oracle_full(w)
    H.compare_full(w, got, want)


@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("window", ["last", "all"])
def test_config1_full(window, path):
    """Config 1: 8/8 heads, d=64, 512-token prompt in 4 chunks of 128 + 16 received tokens,
    keep ratio 0.5; both window readings (last chunk only / every prompt row)."""
    w = wl.config_c1(window)
    got = H.run_library(w, kernel_path=path)
    want = H.oracle_full(w)
    stats = H.compare_full(w, got, want)
    assert got[0]["n_kept"] == 256
    assert stats[0]["band"] < 64          # the keep-set check is not vacuous


@pytest.mark.parametrize("path", PATHS)
def test_outlier_keys_stress_softmax(path):
    """1% of K rows scaled x8 (heavy-tailed attention): large logits, tiny probabilities."""
    w = wl.small_like("outliers", 110, 8, 2, 128, 640, 256, 16, window="all",
                      outlier_frac=0.02, outlier_gain=8.0)
    got = H.run_library(w, kernel_path=path)
    H.compare_full(w, got, H.oracle_full(w))


@pytest.mark.parametrize("path", PATHS)
def test_ragged_batch_small(path):
    """Batched ragged prefill with a shared page pool (config 5 recipe, short lengths)."""
    w = wl.ragged_batch("ragged_small", 4, 8, 2, 128, 5, 40, 600, 128, 20, 0.4, window="last")
    got = H.run_library(w, kernel_path=path)
    H.compare_full(w, got, H.oracle_full(w))


@pytest.mark.parametrize("path", PATHS)
def test_interleaved_received_tokens(path):
    """Received blocks between prompt chunks (config 3's call pattern): they take cache
    positions and collect column mass but are never selectable."""
    calls, kind = wl.make_calls(384, 128, 0, "all", interleave_received=16)
    T = len(kind)
    q, k, v = wl.normal_qkv(wl.rng_for(120), T, 6, 1, 128)
    w = wl.Workload("interleaved", 6, 1, 128, 64, 0.5, [wl.Sequence(q, k, v, kind, calls)], 128,
                    1 / np.sqrt(128.0))
    got = H.run_library(w, kernel_path=path, in_order_calls=True)
    want = H.oracle_full(w)
    H.compare_full(w, got, want)
    assert not got[0]["keep"][kind == wl.RECEIVED].any()
    assert got[0]["n_kept"] == 192


@pytest.mark.parametrize("path", PATHS)
def test_q_zero_closed_form_on_gpu(path):
    """Q = 0: importance of key j over the full window is H_T - H_j, the output is the
    running mean of V, and top-k keeps the first k positions."""
    w = wl.small_like("qzero", 130, 4, 2, 128, 300, 128, 0, keep_ratio=0.25, window="all")
    s = w.seqs[0]
    s.q[:] = 0
    got = H.run_library(w, kernel_path=path)[0]
    T = s.n_tokens
    Hn = np.concatenate([[0.0], np.cumsum(1.0 / np.arange(1, T + 1))])
    want_cs = Hn[T] - Hn[:T]
    for h in range(4):
        np.testing.assert_allclose(got["colsum"][h], want_cs, rtol=1e-4)
    mean_v = np.cumsum(s.v.astype(np.float64), axis=0) / np.arange(1, T + 1)[:, None, None]
    H.check_out(got["out"], np.repeat(mean_v, 2, axis=1))
    assert got["keep"][:75].all() and not got["keep"][75:].any()


def test_kv_roundtrip_and_page_reuse():
    """K/V written through the paged cache read back bit-exactly; reset returns pages and
    zeroes the column sums; a second sequence reuses them."""
    import torch
    from paper_2508_09035_b200 import binding as B
    w = wl.small_like("rt", 140, 4, 2, 128, 200, 64, 10, window="all")
    s = w.seqs[0]
    kv = H.make_cache(w, kernel_path=1)
    for rep in range(2):
        for c in s.calls:
            sl = slice(c.pos0, c.pos0 + c.length)
            fn = kv.prefill_chunk if c.kind == wl.PROMPT else kv.append_received
            fn(H.to_dev(s.q[sl]), H.to_dev(s.k[sl]), H.to_dev(s.v[sl]), window=c.window)
        k, v = kv.export_kv(0)
        np.testing.assert_array_equal(H.from_dev_bf16(k), s.k)
        np.testing.assert_array_equal(H.from_dev_bf16(v), s.v)
        np.testing.assert_array_equal(kv.export_kinds(0).cpu().numpy(), s.kind)
        cs1 = kv.export_colsum(0).cpu().numpy()
        assert abs(cs1.sum() - 4 * 200) < 1e-2
        kv.reset(0)
        assert kv.length(0) == 0
    kv.close()


def test_state_and_capacity_errors():
    """Validation happens before anything is enqueued and leaves the state untouched."""
    import torch
    from paper_2508_09035_b200 import binding as B
    kv = B.KVCache(4, 2, 128, page_tokens=64, max_seqs=2, max_tokens_total=256,
                   max_tokens_per_seq=192, max_rows_per_call=128)
    q = torch.zeros((64, 4, 128), dtype=torch.bfloat16, device="cuda:0")
    k = torch.zeros((64, 2, 128), dtype=torch.bfloat16, device="cuda:0")
    out = torch.empty_like(q)
    kv.prefill_chunk(q, k, k)
    assert kv.length(0) == 64

    def call(seq_ids, pos0, lens, qq=q, kk=k):
        b, keep = B.make_batch(seq_ids, pos0, lens)
        B.pdd_prefill_chunk(kv.h, b, qq.data_ptr(), kk.data_ptr(), kk.data_ptr(), out.data_ptr(),
                            0, kv.stream)

    with pytest.raises(B.PddError) as e:
        call([0], [0], [64])                      # pos0 != current length
    assert e.value.status == B.PDD_ERR_STATE
    with pytest.raises(B.PddError) as e:
        call([0, 0], [64, 64], [32, 32])          # same sequence twice
    assert e.value.status == B.PDD_ERR_INVALID
    with pytest.raises(B.PddError) as e:
        call([3], [0], [8])                       # unknown sequence
    assert e.value.status == B.PDD_ERR_INVALID
    q2 = torch.zeros((192, 4, 128), dtype=torch.bfloat16, device="cuda:0")
    k2 = torch.zeros((192, 2, 128), dtype=torch.bfloat16, device="cuda:0")
    with pytest.raises(B.PddError) as e:
        call([0], [64], [192], q2, k2)            # more rows than a call may carry
    assert e.value.status == B.PDD_ERR_CAPACITY
    kv.prefill_chunk(q, k, k)
    kv.prefill_chunk(q, k, k)
    with pytest.raises(B.PddError) as e:
        call([0], [192], [1])                     # sequence full
    assert e.value.status == B.PDD_ERR_CAPACITY
    assert kv.length(0) == 192 and kv.length(1) == 0
    # an empty call is fine and changes nothing
    b, keep = B.make_batch([1], [0], [0])
    B.pdd_prefill_chunk(kv.h, b, None, None, None, None, 0, kv.stream)
    assert kv.length(1) == 0 and kv.status() == 0
    kv.close()


@pytest.mark.parametrize("pool", [("avg", 1, 7), ("max", 2, 5), ("avg", 1, 1)])
def test_pooling_matches_definition(pool):
    name, kind, width = pool
    w = wl.small_like("pool", 150, 4, 2, 64, 200, 100, 4, window="all")
    got = H.run_library(w, kernel_path=1, pool_kind=kind, pool_k=width)[0]
    want = H.oracle_full(w, name, width)[0]
    atol = H.imp_atol(want["n_window"], 4, w.seqs[0].n_tokens)
    H.check_importance(got["score"], want["score"], atol, "pooled score")


def test_layer_accumulation():
    """accumulate=1 sums layers into one score vector."""
    import torch
    w = wl.small_like("acc", 160, 4, 2, 64, 96, 96, 0, window="all")
    s = w.seqs[0]
    kv = H.make_cache(w, kernel_path=1)
    kv.prefill_chunk(H.to_dev(s.q), H.to_dev(s.k), H.to_dev(s.v), window=True)
    one = kv.token_importance(0)
    acc = one.clone()
    kv.token_importance(0, score=acc, accumulate=True)
    torch.testing.assert_close(acc, 2 * one)
    kv.close()


def _topk_case(rng, n):
    score = rng.random(n).astype(np.float32)
    mode = int(rng.integers(0, 4))
    if mode == 1:
        score = np.round(score * 8).astype(np.float32) / 8          # many exact ties
    elif mode == 2:
        score[:] = 0.5                                              # all equal
    elif mode == 3:
        score = (score * 1e-30).astype(np.float32)                  # tiny values
    kind = (rng.random(n) < 0.1).astype(np.uint8)
    lo = int(rng.integers(0, max(1, n // 4)))
    hi = n - int(rng.integers(0, max(1, n // 4)))
    return score, kind, lo, max(lo, hi), float(rng.choice([0.0, 0.2, 0.37, 0.5, 0.9, 1.0]))


def test_radix_topk_bit_exact_against_sort():
    """Integer/byte work: the mask must equal the stable-sort definition exactly when both
    sides see the same fp32 scores."""
    import torch
    from paper_2508_09035_b200 import binding as B
    orc = _orc()
    rng = wl.rng_for(170)
    for n in [1, 2, 31, 32, 33, 1000, 1024, 1025, 4160, 8191, 33024, 49151, 49152, 49153, 70001]:
        for rep in range(3):
            score, kind, lo, hi, r = _topk_case(rng, n)
            d_score = torch.from_numpy(score).cuda()
            d_kind = torch.from_numpy(kind).cuda()
            keep = torch.empty(n, dtype=torch.uint8, device="cuda:0")
            n_kept = torch.zeros(1, dtype=torch.int32, device="cuda:0")
            B.pdd_refine_topk(d_score.data_ptr(), d_kind.data_ptr(), n, lo, hi, r,
                              keep.data_ptr(), n_kept.data_ptr(),
                              torch.cuda.current_stream().cuda_stream)
            want, want_n, _ = orc.refine_topk(score.astype(np.float64), kind, lo, hi, r)
            np.testing.assert_array_equal(keep.cpu().numpy(), want, err_msg="n=%d r=%g" % (n, r))
            assert int(n_kept.item()) == want_n
            # null kinds = all prompt
            B.pdd_refine_topk(d_score.data_ptr(), None, n, lo, hi, r, keep.data_ptr(),
                              n_kept.data_ptr(), torch.cuda.current_stream().cuda_stream)
            want, want_n, _ = orc.refine_topk(score.astype(np.float64), None, lo, hi, r)
            np.testing.assert_array_equal(keep.cpu().numpy(), want)


def test_radix_topk_batched():
    import torch
    from paper_2508_09035_b200 import binding as B
    orc = _orc()
    rng = wl.rng_for(171)
    lens = [int(x) for x in rng.integers(1, 3000, size=70)]     # more than one launch
    offs = np.concatenate([[0], np.cumsum(lens)])
    cases = [_topk_case(rng, n) for n in lens]
    score = np.concatenate([c[0] for c in cases])
    kind = np.concatenate([c[1] for c in cases])
    keep = torch.empty(len(score), dtype=torch.uint8, device="cuda:0")
    n_kept = torch.zeros(len(lens), dtype=torch.int32, device="cuda:0")
    d_score, d_kind = torch.from_numpy(score).cuda(), torch.from_numpy(kind).cuda()
    B.pdd_refine_topk_batched(d_score.data_ptr(), d_kind.data_ptr(), offs.tolist(),
                              [c[2] for c in cases], [c[3] for c in cases], 0.4,
                              keep.data_ptr(), n_kept.data_ptr(),
                              torch.cuda.current_stream().cuda_stream)
    got = keep.cpu().numpy()
    for i, c in enumerate(cases):
        want, want_n, _ = orc.refine_topk(c[0].astype(np.float64), c[1], c[2], c[3], 0.4)
        np.testing.assert_array_equal(got[offs[i]:offs[i + 1]], want)
        assert int(n_kept[i].item()) == want_n


def test_many_short_sequences_in_one_call():
    """70 sequences of 1..90 tokens in batched calls: the call record outgrows the kernel
    parameter block and travels through its device slot instead (the other record path), and
    most tile pairs are a few rows of one key block."""
    w = wl.ragged_batch("many_short", 120, 8, 2, 128, 70, 1, 90, 48, 5, 0.5, window="all")
    assert len(w.seqs) == 70
    got = H.run_library(w)
    H.compare_full(w, got, H.oracle_full(w))


def test_empty_sequences_inside_a_batch():
    """len = 0 for some sequences of a call: they keep their state, the others see exactly
    what a call without the empty entries gives."""
    import torch
    from paper_2508_09035_b200 import binding as B
    orc = _orc()
    rng = wl.rng_for(121)
    hq, hkv, d = 4, 2, 128
    lens_a, lens_b = [130, 0, 37], [0, 64, 5]
    kv = B.KVCache(hq, hkv, d, page_tokens=64, max_seqs=3, max_tokens_total=512,
                   max_tokens_per_seq=256, max_rows_per_call=256)
    seqs = [dict(q=[], k=[], v=[]) for _ in range(3)]
    outs = [[] for _ in range(3)]
    for lens in (lens_a, lens_b):
        rows = sum(lens)
        q = wl.bf16_round(rng.standard_normal((rows, hq, d)).astype(np.float32))
        k = wl.bf16_round(rng.standard_normal((rows, hkv, d)).astype(np.float32))
        v = wl.bf16_round(rng.standard_normal((rows, hkv, d)).astype(np.float32))
        o = H.from_dev_bf16(kv.prefill_chunk(H.to_dev(q), H.to_dev(k), H.to_dev(v),
                                             seq_ids=[0, 1, 2], lens=lens, window=True))
        r = 0
        for si, n in enumerate(lens):
            seqs[si]["q"].append(q[r:r + n]); seqs[si]["k"].append(k[r:r + n])
            seqs[si]["v"].append(v[r:r + n]); outs[si].append(o[r:r + n])
            r += n
    scale = 1.0 / np.sqrt(d)
    for si in range(3):
        q, k, v = (np.concatenate(seqs[si][n]).astype(np.float64) for n in ("q", "k", "v"))
        T = q.shape[0]
        assert kv.length(si) == T == lens_a[si] + lens_b[si]
        want, _ = orc.attention(q, k, v, scale)
        H.check_out(np.concatenate(outs[si]), want, "seq %d" % si)
        cs = kv.export_colsum(si).cpu().numpy().astype(np.float64)
        want_cs = orc.colsum(q, k, scale, np.ones(T, dtype=np.uint8))
        H.check_importance(cs, want_cs, H.imp_atol(T, hq, T) / hq, "seq %d colsum" % si)
    assert kv.status() == 0
    kv.close()


@pytest.mark.parametrize("pool", [(0, 1), (1, 5), (2, 3)])
def test_fused_importance_topk_equals_the_two_calls_and_the_checker(pool):
    """pdd_importance_topk: scores and mask bit-identical to pdd_token_importance followed by
    pdd_refine_topk, and the mask equal to the checker's exact top-k of those scores."""
    import torch
    from oracle import pdd_oracle as orc
    from paper_2508_09035_b200 import binding as B
    w = wl.small_like("fused", 880, 8, 2, 128, 1500, 512, 40, keep_ratio=0.3, window="all")
    s = w.seqs[0]
    kv = H.make_cache(w, 0)
    for c in s.calls:
        sl = slice(c.pos0, c.pos0 + c.length)
        fn = kv.prefill_chunk if c.kind == wl.PROMPT else kv.append_received
        fn(H.to_dev(s.q[sl]), H.to_dev(s.k[sl]), H.to_dev(s.v[sl]), window=c.window)
    n = s.n_tokens
    score2 = kv.token_importance(0, pool[0], pool[1])
    keep2, n2 = kv.refine_topk(score2, 0.3, 0, 7, n - 5)
    for with_score in (True,):
        score1 = torch.full((n,), -1.0, dtype=torch.float32, device="cuda:0")
        keep1 = torch.full((n,), 9, dtype=torch.uint8, device="cuda:0")
        n1 = torch.full((1,), -1, dtype=torch.int32, device="cuda:0")
        B.pdd_importance_topk(kv.h, 0, pool[0], pool[1], score1.data_ptr() if with_score else None,
                              0, 7, n - 5, 0.3, keep1.data_ptr(), n1.data_ptr(), kv.stream)
        torch.cuda.synchronize()
        if with_score:
            assert torch.equal(score1, score2)
        assert torch.equal(keep1, keep2) and int(n1.item()) == int(n2.item())
    want, want_n, _ = orc.refine_topk(score2.cpu().numpy(), s.kind, 7, n - 5, 0.3)
    np.testing.assert_array_equal(keep2.cpu().numpy(), want)
    # accumulate adds to the caller's vector, as the separate call does
    acc1 = score2.clone()
    acc2 = score2.clone()
    keep1 = torch.empty(n, dtype=torch.uint8, device="cuda:0")
    n1 = torch.zeros(1, dtype=torch.int32, device="cuda:0")
    B.pdd_importance_topk(kv.h, 0, pool[0], pool[1], acc1.data_ptr(), 1, 0, n, 0.3,
                          keep1.data_ptr(), n1.data_ptr(), kv.stream)
    kv.token_importance(0, pool[0], pool[1], score=acc2, accumulate=True)
    assert torch.equal(acc1, acc2)
    keepa, na = kv.refine_topk(acc2, 0.3, 0)
    assert torch.equal(keep1, keepa) and int(n1.item()) == int(na.item())
    kv.close()


def test_batched_importance_equals_single_calls():
    import torch
    from paper_2508_09035_b200 import binding as B
    w = wl.ragged_batch("imp_b", 881, 8, 2, 64, 5, 100, 900, 256, 30, 0.4, "last", page_tokens=64)
    kv = H.make_cache(w, 0)
    res = H.run_library(w, cache=kv)
    offs = [0]
    for s in w.seqs:
        offs.append(offs[-1] + s.n_tokens)
    score = torch.full((offs[-1],), -1.0, dtype=torch.float32, device="cuda:0")
    B.pdd_token_importance_batched(kv.h, list(range(len(w.seqs))), 0, 1, score.data_ptr(), offs, 0,
                                   kv.stream)
    got = score.cpu().numpy()
    for si in range(len(w.seqs)):
        np.testing.assert_array_equal(got[offs[si]:offs[si + 1]], res[si]["score"].astype(np.float32))
    with pytest.raises(B.PddError):
        B.pdd_token_importance_batched(kv.h, [0], 0, 1, score.data_ptr(), [0, 3], 0, kv.stream)
    kv.close()
