"""GPU parity on the named configurations at full size, in the launch configuration the
benchmark times (default tensor-core path, batched calls).

Config 2 is checked element by element (the checker finishes it in seconds).  Configs 4
and 5 are too large for that: outputs are compared on sampled rows the checker computes
one by one, column sums on sampled heads or sequences, and the rest through properties
that hold at any size (probability mass conservation, popcount of the mask, the mask
being the exact top-k of the library's own scores).  Config 3 runs the layer stack with
the checker evaluated on the bf16 q/k/v the GPU produced for the sampled layers.
"""
import numpy as np
import pytest

from paper_2508_09035_b200 import workloads as wl
from tests import helpers as H

pytestmark = pytest.mark.gpu


def _orc():
    from oracle import pdd_oracle as orc
    return orc


def sampled_rows(s: wl.Sequence, n: int, seed: int) -> np.ndarray:
    """Rows spread over the sequence plus tile/chunk boundaries and both ends."""
    T = s.n_tokens
    edges = [0, 1, 63, 64, 127, 128, 129, T - 1, T - 2]
    for c in s.calls:
        edges += [c.pos0, c.pos0 + c.length - 1]
    rng = wl.rng_for(seed, 55)
    rows = np.concatenate([np.array([e for e in edges if 0 <= e < T]),
                           rng.integers(0, T, size=n)])
    return np.unique(rows)


def run_big(w: wl.Workload, schedule: int = 0):
    """All calls through the C ABI; outputs stay on the device per call."""
    import torch
    kv = H.make_cache(w, 0)
    kv.set_schedule(schedule)
    outs = [dict() for _ in w.seqs]          # pos0 -> device tensor
    for kind, win, group in H.batched_steps(w):
        q = np.concatenate([w.seqs[si].q[c.pos0:c.pos0 + c.length] for si, c in group])
        k = np.concatenate([w.seqs[si].k[c.pos0:c.pos0 + c.length] for si, c in group])
        v = np.concatenate([w.seqs[si].v[c.pos0:c.pos0 + c.length] for si, c in group])
        fn = kv.prefill_chunk if kind == wl.PROMPT else kv.append_received
        o = fn(H.to_dev(q), H.to_dev(k), H.to_dev(v), seq_ids=[si for si, _ in group],
               lens=[c.length for _, c in group], window=win)
        r = 0
        for si, c in group:
            outs[si][c.pos0] = o[r:r + c.length]
            r += c.length
    assert kv.status() == 0
    return kv, outs


def gather_rows(s: wl.Sequence, out_by_call: dict, rows: np.ndarray) -> np.ndarray:
    res = np.zeros((len(rows),) + s.q.shape[1:], dtype=np.float64)
    starts = sorted(out_by_call)
    for i, p in enumerate(rows):
        p0 = max(x for x in starts if x <= p)
        res[i] = H.from_dev_bf16(out_by_call[p0][p - p0:p - p0 + 1])[0]
    return res


def check_sequence_properties(w, s, kv, si, n_window):
    """Size-independent checks: mass conservation per head, mask = exact top-k of the
    library's own fp32 scores, popcount = k_total."""
    orc = _orc()
    cs = kv.export_colsum(si).cpu().numpy().astype(np.float64)
    np.testing.assert_allclose(cs.sum(axis=1), np.full(w.n_q_heads, float(n_window)), rtol=2e-4)
    assert (cs >= 0).all() and np.isfinite(cs).all()
    score = kv.token_importance(si)
    keep, n_kept = kv.refine_topk(score, w.keep_ratio, si)
    score_h = score.cpu().numpy()
    np.testing.assert_allclose(score_h, cs.sum(axis=0), rtol=1e-5, atol=1e-6)
    want, want_n, k = orc.refine_topk(score_h.astype(np.float64), s.kind, 0, s.n_tokens,
                                      w.keep_ratio)
    np.testing.assert_array_equal(keep.cpu().numpy(), want)
    assert int(n_kept.item()) == want_n == orc.keep_count(w.keep_ratio, s.n_prompt)
    return cs, score_h, keep.cpu().numpy()


@pytest.mark.parametrize("window", ["last", "all"])
def test_config2_full(window):
    """Config 2, every output element, every column sum, the keep mask (k = 1229)."""
    w = wl.config_c2(window)
    got = H.run_library(w, kernel_path=0)
    want = H.oracle_full(w)
    stats = H.compare_full(w, got, want)
    assert got[0]["n_kept"] == 1229
    # With 512 window rows x 32 heads the scores are concentrated: about a quarter of the
    # positions lie within 1% of the threshold.  Outside that band the mask is compared
    # with the checker's, inside it with the exact top-k of the library's own scores.
    print("config2 %s: %s" % (window, stats[0]))
    assert stats[0]["band"] < 2048
    # Second, tight band: the measured importance error is below 1e-6 relative, so the mask must
    # also equal the checker's wherever the checker's score is more than 1e-4 (relative) away
    # from the threshold, and that band must be small enough for the comparison to bite.
    from oracle import pdd_oracle as orc
    s = w.seqs[0]
    score_o = want[0]["score"]
    keep_o, _, k = orc.refine_topk(score_o, s.kind, 0, s.n_tokens, w.keep_ratio)
    theta = np.sort(score_o[s.kind == 0])[::-1][k - 1]
    tight = np.abs(score_o - theta) <= 1e-4 * abs(theta)
    np.testing.assert_array_equal(got[0]["keep"][~tight], keep_o[~tight])
    assert int(tight.sum()) <= 64, "tight band holds %d positions" % int(tight.sum())


@pytest.mark.parametrize("schedule", [0, 4], ids=["model", "cta_pairs"])
def test_config4_long_prompt_sampled(schedule):
    """Config 4 at full size (32768 + 256 tokens, 1% outlier keys x8): as the cost model cuts
    it, and through the pair-of-CTAs kernel."""
    orc = _orc()
    w = wl.config_c4("last")
    s = w.seqs[0]
    kv, outs = run_big(w, schedule)
    rows = sampled_rows(s, 48, 4)
    q64, k64, v64 = (a.astype(np.float64) for a in (s.q, s.k, s.v))
    want, _ = orc.attention_rows(q64, k64, v64, w.softmax_scale, rows)
    H.check_out(gather_rows(s, outs[0], rows), want, "config4 sampled rows")
    win = H.window_mask(s)
    cs, score, keep = check_sequence_properties(w, s, kv, 0, int(win.sum()))
    assert int(keep.sum()) == 6554
    # column sums of two heads against the checker (all 33024 positions)
    atol = H.imp_atol(int(win.sum()), w.n_q_heads, s.n_tokens) / w.n_q_heads
    for h in (3, 30):
        g = h // 4
        want_cs = orc.colsum(q64[:, h:h + 1], k64[:, g:g + 1], w.softmax_scale, win)[0]
        H.check_importance(cs[h], want_cs, atol, "config4 colsum head %d" % h)
    kv.close()


def test_config5_ragged_batch_sampled():
    """Config 5 at full size: 16 ragged sequences through batched calls, 64-token pages."""
    orc = _orc()
    w = wl.config_c5("last")
    kv, outs = run_big(w)
    order = np.argsort([s.n_tokens for s in w.seqs])
    for si, s in enumerate(w.seqs):
        q64, k64, v64 = (a.astype(np.float64) for a in (s.q, s.k, s.v))
        rows = sampled_rows(s, 6, 100 + si)
        want, _ = orc.attention_rows(q64, k64, v64, w.softmax_scale, rows)
        H.check_out(gather_rows(s, outs[si], rows), want, "config5 seq %d" % si)
        win = H.window_mask(s)
        cs, score, keep = check_sequence_properties(w, s, kv, si, int(win.sum()))
        if si in order[:4]:                      # the four shortest: full column sums
            want_cs = orc.colsum(q64, k64, w.softmax_scale, win)
            atol = H.imp_atol(int(win.sum()), w.n_q_heads, s.n_tokens)
            H.check_importance(cs, want_cs, atol / w.n_q_heads, "config5 colsum seq %d" % si)
            H.check_keep(keep, int(keep.sum()), want_cs.sum(axis=0), s.kind, 0, s.n_tokens,
                         w.keep_ratio, atol, "config5 seq %d" % si)
    kv.close()


def rmsnorm(x):
    import torch
    xf = x.float()
    return (xf * torch.rsqrt(xf.pow(2).mean(-1, keepdim=True) + 1e-6)).to(torch.bfloat16)


def run_stack(st: wl.LayerStack, check_layers, rows_per_layer=24, full_colsum_layers=()):
    """Layer stack of config 3, chunk by chunk through all layers (one cache per layer):
    x -> RMSNorm -> Wq/Wk/Wv -> attention call -> Wo -> residual.  The projections are plain
    torch GEMMs (not part of the attention path).  For the layers in check_layers the
    checker is evaluated on the bf16 q/k/v the GPU produced ("teacher forced"), so drift of
    the residual stream cannot hide a kernel error."""
    import torch
    from paper_2508_09035_b200 import binding as B
    orc = _orc()
    T = len(st.token_ids)
    hq, hkv, d = st.n_q_heads, st.n_kv_heads, st.head_dim
    scale = 1 / np.sqrt(d)
    x_all = H.to_dev(st.embedding_rows(st.token_ids))
    max_rows = max(c.length for c in st.calls)
    caches = [B.KVCache(hq, hkv, d, page_tokens=128, max_seqs=1, max_tokens_total=T,
                        max_tokens_per_seq=T, max_rows_per_call=max_rows)
              for _ in range(st.n_layers)]
    W = [{n: H.to_dev(st.weight(l, n)) for n in "qkvo"} for l in range(st.n_layers)]
    keep_layers = set(check_layers) | (set(range(st.n_layers)) if full_colsum_layers == "all"
                                       else set(full_colsum_layers))
    saved = {l: dict(q=[], k=[], v=[], out=[]) for l in keep_layers}
    for c in st.calls:
        x = x_all[c.pos0:c.pos0 + c.length]
        for l in range(st.n_layers):
            h_in = rmsnorm(x)
            q = (h_in @ W[l]["q"]).view(-1, hq, d).contiguous()
            k = (h_in @ W[l]["k"]).view(-1, hkv, d).contiguous()
            v = (h_in @ W[l]["v"]).view(-1, hkv, d).contiguous()
            fn = caches[l].prefill_chunk if c.kind == wl.PROMPT else caches[l].append_received
            out = fn(q, k, v, window=c.window)
            if l in saved:
                for n, t in (("q", q), ("k", k), ("v", v), ("out", out)):
                    saved[l][n].append(t)
            x = x + (out.view(-1, hq * d) @ W[l]["o"])
    win = np.zeros(T, np.uint8)
    for c in st.calls:
        if c.window:
            win[c.pos0:c.pos0 + c.length] = 1
    n_win = int(win.sum())
    score = torch.zeros(T, dtype=torch.float32, device="cuda:0")
    colsum_want_total = None
    for l in range(st.n_layers):
        assert caches[l].status() == 0
        caches[l].token_importance(0, score=score, accumulate=l > 0)
        if l not in saved:
            continue
        q64, k64, v64, out = (H.from_dev_bf16(torch.cat(saved[l][n])) for n in ("q", "k", "v", "out"))
        if l in check_layers:
            seq = wl.Sequence(q64, k64, v64, st.kind, st.calls)
            rows = sampled_rows(seq, rows_per_layer, 300 + l)
            want, _ = orc.attention_rows(q64, k64, v64, scale, rows)
            H.check_out(out[rows], want, "stack layer %d" % l)
            cs = caches[l].export_colsum(0).cpu().numpy().astype(np.float64)
            np.testing.assert_allclose(cs.sum(axis=1), np.full(hq, float(n_win)), rtol=2e-4)
            atol = H.imp_atol(n_win, hq, T) / hq
            for h in (0, hq - 1):
                g = h // (hq // hkv)
                want_cs = orc.colsum(q64[:, h:h + 1], k64[:, g:g + 1], scale, win)[0]
                H.check_importance(cs[h], want_cs, atol, "stack layer %d head %d" % (l, h))
        if full_colsum_layers == "all" or l in full_colsum_layers:
            c_l = orc.colsum(q64, k64, scale, win).sum(axis=0)
            colsum_want_total = c_l if colsum_want_total is None else colsum_want_total + c_l
    keep, n_kept = caches[0].refine_topk(score, st.keep_ratio, 0)
    score_h = score.cpu().numpy().astype(np.float64)
    total = hq * n_win * st.n_layers
    assert abs(score_h.sum() - total) < 2e-4 * total
    want, want_n, _ = orc.refine_topk(score_h, st.kind, 0, T, st.keep_ratio)
    keep_h = keep.cpu().numpy()
    np.testing.assert_array_equal(keep_h, want)
    assert int(n_kept.item()) == want_n
    assert not keep_h[st.kind == wl.RECEIVED].any()
    for cch in caches:
        cch.close()
    return score_h, colsum_want_total, keep_h, n_win


def test_config3_stack_small_end_to_end():
    """Config 3 recipe at reduced size (4 layers, 1024-token prompt): importance summed over
    layers against the checker on every layer, keep mask with the ambiguity band."""
    st = wl.config_c3(n_layers=4, n_prompt=1024, chunk=256, received_per_chunk=32)
    score, want, keep, n_win = run_stack(st, check_layers=(0, 3), full_colsum_layers="all")
    T = len(st.token_ids)
    atol = H.imp_atol(n_win, st.n_q_heads, T, n_layers=4)
    H.check_importance(score, want, atol, "stack score")
    H.check_keep(keep, int(keep.sum()), want, st.kind, 0, T, st.keep_ratio, atol, "stack keep")
    assert int(keep.sum()) == 512


def test_config3_stack_full_size_sampled():
    """Config 3 at full size: 28 layers, 8192-token prompt in chunks of 1024 with 128
    received tokens after each chunk; sampled rows and heads on three layers."""
    st = wl.config_c3()
    score, _, keep, n_win = run_stack(st, check_layers=(0, 13, 27), rows_per_layer=16)
    assert n_win == 8192 and int(keep.sum()) == 4096
