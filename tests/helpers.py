"""Shared helpers of the GPU parity tests: run a workload through the C ABI, run the CPU
checker on the same seeded inputs, compare with the stated tolerances."""
from __future__ import annotations

import math
from typing import Dict, List, Optional, Sequence

import numpy as np

from paper_2508_09035_b200 import workloads as wl

# Tolerances of the parity bar.
OUT_MAX_ABS = 2e-2        # bf16 attention output vs the fp64 checker
OUT_MEAN_ABS = 2e-3
IMP_REL = 1e-2            # importance scores, relative


def imp_atol(n_window_rows: int, n_q_heads: int, n_tokens: int, n_layers: int = 1) -> float:
    """Absolute floor for importance: 1e-6 of the mean score.  fp32 exp flushes
    probabilities below ~1e-38 that fp64 keeps, and fp32 sums carry ~1e-7 relative
    rounding per addend, so values far below the mean score cannot be held to a purely
    relative bound."""
    return 1e-6 * n_window_rows * n_q_heads * n_layers / max(n_tokens, 1)


def to_dev(x: np.ndarray, device="cuda:0"):
    """bf16-representable float32 numpy array -> torch bf16 tensor on the device (exact)."""
    import torch
    bits = wl.bf16_bits(x).view(np.int16)
    return torch.from_numpy(bits.copy()).to(device).view(torch.bfloat16)


def from_dev_bf16(t) -> np.ndarray:
    import torch
    bits = t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)
    return wl.bf16_bits_to_f32(bits).astype(np.float64)


def make_cache(w: wl.Workload, kernel_path: int = 0, extra_tokens: int = 0):
    from paper_2508_09035_b200 import binding as B
    max_len = max(s.n_tokens for s in w.seqs) + extra_tokens
    total = sum(s.n_tokens for s in w.seqs) + extra_tokens * len(w.seqs)
    max_rows = sum(max(c.length for c in s.calls) for s in w.seqs)
    return B.KVCache(w.n_q_heads, w.n_kv_heads, w.head_dim, page_tokens=w.page_tokens,
                     max_seqs=len(w.seqs), max_tokens_total=total, max_tokens_per_seq=max_len,
                     max_rows_per_call=max(max_rows, 1), softmax_scale=w.softmax_scale,
                     kernel_path=kernel_path, sliding_window=w.sliding_window)


def batched_steps(w: wl.Workload):
    """Group the sequences' calls into batched library calls: prompt chunk t of every
    sequence that still has one goes into one call, then one call with all received
    blocks.  Yields (kind, window, [(seq_index, Call), ...])."""
    n_prompt_steps = max(sum(1 for c in s.calls if c.kind == wl.PROMPT) for s in w.seqs)
    for t in range(n_prompt_steps):
        group = []
        for si, s in enumerate(w.seqs):
            pc = [c for c in s.calls if c.kind == wl.PROMPT]
            if t < len(pc):
                group.append((si, pc[t]))
        for win in (False, True):
            sub = [(si, c) for si, c in group if c.window == win]
            if sub:
                yield wl.PROMPT, win, sub
    group = [(si, c) for si, s in enumerate(w.seqs) for c in s.calls if c.kind == wl.RECEIVED]
    if group:
        yield wl.RECEIVED, False, group


def run_library(w: wl.Workload, kernel_path: int = 0, pool_kind: int = 0, pool_k: int = 1,
                cand=None, cache=None, in_order_calls: bool = False):
    """All calls of the workload through the C ABI.  Returns per-sequence dicts with
    out (float64 [T,Hq,d]), colsum (float64 [Hq,T]), score, keep, n_kept."""
    import torch
    from paper_2508_09035_b200 import binding as B
    kv = cache or make_cache(w, kernel_path)
    outs = [np.zeros(s.q.shape, dtype=np.float64) for s in w.seqs]
    if in_order_calls:
        # one sequence at a time, calls in their original order (interleaved received blocks)
        steps = []
        for si, s in enumerate(w.seqs):
            for c in s.calls:
                steps.append((c.kind, c.window, [(si, c)]))
    else:
        steps = list(batched_steps(w))
    for kind, win, group in steps:
        q = np.concatenate([w.seqs[si].q[c.pos0:c.pos0 + c.length] for si, c in group])
        k = np.concatenate([w.seqs[si].k[c.pos0:c.pos0 + c.length] for si, c in group])
        v = np.concatenate([w.seqs[si].v[c.pos0:c.pos0 + c.length] for si, c in group])
        fn = kv.prefill_chunk if kind == wl.PROMPT else kv.append_received
        o = fn(to_dev(q), to_dev(k), to_dev(v), seq_ids=[si for si, _ in group],
               lens=[c.length for _, c in group], window=win)
        o = from_dev_bf16(o)
        r = 0
        for si, c in group:
            outs[si][c.pos0:c.pos0 + c.length] = o[r:r + c.length]
            r += c.length
    res = []
    for si, s in enumerate(w.seqs):
        assert kv.length(si) == s.n_tokens
        cs = kv.export_colsum(si).cpu().numpy().astype(np.float64)
        score = kv.token_importance(si, pool_kind, pool_k)
        lo, hi = cand[si] if cand else (0, s.n_tokens)
        keep, n_kept = kv.refine_topk(score, w.keep_ratio, si, lo, hi)
        res.append(dict(out=outs[si], colsum=cs, score=score.cpu().numpy().astype(np.float64),
                        keep=keep.cpu().numpy(), n_kept=int(n_kept.item())))
    assert kv.status() == 0
    if cache is None:
        kv.close()
    return res


def window_mask(s: wl.Sequence) -> np.ndarray:
    win = np.zeros(s.n_tokens, dtype=np.uint8)
    for c in s.calls:
        if c.window:
            win[c.pos0:c.pos0 + c.length] = 1
    return win


def check_out(got: np.ndarray, want: np.ndarray, what: str = ""):
    err = np.abs(got - want)
    assert np.isfinite(got).all(), "%s: non-finite output" % what
    assert err.max() <= OUT_MAX_ABS, "%s: max-abs %.4g > %.4g at %s" % (
        what, err.max(), OUT_MAX_ABS, np.unravel_index(err.argmax(), err.shape))
    assert err.mean() <= OUT_MEAN_ABS, "%s: mean-abs %.4g > %.4g" % (what, err.mean(), OUT_MEAN_ABS)
    return float(err.max()), float(err.mean())


def check_importance(got: np.ndarray, want: np.ndarray, atol: float, what: str = ""):
    err = np.abs(got - want)
    bound = IMP_REL * np.abs(want) + atol
    bad = err > bound
    assert not bad.any(), "%s: %d importance values off; worst at %s got %.6g want %.6g" % (
        what, int(bad.sum()), np.unravel_index((err - bound).argmax(), err.shape),
        got.flat[(err - bound).argmax()], want.flat[(err - bound).argmax()])
    nz = np.abs(want) > 100 * atol
    return float((err[nz] / np.abs(want[nz])).max()) if nz.any() else 0.0


def check_keep(keep_gpu: np.ndarray, n_kept_gpu: int, score_oracle: np.ndarray, kind: np.ndarray,
               cand_lo: int, cand_hi: int, keep_ratio: float, atol: float, what: str = ""):
    """Keep set: bit-exact wherever the checker's scores separate a position from the
    threshold by more than the importance tolerance; equal popcount overall."""
    from oracle import pdd_oracle as orc
    keep_o, n_kept_o, k = orc.refine_topk(score_oracle, kind, cand_lo, cand_hi, keep_ratio)
    assert keep_gpu.shape == keep_o.shape
    assert set(np.unique(keep_gpu)) <= {0, 1}
    assert n_kept_gpu == n_kept_o == int(keep_gpu.sum()), "%s: popcount %d vs %d (k=%d)" % (
        what, int(keep_gpu.sum()), n_kept_o, k)
    n = len(keep_o)
    pos = np.arange(n)
    cand = (kind == wl.PROMPT) & (pos >= cand_lo) & (pos < cand_hi)
    band = np.zeros(n, dtype=bool)
    if 0 < k < int(cand.sum()):
        theta = np.sort(score_oracle[cand])[::-1][k - 1]
        band = cand & (np.abs(score_oracle - theta) <= IMP_REL * abs(theta) + atol)
    outside = ~band
    mism = int((keep_gpu[outside] != keep_o[outside]).sum())
    assert mism == 0, "%s: %d keep-mask mismatches outside the ambiguous band (band %d)" % (
        what, mism, int(band.sum()))
    return int(band.sum()), int((keep_gpu != keep_o).sum())


def oracle_full(w: wl.Workload, pool_kind: str = "none", pool_k: int = 1):
    """Checker results for every sequence (small workloads only)."""
    from oracle import pdd_oracle as orc
    res = []
    for s in w.seqs:
        out, lse = orc.attention(s.q, s.k, s.v, w.softmax_scale, w.sliding_window)
        win = window_mask(s)
        cs = orc.colsum(s.q, s.k, w.softmax_scale, win, w.sliding_window)
        score = orc.importance([cs], pool_kind, pool_k)
        res.append(dict(out=out, lse=lse, colsum=cs, score=score, n_window=int(win.sum())))
    return res


def compare_full(w: wl.Workload, got, want, cand=None, what: str = ""):
    stats = []
    for si, s in enumerate(w.seqs):
        tag = "%s seq %d" % (what or w.name, si)
        mx, mean = check_out(got[si]["out"], want[si]["out"], tag)
        atol = imp_atol(want[si]["n_window"], w.n_q_heads, s.n_tokens)
        # per-head column sums: same bound per head
        check_importance(got[si]["colsum"], want[si]["colsum"], atol / w.n_q_heads, tag + " colsum")
        rel = check_importance(got[si]["score"], want[si]["score"], atol, tag + " score")
        lo, hi = cand[si] if cand else (0, s.n_tokens)
        band, diff = check_keep(got[si]["keep"], got[si]["n_kept"], want[si]["score"], s.kind, lo,
                                hi, w.keep_ratio, atol, tag)
        # inside the band several keep sets are correct; there the mask must still be the
        # exact top-k (ties to the lower position) of the library's own fp32 scores
        from oracle import pdd_oracle as orc
        own, own_n, _ = orc.refine_topk(got[si]["score"], s.kind, lo, hi, w.keep_ratio)
        np.testing.assert_array_equal(got[si]["keep"], own, err_msg=tag + " mask vs own scores")
        stats.append(dict(out_max=mx, out_mean=mean, imp_rel=rel, band=band, keep_diff=diff))
    return stats


# ---------------------------------------------------------------------------------------------
# Single-precision replays.  SECONDARY checks only: the parity statements of the sentence and
# vote selections are made against the fp64 checker (bands below); these functions repeat an
# fp32 evaluation (terms added one by one in position / head order, one division) so that a
# test can also say "and the mask is the exact selection for the values the library formed".

def replay_sentence_values_f32(score, kind, seg_start):
    score = np.asarray(score, dtype=np.float32)
    n_seg = len(seg_start) - 1
    kind = np.zeros(len(score), np.uint8) if kind is None else np.asarray(kind, np.uint8)
    value = np.full(n_seg, -np.inf, dtype=np.float32)
    count = np.zeros(n_seg, dtype=np.int64)
    for s in range(n_seg):
        acc = np.float32(0)
        c = 0
        for i in range(int(seg_start[s]), int(seg_start[s + 1])):
            if kind[i] == wl.PROMPT:
                acc = np.float32(acc + score[i])
                c += 1
        count[s] = c
        if c:
            value[s] = np.float32(acc / np.float32(c))
    return value, count


def replay_pool_f32(x, kind: str, width: int):
    x = np.asarray(x, dtype=np.float32)
    if kind == "none" or width == 1:
        return x.copy()
    half = width // 2
    n = x.shape[-1]
    out = np.empty_like(x)
    for j in range(n):
        lo, hi = max(0, j - half), min(n, j + half + 1)
        if kind == "avg":
            acc = np.zeros(x.shape[:-1], dtype=np.float32)
            for t in range(lo, hi):
                acc = (acc + x[..., t]).astype(np.float32)
            out[..., j] = (acc / np.float32(width)).astype(np.float32)
        else:
            out[..., j] = x[..., lo:hi].max(axis=-1)
    return out


def sentence_budget(kind, seg_start, keep_ratio: float) -> int:
    """Token budget of the sentence selection: clamp(k_total - #always_kept, 0, #content)."""
    from oracle import pdd_oracle as orc
    n = len(kind)
    pos = np.arange(n)
    prompt = np.asarray(kind) == wl.PROMPT
    content = prompt & (pos >= int(seg_start[0])) & (pos < int(seg_start[-1]))
    always = prompt & ~content
    k_total = orc.keep_count(keep_ratio, int(prompt.sum()))
    return min(max(k_total - int(always.sum()), 0), int(content.sum()))


def sentence_near_ties(value64, count, rel: float) -> int:
    """Adjacent pairs (in decreasing order) of distinct sentence values closer than rel: the
    pairs whose order an fp32 evaluation of the means may turn round."""
    v = np.sort(np.asarray(value64)[np.asarray(count) > 0])[::-1]
    if len(v) < 2:
        return 0
    gap = v[:-1] - v[1:]
    return int(((gap > 0) & (gap <= rel * np.abs(v[:-1]))).sum())


def check_vote_keep(keep_gpu, n_kept_gpu, votes_gpu, keep_o, n_kept_o, votes_o, total_o, kind,
                    cand_lo: int, cand_hi: int, n_heads: int, what: str = ""):
    """Vote selection against the fp64 checker.  Votes must agree exactly (the caller only
    passes inputs whose per-head decisions are exact in fp32).  The mask must agree outside the
    near-tie band: candidates with the threshold's vote count whose head sum lies within the
    fp32 summation error of the threshold's head sum.  Returns the band size."""
    np.testing.assert_array_equal(votes_gpu, votes_o, err_msg=what + " votes")
    assert n_kept_gpu == n_kept_o == int(keep_gpu.sum()), what + " popcount"
    n = len(keep_o)
    pos = np.arange(n)
    cand = (np.asarray(kind) == wl.PROMPT) & (pos >= cand_lo) & (pos < cand_hi)
    k = int(keep_o[cand].sum())
    band = np.zeros(n, dtype=bool)
    if 0 < k < int(cand.sum()):
        idx = pos[cand]
        order = np.lexsort((idx, -total_o[idx], -votes_o[idx]))
        last = idx[order[k - 1]]
        v_star, theta = votes_o[last], total_o[last]
        eps = (n_heads + 2) * 2.0 ** -24 * np.abs(total_o)
        band = cand & (votes_o == v_star) & (np.abs(total_o - theta) <= 2 * (eps + eps[last]))
    mism = int((keep_gpu[~band] != keep_o[~band]).sum())
    assert mism == 0, "%s: %d mask mismatches outside the near-tie band (band %d)" % (
        what, mism, int(band.sum()))
    return int(band.sum())
