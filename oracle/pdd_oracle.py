"""CPU checker ("oracle") for the chunked-prefill attention path.  TEST INFRASTRUCTURE ONLY.

Slow, plain and fp64.  Only the tests, the smoke check and the benchmark's CPU-baseline
leg may import this module; the library never does, and this module imports nothing
from the CUDA package.

What it follows in the paper:
  * attention  softmax(Q K^T / sqrt(h)) V  -- Sec. 2.2.3 (unnumbered attention equation),
    causal as in any decoder-only model;
  * the refiner signal -- Sec. 3.2 "Prompt Refiner": normalised attention weights of the
    observation window (the last segment of Q) against the entire K, summed along the
    query dimension, then 1-D pooling, then the top values with ratio r;
  * r = refined length / original length -- Sec. 2.2.3 (definition of the refinement
    ratio); mask with 1 = keep -- Sec. 3.2 (mask tensor);
  * chunked prefill and the received tokens that are fed back as forced inputs --
    Sec. 3.3 "LLM Engine" and Algorithm 2.

Readings taken where the paper is silent (each is a parameter here):
  * scale: the caller passes it (1/sqrt(head_dim) in every workload);
  * observation window: the set of rows whose calls were flagged as window rows;
  * pooling: kind in {"none","avg","max"}, odd width, stride 1, same length; avg pads
    with zeros and always divides by the width, max pads with -inf;
  * heads (and layers) are merged by plain summation before ONE top-k;
  * k_total = floor(r*l + 1/2) over the l prompt positions, always-kept prompt
    positions (outside the candidate range) count toward it; received positions are
    never kept; ties go to the lower position.
Parity unpinned: the pooling defaults and the head/layer merge rule are readings, pinned
only as definitions (brute force), not by any value the paper prints.
"""
from __future__ import annotations

import ctypes
import math
import os
import subprocess
from typing import List, Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "pdd_oracle.c")
_LIB = os.path.join(_HERE, "libpdd_oracle.so")
_lib = None

PROMPT = 0
RECEIVED = 1


def build(force: bool = False) -> str:
    """Compile the C part with gcc (OpenMP, no fast-math, no FMA contraction)."""
    if (not force and os.path.exists(_LIB)
            and os.path.getmtime(_LIB) >= os.path.getmtime(_SRC)):
        return _LIB
    cmd = ["gcc", "-O3", "-march=x86-64-v3", "-ffp-contract=off", "-fopenmp", "-shared",
           "-fPIC", "-o", _LIB, _SRC, "-lm"]
    subprocess.run(cmd, check=True)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        lib = ctypes.CDLL(_LIB)
        dp = ctypes.POINTER(ctypes.c_double)
        i64p = ctypes.POINTER(ctypes.c_int64)
        u8p = ctypes.POINTER(ctypes.c_uint8)
        lib.pdd_oracle_attention_rows.argtypes = [dp, dp, dp, ctypes.c_int64, ctypes.c_int,
                                                  ctypes.c_int, ctypes.c_int, ctypes.c_double,
                                                  i64p, ctypes.c_int64, dp, dp, ctypes.c_int64]
        lib.pdd_oracle_colsum.argtypes = [dp, dp, ctypes.c_int64, ctypes.c_int, ctypes.c_int,
                                          ctypes.c_int, ctypes.c_double, u8p, dp, ctypes.c_int64,
                                          ctypes.c_int64]
        lib.pdd_oracle_prob_row.argtypes = [dp, dp, ctypes.c_int64, ctypes.c_int, ctypes.c_int,
                                            ctypes.c_int, ctypes.c_double, ctypes.c_int64,
                                            ctypes.c_int, dp, dp, ctypes.c_int64]
        lib.pdd_oracle_threads.restype = ctypes.c_int
        _lib = lib
    return _lib


def threads() -> int:
    return int(_load().pdd_oracle_threads())


def _f64(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.float64)


def _dp(a: np.ndarray):
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_double))


def attention_rows(q, k, v, scale: float, rows, sliding_window: int = 0) -> tuple:
    """O and LSE of the listed query positions against keys 0..p (Sec. 2.2.3).

    q [T,Hq,d], k,v [T,Hkv,d]; returns (out [n,Hq,d], lse [n,Hq]) in fp64.
    sliding_window = w > 0 restricts row p to keys max(0, p-w+1)..p (the on-device
    sliding-window attention of Sec. 3.3).
    """
    q, k, v = _f64(q), _f64(k), _f64(v)
    T, hq, d = q.shape
    hkv = k.shape[1]
    assert k.shape == (T, hkv, d) and v.shape == (T, hkv, d)
    rows = np.ascontiguousarray(rows, dtype=np.int64)
    out = np.zeros((len(rows), hq, d), dtype=np.float64)
    lse = np.zeros((len(rows), hq), dtype=np.float64)
    if len(rows) == 0:
        return out, lse
    rc = _load().pdd_oracle_attention_rows(
        _dp(q), _dp(k), _dp(v), T, hq, hkv, d, float(scale),
        rows.ctypes.data_as(ctypes.POINTER(ctypes.c_int64)), len(rows), _dp(out), _dp(lse),
        int(sliding_window))
    if rc != 0:
        raise ValueError("pdd_oracle_attention_rows: bad arguments")
    return out, lse


def attention(q, k, v, scale: float, sliding_window: int = 0) -> tuple:
    """One-shot causal attention over all T positions."""
    return attention_rows(q, k, v, scale, np.arange(np.asarray(q).shape[0]), sliding_window)


def colsum(q, k, scale: float, window, sliding_window: int = 0) -> np.ndarray:
    """colsum[h][j] = sum over window rows p >= j of P[h][p][j]  (Sec. 3.2)."""
    q, k = _f64(q), _f64(k)
    T, hq, d = q.shape
    hkv = k.shape[1]
    window = np.ascontiguousarray(window, dtype=np.uint8)
    assert window.shape == (T,)
    cs = np.zeros((hq, T), dtype=np.float64)
    rc = _load().pdd_oracle_colsum(_dp(q), _dp(k), T, hq, hkv, d, float(scale),
                                   window.ctypes.data_as(ctypes.POINTER(ctypes.c_uint8)),
                                   _dp(cs), T, int(sliding_window))
    if rc != 0:
        raise ValueError("pdd_oracle_colsum: bad arguments")
    return cs


def prob_row(q, k, scale: float, p: int, h: int, sliding_window: int = 0) -> np.ndarray:
    q, k = _f64(q), _f64(k)
    T, hq, d = q.shape
    out = np.zeros(p + 1, dtype=np.float64)
    rc = _load().pdd_oracle_prob_row(_dp(q), _dp(k), T, hq, k.shape[1], d, float(scale),
                                     int(p), int(h), _dp(out), None, int(sliding_window))
    if rc != 0:
        raise ValueError("pdd_oracle_prob_row: bad arguments")
    return out


def pool1d(x: np.ndarray, kind: str = "none", width: int = 1) -> np.ndarray:
    """1-D pooling along the last axis, stride 1, same length (Sec. 3.2, "1D pooling")."""
    x = np.asarray(x, dtype=np.float64)
    if kind == "none" or width == 1:
        return x.copy()
    assert width % 2 == 1 and width >= 1
    half = width // 2
    n = x.shape[-1]
    out = np.empty_like(x)
    for j in range(n):
        lo, hi = max(0, j - half), min(n, j + half + 1)
        seg = x[..., lo:hi]
        if kind == "avg":
            out[..., j] = seg.sum(axis=-1) / width      # zero padding, fixed divisor
        elif kind == "max":
            out[..., j] = seg.max(axis=-1)              # -inf padding
        else:
            raise ValueError(kind)
    return out


def importance(colsums: Sequence[np.ndarray], pool_kind: str = "none",
               pool_width: int = 1) -> np.ndarray:
    """score[j] = sum over layers and heads of the pooled per-head column sums."""
    score = None
    for cs in colsums:
        s = pool1d(cs, pool_kind, pool_width).sum(axis=0)
        score = s if score is None else score + s
    return score


def keep_count(keep_ratio: float, n_prompt: int) -> int:
    """k_total = floor(r*l + 1/2), r = refined length / original length (Sec. 2.2.3)."""
    return int(math.floor(float(keep_ratio) * float(n_prompt) + 0.5))


def refine_topk(score, kind, cand_lo: int, cand_hi: int, keep_ratio: float):
    """Keep mask over positions (Sec. 3.2: top values with ratio r; mask 1 = keep).

    Candidates are prompt positions in [cand_lo, cand_hi) (the "content" part); prompt
    positions outside are prefix/suffix and always kept; received positions are 0.
    Returns (keep uint8 [n], n_kept, k) with k the number taken from the candidates.
    """
    score = np.asarray(score, dtype=np.float64)
    n = score.shape[0]
    kind = np.zeros(n, dtype=np.uint8) if kind is None else np.asarray(kind, dtype=np.uint8)
    pos = np.arange(n)
    is_prompt = kind == PROMPT
    cand = is_prompt & (pos >= cand_lo) & (pos < cand_hi)
    always = is_prompt & ~cand
    k_total = keep_count(keep_ratio, int(is_prompt.sum()))
    k = min(max(k_total - int(always.sum()), 0), int(cand.sum()))
    keep = np.zeros(n, dtype=np.uint8)
    keep[always] = 1
    idx = pos[cand]
    order = np.argsort(-score[idx], kind="stable")     # descending, ties -> lower position
    keep[idx[order[:k]]] = 1
    return keep, int(keep.sum()), k


def sentence_values(score, kind, seg_start):
    """Value of each sentence = mean score of its prompt tokens (Sec. 3.2: the KVCache of one
    sentence is treated as a whole).  The aggregator is not given in the paper; the mean is
    this build's reading ("parity unpinned").  Returns (value [n_seg] fp64, count [n_seg]); a
    sentence without prompt tokens has count 0 and value -inf."""
    score = np.asarray(score, dtype=np.float64)
    n_seg = len(seg_start) - 1
    kind = np.zeros(len(score), np.uint8) if kind is None else np.asarray(kind, np.uint8)
    value = np.full(n_seg, -np.inf, dtype=np.float64)
    count = np.zeros(n_seg, dtype=np.int64)
    for s in range(n_seg):
        sl = slice(int(seg_start[s]), int(seg_start[s + 1]))
        prompt = kind[sl] == PROMPT
        count[s] = int(prompt.sum())
        if count[s]:
            value[s] = math.fsum(score[sl][prompt]) / float(count[s])
    return value, count


def select_sentences(value, count, budget: int) -> np.ndarray:
    """Which sentences are taken, given their values, their prompt-token counts and the token
    budget: sentences are visited by decreasing value (ties: lower sentence first) and one is
    taken iff it has prompt tokens and still fits what is left of the budget."""
    value = np.asarray(value, dtype=np.float64)
    order = np.argsort(-value, kind="stable")
    taken = np.zeros(len(value), dtype=bool)
    rem = int(budget)
    for s in order:
        if rem == 0:
            break
        if 0 < count[s] <= rem:
            taken[s] = True
            rem -= int(count[s])
    return taken


def refine_sentences(score, kind, seg_start, keep_ratio: float):
    """Sentence-level selection (Sec. 3.2: choosing KVCache entries amounts to choosing whole
    sentences; Sec. 4, Table 2: the "Refine (Sentences)" variant).

    seg_start [n_seg+1] are sentence boundaries that tile the content range
    [seg_start[0], seg_start[-1]); prompt positions outside it (prefix, suffix) are always kept,
    received positions never.  With the token budget B = clamp(k_total - #always_kept, 0,
    #content prompt tokens), sentences are visited by decreasing value (ties: lower sentence
    first) and a sentence is taken iff it still fits the remaining budget, until the budget
    is used up.  Returns (keep uint8 [n], n_kept, taken [n_seg] bool)."""
    score = np.asarray(score, dtype=np.float64)
    n = len(score)
    kind = np.zeros(n, np.uint8) if kind is None else np.asarray(kind, np.uint8)
    seg_start = np.asarray(seg_start, dtype=np.int64)
    lo, hi = int(seg_start[0]), int(seg_start[-1])
    pos = np.arange(n)
    is_prompt = kind == PROMPT
    content = is_prompt & (pos >= lo) & (pos < hi)
    always = is_prompt & ~content
    k_total = keep_count(keep_ratio, int(is_prompt.sum()))
    budget = min(max(k_total - int(always.sum()), 0), int(content.sum()))
    value, count = sentence_values(score, kind, seg_start)
    taken = select_sentences(value, count, budget)
    keep = np.zeros(n, dtype=np.uint8)
    keep[always] = 1
    for s in np.nonzero(taken)[0]:
        sl = slice(int(seg_start[s]), int(seg_start[s + 1]))
        keep[sl] = is_prompt[sl]
    return keep, int(keep.sum()), taken


def pack_mask_bits(keep) -> np.ndarray:
    """Mask tensor as a bit stream (Sec. 3.2: the mask is treated as a bit stream before
    compression): bit (i mod 8) of byte i // 8 is keep[i], least significant bit first;
    the last byte is padded with zeros."""
    keep = np.asarray(keep, dtype=np.uint8)
    return np.packbits(keep != 0, bitorder="little")


def refine_vote(colsum, kind, cand_lo: int, cand_hi: int, keep_ratio: float,
                pool_kind: str = "none", pool_width: int = 1):
    """Per-head selection followed by a vote (Sec. 3.2 picks the top-valued indices of every
    head at ratio r, yet ONE mask of the prompt's length is sent).  The paper does not say how
    the per-head index sets become one mask; this is the alternative to summing the heads first
    ("parity unpinned" as a reading):

      1. every head h selects its own k candidates with the largest pooled column sums
         (the same candidates, the same k and the same tie rule as refine_topk);
      2. votes[j] = number of heads that selected position j;
      3. the mask keeps the k candidates with the most votes; equal votes are ordered by the
         pooled column sums added over the heads, then by the lower position.

    colsum is [n_heads, n].  Returns (keep uint8 [n], n_kept, votes int32 [n], total fp64 [n])
    with total the head sum of the pooled values."""
    cs = np.asarray(colsum, dtype=np.float64)
    n_heads, n = cs.shape
    kind = np.zeros(n, dtype=np.uint8) if kind is None else np.asarray(kind, dtype=np.uint8)
    pooled = pool1d(cs, pool_kind, pool_width)
    pos = np.arange(n)
    is_prompt = kind == PROMPT
    cand = is_prompt & (pos >= cand_lo) & (pos < cand_hi)
    always = is_prompt & ~cand
    votes = np.zeros(n, dtype=np.int32)
    k = 0
    for h in range(n_heads):
        keep_h, _, k = refine_topk(pooled[h], kind, cand_lo, cand_hi, keep_ratio)
        votes += (keep_h.astype(bool) & cand).astype(np.int32)
    total = pooled.sum(axis=0)
    idx = pos[cand]
    # descending votes, then descending total, then ascending position
    order = np.lexsort((idx, -total[idx], -votes[idx]))
    keep = np.zeros(n, dtype=np.uint8)
    keep[always] = 1
    keep[idx[order[:k]]] = 1
    return keep, int(keep.sum()), votes, total


def solve_rl(l: float, k_c: float, k_d: float, delta: float, delta_c: float, xi: float,
             tau: float, tpot_c: float, tpot_d: float, m_max: int = 1 << 16):
    """Problem P of Sec. 3.4 (Algorithm 1, "Solve r and L upon P"): minimise TTFT_d over the
    refinement ratio r (real, 0 < r <= 1, so the quality floor xi must be positive) and the
    number L of cloud tokens (integer > 1).

    Model, all times in one unit, lengths in tokens:
      TTFT_c(l)   = k_c*l + delta_c                       (Eq. 2: prefill_c + compress + RTT)
      TTFT_d(r)   = k_c*l + delta + k_d*r*l               (Eq. 3 with Sec. 3.4's estimates;
                                                           delta >= compress + decompress + RTT)
      Eq. 5 (r):  xi <= r <= 1 - (k_c + delta/l)/k_d
      Eq. 6 (L):  (k_d*r*l - TTFT_c)/(tau - TPOT_d) <= L-1 <= (TTFT_d - TTFT_c)/TPOT_c
    TTFT_d grows with r, so the optimum is the smallest r for which some integer L-1 >= 1 fits
    Eq. 6; among the L that fit, the smallest is taken (Sec. 4.2: the optimum is reached when L
    matches its lower bound).  Written as the plain scan over m = L-1 = 1..m_max.

    Returns dict(feasible, r, L, ttft_c, ttft_d, tpot_smooth) (r, L = nan, 0 if infeasible)."""
    l, k_c, k_d, delta, delta_c = float(l), float(k_c), float(k_d), float(delta), float(delta_c)
    xi, tau, tpot_c, tpot_d = float(xi), float(tau), float(tpot_c), float(tpot_d)
    ttft_c = k_c * l + delta_c
    r_ub = min(1.0, 1.0 - (k_c + delta / l) / k_d)
    best = None
    if tau > tpot_d and l > 0 and k_d > 0 and k_c >= 0 and tpot_c > 0 and xi > 0 and 0 <= delta_c <= delta:
        for m in range(1, m_max + 1):
            # upper bound of Eq. 5 holds from this r upward
            r_from = (m * tpot_c - (delta - delta_c)) / (k_d * l)
            # lower bound of Eq. 5 holds up to this r
            r_to = (m * (tau - tpot_d) + ttft_c) / (k_d * l)
            lo = max(xi, r_from)
            hi = min(r_ub, r_to)
            if lo <= hi and lo > 0.0 and (best is None or lo < best[0]):
                best = (lo, m)
            if r_from > r_ub:
                break                       # r_from only grows with m
    if best is None:
        return dict(feasible=False, r=float("nan"), L=0, ttft_c=ttft_c, ttft_d=float("nan"),
                    tpot_smooth=float("nan"))
    r, m = best
    return dict(feasible=True, r=r, L=m + 1, ttft_c=ttft_c, ttft_d=k_c * l + delta + k_d * r * l,
                tpot_smooth=tpot_d + (k_d * r * l - ttft_c) / m)


class SequenceOracle:
    """Literal replay of the call sequence on growing arrays (Sec. 3.3, Algorithm 2).

    Every prefill chunk and every block of received tokens appends its rows to the
    arrays and evaluates attention of exactly those rows against everything appended
    so far; window rows add their probability rows to the column sums.
    """

    def __init__(self, n_q_heads: int, n_kv_heads: int, head_dim: int, scale: float,
                 sliding_window: int = 0):
        self.hq, self.hkv, self.d, self.scale = n_q_heads, n_kv_heads, head_dim, float(scale)
        self.sliding_window = int(sliding_window)
        self.q = np.zeros((0, n_q_heads, head_dim))
        self.k = np.zeros((0, n_kv_heads, head_dim))
        self.v = np.zeros((0, n_kv_heads, head_dim))
        self.kind = np.zeros(0, dtype=np.uint8)
        self.window = np.zeros(0, dtype=np.uint8)
        self.colsum = np.zeros((n_q_heads, 0))

    @property
    def n_tokens(self) -> int:
        return self.q.shape[0]

    def _append(self, q, k, v, kind: int, window: bool):
        pos0, n = self.n_tokens, np.asarray(q).shape[0]
        self.q = np.concatenate([self.q, _f64(q)], axis=0)
        self.k = np.concatenate([self.k, _f64(k)], axis=0)
        self.v = np.concatenate([self.v, _f64(v)], axis=0)
        self.kind = np.concatenate([self.kind, np.full(n, kind, dtype=np.uint8)])
        self.window = np.concatenate([self.window, np.full(n, 1 if window else 0, np.uint8)])
        self.colsum = np.concatenate([self.colsum, np.zeros((self.hq, n))], axis=1)
        rows = np.arange(pos0, pos0 + n)
        out, lse = attention_rows(self.q, self.k, self.v, self.scale, rows, self.sliding_window)
        if window and n:
            w = np.zeros(self.n_tokens, dtype=np.uint8)
            w[rows] = 1
            self.colsum += colsum(self.q, self.k, self.scale, w, self.sliding_window)
        return out, lse

    def prefill_chunk(self, q, k, v, window: bool = False):
        return self._append(q, k, v, PROMPT, window)

    def append_received(self, q, k, v, window: bool = False):
        return self._append(q, k, v, RECEIVED, window)

    def token_importance(self, pool_kind: str = "none", pool_width: int = 1) -> np.ndarray:
        return importance([self.colsum], pool_kind, pool_width)
