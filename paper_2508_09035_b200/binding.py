"""ctypes binding of libpdd: the same names as the C ABI, argument marshalling only.

Every computation happens in the library's CUDA kernels.  There is no fallback: if
libpdd.so has not been built (python -m paper_2508_09035_b200.build) loading fails with
an error.  PyTorch is used by the convenience class only for device memory and streams.
"""
from __future__ import annotations

import ctypes
import os
from typing import Dict, List, Optional, Sequence, Tuple

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(HERE, "libpdd.so")

PDD_OK, PDD_ERR_INVALID, PDD_ERR_STATE, PDD_ERR_CAPACITY = 0, 1, 2, 3
PDD_ERR_CUDA, PDD_ERR_TIMEOUT, PDD_ERR_UNSUPPORTED = 4, 5, 6
PDD_WINDOW = 1
PDD_POOL_NONE, PDD_POOL_AVG, PDD_POOL_MAX = 0, 1, 2
PATH_TENSOR_CORE, PATH_SIMT, PATH_TENSOR_CORE_SIMPLE = 0, 1, 2

EXPORTS = [
    "pdd_kv_bytes_required", "pdd_kv_alloc", "pdd_kv_free", "pdd_kv_reset", "pdd_kv_length",
    "pdd_prefill_chunk", "pdd_append_received", "pdd_token_importance",
    "pdd_token_importance_batched", "pdd_importance_topk", "pdd_kv_kinds",
    "pdd_refine_topk", "pdd_refine_topk_batched", "pdd_refine_from_colsum_static", "pdd_refine_sentences", "pdd_pack_mask",
    "pdd_refine_vote", "pdd_refine_vote_workspace", "pdd_solve_rl",
    "pdd_status", "pdd_clear_status", "pdd_selftest_wait_timeout", "pdd_debug_fail_launch",
    "pdd_export_colsum",
    "pdd_export_kv", "pdd_export_kinds", "pdd_last_lse", "pdd_trace_enable", "pdd_trace_read",
    "pdd_set_kernel_path", "pdd_set_schedule", "pdd_strerror", "pdd_last_error_detail",
]


class pdd_kv_config(ctypes.Structure):
    _fields_ = [("n_q_heads", ctypes.c_int32), ("n_kv_heads", ctypes.c_int32),
                ("head_dim", ctypes.c_int32), ("page_tokens", ctypes.c_int32),
                ("max_seqs", ctypes.c_int32), ("sliding_window", ctypes.c_int32),
                ("max_tokens_total", ctypes.c_int64), ("max_tokens_per_seq", ctypes.c_int64),
                ("max_rows_per_call", ctypes.c_int64), ("softmax_scale", ctypes.c_float),
                ("reserved_f", ctypes.c_float)]


class pdd_batch(ctypes.Structure):
    _fields_ = [("n_seqs", ctypes.c_int32), ("seq_id", ctypes.POINTER(ctypes.c_int32)),
                ("pos0", ctypes.POINTER(ctypes.c_int64)), ("len", ctypes.POINTER(ctypes.c_int32)),
                ("tok_offset", ctypes.POINTER(ctypes.c_int64))]


class pdd_rl_problem(ctypes.Structure):
    _fields_ = [(n, ctypes.c_double) for n in
                ("l", "k_c", "k_d", "delta", "delta_c", "xi", "tau", "tpot_c", "tpot_d")]


class pdd_rl_solution(ctypes.Structure):
    _fields_ = [("feasible", ctypes.c_int32), ("L", ctypes.c_int32), ("r", ctypes.c_double),
                ("ttft_c", ctypes.c_double), ("ttft_d", ctypes.c_double),
                ("tpot_smooth", ctypes.c_double)]


class PddError(RuntimeError):
    def __init__(self, status: int, where: str, detail: str):
        self.status = status
        super().__init__("%s: status %d (%s)" % (where, status, detail))


_lib = None


def lib():
    """Load libpdd.so (once).  Raises if it has not been built."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ImportError("libpdd.so is missing at %s; build it with "
                          "`python -m paper_2508_09035_b200.build` (needs nvcc)" % LIB_PATH)
    L = ctypes.CDLL(LIB_PATH)
    vp, i32, i64, u32 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_uint32
    P = ctypes.POINTER
    L.pdd_kv_bytes_required.argtypes = [P(pdd_kv_config), P(ctypes.c_size_t)]
    L.pdd_kv_alloc.argtypes = [P(pdd_kv_config), vp, ctypes.c_size_t, vp, P(vp)]
    L.pdd_kv_free.argtypes = [vp]
    L.pdd_kv_reset.argtypes = [vp, i32, vp]
    L.pdd_kv_length.argtypes = [vp, i32, P(i64)]
    for f in (L.pdd_prefill_chunk, L.pdd_append_received):
        f.argtypes = [vp, P(pdd_batch), vp, vp, vp, vp, u32, vp]
    L.pdd_token_importance.argtypes = [vp, i32, i32, i32, vp, i32, vp]
    L.pdd_token_importance_batched.argtypes = [vp, i32, P(i32), i32, i32, vp, P(i64), i32, vp]
    L.pdd_importance_topk.argtypes = [vp, i32, i32, i32, vp, i32, i64, i64, ctypes.c_double,
                                      vp, vp, vp]
    L.pdd_kv_kinds.argtypes = [vp, i32, P(vp)]
    L.pdd_refine_topk.argtypes = [vp, vp, i64, i64, i64, ctypes.c_double, vp, vp, vp]
    L.pdd_refine_topk_batched.argtypes = [vp, vp, i32, P(i64), P(i64), P(i64), ctypes.c_double,
                                          vp, vp, vp]
    L.pdd_refine_from_colsum_static.argtypes = [vp, i64, i32, vp, i64, i32, i32, i64, i64,
                                                ctypes.c_double, vp, vp, vp]
    L.pdd_refine_sentences.argtypes = [vp, vp, i64, vp, i32, ctypes.c_double, vp, vp, vp, vp]
    L.pdd_pack_mask.argtypes = [vp, i64, vp, vp]
    L.pdd_refine_vote_workspace.argtypes = [i32, i64, P(ctypes.c_size_t)]
    L.pdd_refine_vote.argtypes = [vp, i64, i32, vp, i64, i32, i32, i64, i64, ctypes.c_double,
                                  vp, vp, vp, vp, ctypes.c_size_t, vp]
    L.pdd_solve_rl.argtypes = [P(pdd_rl_problem), i32, P(pdd_rl_solution)]
    L.pdd_status.argtypes = [vp, vp, P(i32)]
    L.pdd_clear_status.argtypes = [vp, vp]
    L.pdd_selftest_wait_timeout.argtypes = [vp, u32, vp]
    L.pdd_debug_fail_launch.argtypes = [vp, i32]
    L.pdd_export_colsum.argtypes = [vp, i32, vp, vp]
    L.pdd_export_kv.argtypes = [vp, i32, vp, vp, vp]
    L.pdd_export_kinds.argtypes = [vp, i32, vp, vp]
    L.pdd_last_lse.argtypes = [vp, P(vp), P(i64)]
    L.pdd_trace_enable.argtypes = [vp, i32]
    L.pdd_trace_read.argtypes = [vp, i32, P(ctypes.c_char_p), P(i64), P(ctypes.c_double), P(i32)]
    L.pdd_set_kernel_path.argtypes = [vp, i32]
    L.pdd_set_schedule.argtypes = [vp, i32]
    L.pdd_strerror.argtypes = [ctypes.c_int]
    L.pdd_strerror.restype = ctypes.c_char_p
    L.pdd_last_error_detail.restype = ctypes.c_char_p
    _lib = L
    return L


def _check(rc: int, where: str):
    if rc != PDD_OK:
        L = lib()
        raise PddError(rc, where, "%s: %s" % (L.pdd_strerror(rc).decode(),
                                             L.pdd_last_error_detail().decode()))


def make_batch(seq_ids: Sequence[int], pos0: Sequence[int], lens: Sequence[int]):
    """Host-side pdd_batch plus the ctypes arrays that keep it alive."""
    n = len(seq_ids)
    a_id = (ctypes.c_int32 * n)(*seq_ids)
    a_p0 = (ctypes.c_int64 * n)(*pos0)
    a_ln = (ctypes.c_int32 * n)(*lens)
    offs = [0]
    for x in lens:
        offs.append(offs[-1] + int(x))
    a_off = (ctypes.c_int64 * (n + 1))(*offs)
    b = pdd_batch(n, a_id, a_p0, a_ln, a_off)
    return b, (a_id, a_p0, a_ln, a_off)


# ------------------------------------------------------------------ same-name thin calls

def pdd_kv_bytes_required(cfg: pdd_kv_config) -> int:
    n = ctypes.c_size_t(0)
    _check(lib().pdd_kv_bytes_required(ctypes.byref(cfg), ctypes.byref(n)), "pdd_kv_bytes_required")
    return int(n.value)


def pdd_kv_alloc(cfg: pdd_kv_config, dev_ptr: int, nbytes: int, stream: int) -> int:
    h = ctypes.c_void_p()
    _check(lib().pdd_kv_alloc(ctypes.byref(cfg), dev_ptr, nbytes, stream, ctypes.byref(h)),
           "pdd_kv_alloc")
    return h.value


def pdd_kv_free(h: int):
    _check(lib().pdd_kv_free(h), "pdd_kv_free")


def pdd_kv_reset(h: int, seq_id: int, stream: int):
    _check(lib().pdd_kv_reset(h, seq_id, stream), "pdd_kv_reset")


def pdd_kv_length(h: int, seq_id: int) -> int:
    n = ctypes.c_int64(0)
    _check(lib().pdd_kv_length(h, seq_id, ctypes.byref(n)), "pdd_kv_length")
    return int(n.value)


def pdd_prefill_chunk(h, batch, q_ptr, k_ptr, v_ptr, out_ptr, flags, stream):
    _check(lib().pdd_prefill_chunk(h, ctypes.byref(batch), q_ptr, k_ptr, v_ptr, out_ptr, flags,
                                   stream), "pdd_prefill_chunk")


def pdd_append_received(h, batch, q_ptr, k_ptr, v_ptr, out_ptr, flags, stream):
    _check(lib().pdd_append_received(h, ctypes.byref(batch), q_ptr, k_ptr, v_ptr, out_ptr, flags,
                                     stream), "pdd_append_received")


def pdd_token_importance(h, seq_id, pool_kind, pool_k, score_ptr, accumulate, stream):
    _check(lib().pdd_token_importance(h, seq_id, pool_kind, pool_k, score_ptr, accumulate, stream),
           "pdd_token_importance")


def pdd_token_importance_batched(h, seq_ids, pool_kind, pool_k, score_ptr, offsets, accumulate,
                                 stream):
    n = len(seq_ids)
    a_id = (ctypes.c_int32 * n)(*seq_ids)
    a_off = (ctypes.c_int64 * (n + 1))(*offsets)
    _check(lib().pdd_token_importance_batched(h, n, a_id, pool_kind, pool_k, score_ptr, a_off,
                                              accumulate, stream), "pdd_token_importance_batched")


def pdd_importance_topk(h, seq_id, pool_kind, pool_k, score_ptr, accumulate, cand_lo, cand_hi,
                        keep_ratio, keep_ptr, n_kept_ptr, stream):
    _check(lib().pdd_importance_topk(h, seq_id, pool_kind, pool_k, score_ptr, accumulate, cand_lo,
                                     cand_hi, keep_ratio, keep_ptr, n_kept_ptr, stream),
           "pdd_importance_topk")


def pdd_kv_kinds(h, seq_id) -> int:
    p = ctypes.c_void_p()
    _check(lib().pdd_kv_kinds(h, seq_id, ctypes.byref(p)), "pdd_kv_kinds")
    return p.value


def pdd_refine_topk(score_ptr, kinds_ptr, n, cand_lo, cand_hi, keep_ratio, keep_ptr, n_kept_ptr,
                    stream):
    _check(lib().pdd_refine_topk(score_ptr, kinds_ptr, n, cand_lo, cand_hi, keep_ratio, keep_ptr,
                                 n_kept_ptr, stream), "pdd_refine_topk")


def pdd_refine_topk_batched(score_ptr, kinds_ptr, offsets, cand_lo, cand_hi, keep_ratio, keep_ptr,
                            n_kept_ptr, stream):
    n = len(cand_lo)
    a_off = (ctypes.c_int64 * (n + 1))(*offsets)
    a_lo = (ctypes.c_int64 * n)(*cand_lo)
    a_hi = (ctypes.c_int64 * n)(*cand_hi)
    _check(lib().pdd_refine_topk_batched(score_ptr, kinds_ptr, n, a_off, a_lo, a_hi, keep_ratio,
                                         keep_ptr, n_kept_ptr, stream), "pdd_refine_topk_batched")


PDD_STATIC_SCORE_MAX = 65536


def pdd_refine_from_colsum_static(colsum_ptr, ld, n_heads, kinds_ptr, n, pool_kind, pool_k,
                                  cand_lo, cand_hi, keep_ratio, keep_ptr, n_kept_ptr, stream):
    """Importance reduction + top-k without any allocation: the intermediate score vector
    lives in a fixed buffer inside libpdd (at most PDD_STATIC_SCORE_MAX positions).  Meant
    for callers that own their inputs and outputs but may not allocate device memory on
    the request path; calls on one device share the buffer and must not overlap."""
    _check(lib().pdd_refine_from_colsum_static(colsum_ptr, ld, n_heads, kinds_ptr, n, pool_kind,
                                               pool_k, cand_lo, cand_hi, keep_ratio, keep_ptr,
                                               n_kept_ptr, stream),
           "pdd_refine_from_colsum_static")


def pdd_refine_sentences(score_ptr, kinds_ptr, n, seg_start_ptr, n_seg, keep_ratio, keep_ptr,
                         n_kept_ptr, seg_value_ptr, stream):
    _check(lib().pdd_refine_sentences(score_ptr, kinds_ptr, n, seg_start_ptr, n_seg, keep_ratio,
                                      keep_ptr, n_kept_ptr, seg_value_ptr, stream),
           "pdd_refine_sentences")


def pdd_pack_mask(keep_ptr, n, bits_ptr, stream):
    _check(lib().pdd_pack_mask(keep_ptr, n, bits_ptr, stream), "pdd_pack_mask")


def pdd_refine_vote_workspace(n_heads: int, n: int) -> int:
    b = ctypes.c_size_t(0)
    _check(lib().pdd_refine_vote_workspace(n_heads, n, ctypes.byref(b)), "pdd_refine_vote_workspace")
    return int(b.value)


def pdd_refine_vote(colsum_ptr, ld, n_heads, kinds_ptr, n, pool_kind, pool_k, cand_lo, cand_hi,
                    keep_ratio, keep_ptr, n_kept_ptr, votes_ptr, workspace_ptr, workspace_bytes,
                    stream):
    _check(lib().pdd_refine_vote(colsum_ptr, ld, n_heads, kinds_ptr, n, pool_kind, pool_k, cand_lo,
                                 cand_hi, keep_ratio, keep_ptr, n_kept_ptr, votes_ptr,
                                 workspace_ptr, workspace_bytes, stream), "pdd_refine_vote")


def pdd_solve_rl(problems: Sequence[Sequence[float]]) -> List[dict]:
    """problems: rows of (l, k_c, k_d, delta, delta_c, xi, tau, tpot_c, tpot_d); host only."""
    n = len(problems)
    arr = (pdd_rl_problem * max(n, 1))(*[pdd_rl_problem(*[float(x) for x in p]) for p in problems])
    out = (pdd_rl_solution * max(n, 1))()
    _check(lib().pdd_solve_rl(arr, n, out), "pdd_solve_rl")
    return [dict(feasible=bool(o.feasible), L=int(o.L), r=o.r, ttft_c=o.ttft_c, ttft_d=o.ttft_d,
                 tpot_smooth=o.tpot_smooth) for o in out[:n]]


def pdd_status(h, stream) -> int:
    v = ctypes.c_int32(0)
    _check(lib().pdd_status(h, stream, ctypes.byref(v)), "pdd_status")
    return int(v.value)


def pdd_clear_status(h, stream):
    _check(lib().pdd_clear_status(h, stream), "pdd_clear_status")


def pdd_selftest_wait_timeout(h, limit_us: int, stream):
    _check(lib().pdd_selftest_wait_timeout(h, limit_us, stream), "pdd_selftest_wait_timeout")


def pdd_debug_fail_launch(h, nth: int):
    _check(lib().pdd_debug_fail_launch(h, nth), "pdd_debug_fail_launch")


def pdd_export_colsum(h, seq_id, dst_ptr, stream):
    _check(lib().pdd_export_colsum(h, seq_id, dst_ptr, stream), "pdd_export_colsum")


def pdd_export_kv(h, seq_id, k_ptr, v_ptr, stream):
    _check(lib().pdd_export_kv(h, seq_id, k_ptr, v_ptr, stream), "pdd_export_kv")


def pdd_export_kinds(h, seq_id, dst_ptr, stream):
    _check(lib().pdd_export_kinds(h, seq_id, dst_ptr, stream), "pdd_export_kinds")


def pdd_last_lse(h) -> Tuple[int, int]:
    p, ld = ctypes.c_void_p(), ctypes.c_int64(0)
    _check(lib().pdd_last_lse(h, ctypes.byref(p), ctypes.byref(ld)), "pdd_last_lse")
    return p.value, int(ld.value)


def pdd_trace_enable(h, on: bool):
    _check(lib().pdd_trace_enable(h, 1 if on else 0), "pdd_trace_enable")


def pdd_trace_read(h) -> Dict[str, Tuple[int, float]]:
    cap = 32
    names = (ctypes.c_char_p * cap)()
    cnt = (ctypes.c_int64 * cap)()
    ms = (ctypes.c_double * cap)()
    n = ctypes.c_int32(0)
    _check(lib().pdd_trace_read(h, cap, names, cnt, ms, ctypes.byref(n)), "pdd_trace_read")
    return {names[i].decode(): (int(cnt[i]), float(ms[i])) for i in range(n.value)}


def pdd_set_kernel_path(h, path: int):
    _check(lib().pdd_set_kernel_path(h, path), "pdd_set_kernel_path")


def pdd_set_schedule(h, mode: int):
    _check(lib().pdd_set_schedule(h, mode), "pdd_set_schedule")


# ------------------------------------------------------------------ convenience wrapper

class KVCache:
    """A pdd_kv handle over a torch-owned device arena.  Marshals tensors to pointers."""

    def __init__(self, n_q_heads: int, n_kv_heads: int, head_dim: int, page_tokens: int = 64,
                 max_seqs: int = 1, max_tokens_total: int = 0, max_tokens_per_seq: int = 0,
                 max_rows_per_call: int = 0, softmax_scale: float = 0.0, device="cuda:0",
                 kernel_path: int = PATH_TENSOR_CORE, sliding_window: int = 0):
        import torch
        self.torch = torch
        self.device = torch.device(device)
        self.cfg = pdd_kv_config(n_q_heads, n_kv_heads, head_dim, page_tokens, max_seqs,
                                 int(sliding_window), max_tokens_total, max_tokens_per_seq,
                                 max_rows_per_call or max_tokens_per_seq, softmax_scale, 0.0)
        nbytes = pdd_kv_bytes_required(self.cfg)
        with torch.cuda.device(self.device):
            self.arena = torch.empty(nbytes + 256, dtype=torch.uint8, device=self.device)
            ptr = (self.arena.data_ptr() + 255) // 256 * 256
            self.h = pdd_kv_alloc(self.cfg, ptr, nbytes, self.stream)
        self.arena_bytes = nbytes
        if kernel_path != PATH_TENSOR_CORE:
            pdd_set_kernel_path(self.h, kernel_path)

    def set_schedule(self, mode: int):
        pdd_set_schedule(self.h, mode)

    @property
    def stream(self) -> int:
        return self.torch.cuda.current_stream(self.device).cuda_stream

    def close(self):
        if getattr(self, "h", None):
            self.torch.cuda.synchronize(self.device)
            pdd_kv_free(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _call(self, fn, seq_ids, q, k, v, lens, window, out):
        torch = self.torch
        pos0 = [pdd_kv_length(self.h, s) for s in seq_ids]
        batch, keep = make_batch(seq_ids, pos0, lens)
        for t in (q, k, v):
            assert t.dtype == torch.bfloat16 and t.is_contiguous() and t.is_cuda
        if out is None:
            out = torch.empty_like(q)
        fn(self.h, batch, q.data_ptr(), k.data_ptr(), v.data_ptr(), out.data_ptr(),
           PDD_WINDOW if window else 0, self.stream)
        return out

    def prefill_chunk(self, q, k, v, seq_ids=(0,), lens=None, window=False, out=None):
        lens = [q.shape[0]] if lens is None else list(lens)
        return self._call(pdd_prefill_chunk, list(seq_ids), q, k, v, lens, window, out)

    def append_received(self, q, k, v, seq_ids=(0,), lens=None, window=False, out=None):
        lens = [q.shape[0]] if lens is None else list(lens)
        return self._call(pdd_append_received, list(seq_ids), q, k, v, lens, window, out)

    def length(self, seq_id: int = 0) -> int:
        return pdd_kv_length(self.h, seq_id)

    def token_importance(self, seq_id: int = 0, pool_kind: int = PDD_POOL_NONE, pool_k: int = 1,
                         score=None, accumulate: bool = False):
        torch = self.torch
        n = self.length(seq_id)
        if score is None:
            score = torch.zeros(n, dtype=torch.float32, device=self.device)
        pdd_token_importance(self.h, seq_id, pool_kind, pool_k, score.data_ptr(),
                             1 if accumulate else 0, self.stream)
        return score

    def kinds_ptr(self, seq_id: int = 0) -> int:
        return pdd_kv_kinds(self.h, seq_id)

    def refine_topk(self, score, keep_ratio: float, seq_id: Optional[int] = 0, cand_lo: int = 0,
                    cand_hi: Optional[int] = None):
        """Keep mask for one sequence; kinds come from the cache when seq_id is given."""
        torch = self.torch
        n = int(score.shape[0])
        keep = torch.empty(n, dtype=torch.uint8, device=self.device)
        n_kept = torch.zeros(1, dtype=torch.int32, device=self.device)
        kinds = self.kinds_ptr(seq_id) if seq_id is not None else None
        pdd_refine_topk(score.data_ptr(), kinds, n, cand_lo, n if cand_hi is None else cand_hi,
                        float(keep_ratio), keep.data_ptr(), n_kept.data_ptr(), self.stream)
        return keep, n_kept

    def export_colsum(self, seq_id: int = 0):
        torch = self.torch
        n = self.length(seq_id)
        dst = torch.empty((self.cfg.n_q_heads, n), dtype=torch.float32, device=self.device)
        pdd_export_colsum(self.h, seq_id, dst.data_ptr(), self.stream)
        return dst

    def export_kv(self, seq_id: int = 0):
        torch = self.torch
        n = self.length(seq_id)
        shape = (n, self.cfg.n_kv_heads, self.cfg.head_dim)
        k = torch.empty(shape, dtype=torch.bfloat16, device=self.device)
        v = torch.empty(shape, dtype=torch.bfloat16, device=self.device)
        pdd_export_kv(self.h, seq_id, k.data_ptr(), v.data_ptr(), self.stream)
        return k, v

    def export_kinds(self, seq_id: int = 0):
        torch = self.torch
        dst = torch.empty(self.length(seq_id), dtype=torch.uint8, device=self.device)
        pdd_export_kinds(self.h, seq_id, dst.data_ptr(), self.stream)
        return dst

    def status(self) -> int:
        return pdd_status(self.h, self.stream)

    def reset(self, seq_id: int = 0):
        pdd_kv_reset(self.h, seq_id, self.stream)

    def trace(self, on: bool):
        pdd_trace_enable(self.h, on)

    def trace_read(self):
        return pdd_trace_read(self.h)
