/*
 * libpdd -- chunked causal prefill attention over a growing, paged KV cache, with the
 * attention-mass statistics and top-k keep mask used for prompt refinement.
 *
 * C ABI.  Plain pointers and sizes only.  Unless a parameter says "host", every data
 * pointer is DEVICE memory owned by the caller; the library allocates no device memory
 * (pdd_kv_alloc carves an arena the caller hands in).  All hot calls enqueue work on
 * the caller's CUDA stream (a cudaStream_t passed as void*) and return without
 * synchronising the host.  Every function returns a pdd status code (0 = PDD_OK);
 * nothing throws, aborts or traps.  Device-side problems (a bounded wait that ran out)
 * set a sticky word that pdd_status reads.
 *
 * One stream per handle.  Every call on a pdd_kv shares the handle's scratch (row
 * normalisers, partial results of split key ranges, the ring of call records, cached tensor
 * maps) without any synchronisation of its own: issue all calls of a handle on ONE stream,
 * or order them with events so that the kernels of two calls never overlap on the GPU.
 * Handles are independent of one another.  The host part of a handle is not thread-safe.
 *
 * After a failure.  A hot call that returns an error before or while it enqueues its kernels
 * leaves the handle's host state (lengths, pages) as it found it, so the same call can be
 * repeated; cache rows a partly enqueued call may have written lie beyond the sequences'
 * lengths and are overwritten by the next call at those positions.  Once the sticky word is
 * PDD_ERR_TIMEOUT, every later kernel of the handle returns without doing any work (outputs
 * are not written) until pdd_clear_status; what the interrupted kernels left in the cache is
 * undefined, so reset the sequences that were in flight (pdd_kv_reset) before reusing them.
 *
 * Conventions
 *   q, out : bf16, token-major [rows][n_q_heads][head_dim], contiguous, 16-byte aligned
 *   k, v   : bf16, token-major [rows][n_kv_heads][head_dim], contiguous, 16-byte aligned
 *   rows of all sequences of one call are packed back to back; sequence i owns rows
 *   tok_offset[i] .. tok_offset[i+1]-1 and len[i] == tok_offset[i+1]-tok_offset[i].
 *   Query head h reads KV head h / (n_q_heads / n_kv_heads).
 *   Position kinds: 0 = prompt token, 1 = token received from the cloud.
 */
#ifndef PDD_H_
#define PDD_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum {
  PDD_OK = 0,
  PDD_ERR_INVALID = 1,     /* bad argument (null, misaligned, out of range)            */
  PDD_ERR_STATE = 2,       /* call does not fit the sequence state (pos0 != length)    */
  PDD_ERR_CAPACITY = 3,    /* page pool, per-sequence or per-call capacity exceeded    */
  PDD_ERR_CUDA = 4,        /* a CUDA runtime/driver call failed                        */
  PDD_ERR_TIMEOUT = 5,     /* a bounded device-side wait ran out (sticky)              */
  PDD_ERR_UNSUPPORTED = 6  /* shape the kernels do not cover, or no sm_100 device      */
};

/* flags of pdd_prefill_chunk / pdd_append_received */
enum {
  PDD_WINDOW = 1u          /* the rows of this call join the observation window        */
};

/* pool_kind of pdd_token_importance */
enum { PDD_POOL_NONE = 0, PDD_POOL_AVG = 1, PDD_POOL_MAX = 2 };

typedef struct pdd_kv pdd_kv;      /* opaque handle; owns host metadata only */

typedef struct {
  int32_t n_q_heads;           /* multiple of n_kv_heads                                  */
  int32_t n_kv_heads;
  int32_t head_dim;            /* 64 or 128                                               */
  int32_t page_tokens;         /* tokens per KV page: 64 or 128                           */
  int32_t max_seqs;            /* sequence ids are 0 .. max_seqs-1                        */
  int32_t sliding_window;      /* w > 0: row p sees keys max(0,p-w+1)..p (the on-device    */
                               /* sliding-window attention of Sec. 3.3); 0 = plain causal  */
  int64_t max_tokens_total;    /* page pool capacity in tokens (rounded up to pages)      */
  int64_t max_tokens_per_seq;  /* longest sequence (prompt + received)                    */
  int64_t max_rows_per_call;   /* most rows (summed over sequences) one call may carry    */
  float softmax_scale;         /* 0 => 1/sqrt(head_dim)                                   */
  float reserved_f;            /* must be 0                                               */
} pdd_kv_config;

/* One call's batch.  All four arrays are HOST memory, read before the call returns. */
typedef struct {
  int32_t n_seqs;
  const int32_t* seq_id;      /* [n_seqs], distinct                                      */
  const int64_t* pos0;        /* [n_seqs], must equal the sequence's current length      */
  const int32_t* len;         /* [n_seqs], rows of this call (0 allowed)                 */
  const int64_t* tok_offset;  /* [n_seqs+1], packed row offsets                          */
} pdd_batch;

/*
 * KV cache set-up.  The KV cache and the other intermediate data stay in HBM and grow with
 * the prompt (Sec. 2.1 and Sec. 3.2, preliminaries): the cache is a pool of fixed-size pages
 * plus a page table per sequence.
 *
 * pdd_kv_bytes_required: size of the device arena for a configuration.
 * pdd_kv_alloc: dev_buf is device memory of at least that size, 256-byte aligned, owned
 *   by the caller and kept alive until pdd_kv_free; the library carves it into K/V page
 *   pools, page tables, position kinds, per-head column sums and per-call scratch, and
 *   clears what must start at zero on `stream` (the caller orders later calls after it).
 *   Must be called with the target device current.  PDD_ERR_UNSUPPORTED for shapes
 *   outside the ranges above or on a device that is not sm_100.
 * pdd_kv_free: releases host metadata only.  pdd_kv_reset: returns a sequence's pages
 *   to the pool and zeroes its column sums (asynchronously on `stream`).
 */
int pdd_kv_bytes_required(const pdd_kv_config* cfg, size_t* bytes);
int pdd_kv_alloc(const pdd_kv_config* cfg, void* dev_buf, size_t bytes, void* stream,
                 pdd_kv** out);
int pdd_kv_free(pdd_kv* kv);
int pdd_kv_reset(pdd_kv* kv, int32_t seq_id, void* stream);
int pdd_kv_length(const pdd_kv* kv, int32_t seq_id, int64_t* n_tokens);

/*
 * pdd_prefill_chunk -- chunked prefill (Sec. 3.3 "LLM Engine": the prompt is prefilled
 * chunk by chunk; attention is softmax(Q K^T / sqrt(h)) V, Sec. 2.2.3, causal).
 * For every sequence of the batch: appends the chunk's K/V rows to the cache at
 * positions pos0 .. pos0+len-1 (kind = prompt), then writes, for each row i and head h,
 *   out[i][h] = softmax_j(scale * q[i][h] . K[j]) V[j],  j = 0 .. pos0+i.
 * With PDD_WINDOW the rows also add their normalised attention weights to the
 * per-head column sums of the sequence (Sec. 3.2: weights of the observation window
 * against the entire K, summed along the query dimension).
 * Errors (checked before anything is enqueued): PDD_ERR_STATE if pos0 differs from the
 * current length, PDD_ERR_CAPACITY if pages, per-sequence or per-call limits would be
 * exceeded, PDD_ERR_INVALID for bad pointers/ids.
 *
 * pdd_append_received -- the same for tokens received from the cloud, which are fed to
 * the on-device model as known inputs (Algorithm 2; Sec. 2.2.2 token-level assist).
 * Positions get kind = received: they are attended to by later rows and collect column
 * mass, but are never selectable by pdd_refine_topk.
 */
int pdd_prefill_chunk(pdd_kv* kv, const pdd_batch* batch, const void* q, const void* k,
                      const void* v, void* out, uint32_t flags, void* stream);
int pdd_append_received(pdd_kv* kv, const pdd_batch* batch, const void* q, const void* k,
                        const void* v, void* out, uint32_t flags, void* stream);

/*
 * pdd_token_importance -- per-position importance of one sequence (Sec. 3.2: after the
 * sum along the query dimension, 1-D pooling, then heads are merged):
 *   score[j] (+)= sum_h pool(colsum[h])[j],  j = 0 .. length-1.
 * pool_k is odd (1 = no pooling); average pooling pads with zeros and divides by pool_k,
 * max pooling pads with -inf.  accumulate != 0 adds to score (to merge layers, Sec. 4.4
 * "layer selection"), otherwise score is overwritten.  score: fp32 [length].
 */
int pdd_token_importance(pdd_kv* kv, int32_t seq_id, int32_t pool_kind, int32_t pool_k,
                         float* score, int32_t accumulate, void* stream);

/*
 * pdd_token_importance_batched -- the same for several sequences in one launch: sequence
 * seq_ids[i] writes (or adds to) score[offsets[i] .. offsets[i+1]-1]; offsets[i+1]-offsets[i]
 * must equal its length.  seq_ids, offsets: HOST arrays.
 *
 * pdd_importance_topk -- pdd_token_importance followed by pdd_refine_topk for one sequence in
 * one call (Sec. 3.2: sum, pooling, top values), with the position kinds taken from the
 * cache: two kernels chained on the stream, the second starting under the first's tail.
 * Results are bit-identical to the two calls.  (Selections of at most 49152 positions per
 * sequence, through any of the top-k calls, stage the scores in shared memory and read them
 * from global memory once; longer ones read them once per radix pass.)
 */
int pdd_token_importance_batched(pdd_kv* kv, int32_t n_seqs, const int32_t* seq_ids,
                                 int32_t pool_kind, int32_t pool_k, float* score,
                                 const int64_t* offsets, int32_t accumulate, void* stream);
int pdd_importance_topk(pdd_kv* kv, int32_t seq_id, int32_t pool_kind, int32_t pool_k,
                        float* score, int32_t accumulate, int64_t cand_lo, int64_t cand_hi,
                        double keep_ratio, uint8_t* keep, int32_t* n_kept, void* stream);

/* Device pointer to a sequence's kind array (uint8 [length]); valid until pdd_kv_free. */
int pdd_kv_kinds(pdd_kv* kv, int32_t seq_id, const uint8_t** kinds);

/*
 * pdd_refine_topk -- keep mask over n positions (Sec. 3.2: indices with the top values,
 * ratio r; mask with 1 at position i = token i kept; prefix and suffix are not refined).
 * Candidates are positions of kind 0 in [cand_lo, cand_hi); kind-0 positions outside
 * that range are always kept; kind-1 positions are never kept.  With l = number of
 * kind-0 positions, k_total = floor(keep_ratio*l + 1/2) (r = refined/original length,
 * Sec. 2.2.3) and the candidates contribute k = clamp(k_total - #always_kept, 0, #cand)
 * positions: the k largest scores, ties broken toward the lower position.
 * score: fp32 [n], finite and >= 0.  kinds: uint8 [n] or NULL (all prompt).
 * keep: uint8 [n] (0/1).  n_kept: int32 on the device, = popcount(keep).
 * n <= 2^24.  No handle: the call works on any score vector.
 */
int pdd_refine_topk(const float* score, const uint8_t* kinds, int64_t n, int64_t cand_lo,
                    int64_t cand_hi, double keep_ratio, uint8_t* keep, int32_t* n_kept,
                    void* stream);

/* Batched form: sequence i owns positions offsets[i] .. offsets[i+1]-1 of score, kinds,
 * keep; cand ranges are relative to the sequence.  offsets, cand_lo, cand_hi: HOST arrays. */
int pdd_refine_topk_batched(const float* score, const uint8_t* kinds, int32_t n_seqs,
                            const int64_t* offsets, const int64_t* cand_lo,
                            const int64_t* cand_hi, double keep_ratio, uint8_t* keep,
                            int32_t* n_kept, void* stream);

/*
 * pdd_refine_sentences -- sentence-level selection (Sec. 3.2: the KVCache of one sentence
 * is treated as a whole, so the selection of KVCache is a selection of sentences; Sec. 4,
 * the "Refine (Sentences)" variant).
 *   seg_start : int32 [n_seg + 1], DEVICE, increasing; sentence s covers positions
 *               seg_start[s] .. seg_start[s+1]-1; the sentences tile the content range
 *               [seg_start[0], seg_start[n_seg]).  Prompt positions outside that range
 *               (prefix, suffix) are always kept; received positions never.
 *   value of a sentence = mean score of its prompt tokens (the paper names no aggregator;
 *               added one by one in position order in fp32, then one division).
 *   budget    = clamp(floor(keep_ratio*l + 1/2) - #always_kept, 0, #content prompt tokens)
 *               tokens; sentences are visited by decreasing value (ties: lower sentence
 *               first) and a sentence is taken iff it still fits what is left of the budget.
 *   keep      : uint8 [n]; n_kept: int32 on the device (<= floor(keep_ratio*l + 1/2)).
 *   seg_value : optional fp32 [n_seg] (device) receiving the sentence values, or NULL.
 * 1 <= n_seg <= 8192 (PDD_ERR_CAPACITY beyond); score, kinds as in pdd_refine_topk.
 * seg_start is device memory, so the host cannot validate it: the kernel checks that every
 * boundary lies in [0, n] and that they do not decrease.  If they do not, nothing is read or
 * written through a bad boundary: keep is all zeros and n_kept is -1.
 */
int pdd_refine_sentences(const float* score, const uint8_t* kinds, int64_t n,
                         const int32_t* seg_start, int32_t n_seg, double keep_ratio,
                         uint8_t* keep, int32_t* n_kept, float* seg_value, void* stream);

/*
 * pdd_pack_mask -- the mask tensor as a bit stream (Sec. 3.2 serialises the mask as a bit
 * stream before it is compressed): bit (i mod 8) of bits[i / 8] = (keep[i] != 0), least
 * significant bit first, the last byte padded with zeros.  bits: uint8 [(n + 7) / 8].
 */
int pdd_pack_mask(const uint8_t* keep, int64_t n, uint8_t* bits, void* stream);

/*
 * pdd_refine_vote -- per-head selection followed by a vote (Sec. 3.2 takes, for every head,
 * the indices with the largest values at ratio r, but sends one mask of the prompt's length;
 * the paper does not say how the per-head index sets are merged.  pdd_token_importance +
 * pdd_refine_topk sum the heads first; this call is the other reading):
 *   1. every head h takes its own k candidates with the largest pooled column sums
 *      (candidates, k and tie rule exactly as in pdd_refine_topk);
 *   2. votes[j] = number of heads that took candidate j;
 *   3. keep = the k candidates with the most votes; equal votes are ordered by the pooled
 *      column sums added over the heads in index order (fp32), then by the lower position.
 * colsum: fp32 [n_heads][ld], ld >= n (for example from pdd_export_colsum); n_heads <= 255;
 * kinds, cand_lo, cand_hi, keep_ratio, keep, n_kept as in pdd_refine_topk; pool_kind, pool_k
 * as in pdd_token_importance.  votes: optional int32 [n] (device) receiving the vote counts
 * (0 outside the candidates), or NULL.  workspace: device scratch, 256-byte aligned, of at
 * least pdd_refine_vote_workspace(n_heads, n) bytes; contents are undefined afterwards.
 */
int pdd_refine_vote_workspace(int32_t n_heads, int64_t n, size_t* bytes);
int pdd_refine_vote(const float* colsum, int64_t ld, int32_t n_heads, const uint8_t* kinds,
                    int64_t n, int32_t pool_kind, int32_t pool_k, int64_t cand_lo,
                    int64_t cand_hi, double keep_ratio, uint8_t* keep, int32_t* n_kept,
                    int32_t* votes, void* workspace, size_t workspace_bytes, void* stream);

/*
 * pdd_solve_rl -- the offline decision of Algorithm 1 ("solve r and L upon P", Sec. 3.4):
 * minimise the on-device TTFT over the refinement ratio r (real, 0 < r <= 1) and the number
 * L of tokens the cloud generates before it terminates early (integer > 1), for a table of
 * <scene, device, prompt length> combinations.  HOST arrays, host arithmetic (fp64); no GPU
 * work.  Times share one unit, lengths are in tokens.  Per problem:
 *   TTFT_c = k_c*l + delta_c                  (Eq. 2: cloud prefill + compress + RTT)
 *   TTFT_d = k_c*l + delta + k_d*r*l          (Eq. 3; delta bounds compress + decompress + RTT,
 *                                              so delta - delta_c is the decompression time)
 *   Eq. 5:  xi <= r <= 1 - (k_c + delta/l)/k_d
 *   Eq. 6:  (k_d*r*l - TTFT_c)/(tau - TPOT_d) <= L-1 <= (TTFT_d - TTFT_c)/TPOT_c
 * TTFT_d grows with r, so the answer is the smallest r for which an integer L-1 >= 1 fits
 * Eq. 6, and the smallest such L (the optimum sits on L's lower bound, Sec. 4.2).
 * tpot_smooth = TPOT_d + (k_d*r*l - TTFT_c)/(L-1) (Eq. 4).  k_d can be fed from this library's
 * measured prefill rate.  A problem with no solution, or with inputs outside
 * l > 0, k_d > 0, k_c >= 0, tpot_c > 0, tau > tpot_d, 0 <= delta_c <= delta, xi > 0, gets
 * feasible = 0, L = 0 and NaN in r, ttft_d, tpot_smooth; the call still returns PDD_OK.
 */
typedef struct {
  double l;         /* prompt length in tokens                                        */
  double k_c, k_d;  /* prefill time per token in the cloud / on the device            */
  double delta;     /* upper bound of compress + decompress + RTT for this length     */
  double delta_c;   /* the part of delta that precedes the first token: compress + RTT */
  double xi;        /* smallest ratio the scene's quality allows                      */
  double tau;       /* largest tolerable time per output token                        */
  double tpot_c, tpot_d;  /* time per output token in the cloud / on the device       */
} pdd_rl_problem;
typedef struct {
  int32_t feasible;
  int32_t L;
  double r, ttft_c, ttft_d, tpot_smooth;
} pdd_rl_solution;
int pdd_solve_rl(const pdd_rl_problem* problems, int32_t n, pdd_rl_solution* solutions);

/*
 * pdd_refine_from_colsum_static -- importance reduction and top-k in one call that
 * allocates nothing.  (The paper has no counterpart; this is a packaging of the two steps
 * above for a particular kind of caller.)
 *
 * Who needs it: a refiner that runs as a plug-in inside a serving engine which hands out
 * all of its device memory at start-up and gives plug-ins no allocator.  Such a caller
 * owns its inputs and outputs but has nowhere to put the intermediate score vector that
 * pdd_token_importance writes and pdd_refine_topk reads, and it must not call cudaMalloc
 * on the request path (the engine forbids it: an allocation there can fail once the
 * engine's pool has taken the device, and it stalls every stream of the device).
 * Here the score vector lives in a fixed buffer inside the library image instead.
 *
 *   colsum : fp32 [n_heads][ld], ld >= n, per-head column sums (for example the output of
 *            pdd_export_colsum); kinds, cand_lo, cand_hi, keep_ratio, keep, n_kept exactly
 *            as in pdd_refine_topk; pool_kind, pool_k as in pdd_token_importance.
 *   Result : keep and n_kept equal those of pdd_token_importance (accumulate = 0) followed
 *            by pdd_refine_topk on the same data.
 *
 * Limits and rules:
 *   - n <= PDD_STATIC_SCORE_MAX positions; larger n returns PDD_ERR_CAPACITY and launches
 *     nothing.  The buffer (PDD_STATIC_SCORE_MAX floats, 256 KiB) is part of the library
 *     image: every GPU that loads libpdd holds it until the process exits.
 *   - The call makes no cudaMalloc/cudaFree and uses no allocating library routine.
 *   - The first call on each device looks up the buffer's device address (with that device
 *     current, as for every call); make that first call before any stream capture begins.
 *   - All calls on a device share the one buffer.  It keeps the previous call's contents,
 *     and each call overwrites positions 0..n-1 before reading them, so nothing has to be
 *     cleared; but two calls whose kernels overlap on the GPU (different streams without
 *     an ordering between them) race on it.  Order them on one stream or with events.
 */
#define PDD_STATIC_SCORE_MAX 65536
int pdd_refine_from_colsum_static(const float* colsum, int64_t ld, int32_t n_heads,
                                  const uint8_t* kinds, int64_t n, int32_t pool_kind,
                                  int32_t pool_k, int64_t cand_lo, int64_t cand_hi,
                                  double keep_ratio, uint8_t* keep, int32_t* n_kept,
                                  void* stream);

/* Sticky device-side status of the handle (PDD_OK or PDD_ERR_TIMEOUT); synchronises `stream`.
 * pdd_clear_status sets it back to PDD_OK (asynchronously on `stream`). */
int pdd_status(pdd_kv* kv, void* stream, int32_t* sticky_device_status);
int pdd_clear_status(pdd_kv* kv, void* stream);

/*
 * Self-tests of the error paths (not part of the hot path; the paper has no counterpart).
 * pdd_selftest_wait_timeout enqueues a one-warp kernel that waits on a barrier nobody ever
 *   arrives at, with a limit of limit_us microseconds (1..100000) instead of the hot kernels'
 *   2 s; when the limit runs out the kernel raises the handle's sticky word exactly as a hot
 *   kernel does (PDD_ERR_TIMEOUT) and returns normally.  Nothing hangs and nothing traps.
 * pdd_debug_fail_launch makes the nth enqueue step (copy or kernel launch, counted from 1)
 *   of the following hot calls on this handle report PDD_ERR_CUDA without being attempted;
 *   0 disarms.  It exists to test that a failed call leaves the host state unchanged.
 */
int pdd_selftest_wait_timeout(pdd_kv* kv, uint32_t limit_us, void* stream);
int pdd_debug_fail_launch(pdd_kv* kv, int32_t nth);

/*
 * Diagnostics.  pdd_export_colsum copies a sequence's per-head column sums
 * (fp32 [n_q_heads][length]) to dst (device).  pdd_export_kv gathers a sequence's
 * cached K and V back to token-major bf16 [length][n_kv_heads][head_dim] (device).
 * pdd_export_kinds copies the position kinds (uint8 [length]) to dst (device).
 * pdd_last_lse: device pointer to the log-sum-exp (natural log) of the last hot call,
 * fp32 [n_q_heads][ld] with ld = *ld_out, column = packed row index of that call.
 */
int pdd_export_colsum(pdd_kv* kv, int32_t seq_id, float* dst, void* stream);
int pdd_export_kv(pdd_kv* kv, int32_t seq_id, void* k_dst, void* v_dst, void* stream);
int pdd_export_kinds(pdd_kv* kv, int32_t seq_id, uint8_t* dst, void* stream);
int pdd_last_lse(pdd_kv* kv, const float** lse, int64_t* ld_out);

/*
 * Per-kernel timing.  With tracing on, every kernel launch of the handle is bracketed by
 * CUDA events on the launch stream.  pdd_trace_read synchronises, then fills up to `cap`
 * entries (host arrays): name (pointer to a static string), launches, total
 * milliseconds; returns the number of distinct kernels in *n and clears the record.
 */
int pdd_trace_enable(pdd_kv* kv, int32_t on);
int pdd_trace_read(pdd_kv* kv, int32_t cap, const char** names, int64_t* launches,
                   double* total_ms, int32_t* n);

/* Which attention / column-sum kernels run: 0 = pipelined tensor-core (tcgen05) kernels,
 * 1 = plain SIMT kernels, 2 = an unpipelined tensor-core attention kernel; 1 and 2 are
 * kept for bring-up and on-device cross-checks.  Default 0. */
int pdd_set_kernel_path(pdd_kv* kv, int32_t path);

/* How the pipelined attention kernel's work is cut among CTAs: 0 = chosen per call by a
 * cost model (default); 1 = whole tile pairs per CTA; 2 = equal shares of the call's
 * (tile pair, key block) units, partial results merged by a second kernel; 3 = a
 * thread-block cluster per tile pair whose CTAs split the pair's key range and merge
 * through distributed shared memory (falls back to the cost model for a call whose pairs
 * do not fit on the device at once); 4 = the pair-of-CTAs kernel: clusters of two CTAs work
 * on four query tiles of one GQA group at a time, every MMA issued once for both CTAs, each
 * CTA holding half of every K and V block (head_dim 128, no sliding window, group size a
 * multiple of 4; any other call is cut as under 0).  The cost model never picks 4: on B200
 * it is the slower kernel, kept so that the comparison can be repeated.  Results are the
 * same up to rounding; 1-4 exist so that tests can pin each one.  The paper has no
 * counterpart (it leaves the attention kernel to the vendor library, Sec. 3.2). */
int pdd_set_schedule(pdd_kv* kv, int32_t mode);

const char* pdd_strerror(int status);
const char* pdd_last_error_detail(void);   /* thread-local text of the last failure */

#ifdef __cplusplus
}
#endif
#endif /* PDD_H_ */
