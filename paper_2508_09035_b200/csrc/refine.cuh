// importance_reduce: pool each head's column sums along positions, merge heads (and,
// with accumulate, layers) into one score vector.
// radix_topk: keep mask of the k largest scores among the candidate positions of each
// sequence; exact ties go to the lower position.  One CTA per sequence.
#pragma once
#include "common.cuh"
#include "ptx.cuh"

namespace pdd {

// score of position j: per-head pooled column sums added over the heads in index order
__device__ __forceinline__ float pooled_head_sum(const float* __restrict__ colsum, int64_t ld,
                                                 int hq, int64_t n, int pool_kind, int pool_k,
                                                 int64_t j) {
  const int half = pool_k / 2;
  const int64_t lo = max((int64_t)0, j - half), hi = min(n - 1, j + half);
  float total = 0.f;
  for (int h = 0; h < hq; ++h) {
    const float* cs = colsum + (size_t)h * ld;
    float r;
    if (pool_kind == 2) {
      r = -INFINITY;
      for (int64_t t = lo; t <= hi; ++t) r = fmaxf(r, cs[t]);
    } else if (pool_kind == 1) {
      r = 0.f;
      for (int64_t t = lo; t <= hi; ++t) r += cs[t];
      r /= (float)pool_k;                       // zero padding, fixed divisor
    } else {
      r = cs[j];
    }
    total += r;
  }
  return total;
}

// Several sequences in one launch: blockIdx.y = sequence of the batch.
constexpr int kImportanceBatch = 64;
struct ImportanceBatch {
  const float* colsum[kImportanceBatch];   // [hq][ld] of the sequence
  float* score[kImportanceBatch];
  int64_t n[kImportanceBatch];
};
__global__ void __launch_bounds__(256)
importance_reduce_batched_kernel(const ImportanceBatch b, int64_t ld, int hq, int pool_kind,
                                 int pool_k, int accumulate) {
  ptx::griddep_launch_dependents();
  ptx::griddep_wait();
  const int s = blockIdx.y;
  const int64_t n = b.n[s];
  const int64_t j = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (j >= n) return;
  const float total = pooled_head_sum(b.colsum[s], ld, hq, n, pool_kind, pool_k, j);
  float* score = b.score[s];
  score[j] = accumulate ? score[j] + total : total;
}

__global__ void __launch_bounds__(256)
importance_reduce_kernel(const float* __restrict__ colsum, int64_t ld, int hq, int64_t n,
                         int pool_kind, int pool_k, float* __restrict__ score, int accumulate) {
  // (may be launched with programmatic serialization: nothing is read or written before the
  // kernels ahead in the stream have finished; without that attribute the wait returns at once)
  ptx::griddep_launch_dependents();
  ptx::griddep_wait();
  const int64_t j = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (j >= n) return;
  const int half = pool_k / 2;
  const int64_t lo = max((int64_t)0, j - half), hi = min(n - 1, j + half);
  float total = 0.f;
  for (int h = 0; h < hq; ++h) {
    const float* cs = colsum + (size_t)h * ld;
    float r;
    if (pool_kind == 2) {
      r = -INFINITY;
      for (int64_t t = lo; t <= hi; ++t) r = fmaxf(r, cs[t]);
    } else if (pool_kind == 1) {
      r = 0.f;
      for (int64_t t = lo; t <= hi; ++t) r += cs[t];
      r /= (float)pool_k;                       // zero padding, fixed divisor
    } else {
      r = cs[j];
    }
    total += r;
  }
  score[j] = accumulate ? score[j] + total : total;
}

struct TopkSeq {
  int64_t offset;     // first position of the sequence in score/keep
  int64_t kinds_offset;  // first position of the sequence in kinds (several rows may share one)
  int64_t n;
  int64_t cand_lo, cand_hi;
};

constexpr int kTopkThreads = 1024;
constexpr int kRadixBits = 11;                // digits of the radix select
constexpr int kRadixBins = 1 << kRadixBits;   // = 2 * kTopkThreads: two bins per thread in the scan
constexpr int kScorePasses = 3;   // radix passes over a 32-bit key
constexpr int kTopkBatch = 64;      // sequences per launch (descriptors travel as parameters)
struct TopkBatch {
  TopkSeq s[kTopkBatch];
};

// fp32 bit pattern -> uint32 whose unsigned order equals the float order.
__device__ __forceinline__ uint32_t order_key(float x) {
  uint32_t b = __float_as_uint(x);
  return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}

// Where the selection keys come from.  ScoreKeys: fp32 scores, 32-bit keys, 3 radix passes of
// 11 bits.  VoteKeys: ready-made 40-bit keys (votes in bits 32-39 above the order key of the
// summed value), 4 passes.
struct ScoreKeys {
  using key_t = uint32_t;
  static constexpr int kPasses = kScorePasses;
  const float* score;
  __device__ __forceinline__ key_t load(int64_t i) const { return order_key(score[i]); }
};
struct VoteKeys {
  using key_t = unsigned long long;
  static constexpr int kPasses = 4;
  const unsigned long long* key;
  __device__ __forceinline__ key_t load(int64_t i) const { return key[i]; }
};

__device__ __forceinline__ int block_sum(int v, int* warp_buf) {
  for (int off = 16; off; off >>= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
  __syncthreads();
  if ((threadIdx.x & 31) == 0) warp_buf[threadIdx.x >> 5] = v;
  __syncthreads();
  int t = 0;
  for (int w = 0; w < kTopkThreads / 32; ++w) t += warp_buf[w];
  return t;
}

// After a counting pass: finds the bin that holds the need-th largest matching key, appends its
// digit to the prefix and reduces the need by the keys in higher bins.  Thread i looks at bins
// B-1-2i and B-2-2i, so an inclusive scan of the pair sums over threads is the count of keys in
// those bins and all higher ones.  Called by all kTopkThreads threads, after a __syncthreads()
// that follows the last update of hist; leaves *s_prefix and *s_need updated but NOT yet
// synchronised.
template <class key_t>
__device__ __forceinline__ void radix_pick_bin(const int* hist, int* warp_buf, key_t* s_prefix,
                                               int* s_need, key_t prefix, int shift) {
  const int tid = threadIdx.x;
  const int need = *s_need;
  __syncthreads();                         // everyone has read s_need before it changes
  const int bin_a = kRadixBins - 1 - 2 * tid, bin_b = bin_a - 1;
  const int va = hist[bin_a], vb = hist[bin_b];
  int incl = va + vb;
  for (int off = 1; off < 32; off <<= 1) {
    const int up = __shfl_up_sync(0xffffffffu, incl, off);
    if ((tid & 31) >= off) incl += up;
  }
  if ((tid & 31) == 31) warp_buf[tid >> 5] = incl;
  __syncthreads();
  for (int w = 0; w < (tid >> 5); ++w) incl += warp_buf[w];
  const int excl = incl - (va + vb);
  // exactly one bin satisfies this (the total count of matching keys is >= need)
  if (excl < need && excl + va >= need) {
    *s_prefix = prefix | ((key_t)bin_a << shift);
    *s_need = need - excl;
  } else if (excl + va < need && incl >= need) {
    *s_prefix = prefix | ((key_t)bin_b << shift);
    *s_need = need - (excl + va);
  }
}

// Selection of one sequence by the whole CTA (kTopkThreads threads), keys and kinds read from
// global memory in every pass: the body of radix_topk_kernel (sequences too long to stage, and
// the 40-bit vote keys).
template <class Keys>
__device__ __forceinline__ void radix_topk_body(const Keys& keys, const uint8_t* __restrict__ kinds,
                                                const TopkSeq& sq, double keep_ratio,
                                                uint8_t* __restrict__ keep,
                                                int32_t* __restrict__ n_kept_out) {
  using key_t = typename Keys::key_t;
  __shared__ int hist[kRadixBins];
  __shared__ int warp_buf[kTopkThreads / 32];
  __shared__ key_t s_prefix;
  __shared__ int s_need;
  const uint8_t* kd = kinds ? kinds + sq.kinds_offset : nullptr;
  uint8_t* kp = keep + sq.offset;
  const int tid = threadIdx.x;

  // Counts: prompt positions, always-kept (prompt outside the candidate range), candidates.
  int c_prompt = 0, c_cand = 0;
  for (int64_t i = tid; i < sq.n; i += kTopkThreads) {
    const bool prompt = !kd || kd[i] == 0;
    const bool cand = prompt && i >= sq.cand_lo && i < sq.cand_hi;
    c_prompt += prompt;
    c_cand += cand;
  }
  const int n_prompt = block_sum(c_prompt, warp_buf);
  const int n_cand = block_sum(c_cand, warp_buf);
  const int n_always = n_prompt - n_cand;
  // k_total = floor(r*l + 1/2) with separately rounded multiply and add
  const long long k_total = (long long)floor(__dadd_rn(__dmul_rn(keep_ratio, (double)n_prompt), 0.5));
  long long kk = k_total - n_always;
  kk = kk < 0 ? 0 : (kk > n_cand ? n_cand : kk);
  const int k = (int)kk;

  // Radix select, 11 bits per pass from the top (three passes for 32-bit keys): after the
  // passes s_prefix is the key of the k-th largest candidate and s_need the number of
  // positions to take at that key.
  if (tid == 0) { s_prefix = 0; s_need = k; }
  __syncthreads();
  if (k > 0) {
    for (int pass = 0; pass < Keys::kPasses; ++pass) {
      const int shift = kRadixBits * (Keys::kPasses - 1 - pass);
      const key_t mask_hi = pass == 0 ? (key_t)0 : (key_t)(~(key_t)0 << (shift + kRadixBits));
      for (int b = tid; b < kRadixBins; b += kTopkThreads) hist[b] = 0;
      __syncthreads();
      const key_t prefix = s_prefix;
      for (int64_t i = tid; i < sq.n; i += kTopkThreads) {
        const bool cand = (!kd || kd[i] == 0) && i >= sq.cand_lo && i < sq.cand_hi;
        if (!cand) continue;
        const key_t key = keys.load(sq.offset + i);
        if ((key & mask_hi) == prefix)
          atomicAdd(&hist[(int)((key >> shift) & (key_t)(kRadixBins - 1))], 1);
      }
      __syncthreads();
      radix_pick_bin(hist, warp_buf, &s_prefix, &s_need, prefix, shift);
      __syncthreads();
    }
  }
  const key_t theta = s_prefix;
  const int need_eq = s_need;

  // Mask: greater than the threshold -> keep; equal -> the first need_eq by position.
  __shared__ int s_run;
  if (tid == 0) s_run = 0;
  __syncthreads();
  for (int64_t base = 0; base < sq.n; base += kTopkThreads) {
    const int64_t i = base + tid;
    bool prompt = false, cand = false, eq = false, gt = false;
    if (i < sq.n) {
      prompt = !kd || kd[i] == 0;
      cand = prompt && i >= sq.cand_lo && i < sq.cand_hi;
      if (cand && k > 0) {
        const key_t key = keys.load(sq.offset + i);
        gt = key > theta;
        eq = key == theta;
      }
    }
    // rank of this thread among the block's "equal" flags, in position order
    const unsigned bal = __ballot_sync(0xffffffffu, eq);
    const int lane = tid & 31, warp = tid >> 5;
    if (lane == 0) warp_buf[warp] = __popc(bal);
    __syncthreads();
    int before = s_run;
    for (int w = 0; w < warp; ++w) before += warp_buf[w];
    before += __popc(bal & ((1u << lane) - 1u));
    if (i < sq.n) {
      uint8_t kv = 0;
      if (prompt && !cand) kv = 1;
      else if (gt) kv = 1;
      else if (eq && before < need_eq) kv = 1;
      kp[i] = kv;
    }
    __syncthreads();
    if (tid == 0) {
      int t = 0;
      for (int w = 0; w < kTopkThreads / 32; ++w) t += warp_buf[w];
      s_run += t;
    }
    __syncthreads();
  }
  if (tid == 0) *n_kept_out = k + n_always;
}

template <class Keys>
__global__ void __launch_bounds__(kTopkThreads)
radix_topk_kernel(const Keys keys, const uint8_t* __restrict__ kinds,
                  const TopkBatch seqs, double keep_ratio,
                  uint8_t* __restrict__ keep, int32_t* __restrict__ n_kept) {
  ptx::griddep_launch_dependents();
  ptx::griddep_wait();          // see importance_reduce_kernel
  radix_topk_body(keys, kinds, seqs.s[blockIdx.x], keep_ratio, keep, n_kept + blockIdx.x);
}

// Selection with everything staged in shared memory: the CTA reads its sequence's scores and
// kinds from global memory ONCE (keys as order-preserving 32-bit words, one bit per position
// for "prompt" and for "candidate"), counting the first radix digit on the way; the remaining
// radix passes and the mask pass touch shared memory only.  The mask pass gives every warp a
// contiguous stretch of positions, so the ordered count of ties needs two block-wide barriers
// instead of two per 1024 positions.  At most kStagedTopkMax positions per sequence.
constexpr int64_t kStagedTopkMax = 49152;
__host__ __device__ constexpr size_t staged_topk_smem_bytes(int64_t n) {
  return (size_t)(((n + 31) & ~(int64_t)31) + 2 * ((n + 31) >> 5)) * 4;
}
__global__ void __launch_bounds__(kTopkThreads)
radix_topk_staged_kernel(const float* __restrict__ score, const uint8_t* __restrict__ kinds,
                         const TopkBatch seqs, double keep_ratio, uint8_t* __restrict__ keep,
                         int32_t* __restrict__ n_kept) {
  extern __shared__ __align__(16) uint32_t s_dyn[];
  __shared__ int hist[kRadixBins];
  __shared__ int warp_buf[kTopkThreads / 32];
  __shared__ uint32_t s_prefix;
  __shared__ int s_need;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const TopkSeq sq = seqs.s[blockIdx.x];
  const int n = (int)sq.n;
  const int n_words = (n + 31) >> 5;
  uint32_t* const s_key = s_dyn;
  uint32_t* const s_cand = s_dyn + ((n + 31) & ~31);
  uint32_t* const s_prompt = s_cand + n_words;
  for (int b = tid; b < kRadixBins; b += kTopkThreads) hist[b] = 0;
  ptx::griddep_launch_dependents();
  ptx::griddep_wait();          // see importance_reduce_kernel
  __syncthreads();

  // Stage: keys, flag bits, counts and the histogram of the first digit.  The loads of the
  // next 1024 positions are in flight while these are handled.
  const float* sc = score + sq.offset;
  const uint8_t* kd = kinds ? kinds + sq.kinds_offset : nullptr;
  constexpr int kShift0 = kRadixBits * (kScorePasses - 1);
  int c_prompt = 0, c_cand = 0;
  constexpr int kU = 8;               // positions per thread whose loads are in flight together
  for (int base = 0; base < n; base += kU * kTopkThreads) {
    float x[kU];
    uint8_t kind[kU];
#pragma unroll
    for (int u = 0; u < kU; ++u) {
      const int i = base + u * kTopkThreads + tid;
      x[u] = i < n ? sc[i] : 0.f;
      kind[u] = (kd && i < n) ? kd[i] : (uint8_t)0;
    }
#pragma unroll
    for (int u = 0; u < kU; ++u) {
      const int i = base + u * kTopkThreads + tid;
      if (base + u * kTopkThreads >= n) break;          // uniform over the block
      const bool prompt = i < n && kind[u] == 0;
      const bool cand = prompt && i >= sq.cand_lo && i < sq.cand_hi;
      const uint32_t key = order_key(x[u]);
      if (i < n) s_key[i] = key;
      const unsigned bp = __ballot_sync(0xffffffffu, prompt);
      const unsigned bc = __ballot_sync(0xffffffffu, cand);
      // (finding the lanes that share a bin first, by match.any or by a ballot against the first
      // lane's bin, was measured: slower and no faster than the plain shared-memory atomics)
      if (cand) atomicAdd(&hist[key >> kShift0], 1);
      if (lane == 0 && i < n) {
        s_prompt[i >> 5] = bp;
        s_cand[i >> 5] = bc;
        c_prompt += __popc(bp);
        c_cand += __popc(bc);
      }
    }
  }
  const int n_prompt = block_sum(c_prompt, warp_buf);
  const int n_cand = block_sum(c_cand, warp_buf);
  const int n_always = n_prompt - n_cand;
  // k_total = floor(r*l + 1/2) with separately rounded multiply and add
  const long long k_total = (long long)floor(__dadd_rn(__dmul_rn(keep_ratio, (double)n_prompt), 0.5));
  long long kk = k_total - n_always;
  kk = kk < 0 ? 0 : (kk > n_cand ? n_cand : kk);
  const int k = (int)kk;

  if (tid == 0) { s_prefix = 0; s_need = k; }
  __syncthreads();
  if (k > 0) {
    radix_pick_bin(hist, warp_buf, &s_prefix, &s_need, 0u, kShift0);
    __syncthreads();
    for (int pass = 1; pass < kScorePasses; ++pass) {
      const int shift = kRadixBits * (kScorePasses - 1 - pass);
      const uint32_t mask_hi = ~0u << (shift + kRadixBits);
      for (int b = tid; b < kRadixBins; b += kTopkThreads) hist[b] = 0;
      __syncthreads();
      const uint32_t prefix = s_prefix;
      for (int base = 0; base < n; base += kTopkThreads) {
        const int i = base + tid;
        const uint32_t key = i < n ? s_key[i] : 0u;
        const bool hit = i < n && ((s_cand[i >> 5] >> lane) & 1u) && (key & mask_hi) == prefix;
        if (hit) atomicAdd(&hist[(key >> shift) & (uint32_t)(kRadixBins - 1)], 1);
      }
      __syncthreads();
      radix_pick_bin(hist, warp_buf, &s_prefix, &s_need, prefix, shift);
      __syncthreads();
    }
  }
  const uint32_t theta = s_prefix;
  const int need_eq = s_need;

  // Mask: greater than the threshold -> keep; equal -> the first need_eq by position.  Warp w
  // owns words [w0, w1) of 32 positions: it counts its ties, learns how many lie before its
  // stretch, and then numbers its own in order.
  const int wpw = (n_words + kTopkThreads / 32 - 1) / (kTopkThreads / 32);
  const int w0 = min(n_words, warp * wpw), w1 = min(n_words, w0 + wpw);
  auto tie = [&](int w) -> bool {
    const int i = w * 32 + lane;
    return k > 0 && i < n && ((s_cand[w] >> lane) & 1u) && s_key[i] == theta;
  };
  int ties = 0;
  for (int w = w0; w < w1; ++w) ties += __popc(__ballot_sync(0xffffffffu, tie(w)));
  if (lane == 0) warp_buf[warp] = ties;
  __syncthreads();
  int run = lane < warp ? warp_buf[lane] : 0;
  for (int off = 16; off; off >>= 1) run += __shfl_xor_sync(0xffffffffu, run, off);
  uint8_t* kp = keep + sq.offset;
  for (int w = w0; w < w1; ++w) {
    const int i = w * 32 + lane;
    const bool prompt = (s_prompt[w] >> lane) & 1u, cand = (s_cand[w] >> lane) & 1u;
    const bool eq = tie(w);
    const bool gt = k > 0 && cand && i < n && s_key[i] > theta;
    const unsigned bal = __ballot_sync(0xffffffffu, eq);
    const int before = run + __popc(bal & ((1u << lane) - 1u));
    if (i < n) kp[i] = (uint8_t)((prompt && !cand) || gt || (eq && before < need_eq));
    run += __popc(bal);
  }
  if (tid == 0) n_kept[blockIdx.x] = k + n_always;
}

}  // namespace pdd
