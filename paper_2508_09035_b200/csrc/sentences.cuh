// Sentence-level selection and the mask bit stream.
//
// refine_sentences_kernel: one CTA.  The sentence boundaries live in device memory, so the
// host cannot check them: the kernel clamps every boundary to [0, n] and verifies that they
// do not decrease; on a violation it keeps nothing, reports n_kept = -1 and returns (no index
// derived from a bad boundary is ever used).  Sentence value = mean score of the sentence's prompt
// tokens (added one by one in position order in fp32, then one division, so that the
// decision can be repeated exactly on the host); sentences are sorted by decreasing value
// (ties: lower sentence first) with a bitonic sort in shared memory, then taken first-fit
// against the token budget.  Latency-bound: a few thousand sentences at most.
// pack_mask_kernel: keep[i] -> bit (i mod 8) of byte i/8.
#pragma once
#include "common.cuh"
#include "refine.cuh"

namespace pdd {

constexpr int kMaxSentences = 8192;
constexpr int kSentenceThreads = 1024;

// dynamic shared memory: uint64 key[n_pad] | int32 count[n_pad] | uint8 take[n_pad]
inline size_t sentence_smem_bytes(int n_pad) { return (size_t)n_pad * (8 + 4 + 1) + 64; }

__global__ void __launch_bounds__(kSentenceThreads)
refine_sentences_kernel(const float* __restrict__ score, const uint8_t* __restrict__ kinds,
                        int64_t n, const int32_t* __restrict__ seg_start, int n_seg, int n_pad,
                        double keep_ratio, uint8_t* __restrict__ keep,
                        int32_t* __restrict__ n_kept, float* __restrict__ seg_value) {
  extern __shared__ __align__(16) uint8_t smem[];
  unsigned long long* key = reinterpret_cast<unsigned long long*>(smem);
  int32_t* count = reinterpret_cast<int32_t*>(smem + (size_t)n_pad * 8);
  uint8_t* take = smem + (size_t)n_pad * 12;
  __shared__ int warp_buf[kSentenceThreads / 32];
  __shared__ int s_used;
  __shared__ int s_bad;
  const int tid = threadIdx.x;
  // boundary s, clamped to [0, n]
  auto bound = [&](int s) -> int64_t {
    const int64_t b = seg_start[s];
    return b < 0 ? 0 : (b > n ? n : b);
  };
  if (tid == 0) s_bad = 0;
  __syncthreads();
  for (int s = tid; s <= n_seg; s += kSentenceThreads) {
    const int64_t b = seg_start[s];
    if (b < 0 || b > n || (s > 0 && b < (int64_t)seg_start[s - 1])) s_bad = 1;
  }
  __syncthreads();
  if (s_bad) {
    for (int64_t i = tid; i < n; i += kSentenceThreads) keep[i] = 0;
    if (tid == 0) *n_kept = -1;
    return;
  }
  const int64_t lo = bound(0), hi = bound(n_seg);

  // prompt positions overall and inside the content range
  int c_prompt = 0, c_content = 0;
  for (int64_t i = tid; i < n; i += kSentenceThreads) {
    const bool prompt = !kinds || kinds[i] == 0;
    c_prompt += prompt;
    c_content += prompt && i >= lo && i < hi;
  }
  const int n_prompt = block_sum(c_prompt, warp_buf);
  const int n_content = block_sum(c_content, warp_buf);
  const int n_always = n_prompt - n_content;
  const long long k_total =
      (long long)floor(__dadd_rn(__dmul_rn(keep_ratio, (double)n_prompt), 0.5));
  long long bb = k_total - n_always;
  bb = bb < 0 ? 0 : (bb > n_content ? n_content : bb);
  const int budget = (int)bb;

  // sentence values and sort keys
  for (int s = tid; s < n_pad; s += kSentenceThreads) {
    unsigned long long kk = 0ull;
    int c = 0;
    if (s < n_seg) {
      float acc = 0.f;
      for (int64_t i = bound(s); i < bound(s + 1); ++i) {
        if (!kinds || kinds[i] == 0) {
          acc = __fadd_rn(acc, score[i]);
          ++c;
        }
      }
      const float v = c > 0 ? __fdiv_rn(acc, (float)c) : -INFINITY;
      if (seg_value) seg_value[s] = v;
      if (c > 0)
        kk = ((unsigned long long)order_key(v) << 32) | (unsigned long long)(0xFFFFFFFFu - (uint32_t)s);
    }
    key[s] = kk;          // sentences without prompt tokens and padding sort last
    count[s] = c;
    take[s] = 0;
  }
  __syncthreads();

  // bitonic sort, descending
  for (int size = 2; size <= n_pad; size <<= 1) {
    for (int stride = size >> 1; stride > 0; stride >>= 1) {
      for (int i = tid; i < n_pad; i += kSentenceThreads) {
        const int j = i ^ stride;
        if (j > i) {
          const bool desc = (i & size) == 0;
          const unsigned long long a = key[i], b = key[j];
          if ((a < b) == desc) {
            key[i] = b;
            key[j] = a;
          }
        }
      }
      __syncthreads();
    }
  }

  // first fit against the budget, in sorted order
  if (tid == 0) {
    int rem = budget;
    for (int i = 0; i < n_seg && rem > 0; ++i) {
      const unsigned long long kk = key[i];
      if (kk == 0ull) break;                       // only empty sentences follow
      const int s = (int)(0xFFFFFFFFu - (uint32_t)(kk & 0xFFFFFFFFull));
      const int c = count[s];
      if (c <= rem) {
        take[s] = 1;
        rem -= c;
      }
    }
    s_used = budget - rem;
  }
  __syncthreads();

  // mask: prefix and suffix prompt tokens, then the tokens of the taken sentences
  for (int64_t i = tid; i < n; i += kSentenceThreads) {
    if (i < lo || i >= hi) keep[i] = (!kinds || kinds[i] == 0) ? 1 : 0;
  }
  for (int s = tid; s < n_seg; s += kSentenceThreads) {
    const uint8_t t = take[s];
    for (int64_t i = bound(s); i < bound(s + 1); ++i)
      keep[i] = (t && (!kinds || kinds[i] == 0)) ? 1 : 0;
  }
  if (tid == 0) *n_kept = n_always + s_used;
}

__global__ void __launch_bounds__(256)
pack_mask_kernel(const uint8_t* __restrict__ keep, int64_t n, uint8_t* __restrict__ bits) {
  const int64_t b = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  const int64_t n_bytes = (n + 7) / 8;
  if (b >= n_bytes) return;
  uint32_t v = 0;
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    const int64_t i = b * 8 + j;
    if (i < n && keep[i]) v |= 1u << j;
  }
  bits[b] = (uint8_t)v;
}

}  // namespace pdd
