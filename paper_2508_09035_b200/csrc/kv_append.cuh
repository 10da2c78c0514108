// kv_append: copy a call's K/V rows into the paged cache, publish the pages the call
// uses in the page table and tag the new positions with their kind.
// HBM-bound: every thread moves 16 bytes of K and 16 bytes of V.
#pragma once
#include "common.cuh"
#include "ptx.cuh"

namespace pdd {

__global__ void __launch_bounds__(256)
kv_append_kernel(CacheGeom g, void* __restrict__ rec_dev, const __grid_constant__ RecParam recp,
                 int rec_in_param, const __nv_bfloat16* __restrict__ k,
                 const __nv_bfloat16* __restrict__ v) {
  // Launched with programmatic serialization: everything this kernel writes (cache rows, page
  // table, kinds, the record's device slot) may still be read by the kernels ahead of it.
  ptx::griddep_wait();
  // Only now may the attention kernel start: whatever it reads before its own wait (the
  // caller's q, cache rows of earlier calls) is then known to be complete.
  ptx::griddep_launch_dependents();
  // a launch that follows a timed-out wait does no work (as in every kernel of the handle)
  if (*reinterpret_cast<volatile int32_t*>(g.dev_status) != 0) return;
  const void* rec = rec_in_param ? reinterpret_cast<const void*>(&recp) : rec_dev;
  if (rec_in_param && blockIdx.x == 0) {
    const int n16 = (reinterpret_cast<const CallHeader*>(rec)->rec_bytes + 15) / 16;
    for (int i = threadIdx.x; i < n16; i += blockDim.x)
      reinterpret_cast<uint4*>(rec_dev)[i] = recp.w[i];
  }
  const CallHeader* hdr = reinterpret_cast<const CallHeader*>(rec);
  const SeqDesc* descs = record_descs(rec);
  const int32_t* pages = record_pages(rec);
  const int n_seqs = hdr->n_seqs;
  const int vec_per_row = g.hkv * g.d / 8;            // 16-byte vectors per token row
  const int64_t n_vec = (int64_t)hdr->n_rows * vec_per_row;
  const int64_t tid = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;

  // Publish page ids: entry e of sequence s is the page of slot pos0/page_tokens + e.
  for (int64_t i = tid; i < hdr->n_page_ids; i += stride) {
    int s = 0;
    while (s + 1 < n_seqs && descs[s + 1].page_off <= i) ++s;
    const SeqDesc& sd = descs[s];
    int slot = (int)(sd.pos0 / g.page_tokens) + (int)(i - sd.page_off);
    g.page_table[(size_t)sd.seq_id * g.pages_per_seq + slot] = pages[i];
  }

  const uint4* k4 = reinterpret_cast<const uint4*>(k);
  const uint4* v4 = reinterpret_cast<const uint4*>(v);
  const uint32_t vec_per_head = (uint32_t)g.d / 8;
  const uint32_t vpr = (uint32_t)vec_per_row;
  const uint32_t page_tokens = (uint32_t)g.page_tokens;
  // destination of vector i (32-bit index arithmetic: a call carries far fewer than 2^31
  // vectors); the sequence of a packed row is found by a scan that starts at the sequence of
  // the thread's previous vector (rows only grow along a thread's stride)
  int s_hint = 0;
  auto dest = [&](uint32_t i, bool& first_of_row, size_t& kind_at) -> size_t {
    const uint32_t row = i / vpr, rem = i - row * vpr;
    const uint32_t kvh = rem / vec_per_head, c = rem - kvh * vec_per_head;
    while (s_hint + 1 < n_seqs && descs[s_hint + 1].tok_offset <= (int64_t)row) ++s_hint;
    const SeqDesc& sd = descs[s_hint];
    const uint32_t pos = (uint32_t)sd.pos0 + (row - (uint32_t)sd.tok_offset);
    const uint32_t e = pos / page_tokens - (uint32_t)sd.pos0 / page_tokens;
    const int32_t page = pages[sd.page_off + e];
    first_of_row = rem == 0;
    kind_at = (size_t)sd.seq_id * g.max_tokens_per_seq + pos;
    return ((((size_t)page * g.hkv + kvh) * page_tokens + pos % page_tokens) * g.d) / 8 + c;
  };
  // four vectors of K and of V in flight per thread before the first store
  constexpr int kUnroll = 4;
  const uint32_t n = (uint32_t)n_vec, t0 = (uint32_t)tid, step = (uint32_t)stride;
  for (uint32_t base = t0; base < n; base += kUnroll * step) {
    uint4 kk[kUnroll], vv[kUnroll];
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
      const uint32_t i = base + u * step;
      if (i < n) {
        kk[u] = k4[i];
        vv[u] = v4[i];
      }
    }
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
      const uint32_t i = base + u * step;
      if (i < n) {
        bool first;
        size_t kind_at;
        const size_t dst = dest(i, first, kind_at);
        reinterpret_cast<uint4*>(g.kpool)[dst] = kk[u];
        reinterpret_cast<uint4*>(g.vpool)[dst] = vv[u];
        if (first) g.kinds[kind_at] = (uint8_t)hdr->kind;
      }
    }
  }
}

// Gather a sequence's cached K and V back to token-major layout (diagnostics).
__global__ void kv_export_kernel(CacheGeom g, int seq_id, int64_t n_tokens,
                                 __nv_bfloat16* __restrict__ k_dst,
                                 __nv_bfloat16* __restrict__ v_dst) {
  const int vec_per_row = g.hkv * g.d / 8;
  const int vec_per_head = g.d / 8;
  const int64_t n_vec = n_tokens * vec_per_row;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n_vec;
       i += (int64_t)gridDim.x * blockDim.x) {
    int64_t pos = i / vec_per_row;
    int rem = (int)(i - pos * vec_per_row);
    int kvh = rem / vec_per_head;
    int c = rem - kvh * vec_per_head;
    size_t src = kv_row_offset(g, seq_id, pos, kvh) / 8 + c;
    reinterpret_cast<uint4*>(k_dst)[i] = reinterpret_cast<const uint4*>(g.kpool)[src];
    reinterpret_cast<uint4*>(v_dst)[i] = reinterpret_cast<const uint4*>(g.vpool)[src];
  }
}

}  // namespace pdd
