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
  const int vec_per_head = g.d / 8;
  for (int64_t i = tid; i < n_vec; i += stride) {
    int64_t row = i / vec_per_row;
    int rem = (int)(i - row * vec_per_row);
    int kvh = rem / vec_per_head;
    int c = rem - kvh * vec_per_head;
    // sequence of this packed row (few sequences per call: linear scan)
    int s = 0;
    while (s + 1 < n_seqs && descs[s + 1].tok_offset <= row) ++s;
    const SeqDesc& sd = descs[s];
    int64_t pos = sd.pos0 + (row - sd.tok_offset);
    int e = (int)(pos / g.page_tokens) - (int)(sd.pos0 / g.page_tokens);
    int32_t page = pages[sd.page_off + e];
    size_t dst = ((((size_t)page * g.hkv + kvh) * g.page_tokens + (size_t)(pos % g.page_tokens)) *
                  g.d) / 8 + c;
    reinterpret_cast<uint4*>(g.kpool)[dst] = k4[i];
    reinterpret_cast<uint4*>(g.vpool)[dst] = v4[i];
    if (rem == 0) g.kinds[(size_t)sd.seq_id * g.max_tokens_per_seq + pos] = (uint8_t)hdr->kind;
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
