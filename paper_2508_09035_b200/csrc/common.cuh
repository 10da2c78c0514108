// Shared device/host declarations of libpdd's kernels.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace pdd {

constexpr int kTileRows = 128;   // query rows per attention tile
constexpr int kKeyBlock = 128;   // keys per K/V block
constexpr int kMaxSeqsPerCall = 1024;
constexpr int kMaxAttnCtas = 160;      // attention CTAs per launch (one per SM)
constexpr int kMinUnitsPerCta = 4;     // a CTA's share is at least this many key blocks

// One sequence's share of a call.  Lives in the call record (device memory).
struct SeqDesc {
  int64_t pos0;        // cache position of the call's first row
  int64_t tok_offset;  // first packed row of the call that belongs to this sequence
  int32_t len;         // rows
  int32_t seq_id;
  int32_t tile0;       // first 128-row tile index of this sequence within the call
  int32_t page_off;    // first entry of this sequence in the record's page list
  int32_t n_pages;     // pages covering [pos0, pos0+len)
  int32_t window;      // rows join the observation window
  int32_t pair0;       // first tile-pair index of this sequence (pipelined attention kernel)
  int32_t pad;
};

// Header of a call record; followed by SeqDesc[n_seqs], then int32 page ids.
struct CallHeader {
  int32_t n_seqs;
  int32_t n_tiles;     // sum over sequences of ceil(len/128)
  int32_t n_rows;      // sum of len
  int32_t n_page_ids;
  int32_t kind;        // 0 prompt, 1 received
  int32_t desc_off;    // byte offset of SeqDesc array from the record start
  int32_t pages_off;   // byte offset of the page id list
  int32_t n_pairs;     // tile pairs (work items of the attention kernel)
  // Attention schedule: every CTA gets an equal share of the call's (pair, key block) units.
  int32_t n_ctas;      // CTAs of the attention launch
  int32_t cta_off;     // byte offset of CtaStart[n_ctas + 1]
  int32_t n_split;     // pairs whose key range is shared by several CTAs
  int32_t split_off;   // byte offset of SplitPair[n_split]
  // > 1: the launch uses thread-block clusters of this many CTAs, one cluster per pair, and
  // the CtaStart / SplitPair tables are not used (n_ctas = n_pairs * cluster).
  int32_t cluster;
  int32_t rec_bytes;   // size of the whole record (header, descriptors, page ids, schedule)
  // 1: the launch is the pair-of-CTAs kernel (clusters of two; the CtaStart table then counts
  // quads, i.e. pairs 2i and 2i+1, and has n_ctas / 2 + 1 entries)
  int32_t pair_of_ctas;
  int32_t pad;
};

// First unit of a CTA's share: key block `kb` of pair `pair`; entry n_ctas is the end.
struct CtaStart {
  int32_t pair;
  int32_t kb;
};

// A pair processed by CTAs cta_first .. cta_first+n_seg-1; each leaves a partial result in
// its scratch slot (slot_first for the first CTA, slot 0 for the others).
struct SplitPair {
  int32_t pair;
  int32_t cta_first;
  int32_t n_seg;
  int32_t slot_first;
};

// A call record small enough travels to kv_append and to the attention kernel as a kernel
// parameter (no copy engine between two calls' kernels, and the attention kernel can decode
// its work before the kernel ahead of it has finished); kv_append also stores it in the
// record's device slot for the kernels that read it from memory.
constexpr int kRecParamBytes = 4096;
struct RecParam {
  uint4 w[kRecParamBytes / 16];
};

// Geometry of the cache; passed by value to kernels.
struct CacheGeom {
  __nv_bfloat16* kpool;     // [n_pages][hkv][page_tokens][d]
  __nv_bfloat16* vpool;
  int32_t* page_table;      // [max_seqs][pages_per_seq]
  uint8_t* kinds;           // [max_seqs][max_tokens_per_seq]
  float* colsum;            // [max_seqs][hq][max_tokens_per_seq]
  float* lse;               // [hq][lse_ld]   natural-log LSE of the current call's rows
  int32_t* dev_status;      // sticky error word
  // Partial results of key-range shares: slot = cta*2 + {0,1};
  //   part_o  [slot][tile 2][d/4][128 rows][4] fp32, unnormalised, relative to its own max
  //   part_ml [slot][tile 2][128 rows] (running max of raw logits, row sum)
  float* part_o;
  float2* part_ml;
  int64_t max_tokens_per_seq;
  int64_t lse_ld;
  int32_t pages_per_seq;
  int32_t page_tokens;
  int32_t hq, hkv, d;
  float scale;              // softmax scale
  // Query at position p sees keys p-window+1 .. p (clipped at 0).  Plain causal attention is
  // stored as a window no sequence can reach, so the kernels have a single code path.
  int32_t window;
};
constexpr int32_t kNoWindow = 0x3fffffff;

// First key block a 128-row tile whose first row sits at position p_first can see.
__host__ __device__ __forceinline__ int first_key_block(int64_t p_first, int32_t window) {
  const int64_t lo = p_first - window + 1;
  return lo > 0 ? (int)(lo / kKeyBlock) : 0;
}

__device__ __forceinline__ const SeqDesc* record_descs(const void* rec) {
  const CallHeader* h = reinterpret_cast<const CallHeader*>(rec);
  return reinterpret_cast<const SeqDesc*>(reinterpret_cast<const char*>(rec) + h->desc_off);
}
__device__ __forceinline__ const int32_t* record_pages(const void* rec) {
  const CallHeader* h = reinterpret_cast<const CallHeader*>(rec);
  return reinterpret_cast<const int32_t*>(reinterpret_cast<const char*>(rec) + h->pages_off);
}

// Element offset of (position, kv head) row in a pool, through the page table.
__device__ __forceinline__ size_t kv_row_offset(const CacheGeom& g, int seq_id, int64_t pos,
                                                int kvh) {
  int32_t page = g.page_table[(size_t)seq_id * g.pages_per_seq + (int32_t)(pos / g.page_tokens)];
  return (((size_t)page * g.hkv + kvh) * g.page_tokens + (size_t)(pos % g.page_tokens)) * g.d;
}

}  // namespace pdd
