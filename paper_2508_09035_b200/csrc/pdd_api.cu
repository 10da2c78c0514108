// libpdd: C ABI and host runtime (page pool, page tables, call records, launches).
// See include/pdd.h for the contract of every entry point.
#include <cuda.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <map>
#include <mutex>
#include <string>
#include <vector>

#include "../../include/pdd.h"
#include "attn_simt.cuh"
#include "attn_tc.cuh"
#include "attn_tc2.cuh"
#include "attn_tc_v0.cuh"
#include "colsum_tc.cuh"
#include "common.cuh"
#include "kv_append.cuh"
#include "refine.cuh"
#include "sentences.cuh"
#include "vote.cuh"

using namespace pdd;

namespace {

thread_local char g_detail[512] = "";

int fail(int code, const char* fmt, ...) {
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(g_detail, sizeof(g_detail), fmt, ap);
  va_end(ap);
  return code;
}

#define PDD_CUDA(expr)                                                                    \
  do {                                                                                    \
    cudaError_t e_ = (expr);                                                              \
    if (e_ != cudaSuccess)                                                                \
      return fail(PDD_ERR_CUDA, "%s failed: %s", #expr, cudaGetErrorString(e_));          \
  } while (0)

size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

using EncodeTiledFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*,
                                   const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                                   const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                   CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) ==
            cudaSuccess && qres == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

// bf16 tensor map with 128-byte swizzle; dims/strides innermost first, strides in bytes
// for dims 1..rank-1.
int make_tmap(CUtensorMap* m, const void* base, int rank, const uint64_t* dims,
              const uint64_t* strides_bytes, const uint32_t* box) {
  EncodeTiledFn fn = get_encode_fn();
  if (!fn) return fail(PDD_ERR_CUDA, "cuTensorMapEncodeTiled entry point not available");
  cuuint64_t gd[5];
  cuuint64_t gs[4];
  cuuint32_t bx[5], es[5];
  for (int i = 0; i < rank; ++i) {
    gd[i] = dims[i];
    bx[i] = box[i];
    es[i] = 1;
    if (i > 0) gs[i - 1] = strides_bytes[i - 1];
  }
  CUresult r = fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, (cuuint32_t)rank, const_cast<void*>(base),
                  gd, gs, bx, es, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                  CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return fail(PDD_ERR_CUDA, "cuTensorMapEncodeTiled failed (%d)", (int)r);
  return PDD_OK;
}

constexpr int kRingSlots = 32;

struct TraceEntry {
  const char* name;
  cudaEvent_t a, b;
};

}  // namespace

struct QMapEntry {
  const void* ptr = nullptr;
  int rows = 0;
  CUtensorMap map;
};

struct pdd_kv {
  pdd_kv_config cfg;
  CacheGeom g;
  uint8_t* arena;
  size_t arena_bytes;
  int64_t n_pages;
  std::vector<int32_t> free_pages;              // stack of free page ids
  std::vector<std::vector<int32_t>> seq_pages;  // per sequence, in slot order
  std::vector<int64_t> seq_len;
  // call records: pinned host ring mirrored into the arena
  uint8_t* ring_host;
  uint8_t* ring_dev;
  size_t rec_bytes;
  cudaEvent_t ring_ev[kRingSlots];
  bool ring_used[kRingSlots];
  int ring_next;
  CUtensorMap tmK, tmV;
  int kernel_path;
  int schedule;                       // 0 cost model, 1 whole pairs, 2 equal shares, 3 clusters, 4 CTA pairs
  int max_clusters[kMaxCluster + 1];  // clusters of c CTAs the device runs at once
  int max_clusters2 = 0;              // CTA pairs of the pair-of-CTAs kernel the device runs at once
  int sm_count;
  bool trace;
  std::vector<TraceEntry> trace_log;
  int64_t last_rows;
  QMapEntry tmq_cache[16];
  int tmq_next = 0;
  std::vector<int32_t> sched_nb;      // per-call scratch of the attention schedule
  std::vector<int64_t> sched_first;
  RecParam rec_param;                 // by-value copy of a small call record
  int fail_countdown = 0;             // > 0: the n-th launch from now reports a failure (test hook)
};

namespace {

// Test hook: true if this launch is the one that has been told to fail.
bool injected_failure(pdd_kv* kv) {
  if (kv->fail_countdown <= 0) return false;
  return --kv->fail_countdown == 0;
}

// Waits on a barrier nobody arrives at; when the limit runs out it raises the sticky status
// word like any hot kernel does and returns through the normal exit.
__global__ void __launch_bounds__(32)
wait_timeout_probe_kernel(int32_t* dev_status, unsigned long long limit_ns) {
  __shared__ uint64_t bar;
  if (threadIdx.x == 0) {
    ptx::mbar_init(&bar, 1);
    ptx::fence_mbar_init();
  }
  __syncwarp();
  if (threadIdx.x == 0) {
    const bool got = ptx::mbar_wait_for(&bar, 0, limit_ns, 0xf);
    if (!got) atomicExch(dev_status, PDD_ERR_TIMEOUT);
  }
}

struct Carve {
  size_t kpool, vpool, page_table, kinds, colsum, lse, status, part_o, part_ml, ring, total;
  int64_t n_pages;
  int32_t pages_per_seq;
  size_t rec_bytes;
};

int validate_cfg(const pdd_kv_config* c) {
  if (!c) return fail(PDD_ERR_INVALID, "config is null");
  if (c->n_q_heads <= 0 || c->n_kv_heads <= 0 || c->n_q_heads % c->n_kv_heads != 0)
    return fail(PDD_ERR_INVALID, "n_q_heads must be a positive multiple of n_kv_heads");
  if (c->head_dim != 64 && c->head_dim != 128)
    return fail(PDD_ERR_UNSUPPORTED, "head_dim %d: only 64 and 128 are supported", c->head_dim);
  if (c->page_tokens != 64 && c->page_tokens != 128)
    return fail(PDD_ERR_UNSUPPORTED, "page_tokens %d: only 64 and 128", c->page_tokens);
  if (c->max_seqs <= 0 || c->max_seqs > kMaxSeqsPerCall)
    return fail(PDD_ERR_INVALID, "max_seqs must be in 1..%d", kMaxSeqsPerCall);
  if (c->max_tokens_total <= 0 || c->max_tokens_per_seq <= 0 || c->max_rows_per_call <= 0)
    return fail(PDD_ERR_INVALID, "token capacities must be positive");
  if (c->max_tokens_per_seq > (1 << 24))
    return fail(PDD_ERR_UNSUPPORTED, "max_tokens_per_seq above 2^24");
  if (c->max_rows_per_call > (1 << 22))
    return fail(PDD_ERR_UNSUPPORTED, "max_rows_per_call above 2^22");
  if (c->sliding_window < 0 || c->reserved_f != 0.f || c->softmax_scale < 0.f)
    return fail(PDD_ERR_INVALID, "sliding_window >= 0, reserved_f must be 0, softmax_scale >= 0");
  return PDD_OK;
}

void carve(const pdd_kv_config& c, Carve* out) {
  const size_t A = 1024;
  Carve k{};
  // every sequence may leave its last page partly filled
  k.n_pages = (c.max_tokens_total + c.page_tokens - 1) / c.page_tokens + c.max_seqs;
  k.pages_per_seq = (int32_t)((c.max_tokens_per_seq + c.page_tokens - 1) / c.page_tokens);
  const size_t pool = (size_t)k.n_pages * c.n_kv_heads * c.page_tokens * c.head_dim * 2;
  // record: header + descs + page ids
  // ... + the attention schedule (CTA starts, shared pairs)
  k.rec_bytes = align_up(sizeof(CallHeader) + sizeof(SeqDesc) * (size_t)c.max_seqs +
                             4 * ((size_t)c.max_rows_per_call / c.page_tokens + 2 * (size_t)c.max_seqs + 2) +
                             16 + sizeof(CtaStart) * (kMaxAttnCtas + 1) + sizeof(SplitPair) * kMaxAttnCtas,
                         256);
  size_t off = 0;
  k.kpool = off; off = align_up(off + pool, A);
  k.vpool = off; off = align_up(off + pool, A);
  k.page_table = off; off = align_up(off + 4 * (size_t)c.max_seqs * k.pages_per_seq, A);
  k.kinds = off; off = align_up(off + (size_t)c.max_seqs * c.max_tokens_per_seq, A);
  k.colsum = off; off = align_up(off + 4 * (size_t)c.max_seqs * c.n_q_heads * c.max_tokens_per_seq, A);
  k.lse = off; off = align_up(off + 4 * (size_t)c.n_q_heads * (c.max_rows_per_call + kTileRows), A);
  k.status = off; off = align_up(off + 256, A);
  k.part_o = off; off = align_up(off + 4 * part_o_floats(c.head_dim) * 2 * kMaxAttnCtas, A);
  k.part_ml = off; off = align_up(off + 8 * part_ml_elems() * 2 * kMaxAttnCtas, A);
  k.ring = off; off = align_up(off + k.rec_bytes * kRingSlots, A);
  k.total = off;
  *out = k;
}

struct Tracer {
  pdd_kv* kv;
  cudaStream_t st;
  TraceEntry e{};
  bool on;
  Tracer(pdd_kv* k, cudaStream_t s, const char* name) : kv(k), st(s), on(k && k->trace) {
    if (on) {
      e.name = name;
      cudaEventCreate(&e.a);
      cudaEventCreate(&e.b);
      cudaEventRecord(e.a, st);
    }
  }
  ~Tracer() {
    if (on) {
      cudaEventRecord(e.b, st);
      kv->trace_log.push_back(e);
    }
  }
};

// Tensor map of a call's q buffer viewed as (d, heads, rows); callers tend to reuse the
// same buffers, so the last few maps are kept.
int q_tensor_map(pdd_kv* kv, const void* q, int n_rows, const CUtensorMap** out) {
  for (auto& e : kv->tmq_cache)
    if (e.ptr == q && e.rows == n_rows) {
      *out = &e.map;
      return PDD_OK;
    }
  const CacheGeom& g = kv->g;
  QMapEntry& e = kv->tmq_cache[kv->tmq_next];
  kv->tmq_next = (kv->tmq_next + 1) % (int)(sizeof(kv->tmq_cache) / sizeof(kv->tmq_cache[0]));
  const uint64_t dims[3] = {(uint64_t)g.d, (uint64_t)g.hq, (uint64_t)n_rows};
  const uint64_t strides[2] = {(uint64_t)g.d * 2, (uint64_t)g.hq * g.d * 2};
  const uint32_t box[3] = {64, 1, (uint32_t)kTileRows};
  e.ptr = nullptr;
  int rc = make_tmap(&e.map, q, 3, dims, strides, box);
  if (rc) return rc;
  e.ptr = q;
  e.rows = n_rows;
  *out = &e.map;
  return PDD_OK;
}

int launch_attention(pdd_kv* kv, const void* rec_dev, const RecParam& recp, int rec_in_param,
                     const CallHeader& hdr, const void* q, void* out, cudaStream_t st) {
  const CacheGeom& g = kv->g;
  const int D = g.d;
  if (kv->kernel_path == 1) {
    Tracer t(kv, st, "attn_simt");
    dim3 grid((hdr.n_rows + 3) / 4, g.hq);
    if (D == 128)
      attn_simt_kernel<128><<<grid, 128, 0, st>>>(g, rec_dev, (const __nv_bfloat16*)q,
                                                  (__nv_bfloat16*)out);
    else
      attn_simt_kernel<64><<<grid, 128, 0, st>>>(g, rec_dev, (const __nv_bfloat16*)q,
                                                 (__nv_bfloat16*)out);
    PDD_CUDA(cudaGetLastError());
    return PDD_OK;
  }
  // tensor-core paths: Q viewed as (d, heads, rows)
  const CUtensorMap* tmq_ptr = nullptr;
  int rc = q_tensor_map(kv, q, hdr.n_rows, &tmq_ptr);
  if (rc) return rc;
  const CUtensorMap& tmQ = *tmq_ptr;
  if (kv->kernel_path == 2) {
    Tracer t(kv, st, "attn_tc_v0");
    dim3 grid(hdr.n_tiles, g.hq);
    if (D == 128) {
      attn_tc_v0_kernel<128><<<grid, 128, AttnV0Smem<128>::kBytes, st>>>(
          g, rec_dev, tmQ, kv->tmK, kv->tmV, (__nv_bfloat16*)out, nullptr);
    } else {
      attn_tc_v0_kernel<64><<<grid, 128, AttnV0Smem<64>::kBytes, st>>>(
          g, rec_dev, tmQ, kv->tmK, kv->tmV, (__nv_bfloat16*)out, nullptr);
    }
    PDD_CUDA(cudaGetLastError());
    return PDD_OK;
  }
  cudaError_t e;
  {
    Tracer t(kv, st, "fwd_attn");
    e = hdr.pair_of_ctas ? launch_attn_tc2(g, rec_dev, recp, rec_in_param, hdr, tmQ, kv->tmK,
                                           kv->tmV, (__nv_bfloat16*)out, st)
                         : launch_attn_tc(g, rec_dev, recp, rec_in_param, hdr, tmQ, kv->tmK, kv->tmV,
                                          (__nv_bfloat16*)out, st);
  }
  if (e == cudaSuccess && hdr.n_split > 0) {
    Tracer t(kv, st, "attn_combine");
    e = launch_attn_combine(g, rec_dev, hdr, (__nv_bfloat16*)out, st);
  }
  return e == cudaSuccess ? PDD_OK
                          : fail(PDD_ERR_CUDA, "fwd_attn launch failed: %s", cudaGetErrorString(e));
}

int launch_colsum(pdd_kv* kv, const void* rec_dev, const CallHeader& hdr,
                  const std::vector<SeqDesc>& descs, const void* q, cudaStream_t st) {
  const CacheGeom& g = kv->g;
  if (kv->kernel_path != 0) {
    Tracer t(kv, st, "colsum_simt");
    for (int s = 0; s < hdr.n_seqs; ++s) {
      if (!descs[s].window || descs[s].len == 0) continue;
      const int64_t T = descs[s].pos0 + descs[s].len;
      dim3 grid((unsigned)((T + 127) / 128), g.hq);
      if (g.d == 128)
        colsum_simt_kernel<128><<<grid, 128, 0, st>>>(g, rec_dev, s, (const __nv_bfloat16*)q);
      else
        colsum_simt_kernel<64><<<grid, 128, 0, st>>>(g, rec_dev, s, (const __nv_bfloat16*)q);
    }
    PDD_CUDA(cudaGetLastError());
    return PDD_OK;
  }
  const CUtensorMap* tmq_ptr = nullptr;
  int rc = q_tensor_map(kv, q, hdr.n_rows, &tmq_ptr);
  if (rc) return rc;
  const CUtensorMap& tmQ = *tmq_ptr;
  Tracer t(kv, st, "colsum");
  int n_kb_total = 0;
  for (int s = 0; s < hdr.n_seqs; ++s)
    if (descs[s].window && descs[s].len > 0)
      n_kb_total += (int)((descs[s].pos0 + descs[s].len + kKeyBlock - 1) / kKeyBlock);
  if (launch_colsum_tc(g, rec_dev, n_kb_total, tmQ, kv->tmK, kv->sm_count, st) != cudaSuccess)
    return fail(PDD_ERR_CUDA, "colsum launch failed: %s", cudaGetErrorString(cudaGetLastError()));
  return PDD_OK;
}

int run_call(pdd_kv* kv, const pdd_batch* b, const void* q, const void* k, const void* v,
             void* out, uint32_t flags, int kind, void* stream) {
  if (!kv || !b) return fail(PDD_ERR_INVALID, "null handle or batch");
  if (b->n_seqs <= 0 || b->n_seqs > kv->cfg.max_seqs)
    return fail(PDD_ERR_INVALID, "n_seqs %d outside 1..%d", b->n_seqs, kv->cfg.max_seqs);
  if (!b->seq_id || !b->pos0 || !b->len || !b->tok_offset)
    return fail(PDD_ERR_INVALID, "batch arrays must not be null");
  if (flags & ~(uint32_t)PDD_WINDOW) return fail(PDD_ERR_INVALID, "unknown flag bits");
  const pdd_kv_config& c = kv->cfg;
  cudaStream_t st = (cudaStream_t)stream;

  // ---- validation (nothing is enqueued or changed before it passes) ----
  std::vector<char> seen(c.max_seqs, 0);
  int64_t rows = 0, pages_needed = 0;
  for (int i = 0; i < b->n_seqs; ++i) {
    const int32_t s = b->seq_id[i];
    if (s < 0 || s >= c.max_seqs) return fail(PDD_ERR_INVALID, "seq_id %d out of range", s);
    if (seen[s]) return fail(PDD_ERR_INVALID, "seq_id %d appears twice in one call", s);
    seen[s] = 1;
    if (b->len[i] < 0) return fail(PDD_ERR_INVALID, "negative len");
    if (b->tok_offset[i] != rows || b->tok_offset[i + 1] - b->tok_offset[i] != b->len[i])
      return fail(PDD_ERR_INVALID, "tok_offset does not match len at sequence %d", i);
    if (b->pos0[i] != kv->seq_len[s])
      return fail(PDD_ERR_STATE, "sequence %d: pos0 %lld but current length is %lld", s,
                  (long long)b->pos0[i], (long long)kv->seq_len[s]);
    const int64_t new_len = kv->seq_len[s] + b->len[i];
    if (new_len > c.max_tokens_per_seq)
      return fail(PDD_ERR_CAPACITY, "sequence %d would reach %lld tokens (max %lld)", s,
                  (long long)new_len, (long long)c.max_tokens_per_seq);
    const int64_t have = (int64_t)kv->seq_pages[s].size();
    const int64_t need = (new_len + c.page_tokens - 1) / c.page_tokens;
    pages_needed += std::max<int64_t>(0, need - have);
    rows += b->len[i];
  }
  if (rows > c.max_rows_per_call)
    return fail(PDD_ERR_CAPACITY, "%lld rows in one call (max %lld)", (long long)rows,
                (long long)c.max_rows_per_call);
  if (pages_needed > (int64_t)kv->free_pages.size())
    return fail(PDD_ERR_CAPACITY, "page pool exhausted: need %lld pages, %zu free",
                (long long)pages_needed, kv->free_pages.size());
  if (rows == 0) return PDD_OK;
  if (!q || !k || !v || !out) return fail(PDD_ERR_INVALID, "q/k/v/out must not be null");
  if (((uintptr_t)q | (uintptr_t)k | (uintptr_t)v | (uintptr_t)out) & 15)
    return fail(PDD_ERR_INVALID, "q/k/v/out must be 16-byte aligned");

  // ---- record ----
  // Built in a pinned ring slot (its copy engine transfer reads it after this call returns).
  // A record of at most kRecParamBytes is afterwards passed to the kernels by value instead,
  // and no copy is enqueued; which of the two it will be is known only once it is built.
  const int slot = kv->ring_next;
  if (kv->ring_used[slot]) {
    PDD_CUDA(cudaEventSynchronize(kv->ring_ev[slot]));
    kv->ring_used[slot] = false;
  }
  uint8_t* rec_h = kv->ring_host + (size_t)slot * kv->rec_bytes;
  uint8_t* rec_d = kv->ring_dev + (size_t)slot * kv->rec_bytes;
  CallHeader hdr{};
  hdr.n_seqs = b->n_seqs;
  hdr.kind = kind;
  hdr.desc_off = (int32_t)sizeof(CallHeader);
  hdr.pages_off = (int32_t)(sizeof(CallHeader) + sizeof(SeqDesc) * (size_t)b->n_seqs);
  std::vector<SeqDesc> descs(b->n_seqs);
  int32_t* page_ids = reinterpret_cast<int32_t*>(rec_h + hdr.pages_off);
  // The host state (lengths, page lists, free pages, ring position) moves forward while the
  // record is built; if anything fails before the call's last launch has been accepted it is
  // put back, so that a failed call leaves the handle as it found it.
  struct Undo { int32_t seq; int64_t len; size_t n_pages; };
  std::vector<Undo> undo;
  undo.reserve(b->n_seqs);
  const int ring_next_before = kv->ring_next;
  const int64_t last_rows_before = kv->last_rows;
  auto roll_back = [&](int rc) {
    for (auto it = undo.rbegin(); it != undo.rend(); ++it) {
      auto& pages = kv->seq_pages[it->seq];
      while (pages.size() > it->n_pages) {
        kv->free_pages.push_back(pages.back());
        pages.pop_back();
      }
      kv->seq_len[it->seq] = it->len;
    }
    kv->ring_next = ring_next_before;
    kv->last_rows = last_rows_before;
    return rc;
  };
  int tile0 = 0, page_off = 0, pair0 = 0;
  const int G = c.n_q_heads / c.n_kv_heads;
  for (int i = 0; i < b->n_seqs; ++i) {
    const int32_t s = b->seq_id[i];
    SeqDesc& d = descs[i];
    d.pos0 = b->pos0[i];
    d.tok_offset = b->tok_offset[i];
    d.len = b->len[i];
    d.seq_id = s;
    d.tile0 = tile0;
    d.pair0 = pair0;
    d.pad = 0;
    d.page_off = page_off;
    d.window = (flags & PDD_WINDOW) ? 1 : 0;
    d.n_pages = 0;
    if (d.len > 0) {
      const int64_t new_len = d.pos0 + d.len;
      const int64_t need = (new_len + c.page_tokens - 1) / c.page_tokens;
      undo.push_back(Undo{s, kv->seq_len[s], kv->seq_pages[s].size()});
      while ((int64_t)kv->seq_pages[s].size() < need) {
        kv->seq_pages[s].push_back(kv->free_pages.back());
        kv->free_pages.pop_back();
      }
      const int first = (int)(d.pos0 / c.page_tokens);
      d.n_pages = (int)need - first;
      for (int e = 0; e < d.n_pages; ++e) page_ids[page_off + e] = kv->seq_pages[s][first + e];
      page_off += d.n_pages;
      const int ntile = (d.len + kTileRows - 1) / kTileRows;
      tile0 += ntile;
      pair0 += (G % 2 == 0) ? ntile * (c.n_q_heads / 2) : ((ntile + 1) / 2) * c.n_q_heads;
      kv->seq_len[s] = new_len;
    }
  }
  hdr.n_tiles = tile0;
  hdr.n_rows = (int32_t)rows;
  hdr.n_page_ids = page_off;
  hdr.n_pairs = pair0;
  // Attention schedule: key blocks per pair, then equal shares of the total per CTA.
  size_t used = align_up(hdr.pages_off + 4 * (size_t)page_off, 16);
  {
    std::vector<int32_t>& nb = kv->sched_nb;
    nb.assign(pair0, 0);
    for (const SeqDesc& d : descs) {
      if (d.len <= 0) continue;
      const int ntile = (d.len + kTileRows - 1) / kTileRows;
      const int32_t win = c.sliding_window > 0 ? c.sliding_window : kNoWindow;
      // key blocks of a pair whose first tile is rb_first and last tile rb_last: from the
      // first block the first tile's first row can see to the block of the last valid row
      auto pair_blocks = [&](int rb_first, int rb_last) {
        const int64_t p_last0 = d.pos0 + (int64_t)rb_last * kTileRows;
        const int rv = std::min(kTileRows, d.len - rb_last * kTileRows);
        const int end = (int)((p_last0 + rv - 1) / kKeyBlock + 1);
        return (int32_t)(end - first_key_block(d.pos0 + (int64_t)rb_first * kTileRows, win));
      };
      if (G % 2 == 0) {
        for (int rb = 0; rb < ntile; ++rb)
          for (int hp = 0; hp < c.n_q_heads / 2; ++hp)
            nb[d.pair0 + rb * (c.n_q_heads / 2) + hp] = pair_blocks(rb, rb);
      } else {
        for (int rbp = 0; rbp < (ntile + 1) / 2; ++rbp)
          for (int h = 0; h < c.n_q_heads; ++h)
            nb[d.pair0 + rbp * c.n_q_heads + h] =
                pair_blocks(2 * rbp, std::min(2 * rbp + 1, ntile - 1));
      }
    }
    int64_t total_units = 0;
    for (int32_t x : nb) total_units += x;
    const int max_ctas = std::min(kv->sm_count, kMaxAttnCtas);
    // Three ways to cut the work: (A) whole pairs per CTA, no partial results; (B) exactly
    // equal shares, which leaves up to two partial results per CTA for the merge kernel;
    // (C) a cluster of c CTAs per pair, each taking 1/c of the pair's key blocks and merging
    // through distributed shared memory (only when all clusters run at once).
    // A rough cost model in microseconds, fitted to per-call timings on B200 (whole pairs:
    // 10 + 1.95 per key block of the largest share; equal shares: 28 with the merge + 1.9;
    // clusters: 16.5 with the merge + 2.05 per key block of the largest part)
    const int n_b =
        (int)std::max<int64_t>(1, std::min<int64_t>(max_ctas, total_units / kMinUnitsPerCta));
    const int n_a = std::min(max_ctas, pair0);
    std::vector<int64_t>& first_unit = kv->sched_first;     // unit at which each CTA starts
    first_unit.assign(n_a + 1, 0);
    int64_t share_a = 0;
    {
      int pair = 0;
      int64_t prefix = 0;
      for (int i = 1; i <= n_a; ++i) {
        const int64_t target = total_units * i / n_a;
        // at least one pair per CTA, and leave one for each CTA still to come
        do prefix += nb[pair++];
        while (pair < pair0 - (n_a - i) && prefix + nb[pair] / 2 <= target);
        if (i == n_a)
          while (pair < pair0) prefix += nb[pair++];
        first_unit[i] = prefix;
        share_a = std::max(share_a, first_unit[i] - first_unit[i - 1]);
      }
    }
    double est_a = 10.0 + 1.95 * (double)share_a;
    double est_b = 28.0 + 1.9 * (double)((total_units + n_b - 1) / n_b);
    int32_t nb_max = 0;
    for (int32_t x : nb) nb_max = std::max(nb_max, x);
    int best_c = 0;
    double est_c = 1e30;
    for (int cl = 2; cl <= kMaxCluster; ++cl) {
      if (pair0 > kv->max_clusters[cl] || pair0 * cl > kMaxAttnCtas) continue;
      const double e = 16.5 + 2.05 * (double)((nb_max + cl - 1) / cl);
      if (e < est_c) {
        est_c = e;
        best_c = cl;
      }
    }
    if (kv->schedule == 1) est_b = est_c = 1e30;
    if (kv->schedule == 2) est_a = est_c = 1e30;
    if (kv->schedule == 3 && best_c > 0) est_a = est_b = 1e30;
    // Schedule 4, never picked by the model: the pair-of-CTAs kernel, where the call has the
    // shape it needs (head_dim 128, no sliding window, groups of a multiple of four query heads,
    // so that pairs 2i and 2i+1 cover the same rows of one KV head).
    const bool use2 = kv->schedule == 4 && G % 4 == 0 && c.head_dim == 128 && c.sliding_window <= 0 &&
                      kv->max_clusters2 > 0 && kv->kernel_path == 0 && pair0 % 2 == 0;
    hdr.cluster = 0;
    hdr.pair_of_ctas = 0;
    if (!use2 && best_c > 0 && est_c < est_a && est_c < est_b) {
      // the kernel derives every CTA's part from the pair itself; no tables
      hdr.cluster = best_c;
      hdr.n_ctas = pair0 * best_c;
      hdr.cta_off = hdr.split_off = (int32_t)used;
      hdr.n_split = 0;
    }
    const bool exact = est_b < est_a;
    const int n_ctas = exact ? n_b : n_a;
    if (use2) {
      // The unit is a quad (pairs 2i and 2i+1), the shares are equal over the clusters, and CTA
      // `rank` of cluster i takes pair 2 * quad + rank.  Scratch slots: CTA (rank, i) has index
      // rank * n_cl + i, so the segments of a split pair lie in consecutive indices, which is
      // what the merge kernel expects.
      const int n_quads = pair0 / 2;
      int64_t total_q = 0;
      for (int i = 0; i < n_quads; ++i) total_q += nb[2 * i];
      const int n_cl = (int)std::max<int64_t>(
          1, std::min<int64_t>(std::min(kv->max_clusters2, kMaxAttnCtas / 2), total_q / kMinUnitsPerCta));
      hdr.pair_of_ctas = 1;
      hdr.n_ctas = 2 * n_cl;
      hdr.cta_off = (int32_t)used;
      CtaStart* cs = reinterpret_cast<CtaStart*>(rec_h + used);
      first_unit.assign(n_cl + 1, 0);
      for (int i = 0; i <= n_cl; ++i) first_unit[i] = total_q * i / n_cl;
      int quad = 0;
      int64_t quad_first = 0;
      for (int i = 0; i <= n_cl; ++i) {
        const int64_t u = first_unit[i];
        while (quad < n_quads && quad_first + nb[2 * quad] <= u) quad_first += nb[2 * quad++];
        cs[i].pair = quad;
        cs[i].kb = (int32_t)(u - quad_first);
      }
      used += sizeof(CtaStart) * (size_t)(n_cl + 1);
      hdr.split_off = (int32_t)used;
      SplitPair* sp = reinterpret_cast<SplitPair*>(rec_h + used);
      int n_split = 0;
      for (int i = 1; i < n_cl; ++i) {
        if (cs[i].kb == 0) continue;
        if (n_split > 0 && sp[n_split - 1].pair == 2 * cs[i].pair + 1) {
          ++sp[n_split - 2].n_seg;
          ++sp[n_split - 1].n_seg;
          continue;
        }
        const int64_t quad_start = first_unit[i] - cs[i].kb;
        for (int rk = 0; rk < 2; ++rk) {
          sp[n_split].pair = 2 * cs[i].pair + rk;
          sp[n_split].cta_first = rk * n_cl + i - 1;
          sp[n_split].n_seg = 2;
          sp[n_split].slot_first = first_unit[i - 1] < quad_start ? 1 : 0;
          ++n_split;
        }
      }
      hdr.n_split = n_split;
      used += sizeof(SplitPair) * (size_t)n_split;
    } else if (hdr.cluster == 0) {
      hdr.n_ctas = n_ctas;
      hdr.cta_off = (int32_t)used;
      CtaStart* cs = reinterpret_cast<CtaStart*>(rec_h + used);
      if (exact) {
        first_unit.assign(n_ctas + 1, 0);
        for (int i = 0; i <= n_ctas; ++i) first_unit[i] = total_units * i / n_ctas;
      }
      int pair = 0;
      int64_t pair_first = 0;                                 // first unit of `pair`
      for (int i = 0; i <= n_ctas; ++i) {
        const int64_t u = first_unit[i];
        while (pair < pair0 && pair_first + nb[pair] <= u) pair_first += nb[pair++];
        cs[i].pair = pair;
        cs[i].kb = (int32_t)(u - pair_first);
      }
      used += sizeof(CtaStart) * (size_t)(n_ctas + 1);
      hdr.split_off = (int32_t)used;
      SplitPair* sp = reinterpret_cast<SplitPair*>(rec_h + used);
      int n_split = 0;
      // every interior boundary that falls inside a pair marks a shared pair
      for (int i = 1; i < n_ctas; ++i) {
        if (cs[i].kb == 0) continue;
        if (n_split > 0 && sp[n_split - 1].pair == cs[i].pair) {
          ++sp[n_split - 1].n_seg;
          continue;
        }
        const int64_t pair_start = first_unit[i] - cs[i].kb;
        // CTA i-1 holds the pair's first key blocks; it may have started before the pair
        sp[n_split].pair = cs[i].pair;
        sp[n_split].cta_first = i - 1;
        sp[n_split].n_seg = 2;
        sp[n_split].slot_first = first_unit[i - 1] < pair_start ? 1 : 0;
        ++n_split;
      }
      hdr.n_split = n_split;
      used += sizeof(SplitPair) * (size_t)n_split;
    }
  }
  hdr.rec_bytes = (int32_t)used;
  memcpy(rec_h, &hdr, sizeof(hdr));
  memcpy(rec_h + hdr.desc_off, descs.data(), sizeof(SeqDesc) * descs.size());
  const int rec_in_param = used <= (size_t)kRecParamBytes ? 1 : 0;
  RecParam& recp = kv->rec_param;
  if (rec_in_param) {
    memcpy(&recp, rec_h, used);
  } else {
    cudaError_t ce = injected_failure(kv) ? cudaErrorUnknown
                                          : cudaMemcpyAsync(rec_d, rec_h, used, cudaMemcpyHostToDevice, st);
    if (ce == cudaSuccess) ce = cudaEventRecord(kv->ring_ev[slot], st);
    if (ce != cudaSuccess)
      return roll_back(fail(PDD_ERR_CUDA, "copy of the call record failed: %s", cudaGetErrorString(ce)));
    kv->ring_used[slot] = true;
  }
  // The device slots rotate in both cases: the slot's last readers are kernels of the call
  // kRingSlots calls back on this stream, and kv_append writes it only after the kernels
  // ahead of it have finished.
  kv->ring_next = (slot + 1) % kRingSlots;
  kv->last_rows = rows;

  // ---- launches ----
  {
    Tracer t(kv, st, "kv_append");
    const int64_t n_vec = rows * c.n_kv_heads * c.head_dim / 8;
    const int blocks = (int)std::min<int64_t>((n_vec / 4 + 255) / 256, (int64_t)kv->sm_count * 8);
    if (injected_failure(kv) ||
        launch_pdl(kv_append_kernel, dim3(std::max(blocks, 1)), dim3(256), 0, st, kv->g,
                   (void*)rec_d, recp, rec_in_param, (const __nv_bfloat16*)k,
                   (const __nv_bfloat16*)v) != cudaSuccess)
      return roll_back(fail(PDD_ERR_CUDA, "kv_append launch failed: %s",
                            cudaGetErrorString(cudaGetLastError())));
  }
  int rc = injected_failure(kv) ? fail(PDD_ERR_CUDA, "fwd_attn launch failed: injected")
                                : launch_attention(kv, rec_d, recp, rec_in_param, hdr, q, out, st);
  if (rc) return roll_back(rc);
  if (flags & PDD_WINDOW) {
    rc = injected_failure(kv) ? fail(PDD_ERR_CUDA, "colsum launch failed: injected")
                              : launch_colsum(kv, rec_d, hdr, descs, q, st);
    if (rc) return roll_back(rc);
  }
  return PDD_OK;
}

// Score vector of pdd_refine_from_colsum_static.  It lives in the library image, so every
// GPU that loads libpdd holds these 256 KiB until the process exits, and no call ever
// allocates it.  In host code this name is only a handle for the runtime: the device
// address has to be asked for with cudaGetSymbolAddress, once per device.
static __device__ __align__(256) float g_static_score[PDD_STATIC_SCORE_MAX];

constexpr int kMaxDevices = 64;
std::mutex g_static_mutex;
float* g_static_score_ptr[kMaxDevices] = {};

// Device address of g_static_score on the current device (looked up on first use).
int static_score_buffer(float** out) {
  int dev = -1;
  PDD_CUDA(cudaGetDevice(&dev));
  if (dev < 0 || dev >= kMaxDevices)
    return fail(PDD_ERR_UNSUPPORTED, "device ordinal %d outside 0..%d", dev, kMaxDevices - 1);
  std::lock_guard<std::mutex> lock(g_static_mutex);
  if (!g_static_score_ptr[dev]) {
    float* p = nullptr;
    cudaError_t e = cudaGetSymbolAddress((void**)&p, g_static_score);
    if (e != cudaSuccess || !p)
      return fail(PDD_ERR_CUDA, "cudaGetSymbolAddress(g_static_score) failed on device %d: %s", dev,
                  cudaGetErrorString(e));
    g_static_score_ptr[dev] = p;
  }
  *out = g_static_score_ptr[dev];
  return PDD_OK;
}

}  // namespace

extern "C" {

int pdd_kv_bytes_required(const pdd_kv_config* cfg, size_t* bytes) {
  int rc = validate_cfg(cfg);
  if (rc) return rc;
  if (!bytes) return fail(PDD_ERR_INVALID, "bytes is null");
  Carve k;
  carve(*cfg, &k);
  *bytes = k.total;
  return PDD_OK;
}

int pdd_kv_alloc(const pdd_kv_config* cfg, void* dev_buf, size_t bytes, void* stream,
                 pdd_kv** out) {
  int rc = validate_cfg(cfg);
  if (rc) return rc;
  if (!dev_buf || !out) return fail(PDD_ERR_INVALID, "dev_buf/out is null");
  if ((uintptr_t)dev_buf & 255) return fail(PDD_ERR_INVALID, "dev_buf must be 256-byte aligned");
  Carve k;
  carve(*cfg, &k);
  if (bytes < k.total)
    return fail(PDD_ERR_CAPACITY, "arena of %zu bytes, %zu required", bytes, k.total);
  int dev = 0;
  PDD_CUDA(cudaGetDevice(&dev));
  cudaDeviceProp prop;
  PDD_CUDA(cudaGetDeviceProperties(&prop, dev));
  if (prop.major != 10)
    return fail(PDD_ERR_UNSUPPORTED, "device is sm_%d%d; this library is built for sm_100a only",
                prop.major, prop.minor);
  cudaStream_t st = (cudaStream_t)stream;
  pdd_kv* kv = new pdd_kv();
  kv->cfg = *cfg;
  if (kv->cfg.softmax_scale == 0.f) kv->cfg.softmax_scale = 1.f / sqrtf((float)cfg->head_dim);
  uint8_t* a = reinterpret_cast<uint8_t*>(dev_buf);
  kv->arena = a;
  kv->arena_bytes = bytes;
  kv->n_pages = k.n_pages;
  CacheGeom& g = kv->g;
  g.kpool = reinterpret_cast<__nv_bfloat16*>(a + k.kpool);
  g.vpool = reinterpret_cast<__nv_bfloat16*>(a + k.vpool);
  g.page_table = reinterpret_cast<int32_t*>(a + k.page_table);
  g.kinds = a + k.kinds;
  g.colsum = reinterpret_cast<float*>(a + k.colsum);
  g.lse = reinterpret_cast<float*>(a + k.lse);
  g.dev_status = reinterpret_cast<int32_t*>(a + k.status);
  g.part_o = reinterpret_cast<float*>(a + k.part_o);
  g.part_ml = reinterpret_cast<float2*>(a + k.part_ml);
  g.max_tokens_per_seq = cfg->max_tokens_per_seq;
  g.lse_ld = cfg->max_rows_per_call + kTileRows;
  g.pages_per_seq = k.pages_per_seq;
  g.page_tokens = cfg->page_tokens;
  g.hq = cfg->n_q_heads;
  g.hkv = cfg->n_kv_heads;
  g.d = cfg->head_dim;
  g.scale = kv->cfg.softmax_scale;
  g.window = kv->cfg.sliding_window > 0 ? kv->cfg.sliding_window : kNoWindow;
  kv->ring_dev = a + k.ring;
  kv->rec_bytes = k.rec_bytes;
  kv->ring_next = 0;
  kv->kernel_path = 0;
  kv->schedule = 0;
  kv->sm_count = prop.multiProcessorCount;
  kv->trace = false;
  kv->last_rows = 0;
  kv->ring_host = nullptr;
  for (int i = 0; i < kRingSlots; ++i) kv->ring_used[i] = false;
  cudaError_t e = cudaHostAlloc((void**)&kv->ring_host, k.rec_bytes * kRingSlots, cudaHostAllocDefault);
  if (e != cudaSuccess) {
    delete kv;
    return fail(PDD_ERR_CUDA, "cudaHostAlloc failed: %s", cudaGetErrorString(e));
  }
  for (int i = 0; i < kRingSlots; ++i) cudaEventCreateWithFlags(&kv->ring_ev[i], cudaEventDisableTiming);
  kv->free_pages.resize(k.n_pages);
  for (int64_t i = 0; i < k.n_pages; ++i) kv->free_pages[i] = (int32_t)(k.n_pages - 1 - i);
  kv->seq_pages.assign(cfg->max_seqs, {});
  kv->seq_len.assign(cfg->max_seqs, 0);
  // K/V pools as (d, page_tokens, kv_head, page); 64 x 64 boxes
  const uint64_t dims[4] = {(uint64_t)g.d, (uint64_t)g.page_tokens, (uint64_t)g.hkv,
                            (uint64_t)k.n_pages};
  const uint64_t strides[3] = {(uint64_t)g.d * 2, (uint64_t)g.page_tokens * g.d * 2,
                               (uint64_t)g.hkv * g.page_tokens * g.d * 2};
  const uint32_t box[4] = {64, 64, 1, 1};
  rc = make_tmap(&kv->tmK, g.kpool, 4, dims, strides, box);
  if (!rc) rc = make_tmap(&kv->tmV, g.vpool, 4, dims, strides, box);
  if (!rc) {
    // kernel attributes once per handle, not per launch
    cudaError_t pe = prepare_attn_tc(g.d, g.window != kNoWindow, kv->max_clusters);
    if (pe == cudaSuccess && g.d == 128 && g.window == kNoWindow) pe = prepare_attn_tc2(&kv->max_clusters2);
    if (pe == cudaSuccess) pe = prepare_colsum_tc(g.d);
    if (pe == cudaSuccess)
      pe = g.d == 128 ? cudaFuncSetAttribute(attn_tc_v0_kernel<128>,
                                             cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             AttnV0Smem<128>::kBytes)
                      : cudaFuncSetAttribute(attn_tc_v0_kernel<64>,
                                             cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             AttnV0Smem<64>::kBytes);
    if (pe != cudaSuccess)
      rc = fail(PDD_ERR_CUDA, "kernel set-up failed: %s", cudaGetErrorString(pe));
  }
  if (rc) {
    pdd_kv_free(kv);
    return rc;
  }
  // Everything starts at zero: pools (so that never-written rows hold finite values),
  // page tables (slot -> page 0), column sums, status.
  e = cudaMemsetAsync(a, 0, k.total, st);
  if (e != cudaSuccess) {
    pdd_kv_free(kv);
    return fail(PDD_ERR_CUDA, "cudaMemsetAsync failed: %s", cudaGetErrorString(e));
  }
  *out = kv;
  return PDD_OK;
}

int pdd_kv_free(pdd_kv* kv) {
  if (!kv) return PDD_OK;
  for (auto& t : kv->trace_log) {
    cudaEventDestroy(t.a);
    cudaEventDestroy(t.b);
  }
  for (int i = 0; i < kRingSlots; ++i) cudaEventDestroy(kv->ring_ev[i]);
  if (kv->ring_host) cudaFreeHost(kv->ring_host);
  delete kv;
  return PDD_OK;
}

int pdd_kv_reset(pdd_kv* kv, int32_t seq_id, void* stream) {
  if (!kv) return fail(PDD_ERR_INVALID, "null handle");
  if (seq_id < 0 || seq_id >= kv->cfg.max_seqs) return fail(PDD_ERR_INVALID, "seq_id out of range");
  const int64_t n = kv->seq_len[seq_id];
  for (auto it = kv->seq_pages[seq_id].rbegin(); it != kv->seq_pages[seq_id].rend(); ++it)
    kv->free_pages.push_back(*it);
  kv->seq_pages[seq_id].clear();
  kv->seq_len[seq_id] = 0;
  if (n > 0) {
    const CacheGeom& g = kv->g;
    PDD_CUDA(cudaMemset2DAsync(g.colsum + (size_t)seq_id * g.hq * g.max_tokens_per_seq,
                               4 * (size_t)g.max_tokens_per_seq, 0, 4 * (size_t)n, g.hq,
                               (cudaStream_t)stream));
  }
  return PDD_OK;
}

int pdd_kv_length(const pdd_kv* kv, int32_t seq_id, int64_t* n_tokens) {
  if (!kv || !n_tokens) return fail(PDD_ERR_INVALID, "null argument");
  if (seq_id < 0 || seq_id >= kv->cfg.max_seqs) return fail(PDD_ERR_INVALID, "seq_id out of range");
  *n_tokens = kv->seq_len[seq_id];
  return PDD_OK;
}

int pdd_prefill_chunk(pdd_kv* kv, const pdd_batch* batch, const void* q, const void* k,
                      const void* v, void* out, uint32_t flags, void* stream) {
  return run_call(kv, batch, q, k, v, out, flags, 0, stream);
}

int pdd_append_received(pdd_kv* kv, const pdd_batch* batch, const void* q, const void* k,
                        const void* v, void* out, uint32_t flags, void* stream) {
  return run_call(kv, batch, q, k, v, out, flags, 1, stream);
}

int pdd_token_importance(pdd_kv* kv, int32_t seq_id, int32_t pool_kind, int32_t pool_k,
                         float* score, int32_t accumulate, void* stream) {
  if (!kv || !score) return fail(PDD_ERR_INVALID, "null argument");
  if (seq_id < 0 || seq_id >= kv->cfg.max_seqs) return fail(PDD_ERR_INVALID, "seq_id out of range");
  if (pool_kind < 0 || pool_kind > 2) return fail(PDD_ERR_INVALID, "pool_kind must be 0, 1 or 2");
  if (pool_k < 1 || pool_k % 2 == 0 || pool_k > 1025)
    return fail(PDD_ERR_INVALID, "pool_k must be odd and in 1..1025");
  const int64_t n = kv->seq_len[seq_id];
  if (n == 0) return PDD_OK;
  const CacheGeom& g = kv->g;
  cudaStream_t st = (cudaStream_t)stream;
  Tracer t(kv, st, "importance_reduce");
  PDD_CUDA(launch_pdl(importance_reduce_kernel, dim3((unsigned)((n + 255) / 256)), dim3(256), 0, st,
                      (const float*)(g.colsum + (size_t)seq_id * g.hq * g.max_tokens_per_seq),
                      (int64_t)g.max_tokens_per_seq, (int)g.hq, n, pool_k == 1 ? 0 : pool_kind,
                      pool_k, score, accumulate));
  return PDD_OK;
}

int pdd_token_importance_batched(pdd_kv* kv, int32_t n_seqs, const int32_t* seq_ids,
                                 int32_t pool_kind, int32_t pool_k, float* score,
                                 const int64_t* offsets, int32_t accumulate, void* stream) {
  if (!kv || !score || !seq_ids || !offsets) return fail(PDD_ERR_INVALID, "null argument");
  if (n_seqs <= 0) return fail(PDD_ERR_INVALID, "n_seqs must be positive");
  if (pool_kind < 0 || pool_kind > 2) return fail(PDD_ERR_INVALID, "pool_kind must be 0, 1 or 2");
  if (pool_k < 1 || pool_k % 2 == 0 || pool_k > 1025)
    return fail(PDD_ERR_INVALID, "pool_k must be odd and in 1..1025");
  for (int i = 0; i < n_seqs; ++i) {
    if (seq_ids[i] < 0 || seq_ids[i] >= kv->cfg.max_seqs)
      return fail(PDD_ERR_INVALID, "seq_id out of range");
    if (offsets[i + 1] - offsets[i] != kv->seq_len[seq_ids[i]])
      return fail(PDD_ERR_INVALID, "offsets[%d+1] - offsets[%d] differs from the sequence's length", i, i);
  }
  const CacheGeom& g = kv->g;
  cudaStream_t st = (cudaStream_t)stream;
  Tracer t(kv, st, "importance_reduce");
  for (int base = 0; base < n_seqs; base += kImportanceBatch) {
    ImportanceBatch ib{};
    const int cnt = std::min(kImportanceBatch, n_seqs - base);
    int64_t n_max = 0;
    for (int i = 0; i < cnt; ++i) {
      const int32_t s = seq_ids[base + i];
      ib.colsum[i] = g.colsum + (size_t)s * g.hq * g.max_tokens_per_seq;
      ib.score[i] = score + offsets[base + i];
      ib.n[i] = kv->seq_len[s];
      n_max = std::max(n_max, ib.n[i]);
    }
    if (n_max == 0) continue;
    PDD_CUDA(launch_pdl(importance_reduce_batched_kernel, dim3((unsigned)((n_max + 255) / 256), cnt),
                        dim3(256), 0, st, ib, (int64_t)g.max_tokens_per_seq, (int)g.hq,
                        pool_k == 1 ? 0 : pool_kind, pool_k, accumulate));
  }
  return PDD_OK;
}

int pdd_importance_topk(pdd_kv* kv, int32_t seq_id, int32_t pool_kind, int32_t pool_k,
                        float* score, int32_t accumulate, int64_t cand_lo, int64_t cand_hi,
                        double keep_ratio, uint8_t* keep, int32_t* n_kept, void* stream) {
  if (!kv || !keep || !n_kept) return fail(PDD_ERR_INVALID, "null argument");
  if (seq_id < 0 || seq_id >= kv->cfg.max_seqs) return fail(PDD_ERR_INVALID, "seq_id out of range");
  if (pool_kind < 0 || pool_kind > 2) return fail(PDD_ERR_INVALID, "pool_kind must be 0, 1 or 2");
  if (pool_k < 1 || pool_k % 2 == 0 || pool_k > 1025)
    return fail(PDD_ERR_INVALID, "pool_k must be odd and in 1..1025");
  if (!(keep_ratio >= 0.0 && keep_ratio <= 1.0))
    return fail(PDD_ERR_INVALID, "keep_ratio must be in [0,1]");
  const int64_t n = kv->seq_len[seq_id];
  if (n <= 0) return fail(PDD_ERR_STATE, "the sequence is empty");
  if (cand_lo < 0 || cand_hi > n || cand_lo > cand_hi)
    return fail(PDD_ERR_INVALID, "candidate range outside [0,n]");
  if (!score) return fail(PDD_ERR_INVALID, "score must not be null");
  const CacheGeom& g = kv->g;
  const uint8_t* kinds = g.kinds + (size_t)seq_id * g.max_tokens_per_seq;
  int rc = pdd_token_importance(kv, seq_id, pool_kind, pool_k, score, accumulate, stream);
  if (rc) return rc;
  Tracer t(kv, (cudaStream_t)stream, "radix_topk");
  return pdd_refine_topk(score, kinds, n, cand_lo, cand_hi, keep_ratio, keep, n_kept, stream);
}

int pdd_kv_kinds(pdd_kv* kv, int32_t seq_id, const uint8_t** kinds) {
  if (!kv || !kinds) return fail(PDD_ERR_INVALID, "null argument");
  if (seq_id < 0 || seq_id >= kv->cfg.max_seqs) return fail(PDD_ERR_INVALID, "seq_id out of range");
  *kinds = kv->g.kinds + (size_t)seq_id * kv->g.max_tokens_per_seq;
  return PDD_OK;
}

int pdd_refine_topk_batched(const float* score, const uint8_t* kinds, int32_t n_seqs,
                            const int64_t* offsets, const int64_t* cand_lo,
                            const int64_t* cand_hi, double keep_ratio, uint8_t* keep,
                            int32_t* n_kept, void* stream) {
  if (!score || !keep || !n_kept || !offsets || !cand_lo || !cand_hi)
    return fail(PDD_ERR_INVALID, "null argument");
  if (n_seqs <= 0) return fail(PDD_ERR_INVALID, "n_seqs must be positive");
  if (!(keep_ratio >= 0.0 && keep_ratio <= 1.0))
    return fail(PDD_ERR_INVALID, "keep_ratio must be in [0,1]");
  for (int i = 0; i < n_seqs; ++i) {
    const int64_t n = offsets[i + 1] - offsets[i];
    if (n < 0 || n > (1 << 24)) return fail(PDD_ERR_INVALID, "sequence %d: length out of range", i);
    if (cand_lo[i] < 0 || cand_hi[i] > n || cand_lo[i] > cand_hi[i])
      return fail(PDD_ERR_INVALID, "sequence %d: candidate range outside [0,n]", i);
  }
  cudaStream_t st = (cudaStream_t)stream;
  int64_t n_max = 0;
  for (int i = 0; i < n_seqs; ++i) n_max = std::max(n_max, offsets[i + 1] - offsets[i]);
  const bool staged = n_max <= kStagedTopkMax;
  if (staged) {
    static bool attr_set[kMaxDevices] = {};
    int dev = 0;
    PDD_CUDA(cudaGetDevice(&dev));
    if (dev >= 0 && dev < kMaxDevices && !attr_set[dev]) {
      PDD_CUDA(cudaFuncSetAttribute(radix_topk_staged_kernel,
                                    cudaFuncAttributeMaxDynamicSharedMemorySize,
                                    (int)staged_topk_smem_bytes(kStagedTopkMax)));
      attr_set[dev] = true;
    }
  }
  for (int base = 0; base < n_seqs; base += kTopkBatch) {
    TopkBatch tb{};
    const int cnt = std::min(kTopkBatch, n_seqs - base);
    for (int i = 0; i < cnt; ++i) {
      tb.s[i].offset = offsets[base + i];
      tb.s[i].kinds_offset = offsets[base + i];
      tb.s[i].n = offsets[base + i + 1] - offsets[base + i];
      tb.s[i].cand_lo = cand_lo[base + i];
      tb.s[i].cand_hi = cand_hi[base + i];
    }
    if (staged)
      PDD_CUDA(launch_pdl(radix_topk_staged_kernel, dim3(cnt), dim3(kTopkThreads),
                          staged_topk_smem_bytes(std::max<int64_t>(n_max, 1)), st, score, kinds, tb, keep_ratio,
                          keep, n_kept + base));
    else
      PDD_CUDA(launch_pdl(radix_topk_kernel<ScoreKeys>, dim3(cnt), dim3(kTopkThreads), 0, st,
                          ScoreKeys{score}, kinds, tb, keep_ratio, keep, n_kept + base));
  }
  return PDD_OK;
}

int pdd_refine_topk(const float* score, const uint8_t* kinds, int64_t n, int64_t cand_lo,
                    int64_t cand_hi, double keep_ratio, uint8_t* keep, int32_t* n_kept,
                    void* stream) {
  if (n <= 0) return fail(PDD_ERR_INVALID, "n must be positive");
  const int64_t offsets[2] = {0, n};
  return pdd_refine_topk_batched(score, kinds, 1, offsets, &cand_lo, &cand_hi, keep_ratio, keep,
                                 n_kept, stream);
}

int pdd_refine_sentences(const float* score, const uint8_t* kinds, int64_t n,
                         const int32_t* seg_start, int32_t n_seg, double keep_ratio,
                         uint8_t* keep, int32_t* n_kept, float* seg_value, void* stream) {
  if (!score || !seg_start || !keep || !n_kept) return fail(PDD_ERR_INVALID, "null argument");
  if (n <= 0 || n > (1 << 24)) return fail(PDD_ERR_INVALID, "n must be in 1..2^24");
  if (n_seg < 1) return fail(PDD_ERR_INVALID, "n_seg must be positive");
  if (n_seg > kMaxSentences)
    return fail(PDD_ERR_CAPACITY, "%d sentences, at most %d are supported", n_seg, kMaxSentences);
  if (!(keep_ratio >= 0.0 && keep_ratio <= 1.0))
    return fail(PDD_ERR_INVALID, "keep_ratio must be in [0,1]");
  int n_pad = 2;
  while (n_pad < n_seg) n_pad <<= 1;
  const size_t smem = sentence_smem_bytes(n_pad);
  PDD_CUDA(cudaFuncSetAttribute(refine_sentences_kernel,
                                cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  refine_sentences_kernel<<<1, kSentenceThreads, smem, (cudaStream_t)stream>>>(
      score, kinds, n, seg_start, n_seg, n_pad, keep_ratio, keep, n_kept, seg_value);
  PDD_CUDA(cudaGetLastError());
  return PDD_OK;
}

int pdd_pack_mask(const uint8_t* keep, int64_t n, uint8_t* bits, void* stream) {
  if (!keep || !bits) return fail(PDD_ERR_INVALID, "null argument");
  if (n <= 0) return fail(PDD_ERR_INVALID, "n must be positive");
  const int64_t n_bytes = (n + 7) / 8;
  pack_mask_kernel<<<(unsigned)((n_bytes + 255) / 256), 256, 0, (cudaStream_t)stream>>>(keep, n,
                                                                                       bits);
  PDD_CUDA(cudaGetLastError());
  return PDD_OK;
}

int pdd_refine_vote_workspace(int32_t n_heads, int64_t n, size_t* bytes) {
  if (!bytes) return fail(PDD_ERR_INVALID, "bytes is null");
  if (n_heads <= 0 || n_heads > 255) return fail(PDD_ERR_INVALID, "n_heads must be in 1..255");
  if (n <= 0 || n > (1 << 24)) return fail(PDD_ERR_INVALID, "n must be in 1..2^24");
  *bytes = vote_scratch(n_heads, n).total;
  return PDD_OK;
}

int pdd_refine_vote(const float* colsum, int64_t ld, int32_t n_heads, const uint8_t* kinds,
                    int64_t n, int32_t pool_kind, int32_t pool_k, int64_t cand_lo,
                    int64_t cand_hi, double keep_ratio, uint8_t* keep, int32_t* n_kept,
                    int32_t* votes, void* workspace, size_t workspace_bytes, void* stream) {
  if (!colsum || !keep || !n_kept || !workspace) return fail(PDD_ERR_INVALID, "null argument");
  if (n_heads <= 0 || n_heads > 255) return fail(PDD_ERR_INVALID, "n_heads must be in 1..255");
  if (n <= 0 || n > (1 << 24)) return fail(PDD_ERR_INVALID, "n must be in 1..2^24");
  if (ld < n) return fail(PDD_ERR_INVALID, "need ld >= n");
  if (pool_kind < 0 || pool_kind > 2) return fail(PDD_ERR_INVALID, "pool_kind must be 0, 1 or 2");
  if (pool_k < 1 || pool_k % 2 == 0 || pool_k > 1025)
    return fail(PDD_ERR_INVALID, "pool_k must be odd and in 1..1025");
  if (cand_lo < 0 || cand_hi > n || cand_lo > cand_hi)
    return fail(PDD_ERR_INVALID, "candidate range outside [0,n]");
  if (!(keep_ratio >= 0.0 && keep_ratio <= 1.0))
    return fail(PDD_ERR_INVALID, "keep_ratio must be in [0,1]");
  if ((uintptr_t)workspace & 255) return fail(PDD_ERR_INVALID, "workspace must be 256-byte aligned");
  const VoteScratch vs = vote_scratch(n_heads, n);
  if (workspace_bytes < vs.total)
    return fail(PDD_ERR_CAPACITY, "workspace of %zu bytes, %zu required", workspace_bytes, vs.total);
  uint8_t* w = reinterpret_cast<uint8_t*>(workspace);
  float* pooled = reinterpret_cast<float*>(w + vs.pooled_off);
  uint8_t* head_keep = w + vs.head_keep_off;
  unsigned long long* key = reinterpret_cast<unsigned long long*>(w + vs.key_off);
  int32_t* head_n = reinterpret_cast<int32_t*>(w + vs.head_n_off);
  cudaStream_t st = (cudaStream_t)stream;
  const unsigned blocks = (unsigned)((n + 255) / 256);
  pool_heads_kernel<<<dim3(blocks, (unsigned)n_heads), 256, 0, st>>>(
      colsum, ld, n, pool_k == 1 ? 0 : pool_kind, pool_k, pooled);
  PDD_CUDA(cudaGetLastError());
  for (int base = 0; base < n_heads; base += kTopkBatch) {
    TopkBatch tb{};
    const int cnt = std::min(kTopkBatch, n_heads - base);
    for (int i = 0; i < cnt; ++i) {
      tb.s[i].offset = (int64_t)(base + i) * n;
      tb.s[i].kinds_offset = 0;                 // every head reads the same kinds
      tb.s[i].n = n;
      tb.s[i].cand_lo = cand_lo;
      tb.s[i].cand_hi = cand_hi;
    }
    radix_topk_kernel<ScoreKeys><<<cnt, kTopkThreads, 0, st>>>(ScoreKeys{pooled}, kinds, tb,
                                                               keep_ratio, head_keep, head_n + base);
    PDD_CUDA(cudaGetLastError());
  }
  vote_key_kernel<<<blocks, 256, 0, st>>>(pooled, head_keep, kinds, n_heads, n, cand_lo, cand_hi,
                                          key, votes);
  PDD_CUDA(cudaGetLastError());
  TopkBatch tb{};
  tb.s[0].offset = 0;
  tb.s[0].kinds_offset = 0;
  tb.s[0].n = n;
  tb.s[0].cand_lo = cand_lo;
  tb.s[0].cand_hi = cand_hi;
  radix_topk_kernel<VoteKeys><<<1, kTopkThreads, 0, st>>>(VoteKeys{key}, kinds, tb, keep_ratio,
                                                          keep, n_kept);
  PDD_CUDA(cudaGetLastError());
  return PDD_OK;
}

int pdd_solve_rl(const pdd_rl_problem* problems, int32_t n, pdd_rl_solution* solutions) {
  if (!problems || !solutions) return fail(PDD_ERR_INVALID, "null argument");
  if (n < 0) return fail(PDD_ERR_INVALID, "n must not be negative");
  for (int32_t i = 0; i < n; ++i) {
    const pdd_rl_problem& p = problems[i];
    pdd_rl_solution& o = solutions[i];
    const double nan = std::nan("");
    o.feasible = 0;
    o.L = 0;
    o.r = o.ttft_d = o.tpot_smooth = nan;
    o.ttft_c = p.k_c * p.l + p.delta_c;
    if (!(p.l > 0.0) || !(p.k_d > 0.0) || !(p.tpot_c > 0.0) || !(p.tau > p.tpot_d) ||
        !(p.k_c >= 0.0) || !(p.delta >= p.delta_c) || !(p.delta_c >= 0.0) || !(p.xi > 0.0))
      continue;
    const double kdl = p.k_d * p.l;
    const double r_ub = std::min(1.0, 1.0 - (p.k_c + p.delta / p.l) / p.k_d);
    const double gap = p.tau - p.tpot_d;
    // With m = L - 1: the lower bound of L holds for r <= (m*gap + TTFT_c)/(k_d l), the
    // upper bound for r >= (m*TPOT_c - decompress)/(k_d l); both ends grow with m, so the
    // first m whose interval meets [xi, r_ub] gives the smallest r.  Start one below the m at
    // which the first end reaches xi (rounding) and stop once the second end passes r_ub.
    double m0 = std::ceil((kdl * p.xi - o.ttft_c) / gap) - 1.0;
    if (!(m0 >= 1.0)) m0 = 1.0;
    if (m0 > 2147483000.0) continue;
    for (long long m = (long long)m0; m < (long long)m0 + 4 && m < 2147483647LL; ++m) {
      const double r_from = ((double)m * p.tpot_c - (p.delta - p.delta_c)) / kdl;
      const double r_to = ((double)m * gap + o.ttft_c) / kdl;
      const double lo = std::max(p.xi, r_from), hi = std::min(r_ub, r_to);
      if (r_from > r_ub) break;
      if (lo <= hi && lo > 0.0) {
        o.feasible = 1;
        o.r = lo;
        o.L = (int32_t)(m + 1);
        o.ttft_d = p.k_c * p.l + p.delta + p.k_d * lo * p.l;
        o.tpot_smooth = p.tpot_d + (p.k_d * lo * p.l - o.ttft_c) / (double)m;
        break;
      }
      // r_to < xi cannot happen past m0 + 1, so an empty interval here means r_from > r_to:
      // larger m only helps if the interval's ends are moving apart
      if (r_to >= p.xi && p.tpot_c >= gap) break;
    }
  }
  return PDD_OK;
}

int pdd_refine_from_colsum_static(const float* colsum, int64_t ld, int32_t n_heads,
                                  const uint8_t* kinds, int64_t n, int32_t pool_kind,
                                  int32_t pool_k, int64_t cand_lo, int64_t cand_hi,
                                  double keep_ratio, uint8_t* keep, int32_t* n_kept,
                                  void* stream) {
  if (!colsum || !keep || !n_kept) return fail(PDD_ERR_INVALID, "null argument");
  if (n <= 0) return fail(PDD_ERR_INVALID, "n must be positive");
  if (n > PDD_STATIC_SCORE_MAX)
    return fail(PDD_ERR_CAPACITY,
                "pdd_refine_from_colsum_static: n = %lld positions, but the built-in score "
                "buffer holds at most %d; use pdd_token_importance + pdd_refine_topk with a "
                "caller-owned score vector for longer sequences",
                (long long)n, (int)PDD_STATIC_SCORE_MAX);
  if (n_heads <= 0 || ld < n) return fail(PDD_ERR_INVALID, "need n_heads > 0 and ld >= n");
  if (pool_kind < 0 || pool_kind > 2) return fail(PDD_ERR_INVALID, "pool_kind must be 0, 1 or 2");
  if (pool_k < 1 || pool_k % 2 == 0 || pool_k > 1025)
    return fail(PDD_ERR_INVALID, "pool_k must be odd and in 1..1025");
  if (cand_lo < 0 || cand_hi > n || cand_lo > cand_hi)
    return fail(PDD_ERR_INVALID, "candidate range outside [0,n]");
  if (!(keep_ratio >= 0.0 && keep_ratio <= 1.0))
    return fail(PDD_ERR_INVALID, "keep_ratio must be in [0,1]");
  float* score = nullptr;
  int rc = static_score_buffer(&score);
  if (rc) return rc;
  cudaStream_t st = (cudaStream_t)stream;
  // The buffer keeps whatever the previous call left; positions 0..n-1 are overwritten
  // here (accumulate = 0) before the selection reads them, so nothing needs clearing.
  importance_reduce_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(
      colsum, ld, n_heads, n, pool_k == 1 ? 0 : pool_kind, pool_k, score, 0);
  PDD_CUDA(cudaGetLastError());
  TopkBatch tb{};
  tb.s[0].offset = 0;
  tb.s[0].kinds_offset = 0;
  tb.s[0].n = n;
  tb.s[0].cand_lo = cand_lo;
  tb.s[0].cand_hi = cand_hi;
  radix_topk_kernel<ScoreKeys><<<1, kTopkThreads, 0, st>>>(ScoreKeys{score}, kinds, tb, keep_ratio,
                                                           keep, n_kept);
  PDD_CUDA(cudaGetLastError());
  return PDD_OK;
}

int pdd_status(pdd_kv* kv, void* stream, int32_t* sticky_device_status) {
  if (!kv || !sticky_device_status) return fail(PDD_ERR_INVALID, "null argument");
  int32_t v = 0;
  PDD_CUDA(cudaMemcpyAsync(&v, kv->g.dev_status, 4, cudaMemcpyDeviceToHost, (cudaStream_t)stream));
  PDD_CUDA(cudaStreamSynchronize((cudaStream_t)stream));
  *sticky_device_status = v;
  return PDD_OK;
}

int pdd_clear_status(pdd_kv* kv, void* stream) {
  if (!kv) return fail(PDD_ERR_INVALID, "null handle");
  PDD_CUDA(cudaMemsetAsync(kv->g.dev_status, 0, 4, (cudaStream_t)stream));
  return PDD_OK;
}

int pdd_selftest_wait_timeout(pdd_kv* kv, uint32_t limit_us, void* stream) {
  if (!kv) return fail(PDD_ERR_INVALID, "null handle");
  if (limit_us == 0 || limit_us > 100000)
    return fail(PDD_ERR_INVALID, "limit_us must be in 1..100000");
  wait_timeout_probe_kernel<<<1, 32, 0, (cudaStream_t)stream>>>(kv->g.dev_status,
                                                              1000ull * limit_us);
  PDD_CUDA(cudaGetLastError());
  return PDD_OK;
}

int pdd_debug_fail_launch(pdd_kv* kv, int32_t nth) {
  if (!kv) return fail(PDD_ERR_INVALID, "null handle");
  if (nth < 0) return fail(PDD_ERR_INVALID, "nth must not be negative");
  kv->fail_countdown = nth;
  return PDD_OK;
}

int pdd_export_colsum(pdd_kv* kv, int32_t seq_id, float* dst, void* stream) {
  if (!kv || !dst) return fail(PDD_ERR_INVALID, "null argument");
  if (seq_id < 0 || seq_id >= kv->cfg.max_seqs) return fail(PDD_ERR_INVALID, "seq_id out of range");
  const int64_t n = kv->seq_len[seq_id];
  if (n == 0) return PDD_OK;
  const CacheGeom& g = kv->g;
  PDD_CUDA(cudaMemcpy2DAsync(dst, 4 * (size_t)n,
                             g.colsum + (size_t)seq_id * g.hq * g.max_tokens_per_seq,
                             4 * (size_t)g.max_tokens_per_seq, 4 * (size_t)n, g.hq,
                             cudaMemcpyDeviceToDevice, (cudaStream_t)stream));
  return PDD_OK;
}

int pdd_export_kv(pdd_kv* kv, int32_t seq_id, void* k_dst, void* v_dst, void* stream) {
  if (!kv || !k_dst || !v_dst) return fail(PDD_ERR_INVALID, "null argument");
  if (seq_id < 0 || seq_id >= kv->cfg.max_seqs) return fail(PDD_ERR_INVALID, "seq_id out of range");
  const int64_t n = kv->seq_len[seq_id];
  if (n == 0) return PDD_OK;
  kv_export_kernel<<<(unsigned)std::min<int64_t>((n * kv->g.hkv * kv->g.d / 8 + 255) / 256, 4096),
                     256, 0, (cudaStream_t)stream>>>(kv->g, seq_id, n, (__nv_bfloat16*)k_dst,
                                                     (__nv_bfloat16*)v_dst);
  PDD_CUDA(cudaGetLastError());
  return PDD_OK;
}

int pdd_export_kinds(pdd_kv* kv, int32_t seq_id, uint8_t* dst, void* stream) {
  if (!kv || !dst) return fail(PDD_ERR_INVALID, "null argument");
  if (seq_id < 0 || seq_id >= kv->cfg.max_seqs) return fail(PDD_ERR_INVALID, "seq_id out of range");
  const int64_t n = kv->seq_len[seq_id];
  if (n == 0) return PDD_OK;
  PDD_CUDA(cudaMemcpyAsync(dst, kv->g.kinds + (size_t)seq_id * kv->g.max_tokens_per_seq, (size_t)n,
                           cudaMemcpyDeviceToDevice, (cudaStream_t)stream));
  return PDD_OK;
}

int pdd_last_lse(pdd_kv* kv, const float** lse, int64_t* ld_out) {
  if (!kv || !lse || !ld_out) return fail(PDD_ERR_INVALID, "null argument");
  *lse = kv->g.lse;
  *ld_out = kv->g.lse_ld;
  return PDD_OK;
}

int pdd_trace_enable(pdd_kv* kv, int32_t on) {
  if (!kv) return fail(PDD_ERR_INVALID, "null handle");
  kv->trace = on != 0;
  return PDD_OK;
}

int pdd_trace_read(pdd_kv* kv, int32_t cap, const char** names, int64_t* launches,
                   double* total_ms, int32_t* n) {
  if (!kv || !names || !launches || !total_ms || !n) return fail(PDD_ERR_INVALID, "null argument");
  std::map<std::string, std::pair<const char*, std::pair<int64_t, double>>> agg;
  for (auto& t : kv->trace_log) {
    PDD_CUDA(cudaEventSynchronize(t.b));
    float ms = 0.f;
    PDD_CUDA(cudaEventElapsedTime(&ms, t.a, t.b));
    auto& e = agg[t.name];
    e.first = t.name;
    e.second.first += 1;
    e.second.second += ms;
    cudaEventDestroy(t.a);
    cudaEventDestroy(t.b);
  }
  kv->trace_log.clear();
  int i = 0;
  for (auto& kvp : agg) {
    if (i >= cap) break;
    names[i] = kvp.second.first;
    launches[i] = kvp.second.second.first;
    total_ms[i] = kvp.second.second.second;
    ++i;
  }
  *n = i;
  return PDD_OK;
}

int pdd_set_kernel_path(pdd_kv* kv, int32_t path) {
  if (!kv) return fail(PDD_ERR_INVALID, "null handle");
  if (path < 0 || path > 2) return fail(PDD_ERR_INVALID, "path must be 0, 1 or 2");
  kv->kernel_path = path;
  return PDD_OK;
}

int pdd_set_schedule(pdd_kv* kv, int32_t mode) {
  if (!kv) return fail(PDD_ERR_INVALID, "null handle");
  if (mode < 0 || mode > 4) return fail(PDD_ERR_INVALID, "mode must be 0..4");
  kv->schedule = mode;
  return PDD_OK;
}

const char* pdd_strerror(int status) {
  switch (status) {
    case PDD_OK: return "ok";
    case PDD_ERR_INVALID: return "invalid argument";
    case PDD_ERR_STATE: return "call does not match the sequence state";
    case PDD_ERR_CAPACITY: return "capacity exceeded";
    case PDD_ERR_CUDA: return "CUDA call failed";
    case PDD_ERR_TIMEOUT: return "a bounded device-side wait ran out";
    case PDD_ERR_UNSUPPORTED: return "unsupported shape or device";
    default: return "unknown status";
  }
}

const char* pdd_last_error_detail(void) { return g_detail; }

}  // extern "C"
