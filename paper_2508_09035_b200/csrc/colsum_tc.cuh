// colsum: attention mass per key position from the call's observation-window rows.
//
//   colsum[h][j] += sum over window rows i of this call with pos(i) >= j of
//                   exp(scale * q_i . k_j - LSE_i)
//
// K-stationary, transposed scores: a CTA owns 128 keys of one KV head and computes
// S^T = K_tile Q_tile^T with tcgen05.mma (A = K tile, B = Q tile, both K-major in
// 128B-swizzled shared memory), so that a TMEM lane is a KEY and the columns run along
// QUERIES.  Each consumer thread owns one key: it adds exp2(s*c - lse2[i]) over its row
// of the accumulator for every (query head of the group, query tile) and finally does one
// plain read-modify-write of colsum[h][j]: no shuffles, no atomics, and the same bits
// on every run.  The row normaliser must be final before a probability can be summed, so
// this is a second score pass that reads the LSE the attention kernel wrote.
//   warp 0    TMA producer (K tile once, Q tiles through a 2-stage ring)
//   warp 1    MMA issuer; two 128-column accumulators in TMEM alternate
//   warps 2-5 consumers of the even items (accumulator 0), warps 6-9 of the odd items
//             (accumulator 1): with two CTAs per SM four consumer warps share a scheduler,
//             which is what keeps the MUFU unit busy (two left it idle half of the time)
// A head's items go to both consumer groups, so each group leaves its partial sum of a
// (head, key) in shared memory and one thread adds the two in a fixed order at the end.
#pragma once
#include "common.cuh"
#include "ptx.cuh"

namespace pdd {

constexpr int kColsumThreads = 320;
constexpr int kColsumMaxHeads = 8;      // query heads per CTA (more are dealt out to further CTAs)
// Pairs of every 4 whose exp2 is a polynomial on the FMA pipe (measured on the long-prompt
// window pass: 0 -> 0.83 ms, 1 -> 0.78, 2 -> 0.80, 3 -> 0.91).
constexpr int kColsumPoly = 1;

__device__ __forceinline__ float ex2f_cs(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

template <int D>
struct ColsumSmem {
  static constexpr int kSub = D / 64;
  static constexpr int kSubBytes = 128 * 128;
  static constexpr int kTileBytes = kSub * kSubBytes;
  static constexpr int kKOff = 0;
  static constexpr int kQOff = kTileBytes;                 // 2 stages
  static constexpr int kLseOff = 3 * kTileBytes;           // 2 groups x 2 buffers x 128 floats
  static constexpr int kPartOff = kLseOff + 2048;          // 2 groups x kColsumMaxHeads x 128 floats
  static constexpr int kBarOff = kPartOff + 2 * kColsumMaxHeads * 512;
  static constexpr int kBytes = kBarOff + 256 + 1024;
};

struct ColsumBars {
  uint64_t k_full;
  uint64_t q_full[2], q_empty[2];
  uint64_t s_full[2], s_empty[2];
  uint64_t lse_ready[2];
  uint32_t tmem_base;
  int32_t abort_flag;
};

template <int D>
__global__ void __launch_bounds__(kColsumThreads, 2)
colsum_tc_kernel(CacheGeom g, const void* __restrict__ rec, int hsplit,
                 const __grid_constant__ CUtensorMap tmQ,
                 const __grid_constant__ CUtensorMap tmK) {
  using L = ColsumSmem<D>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) &
                                             ~(uintptr_t)1023);
  uint8_t* sK = base + L::kKOff;
  uint8_t* sQ = base + L::kQOff;
  float* sLse = reinterpret_cast<float*>(base + L::kLseOff);
  float* sPart = reinterpret_cast<float*>(base + L::kPartOff);
  ColsumBars* bars = reinterpret_cast<ColsumBars*>(base + L::kBarOff);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  // The record's device slot is filled by kv_append, and this kernel may be scheduled as soon
  // as the attention kernel has started: nothing is read before the kernels ahead are done
  // (their LSE rows and cache rows are needed anyway).
  ptx::griddep_launch_dependents();
  ptx::griddep_wait();
  // blockIdx.x runs over the key blocks of all window sequences of the call, one after another
  const CallHeader* hdr = reinterpret_cast<const CallHeader*>(rec);
  const SeqDesc* descs = record_descs(rec);
  int kt = blockIdx.x, seq_slot = 0;
  for (; seq_slot < hdr->n_seqs; ++seq_slot) {
    const SeqDesc& d = descs[seq_slot];
    if (!d.window || d.len <= 0) continue;
    const int n_kb = (int)((d.pos0 + d.len + kKeyBlock - 1) / kKeyBlock);
    if (kt < n_kb) break;
    kt -= n_kb;
  }
  if (seq_slot >= hdr->n_seqs) return;
  const SeqDesc sd = descs[seq_slot];
  const int G = g.hq / g.hkv;
  // blockIdx.y = (KV head, part): with few key blocks and KV heads the query heads of a group
  // are dealt out to `hsplit` CTAs (each still the only writer of its heads' column sums)
  const int kvh = blockIdx.y / hsplit;
  const int hpc = G / hsplit;                                   // query heads per CTA
  const int h_first = kvh * G + (blockIdx.y % hsplit) * hpc;
  const int64_t key0 = (int64_t)kt * kKeyBlock;
  const int64_t T = sd.pos0 + sd.len;
  const int n_qt = (sd.len + kTileRows - 1) / kTileRows;
  // first query tile that holds a row at or after this key tile's first key
  const int qt_min = key0 > sd.pos0 ? (int)((key0 - sd.pos0) / kTileRows) : 0;
  // last query tile with a row that still sees this key tile's LAST key under the sliding
  // window (rows key .. key+window-1 see a key)
  const int64_t p_hi = key0 + kKeyBlock - 1 + g.window - 1;
  const int qt_end = p_hi < sd.pos0 ? 0 : (int)min((int64_t)n_qt, (p_hi - sd.pos0) / kTileRows + 1);
  const int n_qt_act = qt_end - qt_min;
  const int n_items = hpc * n_qt_act;             // item = (head of this CTA, query tile)
  if (n_items <= 0 || key0 >= T) return;
  __shared__ int s_skip;   // a launch that follows a timed-out wait does no work
  if (tid == 0) s_skip = *reinterpret_cast<volatile int32_t*>(g.dev_status);
  __syncthreads();
  if (s_skip) return;

  if (tid == 0) {
    ptx::mbar_init(&bars->k_full, 1);
    for (int s = 0; s < 2; ++s) {
      ptx::mbar_init(&bars->q_full[s], 1);
      ptx::mbar_init(&bars->q_empty[s], 1);
      ptx::mbar_init(&bars->s_full[s], 1);
      ptx::mbar_init(&bars->s_empty[s], 128);
      ptx::mbar_init(&bars->lse_ready[s], 128);
    }
    bars->abort_flag = 0;
    ptx::fence_mbar_init();
  }
  for (int i = tid; i < 2 * kColsumMaxHeads * 128; i += kColsumThreads) sPart[i] = 0.f;
  if (warp == 1) {
    ptx::tmem_alloc(&bars->tmem_base, 256);
    ptx::tmem_relinquish();
  }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem = bars->tmem_base;
  volatile int32_t* abort_flag = &bars->abort_flag;

  if (warp == 0) {
    if (lane == 0) {
      ptx::prefetch_tensormap(&tmQ);
      ptx::prefetch_tensormap(&tmK);
      ptx::mbar_expect_tx(&bars->k_full, L::kTileBytes);
      for (int hh = 0; hh < 2; ++hh) {
        const int64_t pos = key0 + 64 * hh;
        const int slot = (int)(pos / g.page_tokens);
        const int page = slot < g.pages_per_seq
                             ? g.page_table[(size_t)sd.seq_id * g.pages_per_seq + slot] : 0;
        const int rin = (int)(pos % g.page_tokens);
        for (int sub = 0; sub < L::kSub; ++sub)
          ptx::tma_load_4d(sK + sub * L::kSubBytes + hh * 8192, &tmK, &bars->k_full, 64 * sub, rin,
                           kvh, page);
      }
      bool ok = true;
      int h = h_first, qt = qt_min;
      for (int it = 0; it < n_items && ok; ++it) {
        const int st = it & 1;
        if (it >= 2) ok = ptx::mbar_wait(&bars->q_empty[st], (uint32_t)((it >> 1) - 1) & 1);
        if (!ok) break;
        ptx::mbar_expect_tx(&bars->q_full[st], L::kTileBytes);
        for (int sub = 0; sub < L::kSub; ++sub)
          ptx::tma_load_3d(sQ + st * L::kTileBytes + sub * L::kSubBytes, &tmQ, &bars->q_full[st],
                           64 * sub, h, (int)(sd.tok_offset + (int64_t)qt * kTileRows));
        if (++qt == qt_end) {
          qt = qt_min;
          ++h;
        }
      }
      if (!ok) *abort_flag = 1;
    }
  } else if (warp == 1) {
    if (lane == 0) {
      constexpr uint32_t idesc = ptx::instr_desc_bf16(128, 128, 0, 0);
      const uint32_t k_addr = ptx::smem_u32(sK), q_addr = ptx::smem_u32(sQ);
      bool ok = ptx::mbar_wait(&bars->k_full, 0);
      for (int it = 0; it < n_items && ok; ++it) {
        const int st = it & 1;
        const uint32_t ph = (uint32_t)(it >> 1) & 1;
        ok = ptx::mbar_wait(&bars->q_full[st], ph);
        if (ok && it >= 2) ok = ptx::mbar_wait(&bars->s_empty[st], ph ^ 1);
        if (!ok) break;
        ptx::tc_fence_after();
#pragma unroll
        for (int ks = 0; ks < D / 16; ++ks) {
          const uint32_t off = (ks / 4) * L::kSubBytes + (ks % 4) * 32;
          ptx::mma_ss(tmem + 128 * st, ptx::smem_desc_sw128(k_addr + off, 16, 1024),
                      ptx::smem_desc_sw128(q_addr + st * L::kTileBytes + off, 16, 1024), idesc,
                      ks > 0);
        }
        ptx::mma_commit(&bars->s_full[st]);
        ptx::mma_commit(&bars->q_empty[st]);
      }
      if (!ok) *abort_flag = 1;
    }
  } else {
    const int cg = (warp - 2) >> 2;                   // consumer group: items cg, cg + 2, ...
    const int wq = warp & 3;                          // TMEM lane quarter this warp may read
    const int r = wq * 32 + lane;                     // key row of the tile
    const int ct = (tid - 64) & 127;                  // 0..127 inside the group
    const uint32_t lane_base = (uint32_t)(wq * 32) << 16;
    const int64_t key = key0 + r;
    const float sl2 = g.scale * 1.4426950408889634f;
    const float2 sl2v = make_float2(sl2, sl2);
    float acc = 0.f;
    bool ok = true;
    float* const part = sPart + (size_t)cg * kColsumMaxHeads * 128 + r;    // [head of the CTA][key]
    // Minus the LSE (exp2 domain) of the rows of an item's query tile; fetched one item ahead so
    // that the global-memory latency falls under the previous item's exponentials.
    auto fetch_lse = [&](int h, int qt) -> float {
      const int rows_valid = min(kTileRows, sd.len - qt * kTileRows);
      const int64_t row0 = sd.tok_offset + (int64_t)qt * kTileRows;
      return ct < rows_valid ? g.lse[(size_t)h * g.lse_ld + row0 + ct] * -1.4426950408889634f : 0.f;
    };
    // item it = (head h_first + it / n_qt_act, query tile qt_min + it % n_qt_act), stepped
    // without divisions; this group takes items cg, cg + 2, ...; (hn, qn) is its next item
    auto advance = [&](int& hh, int& qq) {
      if (++qq == qt_end) {
        qq = qt_min;
        ++hh;
      }
    };
    int h = h_first, qt = qt_min;
    if (cg) advance(h, qt);
    int hn = h, qn = qt, cur_h = h;
    float lse_next = cg < n_items ? fetch_lse(h, qt) : 0.f;
    for (int it = cg, n = 0; it < n_items; it += 2, ++n, h = hn, qt = qn) {
      const int st = cg;                          // the group's accumulator and Q stage
      const uint32_t ph = (uint32_t)n & 1;
      advance(hn, qn);
      advance(hn, qn);
      if (h != cur_h) {
        part[(cur_h - h_first) * 128] = acc;
        acc = 0.f;
        cur_h = h;
      }
      const int rows_valid = min(kTileRows, sd.len - qt * kTileRows);
      const int64_t pq0 = sd.pos0 + (int64_t)qt * kTileRows;     // position of query column 0
      // (two LSE buffers per group: a thread that is already at item n + 1 writes the other one
      // than the threads still reading item n)
      float* const lse_buf = sLse + (cg * 2 + (n & 1)) * 128;
      lse_buf[ct] = lse_next;
      ptx::mbar_arrive(&bars->lse_ready[st]);
      if (it + 2 < n_items) lse_next = fetch_lse(hn, qn);
      ok = ptx::mbar_wait(&bars->lse_ready[st], ph);
      if (ok) ok = ptx::mbar_wait(&bars->s_full[st], ph);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      ptx::tc_fence_after();
      const bool full = rows_valid == kTileRows && pq0 >= key0 + kKeyBlock - 1 &&
                        pq0 + kTileRows - 1 - key0 < g.window;
      // LSE of the 16 columns in hand, as four 16-byte shared-memory loads (every thread of
      // the warp reads the same words: one broadcast each).  Going through the generic float
      // pointer instead costs one load instruction per exponential, and those loads, not the
      // MUFU unit, then bound the kernel.
      const uint32_t ls_addr = ptx::smem_u32(lse_buf);
      // 16 query columns at a time; the next 16 are on their way while these are
      // exponentiated, and the accumulator goes back to the MMA thread as soon as the last
      // ones have landed in registers.  Two partial sums, added in a fixed order.
      float acc0 = 0.f, acc1 = 0.f;
      auto add16 = [&](int c16, const uint32_t* v) {
        float ls[16];
#pragma unroll
        for (int i = 0; i < 4; ++i)
          asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];"
                       : "=f"(ls[4 * i]), "=f"(ls[4 * i + 1]), "=f"(ls[4 * i + 2]), "=f"(ls[4 * i + 3])
                       : "r"(ls_addr + (uint32_t)(c16 * 64 + i * 16)));
        if (full) {
          // kColsumPoly of every 4 pairs go through a cubic on the FMA pipe instead of the MUFU
          // unit (7.5e-5 relative error against a 1e-2 bound on the sums).
          // (packed fp32x2 multiply-add and add: the issue slots, 60 % busy, are the next bound)
          float2 a01 = make_float2(acc0, acc1);
#pragma unroll
          for (int c = 0; c < 16; c += 8) {
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              const float2 x = __ffma2_rn(make_float2(__uint_as_float(v[c + 2 * i]),
                                                      __uint_as_float(v[c + 2 * i + 1])),
                                          sl2v, make_float2(ls[c + 2 * i], ls[c + 2 * i + 1]));
              const float2 e = i < kColsumPoly ? ptx::ex2_poly2(x)
                                               : make_float2(ex2f_cs(x.x), ex2f_cs(x.y));
              a01 = __fadd2_rn(a01, e);
            }
          }
          acc0 = a01.x;
          acc1 = a01.y;
        } else {
#pragma unroll
          for (int c = 0; c < 16; ++c) {
            const int col = c16 * 16 + c;
            const float e = ex2f_cs(fmaf(__uint_as_float(v[c]), sl2, ls[c]));
            const float ee = (col < rows_valid && pq0 + col >= key && pq0 + col - key < g.window) ? e : 0.f;
            if (c & 1) acc1 += ee; else acc0 += ee;
          }
        }
      };
      const uint32_t tacc = tmem + 128 * st + lane_base;
      uint32_t va[16], vb[16];
      ptx::tmem_ld16(tacc, va);
#pragma unroll
      for (int c16 = 0; c16 < 8; c16 += 2) {
        ptx::tmem_ld_wait();
        ptx::tmem_ld16(tacc + 16 * (c16 + 1), vb);
        add16(c16, va);
        ptx::tmem_ld_wait();
        if (c16 + 2 < 8) {
          ptx::tmem_ld16(tacc + 16 * (c16 + 2), va);
        } else {
          ptx::tc_fence_before();
          ptx::mbar_arrive(&bars->s_empty[st]);
        }
        add16(c16 + 1, vb);
      }
      acc += acc0 + acc1;
    }
    if (cg < n_items) part[(cur_h - h_first) * 128] = acc;
    if (!ok && lane == 0) *abort_flag = 1;
    // Both groups' partial sums stand: the threads of group cg finish heads cg, cg + 2, ... of
    // the CTA, each the only writer of its (head, key) in global memory.
    ptx::named_bar_sync(1, 256);
    if (!*abort_flag && key < T) {
      for (int hl = cg; hl < hpc; hl += 2) {
        const float sum = sPart[hl * 128 + r] + sPart[(kColsumMaxHeads + hl) * 128 + r];
        g.colsum[((size_t)sd.seq_id * g.hq + h_first + hl) * g.max_tokens_per_seq + key] += sum;
      }
    }
  }

  ptx::tc_fence_before();
  __syncthreads();
  if (tid == 0 && *abort_flag) atomicExch(g.dev_status, 5);
  if (warp == 1) {
    __syncwarp();
    ptx::tc_fence_after();
    ptx::tmem_dealloc(tmem, 256);
  }
}

// One-time set-up on the current device: dynamic shared memory limit.
inline cudaError_t prepare_colsum_tc(int d) {
  return d == 128 ? cudaFuncSetAttribute(colsum_tc_kernel<128>,
                                         cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         ColsumSmem<128>::kBytes)
                  : cudaFuncSetAttribute(colsum_tc_kernel<64>,
                                         cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         ColsumSmem<64>::kBytes);
}

// One launch for all window sequences of a call: n_kb_total = their key blocks, added up.
inline cudaError_t launch_colsum_tc(const CacheGeom& g, const void* rec_dev, int n_kb_total,
                                    const CUtensorMap& tmQ, const CUtensorMap& tmK, int sm_count,
                                    cudaStream_t st) {
  if (n_kb_total <= 0) return cudaSuccess;
  // Two CTAs fit on an SM.  When (key blocks x KV heads) leaves most of those slots empty, the
  // heads of a GQA group go to separate CTAs: the largest divisor of the group size that
  // still fits one wave (the K tile is then fetched once per part, from L2).
  const int G = g.hq / g.hkv, slots = 2 * sm_count;
  int hsplit = 1;
  while (G % hsplit != 0 || G / hsplit > kColsumMaxHeads) ++hsplit;     // ends at G at the latest
  for (int s = hsplit + 1; s <= G; ++s)
    if (G % s == 0 && (int64_t)n_kb_total * g.hkv * s <= slots) hsplit = s;
  dim3 grid((unsigned)n_kb_total, (unsigned)(g.hkv * hsplit));
  if (g.d == 128)
    return launch_pdl(colsum_tc_kernel<128>, grid, dim3(kColsumThreads), ColsumSmem<128>::kBytes,
                      st, g, rec_dev, hsplit, tmQ, tmK);
  return launch_pdl(colsum_tc_kernel<64>, grid, dim3(kColsumThreads), ColsumSmem<64>::kBytes,
                    st, g, rec_dev, hsplit, tmQ, tmK);
}

}  // namespace pdd
