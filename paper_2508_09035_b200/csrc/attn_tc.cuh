// fwd_attn: pipelined tensor-core causal attention over the paged KV cache.
//
// Work item = a PAIR of 128-row query tiles that read the same KV head of the same
// sequence (two query heads of one GQA group on the same rows, or, when the group size
// is odd, two consecutive row blocks of one head), so every K/V block staged in shared
// memory feeds two tiles.  The call's (pair, key block) units are cut into equal shares,
// one per CTA (one CTA per SM): a CTA walks its share pair by pair.  Where a share ends
// inside a pair, the CTA leaves a partial result (unnormalised O, running max, row sum)
// in its scratch slot and attn_combine_kernel merges the partials of that pair.
// Third way to cut the work, for calls with few pairs: a thread-block cluster of c CTAs per
// pair, CTA k taking the k-th of c equal parts of the pair's key blocks; the c partial
// results are merged through distributed shared memory (the merge's (tile, column group)
// jobs are dealt out to the cluster's CTAs, each reading the others' exported partials),
// with no scratch traffic and no second kernel.
//
// Roles inside a CTA:
//   warp 0      TMA producer: Q tiles per pair, K and V blocks through two 2-stage rings
//   warp 1      MMA issuer of the scores (one thread): S_t(j) = Q_t K(j)^T with tcgen05.mma,
//               S_0(j), S_1(j), S_0(j+1), ... (the warp also owns the TMEM allocation)
//   warp 2      MMA issuer of the PV products (one thread): O_t += P_t(j) V(j).
//               The scores of block j+1 do not wait for the PV product of block j (P has
//               TMEM columns of its own), so a tile's softmax has a whole round of the other
//               MMAs to finish in, and the tensor pipe, not the chain MMA -> softmax -> MMA,
//               bounds the loop.  Two issuing threads, because each barrier wait costs the
//               waiting thread ~100 cycles even when the barrier has completed, and the
//               pipe's queue is too short to bridge that.
//   warp 3      idle (it completes the control warpgroup)
//   warps 4-7   softmax of tile 0 (one row per thread, the whole S row in registers),
//               rescale of O_0, epilogue
//   warps 8-11  the same for tile 1
// The control warpgroup gives registers back (setmaxnreg.dec) and the two softmax
// warpgroups take them (setmaxnreg.inc); the host checks the split against the kernel's
// register count before the first launch, because a split above it would wait forever.
// TMEM (512 columns): S | P_0 | P_1 | O_0 | O_1.  S (128 fp32 columns) is shared by the two
// tiles: a softmax warpgroup takes its whole row of S into registers as soon as it is
// complete and hands the columns back (s_free), so they are free for the other tile's next
// scores long before they are needed.  P_t (64 columns, packed bf16) has columns of its own
// and is the TMEM A operand of the PV product; because it does not lie over S, the scores of
// block j+1 can be computed while P_t(j) still waits for its PV product.  O_t: 128 columns
// each (head_dim of them used).  All waits are bounded; on expiry the kernel raises the sticky
// status word and every role leaves through the common exit that frees TMEM.
#pragma once
#include <type_traits>

#include "common.cuh"
#include "ptx.cuh"

namespace pdd {

constexpr int kAttnThreads = 384;
constexpr int kMaxCluster = 8;     // largest thread-block cluster the cluster schedule uses
constexpr int kKvStages = 2;
constexpr bool kPolyExp = false;     // measured slower on B200 (1167 -> 987 TFLOP/s): the softmax is not MUFU-bound
constexpr int kCtrlRegs = 64;       // registers per thread kept by the control warpgroup
constexpr int kSoftmaxRegs = 216;   // registers per thread taken by each softmax warpgroup

__device__ __forceinline__ void setmaxnreg_dec_ctrl() {
  asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kCtrlRegs));
}
__device__ __forceinline__ void setmaxnreg_inc_softmax() {
  asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(kSoftmaxRegs));
}

template <int D>
struct AttnSmem {
  static constexpr int kSub = D / 64;
  static constexpr int kSubBytes = 128 * 128;            // [128 rows][64 bf16] swizzled
  static constexpr int kTileBytes = kSub * kSubBytes;    // one 128 x D operand tile
  static constexpr int kQOff = 0;                        // 2 tiles
  static constexpr int kKOff = 2 * kTileBytes;           // kKvStages tiles
  static constexpr int kVOff = kKOff + kKvStages * kTileBytes;
  static constexpr int kBarOff = kVOff + kKvStages * kTileBytes;
  static constexpr int kBytes = kBarOff + 512 + 1024;    // barriers + alignment slack
};

struct AttnBars {
  uint64_t q_full[2], q_empty[2];
  uint64_t k_full[kKvStages], k_empty[kKvStages];
  uint64_t v_full[kKvStages], v_empty[kKvStages];
  uint64_t s_ready[2];    // MMA -> softmax: S_t(j) complete (and all earlier MMAs)
  uint64_t p_ready[2];    // softmax -> MMA: P_t(j) in TMEM, O_t rescaled
  uint64_t o_done[2];     // MMA -> softmax: last PV of tile t in this segment complete
  uint64_t pv_done[2];    // MMA -> softmax: PV_t(j) complete (P_t may be overwritten, O_t rescaled)
  uint64_t s_free;        // softmax -> MMA: the shared S columns have been read
  // cluster mode: x_full[t] collects, in every CTA, the other CTAs' "my export of tile t
  // stands"; x_free[t] their "I am done reading your export of tile t"
  uint64_t x_full[2], x_free[2];
  uint32_t tmem_base;
  int32_t abort_flag;
};

// Size of one scratch slot (both tiles) in floats / float2s.
__host__ __device__ constexpr size_t part_o_floats(int d) { return (size_t)2 * 128 * d; }
__host__ __device__ constexpr size_t part_ml_elems() { return (size_t)2 * 128; }

// Decoded tile pair.
struct PairWork {
  int seq_slot;
  int head[2];
  int t_local[2];       // 128-row tile index inside the sequence's rows of this call
  int active[2];
  int kvh;
};

// Pairs are numbered per sequence; with an even group size pair p covers heads
// (2*(p % (hq/2)), +1) of row block p / (hq/2); with an odd group size it covers row
// blocks (2*(p / hq), +1) of head p % hq.
__device__ __forceinline__ PairWork decode_pair(const CallHeader* hdr, const SeqDesc* descs,
                                                int pair, int hq, int hkv) {
  PairWork w;
  int s = 0;
  while (s + 1 < hdr->n_seqs && descs[s + 1].pair0 <= pair) ++s;
  const int p = pair - descs[s].pair0;
  const int G = hq / hkv;
  const int ntile = (descs[s].len + kTileRows - 1) / kTileRows;
  w.seq_slot = s;
  if ((G & 1) == 0) {
    const int hp = p % (hq / 2), rb = p / (hq / 2);
    w.head[0] = 2 * hp;
    w.head[1] = 2 * hp + 1;
    w.t_local[0] = w.t_local[1] = rb;
    w.active[0] = w.active[1] = 1;
  } else {
    const int h = p % hq, rbp = p / hq;
    w.head[0] = w.head[1] = h;
    w.t_local[0] = 2 * rbp;
    w.t_local[1] = 2 * rbp + 1;
    w.active[0] = 1;
    w.active[1] = (2 * rbp + 1) < ntile;
  }
  w.kvh = w.head[0] / G;
  return w;
}

// One stretch of a CTA's share: key blocks [kb_lo, kb_hi) of one pair.  A pair's blocks run
// from kb_first (the first block its first tile can see under the sliding window; 0 without
// one) to the causal end of its last tile; the schedule counts them from kb_first.
struct Segment {
  PairWork w;
  int seq_id;
  int kb_lo, kb_hi;
  int kb_first;
  int n_kb[2];          // one past the last key block each tile needs (causal extent)
  int nblk[2];          // key blocks of this segment that each tile takes part in
  int rows_valid[2];
  int seq_pos0;         // cache position of the sequence's first row of this call
  int row0[2];          // packed row of tile row 0
  int p0[2];            // cache position of tile row 0
  int full;             // the segment covers the pair's whole key range
  int slot;             // scratch slot of this CTA for a partial result
};

__device__ __forceinline__ void describe_pair(const CallHeader* hdr, const SeqDesc* descs,
                                              const CacheGeom& g, int pair, Segment& sg) {
  sg.w = decode_pair(hdr, descs, pair, g.hq, g.hkv);
  const SeqDesc& sd = descs[sg.w.seq_slot];
  sg.seq_id = sd.seq_id;
  sg.seq_pos0 = (int)sd.pos0;
#pragma unroll
  for (int t = 0; t < 2; ++t) {
    sg.rows_valid[t] = sg.w.active[t] ? min(kTileRows, sd.len - sg.w.t_local[t] * kTileRows) : 0;
    sg.row0[t] = (int)sd.tok_offset + sg.w.t_local[t] * kTileRows;
    sg.p0[t] = (int)sd.pos0 + sg.w.t_local[t] * kTileRows;
    sg.n_kb[t] = sg.rows_valid[t] > 0 ? (sg.p0[t] + sg.rows_valid[t] - 1) / kKeyBlock + 1 : 0;
  }
  sg.kb_first = 0;
}

// Walks the segments of a CTA's share.  Every role runs the same walk.  kBand: the cache
// has a sliding window (the plain causal kernel is compiled without any of the band code).
template <bool kBand, bool kCluster>
struct SegmentWalk {
  const CallHeader* hdr;
  const SeqDesc* descs;
  CtaStart cs, ce;
  int pair, index;
  int csize, crank;     // cluster mode (csize > 1): the crank-th of csize parts of pair cta/csize
  __device__ __forceinline__ SegmentWalk(const void* rec, int cta, int csize_, int crank_) {
    hdr = reinterpret_cast<const CallHeader*>(rec);
    descs = record_descs(rec);
    csize = csize_;
    crank = crank_;
    index = 0;
    if (kCluster) {
      pair = cta / csize;
      return;
    }
    const CtaStart* st =
        reinterpret_cast<const CtaStart*>(reinterpret_cast<const char*>(rec) + hdr->cta_off);
    cs = st[cta];
    ce = st[cta + 1];
    pair = cs.pair;
  }
  __device__ __forceinline__ bool next(const CacheGeom& g, Segment& sg) {
    if (kCluster) {
      // exactly one segment, possibly empty (the CTA still takes part in the merge)
      if (index > 0 || pair >= hdr->n_pairs) return false;
      describe_pair(hdr, descs, g, pair, sg);
      if (kBand) sg.kb_first = first_key_block(sg.p0[0], g.window);
      const int units = max(sg.n_kb[0], sg.n_kb[1]) - sg.kb_first;
      sg.kb_lo = sg.kb_first + units * crank / csize;
      sg.kb_hi = sg.kb_first + units * (crank + 1) / csize;
      sg.full = 0;
      sg.slot = 0;
#pragma unroll
      for (int t = 0; t < 2; ++t)
        sg.nblk[t] = max(0, min(sg.kb_hi, sg.n_kb[t]) - sg.kb_lo);
      ++index;
      return true;
    }
    if (pair > ce.pair || pair >= hdr->n_pairs) return false;
    if (pair == ce.pair && ce.kb == 0) return false;
    describe_pair(hdr, descs, g, pair, sg);
    // Tile 0 is the earlier one, so its first visible block is the pair's.  The later tile
    // of a row-block pair may meet one leading block wholly below its band: the mask
    // zeroes it.
    if (kBand) sg.kb_first = first_key_block(sg.p0[0], g.window);
    const int nb = max(sg.n_kb[0], sg.n_kb[1]);
    sg.kb_lo = sg.kb_first + ((pair == cs.pair) ? cs.kb : 0);
    sg.kb_hi = (pair == ce.pair) ? sg.kb_first + ce.kb : nb;
    sg.full = sg.kb_lo == sg.kb_first && sg.kb_hi == nb;
    sg.slot = index == 0 ? 0 : 1;
#pragma unroll
    for (int t = 0; t < 2; ++t)
      sg.nblk[t] = max(0, min(sg.kb_hi, sg.n_kb[t]) - sg.kb_lo);
    ++pair;
    ++index;
    return true;
  }
};

template <int D, bool kBand, bool kCluster, bool kRecInParam>
__global__ void __launch_bounds__(kAttnThreads, 1)
fwd_attn_kernel(CacheGeom g, const void* __restrict__ rec_global,
                const __grid_constant__ RecParam recp,
                const __grid_constant__ CUtensorMap tmQ,
                const __grid_constant__ CUtensorMap tmK,
                const __grid_constant__ CUtensorMap tmV, __nv_bfloat16* __restrict__ out) {
  using L = AttnSmem<D>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) &
                                             ~(uintptr_t)1023);
  uint8_t* sQ = base + L::kQOff;
  uint8_t* sK = base + L::kKOff;
  uint8_t* sV = base + L::kVOff;
  AttnBars* bars = reinterpret_cast<AttnBars*>(base + L::kBarOff);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int cta = blockIdx.x;
  // kCluster: launched with one thread-block cluster per pair (compiled apart, so that the
  // merge through distributed shared memory costs the other schedules no registers)
  const int csize = kCluster ? (int)ptx::cluster_nctarank() : 1;
  const int crank = kCluster ? (int)ptx::cluster_ctarank() : 0;

  ptx::griddep_launch_dependents();     // merge / column-sum kernels may be scheduled early
  if (tid == 0) {
    for (int t = 0; t < 2; ++t) {
      ptx::mbar_init(&bars->q_full[t], 1);
      ptx::mbar_init(&bars->q_empty[t], 1);
      ptx::mbar_init(&bars->s_ready[t], 1);
      ptx::mbar_init(&bars->p_ready[t], 128);
      ptx::mbar_init(&bars->o_done[t], 1);
      ptx::mbar_init(&bars->pv_done[t], 1);
      ptx::mbar_init(&bars->x_full[t], kCluster && csize > 1 ? 128 * (csize - 1) : 1);
      ptx::mbar_init(&bars->x_free[t], kCluster && csize > 1 ? 128 * (csize - 1) : 1);
    }
    for (int s = 0; s < kKvStages; ++s) {
      ptx::mbar_init(&bars->k_full[s], 1);
      ptx::mbar_init(&bars->k_empty[s], 1);
      ptx::mbar_init(&bars->v_full[s], 1);
      ptx::mbar_init(&bars->v_empty[s], 1);
    }
    ptx::mbar_init(&bars->s_free, 128);
    bars->abort_flag = 0;
    ptx::fence_mbar_init();
  }
  if (warp == 1) {
    ptx::tmem_alloc(&bars->tmem_base, 512);
    ptx::tmem_relinquish();
  }
  // A small call record arrives as a kernel parameter, so every role can decode its work
  // while the kernel ahead in the stream (kv_append) is still running; a large one is read
  // from its device slot, which that kernel's predecessor in the stream (a copy) filled.
  // (a compile-time choice: a pointer that may be either costs the key-block loop registers)
  const void* rec = kRecInParam ? reinterpret_cast<const void*>(&recp) : rec_global;
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  // Other CTAs of the cluster arrive on this CTA's barriers at the end of their work: they
  // must not do so before the barriers exist.  Every thread of the cluster gets here.
  if (kCluster) ptx::cluster_sync_all();
  const uint32_t tmem = bars->tmem_base;
  volatile int32_t* abort_flag = &bars->abort_flag;
  // When this kernel starts, every kernel before the call's kv_append has completed (kv_append
  // lets its dependents go only after its own wait), so the only work that may still be in
  // flight is kv_append's: the call's new cache rows and the page-table entries of their pages.
  // Nothing else this kernel touches depends on it.  Only the producer therefore waits for the
  // kernel ahead, and only when it reaches the first key block that holds a new row: key blocks
  // below pos0 are fetched and multiplied while kv_append is still copying.  A launch that
  // follows a timed-out wait (sticky status) does no work.
  auto status_set = [&]() -> bool {
    return *reinterpret_cast<volatile int32_t*>(g.dev_status) != 0;
  };

  if (warp < 4) {
    setmaxnreg_dec_ctrl();
    if (warp == 0 && lane == 0) {
      // ---------------------------------------------------------------- producer
      ptx::prefetch_tensormap(&tmQ);
      ptx::prefetch_tensormap(&tmK);
      ptx::prefetch_tensormap(&tmV);
      SegmentWalk<kBand, kCluster> walk(rec, cta, csize, crank);
      Segment sg;
      int kv_it = 0;
      uint32_t q_cnt0 = 0, q_cnt1 = 0;
      bool ok = true;
      auto load_q = [&](auto tc, uint32_t& q_cnt) -> bool {
        constexpr int t = decltype(tc)::value;
        if (q_cnt > 0 && !ptx::mbar_wait(&bars->q_empty[t], (q_cnt - 1) & 1)) return false;
        ++q_cnt;
        ptx::mbar_expect_tx(&bars->q_full[t], L::kTileBytes);
#pragma unroll
        for (int sub = 0; sub < L::kSub; ++sub)
          ptx::tma_load_3d(sQ + t * L::kTileBytes + sub * L::kSubBytes, &tmQ, &bars->q_full[t],
                           64 * sub, sg.w.head[t], sg.row0[t]);
        return true;
      };
      // The query rows are the caller's input, not the work of the kernel ahead: the Q tiles
      // of the first stretch are fetched before waiting for it.
      bool more_work = walk.next(g, sg);
      if (more_work) {
        if (sg.nblk[0] > 0) load_q(std::integral_constant<int, 0>{}, q_cnt0);
        if (sg.nblk[1] > 0) load_q(std::integral_constant<int, 1>{}, q_cnt1);
      }
      bool waited = false;
      if (status_set()) {
        // nothing to do, but the loads in flight must land before the CTA may exit
        if (q_cnt0 > 0 && !ptx::mbar_wait(&bars->q_full[0], 0)) ok = false;
        if (q_cnt1 > 0 && !ptx::mbar_wait(&bars->q_full[1], 0)) ok = false;
        more_work = false;
      }
      for (bool first = true; ok && more_work; first = false, more_work = walk.next(g, sg)) {
        if (!first) {
          if (sg.nblk[0] > 0) ok = load_q(std::integral_constant<int, 0>{}, q_cnt0);
          if (ok && sg.nblk[1] > 0) ok = load_q(std::integral_constant<int, 1>{}, q_cnt1);
          if (!ok) break;
        }
        const int nmax = max(sg.nblk[0], sg.nblk[1]);
        for (int jj = 0; jj < nmax && ok; ++jj, ++kv_it) {
          const int st = kv_it % kKvStages;
          const uint32_t ph = (uint32_t)(kv_it / kKvStages) & 1;
          if (!waited && (sg.kb_lo + jj + 1) * kKeyBlock > sg.seq_pos0) {
            ptx::griddep_wait();           // this block holds rows that kv_append is writing
            waited = true;
          }
          int page[2], rin[2];
          for (int hh = 0; hh < 2; ++hh) {
            const int pos = (sg.kb_lo + jj) * kKeyBlock + 64 * hh;
            const int slot = pos / g.page_tokens;
            page[hh] = slot < g.pages_per_seq
                           ? g.page_table[(size_t)sg.seq_id * g.pages_per_seq + slot] : 0;
            rin[hh] = pos % g.page_tokens;
          }
          if (kv_it >= kKvStages) ok = ptx::mbar_wait(&bars->k_empty[st], ph ^ 1);
          if (!ok) break;
          ptx::mbar_expect_tx(&bars->k_full[st], L::kTileBytes);
          for (int hh = 0; hh < 2; ++hh)
            for (int sub = 0; sub < L::kSub; ++sub)
              ptx::tma_load_4d(sK + st * L::kTileBytes + sub * L::kSubBytes + hh * 8192, &tmK,
                               &bars->k_full[st], 64 * sub, rin[hh], sg.w.kvh, page[hh]);
          if (kv_it >= kKvStages) ok = ptx::mbar_wait(&bars->v_empty[st], ph ^ 1);
          if (!ok) break;
          ptx::mbar_expect_tx(&bars->v_full[st], L::kTileBytes);
          for (int hh = 0; hh < 2; ++hh)
            for (int sub = 0; sub < L::kSub; ++sub)
              ptx::tma_load_4d(sV + st * L::kTileBytes + sub * L::kSubBytes + hh * 8192, &tmV,
                               &bars->v_full[st], 64 * sub, rin[hh], sg.w.kvh, page[hh]);
        }
      }
      if (!ok) *abort_flag = 1;
    } else if (warp == 1 && lane == 0) {
      // ---------------------------------------------------------------- MMA issuer: scores
      // S_t(j) = Q_t K(j)^T into the shared S columns, S_0(j), S_1(j), S_0(j+1), ...: each
      // once the scores before it (the other tile's) have been taken into registers by their
      // softmax warpgroup.  Nothing here depends on the PV products, which another thread
      // issues: a barrier wait of one (~100 cycles even when it has completed) falls under the
      // other's MMAs instead of leaving the tensor pipe idle.
      constexpr uint32_t idesc_qk = ptx::instr_desc_bf16(128, 128, 0, 0);
      // Descriptors are built once; a K step only adds a constant to the address field.
      const uint64_t dq0 = ptx::smem_desc_sw128(ptx::smem_u32(sQ), 16, 1024);
      const uint64_t dk0 = ptx::smem_desc_sw128(ptx::smem_u32(sK), 16, 1024);
      SegmentWalk<kBand, kCluster> walk(rec, cta, csize, crank);
      Segment sg;
      uint32_t kv_it = 0, q_cnt0 = 0, q_cnt1 = 0, n_qk = 0;
      bool ok = true;
      const bool skip = status_set();
      auto qk = [&](int t, uint32_t st_k) -> bool {
        if (n_qk > 0 && !ptx::mbar_wait(&bars->s_free, (n_qk - 1) & 1)) return false;
        ++n_qk;
        ptx::tc_fence_after();
        const uint64_t da = dq0 + (uint64_t)((t * L::kTileBytes) >> 4);
        const uint64_t db = dk0 + (uint64_t)((st_k * L::kTileBytes) >> 4);
        ptx::mma_ss_k64_first(tmem, da, db, idesc_qk);
        if (D == 128)      // second 64-column sub-tile of Q and K
          ptx::mma_ss_k64_acc(tmem, da + (L::kSubBytes >> 4), db + (L::kSubBytes >> 4), idesc_qk);
        ptx::mma_commit(&bars->s_ready[t]);
        return true;
      };
      while (ok && !skip && walk.next(g, sg)) {
        const int nb0 = sg.nblk[0], nb1 = sg.nblk[1];
        const int nmax = max(nb0, nb1);
        if (nmax == 0) continue;
        if (nb0 > 0) {
          ok = ptx::mbar_wait(&bars->q_full[0], q_cnt0 & 1);
          ++q_cnt0;
        }
        if (ok && nb1 > 0) {
          ok = ptx::mbar_wait(&bars->q_full[1], q_cnt1 & 1);
          ++q_cnt1;
        }
        for (int jj = 0; jj < nmax && ok; ++jj, ++kv_it) {
          const uint32_t st = kv_it % kKvStages;
          ok = ptx::mbar_wait(&bars->k_full[st], (kv_it / kKvStages) & 1);
          if (ok && jj < nb0) {
            ok = qk(0, st);
            if (jj + 1 == nb0) ptx::mma_commit(&bars->q_empty[0]);
          }
          if (ok && jj < nb1) {
            ok = qk(1, st);
            if (jj + 1 == nb1) ptx::mma_commit(&bars->q_empty[1]);
          }
          ptx::mma_commit(&bars->k_empty[st]);
        }
      }
      if (!ok) *abort_flag = 1;
    } else if (warp == 2 && lane == 0) {
      // ---------------------------------------------------------------- MMA issuer: PV products
      // O_t (+)= P_t(j) V(j), tile 0 then tile 1 for every key block, each as soon as its
      // softmax warpgroup has stored P_t(j).  tcgen05.commit covers the MMAs of the thread
      // that executes it, so pv_done / o_done / v_empty follow the PV products alone.
      constexpr uint32_t idesc_pv = ptx::instr_desc_bf16(128, D, 0, 1);
      const uint64_t dv0 = ptx::smem_desc_sw128(ptx::smem_u32(sV), L::kSubBytes, 1024);
      SegmentWalk<kBand, kCluster> walk(rec, cta, csize, crank);
      Segment sg;
      uint32_t kv_it = 0, blk0 = 0, blk1 = 0;
      bool ok = true;
      const bool skip = status_set();
      auto pv = [&](int t, uint32_t st_v, bool first, bool last, uint32_t& blk) -> bool {
        if (!ptx::mbar_wait(&bars->p_ready[t], blk & 1)) return false;
        ++blk;
        ptx::tc_fence_after();
        // keys 0-63 of the block, then keys 64-127
#pragma unroll
        for (int half = 0; half < 2; ++half)
          ptx::mma_ts_k64(tmem + 256 + 128 * t, tmem + 128 + 64 * t + half * 32,
                          dv0 + (uint64_t)((st_v * L::kTileBytes + half * 8192) >> 4), idesc_pv,
                          (first && half == 0) ? 0u : 1u);
        ptx::mma_commit(last ? &bars->o_done[t] : &bars->pv_done[t]);
        return true;
      };
      while (ok && !skip && walk.next(g, sg)) {
        const int nb0 = sg.nblk[0], nb1 = sg.nblk[1];
        const int nmax = max(nb0, nb1);
        for (int jj = 0; jj < nmax && ok; ++jj, ++kv_it) {
          const uint32_t st = kv_it % kKvStages;
          ok = ptx::mbar_wait(&bars->v_full[st], (kv_it / kKvStages) & 1);
          if (ok && jj < nb0) ok = pv(0, st, jj == 0, jj + 1 == nb0, blk0);
          if (ok && jj < nb1) ok = pv(1, st, jj == 0, jj + 1 == nb1, blk1);
          ptx::mma_commit(&bars->v_empty[st]);
        }
      }
      if (!ok) *abort_flag = 1;
    }
  } else {
    // ------------------------------------------------------------------ softmax + epilogue
    setmaxnreg_inc_softmax();
    const int t = (warp - 4) >> 2;                   // tile of this warpgroup
    const int wq = warp & 3;                         // TMEM lane quarter of this warp
    const int r = wq * 32 + lane;                    // row of the tile
    const uint32_t lane_base = (uint32_t)(wq * 32) << 16;
    const uint32_t tS = tmem + lane_base;                       // shared by the two tiles
    const uint32_t tP = tmem + 128 + 64 * t + lane_base;
    const uint32_t tO = tmem + 256 + 128 * t + lane_base;
    const float sl2 = g.scale * 1.4426950408889634f;
    uint64_t* const bar_s = &bars->s_ready[t];
    uint64_t* const bar_p = &bars->p_ready[t];
    SegmentWalk<kBand, kCluster> walk(rec, cta, csize, crank);
    Segment sg;
    int blk = 0, o_cnt = 0, pv_cnt = 0;
    bool ok = !status_set();     // (a skipped launch is not a failure: see below)
    const bool skipped = !ok;
    while (ok && walk.next(g, sg)) {
      const int p_tile = sg.p0[t];
      const int p_row = p_tile + r;
      const int n_blocks = sg.nblk[t];
      float m = -INFINITY, l = 0.f;
      for (int jj = 0; jj < n_blocks; ++jj, ++blk) {
        ok = ptx::mbar_wait(bar_s, (uint32_t)blk & 1);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        ptx::tc_fence_after();
        const int key0 = (sg.kb_lo + jj) * kKeyBlock;
        const bool need_mask = key0 + kKeyBlock - 1 > p_tile;    // a block on the diagonal
        // a block that starts below the band of the tile's last row (sliding window only)
        const bool need_band = kBand && key0 < p_tile + kTileRows - g.window;
        // The whole row of S (128 fp32) comes into registers with one wait.
        uint32_t s[128];
#pragma unroll
        for (int c4 = 0; c4 < 4; ++c4) ptx::tmem_ld32(tS + c4 * 32, s + c4 * 32);
        ptx::tmem_ld_wait();
        // the S columns may take the next scores (the other tile's, as a rule)
        ptx::tc_fence_before();
        ptx::mbar_arrive(&bars->s_free);
        if (need_mask) {     // only the block(s) on the diagonal: masked logits become -inf
          const int n_vis = min(kKeyBlock, p_row - key0 + 1);   // may be <= 0
#pragma unroll
          for (int c = 0; c < 128; ++c)
            if (c >= n_vis) s[c] = 0xff800000u;
        }
        if (need_band) {     // keys before p_row - window + 1 are out of the row's band
          const int n_lo = p_row - g.window + 1 - key0;         // may be <= 0 or >= 128
#pragma unroll
          for (int c = 0; c < 128; ++c)
            if (c < n_lo) s[c] = 0xff800000u;
        }
        float bm0 = -INFINITY, bm1 = -INFINITY;
#pragma unroll
        for (int c = 0; c < 128; c += 4) {
          bm0 = ptx::max3(bm0, __uint_as_float(s[c]), __uint_as_float(s[c + 1]));
          bm1 = ptx::max3(bm1, __uint_as_float(s[c + 2]), __uint_as_float(s[c + 3]));
        }
        const float bm = fmaxf(bm0, bm1);
        // Rescale only when the maximum grew by more than 2^8 in the exponent domain (the
        // stale maximum is carried into the final normalisation, so the result is exact).
        // A row that has seen no key yet has m = -inf; a share that starts on the diagonal
        // can leave it there for a whole block.
        const bool grow = bm > m && (m == -INFINITY || (bm - m) * sl2 > 8.f);
        // PV_t(j-1) was issued after this block's scores: it must have completed before O_t is
        // rescaled or P_t is overwritten.  The rescale (rare) waits here, the common path
        // only before the store of P, when the product has long finished.
        bool pv_waited = jj == 0;
        auto wait_pv = [&]() -> bool {
          if (pv_waited) return true;
          pv_waited = true;
          const bool got = ptx::mbar_wait(&bars->pv_done[t], (uint32_t)pv_cnt & 1);
          ++pv_cnt;
          ptx::tc_fence_after();
          return got;
        };
        if (__any_sync(0xffffffffu, grow)) {
          ok = __all_sync(0xffffffffu, wait_pv());
          if (!ok) break;
          const float m_new = fmaxf(m, bm);
          const float alpha = (m == -INFINITY) ? 0.f : ptx::ex2((m - m_new) * sl2);
          l *= alpha;
          m = m_new;
          if (jj > 0) {
#pragma unroll
            for (int c4 = 0; c4 < D / 32; ++c4) {
              uint32_t v[32];
              ptx::tmem_ld32(tO + c4 * 32, v);
              ptx::tmem_ld_wait();
#pragma unroll
              for (int c = 0; c < 32; ++c) v[c] = __float_as_uint(__uint_as_float(v[c]) * alpha);
              ptx::tmem_st32(tO + c4 * 32, v);
            }
          }
        }
        // P = exp2(s*c - m*c) with packed fp32x2 multiply-adds, row sum, bf16 pairs written
        // over the registers already consumed, then into the first 64 columns of S.
        const float m_fin = (m == -INFINITY) ? 0.f : m;      // all logits are -inf then
        const float2 sl2v = make_float2(sl2, sl2);
        const float2 nmb = make_float2(-m_fin * sl2, -m_fin * sl2);
        float2 ps0 = make_float2(0.f, 0.f), ps1 = make_float2(0.f, 0.f);
        // All of P is formed in registers first, then stored; one arrival hands the whole
        // block to the MMA thread.  Off the diagonal half of the exponentials
        // are evaluated with a polynomial on the FMA pipe (kPolyExp), because the MUFU unit
        // (16 ex2 per clock per SM) is as loaded as the tensor pipe here: 128x128 ex2 per
        // tile and key block take as long as the tile's two MMAs.  Diagonal blocks keep the
        // MUFU path so that masked logits (-inf) give exactly zero.
        auto exp_block = [&](auto poly_c) {
          constexpr bool kPoly = decltype(poly_c)::value;
#pragma unroll
          for (int half = 0; half < 2; ++half) {
#pragma unroll
            for (int c = 64 * half; c < 64 * half + 64; c += 4) {
              const float2 x0 = __ffma2_rn(
                  make_float2(__uint_as_float(s[c]), __uint_as_float(s[c + 1])), sl2v, nmb);
              const float2 x1 = __ffma2_rn(
                  make_float2(__uint_as_float(s[c + 2]), __uint_as_float(s[c + 3])), sl2v, nmb);
              const float2 e0 = make_float2(ptx::ex2(x0.x), ptx::ex2(x0.y));
              const float2 e1 = kPoly ? ptx::ex2_poly2(x1)
                                      : make_float2(ptx::ex2(x1.x), ptx::ex2(x1.y));
              ps0 = __fadd2_rn(ps0, e0);
              ps1 = __fadd2_rn(ps1, e1);
              __nv_bfloat162 b0 = __floats2bfloat162_rn(e0.x, e0.y);
              __nv_bfloat162 b1 = __floats2bfloat162_rn(e1.x, e1.y);
              s[c / 2] = *reinterpret_cast<uint32_t*>(&b0);
              s[c / 2 + 1] = *reinterpret_cast<uint32_t*>(&b1);
            }
          }
        };
        if (need_mask || need_band || !kPolyExp)
          exp_block(std::false_type{});
        else
          exp_block(std::true_type{});
        ok = __all_sync(0xffffffffu, wait_pv());
        if (!ok) break;
        ptx::tmem_st32(tP, s);
        ptx::tmem_st32(tP + 32, s + 32);
        ptx::tmem_st_wait();
        ptx::tc_fence_before();
        ptx::mbar_arrive(bar_p);
        l += (ps0.x + ps0.y) + (ps1.x + ps1.y);
      }
      if (kCluster) {
        // ---- cluster mode: merge the cluster's partial results of this pair -------------
        // Runs to the end even after a timed-out wait (the status word is raised below), so
        // that no CTA of the cluster is left waiting for this one.
        if (ok && n_blocks > 0) {
          ok = ptx::mbar_wait(&bars->o_done[t], (uint32_t)o_cnt & 1);
          ok = __all_sync(0xffffffffu, ok);
          ++o_cnt;
          ptx::tc_fence_after();
        }
        // Both warpgroups are past their last MMA: Q, K and V tiles in shared memory are dead
        // and carry the exports: O [column group of 4][row][4] fp32 over the K/V rings (a row's
        // 16-byte words of consecutive rows are consecutive), (max, sum) over Q.
        ptx::named_bar_sync(1, 256);
        float4* exp_o = reinterpret_cast<float4*>(sK) + (size_t)t * 128 * (D / 4);
        float2* exp_ml = reinterpret_cast<float2*>(sQ) + t * 128;
        // tcgen05.ld is warp-collective: whether O is read must not depend on the row
        const bool have_o = ok && n_blocks > 0;              // warp-uniform
        const bool have = have_o && l > 0.f;                 // this row saw at least one key
        // Every CTA of the cluster finishes some of the (tile, 32-column group) jobs: job
        // (t, c4) belongs to rank (t + 2*c4) mod csize, so the round trips to the peers' shared
        // memory that a merge costs are spread over the cluster (with two CTAs rank t finishes
        // all of tile t).  A warpgroup exports what other ranks finish, tells them, waits for
        // their exports, merges its own jobs, and leaves once nobody reads its export any more.
        auto owner = [&](int c4) { return (t + 2 * c4) % csize; };
        exp_ml[r] = make_float2(m, have ? l : 0.f);     // a row that saw no key: zero sum
        if (have_o) {
#pragma unroll
          for (int c4 = 0; c4 < D / 32; ++c4) {
            if (owner(c4) == crank) continue;           // warp-uniform
            uint32_t v[32];
            ptx::tmem_ld32(tO + c4 * 32, v);
            ptx::tmem_ld_wait();
#pragma unroll
            for (int c = 0; c < 32; c += 4)
              exp_o[(c4 * 8 + c / 4) * 128 + r] =
                  make_float4(__uint_as_float(v[c]), __uint_as_float(v[c + 1]),
                              __uint_as_float(v[c + 2]), __uint_as_float(v[c + 3]));
          }
        }
#pragma unroll 1
        for (int k = 0; k < csize; ++k)
          if (k != crank)
            ptx::mbar_arrive_remote(ptx::mapa(ptx::smem_u32(&bars->x_full[t]), (uint32_t)k));
        if (!ptx::mbar_wait_cluster(&bars->x_full[t], 0)) ok = false;
        ok = __all_sync(0xffffffffu, ok);
        bool any_job = false;
#pragma unroll
        for (int c4 = 0; c4 < D / 32; ++c4) any_job |= owner(c4) == crank;
        if (any_job) {
          const uint32_t ml_addr = ptx::smem_u32(exp_ml + r);
          const uint32_t o_addr = ptx::smem_u32(exp_o + r);
          // A load from another CTA's shared memory is a round trip of a few hundred
          // nanoseconds: every peer's (max, sum) of this row is fetched once, all peers at a
          // time, and kept as a weight (0 for a peer's row that saw no key).
          float pm[kMaxCluster], pl[kMaxCluster], pw[kMaxCluster];   // constant indices: registers
#pragma unroll
          for (int k = 0; k < kMaxCluster; ++k) {
            pm[k] = -INFINITY;
            pl[k] = 0.f;
            if (ok && k < csize && k != crank) {
              const float2 ml = ptx::ld_dsmem_f32x2(ptx::mapa(ml_addr, (uint32_t)k));
              pm[k] = ml.x;
              pl[k] = ml.y;
            }
          }
          float M = have ? m : -INFINITY;
#pragma unroll
          for (int k = 0; k < kMaxCluster; ++k)
            if (pl[k] > 0.f) M = fmaxf(M, pm[k]);
          const float w_own = have ? ptx::ex2((m - M) * sl2) : 0.f;
          float Lsum = w_own * l;
#pragma unroll
          for (int k = 0; k < kMaxCluster; ++k) {
            pw[k] = pl[k] > 0.f ? ptx::ex2((pm[k] - M) * sl2) : 0.f;
            Lsum = fmaf(pw[k], pl[k], Lsum);
          }
          const float inv = 1.f / Lsum;
          const bool valid = ok && r < sg.rows_valid[t];
          __nv_bfloat16* orow = out + ((size_t)(sg.row0[t] + r) * g.hq + sg.w.head[t]) * D;
#pragma unroll
          for (int c4 = 0; c4 < D / 32; ++c4) {
            if (owner(c4) != crank) continue;           // warp-uniform
            float acc[32];
            if (have_o) {
              uint32_t v[32];
              ptx::tmem_ld32(tO + c4 * 32, v);
              ptx::tmem_ld_wait();
#pragma unroll
              for (int c = 0; c < 32; ++c) acc[c] = w_own * __uint_as_float(v[c]);
            } else {
#pragma unroll
              for (int c = 0; c < 32; ++c) acc[c] = 0.f;
            }
            if (ok) {
#pragma unroll 1
              for (int k = 0; k < csize; ++k) {
                if (k == crank) continue;
                float wk = 0.f;
#pragma unroll
                for (int kk = 0; kk < kMaxCluster; ++kk) wk = kk == k ? pw[kk] : wk;
                if (wk > 0.f) {           // a peer's row that saw no key has no O to add
                  const uint32_t base = ptx::mapa(o_addr + (uint32_t)(c4 * 8) * 2048u, (uint32_t)k);
                  float4 pv[8];
#pragma unroll
                  for (int c = 0; c < 8; ++c) pv[c] = ptx::ld_dsmem_f32x4(base + (uint32_t)c * 2048u);
#pragma unroll
                  for (int c = 0; c < 8; ++c) {
                    acc[4 * c + 0] = fmaf(wk, pv[c].x, acc[4 * c + 0]);
                    acc[4 * c + 1] = fmaf(wk, pv[c].y, acc[4 * c + 1]);
                    acc[4 * c + 2] = fmaf(wk, pv[c].z, acc[4 * c + 2]);
                    acc[4 * c + 3] = fmaf(wk, pv[c].w, acc[4 * c + 3]);
                  }
                }
              }
            }
            uint4 wv[4];
            uint32_t* wp = reinterpret_cast<uint32_t*>(wv);
#pragma unroll
            for (int c = 0; c < 32; c += 2) {
              __nv_bfloat162 b = __floats2bfloat162_rn(acc[c] * inv, acc[c + 1] * inv);
              wp[c / 2] = *reinterpret_cast<uint32_t*>(&b);
            }
            if (valid) {
#pragma unroll
              for (int i = 0; i < 4; ++i) reinterpret_cast<uint4*>(orow + c4 * 32)[i] = wv[i];
            }
          }
          if (valid && owner(0) == crank)
            g.lse[(size_t)sg.w.head[t] * g.lse_ld + sg.row0[t] + r] = M * g.scale + __logf(Lsum);
        }
        // done reading the peers' exports; this CTA's own must outlive its readers
#pragma unroll 1
        for (int k = 0; k < csize; ++k)
          if (k != crank)
            ptx::mbar_arrive_remote(ptx::mapa(ptx::smem_u32(&bars->x_free[t]), (uint32_t)k));
        if (!ptx::mbar_wait_cluster(&bars->x_free[t], 0)) ok = false;
        if (!ok) break;
        continue;
      }
      if (!ok) break;
      const bool valid = r < sg.rows_valid[t];
      if (n_blocks > 0) {
        ok = ptx::mbar_wait(&bars->o_done[t], (uint32_t)o_cnt & 1);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        ++o_cnt;
        ptx::tc_fence_after();
        if (sg.full) {
          // final result: normalise, bf16, token-major output and the row's LSE
          const float inv = 1.f / l;
          __nv_bfloat16* orow = out + ((size_t)(sg.row0[t] + r) * g.hq + sg.w.head[t]) * D;
#pragma unroll
          for (int c4 = 0; c4 < D / 32; ++c4) {
            uint32_t v[32];
            ptx::tmem_ld32(tO + c4 * 32, v);
            ptx::tmem_ld_wait();
            uint4 wv[4];
            uint32_t* wp = reinterpret_cast<uint32_t*>(wv);
#pragma unroll
            for (int c = 0; c < 32; c += 2) {
              __nv_bfloat162 b = __floats2bfloat162_rn(__uint_as_float(v[c]) * inv,
                                                       __uint_as_float(v[c + 1]) * inv);
              wp[c / 2] = *reinterpret_cast<uint32_t*>(&b);
            }
            if (valid) {
#pragma unroll
              for (int i = 0; i < 4; ++i) reinterpret_cast<uint4*>(orow + c4 * 32)[i] = wv[i];
            }
          }
          if (valid)
            g.lse[(size_t)sg.w.head[t] * g.lse_ld + sg.row0[t] + r] = m * g.scale + __logf(l);
        } else {
          // partial result of a shared pair: O as it stands, with its max and row sum
          const size_t slot = (size_t)cta * 2 + sg.slot;
          float4* po = reinterpret_cast<float4*>(g.part_o + slot * part_o_floats(D)) +
                       (size_t)t * 128 * (D / 4);
#pragma unroll
          for (int c4 = 0; c4 < D / 32; ++c4) {
            uint32_t v[32];
            ptx::tmem_ld32(tO + c4 * 32, v);
            ptx::tmem_ld_wait();
#pragma unroll
            for (int c = 0; c < 32; c += 4)
              po[(size_t)(c4 * 8 + c / 4) * 128 + r] =
                  make_float4(__uint_as_float(v[c]), __uint_as_float(v[c + 1]),
                              __uint_as_float(v[c + 2]), __uint_as_float(v[c + 3]));
          }
          g.part_ml[slot * part_ml_elems() + t * 128 + r] = make_float2(m, l);
        }
      } else if (!sg.full && sg.w.active[t]) {
        // this tile has no key block in this share: an empty partial
        const size_t slot = (size_t)cta * 2 + sg.slot;
        g.part_ml[slot * part_ml_elems() + t * 128 + r] = make_float2(-INFINITY, 0.f);
      }
    }
    if (!ok && !skipped && lane == 0) *abort_flag = 1;
  }

  ptx::tc_fence_before();
  __syncthreads();
  if (tid == 0 && *abort_flag) atomicExch(g.dev_status, 5);
  // A CTA of a cluster must not leave while a peer may still read its shared memory (after a
  // wait that ran out the x_free hand-shake of the merge can be cut short).  Every wait in
  // this kernel is bounded, so every thread of every CTA of the cluster gets here.
  if (kCluster) ptx::cluster_sync_all();
  if (warp == 1) {
    __syncwarp();
    ptx::tc_fence_after();
    ptx::tmem_dealloc(tmem, 512);
  }
}

// Merges the partial results of the pairs whose key range was shared by several CTAs:
//   M = max_s m_s,  w_s = exp2((m_s - M) c),  O = sum_s w_s O_s / sum_s w_s l_s.
// One block per (shared pair, tile, group of 32 output columns); one thread per row; the
// partial O tiles are read with consecutive rows in consecutive 16-byte words.
template <int D>
__global__ void __launch_bounds__(128)
attn_combine_kernel(CacheGeom g, const void* __restrict__ rec, __nv_bfloat16* __restrict__ out) {
  ptx::griddep_launch_dependents();
  ptx::griddep_wait();                  // the partial results of the attention kernel
  const CallHeader* hdr = reinterpret_cast<const CallHeader*>(rec);
  const SeqDesc* descs = record_descs(rec);
  const SplitPair sp = reinterpret_cast<const SplitPair*>(
      reinterpret_cast<const char*>(rec) + hdr->split_off)[blockIdx.x >> 1];
  const int t = blockIdx.x & 1, r = threadIdx.x, cg = blockIdx.y;   // cg: 32-column group
  Segment sg;
  describe_pair(hdr, descs, g, sp.pair, sg);
  if (!sg.w.active[t] || r >= sg.rows_valid[t]) return;
  const float sl2 = g.scale * 1.4426950408889634f;
  auto slot_of = [&](int s) {
    return (size_t)(sp.cta_first + s) * 2 + (s == 0 ? sp.slot_first : 0);
  };
  // pass 1: maximum over the segments that saw a key, then weights and the row sum
  // Segments are taken four at a time with every load issued before its use and no branch
  // around a load (an empty segment gets weight 0; its slot holds finite stale values), so
  // that the L2 round trips of the segments overlap instead of adding up.
  // (two at a time when the pair has only two segments, by far the most common case: no slot
  // is then read twice)
  float M = -INFINITY;
  float Lsum = 0.f;
  float acc[32];
#pragma unroll
  for (int c = 0; c < 32; ++c) acc[c] = 0.f;
  auto merge = [&](auto width) {
    constexpr int U = decltype(width)::value;
    for (int s0 = 0; s0 < sp.n_seg; s0 += U) {
      float2 ml[U];
#pragma unroll
      for (int u = 0; u < U; ++u)
        ml[u] = g.part_ml[slot_of(min(s0 + u, sp.n_seg - 1)) * part_ml_elems() + t * 128 + r];
#pragma unroll
      for (int u = 0; u < U; ++u)
        if (ml[u].y > 0.f) M = fmaxf(M, ml[u].x);
    }
    for (int s0 = 0; s0 < sp.n_seg; s0 += U) {
      float2 ml[U];
      float4 v[U][8];
#pragma unroll
      for (int u = 0; u < U; ++u) {
        const size_t slot = slot_of(min(s0 + u, sp.n_seg - 1));
        ml[u] = g.part_ml[slot * part_ml_elems() + t * 128 + r];
        const float4* po = reinterpret_cast<const float4*>(g.part_o + slot * part_o_floats(D)) +
                           ((size_t)t * (D / 4) + cg * 8) * 128 + r;
#pragma unroll
        for (int c4 = 0; c4 < 8; ++c4) v[u][c4] = po[(size_t)c4 * 128];
      }
#pragma unroll
      for (int u = 0; u < U; ++u) {
        const bool live = s0 + u < sp.n_seg && ml[u].y > 0.f;
        const float wgt = live ? ptx::ex2((ml[u].x - M) * sl2) : 0.f;
        Lsum = fmaf(wgt, live ? ml[u].y : 0.f, Lsum);
#pragma unroll
        for (int c4 = 0; c4 < 8; ++c4) {
          acc[4 * c4 + 0] = fmaf(wgt, v[u][c4].x, acc[4 * c4 + 0]);
          acc[4 * c4 + 1] = fmaf(wgt, v[u][c4].y, acc[4 * c4 + 1]);
          acc[4 * c4 + 2] = fmaf(wgt, v[u][c4].z, acc[4 * c4 + 2]);
          acc[4 * c4 + 3] = fmaf(wgt, v[u][c4].w, acc[4 * c4 + 3]);
        }
      }
    }
  };
  if (sp.n_seg <= 2)
    merge(std::integral_constant<int, 2>{});
  else
    merge(std::integral_constant<int, 4>{});
  const float inv = 1.f / Lsum;
  __nv_bfloat16* orow =
      out + ((size_t)(sg.row0[t] + r) * g.hq + sg.w.head[t]) * D + cg * 32;
#pragma unroll
  for (int c8 = 0; c8 < 4; ++c8) {
    uint4 wv;
    uint32_t* wp = reinterpret_cast<uint32_t*>(&wv);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      __nv_bfloat162 b =
          __floats2bfloat162_rn(acc[8 * c8 + 2 * i] * inv, acc[8 * c8 + 2 * i + 1] * inv);
      wp[i] = *reinterpret_cast<uint32_t*>(&b);
    }
    reinterpret_cast<uint4*>(orow)[c8] = wv;
  }
  if (cg == 0)
    g.lse[(size_t)sg.w.head[t] * g.lse_ld + sg.row0[t] + r] = M * g.scale + __logf(Lsum);
}

// One-time set-up on the current device: checks the register split against the registers
// the block is launched with (128 control threads + 256 softmax threads against
// 384 x registers per thread; a split above that would wait forever) and raises the
// dynamic shared memory limit.
// max_clusters[c], c = 2..8: how many clusters of c CTAs the device runs at once (0 if none).
template <int D, bool kBand, bool kCluster, bool kRecInParam>
inline cudaError_t prepare_attn_tc_kernel() {
  cudaFuncAttributes fa;
  cudaError_t e = cudaFuncGetAttributes(&fa, fwd_attn_kernel<D, kBand, kCluster, kRecInParam>);
  if (e != cudaSuccess) return e;
  if (128 * kCtrlRegs + 256 * kSoftmaxRegs > kAttnThreads * fa.numRegs)
    return cudaErrorLaunchOutOfResources;
  return cudaFuncSetAttribute(fwd_attn_kernel<D, kBand, kCluster, kRecInParam>,
                              cudaFuncAttributeMaxDynamicSharedMemorySize, AttnSmem<D>::kBytes);
}
template <int D, bool kBand>
inline cudaError_t prepare_attn_tc_one(int* max_clusters) {
  cudaError_t e = prepare_attn_tc_kernel<D, kBand, false, false>();
  if (e == cudaSuccess) e = prepare_attn_tc_kernel<D, kBand, false, true>();
  if (e == cudaSuccess) e = prepare_attn_tc_kernel<D, kBand, true, false>();
  if (e == cudaSuccess) e = prepare_attn_tc_kernel<D, kBand, true, true>();
  if (e != cudaSuccess) return e;
  for (int c = 0; c <= kMaxCluster; ++c) max_clusters[c] = 0;
  for (int c = 2; c <= kMaxCluster; ++c) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(c * 64);
    cfg.blockDim = dim3(kAttnThreads);
    cfg.dynamicSmemBytes = AttnSmem<D>::kBytes;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = (unsigned)c;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, fwd_attn_kernel<D, kBand, true, true>, &cfg) == cudaSuccess)
      max_clusters[c] = n;
    else
      (void)cudaGetLastError();       // this cluster size is simply not used
  }
  return cudaSuccess;
}
inline cudaError_t prepare_attn_tc(int d, bool band, int* max_clusters) {
  if (d == 128)
    return band ? prepare_attn_tc_one<128, true>(max_clusters)
                : prepare_attn_tc_one<128, false>(max_clusters);
  return band ? prepare_attn_tc_one<64, true>(max_clusters)
              : prepare_attn_tc_one<64, false>(max_clusters);
}

// Launches the attention kernel over hdr.n_ctas CTAs.
inline cudaError_t launch_attn_tc(const CacheGeom& g, const void* rec_dev, const RecParam& recp,
                                  int rec_in_param, const CallHeader& hdr, const CUtensorMap& tmQ, const CUtensorMap& tmK,
                                  const CUtensorMap& tmV, __nv_bfloat16* out, cudaStream_t st) {
  if (hdr.n_ctas <= 0) return cudaSuccess;
  const bool band = g.window != kNoWindow;
  const int cl = hdr.cluster > 1 ? hdr.cluster : 1;
  auto go = [&](auto kernel, size_t smem) {
    return launch_pdl_cluster(kernel, cl, dim3(hdr.n_ctas), dim3(kAttnThreads), smem, st, g,
                              rec_dev, recp, tmQ, tmK, tmV, out);
  };
  auto pick = [&](auto dc, auto bandc, auto clc) {
    constexpr int kD = decltype(dc)::value;
    constexpr bool kB = decltype(bandc)::value, kC = decltype(clc)::value;
    return rec_in_param ? go(fwd_attn_kernel<kD, kB, kC, true>, AttnSmem<kD>::kBytes)
                        : go(fwd_attn_kernel<kD, kB, kC, false>, AttnSmem<kD>::kBytes);
  };
  using T = std::true_type;
  using F = std::false_type;
  using D128 = std::integral_constant<int, 128>;
  using D64 = std::integral_constant<int, 64>;
  if (g.d == 128) {
    if (cl > 1) return band ? pick(D128{}, T{}, T{}) : pick(D128{}, F{}, T{});
    return band ? pick(D128{}, T{}, F{}) : pick(D128{}, F{}, F{});
  }
  if (cl > 1) return band ? pick(D64{}, T{}, T{}) : pick(D64{}, F{}, T{});
  return band ? pick(D64{}, T{}, F{}) : pick(D64{}, F{}, F{});
}

// Merge of the pairs whose key range was shared (nothing to do if there are none).
inline cudaError_t launch_attn_combine(const CacheGeom& g, const void* rec_dev,
                                       const CallHeader& hdr, __nv_bfloat16* out,
                                       cudaStream_t st) {
  if (hdr.n_split <= 0) return cudaSuccess;
  if (g.d == 128)
    return launch_pdl(attn_combine_kernel<128>, dim3(2 * hdr.n_split, 4), dim3(128), 0, st, g,
                      rec_dev, out);
  else
    return launch_pdl(attn_combine_kernel<64>, dim3(2 * hdr.n_split, 2), dim3(128), 0, st, g,
                      rec_dev, out);
  return cudaGetLastError();
}

}  // namespace pdd
