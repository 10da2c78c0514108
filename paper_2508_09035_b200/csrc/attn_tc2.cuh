// fwd_attn2: the pair-of-CTAs form of the attention kernel (head_dim 128, plain causal).
//
// Work item = a QUAD: two tile pairs that read the same KV head on the same rows (four query
// heads of one GQA group), one pair per CTA of a two-CTA cluster.  Every MMA is issued once, by
// the leader CTA, for both CTAs (tcgen05 cta_group::2, M = 256: rows 0-127 are the leader's
// tile, rows 128-255 the peer's); each CTA stages only HALF of every K block (64 keys) and half
// of every V block (64 of the 128 head-dim columns), which is what leaves room for a full P tile
// per query tile in shared memory: both products take both operands from shared memory, the
// score columns S_t are private to their tile (TMEM: S_0 | S_1 | O_0 | O_1) and nothing is
// handed over between the tiles.
//   warp 0      TMA producer of the CTA's own Q tiles and K / V halves
//   warp 1      leader: issues the score MMAs (both CTAs: owns the TMEM allocation);
//               peer: relays "S_t read" of its softmax warpgroups to the leader
//   warp 2      leader: issues the PV MMAs; peer: relays "P_t stored"
//   warp 3      peer: relays "Q / K / V landed"
//   warps 4-7   softmax of tile 0 of this CTA, 8-11 of tile 1
// Barriers written by tcgen05.commit are multicast to both CTAs.  The softmax threads arrive on
// barriers of their own CTA; what the leader's issuing threads must know of the peer reaches
// them through one relay thread per kind of event, which waits on the peer's local barrier and
// arrives once on its twin in the leader through the cluster address space (128 softmax
// threads arriving there directly cost 12 % of the kernel's throughput).  All waits are bounded.
//
// Measured on B200 this kernel is slower than the one-CTA kernel (long-prompt workload: 977
// against 1200 TFLOP/s): S_t and P_t are single-buffered across the pair, so the two CTAs run
// in lock-step through relayed hand-overs, and the two tiles of a CTA do their exponentials at
// the same time.  It is never chosen by the cost model; pdd_set_schedule(kv, 4) selects it.
#pragma once
#include "attn_tc.cuh"

namespace pdd {

struct Attn2Smem {
  static constexpr int kSubBytes = 128 * 128;          // [128 rows][64 bf16] swizzled
  static constexpr int kQTile = 2 * kSubBytes;         // one 128 x 128 Q tile
  static constexpr int kKHalf = 2 * 8192;              // [64 keys][128 d]: two [64][64] sub-tiles
  static constexpr int kVHalf = kSubBytes;             // [128 keys][64 d]
  static constexpr int kPTile = 2 * kSubBytes;         // [128 rows][128 keys]
  static constexpr int kQOff = 0;
  static constexpr int kKOff = 2 * kQTile;
  static constexpr int kVOff = kKOff + kKvStages * kKHalf;
  static constexpr int kPOff = kVOff + kKvStages * kVHalf;
  static constexpr int kBarOff = kPOff + 2 * kPTile;
  static constexpr int kBytes = kBarOff + 1024 + 1024;
};

struct Attn2Bars {
  uint64_t q_full[2], k_full[kKvStages], v_full[kKvStages];        // local TMA
  uint64_t q_empty[2], k_empty[kKvStages], v_empty[kKvStages];     // commit, both CTAs
  uint64_t s_ready[2], pv_done[2], o_done[2];                      // commit, both CTAs
  uint64_t s_free[2], p_ready[2];                                  // local: 128 arrivals
  uint64_t peer_s_free[2], peer_p_ready[2];                        // leader: 1 arrival (relayed)
  uint64_t peer_q_full[2], peer_k_full[kKvStages], peer_v_full[kKvStages];   // leader: 1 arrival
  uint32_t tmem_base;
  int32_t abort_flag;
};

// Walk over the quads of a cluster's share; CTA `rank` describes pair 2 * quad + rank.
struct QuadWalk {
  const CallHeader* hdr;
  const SeqDesc* descs;
  CtaStart cs, ce;
  int quad, index, rank;
  __device__ __forceinline__ QuadWalk(const void* rec, int cluster_id, int rank_) {
    hdr = reinterpret_cast<const CallHeader*>(rec);
    descs = record_descs(rec);
    rank = rank_;
    index = 0;
    const CtaStart* st =
        reinterpret_cast<const CtaStart*>(reinterpret_cast<const char*>(rec) + hdr->cta_off);
    cs = st[cluster_id];
    ce = st[cluster_id + 1];
    quad = cs.pair;
  }
  __device__ __forceinline__ bool next(const CacheGeom& g, Segment& sg) {
    if (quad > ce.pair || 2 * quad >= hdr->n_pairs) return false;
    if (quad == ce.pair && ce.kb == 0) return false;
    describe_pair(hdr, descs, g, 2 * quad + rank, sg);
    const int nb = max(sg.n_kb[0], sg.n_kb[1]);
    sg.kb_lo = (quad == cs.pair) ? cs.kb : 0;
    sg.kb_hi = (quad == ce.pair) ? ce.kb : nb;
    sg.full = sg.kb_lo == 0 && sg.kb_hi == nb;
    sg.slot = index == 0 ? 0 : 1;
#pragma unroll
    for (int t = 0; t < 2; ++t) sg.nblk[t] = max(0, min(sg.kb_hi, sg.n_kb[t]) - sg.kb_lo);
    ++quad;
    ++index;
    return true;
  }
};

template <bool kRecInParam>
__global__ void __launch_bounds__(kAttnThreads, 1)
fwd_attn2_kernel(CacheGeom g, const void* __restrict__ rec_global,
                 const __grid_constant__ RecParam recp,
                 const __grid_constant__ CUtensorMap tmQ,
                 const __grid_constant__ CUtensorMap tmK,
                 const __grid_constant__ CUtensorMap tmV, __nv_bfloat16* __restrict__ out) {
  constexpr int D = 128;
  using L = Attn2Smem;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) &
                                             ~(uintptr_t)1023);
  uint8_t* sQ = base + L::kQOff;
  uint8_t* sK = base + L::kKOff;
  uint8_t* sV = base + L::kVOff;
  uint8_t* sP = base + L::kPOff;
  Attn2Bars* bars = reinterpret_cast<Attn2Bars*>(base + L::kBarOff);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int rank = (int)ptx::cluster_ctarank();
  const int cluster_id = blockIdx.x >> 1, n_clusters = gridDim.x >> 1;
  const int cta = rank * n_clusters + cluster_id;       // scratch slots: see the host schedule
  const bool leader = rank == 0;

  ptx::griddep_launch_dependents();
  if (tid == 0) {
    for (int t = 0; t < 2; ++t) {
      ptx::mbar_init(&bars->q_full[t], 1);
      ptx::mbar_init(&bars->q_empty[t], 1);
      ptx::mbar_init(&bars->s_ready[t], 1);
      ptx::mbar_init(&bars->pv_done[t], 1);
      ptx::mbar_init(&bars->o_done[t], 1);
      ptx::mbar_init(&bars->s_free[t], 128);
      ptx::mbar_init(&bars->p_ready[t], 128);
      ptx::mbar_init(&bars->peer_s_free[t], 1);
      ptx::mbar_init(&bars->peer_p_ready[t], 1);
      ptx::mbar_init(&bars->peer_q_full[t], 1);
    }
    for (int s = 0; s < kKvStages; ++s) {
      ptx::mbar_init(&bars->k_full[s], 1);
      ptx::mbar_init(&bars->k_empty[s], 1);
      ptx::mbar_init(&bars->v_full[s], 1);
      ptx::mbar_init(&bars->v_empty[s], 1);
      ptx::mbar_init(&bars->peer_k_full[s], 1);
      ptx::mbar_init(&bars->peer_v_full[s], 1);
    }
    bars->abort_flag = 0;
    ptx::fence_mbar_init();
  }
  if (warp == 1) {
    ptx::tmem_alloc2(&bars->tmem_base, 512);
    ptx::tmem_relinquish2();
  }
  const void* rec = kRecInParam ? reinterpret_cast<const void*>(&recp) : rec_global;
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  // the peer arrives on the leader's barriers and the leader's MMAs read the peer's shared
  // memory: both CTAs' barriers and TMEM must exist first
  ptx::cluster_sync_all();
  const uint32_t tmem = bars->tmem_base;
  volatile int32_t* abort_flag = &bars->abort_flag;
  auto status_set = [&]() -> bool {
    return *reinterpret_cast<volatile int32_t*>(g.dev_status) != 0;
  };
  // the leader's copy of a barrier, as a cluster address
  auto in_leader = [&](uint64_t* bar) -> uint32_t { return ptx::mapa(ptx::smem_u32(bar), 0u); };

  if (warp < 4) {
    setmaxnreg_dec_ctrl();
    if (warp == 0 && lane == 0) {
      // ---------------------------------------------------------------- producer (both CTAs)
      ptx::prefetch_tensormap(&tmQ);
      ptx::prefetch_tensormap(&tmK);
      ptx::prefetch_tensormap(&tmV);
      QuadWalk walk(rec, cluster_id, rank);
      Segment sg;
      int kv_it = 0;
      uint32_t q_cnt0 = 0, q_cnt1 = 0;
      bool ok = true;
      auto load_q = [&](auto tc, uint32_t& q_cnt) -> bool {
        constexpr int t = decltype(tc)::value;
        if (q_cnt > 0 && !ptx::mbar_wait(&bars->q_empty[t], (q_cnt - 1) & 1)) return false;
        ++q_cnt;
        ptx::mbar_expect_tx(&bars->q_full[t], L::kQTile);
#pragma unroll
        for (int sub = 0; sub < 2; ++sub)
          ptx::tma_load_3d(sQ + t * L::kQTile + sub * L::kSubBytes, &tmQ, &bars->q_full[t],
                           64 * sub, sg.w.head[t], sg.row0[t]);
        return true;
      };
      bool more_work = walk.next(g, sg);
      if (more_work) {
        if (sg.nblk[0] > 0) load_q(std::integral_constant<int, 0>{}, q_cnt0);
        if (sg.nblk[1] > 0) load_q(std::integral_constant<int, 1>{}, q_cnt1);
      }
      bool waited = false;
      if (status_set()) {
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
          // K: this CTA's 64 keys of the block, all of head_dim
          if (kv_it >= kKvStages) ok = ptx::mbar_wait(&bars->k_empty[st], ph ^ 1);
          if (!ok) break;
          ptx::mbar_expect_tx(&bars->k_full[st], L::kKHalf);
          for (int sub = 0; sub < 2; ++sub)
            ptx::tma_load_4d(sK + st * L::kKHalf + sub * 8192, &tmK, &bars->k_full[st], 64 * sub,
                             rin[rank], sg.w.kvh, page[rank]);
          // V: all 128 keys of the block, this CTA's 64 columns of head_dim
          if (kv_it >= kKvStages) ok = ptx::mbar_wait(&bars->v_empty[st], ph ^ 1);
          if (!ok) break;
          ptx::mbar_expect_tx(&bars->v_full[st], L::kVHalf);
          for (int hh = 0; hh < 2; ++hh)
            ptx::tma_load_4d(sV + st * L::kVHalf + hh * 8192, &tmV, &bars->v_full[st], 64 * rank,
                             rin[hh], sg.w.kvh, page[hh]);
        }
      }
      if (!ok) *abort_flag = 1;
    } else if (warp == 3 && lane == 0 && !leader) {
      // ---------------------------------------------------------------- peer: relay of "loaded"
      QuadWalk walk(rec, cluster_id, rank);
      Segment sg;
      uint32_t kv_it = 0, q_cnt0 = 0, q_cnt1 = 0;
      bool ok = true;
      const bool skip = status_set();
      while (ok && !skip && walk.next(g, sg)) {
        const int nmax = max(sg.nblk[0], sg.nblk[1]);
        if (nmax == 0) continue;
        if (sg.nblk[0] > 0) {
          ok = ptx::mbar_wait(&bars->q_full[0], q_cnt0 & 1);
          ++q_cnt0;
          ptx::mbar_arrive_remote(in_leader(&bars->peer_q_full[0]));
        }
        if (ok && sg.nblk[1] > 0) {
          ok = ptx::mbar_wait(&bars->q_full[1], q_cnt1 & 1);
          ++q_cnt1;
          ptx::mbar_arrive_remote(in_leader(&bars->peer_q_full[1]));
        }
        for (int jj = 0; jj < nmax && ok; ++jj, ++kv_it) {
          const uint32_t st = kv_it % kKvStages, ph = (kv_it / kKvStages) & 1;
          ok = ptx::mbar_wait(&bars->k_full[st], ph);
          if (!ok) break;
          ptx::mbar_arrive_remote(in_leader(&bars->peer_k_full[st]));
          ok = ptx::mbar_wait(&bars->v_full[st], ph);
          if (!ok) break;
          ptx::mbar_arrive_remote(in_leader(&bars->peer_v_full[st]));
        }
      }
      if (!ok) *abort_flag = 1;
    } else if ((warp == 1 || warp == 2) && lane < 2 && !leader) {
      // ---------------------------------------------------------------- peer: relay of the softmax
      // warpgroups' hand-offs (warp 1: "S_t read", warp 2: "P_t stored"; lane t for tile t), so
      // that no softmax thread pays for an arrival across the cluster network
      const int t = lane;
      uint64_t* const local = warp == 1 ? &bars->s_free[t] : &bars->p_ready[t];
      const uint32_t remote = in_leader(warp == 1 ? &bars->peer_s_free[t] : &bars->peer_p_ready[t]);
      QuadWalk walk(rec, cluster_id, rank);
      Segment sg;
      uint32_t n = 0;
      bool ok = true;
      const bool skip = status_set();
      while (ok && !skip && walk.next(g, sg)) {
        for (int jj = 0; jj < sg.nblk[t] && ok; ++jj, ++n) {
          ok = ptx::mbar_wait(local, n & 1);
          if (ok) ptx::mbar_arrive_remote(remote);
        }
      }
      if (!ok) *abort_flag = 1;
    } else if (warp == 1 && lane == 0 && leader) {
      // ---------------------------------------------------------------- leader: score MMAs
      constexpr uint32_t idesc_qk = ptx::instr_desc_bf16(256, 128, 0, 0);
      const uint64_t dq0 = ptx::smem_desc_sw128(ptx::smem_u32(sQ), 16, 1024);
      const uint64_t dk0 = ptx::smem_desc_sw128(ptx::smem_u32(sK), 16, 1024);
      QuadWalk walk(rec, cluster_id, rank);
      Segment sg;
      uint32_t kv_it = 0, q_cnt0 = 0, q_cnt1 = 0, n_qk[2] = {0, 0};
      bool ok = true;
      const bool skip = status_set();
      auto qk = [&](int t, uint32_t st_k) -> bool {
        // S_t (in both CTAs) may be overwritten once both softmax warpgroups have it in registers
        if (n_qk[t] > 0 && !(ptx::mbar_wait(&bars->s_free[t], (n_qk[t] - 1) & 1) &&
                             ptx::mbar_wait_cluster(&bars->peer_s_free[t], (n_qk[t] - 1) & 1)))
          return false;
        ++n_qk[t];
        ptx::tc_fence_after();
        const uint32_t tS = tmem + 128 * t;
        const uint64_t da = dq0 + (uint64_t)((t * L::kQTile) >> 4);
        const uint64_t db = dk0 + (uint64_t)((st_k * L::kKHalf) >> 4);
        ptx::mma2_ss_k64_first(tS, da, db, idesc_qk);
        ptx::mma2_ss_k64_acc(tS, da + (L::kSubBytes >> 4), db + (8192 >> 4), idesc_qk);
        ptx::mma2_commit_both(&bars->s_ready[t]);
        return true;
      };
      while (ok && !skip && walk.next(g, sg)) {
        const int nb0 = sg.nblk[0], nb1 = sg.nblk[1];
        const int nmax = max(nb0, nb1);
        if (nmax == 0) continue;
        if (nb0 > 0) {
          ok = ptx::mbar_wait(&bars->q_full[0], q_cnt0 & 1) &&
               ptx::mbar_wait_cluster(&bars->peer_q_full[0], q_cnt0 & 1);
          ++q_cnt0;
        }
        if (ok && nb1 > 0) {
          ok = ptx::mbar_wait(&bars->q_full[1], q_cnt1 & 1) &&
               ptx::mbar_wait_cluster(&bars->peer_q_full[1], q_cnt1 & 1);
          ++q_cnt1;
        }
        for (int jj = 0; jj < nmax && ok; ++jj, ++kv_it) {
          const uint32_t st = kv_it % kKvStages, ph = (kv_it / kKvStages) & 1;
          ok = ptx::mbar_wait(&bars->k_full[st], ph) && ptx::mbar_wait_cluster(&bars->peer_k_full[st], ph);
          if (ok && jj < nb0) {
            ok = qk(0, st);
            if (jj + 1 == nb0) ptx::mma2_commit_both(&bars->q_empty[0]);
          }
          if (ok && jj < nb1) {
            ok = qk(1, st);
            if (jj + 1 == nb1) ptx::mma2_commit_both(&bars->q_empty[1]);
          }
          ptx::mma2_commit_both(&bars->k_empty[st]);
        }
      }
      if (!ok) *abort_flag = 1;
    } else if (warp == 2 && lane == 0 && leader) {
      // ---------------------------------------------------------------- leader: PV MMAs
      constexpr uint32_t idesc_pv = ptx::instr_desc_bf16(256, 128, 0, 1);
      const uint64_t dv0 = ptx::smem_desc_sw128(ptx::smem_u32(sV), L::kSubBytes, 1024);
      const uint64_t dp0 = ptx::smem_desc_sw128(ptx::smem_u32(sP), 16, 1024);
      QuadWalk walk(rec, cluster_id, rank);
      Segment sg;
      uint32_t kv_it = 0, blk0 = 0, blk1 = 0;
      bool ok = true;
      const bool skip = status_set();
      auto pv = [&](int t, uint32_t st_v, bool first, bool last, uint32_t& blk) -> bool {
        if (!(ptx::mbar_wait(&bars->p_ready[t], blk & 1) &&
              ptx::mbar_wait_cluster(&bars->peer_p_ready[t], blk & 1)))
          return false;
        ++blk;
        ptx::tc_fence_after();
        // keys 0-63 of the block, then keys 64-127
#pragma unroll
        for (int half = 0; half < 2; ++half)
          ptx::mma2_ss_pv_k64(tmem + 256 + 128 * t,
                              dp0 + (uint64_t)((t * L::kPTile + half * L::kSubBytes) >> 4),
                              dv0 + (uint64_t)((st_v * L::kVHalf + half * 8192) >> 4), idesc_pv,
                              (first && half == 0) ? 0u : 1u);
        ptx::mma2_commit_both(last ? &bars->o_done[t] : &bars->pv_done[t]);
        return true;
      };
      while (ok && !skip && walk.next(g, sg)) {
        const int nb0 = sg.nblk[0], nb1 = sg.nblk[1];
        const int nmax = max(nb0, nb1);
        for (int jj = 0; jj < nmax && ok; ++jj, ++kv_it) {
          const uint32_t st = kv_it % kKvStages, ph = (kv_it / kKvStages) & 1;
          ok = ptx::mbar_wait(&bars->v_full[st], ph) && ptx::mbar_wait_cluster(&bars->peer_v_full[st], ph);
          if (ok && jj < nb0) ok = pv(0, st, jj == 0, jj + 1 == nb0, blk0);
          if (ok && jj < nb1) ok = pv(1, st, jj == 0, jj + 1 == nb1, blk1);
          ptx::mma2_commit_both(&bars->v_empty[st]);
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
    const uint32_t tS = tmem + 128 * t + lane_base;
    const uint32_t tO = tmem + 256 + 128 * t + lane_base;
    // this thread's row of the tile's P buffer: 128-byte swizzle, 8-row groups 1024 bytes apart
    const uint32_t p_row_addr = ptx::smem_u32(sP) + t * L::kPTile + (r >> 3) * 1024 + (r & 7) * 128;
    const float sl2 = g.scale * 1.4426950408889634f;
    uint64_t* const bar_s = &bars->s_ready[t];
    uint64_t* const bar_s_free = &bars->s_free[t];
    uint64_t* const bar_p = &bars->p_ready[t];
    QuadWalk walk(rec, cluster_id, rank);
    Segment sg;
    int blk = 0, o_cnt = 0, pv_cnt = 0;
    bool ok = !status_set();     // (a skipped launch is not a failure)
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
        uint32_t s[128];
#pragma unroll
        for (int c4 = 0; c4 < 4; ++c4) ptx::tmem_ld32(tS + c4 * 32, s + c4 * 32);
        ptx::tmem_ld_wait();
        // S_t may take the tile's next scores
        ptx::tc_fence_before();
        ptx::mbar_arrive(bar_s_free);
        if (need_mask) {     // only the block(s) on the diagonal: masked logits become -inf
          const int n_vis = min(kKeyBlock, p_row - key0 + 1);   // may be <= 0
#pragma unroll
          for (int c = 0; c < 128; ++c)
            if (c >= n_vis) s[c] = 0xff800000u;
        }
        float bm0 = -INFINITY, bm1 = -INFINITY;
#pragma unroll
        for (int c = 0; c < 128; c += 4) {
          bm0 = ptx::max3(bm0, __uint_as_float(s[c]), __uint_as_float(s[c + 1]));
          bm1 = ptx::max3(bm1, __uint_as_float(s[c + 2]), __uint_as_float(s[c + 3]));
        }
        const float bm = fmaxf(bm0, bm1);
        const bool grow = bm > m && (m == -INFINITY || (bm - m) * sl2 > 8.f);
        // PV_t(j-1) must have completed before O_t is rescaled or P_t is overwritten
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
            // the rescaled O must be in TMEM before the PV product that p_ready releases
            ptx::tmem_st_wait();
            ptx::tc_fence_before();
          }
        }
        const float m_fin = (m == -INFINITY) ? 0.f : m;      // all logits are -inf then
        const float2 sl2v = make_float2(sl2, sl2);
        const float2 nmb = make_float2(-m_fin * sl2, -m_fin * sl2);
        float2 ps0 = make_float2(0.f, 0.f), ps1 = make_float2(0.f, 0.f);
#pragma unroll
        for (int c = 0; c < 128; c += 4) {
          const float2 x0 = __ffma2_rn(
              make_float2(__uint_as_float(s[c]), __uint_as_float(s[c + 1])), sl2v, nmb);
          const float2 x1 = __ffma2_rn(
              make_float2(__uint_as_float(s[c + 2]), __uint_as_float(s[c + 3])), sl2v, nmb);
          const float2 e0 = make_float2(ptx::ex2(x0.x), ptx::ex2(x0.y));
          const float2 e1 = make_float2(ptx::ex2(x1.x), ptx::ex2(x1.y));
          ps0 = __fadd2_rn(ps0, e0);
          ps1 = __fadd2_rn(ps1, e1);
          __nv_bfloat162 b0 = __floats2bfloat162_rn(e0.x, e0.y);
          __nv_bfloat162 b1 = __floats2bfloat162_rn(e1.x, e1.y);
          s[c / 2] = *reinterpret_cast<uint32_t*>(&b0);
          s[c / 2 + 1] = *reinterpret_cast<uint32_t*>(&b1);
        }
        ok = __all_sync(0xffffffffu, wait_pv());
        if (!ok) break;
        // the row's 128 bf16 as sixteen 16-byte words (chunk c of a 64-key half at c ^ row % 8)
#pragma unroll
        for (int half = 0; half < 2; ++half)
#pragma unroll
          for (int c8 = 0; c8 < 8; ++c8)
            asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(
                             p_row_addr + (uint32_t)(half * L::kSubBytes) +
                             (uint32_t)((c8 ^ (r & 7)) << 4)),
                         "r"(s[32 * half + 4 * c8]), "r"(s[32 * half + 4 * c8 + 1]),
                         "r"(s[32 * half + 4 * c8 + 2]), "r"(s[32 * half + 4 * c8 + 3])
                         : "memory");
        ptx::fence_async_smem();         // generic-proxy stores before the MMA's async-proxy reads
        ptx::mbar_arrive(bar_p);
        l += (ps0.x + ps0.y) + (ps1.x + ps1.y);
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
        const size_t slot = (size_t)cta * 2 + sg.slot;
        g.part_ml[slot * part_ml_elems() + t * 128 + r] = make_float2(-INFINITY, 0.f);
      }
    }
    if (!ok && !skipped && lane == 0) *abort_flag = 1;
  }

  ptx::tc_fence_before();
  __syncthreads();
  if (tid == 0 && *abort_flag) atomicExch(g.dev_status, 5);
  // Neither CTA may leave while the other may still arrive on its barriers or while MMAs that
  // read its shared memory may be in flight.  Every wait is bounded: every thread gets here.
  ptx::cluster_sync_all();
  if (warp == 1) {
    __syncwarp();
    ptx::tc_fence_after();
    ptx::tmem_dealloc2(tmem, 512);
  }
}

inline cudaError_t prepare_attn_tc2(int* max_clusters2) {
  *max_clusters2 = 0;
  cudaFuncAttributes fa;
  cudaError_t e = cudaFuncGetAttributes(&fa, fwd_attn2_kernel<true>);
  if (e != cudaSuccess) return e;
  if (128 * kCtrlRegs + 256 * kSoftmaxRegs > kAttnThreads * fa.numRegs)
    return cudaErrorLaunchOutOfResources;
  e = cudaFuncSetAttribute(fwd_attn2_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           Attn2Smem::kBytes);
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(fwd_attn2_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             Attn2Smem::kBytes);
  if (e != cudaSuccess) return e;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(2 * 64);
  cfg.blockDim = dim3(kAttnThreads);
  cfg.dynamicSmemBytes = Attn2Smem::kBytes;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  int n = 0;
  if (cudaOccupancyMaxActiveClusters(&n, fwd_attn2_kernel<true>, &cfg) == cudaSuccess)
    *max_clusters2 = n;
  else
    (void)cudaGetLastError();
  return cudaSuccess;
}

inline cudaError_t launch_attn_tc2(const CacheGeom& g, const void* rec_dev, const RecParam& recp,
                                   int rec_in_param, const CallHeader& hdr, const CUtensorMap& tmQ,
                                   const CUtensorMap& tmK, const CUtensorMap& tmV,
                                   __nv_bfloat16* out, cudaStream_t st) {
  if (hdr.n_ctas <= 0) return cudaSuccess;
  if (rec_in_param)
    return launch_pdl_cluster(fwd_attn2_kernel<true>, 2, dim3(hdr.n_ctas), dim3(kAttnThreads),
                              Attn2Smem::kBytes, st, g, rec_dev, recp, tmQ, tmK, tmV, out);
  return launch_pdl_cluster(fwd_attn2_kernel<false>, 2, dim3(hdr.n_ctas), dim3(kAttnThreads),
                            Attn2Smem::kBytes, st, g, rec_dev, recp, tmQ, tmK, tmV, out);
}

}  // namespace pdd
