// 3x3 stride-1 convolution (forward and input gradient) on CTA pairs: tcgen05.mma with cta_group::2.
//
// Same GEMM view and the same "halo" operand scheme as conv_tc_kernel (one activation box with a one-pixel
// halo per 64-channel K chunk serves all nine taps), but two CTAs of a cluster work on one weight stage:
// every tcgen05.mma multiplies 256 rows -- a 128-pixel tile held by each CTA -- with the whole channel
// tile, of which each CTA fetches HALF (n_tile / 2 weight rows) with an ordinary TMA load into its own
// shared memory.  The instruction reads both halves, so the weight bytes that cross L2 -> SM per FLOP are
// halved without any multicast copy.  Why that matters: with pairs of tiles per CTA the one-CTA kernel
// moves 25 KB per weight stage for 640 cycles of tensor work, which is what an SM can draw from L2; a
// unit of fewer tiles (the last unit of most CTAs) costs as much as a full one because the 20 KB weight
// stage is the same.  Here a full unit is four tiles (two per CTA) on 10 KB of weights per CTA, and a
// half unit (one tile per CTA) costs about half of it.
//
// Protocol (rank 0 of the pair = leader):
//   * producers (warp 0 of both CTAs) wait on their own "empty" barriers and load into their own shared
//     memory; every load signals the LEADER's "full" barrier (cp.async.bulk.tensor ... cta_group::2 with
//     the barrier's cluster address), which the leader arms with the bytes of both CTAs;
//   * the leader's warps 1 and 2 issue the MMAs (one accumulator of the pair each, as in the one-CTA
//     kernel) and commit with multicast to the "empty" / "accumulator full" barriers of both CTAs;
//   * the epilogue warps of both CTAs drain their own 128 lanes of tensor memory and release the
//     accumulator slot on the leader's barrier (the peer's warps arrive remotely);
//   * cluster barriers separate barrier initialisation from the first remote signal and the last remote
//     signal from exit.
// Every mbarrier wait is bounded as in the one-CTA kernel.
#pragma once
#include "conv_tc.cuh"

namespace lp {
namespace tc {

__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
// Address of the same shared-memory object in CTA `rank` of the cluster (shared::cluster window).
__device__ __forceinline__ uint32_t mapa_u32(uint32_t local_addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(local_addr), "r"(rank));
  return r;
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// TMA loads into this CTA's shared memory whose completion is counted on a barrier given by its cluster
// address (the leader's barrier): the cta_group::2 form allows the barrier to live in the peer CTA.
__device__ __forceinline__ void tma2_load_2d(void* dst, const CUtensorMap* map, uint32_t bar_cluster_addr, int c0, int c1) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(smem_u32(dst)), "l"(map), "r"(bar_cluster_addr), "r"(c0), "r"(c1)
      : "memory");
}
__device__ __forceinline__ void tma2_load_4d(void* dst, const CUtensorMap* map, uint32_t bar_cluster_addr, int c0, int c1,
                                             int c2, int c3) {
  asm volatile(
      "cp.async.bulk.tensor.4d.cta_group::2.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
      ::"r"(smem_u32(dst)), "l"(map), "r"(bar_cluster_addr), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
      : "memory");
}
__device__ __forceinline__ void tmem2_alloc(uint32_t* smem_dst, uint32_t ncols) {  // one warp of EACH CTA of the pair
  asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(smem_dst)), "r"(ncols)
               : "memory");
}
__device__ __forceinline__ void tmem2_relinquish() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem2_dealloc(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
// D[tmem of both CTAs] (+)= A[128 rows in each CTA's smem] * B[half of the N rows in each CTA's smem]
__device__ __forceinline__ void mma2_bf16(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// Arrive on the barrier at this shared-memory offset in BOTH CTAs once the MMAs issued so far have completed.
__device__ __forceinline__ void mma2_commit_both(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
               ::"r"(smem_u32(bar)), "h"((uint16_t)3)
               : "memory");
}

// Tiles of one unit: up to four consecutive pixel tiles of one channel tile.  The leader takes the first
// `npair` of them (two when there are three or four, else one), the peer the rest.
struct Unit2 {
  int cnt, npair, mine, my_first;
};
__device__ __forceinline__ Unit2 unit2_at(int t, int t_end, int m_tiles, uint32_t rank) {
  Unit2 u;
  const int m = t % m_tiles;
  u.cnt = min(4, min(t_end - t, m_tiles - m));
  u.npair = u.cnt >= 3 ? 2 : 1;
  u.mine = rank == 0 ? u.npair : u.cnt - u.npair;
  u.my_first = rank == 0 ? t : t + u.npair;
  return u;
}

template <bool kAddend>
__global__ void __launch_bounds__(kConvThreads, 1)
conv_tc2_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                const __grid_constant__ ConvTcParams p) {
  extern __shared__ uint8_t smem_raw[];
  // the dynamic shared-memory window starts at the same offset in both CTAs, so the rounded-up offsets agree
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  TcSmemTail* tail = reinterpret_cast<TcSmemTail*>(smem + p.tail_offset);
  TcStatScratch* scratch = reinterpret_cast<TcStatScratch*>(smem + p.tail_offset + kTailBytes);
  volatile int* abort_flag = &tail->abort_flag;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();
  const bool leader = rank == 0;

  // contiguous tile range of this CTA pair
  const int pair_id = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;
  const int t_begin = (int)(((long long)p.total_tiles * pair_id) / n_pairs);
  const int t_end = (int)(((long long)p.total_tiles * (pair_id + 1)) / n_pairs);

  if (threadIdx.x == 0) {
    for (int s = 0; s < kMaxStages; ++s) {
      mbar_init(&tail->full[s], 1);      // leader: one arming arrival; bytes of both CTAs
      mbar_init(&tail->empty[s], 2);     // one (multicast) arrival per MMA warp of the leader
      mbar_init(&tail->full_b[s], 1);
      mbar_init(&tail->empty_b[s], 2);
    }
    for (int b = 0; b < kMaxSlots; ++b) {
      mbar_init(&tail->tmem_full[b], 1);
      mbar_init(&tail->tmem_empty[b], 2 * (kEpiThreads / 32));   // epilogue warps of both CTAs (leader's barrier)
    }
    mbar_init(&tail->add_full, 1);
    tail->abort_flag = 0;
    fence_barrier_init();
    prefetch_tmap(&tmA);
    prefetch_tmap(&tmB);
  }
  if (p.stats) {   // (without statistics the scratch is not part of the allocation)
    for (int i = threadIdx.x; i < LP_EPI_WARPS * 256; i += blockDim.x) {
      (&scratch->ssum[0][0])[i] = 0.f;
      (&scratch->ssq[0][0])[i] = 0.f;
    }
  }
  if (warp == kFirstEpiWarp) {
    tmem2_alloc(&tail->tmem_base, kTmemCols);
    tmem2_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();          // both CTAs' barriers exist before anything signals them from the other side
  tc_fence_after();
  pdl_wait();
  pdl_launch_dependents();
  const uint32_t tmem_base = tail->tmem_base;
  bool failed = false;

  if (warp == 0) {
    // ------------------------------- TMA producer (both CTAs) ---------------------------
    uint32_t sa = 0, pha = 0, sb = 0, phb = 0;
    uint8_t* b_ring = smem + p.b_ring_offset;
    const int n_half = p.n_tile_cols >> 1;
    for (int t = t_begin; t < t_end && !failed;) {
      const Unit2 u = unit2_at(t, t_end, p.m_tiles, rank);
      const int nt = t / p.m_tiles;
      int w0[2], h0[2], n0[2];
      for (int a = 0; a < 2; ++a) {
        const int mm = (u.my_first + a) % p.m_tiles;
        w0[a] = (mm % p.tiles_w) * p.BW;
        h0[a] = ((mm / p.tiles_w) % p.tiles_h) * p.BH;
        n0[a] = (mm / (p.tiles_w * p.tiles_h)) * p.BNI;
      }
      const int col0 = nt * p.n_tile_cols + (int)rank * n_half;   // this CTA's half of the weight rows
      for (int c = 0; c < p.chunks && !failed; ++c) {
        if (!mbar_wait_warp(&tail->empty[sa], pha ^ 1, abort_flag)) { failed = true; break; }
        uint8_t* pa = smem + sa * p.a_stage_bytes;
        if (elect_one()) {
          const uint32_t fb = mapa_u32(smem_u32(&tail->full[sa]), 0);
          if (leader) mbar_expect_tx(&tail->full[sa], (uint32_t)u.cnt * p.tx_a);
          for (int a = 0; a < u.mine; ++a)
            tma2_load_4d(pa + a * p.a_halo_bytes, &tmA, fb, c * p.KC, w0[a] - 1, n0[a], h0[a] - 1);
        }
        __syncwarp();
        if (++sa == (uint32_t)p.nA) { sa = 0; pha ^= 1; }
        for (int ti0 = 0; ti0 < 9; ti0 += p.tps) {      // a weight stage holds this CTA's half of p.tps taps
          const int n_taps = min(p.tps, 9 - ti0);
          if (!mbar_wait_warp(&tail->empty_b[sb], phb ^ 1, abort_flag)) { failed = true; break; }
          if (elect_one()) {
            const uint32_t fb = mapa_u32(smem_u32(&tail->full_b[sb]), 0);
            if (leader) mbar_expect_tx(&tail->full_b[sb], 2 * (uint32_t)n_taps * p.tx_b);
            for (int i = 0; i < n_taps; ++i)
              tma2_load_2d(b_ring + sb * p.b_stage_bytes + i * p.b_tile_bytes, &tmB, fb,
                           p.tap_widx9[ti0 + i] * p.Cin + c * p.KC, col0);
          }
          __syncwarp();
          if (++sb == (uint32_t)p.nB) { sb = 0; phb ^= 1; }
        }
      }
      t += u.cnt;
    }
  } else if ((warp == 1 || warp == 2) && leader) {
    // ------------------------------- MMA issuers (leader CTA only) ----------------------
    // Warp 1 owns the first accumulator of every unit, warp 2 the second one where the unit has two per
    // CTA.  Every "empty" barrier (of BOTH CTAs) takes two multicast commits per stage: one from each warp,
    // or both from warp 1 in a unit of one accumulator.
    const int me = warp - 1;
    uint32_t sa = 0, pha = 0, sb = 0, phb = 0;
    const uint32_t smem_base = smem_u32(smem);
    const int nk = p.KC >> 4;
    uint32_t slot = 0, slot_phase = 0;
    for (int t = t_begin; t < t_end && !failed;) {
      const Unit2 u = unit2_at(t, t_end, p.m_tiles, 0);
      uint32_t sl[2];
      sl[0] = slot;
      sl[1] = slot + 1 == (uint32_t)p.nslots ? 0 : slot + 1;
      const bool active = me < u.npair;
      if (!active) {
        // nothing for the second warp in a unit of one accumulator: it only advances its ring positions (a
        // second warp polling the barriers slowed the active one down), and the active warp signals twice
        const uint32_t tb = sb + (uint32_t)(p.chunks * ((9 + p.tps - 1) / p.tps)), ta = sa + (uint32_t)p.chunks;
        phb ^= (tb / (uint32_t)p.nB) & 1; sb = tb % (uint32_t)p.nB;
        pha ^= (ta / (uint32_t)p.nA) & 1; sa = ta % (uint32_t)p.nA;
        slot_phase ^= 1u << sl[0];
        slot = sl[1];
        t += u.cnt;
        continue;
      }
      const bool alone = u.npair == 1;
      if (!mbar_wait_warp(&tail->tmem_empty[sl[me]], ((slot_phase >> sl[me]) & 1) ^ 1, abort_flag)) { failed = true; break; }
      tc_fence_after();
      const uint32_t d = tmem_base + sl[me] * p.acc_stride;
      uint32_t accum = 0;
      for (int c = 0; c < p.chunks && !failed; ++c) {
        const uint32_t a_addr = smem_base + sa * p.a_stage_bytes + me * p.a_halo_bytes;
        const int nkc = c + 1 == p.chunks ? p.nk_last : nk;
        for (int ti0 = 0; ti0 < 9; ti0 += p.tps) {
          const int n_taps = min(p.tps, 9 - ti0);
          bool ok = ti0 ? true : mbar_wait(&tail->full[sa], pha, abort_flag);
          ok = mbar_wait(&tail->full_b[sb], phb, abort_flag) && ok;
          if (!__all_sync(0xffffffffu, ok)) { failed = true; break; }
          tc_fence_after();
          const uint32_t b_addr = smem_base + p.b_ring_offset + sb * p.b_stage_bytes;
          if (elect_one()) {
            for (int i = 0; i < n_taps; ++i) {
              const uint64_t ad = smem_desc(p.desc_hi_a, a_addr + p.tap_off9[ti0 + i]);
              const uint64_t bd = smem_desc(p.desc_hi, b_addr + i * p.b_tile_bytes);
              for (int j = 0; j < nkc; ++j)
                mma2_bf16(d, ad + (uint64_t)(2 * j), bd + (uint64_t)(2 * j), p.idesc, (accum | i | j) ? 1u : 0u);
            }
            mma2_commit_both(&tail->empty_b[sb]);
            if (alone) mma2_commit_both(&tail->empty_b[sb]);
            if (ti0 + n_taps == 9) {
              mma2_commit_both(&tail->empty[sa]);
              if (alone) mma2_commit_both(&tail->empty[sa]);
            }
          }
          __syncwarp();
          accum = 1;
          if (++sb == (uint32_t)p.nB) { sb = 0; phb ^= 1; }
        }
        if (failed) break;
        if (++sa == (uint32_t)p.nA) { sa = 0; pha ^= 1; }
      }
      if (failed) break;
      if (active && elect_one()) mma2_commit_both(&tail->tmem_full[sl[me]]);
      __syncwarp();
      for (int a = 0; a < u.npair; ++a) slot_phase ^= 1u << sl[a];
      slot = u.npair == 2 ? (sl[1] + 1 == (uint32_t)p.nslots ? 0 : sl[1] + 1) : sl[1];
      t += u.cnt;
    }
  } else if (warp >= kFirstEpiWarp) {
    // ------------------------------- epilogue (both CTAs, own 128 lanes of tensor memory) ----
    const int q = warp & 3;
    const int row = q * 32 + lane;
    const int et = threadIdx.x - 32 * kFirstEpiWarp;
    const int rows_used = p.BW * p.BH * p.BNI;
    const int ngroups = (p.n_tile_cols + 31) >> 5;
    uint32_t slot = 0, slot_phase = 0;
    int epi_turn = 0;
    for (int t = t_begin; t < t_end && !failed;) {
      const Unit2 u = unit2_at(t, t_end, p.m_tiles, rank);
      const int nt = t / p.m_tiles;
      const int col0 = nt * p.n_tile_cols;
      for (int a = 0; a < u.npair && !failed; ++a) {
        const bool have = a < u.mine;       // this CTA holds a real tile in accumulator `a` of the unit
        const int m = (u.my_first + a) % p.m_tiles;
        const uint32_t buf = slot;
        const int w0 = (m % p.tiles_w) * p.BW;
        const int h0 = ((m / p.tiles_w) % p.tiles_h) * p.BH;
        const int n0 = (m / (p.tiles_w * p.tiles_h)) * p.BNI;
        const int ow = w0 + row % p.BW;                 // rows of a tile: (w, image, h)
        const int oh = h0 + row / (p.BW * p.BNI);
        const int n = n0 + (row / p.BW) % p.BNI;
        const bool valid = have && row < rows_used && ow < p.OWl && oh < p.OHl && n < p.Nimg;
        const long long obase = (((long long)n * p.out_H + oh) * p.out_W + ow) * p.out_C;
        if (et == 0) tail->epi_ok[epi_turn] = mbar_wait(&tail->tmem_full[buf], (slot_phase >> buf) & 1, abort_flag) ? 1 : 0;
        asm volatile("bar.sync 1, %0;" ::"n"(kEpiThreads) : "memory");
        const int wait_ok = *(volatile int*)&tail->epi_ok[epi_turn];
        epi_turn ^= 1;
        if (!wait_ok) { failed = true; break; }
        tc_fence_after();
        const uint32_t taddr = tmem_base + buf * p.acc_stride + ((uint32_t)(q * 32) << 16);
        const uint32_t release_addr = mapa_u32(smem_u32(&tail->tmem_empty[buf]), 0);   // the leader's barrier
        constexpr int kBatch = LP_EPI_BATCH;
        auto load_addend = [&](int g, uint4 (&ad)[4]) {
          const int c_in_tile = g * 32;
          const int nv = c_in_tile + 32 <= p.n_tile_cols ? 4 : 2;
#pragma unroll
          for (int v4 = 0; v4 < 4; ++v4)
            ad[v4] = (g < ngroups && v4 < nv && valid && col0 + c_in_tile + 8 * v4 < p.Cout)
                         ? ld_raw(p.addend + obase + col0 + c_in_tile + 8 * v4) : make_uint4(0u, 0u, 0u, 0u);
        };
        if (!have) {   // nothing of this CTA in the accumulator: hand the slot back at once
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive_cluster(release_addr);
        }
        for (int g0 = 0; have && g0 < ngroups; g0 += kBatch) {
          uint32_t raw[kBatch][32];
          uint4 add_cur[4], add_next[4];
          if constexpr (kAddend) load_addend(g0, add_cur);
#pragma unroll
          for (int i = 0; i < kBatch; ++i) {
            const int g = g0 + i;
            if (g < ngroups) {
              if (g * 32 + 32 <= p.n_tile_cols) tmem_ld32_issue(taddr + g * 32, raw[i]);
              else tmem_ld16_issue(taddr + g * 32, raw[i]);
            }
          }
          tmem_ld_wait();
#pragma unroll
          for (int i = 0; i < kBatch; ++i) tmem_ld_fence(raw[i]);
          if (g0 + kBatch >= ngroups) {
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(release_addr);
          }
#pragma unroll
          for (int i = 0; i < kBatch; ++i) {
            const int g = g0 + i;
            if (g >= ngroups) continue;
            const int c_in_tile = g * 32;
            const int col = col0 + c_in_tile;
            const bool wide = c_in_tile + 32 <= p.n_tile_cols;
            const int nv = wide ? 4 : 2;
            float v[32];
#pragma unroll
            for (int j = 0; j < 32; ++j) v[j] = (wide || j < 16) ? __uint_as_float(raw[i][j]) : 0.f;
            if constexpr (kAddend) {
              if (i + 1 < kBatch) load_addend(g + 1, add_next);
#pragma unroll
              for (int v4 = 0; v4 < 4; ++v4) {
                float f[8];
                cvt_raw(add_cur[v4], f);
#pragma unroll
                for (int j = 0; j < 8; ++j) v[8 * v4 + j] += f[j];
                add_cur[v4] = add_next[v4];
              }
            }
            uint32_t pk[16];
#pragma unroll
            for (int j = 0; j < 16; ++j) pk[j] = pack_bf16x2(v[2 * j], v[2 * j + 1]);
            if (p.wide32) {
#pragma unroll
              for (int v2 = 0; v2 < 2; ++v2)
                if (2 * v2 < nv && valid && col + 16 * v2 < p.Cout) st_global_32B(p.out + obase + col + 16 * v2, &pk[8 * v2]);
            } else {
#pragma unroll
              for (int v4 = 0; v4 < 4; ++v4)
                if (v4 < nv && valid && col + 8 * v4 < p.Cout)
                  *reinterpret_cast<uint4*>(p.out + obase + col + 8 * v4) =
                      make_uint4(pk[4 * v4], pk[4 * v4 + 1], pk[4 * v4 + 2], pk[4 * v4 + 3]);
            }
            if (p.stats) {   // statistics of the tensor as stored, by a per-warp transposition (see conv_tc_kernel)
              uint32_t* T = scratch->tr[warp - kFirstEpiWarp];
#pragma unroll
              for (int j = 0; j < 16; ++j) T[j * 33 + lane] = (valid && (wide || j < 8)) ? pk[j] : 0u;
              __syncwarp();
              const int jc = lane & 15, hh = lane >> 4;
              const uint32_t* col_t = T + jc * 33 + hh * 16;
              float s0 = 0.f, s1 = 0.f, q0 = 0.f, q1 = 0.f;
#pragma unroll
              for (int r = 0; r < 16; ++r) {
                const uint32_t w2 = col_t[r];
                const float lo = __uint_as_float(w2 << 16), hi = __uint_as_float(w2 & 0xFFFF0000u);
                s0 += lo; s1 += hi;
                q0 = fmaf(lo, lo, q0); q1 = fmaf(hi, hi, q1);
              }
              __syncwarp();
              s0 += __shfl_xor_sync(0xffffffffu, s0, 16);
              s1 += __shfl_xor_sync(0xffffffffu, s1, 16);
              q0 += __shfl_xor_sync(0xffffffffu, q0, 16);
              q1 += __shfl_xor_sync(0xffffffffu, q1, 16);
              float* dst = hh ? scratch->ssq[warp - kFirstEpiWarp] : scratch->ssum[warp - kFirstEpiWarp];
              dst[c_in_tile + 2 * jc] += hh ? q0 : s0;
              dst[c_in_tile + 2 * jc + 1] += hh ? q1 : s1;
            }
          }
        }
        slot_phase ^= 1u << buf;
        slot = slot + 1 == (uint32_t)p.nslots ? 0 : slot + 1;
      }
      // flush the column sums when the channel tile is about to change (or at the very end)
      if (!failed && p.stats && (t + u.cnt >= t_end || (t + u.cnt) / p.m_tiles != nt)) {
        asm volatile("bar.sync 1, %0;" ::"n"(kEpiThreads) : "memory");
        for (int c = et; c < p.n_tile_cols; c += kEpiThreads) {
          float a_s = 0.f, a_q = 0.f;
          for (int wi = 0; wi < kEpiThreads / 32; ++wi) {
            a_s += scratch->ssum[wi][c];
            a_q += scratch->ssq[wi][c];
            scratch->ssum[wi][c] = 0.f;
            scratch->ssq[wi][c] = 0.f;
          }
          if (col0 + c < p.Cout) {
            atomicAdd(&p.stats[col0 + c], (double)a_s);
            atomicAdd(&p.stats[p.Cout + col0 + c], (double)a_q);
          }
        }
        asm volatile("bar.sync 1, %0;" ::"n"(kEpiThreads) : "memory");
      }
      t += u.cnt;
    }
  }

  if (failed) {
    *abort_flag = 1;
    atomicExch(p.err, 1);
    // let copies and MMAs already in flight land before shared / tensor memory is released
    for (int i = 0; i < 2000; ++i) __nanosleep(1000);
  }
  __syncwarp();
  tc_fence_before();
  __syncthreads();
  if (*abort_flag && !failed) {
    for (int i = 0; i < 2000; ++i) __nanosleep(1000);
  }
  // neither CTA leaves while the other may still signal its barriers or read its shared memory
  cluster_sync_all();
  if (warp == kFirstEpiWarp) {
    tc_fence_after();
    tmem2_dealloc(tmem_base, kTmemCols);
  }
}

}  // namespace tc
}  // namespace lp
