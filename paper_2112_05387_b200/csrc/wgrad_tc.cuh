// Weight gradient of a convolution on the tensor cores.
//
// dw[co][r][s][ci] = sum over output pixels of dy[pix][co] * x[pix shifted by (r,s)][ci].
// GEMM view: M = rows (tap, ci) in tiles of 128, N = output channels (tile <= 256), K = pixels.
// Both operands are stored pixel-major in memory (NHWC), i.e. MN-major for this product: a TMA
// box [pixels][SC channels] lands in shared memory as rows of SC*2 bytes (swizzled), which is the
// MN-major canonical layout with the 8-pixel group stride as SBO and the sub-box size as LBO.
// An M tile is made of 128/SC_A sub-boxes, each with its own tap shift and channel offset, so
// tiles stay full even when C_in is not a multiple of 128.  The pixel range is split over CTAs
// (split-K); partial sums are added to dw with fp32 atomics (dw is zeroed by the caller).
// A CTA computes two row tiles at once where there are at least two: both multiply the same dy
// stage, which cuts the L2 -> SM traffic per FLOP by about 30 %.
//
// 3x3 stride-1 convolutions with C_out tiles of at most 160 take wgrad_halo_kernel instead: the
// three taps of one kernel row read the same x pixels shifted by one pixel each, so ONE x box with
// a one-pixel halo in w serves all three (see that kernel), which halves the bytes per MMA.
//
// Roles (256 threads): warps 0 and 6 = TMA producers (x and dy), warps 1 and 7 = MMA issuers, warps 2..5 =
// epilogue.
#pragma once
#include <algorithm>

#include "common.cuh"
#include "tc_ptx.cuh"

namespace lp {
namespace tc {

constexpr int kWgMaxStages = 8;

// pixels per K block of wgrad_halo_kernel (128 or 64)
#ifndef LP_WGRAD_HALO_KBLOCK
#define LP_WGRAD_HALO_KBLOCK 128
#endif

struct WgradParams {
  int Nimg, OH, OW;
  int BW, BH, BNI, tiles_w, tiles_h, pix_tiles;
  int rows, rows_pad;            // pixels per K block, padded to a multiple of 16
  int stride, pad, R;
  int Cin, Cout, taps;
  int sca, rpt, cin_chunks, total_chunks, m_tiles;   // A: sub-box channels, sub-boxes per tile
  int scb, nb, n_tile, n_tiles;                      // B: sub-box channels, sub-boxes per tile
  int splits;
  int stages;
  int mpair, pair_tiles;                             // row tiles per CTA (1 or 2)
  uint32_t a_sub_bytes, b_sub_bytes, a_region, stage_bytes, tx_a, tx_b;
  uint32_t idesc;
  uint64_t adesc_hi, bdesc_hi;
  uint32_t tmem_cols;
  float* dw;
  int* err;
  // halo kernel (3x3, stride 1)
  int groups, acc_stride;        // (ci chunk, kernel row) groups; TMEM column stride of an accumulator
  uint32_t a_box_bytes;          // one x box: (8+2) x BNI x BH pixels x 64 channels
  uint32_t a_start3[3];          // first row of the three accumulators' A operands (bytes into the A region)
  uint64_t adesc_hi3[3];         // their descriptors (the leading byte offset differs)
  uint32_t a_kstep_bytes;        // 16 pixels further along K
  int epi_bufs;                  // 0: fp32 atomics; else number of 64-row staging buffers of the bulk-reduction epilogue
  uint32_t epi_buf_bytes;
};

struct WgSmemTail {
  uint64_t full[kWgMaxStages];
  uint64_t empty[kWgMaxStages];
  uint64_t acc_full;
  uint32_t tmem_base;
  int abort_flag;
  int epi_ok;
};

__global__ void __launch_bounds__(256, 1)
wgrad_tc_kernel(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmDY,
                const __grid_constant__ CUtensorMap tmDW, const __grid_constant__ WgradParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  WgSmemTail* tail = reinterpret_cast<WgSmemTail*>(smem + (size_t)p.stages * p.stage_bytes);
  volatile int* abort_flag = &tail->abort_flag;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int tile = blockIdx.x;
  const int m_tile = (tile % p.pair_tiles) * p.mpair, n_tile = tile / p.pair_tiles;
  const int cnt = (p.mpair == 2 && m_tile + 1 < p.m_tiles) ? 2 : 1;
  const int split = blockIdx.y;
  const int pt_begin = (int)(((long long)p.pix_tiles * split) / p.splits);
  const int pt_end = (int)(((long long)p.pix_tiles * (split + 1)) / p.splits);
  const int n_iter = pt_end - pt_begin;

  if (threadIdx.x == 0) {
    for (int s = 0; s < p.stages; ++s) {
      mbar_init(&tail->full[s], 2);    // one expect_tx arrival per producer warp
      mbar_init(&tail->empty[s], 2);   // one arrival per MMA warp
    }
    mbar_init(&tail->acc_full, 2);
    tail->abort_flag = 0;
    fence_barrier_init();
    prefetch_tmap(&tmX);
    prefetch_tmap(&tmDY);
  }
  // rows beyond the pixel box are never written by TMA: they must read as zero in the K dimension
  if (p.rows_pad > p.rows) {
    const int a_row_b = p.sca * 2, b_row_b = p.scb * 2;
    for (int s = 0; s < p.stages; ++s) {
      uint8_t* sa = smem + (size_t)s * p.stage_bytes;
      for (int j = 0; j < p.rpt * p.mpair; ++j) {
        uint8_t* base = sa + (size_t)j * p.a_sub_bytes + (size_t)p.rows * a_row_b;
        const int nbytes = (p.rows_pad - p.rows) * a_row_b;
        for (int i = threadIdx.x * 16; i < nbytes; i += blockDim.x * 16) *reinterpret_cast<uint4*>(base + i) = make_uint4(0, 0, 0, 0);
      }
      for (int j = 0; j < p.nb; ++j) {
        uint8_t* base = sa + p.a_region + (size_t)j * p.b_sub_bytes + (size_t)p.rows * b_row_b;
        const int nbytes = (p.rows_pad - p.rows) * b_row_b;
        for (int i = threadIdx.x * 16; i < nbytes; i += blockDim.x * 16) *reinterpret_cast<uint4*>(base + i) = make_uint4(0, 0, 0, 0);
      }
    }
    fence_proxy_async();
  }
  if (warp == 2) {
    tmem_alloc(&tail->tmem_base, p.tmem_cols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  pdl_wait();
  pdl_launch_dependents();
  const uint32_t tmem_base = tail->tmem_base;
  bool failed = false;

  if (warp == 0 || warp == 6) {
    // TMA producers: warp 0 copies the x sub-boxes, warp 6 the dy sub-boxes (a copy costs its
    // issuing thread about 100 cycles, and a stage has up to 11 of them for 16 MMAs); warp-uniform
    // loops, one elected lane issues
    const bool do_a = warp == 0;
    uint32_t s = 0, ph = 0;
    // Nothing in the loop divides: the pixel tile advances by one per iteration (its three coordinates are
    // counted up), and a sub-box's channel offset and tap shift do not depend on the iteration (lane j keeps
    // those of sub-box j and hands them to the issuing lane).  On layers of few channels the divide
    // instructions of 8 to 16 copies per stage were what the producer spent its time on.
    int tw, th, tn;
    {
      const int q1 = pt_begin / p.tiles_w;
      tw = pt_begin - q1 * p.tiles_w;
      tn = q1 / p.tiles_h;
      th = q1 - tn * p.tiles_h;
    }
    int my_c0 = 0, my_dw = 0, my_dh = 0;
    if (do_a && lane < p.rpt * cnt) {
      int g = m_tile * p.rpt + lane;
      if (g >= p.total_chunks) g = p.total_chunks - 1;  // padding rows of the last tile: any finite data
      const int tap = g / p.cin_chunks;
      my_c0 = (g - tap * p.cin_chunks) * p.sca;
      const int r = tap / p.R;
      my_dh = r - p.pad;
      my_dw = tap - r * p.R - p.pad;
    }
    for (int it = 0; it < n_iter; ++it) {
      const int w0 = tw * p.BW, h0 = th * p.BH, n0 = tn * p.BNI;
      if (++tw == p.tiles_w) { tw = 0; if (++th == p.tiles_h) { th = 0; ++tn; } }
      if (!mbar_wait_warp(&tail->empty[s], ph ^ 1, abort_flag)) { failed = true; break; }
      uint8_t* sa = smem + s * p.stage_bytes;
      const bool leader = elect_one();
      if (do_a) {
        if (leader) mbar_expect_tx(&tail->full[s], cnt * p.tx_a);
        for (int j = 0; j < p.rpt * cnt; ++j) {
          const int c0 = __shfl_sync(0xffffffffu, my_c0, j);
          const int dw = __shfl_sync(0xffffffffu, my_dw, j);
          const int dh = __shfl_sync(0xffffffffu, my_dh, j);
          if (leader)
            tma_load_4d(sa + j * p.a_sub_bytes, &tmX, &tail->full[s], c0, w0 * p.stride + dw, h0 * p.stride + dh, n0);
        }
      } else if (leader) {
        mbar_expect_tx(&tail->full[s], p.tx_b);
        for (int j = 0; j < p.nb; ++j)
          tma_load_4d(sa + p.a_region + j * p.b_sub_bytes, &tmDY, &tail->full[s], n_tile * p.n_tile + j * p.scb, w0,
                      h0, n0);
      }
      __syncwarp();
      if (++s == (uint32_t)p.stages) { s = 0; ph ^= 1; }
    }
  } else if (warp == 1 || warp == 7) {
    // Two MMA-issuing warps (one thread cannot keep the tensor pipe full): warp 1 owns the first row tile of
    // the CTA, warp 7 the second one of a pair.  Both wait for every stage and both arrive on its "empty"
    // barrier: with a commit after their MMAs, or (warp 7 with a single row tile) with a plain arrive.
    const bool active = warp == 1 || cnt == 2;
    const uint32_t acc_col = warp == 1 ? 0u : 256u;
    uint32_t s = 0, ph = 0;
    const uint32_t smem_base = smem_u32(smem);
    const int ksteps = p.rows_pad >> 4;
    const uint32_t a_kstep = (uint32_t)(16 * p.sca * 2) >> 4, b_kstep = (uint32_t)(16 * p.scb * 2) >> 4;
    for (int it = 0; it < n_iter; ++it) {
      if (!mbar_wait_warp(&tail->full[s], ph, abort_flag)) { failed = true; break; }
      tc_fence_after();
      const uint32_t a_addr = smem_base + s * p.stage_bytes;
      const uint64_t bd = smem_desc(p.bdesc_hi, a_addr + p.a_region);
      const uint64_t ad = smem_desc(p.adesc_hi, a_addr + (warp == 1 ? 0u : (uint32_t)(p.rpt * p.a_sub_bytes)));
      if (elect_one()) {
        if (active) {
          for (int j = 0; j < ksteps; ++j)
            mma_bf16(tmem_base + acc_col, ad + (uint64_t)(j * a_kstep), bd + (uint64_t)(j * b_kstep), p.idesc, (it | j) ? 1u : 0u);
          mma_commit(&tail->empty[s]);
        } else {
          mbar_arrive(&tail->empty[s]);
        }
      }
      __syncwarp();
      if (++s == (uint32_t)p.stages) { s = 0; ph ^= 1; }
    }
    if (!failed && n_iter > 0) {
      if (elect_one()) {
        if (active) mma_commit(&tail->acc_full);
        else mbar_arrive(&tail->acc_full);
      }
      __syncwarp();
    }
  } else {
    const int q = warp & 3;
    const int row = q * 32 + lane;
    const int et = threadIdx.x - 64;
    if (et == 0) tail->epi_ok = (n_iter > 0 && mbar_wait(&tail->acc_full, 0, abort_flag)) ? 1 : 0;
    asm volatile("bar.sync 1, 128;" ::: "memory");
    if (*(volatile int*)&tail->epi_ok && p.epi_bufs) {
      // Bulk-reduction epilogue (see wgrad_halo_kernel): an accumulator is transposed into its rpt
      // [channel-out][sca channel-in] fp32 tiles in the free operand ring, each added to dw by a TMA
      // reduction; the second accumulator of a pair reuses the buffers once they have been read.
      tc_fence_after();
      const int sub = row / p.sca, ci_l = row % p.sca;
      const int co0 = n_tile * p.n_tile;
      for (int a = 0; a < cnt; ++a) {
        if (a > 0) {
          if (et == 0) bulk_wait_read(0);
          asm volatile("bar.sync 1, 128;" ::: "memory");
        }
        float* buf = reinterpret_cast<float*>(smem + (size_t)sub * p.epi_buf_bytes);
        const uint32_t taddr = tmem_base + a * 256 + ((uint32_t)(q * 32) << 16);
        for (int cc = 0; cc < (p.n_tile >> 4); ++cc) {
          float v[16];
          tmem_ld16(taddr + cc * 16, v);
#pragma unroll
          for (int j = 0; j < 16; ++j) buf[(cc * 16 + j) * p.sca + ci_l] = v[j];
        }
        fence_proxy_async();
        asm volatile("bar.sync 1, 128;" ::: "memory");
        if (et == 0) {
          for (int sb = 0; sb < p.rpt; ++sb) {
            const int g = (m_tile + a) * p.rpt + sb;
            if (g < p.total_chunks)
              tma_reduce_add_3d(&tmDW, smem + (size_t)sb * p.epi_buf_bytes, (g % p.cin_chunks) * p.sca, g / p.cin_chunks, co0);
          }
          bulk_commit_group();
        }
      }
      if (et == 0) bulk_wait_read(0);
      tc_fence_before();
    } else if (*(volatile int*)&tail->epi_ok) {
      tc_fence_after();
      for (int a = 0; a < cnt; ++a) {
        const int g = (m_tile + a) * p.rpt + row / p.sca;
        const int ci_raw = (g % p.cin_chunks) * p.sca + row % p.sca;
        const bool valid = g < p.total_chunks && ci_raw < p.Cin;
        const int tap = valid ? g / p.cin_chunks : 0;
        const int ci = valid ? ci_raw : 0;
        const uint32_t taddr = tmem_base + a * 256 + ((uint32_t)(q * 32) << 16);
        const int co0 = n_tile * p.n_tile;
        for (int cc = 0; cc < (p.n_tile >> 4); ++cc) {
          float v[16];
          tmem_ld16(taddr + cc * 16, v);
          if (valid) {
#pragma unroll
            for (int j = 0; j < 16; ++j) {
              const int co = co0 + cc * 16 + j;
              if (co < p.Cout) atomicAdd(&p.dw[((long long)co * p.taps + tap) * p.Cin + ci], v[j]);
            }
          }
        }
      }
      tc_fence_before();
    } else if (n_iter > 0) {
      failed = true;
    }
  }

  if (failed) {
    *abort_flag = 1;
    atomicExch(p.err, 1);
    for (int i = 0; i < 2000; ++i) __nanosleep(1000);
  }
  __syncwarp();
  tc_fence_before();
  __syncthreads();
  if (*abort_flag && !failed) {
    for (int i = 0; i < 2000; ++i) __nanosleep(1000);
  }
  __syncthreads();
  if (warp == 2) {
    tc_fence_after();
    tmem_dealloc(tmem_base, p.tmem_cols);
  }
}

// ---------------------------------------------------------------------------------------------
// Weight gradient of a 3x3 stride-1 convolution with tap reuse.
//
// K block = 128 (or 64) output pixels: an 8 (w) x BH x BNI box, rows ordered (w, image, h) in both operands.
// A "group" is a 64-channel chunk of C_in together with one kernel row r; its three taps (s = 0,1,2)
// read x at pixels shifted by s - 1 in w.  The x box of a group is 10 pixels wide (halo of one on
// each side), so the operand of tap s is the same box started s rows (of 128 bytes) further on; an
// 8-pixel group of K is 8 consecutive box rows and the next one starts 10 rows later (SBO = 1280).
// As in the forward kernel this relies on the 128-byte swizzle being a function of the address
// bits.  A CTA holds two groups = six 64-row chunks = three 128-row accumulators in tensor memory:
//   acc 0 = (g0,s0),(g0,s1)   acc 1 = (g0,s2),(g1,s0)   acc 2 = (g1,s1),(g1,s2)
// The two chunks of an accumulator are the two 64-element M blocks of an MN-major operand; the
// descriptor's leading byte offset is the distance between their first rows: 128 bytes inside a
// box, (box size - 256) across the two boxes.  Per 128 pixels of K a CTA fetches x boxes of 40 KB and
// the dy tile (128 x n_tile) for 24 MMAs, against 6 sub-boxes (96 KB) without the reuse.
// Roles as in wgrad_tc_kernel, plus a second MMA-issuing warp (warp 7; 256 threads).
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256, 1)
wgrad_halo_kernel(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmDY,
                  const __grid_constant__ CUtensorMap tmDW, const __grid_constant__ WgradParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  WgSmemTail* tail = reinterpret_cast<WgSmemTail*>(smem + (size_t)p.stages * p.stage_bytes);
  volatile int* abort_flag = &tail->abort_flag;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int m_tile = blockIdx.x % p.m_tiles, n_tile = blockIdx.x / p.m_tiles;
  const int g0 = 2 * m_tile;                       // groups g0 and g0 + 1 (the second may not exist)
  const int split = blockIdx.y;
  const int pt_begin = (int)(((long long)p.pix_tiles * split) / p.splits);
  const int pt_end = (int)(((long long)p.pix_tiles * (split + 1)) / p.splits);
  const int n_iter = pt_end - pt_begin;

  if (threadIdx.x == 0) {
    for (int s = 0; s < p.stages; ++s) {
      mbar_init(&tail->full[s], 2);
      mbar_init(&tail->empty[s], 2);     // one commit per MMA-issuing warp
    }
    mbar_init(&tail->acc_full, 2);
    tail->abort_flag = 0;
    fence_barrier_init();
    prefetch_tmap(&tmX);
    prefetch_tmap(&tmDY);
  }
  if (warp == 2) {
    tmem_alloc(&tail->tmem_base, p.tmem_cols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  pdl_wait();
  pdl_launch_dependents();
  const uint32_t tmem_base = tail->tmem_base;
  bool failed = false;

  if (warp == 0 || warp == 6) {
    const bool do_a = warp == 0;
    uint32_t s = 0, ph = 0;
    int tw, th, tn;      // the pixel tile advances by one per iteration: its coordinates are counted up, not divided out
    {
      const int q1 = pt_begin / p.tiles_w;
      tw = pt_begin - q1 * p.tiles_w;
      tn = q1 / p.tiles_h;
      th = q1 - tn * p.tiles_h;
    }
    for (int it = 0; it < n_iter; ++it) {
      const int w0 = tw * 8, h0 = th * p.BH, n0 = tn * p.BNI;
      if (++tw == p.tiles_w) { tw = 0; if (++th == p.tiles_h) { th = 0; ++tn; } }
      if (!mbar_wait_warp(&tail->empty[s], ph ^ 1, abort_flag)) { failed = true; break; }
      uint8_t* sa = smem + s * p.stage_bytes;
      const bool leader = elect_one();
      if (leader && do_a) {
        mbar_expect_tx(&tail->full[s], 2 * p.tx_a);
        for (int j = 0; j < 2; ++j) {
          const int g = min(g0 + j, p.groups - 1);   // a missing second group: any finite data
          const int c0 = (g / 3) * 64, r = g % 3;
          tma_load_4d(sa + j * p.a_box_bytes, &tmX, &tail->full[s], c0, w0 - 1, n0, h0 + r - 1);
        }
      } else if (leader) {
        mbar_expect_tx(&tail->full[s], p.tx_b);
        for (int j = 0; j < p.nb; ++j)
          tma_load_4d(sa + p.a_region + j * p.b_sub_bytes, &tmDY, &tail->full[s], n_tile * p.n_tile + j * p.scb, w0,
                      n0, h0);
      }
      __syncwarp();
      if (++s == (uint32_t)p.stages) { s = 0; ph ^= 1; }
    }
  } else if (warp == 1 || warp == 7) {
    // Two MMA-issuing warps: a tcgen05.mma costs its issuing thread nearly as long as the tensor pipe works on
    // it, so one thread cannot keep the pipe full.  Warp 1 owns accumulators 0 and 1, warp 7 accumulator 2;
    // both wait for every stage and both commit on its "empty" barrier.
    const bool first = warp == 1;
    uint32_t s = 0, ph = 0;
    const uint32_t smem_base = smem_u32(smem);
    const uint32_t a_kstep = p.a_kstep_bytes >> 4, b_kstep = (uint32_t)(16 * p.scb * 2) >> 4;
    const int ksteps = p.rows >> 4;   // K = 16 pixels per MMA
    for (int it = 0; it < n_iter; ++it) {
      if (!mbar_wait_warp(&tail->full[s], ph, abort_flag)) { failed = true; break; }
      tc_fence_after();
      const uint32_t a_addr = smem_base + s * p.stage_bytes;
      const uint64_t bd = smem_desc(p.bdesc_hi, a_addr + p.a_region);
      const uint64_t ad0 = smem_desc(p.adesc_hi3[0], a_addr + p.a_start3[0]);
      const uint64_t ad1 = smem_desc(p.adesc_hi3[1], a_addr + p.a_start3[1]);
      const uint64_t ad2 = smem_desc(p.adesc_hi3[2], a_addr + p.a_start3[2]);
      if (elect_one()) {
#pragma unroll 1
        for (int j = 0; j < ksteps; ++j) {
          const uint32_t acc = (it | j) ? 1u : 0u;
          if (first) {
            mma_bf16(tmem_base, ad0 + (uint64_t)(j * a_kstep), bd + (uint64_t)(j * b_kstep), p.idesc, acc);
            mma_bf16(tmem_base + p.acc_stride, ad1 + (uint64_t)(j * a_kstep), bd + (uint64_t)(j * b_kstep), p.idesc, acc);
          } else {
            mma_bf16(tmem_base + 2 * p.acc_stride, ad2 + (uint64_t)(j * a_kstep), bd + (uint64_t)(j * b_kstep), p.idesc, acc);
          }
        }
        mma_commit(&tail->empty[s]);
      }
      __syncwarp();
      if (++s == (uint32_t)p.stages) { s = 0; ph ^= 1; }
    }
    if (!failed && n_iter > 0) {
      if (elect_one()) mma_commit(&tail->acc_full);
      __syncwarp();
    }
  } else {
    const int q = warp & 3;
    const int row = q * 32 + lane;
    const int et = threadIdx.x - 64;
    if (et == 0) tail->epi_ok = (n_iter > 0 && mbar_wait(&tail->acc_full, 0, abort_flag)) ? 1 : 0;
    asm volatile("bar.sync 1, 128;" ::: "memory");
    if (*(volatile int*)&tail->epi_ok && p.epi_bufs >= 2) {
      // Bulk-reduction epilogue.  The operand ring is free now (every MMA has completed); each
      // accumulator is transposed into two [channel-out][64 channel-in] fp32 tiles there, and one
      // thread adds each tile to dw with a TMA reduction (whole 256-byte rows, asynchronous), in
      // place of 61 440 scalar atomics per CTA.  Tiles of a later accumulator reuse a buffer once the
      // reduction that read it has finished reading.
      tc_fence_after();
      const int hh = q >> 1;                       // which 64-row chunk of the accumulator this warp holds
      const int ci_l = (q & 1) * 32 + lane;        // input channel within the chunk
      const int rounds_in_flight = p.epi_bufs >> 1;
      const int co0 = n_tile * p.n_tile;
      for (int a = 0; a < 3; ++a) {
        if (a >= rounds_in_flight) {
          if (et == 0) bulk_wait_read(rounds_in_flight - 1);
          asm volatile("bar.sync 1, 128;" ::: "memory");
        }
        const int slot = (a % rounds_in_flight) * 2;
        float* buf = reinterpret_cast<float*>(smem + (size_t)(slot + hh) * p.epi_buf_bytes);
        const uint32_t taddr = tmem_base + a * p.acc_stride + ((uint32_t)(q * 32) << 16);
        for (int cc = 0; cc < (p.n_tile >> 4); ++cc) {
          float v[16];
          tmem_ld16(taddr + cc * 16, v);
#pragma unroll
          for (int j = 0; j < 16; ++j) buf[(cc * 16 + j) * 64 + ci_l] = v[j];
        }
        fence_proxy_async();
        asm volatile("bar.sync 1, 128;" ::: "memory");
        if (et == 0) {
          for (int h2 = 0; h2 < 2; ++h2) {
            const int chunk = 2 * a + h2;
            const int g = g0 + chunk / 3, sx = chunk % 3;
            if (g < p.groups)
              tma_reduce_add_3d(&tmDW, smem + (size_t)(slot + h2) * p.epi_buf_bytes, (g / 3) * 64, (g % 3) * 3 + sx, co0);
          }
          bulk_commit_group();
        }
      }
      if (et == 0) bulk_wait_read(0);
      tc_fence_before();
    } else if (*(volatile int*)&tail->epi_ok) {
      tc_fence_after();
      for (int a = 0; a < 3; ++a) {
        const int chunk = 2 * a + (row >> 6);          // 0..5: group chunk/3, kernel column chunk%3
        const int g = g0 + chunk / 3, sx = chunk % 3;
        const int ci_raw = (g / 3) * 64 + (row & 63);
        const bool valid = g < p.groups && ci_raw < p.Cin;
        const int tap = valid ? (g % 3) * 3 + sx : 0;
        const int ci = valid ? ci_raw : 0;
        const uint32_t taddr = tmem_base + a * p.acc_stride + ((uint32_t)(q * 32) << 16);
        const int co0 = n_tile * p.n_tile;
        for (int cc = 0; cc < (p.n_tile >> 4); ++cc) {
          float v[16];
          tmem_ld16(taddr + cc * 16, v);
          if (valid) {
#pragma unroll
            for (int j = 0; j < 16; ++j) {
              const int co = co0 + cc * 16 + j;
              if (co < p.Cout) atomicAdd(&p.dw[((long long)co * 9 + tap) * p.Cin + ci], v[j]);
            }
          }
        }
      }
      tc_fence_before();
    } else if (n_iter > 0) {
      failed = true;
    }
  }

  if (failed) {
    *abort_flag = 1;
    atomicExch(p.err, 1);
    for (int i = 0; i < 2000; ++i) __nanosleep(1000);
  }
  __syncwarp();
  tc_fence_before();
  __syncthreads();
  if (*abort_flag && !failed) {
    for (int i = 0; i < 2000; ++i) __nanosleep(1000);
  }
  __syncthreads();
  if (warp == 2) {
    tc_fence_after();
    tmem_dealloc(tmem_base, p.tmem_cols);
  }
}

}  // namespace tc

typedef CUresult (*WgEncodeFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                               const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                               CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static int wg_encode(WgEncodeFn enc, CUtensorMap* m, const void* base, int N, int H, int W, int C, int boxC, int BW,
                     int BH, int BNI, int step) {
  cuuint64_t dims[4] = {(cuuint64_t)C, (cuuint64_t)W, (cuuint64_t)H, (cuuint64_t)N};
  cuuint64_t strides[3] = {(cuuint64_t)C * 2, (cuuint64_t)W * C * 2, (cuuint64_t)H * W * C * 2};
  cuuint32_t box[4] = {(cuuint32_t)boxC, (cuuint32_t)((BW - 1) * step + 1), (cuuint32_t)((BH - 1) * step + 1),
                       (cuuint32_t)BNI};
  cuuint32_t es[4] = {1, (cuuint32_t)step, (cuuint32_t)step, 1};
  const int row_bytes = boxC * 2;
  const CUtensorMapSwizzle sw = row_bytes == 128 ? CU_TENSOR_MAP_SWIZZLE_128B
                                : row_bytes == 64 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_32B;
  CUresult r = enc(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, es,
                   CU_TENSOR_MAP_INTERLEAVE_NONE, sw, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? 0 : -8;
}

// Tensor maps with the dimension order (C, W, image, H), as the halo kernel's boxes want them.
static int wg_encode_wnh(WgEncodeFn enc, CUtensorMap* m, const void* base, int N, int H, int W, int C, int boxC, int boxW,
                         int BNI, int BH) {
  cuuint64_t dims[4] = {(cuuint64_t)C, (cuuint64_t)W, (cuuint64_t)N, (cuuint64_t)H};
  cuuint64_t strides[3] = {(cuuint64_t)C * 2, (cuuint64_t)H * W * C * 2, (cuuint64_t)W * C * 2};
  cuuint32_t box[4] = {(cuuint32_t)boxC, (cuuint32_t)boxW, (cuuint32_t)BNI, (cuuint32_t)BH};
  cuuint32_t es[4] = {1, 1, 1, 1};
  const int row_bytes = boxC * 2;
  const CUtensorMapSwizzle sw = row_bytes == 128 ? CU_TENSOR_MAP_SWIZZLE_128B
                                : row_bytes == 64 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_32B;
  return enc(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, es,
             CU_TENSOR_MAP_INTERLEAVE_NONE, sw, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS ? 0 : -1;
}

// Returns 1 when the shape is not one the halo kernel takes (the caller then uses wgrad_tc_kernel).
// shared_sm: the launch is sized to share an SM with other kernels (tensor memory to need, at most
// kWgSharedSmem of shared memory) instead of taking the SM for itself; for small layers that several
// modules run at the same time.
static const size_t kWgSharedSmem = 100 * 1024;
static int launch_wgrad_halo(WgEncodeFn enc, int sm_count, bool* attr_done, const bf16* x, const bf16* dy, float* dw, int N, int H, int W,
                             int Cin, int Cout, int* dev_err, cudaStream_t st, bool shared_sm) {
  if (W % 8 || Cin < 64) return 1;
  tc::WgradParams p;
  memset(&p, 0, sizeof(p));
  p.Nimg = N; p.OH = H; p.OW = W; p.stride = 1; p.pad = 1; p.R = 3;
  p.Cin = Cin; p.Cout = Cout; p.taps = 9;
  // pixel box (K block): 8 x BH x BNI = LP_WGRAD_HALO_KBLOCK pixels.  Blocks of 64 make a stage 40 KB
  // instead of 80 KB for a 160-channel tile (five stages in flight instead of two); measured, that is
  // no faster (0.079 against 0.078 ms at 160 channels), so the copy latency is not what limits it.
  constexpr int per_col = LP_WGRAD_HALO_KBLOCK / 8;
  if (H >= per_col) { p.BH = per_col; p.BNI = 1; }
  else if (H == 8 || H == 4 || H == 2) { p.BH = H; p.BNI = per_col / H; }
  else return 1;
  if (p.BNI > N) return 1;
  p.BW = 8;
  p.tiles_w = W / 8;
  p.tiles_h = (H + p.BH - 1) / p.BH;
  p.pix_tiles = p.tiles_w * p.tiles_h * ((N + p.BNI - 1) / p.BNI);
  p.rows = p.rows_pad = LP_WGRAD_HALO_KBLOCK;
  // dy sub-boxes as in the plain kernel, one channel tile of at most 160 so that three accumulators fit
  int best_tile = 0;
  for (int sc : {64, 32, 16}) {
    if (Cout % sc && sc != 16) continue;
    const int chunks = (Cout + sc - 1) / sc;
    int nb = 1;
    for (int d = 1; d <= chunks && d * sc <= 160; ++d)
      if (chunks % d == 0) nb = d;
    if (nb * sc > best_tile) { best_tile = nb * sc; p.scb = sc; p.nb = nb; }
  }
  if (best_tile < 64) return 1;
  p.n_tile = best_tile;
  p.n_tiles = (Cout + p.n_tile - 1) / p.n_tile;
  p.acc_stride = (p.n_tile + 31) / 32 * 32;
  if (3 * p.acc_stride > 512) return 1;
  p.tmem_cols = 512;
  if (shared_sm) {
    p.tmem_cols = 32;
    while ((int)p.tmem_cols < 3 * p.acc_stride) p.tmem_cols *= 2;
  }
  const size_t max_smem = shared_sm ? kWgSharedSmem : (size_t)220 * 1024;
  p.cin_chunks = (Cin + 63) / 64;
  p.groups = 3 * p.cin_chunks;
  p.m_tiles = (p.groups + 1) / 2;
  const int box_rows = 10 * p.BNI * p.BH;
  p.a_box_bytes = (uint32_t)(box_rows * 128);
  p.a_region = 2 * p.a_box_bytes;
  p.b_sub_bytes = (uint32_t)((p.rows * p.scb * 2 + 1023) / 1024 * 1024);
  p.stage_bytes = p.a_region + p.b_sub_bytes * p.nb;
  p.tx_a = p.a_box_bytes;
  p.tx_b = (uint32_t)(p.rows * p.nb * p.scb * 2);
  const size_t tail = sizeof(tc::WgSmemTail) + 1024;
  int stages = (int)((max_smem - tail) / p.stage_bytes);
  stages = std::min(stages, tc::kWgMaxStages);
  if (stages < 2) return 1;
  p.stages = stages;
  // A operands: rows of 128 bytes; an 8-pixel K group is 8 rows, the next group 10 rows further
  const uint32_t sbo = 10 * 128;
  const uint32_t lbo_in = 128, lbo_across = p.a_box_bytes - 2 * 128;
  p.a_start3[0] = 0;                p.adesc_hi3[0] = tc::smem_desc_hi(lbo_in, sbo, 2);
  p.a_start3[1] = 2 * 128;          p.adesc_hi3[1] = tc::smem_desc_hi(lbo_across, sbo, 2);
  p.a_start3[2] = p.a_box_bytes + 128; p.adesc_hi3[2] = tc::smem_desc_hi(lbo_in, sbo, 2);
  p.a_kstep_bytes = 2 * sbo;                             // 16 pixels = two groups
  p.bdesc_hi = tc::smem_desc_hi(p.b_sub_bytes, 8 * p.scb * 2, tc::swizzle_code_for_row_bytes(p.scb * 2));
  p.idesc = tc::instr_desc_bf16(128, p.n_tile, 1, 1);
  const int tiles = p.m_tiles * p.n_tiles;
  {
    int best_s = 1;
    double best_t = 1e30;
    const int max_s = std::min(p.pix_tiles, 64);
    for (int sp = 1; sp <= max_s; ++sp) {
      const int waves = (tiles * sp + sm_count - 1) / sm_count;
      const double t = waves * ((double)((p.pix_tiles + sp - 1) / sp) * 1.5 * (p.rows / 128.0) + 4.0);
      if (t < best_t - 1e-9) { best_t = t; best_s = sp; }
    }
    p.splits = best_s;
  }
  p.dw = dw; p.err = dev_err;
  CUtensorMap tmX, tmDY;
  if (wg_encode_wnh(enc, &tmX, x, N, H, W, Cin, 64, 10, p.BNI, p.BH)) return -8;
  if (wg_encode_wnh(enc, &tmDY, dy, N, H, W, Cout, p.scb, 8, p.BNI, p.BH)) return -8;
  // dw as a (C_in, tap, C_out) fp32 tensor for the bulk-reduction epilogue: boxes of 64 input channels
  // of one tap and the CTA's output channels; staged in the operand ring after the main loop
  CUtensorMap tmDW;
  memset(&tmDW, 0, sizeof(tmDW));
  p.epi_buf_bytes = (uint32_t)(p.n_tile * 64 * 4);
  p.epi_bufs = 0;
  {
    cuuint64_t dims[3] = {(cuuint64_t)Cin, 9, (cuuint64_t)Cout};
    cuuint64_t strides[2] = {(cuuint64_t)Cin * 4, (cuuint64_t)Cin * 9 * 4};
    cuuint32_t box[3] = {64, 1, (cuuint32_t)p.n_tile};
    cuuint32_t es[3] = {1, 1, 1};
    const int fit = (int)std::min<size_t>(6, ((size_t)stages * p.stage_bytes) / p.epi_buf_bytes);
    if (fit >= 2 && (reinterpret_cast<uintptr_t>(dw) & 15) == 0 && Cin % 4 == 0 &&
        enc(&tmDW, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, dw, dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
            CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS)
      p.epi_bufs = fit & ~1;
  }
  size_t smem = (size_t)stages * p.stage_bytes + tail;
  if (!shared_sm) smem = std::max(smem, (size_t)120 * 1024);   // one CTA, and one owner of all tensor memory, per SM
  if (!*attr_done) {   // per device
    if (cudaFuncSetAttribute(tc::wgrad_halo_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 220 * 1024) != cudaSuccess)
      return -8;
    *attr_done = true;
  }
  dim3 grid(tiles, p.splits);
  return launch_pdl(tc::wgrad_halo_kernel, grid, dim3(256), smem, st, tmX, tmDY, tmDW, p) == cudaSuccess ? 0 : -8;
}

static int launch_wgrad_tc(WgEncodeFn enc, int sm_count, bool* attr_done, bool* halo_attr_done, const bf16* x,
                           const bf16* dy, float* dw, int N, int H, int W, int Cin, int OH, int OW, int Cout, int R,
                           int stride, int pad, int* dev_err, cudaStream_t st, bool shared_sm = false) {
  if (R == 3 && stride == 1 && pad == 1) {
    const int rc = launch_wgrad_halo(enc, sm_count, halo_attr_done, x, dy, dw, N, H, W, Cin, Cout, dev_err, st, shared_sm);
    if (rc != 1) return rc;
  }
  const size_t max_smem = shared_sm ? kWgSharedSmem : (size_t)220 * 1024;
  tc::WgradParams p;
  memset(&p, 0, sizeof(p));
  p.Nimg = N; p.OH = OH; p.OW = OW;
  p.stride = stride; p.pad = pad; p.R = R;
  p.Cin = Cin; p.Cout = Cout; p.taps = R * R;
  // sub-box width of x: the widest that divides C_in; otherwise 16 with zero fill past the last
  // channel (C_in = 40: chunks 0-15, 16-31, 32-47)
  p.sca = Cin % 64 == 0 ? 64 : (Cin % 32 == 0 ? 32 : 16);
  p.rpt = 128 / p.sca;
  p.cin_chunks = (Cin + p.sca - 1) / p.sca;
  p.total_chunks = p.taps * p.cin_chunks;
  p.m_tiles = (p.total_chunks + p.rpt - 1) / p.rpt;
  int best_tile = 0;
  for (int sc : {64, 32, 16}) {
    // 16-channel sub-boxes also serve a C_out that is only a multiple of 8: the last sub-box is
    // half zero fill (C_out = 40: 32 + 16) and the epilogue skips the channels past C_out
    if (Cout % sc && sc != 16) continue;
    const int chunks = (Cout + sc - 1) / sc;
    int nb = 1;
    for (int d = 1; d <= chunks && d * sc <= 256; ++d)
      if (chunks % d == 0) nb = d;
    if (nb * sc > best_tile) { best_tile = nb * sc; p.scb = sc; p.nb = nb; }
  }
  if (!best_tile) return -10;
  p.n_tile = best_tile;
  p.n_tiles = (Cout + p.n_tile - 1) / p.n_tile;
  // two row tiles per CTA pay off with 64-channel sub-boxes (few, large copies per stage); with
  // narrower sub-boxes the two pipeline stages that still fit do not hide the copy latency
  p.mpair = (p.m_tiles >= 2 && p.sca == 64 && !shared_sm) ? 2 : 1;
  p.pair_tiles = (p.m_tiles + p.mpair - 1) / p.mpair;
  const size_t tail = sizeof(tc::WgSmemTail) + 1024;
  // pixel box (K block): 128 output pixels, or 64 where three stages of 128 would not fit
  int target_rows = 128;
  if ((max_smem - tail) / ((size_t)128 * 2 * (p.mpair * 128 + p.n_tile)) < 2) target_rows = 64;
  p.BW = std::min(OW, target_rows);
  int bh = std::min(std::max(1, target_rows / p.BW), OH);
  const int th = (OH + bh - 1) / bh;
  p.BH = (OH + th - 1) / th;
  int bn = std::min(std::max(1, target_rows / (p.BW * p.BH)), N);
  const int tn = (N + bn - 1) / bn;
  p.BNI = (N + tn - 1) / tn;
  p.tiles_w = (OW + p.BW - 1) / p.BW;
  p.tiles_h = (OH + p.BH - 1) / p.BH;
  p.pix_tiles = p.tiles_w * p.tiles_h * ((N + p.BNI - 1) / p.BNI);
  p.rows = p.BW * p.BH * p.BNI;
  p.rows_pad = (p.rows + 15) / 16 * 16;
  const int tiles = p.pair_tiles * p.n_tiles;
  // split the pixel range so that the CTAs fill whole waves of SMs: time ~ waves x (K blocks per
  // CTA + fixed prologue/epilogue worth about 4 K blocks)
  {
    int best_s = 1;
    double best_t = 1e30;
    const int max_s = std::min(p.pix_tiles, 64);
    for (int sp = 1; sp <= max_s; ++sp) {
      const int waves = (tiles * sp + sm_count - 1) / sm_count;
      const double t = waves * ((double)((p.pix_tiles + sp - 1) / sp) + 4.0);
      if (t < best_t - 1e-9) { best_t = t; best_s = sp; }
    }
    p.splits = best_s;
  }
  p.a_sub_bytes = (uint32_t)(p.rows_pad * p.sca * 2);
  p.b_sub_bytes = (uint32_t)(p.rows_pad * p.scb * 2);
  p.a_sub_bytes = (p.a_sub_bytes + 1023) / 1024 * 1024;
  p.b_sub_bytes = (p.b_sub_bytes + 1023) / 1024 * 1024;
  p.a_region = p.a_sub_bytes * p.rpt * p.mpair;
  p.stage_bytes = p.a_region + p.b_sub_bytes * p.nb;
  p.tx_a = (uint32_t)(p.rows * p.rpt * p.sca * 2);
  p.tx_b = (uint32_t)(p.rows * p.nb * p.scb * 2);
  int stages = (int)((max_smem - tail) / p.stage_bytes);
  stages = std::min(stages, tc::kWgMaxStages);
  if (stages < 2) return shared_sm ? launch_wgrad_tc(enc, sm_count, attr_done, halo_attr_done, x, dy, dw, N, H, W, Cin, OH, OW, Cout,
                                                     R, stride, pad, dev_err, st, false)
                                   : -10;
  p.stages = stages;
  p.idesc = tc::instr_desc_bf16(128, p.n_tile, 1, 1);
  p.adesc_hi = tc::smem_desc_hi(p.a_sub_bytes, 8 * p.sca * 2, tc::swizzle_code_for_row_bytes(p.sca * 2));
  p.bdesc_hi = tc::smem_desc_hi(p.b_sub_bytes, 8 * p.scb * 2, tc::swizzle_code_for_row_bytes(p.scb * 2));
  uint32_t cols = 32;
  while ((int)cols < p.n_tile) cols *= 2;
  p.tmem_cols = p.mpair == 2 ? 512 : cols;   // second accumulator at column 256
  p.dw = dw; p.err = dev_err;
  CUtensorMap tmX, tmDY;
  if (wg_encode(enc, &tmX, x, N, H, W, Cin, p.sca, p.BW, p.BH, p.BNI, stride)) return -8;
  if (wg_encode(enc, &tmDY, dy, N, OH, OW, Cout, p.scb, p.BW, p.BH, p.BNI, 1)) return -8;
  // dw as a (C_in, tap, C_out) fp32 tensor for the bulk-reduction epilogue (boxes of one sub-box of
  // input channels, one tap, the CTA's output channels), where the operand ring can hold an accumulator
  CUtensorMap tmDW;
  memset(&tmDW, 0, sizeof(tmDW));
  p.epi_buf_bytes = (uint32_t)(p.n_tile * p.sca * 4);
  p.epi_bufs = 0;
  {
    cuuint64_t dims[3] = {(cuuint64_t)Cin, (cuuint64_t)p.taps, (cuuint64_t)Cout};
    cuuint64_t strides[2] = {(cuuint64_t)Cin * 4, (cuuint64_t)Cin * p.taps * 4};
    cuuint32_t box[3] = {(cuuint32_t)p.sca, 1, (cuuint32_t)p.n_tile};
    cuuint32_t es[3] = {1, 1, 1};
    if ((size_t)p.rpt * p.epi_buf_bytes <= (size_t)stages * p.stage_bytes && p.epi_buf_bytes % 128 == 0 &&
        (reinterpret_cast<uintptr_t>(dw) & 15) == 0 && Cin % 4 == 0 &&
        enc(&tmDW, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, dw, dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
            CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS)
      p.epi_bufs = p.rpt;
  }
  size_t smem = (size_t)stages * p.stage_bytes + tail;
  if (!shared_sm) smem = std::max(smem, (size_t)120 * 1024);   // one CTA, and one owner of all tensor memory, per SM
  if (!*attr_done) {   // per device
    if (cudaFuncSetAttribute(tc::wgrad_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 220 * 1024) != cudaSuccess)
      return -8;
    *attr_done = true;
  }
  dim3 grid(tiles, p.splits);
  return launch_pdl(tc::wgrad_tc_kernel, grid, dim3(256), smem, st, tmX, tmDY, tmDW, p) == cudaSuccess ? 0 : -8;
}

}  // namespace lp
