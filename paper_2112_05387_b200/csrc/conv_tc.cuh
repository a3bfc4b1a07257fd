// Implicit-GEMM convolution on the 5th-generation tensor cores (forward and input gradient).
//
// GEMM view: M = output pixels (tiles of up to 128: a BW x BH x BNI box of the output grid),
// N = output channels (tile of N_TILE <= 256), K = taps x input channels.  For every tap the
// A operand is a 4-D TMA box of the NHWC activation tensor shifted by the tap offset (zero fill
// outside the image supplies the padding; element strides supply the convolution stride); the B
// operand is a 2-D TMA box of the bf16 weights [C_out][taps*C_in].  Both land in shared memory
// in the K-major swizzled layout tcgen05.mma reads; accumulators live in tensor memory.
//
// Operand reuse: a CTA works on up to two consecutive pixel tiles at once ("pair"): both A tiles
// are multiplied with the same B stage, which halves the weight traffic per FLOP (the kernel is
// otherwise bound by L2 -> SM bandwidth).  The accumulators form a ring of 512 / N_TILE slots in
// tensor memory (3 for N_TILE = 160), so the epilogue of one unit overlaps the MMAs of the next
// as far as slots are free.
//
// Tap reuse ("halo" mode, 3x3 stride-1 convolutions; described for 64-channel K chunks, i.e. rows of
// 128 bytes -- chunks of 32 and 16 channels work the same way with 64- and 32-byte rows and their
// swizzles): all nine taps of
// a K chunk read the same activations, shifted by whole pixels.  The tile is 8 pixels wide and its
// rows are ordered (w, image, h); ONE box with a one-pixel halo all round, (8+2) x BNI x (BH+2)
// rows of 128 bytes, is fetched per K chunk and tile.  An 8-row group of the A operand (one image
// row segment) is then 8 consecutive box rows, consecutive groups are 10 rows (1280 bytes)
// apart, and tap (dy, dx) starts dy*10*BNI + dx rows into the box.  The shared-memory descriptor
// takes exactly that: its start address moves by whole 128-byte rows and its stride byte offset is
// 1280.  Neither is a multiple of the 1024-byte swizzle atom; that works because the 128-byte
// swizzle is a function of the shared-memory address bits (16-byte chunk index ^= address bits
// 7..9), for the TMA write and for the MMA read alike, so any row of the box can be the first row
// of an operand (checked against the CPU oracle by the parity tests).  Activations and weights
// travel in separate rings: an activation stage per K chunk (nine taps), a weight stage per group of
// taps (as many taps as leave three stages: all nine for 16 or 32 channels, two for 160).
// This cuts the bytes fetched per MMA from 52 KB to 25 KB per eight instructions.
//
// Roles: warp 0 = TMA producer; warps 1 and 2 = MMA issuers, one per accumulator of a pair (a
// tcgen05.mma costs its issuing thread about 65 cycles, close to the 80 cycles of tensor work of
// an N = 160 instruction, so one issuer cannot keep the pipe full); warps 3.. = epilogue
// (TMEM -> registers -> optional residual add -> bf16 store, per-channel sum / sum of squares
// for the batch-norm that follows).  One persistent CTA per SM walks a contiguous tile range.
#pragma once
#include "common.cuh"
#include "tc_ptx.cuh"

namespace lp {
namespace tc {

constexpr int kMaxStages = 12;
constexpr int kTmemCols = 512;
constexpr int kMaxSlots = 4;     // accumulator slots in tensor memory

#ifndef LP_EPI_WARPS
#define LP_EPI_WARPS 4
#endif
#ifndef LP_CONV_MIN_BLOCKS
#define LP_CONV_MIN_BLOCKS 1
#endif
#ifndef LP_EPI_BATCH
#define LP_EPI_BATCH 5
#endif

// Division by a run-time constant without the divide instruction (Granlund-Montgomery): for 0 <= n < 2^31,
// n / d = (umulhi(n, mul) + n) >> shift with shift = ceil(log2 d), mul = floor(2^32 (2^shift - d) / d) + 1.
// The tile loops of all roles split tile numbers several times per tile; with divide instructions that was a
// quarter of the life of a CTA on small layers.
struct FastDiv {
  uint32_t d, mul, shift;
};
__host__ inline FastDiv make_fastdiv(int d) {
  FastDiv f;
  f.d = (uint32_t)d; f.mul = 0; f.shift = 0;
  if (d > 1) {
    uint32_t s = 0;
    while ((1u << s) < (uint32_t)d) ++s;
    f.shift = s;
    f.mul = (uint32_t)((((uint64_t)1 << 32) * (((uint64_t)1 << s) - (uint64_t)d)) / (uint64_t)d + 1);
  }
  return f;
}
__device__ __forceinline__ int fd_div(int n, const FastDiv& f) {
  return f.d == 1 ? n : (int)((__umulhi((uint32_t)n, f.mul) + (uint32_t)n) >> f.shift);
}
// q = n / d, r = n % d
__device__ __forceinline__ void fd_divmod(int n, const FastDiv& f, int& q, int& r) {
  q = fd_div(n, f);
  r = n - q * (int)f.d;
}

struct ConvTcParams {
  int Nimg, OHl, OWl;            // logical output grid
  int BW, BH, BNI;               // tile box (logical pixels), BW*BH*BNI <= 128
  int tiles_w, tiles_h, m_tiles, n_tiles, total_tiles;
  FastDiv fd_tiles_w, fd_tiles_h, fd_m_tiles, fd_n_tiles, fd_chunks;   // the same numbers as divisors
  int in_step;                   // input coordinate = logical * in_step + tap offset
  int out_H, out_W, out_C;       // physical output tensor
  int os, oo_h, oo_w;            // physical pixel = logical * os + oo
  int n_tile_cols, Cout;
  int ntaps;
  int tap_dh[16], tap_dw[16], tap_w[16];   // up to 16 taps (plain mode; the space-to-depth stem has 4x4)
  // Tile classes (plain mode, direct epilogue): a stride-2 input gradient is one convolution per parity class of
  // the input pixels -- same logical grid and tiles, but its own subset of the taps and its own offset into the
  // physical output -- and one launch walks the classes one after another: tile t belongs to class
  // (t / m_tiles) / n_tiles and to channel tile (t / m_tiles) % n_tiles.  Every other launch has one class.
  int n_cls;
  int cls_ntaps[4], cls_tap0[4];           // taps of the class: tap_*[cls_tap0 .. cls_tap0 + cls_ntaps)
  int cls_oo_h[4], cls_oo_w[4];            // physical pixel = logical * os + cls_oo
  int Cin, KC, chunks;
  int nk_last;                   // K = 16 slices of the last chunk that hold real channels (the rest is zero fill)
  int stages;
  int ips;                       // (tap, K chunk) items per pipeline stage (plain mode): thin layers (few channels) put
                                 // several taps into one stage, so that the fixed cost of a stage -- a barrier round
                                 // trip, several hundred cycles -- is paid once per `ips` items instead of once each
  uint32_t item_bytes;           // one item: mpair activation tiles + the weight tile
  int mpair;                     // pixel tiles per unit: 1 or 2
  int nslots, acc_stride;        // accumulator ring: slots and their TMEM column stride
  int tmem_cols;                 // tensor-memory columns the CTA allocates: a power of two >= nslots * acc_stride
  uint32_t stage_bytes, a_region_bytes, b_offset, tx_a, tx_b;
  uint32_t idesc;
  uint64_t desc_hi;
  bf16* out;
  const bf16* addend;            // nullable; same geometry as out
  double* stats;                 // nullable; [2*Cout]
  int* err;
  // halo mode
  int halo;                      // 1: one activation box with a halo per K chunk serves all nine taps
  int nA, nB;                    // ring depths
  uint32_t a_halo_bytes;         // one activation box (1024-aligned)
  uint32_t a_stage_bytes;        // mpair boxes
  uint32_t b_stage_bytes, b_ring_offset;
  int tps;                       // halo mode: taps per weight stage.  A stage costs roughly 450 cycles plus 12 per KB
                                 // whatever it holds: with one tap (20 KB; 640 cycles of tensor work for a pair of
                                 // tiles) that is more than the tensor work, with two taps per stage it is less
  uint32_t b_tile_bytes;         // weights of one tap inside a weight stage
  uint32_t tail_offset;          // barriers and scratch after the rings
  int tap_widx9[16];             // weight tap index of the taps in (dy, dx) order (nine for 3x3, sixteen for 4x4)
  uint32_t tap_off9[16];         // byte offset of the tap's first row inside the box
  int halo_dw0, halo_dh0;        // offset of the first tap: the box starts that many pixels from the tile (-1 for 3x3)
  uint64_t desc_hi_a;            // descriptor of the activation operand (row-group stride of the box)
  // local loss of an interior module, fused into the epilogue of the module's last convolution
  // (kLoss instantiation): r = out - x_next, sums of r^2 and kappa*r, seed = rho*r + kappa
  const bf16* x_next;            // same geometry as out
  const bf16* kappa;             // nullable (penalty method)
  bf16* r_out;
  bf16* seed_out;
  float rho;
  double* loss_acc;              // [2]: sum r^2, sum kappa*r (atomically added)
  int wide32;                    // output (and residual) rows can be accessed in 32-byte pieces
  // staged epilogue (kStaged instantiations): the output tile goes through shared memory and leaves by TMA
  uint32_t stage_offset;         // staging region: one 128-row x 64-byte group per 32 output channels of the tile
  // Reduction pass of a batch-norm backward, fused into the epilogue (kBnBwd instantiations).  The
  // output of this convolution is dy, the gradient with respect to the result of y = [relu](bn(x));
  // the epilogue adds  sum dy_m  to dbeta and  rstd * sum dy_m (x - mean)  to dgamma, with
  // dy_m = dy where the ReLU let the value pass (recomputed from x as the forward kernel did), so
  // that only the apply pass of the batch-norm backward is left to run afterwards.
  const bf16* bwd_x;             // the tensor the batch norm normalised; same geometry as out
  BnArgs bwd_bn;                 // its statistics and affine parameters
  float* bwd_dgamma;             // [Cout], atomically added
  float* bwd_dbeta;
  int bwd_relu;                  // 1: a ReLU followed the batch norm
};

struct TcSmemTail {
  uint64_t full[kMaxStages];
  uint64_t empty[kMaxStages];
  uint64_t full_b[kMaxStages];
  uint64_t empty_b[kMaxStages];
  uint64_t tmem_full[kMaxSlots];
  uint64_t tmem_empty[kMaxSlots];
  uint64_t add_full;               // staged epilogue: the residual tile has landed in the staging region
  uint32_t tmem_base;
  int abort_flag;
  int epi_ok[2];                   // outcome of the epilogue's wait, alternating by accumulator (see the epilogue)
};
// Scratch of the direct (register -> global) epilogue's statistics, placed right after the tail.
struct TcStatScratch {
  float ssum[LP_EPI_WARPS][256];   // per epilogue warp: plain read-modify-write, no shared-memory atomics
  float ssq[LP_EPI_WARPS][256];
  uint32_t tr[LP_EPI_WARPS][16 * 33];   // per epilogue warp: transposition scratch of the statistics
};
// Additional scratch of the fused batch-norm-backward sums, placed right after TcStatScratch.
struct TcBnBwdScratch {
  uint32_t tr2[LP_EPI_WARPS][16 * 33];  // transposition scratch of the normalised tensor's tile
  float4 consts[256];                   // per channel of the current channel tile: scale, shift, mean, rstd
};
constexpr uint32_t kTailBytes = (uint32_t)((sizeof(TcSmemTail) + 127) / 128 * 128);
constexpr uint32_t kStageGroupBytes = 128 * 64;   // staging: 128 tile rows x 32 bf16 channels

// 32-byte global accesses (sm_100: 256-bit vector loads and stores); the address must be 32-byte aligned.
__device__ __forceinline__ void st_global_32B(void* p, const uint32_t* v) {
  asm volatile("st.global.v8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" ::"l"(p), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]),
               "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7])
               : "memory");
}
__device__ __forceinline__ void ld_global_32B(const void* p, uint4& lo, uint4& hi) {
  asm volatile("ld.global.v8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
               : "=r"(lo.x), "=r"(lo.y), "=r"(lo.z), "=r"(lo.w), "=r"(hi.x), "=r"(hi.y), "=r"(hi.z), "=r"(hi.w)
               : "l"(p)
               : "memory");
}

// first pixel (w0, h0) and first image n0 of pixel tile m
__device__ __forceinline__ void tile_first_pixel(const ConvTcParams& p, int m, int& w0, int& h0, int& n0) {
  int q1, r1, q2, r2;
  fd_divmod(m, p.fd_tiles_w, q1, r1);
  fd_divmod(q1, p.fd_tiles_h, q2, r2);
  w0 = r1 * p.BW; h0 = r2 * p.BH; n0 = q2 * p.BNI;
}

constexpr int kEpiThreads = 32 * LP_EPI_WARPS;
constexpr int kConvThreads = 96 + kEpiThreads;
constexpr int kFirstEpiWarp = 3;
constexpr int kEpiGroups = LP_EPI_WARPS / 4;

// kAddend: a residual operand is added in the epilogue (its loads run one channel group ahead);
// kLoss: the epilogue also takes the local loss of an interior module (implies kAddend);
// kStaged: the epilogue writes the bf16 tile into shared memory (64-byte swizzled rows of 32 channels)
//   and one thread sends it to global memory with TMA tile stores; the residual tile, when there is
//   one, arrives in the same region by TMA loads issued a tile ahead and is added in place.  Global
//   memory then sees whole 64-byte row pieces written by the copy engine instead of 16- or 32-byte
//   stores 2 x C_out bytes apart across the lanes of a warp, and the per-channel statistics are column
//   sums over the staged tile.  tmOut / tmAdd are only read by these instantiations.
// kBnBwd: the direct epilogue also takes the reduction pass of the batch-norm backward that consumes
//   this convolution's output (see ConvTcParams::bwd_x).
// kMinBlocks: CTAs of this kernel that must fit on one SM.  Layers of few channels (a channel tile of at most
//   64 columns) are launched as the two-per-SM instantiation -- registers capped accordingly (the epilogue
//   drains 64 accumulator columns per pass instead of 160), tensor memory and shared memory sized to need --
//   so that the kernels of several modules, each bound by latency rather than by any unit, share the SMs.
template <bool kLoss, bool kAddend, bool kStaged, bool kBnBwd = false, int kMinBlocks = LP_CONV_MIN_BLOCKS>
__global__ void __launch_bounds__(kConvThreads, kMinBlocks)
conv_tc_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
               const __grid_constant__ CUtensorMap tmOut, const __grid_constant__ CUtensorMap tmAdd,
               const __grid_constant__ ConvTcParams p) {
  static_assert(!(kStaged && kLoss), "the fused local loss uses the direct epilogue");
  static_assert(!(kBnBwd && (kStaged || kLoss)), "the fused batch-norm sums use the plain direct epilogue");
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  TcSmemTail* tail = reinterpret_cast<TcSmemTail*>(smem + p.tail_offset);
  TcStatScratch* scratch = reinterpret_cast<TcStatScratch*>(smem + p.tail_offset + kTailBytes);
  TcBnBwdScratch* bscratch = reinterpret_cast<TcBnBwdScratch*>(smem + p.tail_offset + kTailBytes + sizeof(TcStatScratch));
  volatile int* abort_flag = &tail->abort_flag;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  // contiguous tile range of this CTA
  const int t_begin = (int)(((long long)p.total_tiles * blockIdx.x) / gridDim.x);
  const int t_end = (int)(((long long)p.total_tiles * (blockIdx.x + 1)) / gridDim.x);

  // barrier set-up spread over the first threads (one thread doing all 57 took about a thousand cycles)
  if (threadIdx.x < kMaxStages) {
    const int s = threadIdx.x;
    mbar_init(&tail->full[s], 1);
    mbar_init(&tail->empty[s], 2);   // one arrival per MMA warp
    mbar_init(&tail->full_b[s], 1);
    mbar_init(&tail->empty_b[s], 2);
    fence_barrier_init();
  } else if (threadIdx.x >= 32 && threadIdx.x < 32 + kMaxSlots) {
    const int b = threadIdx.x - 32;
    mbar_init(&tail->tmem_full[b], 1);
    mbar_init(&tail->tmem_empty[b], kEpiThreads / 32);
    fence_barrier_init();
  }
  if (threadIdx.x == 64) {
    mbar_init(&tail->add_full, 1);
    tail->abort_flag = 0;
    fence_barrier_init();
    prefetch_tmap(&tmA);
    prefetch_tmap(&tmB);
    if constexpr (kStaged) {
      prefetch_tmap(&tmOut);
      if constexpr (kAddend) prefetch_tmap(&tmAdd);
    }
  }
  if (!kStaged && (p.stats || kBnBwd)) {   // (without statistics the scratch is not part of the allocation)
    for (int i = threadIdx.x; i < LP_EPI_WARPS * 256; i += blockDim.x) {
      (&scratch->ssum[0][0])[i] = 0.f;
      (&scratch->ssq[0][0])[i] = 0.f;
    }
  }
  if (warp == kFirstEpiWarp) {
    tmem_alloc(&tail->tmem_base, (uint32_t)p.tmem_cols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  pdl_wait();                 // the set-up above overlapped the tail of the preceding kernel
  pdl_launch_dependents();
  const uint32_t tmem_base = tail->tmem_base;
  bool failed = false;

  // All three roles walk the same sequence of units: a unit is one pixel tile, or two consecutive
  // ones of the same channel tile, and takes the next one or two accumulator slots of the ring.
  if (warp == 0 && p.halo) {
    // ------------------------------- TMA producer, halo mode ----------------------------
    uint32_t sa = 0, pha = 0, sb = 0, phb = 0;
    uint8_t* b_ring = smem + p.b_ring_offset;
    for (int t = t_begin; t < t_end && !failed;) {
      int nt, m;
      fd_divmod(t, p.fd_m_tiles, nt, m);
      const int cnt = (p.mpair == 2 && t + 1 < t_end && m + 1 < p.m_tiles) ? 2 : 1;
      int w0[2], h0[2], n0[2];
      for (int a = 0; a < 2; ++a) tile_first_pixel(p, m + a, w0[a], h0[a], n0[a]);
      const int col0 = nt * p.n_tile_cols;
      for (int c = 0; c < p.chunks && !failed; ++c) {
        if (!mbar_wait_warp(&tail->empty[sa], pha ^ 1, abort_flag)) { failed = true; break; }
        uint8_t* pa = smem + sa * p.a_stage_bytes;
        if (elect_one()) {
          mbar_expect_tx(&tail->full[sa], cnt * p.tx_a);
          tma_load_4d(pa, &tmA, &tail->full[sa], c * p.KC, w0[0] + p.halo_dw0, n0[0], h0[0] + p.halo_dh0);
          if (cnt == 2) tma_load_4d(pa + p.a_halo_bytes, &tmA, &tail->full[sa], c * p.KC, w0[1] + p.halo_dw0, n0[1], h0[1] + p.halo_dh0);
        }
        __syncwarp();
        if (++sa == (uint32_t)p.nA) { sa = 0; pha ^= 1; }
        for (int ti0 = 0; ti0 < p.ntaps; ti0 += p.tps) {
          const int n_taps = min(p.tps, p.ntaps - ti0);
          if (!mbar_wait_warp(&tail->empty_b[sb], phb ^ 1, abort_flag)) { failed = true; break; }
          if (elect_one()) {
            mbar_expect_tx(&tail->full_b[sb], n_taps * p.tx_b);
            for (int i = 0; i < n_taps; ++i)
              tma_load_2d(b_ring + sb * p.b_stage_bytes + i * p.b_tile_bytes, &tmB, &tail->full_b[sb],
                          p.tap_widx9[ti0 + i] * p.Cin + c * p.KC, col0);
          }
          __syncwarp();
          if (++sb == (uint32_t)p.nB) { sb = 0; phb ^= 1; }
        }
      }
      t += cnt;
    }
  } else if ((warp == 1 || warp == 2) && p.halo) {
    // ------------------------------- MMA issuers, halo mode -----------------------------
    const int me = warp - 1;
    uint32_t sa = 0, pha = 0, sb = 0, phb = 0;
    const uint32_t smem_base = smem_u32(smem);
    const int nk = p.KC >> 4;
    uint32_t slot = 0, slot_phase = 0;
    for (int t = t_begin; t < t_end && !failed;) {
      const int m = t - fd_div(t, p.fd_m_tiles) * p.m_tiles;
      const int cnt = (p.mpair == 2 && t + 1 < t_end && m + 1 < p.m_tiles) ? 2 : 1;
      uint32_t sl[2];
      sl[0] = slot;
      sl[1] = slot + 1 == (uint32_t)p.nslots ? 0 : slot + 1;
      const bool active = me < cnt;
      if (active) {
        if (!mbar_wait_warp(&tail->tmem_empty[sl[me]], ((slot_phase >> sl[me]) & 1) ^ 1, abort_flag)) { failed = true; break; }
        tc_fence_after();
      }
      const uint32_t d = tmem_base + sl[me] * p.acc_stride;
      uint32_t accum = 0;
      for (int c = 0; c < p.chunks && !failed; ++c) {
        const uint32_t a_addr = smem_base + sa * p.a_stage_bytes + me * p.a_halo_bytes;
        const int nkc = c + 1 == p.chunks ? p.nk_last : nk;   // slices of pure zero fill are not multiplied
        for (int ti0 = 0; ti0 < p.ntaps; ti0 += p.tps) {
          const int n_taps = min(p.tps, p.ntaps - ti0);
          const bool last_of_chunk = ti0 + n_taps == p.ntaps;
          // The box barrier is polled together with the first weight stage and released together
          // with the last one: a separate trip (poll, election, commit) at every chunk boundary
          // costs about 500 cycles in which the tensor pipe runs dry.
          bool ok = ti0 ? true : mbar_wait(&tail->full[sa], pha, abort_flag);
          ok = mbar_wait(&tail->full_b[sb], phb, abort_flag) && ok;
          if (!__all_sync(0xffffffffu, ok)) { failed = true; break; }
          tc_fence_after();
          const uint32_t b_addr = smem_base + p.b_ring_offset + sb * p.b_stage_bytes;
          if (elect_one()) {
            if (active) {
              for (int i = 0; i < n_taps; ++i) {
                const uint64_t ad = smem_desc(p.desc_hi_a, a_addr + p.tap_off9[ti0 + i]);
                const uint64_t bd = smem_desc(p.desc_hi, b_addr + i * p.b_tile_bytes);
                for (int j = 0; j < nkc; ++j)
                  mma_bf16(d, ad + (uint64_t)(2 * j), bd + (uint64_t)(2 * j), p.idesc, (accum | i | j) ? 1u : 0u);
              }
              mma_commit(&tail->empty_b[sb]);
              if (last_of_chunk) mma_commit(&tail->empty[sa]);
            } else {
              mbar_arrive(&tail->empty_b[sb]);
              if (last_of_chunk) mbar_arrive(&tail->empty[sa]);
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
      if (active && elect_one()) mma_commit(&tail->tmem_full[sl[me]]);
      __syncwarp();
      for (int a = 0; a < cnt; ++a) slot_phase ^= 1u << sl[a];
      slot = cnt == 2 ? (sl[1] + 1 == (uint32_t)p.nslots ? 0 : sl[1] + 1) : sl[1];
      t += cnt;
    }
  } else if (warp == 0) {
    // ------------------------------- TMA producer (warp-uniform loop, elected issue) ----
    uint32_t s = 0, ph = 0;
    for (int t = t_begin; t < t_end && !failed;) {
      int ntg, m, cls, nt;
      fd_divmod(t, p.fd_m_tiles, ntg, m);
      fd_divmod(ntg, p.fd_n_tiles, cls, nt);
      const int kiters = p.cls_ntaps[cls] * p.chunks;
      const int cnt = (p.mpair == 2 && t + 1 < t_end && m + 1 < p.m_tiles) ? 2 : 1;
      int w0[2], h0[2], n0[2];
      for (int a = 0; a < 2; ++a) tile_first_pixel(p, m + a, w0[a], h0[a], n0[a]);
      const int col0 = nt * p.n_tile_cols;
      const uint32_t tx = p.tx_b + cnt * p.tx_a;
      for (int k0 = 0; k0 < kiters && !failed; k0 += p.ips) {
        const int n_items = min(p.ips, kiters - k0);
        if (!mbar_wait_warp(&tail->empty[s], ph ^ 1, abort_flag)) { failed = true; break; }
        uint8_t* sa = smem + s * p.stage_bytes;
        if (elect_one()) {
          mbar_expect_tx(&tail->full[s], n_items * tx);
          for (int i = 0; i < n_items; ++i) {
            int tap, c;
            fd_divmod(k0 + i, p.fd_chunks, tap, c);
            tap += p.cls_tap0[cls];
            const int kb = p.tap_w[tap] * p.Cin;
            uint8_t* si = sa + i * p.item_bytes;
            tma_load_4d(si, &tmA, &tail->full[s], c * p.KC, w0[0] * p.in_step + p.tap_dw[tap],
                        h0[0] * p.in_step + p.tap_dh[tap], n0[0]);
            if (cnt == 2)
              tma_load_4d(si + p.a_region_bytes, &tmA, &tail->full[s], c * p.KC, w0[1] * p.in_step + p.tap_dw[tap],
                          h0[1] * p.in_step + p.tap_dh[tap], n0[1]);
            tma_load_2d(si + p.b_offset, &tmB, &tail->full[s], kb + c * p.KC, col0);
          }
        }
        __syncwarp();
        if (++s == (uint32_t)p.stages) { s = 0; ph ^= 1; }
      }
      t += cnt;
    }
  } else if (warp == 1 || warp == 2) {
    // ------------------------------- MMA issuers (warp-uniform loops, elected issue) ----
    // Warp 1 owns the first accumulator of every unit, warp 2 the second one of a pair.  Both
    // wait for every stage and both arrive on its "empty" barrier: with a commit after their
    // MMAs, or (warp 2 in a single-tile unit) with a plain arrive.
    const int me = warp - 1;
    uint32_t s = 0, ph = 0;
    const uint32_t smem_base = smem_u32(smem);
    const int nk = p.KC >> 4;
    uint32_t slot = 0, slot_phase = 0;  // bit b of slot_phase: parity of the number of uses of slot b
    for (int t = t_begin; t < t_end && !failed;) {
      int ntg, m;
      fd_divmod(t, p.fd_m_tiles, ntg, m);
      const int kiters = p.cls_ntaps[fd_div(ntg, p.fd_n_tiles)] * p.chunks;
      const int cnt = (p.mpair == 2 && t + 1 < t_end && m + 1 < p.m_tiles) ? 2 : 1;
      uint32_t sl[2];
      sl[0] = slot;
      sl[1] = slot + 1 == (uint32_t)p.nslots ? 0 : slot + 1;
      const bool active = me < cnt;
      if (active) {
        if (!mbar_wait_warp(&tail->tmem_empty[sl[me]], ((slot_phase >> sl[me]) & 1) ^ 1, abort_flag)) { failed = true; break; }
        tc_fence_after();
      }
      const uint32_t d = tmem_base + sl[me] * p.acc_stride;
      for (int k0 = 0; k0 < kiters; k0 += p.ips) {
        const int n_items = min(p.ips, kiters - k0);
        if (!mbar_wait_warp(&tail->full[s], ph, abort_flag)) { failed = true; break; }
        tc_fence_after();
        const uint32_t a_addr = smem_base + s * p.stage_bytes;
        if (elect_one()) {
          if (active) {
            for (int i = 0; i < n_items; ++i) {
              const int kc = k0 + i - fd_div(k0 + i, p.fd_chunks) * p.chunks;
              const int nkc = kc + 1 == p.chunks ? p.nk_last : nk;
              const uint64_t ad = smem_desc(p.desc_hi, a_addr + i * p.item_bytes + me * p.a_region_bytes);
              const uint64_t bd = smem_desc(p.desc_hi, a_addr + i * p.item_bytes + p.b_offset);
              for (int j = 0; j < nkc; ++j)  // +32 bytes (one K = 16 slice) per step, in 16-byte units
                mma_bf16(d, ad + (uint64_t)(2 * j), bd + (uint64_t)(2 * j), p.idesc, (k0 | i | j) ? 1u : 0u);
            }
            mma_commit(&tail->empty[s]);
          } else {
            mbar_arrive(&tail->empty[s]);
          }
        }
        __syncwarp();
        if (++s == (uint32_t)p.stages) { s = 0; ph ^= 1; }
      }
      if (failed) break;
      if (active && elect_one()) mma_commit(&tail->tmem_full[sl[me]]);
      __syncwarp();
      for (int a = 0; a < cnt; ++a) slot_phase ^= 1u << sl[a];
      slot = cnt == 2 ? (sl[1] + 1 == (uint32_t)p.nslots ? 0 : sl[1] + 1) : sl[1];
      t += cnt;
    }
  } else {
    if constexpr (kStaged) {
    // ------------------------------- epilogue, staged through shared memory -------------
    // Requires (checked by the launcher): output grid = logical grid (os = 1), channel tile a multiple
    // of 32, kEpiThreads = 128.  Thread `row` owns tile row `row` (one pixel) as in the direct epilogue.
    const int q = warp & 3;
    const int row = q * 32 + lane;
    const int et = threadIdx.x - 32 * kFirstEpiWarp;
    const int rows_used = p.BW * p.BH * p.BNI;
    // rows of a tile are ordered (w, h, image), or (w, image, h) in halo mode: this thread's place in every tile
    const int row_w = row % p.BW;
    const int row_h = p.halo ? row / (p.BW * p.BNI) : (row / p.BW) % p.BH;
    const int row_n = p.halo ? (row / p.BW) % p.BNI : row / (p.BW * p.BH);
    const int ngroups = p.n_tile_cols >> 5;
    uint8_t* stg = smem + p.stage_offset;
    // 64-byte swizzle of the staging rows, as the TMA unit applies it: 16-byte piece index ^= address bits 7..8
    uint8_t* my_row = stg + row * 64;
    const uint32_t swz = (uint32_t)((row >> 1) & 3);
    uint32_t slot = 0, slot_phase = 0, add_phase = 0;
    int epi_turn = 0;
    // per-channel statistics: thread (group sg, word sw) owns two channels and sums them over the rows
    const int sg = et >> 4, sw = et & 15;
    const bool stat_owner = p.stats != nullptr && sg < ngroups;
    float st_s0 = 0.f, st_s1 = 0.f, st_q0 = 0.f, st_q1 = 0.f;
    auto tile_origin = [&](int tile, int& col0, int& c1, int& c2, int& c3) {
      int nt, m, w0, h0, n0;
      fd_divmod(tile, p.fd_m_tiles, nt, m);
      tile_first_pixel(p, m, w0, h0, n0);
      col0 = nt * p.n_tile_cols;
      c1 = w0;
      c2 = p.halo ? n0 : h0;      // box dimension order (C, W, image, H) in halo mode, (C, W, H, image) otherwise
      c3 = p.halo ? h0 : n0;
    };
    auto load_addend_tile = [&](int tile) {   // elected thread only
      int col0, c1, c2, c3;
      tile_origin(tile, col0, c1, c2, c3);
      mbar_expect_tx(&tail->add_full, (uint32_t)(ngroups * rows_used * 64));
      for (int g = 0; g < ngroups; ++g)
        tma_load_4d(stg + g * kStageGroupBytes, &tmAdd, &tail->add_full, col0 + 32 * g, c1, c2, c3);
    };
    auto flush_stats = [&](int col0) {
      if (stat_owner) {
        const int c = col0 + sg * 32 + 2 * sw;
        if (c < p.Cout) {
          atomicAdd(&p.stats[c], (double)st_s0);
          atomicAdd(&p.stats[p.Cout + c], (double)st_q0);
        }
        if (c + 1 < p.Cout) {
          atomicAdd(&p.stats[c + 1], (double)st_s1);
          atomicAdd(&p.stats[p.Cout + c + 1], (double)st_q1);
        }
      }
      st_s0 = st_s1 = st_q0 = st_q1 = 0.f;
    };
    if constexpr (kAddend) {
      if (et == 0 && t_begin < t_end) load_addend_tile(t_begin);
    }
    for (int t = t_begin; t < t_end && !failed;) {
      int nt, m0;
      fd_divmod(t, p.fd_m_tiles, nt, m0);
      const int cnt = (p.mpair == 2 && t + 1 < t_end && m0 + 1 < p.m_tiles) ? 2 : 1;
      for (int a = 0; a < cnt && !failed; ++a) {
        const int tile = t + a;
        const int m = m0 + a;
        const uint32_t buf = slot;
        int w0, h0, n0;
        tile_first_pixel(p, m, w0, h0, n0);
        const int ow = w0 + row_w;
        const int oh = h0 + row_h;
        const int n = n0 + row_n;
        const bool valid = row < rows_used && ow < p.OWl && oh < p.OHl && n < p.Nimg;
        // One thread waits (bounded) for the accumulator, for the residual tile, and until the stores of
        // the previous tile have read the staging region; all epilogue threads then agree on the outcome.
        if (et == 0) {
          bool ok = mbar_wait(&tail->tmem_full[buf], (slot_phase >> buf) & 1, abort_flag);
          if constexpr (kAddend) ok = mbar_wait(&tail->add_full, add_phase, abort_flag) && ok;
          else bulk_wait_read(0);
          tail->epi_ok[epi_turn] = ok ? 1 : 0;
        }
        asm volatile("bar.sync 1, %0;" ::"n"(kEpiThreads) : "memory");
        const int wait_ok = *(volatile int*)&tail->epi_ok[epi_turn];
        epi_turn ^= 1;
        add_phase ^= 1;
        if (!wait_ok) { failed = true; break; }
        tc_fence_after();
        const uint32_t taddr = tmem_base + buf * p.acc_stride + ((uint32_t)(q * 32) << 16);
        constexpr int kBatch = LP_EPI_BATCH;
        for (int g0 = 0; g0 < ngroups; g0 += kBatch) {
          uint32_t raw[kBatch][32];
#pragma unroll
          for (int i = 0; i < kBatch; ++i)
            if (g0 + i < ngroups) tmem_ld32_issue(taddr + (g0 + i) * 32, raw[i]);
          tmem_ld_wait();
#pragma unroll
          for (int i = 0; i < kBatch; ++i) tmem_ld_fence(raw[i]);
          if (g0 + kBatch >= ngroups) {      // the accumulator is in registers: hand the slot back
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&tail->tmem_empty[buf]);
          }
#pragma unroll
          for (int i = 0; i < kBatch; ++i) {
            const int g = g0 + i;
            if (g >= ngroups) continue;
            uint8_t* grow = my_row + g * kStageGroupBytes;
#pragma unroll
            for (int u = 0; u < 4; ++u) {
              uint4* dst = reinterpret_cast<uint4*>(grow + ((u ^ swz) << 4));
              float v[8];
#pragma unroll
              for (int j = 0; j < 8; ++j) v[j] = valid ? __uint_as_float(raw[i][8 * u + j]) : 0.f;
              if constexpr (kAddend) {
                float f[8];
                cvt_raw(*dst, f);     // residual piece (zero where the tile leaves the tensor)
#pragma unroll
                for (int j = 0; j < 8; ++j) v[j] += f[j];
              }
              if (row < rows_used)
                *dst = make_uint4(pack_bf16x2(v[0], v[1]), pack_bf16x2(v[2], v[3]), pack_bf16x2(v[4], v[5]),
                                  pack_bf16x2(v[6], v[7]));
            }
          }
        }
        fence_proxy_async();     // the staged tile is read by the copy engine
        asm volatile("bar.sync 1, %0;" ::"n"(kEpiThreads) : "memory");
        if (et == 0) {
          int col0, c1, c2, c3;
          tile_origin(tile, col0, c1, c2, c3);
          for (int g = 0; g < ngroups; ++g)
            tma_store_4d(&tmOut, stg + g * kStageGroupBytes, col0 + 32 * g, c1, c2, c3);
          bulk_commit_group();
        }
        if (stat_owner) {
          // Statistics of the tensor as stored (bf16).  Lanes 0-15 and 16-31 of a warp read different
          // groups at the same offset: the second half walks the rows in swapped pairs so that the two
          // halves touch different 64-byte halves of a 128-byte line of banks.
          const uint8_t* gbase = stg + sg * kStageGroupBytes;
          const int flip = sg & 1;
          for (int r = 0; r < rows_used; ++r) {
            int rr = r ^ flip;
            if (rr >= rows_used) rr = r;
            const uint32_t w2 = *reinterpret_cast<const uint32_t*>(
                gbase + rr * 64 + ((((uint32_t)sw >> 2) ^ ((uint32_t)(rr >> 1) & 3)) << 4) + ((sw & 3) << 2));
            const float lo = __uint_as_float(w2 << 16), hi = __uint_as_float(w2 & 0xFFFF0000u);
            st_s0 += lo; st_s1 += hi;
            st_q0 = fmaf(lo, lo, st_q0); st_q1 = fmaf(hi, hi, st_q1);
          }
        }
        if constexpr (kAddend) {
          // the next residual tile may overwrite the staging region once the stores have read it and the
          // statistics above are done with it
          if (p.stats) asm volatile("bar.sync 1, %0;" ::"n"(kEpiThreads) : "memory");
          if (et == 0) {
            bulk_wait_read(0);
            if (tile + 1 < t_end) load_addend_tile(tile + 1);
          }
        }
        slot_phase ^= 1u << buf;
        slot = slot + 1 == (uint32_t)p.nslots ? 0 : slot + 1;
        const bool last_of_unit = a + 1 == cnt;
        if (p.stats && last_of_unit && (t + cnt >= t_end || m0 + cnt >= p.m_tiles)) flush_stats(nt * p.n_tile_cols);
      }
      t += cnt;
    }
    if (et == 0) bulk_wait_read(0);   // shared memory must outlive the last stores' reads
    } else {
    // ------------------------------- epilogue -----------------------------------------
    const int q = warp & 3;              // TMEM lane quarter this warp may read
    const int grp = (warp - kFirstEpiWarp) >> 2;  // which warp of the quarter (more than four epilogue warps)
    const int row = q * 32 + lane;
    const int et = threadIdx.x - 32 * kFirstEpiWarp;
    const int rows_used = p.BW * p.BH * p.BNI;
    // rows of a tile are ordered (w, h, image), or (w, image, h) in halo mode: this thread's place in every tile
    const int row_w = row % p.BW;
    const int row_h = p.halo ? row / (p.BW * p.BNI) : (row / p.BW) % p.BH;
    const int row_n = p.halo ? (row / p.BW) % p.BNI : row / (p.BW * p.BH);
    const int ngroups = (p.n_tile_cols + 31) >> 5;
    uint32_t slot = 0, slot_phase = 0;
    float sum_rr = 0.f, sum_kr = 0.f;    // local-loss sums of this thread (kLoss)
    int epi_turn = 0;
    // The residual operand (and the tensor of a fused batch-norm backward) was written several kernels
    // ago and is no longer in L2.  Each thread asks for the row of the NEXT tile it will read while it
    // works on the current one, so that the loads of the epilogue find their lines in L2 instead of
    // waiting for DRAM.
    auto prefetch_rows = [&](const bf16* base, int tile) {
      if (tile >= t_end) return;
      int pntg, pm, pcls, pnt, pw, phh, pn;
      fd_divmod(tile, p.fd_m_tiles, pntg, pm);
      fd_divmod(pntg, p.fd_n_tiles, pcls, pnt);
      tile_first_pixel(p, pm, pw, phh, pn);
      pw += row_w; phh += row_h; pn += row_n;
      if (row >= rows_used || pw >= p.OWl || phh >= p.OHl || pn >= p.Nimg || grp) return;
      const long long pb =
          (((long long)pn * p.out_H + (phh * p.os + p.cls_oo_h[pcls])) * p.out_W + (pw * p.os + p.cls_oo_w[pcls])) * p.out_C +
          pnt * p.n_tile_cols;
      const int ncols = min(p.n_tile_cols, p.Cout - pnt * p.n_tile_cols);
      const uintptr_t b = reinterpret_cast<uintptr_t>(base + pb);
      for (uintptr_t l = b & ~(uintptr_t)127; l < b + 2 * (uintptr_t)ncols; l += 128)
        asm volatile("prefetch.global.L2 [%0];" ::"l"(l));
    };
    auto prefetch_addend = [&](int tile) {
      if constexpr (kAddend) prefetch_rows(p.addend, tile);
      if constexpr (kBnBwd) prefetch_rows(p.bwd_x, tile);
    };
    prefetch_addend(t_begin);
    int consts_nt = -1;                  // channel tile whose batch-norm constants are in shared memory (kBnBwd)
    for (int t = t_begin; t < t_end && !failed;) {
      int nt, m0, cls, nt_c;                               // nt counts (class, channel tile) pairs
      fd_divmod(t, p.fd_m_tiles, nt, m0);
      fd_divmod(nt, p.fd_n_tiles, cls, nt_c);
      const int cnt = (p.mpair == 2 && t + 1 < t_end && m0 + 1 < p.m_tiles) ? 2 : 1;
      const int col0 = nt_c * p.n_tile_cols;
      if constexpr (kBnBwd) {
        if (nt != consts_nt) {
          // scale, shift (the forward kernel's, for the ReLU mask), mean and rstd of this channel tile
          asm volatile("bar.sync 1, %0;" ::"n"(kEpiThreads) : "memory");
          for (int c = et; c < 256; c += kEpiThreads) {
            float4 k4 = make_float4(0.f, 0.f, 0.f, 0.f);
            if (c < p.n_tile_cols && col0 + c < p.Cout) {
              float mean, rstd;
              bn_mean_rstd(p.bwd_bn.stats[col0 + c], p.bwd_bn.stats[p.Cout + col0 + c], p.bwd_bn.inv_count, p.bwd_bn.eps,
                           mean, rstd);
              const float sa = p.bwd_bn.gamma[col0 + c] * rstd;
              k4 = make_float4(sa, p.bwd_bn.beta[col0 + c] - mean * sa, mean, rstd);
            }
            bscratch->consts[c] = k4;
          }
          asm volatile("bar.sync 1, %0;" ::"n"(kEpiThreads) : "memory");
          consts_nt = nt;
        }
      }
      for (int a = 0; a < cnt && !failed; ++a) {
        prefetch_addend(t + a + 1);
        const int m = m0 + a;
        const uint32_t buf = slot;
        int w0, h0, n0;
        tile_first_pixel(p, m, w0, h0, n0);
        const int ow = w0 + row_w;
        const int oh = h0 + row_h;
        const int n = n0 + row_n;
        const bool valid = row < rows_used && ow < p.OWl && oh < p.OHl && n < p.Nimg;
        const long long obase =
            (((long long)n * p.out_H + (oh * p.os + p.cls_oo_h[cls])) * p.out_W + (ow * p.os + p.cls_oo_w[cls])) * p.out_C;
        // one thread waits (bounded) and all epilogue threads agree on the outcome, so that the
        // named barriers below are reached by all of them or by none
        // (two words used in turn: the one of the previous accumulator may still be read by a slower warp
        // when thread 0 writes the next outcome; the barrier below separates uses two apart)
        if (et == 0) tail->epi_ok[epi_turn] = mbar_wait(&tail->tmem_full[buf], (slot_phase >> buf) & 1, abort_flag) ? 1 : 0;
        asm volatile("bar.sync 1, %0;" ::"n"(kEpiThreads) : "memory");
        const int wait_ok = *(volatile int*)&tail->epi_ok[epi_turn];
        epi_turn ^= 1;
        if (!wait_ok) { failed = true; break; }
        tc_fence_after();
        const uint32_t taddr = tmem_base + buf * p.acc_stride + ((uint32_t)(q * 32) << 16);
        // Drain the accumulator into registers first (up to kBatch x 32 columns per pass) and hand
        // the TMEM slot back to the MMA warp; stores and statistics then work from registers.
        constexpr int kBatch = kMinBlocks > 1 ? 2 : LP_EPI_BATCH;
        // Residual operand of one 32-channel group, as raw 16-byte pieces (zero where nothing is added).
        // A group's pieces are requested while the group before it is processed.
        auto load_addend = [&](int g, uint4 (&a)[4]) {
          const int c_in_tile = g * 32;
          const int nv = c_in_tile + 32 <= p.n_tile_cols ? 4 : 2;
          if (p.wide32) {
#pragma unroll
            for (int u = 0; u < 2; ++u) {
              if (g < ngroups && 2 * u < nv && valid && col0 + c_in_tile + 16 * u < p.Cout) {
                ld_global_32B(p.addend + obase + col0 + c_in_tile + 16 * u, a[2 * u], a[2 * u + 1]);
              } else {
                a[2 * u] = a[2 * u + 1] = make_uint4(0u, 0u, 0u, 0u);
              }
            }
            return;
          }
#pragma unroll
          for (int u = 0; u < 4; ++u)
            a[u] = (g < ngroups && u < nv && valid && col0 + c_in_tile + 8 * u < p.Cout)
                       ? ld_raw(p.addend + obase + col0 + c_in_tile + 8 * u) : make_uint4(0u, 0u, 0u, 0u);
        };
        for (int g0 = grp; g0 < ngroups; g0 += kBatch * kEpiGroups) {
          uint32_t raw[kBatch][32];
          uint4 add_cur[4], add_next[4];
          if constexpr (kAddend) load_addend(g0, add_cur);
#pragma unroll
          for (int i = 0; i < kBatch; ++i) {
            const int g = g0 + i * kEpiGroups;
            if (g < ngroups) {
              if (g * 32 + 32 <= p.n_tile_cols) tmem_ld32_issue(taddr + g * 32, raw[i]);
              else tmem_ld16_issue(taddr + g * 32, raw[i]);
            }
          }
          tmem_ld_wait();
#pragma unroll
          for (int i = 0; i < kBatch; ++i) tmem_ld_fence(raw[i]);
          if (g0 + kBatch * kEpiGroups >= ngroups) {
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&tail->tmem_empty[buf]);
          }
#pragma unroll
          for (int i = 0; i < kBatch; ++i) {
            const int g = g0 + i * kEpiGroups;
            if (g >= ngroups) continue;
            const int c_in_tile = g * 32;
            const int col = col0 + c_in_tile;
            const bool wide = c_in_tile + 32 <= p.n_tile_cols;   // a 16-column tail otherwise
            const int nv = wide ? 4 : 2;                         // 8-channel vectors in this group
            float v[32];
#pragma unroll
            for (int j = 0; j < 32; ++j) v[j] = (wide || j < 16) ? __uint_as_float(raw[i][j]) : 0.f;
            // this pixel's 32 channels of the tensor the batch norm normalised, asked for before the
            // stores so that they have arrived when the sums need them
            uint4 xr[kBnBwd ? 4 : 1];
            if constexpr (kBnBwd) {
#pragma unroll
              for (int u = 0; u < 4; ++u)
                xr[u] = (u < nv && valid && col + 8 * u < p.Cout) ? ld_raw(p.bwd_x + obase + col + 8 * u)
                                                                  : make_uint4(0u, 0u, 0u, 0u);
            }
            if constexpr (kAddend) {
              if (i + 1 < kBatch) load_addend(g + kEpiGroups, add_next);
#pragma unroll
              for (int u = 0; u < 4; ++u) {
                float f[8];
                cvt_raw(add_cur[u], f);
#pragma unroll
                for (int j = 0; j < 8; ++j) v[8 * u + j] += f[j];
                add_cur[u] = add_next[u];
              }
            }
            // bf16 pairs as they go to memory: the store and the statistics both work from them
            uint32_t pk[16];
#pragma unroll
            for (int j = 0; j < 16; ++j) pk[j] = pack_bf16x2(v[2 * j], v[2 * j + 1]);
            if (p.wide32) {
              // whole 32-byte sectors per lane: half as many store instructions, no partial sectors
#pragma unroll
              for (int u = 0; u < 2; ++u)
                if (2 * u < nv && valid && col + 16 * u < p.Cout) st_global_32B(p.out + obase + col + 16 * u, &pk[8 * u]);
            } else {
#pragma unroll
              for (int u = 0; u < 4; ++u)
                if (u < nv && valid && col + 8 * u < p.Cout)
                  *reinterpret_cast<uint4*>(p.out + obase + col + 8 * u) =
                      make_uint4(pk[4 * u], pk[4 * u + 1], pk[4 * u + 2], pk[4 * u + 3]);
            }
            if constexpr (kLoss) {
              // The module output is what was just stored (bf16); the residual against the
              // auxiliary variable, the loss sums and the terminal adjoint follow from it.
#pragma unroll
              for (int u = 0; u < 4; ++u)
                if (u < nv && valid && col + 8 * u < p.Cout) {
                  float xn[8], r[8], sd[8];
                  ldv(p.x_next + obase + col + 8 * u, xn);
#pragma unroll
                  for (int j = 0; j < 8; ++j) {
                    r[j] = round_storage<bf16>(v[8 * u + j]) - xn[j];
                    sum_rr += r[j] * r[j];
                  }
                  stv(p.r_out + obase + col + 8 * u, r);
                  if (p.kappa) {
                    float kp[8];
                    ldv(p.kappa + obase + col + 8 * u, kp);
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                      sum_kr += kp[j] * r[j];
                      sd[j] = p.rho * r[j] + kp[j];
                    }
                  } else {
#pragma unroll
                    for (int j = 0; j < 8; ++j) sd[j] = p.rho * r[j];
                  }
                  stv(p.seed_out + obase + col + 8 * u, sd);
                }
            }
            if (kBnBwd || p.stats) {
              // Statistics of the tensor as stored (bf16), so that the batch-norm that follows
              // normalises exactly the values it reads.  A thread holds one pixel and 32 channels;
              // the sums run over pixels, so the warp transposes through shared memory: every lane
              // writes its 16 channel pairs, then lane l sums channel pair (l & 15) over 16 of the
              // warp's 32 pixels (both phases conflict-free with the row pitch of 33 words).
              // kBnBwd: the two sums are those of a batch-norm backward, sum dy_m and
              // sum dy_m (x - mean), and the tile of x is transposed beside the tile of dy.
              uint32_t* T = scratch->tr[warp - kFirstEpiWarp];
#pragma unroll
              for (int j = 0; j < 16; ++j) T[j * 33 + lane] = (valid && (wide || j < 8)) ? pk[j] : 0u;
              if constexpr (kBnBwd) {
                uint32_t* T2 = bscratch->tr2[warp - kFirstEpiWarp];
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                  const bool on = valid && (wide || u < 2);
                  T2[(4 * u + 0) * 33 + lane] = on ? xr[u].x : 0u;
                  T2[(4 * u + 1) * 33 + lane] = on ? xr[u].y : 0u;
                  T2[(4 * u + 2) * 33 + lane] = on ? xr[u].z : 0u;
                  T2[(4 * u + 3) * 33 + lane] = on ? xr[u].w : 0u;
                }
              }
              __syncwarp();
              const int jc = lane & 15, hh = lane >> 4;
              const uint32_t* col_t = T + jc * 33 + hh * 16;
              float s0 = 0.f, s1 = 0.f, q0 = 0.f, q1 = 0.f;
              if constexpr (kBnBwd) {
                const uint32_t* col_x = bscratch->tr2[warp - kFirstEpiWarp] + jc * 33 + hh * 16;
                const float4 k0 = bscratch->consts[c_in_tile + 2 * jc], k1 = bscratch->consts[c_in_tile + 2 * jc + 1];
                const bool relu = p.bwd_relu != 0;
#pragma unroll
                for (int i2 = 0; i2 < 16; ++i2) {
                  const uint32_t w2 = col_t[i2], x2 = col_x[i2];
                  float dlo = __uint_as_float(w2 << 16), dhi = __uint_as_float(w2 & 0xFFFF0000u);
                  const float xlo = __uint_as_float(x2 << 16), xhi = __uint_as_float(x2 & 0xFFFF0000u);
                  if (relu) {
                    dlo = fmaf(xlo, k0.x, k0.y) > 0.f ? dlo : 0.f;
                    dhi = fmaf(xhi, k1.x, k1.y) > 0.f ? dhi : 0.f;
                  }
                  s0 += dlo; s1 += dhi;
                  q0 = fmaf(dlo, xlo - k0.z, q0); q1 = fmaf(dhi, xhi - k1.z, q1);
                }
              } else {
#pragma unroll
                for (int i2 = 0; i2 < 16; ++i2) {
                  const uint32_t w2 = col_t[i2];
                  const float lo = __uint_as_float(w2 << 16), hi = __uint_as_float(w2 & 0xFFFF0000u);
                  s0 += lo; s1 += hi;
                  q0 = fmaf(lo, lo, q0); q1 = fmaf(hi, hi, q1);
                }
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
        // flush the column sums when the channel tile is about to change (or at the very end)
        const bool last_of_unit = a + 1 == cnt;
        const bool flush = (kBnBwd || p.stats) && last_of_unit && (t + cnt >= t_end || m0 + cnt >= p.m_tiles);
        if (flush) {
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
              if constexpr (kBnBwd) {
                atomicAdd(&p.bwd_dbeta[col0 + c], a_s);
                atomicAdd(&p.bwd_dgamma[col0 + c], a_q * bscratch->consts[c].w);
              } else {
                atomicAdd(&p.stats[col0 + c], (double)a_s);
                atomicAdd(&p.stats[p.Cout + col0 + c], (double)a_q);
              }
            }
          }
          asm volatile("bar.sync 1, %0;" ::"n"(kEpiThreads) : "memory");
        }
      }
      t += cnt;
    }
    if constexpr (kLoss) {
      __syncwarp();
      sum_rr = warp_sum(sum_rr);
      sum_kr = warp_sum(sum_kr);
      if (lane == 0 && !failed) {
        atomicAdd(&p.loss_acc[0], (double)sum_rr);
        atomicAdd(&p.loss_acc[1], (double)sum_kr);
      }
    }
    }   // direct epilogue
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
  __syncthreads();
  if (warp == kFirstEpiWarp) {
    tc_fence_after();
    tmem_dealloc(tmem_base, (uint32_t)p.tmem_cols);
  }
}

}  // namespace tc
}  // namespace lp
