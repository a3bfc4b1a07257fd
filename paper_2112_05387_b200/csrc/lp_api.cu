// C ABI of the layer-parallel training step: descriptor parsing, workspace planning, the per-module
// operation lists (forward, local loss, backward), and their execution on CUDA streams.
#include <cuda.h>
#include <cuda_runtime.h>
#include <math.h>
#include <stdio.h>
#include <string.h>

#include <algorithm>
#include <mutex>
#include <string>
#include <vector>

#include "../../include/lp.h"
#include "conv_simt.cuh"
#include "conv_tc.cuh"
#include "conv_tc2.cuh"
#include "kernels_elem.cuh"
#include "net.h"
#include "wgrad_tc.cuh"

namespace lp {

// ---------------------------------------------------------------------------------------------
// small utilities
// ---------------------------------------------------------------------------------------------
static inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }
static inline size_t esize(int dtype) { return dtype == LP_F32 ? 4 : 2; }

enum ExtSlot { EXT_NONE = 0, EXT_X, EXT_XNEXT, EXT_KAPPA, EXT_DX, EXT_IMAGES, EXT_XOUT0 /* + k */ };

struct Tensor {
  void* p = nullptr;  // workspace address (or fallback when ext != EXT_NONE)
  int ext = EXT_NONE;
  int n = 0, h = 0, w = 0, c = 0;
  long long elems() const { return (long long)n * h * w * c; }
  bool defined() const { return p != nullptr || ext != EXT_NONE; }
};

struct ConvDef {
  int cin, cout, R, stride, pad;
  int H, W, OH, OW;          // input / output spatial size
  float* w = nullptr;        // fp32 master [cout][R][R][cin]
  float* gw = nullptr;       // gradient, same layout
  bf16* wf = nullptr;        // bf16 [cout][R*R*cin]
  bf16* wt = nullptr;        // bf16 [cin][R*R*cout] (input-gradient operand), optional
  bool need_dgrad = true;
  // 7x7 / stride-2 stem on the tensor cores by space-to-depth (see kernels_elem.cuh): the regrouped input,
  // the regrouped bf16 weights [cout][16 taps][16] (in wf) and the weight gradient in that layout
  bool s2d = false;
  bf16* xs = nullptr;        // [N][H/2][W/2][16]
  float* dws = nullptr;      // [cout][16][16]
};
struct BnDef {
  int C;
  long long count;           // N*H*W of the normalised tensor
  float *gamma = nullptr, *beta = nullptr, *dgamma = nullptr, *dbeta = nullptr;
  double* stats = nullptr;   // [2*C]
};

enum OpType {
  OP_CONV_FWD, OP_CONV_DGRAD, OP_CONV_WGRAD, OP_BN_STATS, OP_BN_APPLY, OP_OUT_LOSS, OP_BN_BWD, OP_MAXPOOL_FWD,
  OP_MAXPOOL_BWD, OP_HEAD_FWD, OP_HEAD_BWD, OP_COPY
};

static_assert(OP_CONV_FWD == LP_OP_CONV_FWD && OP_BN_BWD == LP_OP_BN_BWD && OP_COPY == LP_OP_COPY && LP_OP_UPDATE == OP_COPY + 1,
              "operation codes of the time line follow OpType");

struct Op {
  OpType type;
  Tensor in, in2, addend, mask, out;
  int conv = -1, bn = -1, bn2 = -1, stats_bn = -1;
  int relu = 0;
  int fuse_loss = 0;       // conv: its epilogue takes the module's local loss; out_loss: only the final scalars are left
  // Reduction pass of a batch-norm backward taken by the epilogue of the input-gradient convolution
  // that writes its dy.  On the convolution: bwd_bn >= 0 names the batch norm, bwd_x the tensor it
  // normalised, bwd_relu whether a ReLU followed.  On the batch-norm backward: reduce_fused = 1,
  // only the apply pass is left.
  int bwd_bn = -1, bwd_relu = 0, reduce_fused = 0;
  Tensor bwd_x;
  uint8_t* arg = nullptr;  // max-pool argmax
};

struct ParamSet {
  std::vector<lp_param_entry> layout;
  size_t n = 0;
  float *p = nullptr, *g = nullptr, *m = nullptr;
  PackEntry* dev_pack = nullptr;
  std::vector<PackEntry> host_pack;
  std::vector<SgdRange> host_ranges;   // the parts of the blob that have no packed copy
  SgdRange* dev_ranges = nullptr;
  long long pack_total = 0;
  long long pack_tiles = 0;
  long long pack_tiles64 = 0;   // 64x64 tiles of the update kernel with 16-byte accesses
  bool pack64_ok = true;        // every packed weight tensor starts on a 16-byte boundary of the blobs
  bool grads_fresh = false;
  bool momentum_used = false;
};

struct HeadDef {
  int C = 0, classes = 0, HW = 0, N = 0;
  float *W = nullptr, *b = nullptr, *dW = nullptr, *db = nullptr;
  float *pooled = nullptr, *logits = nullptr, *dlogits = nullptr;
};

struct Plan {  // one module or one AuxNet
  std::vector<Op> fwd, bwd;
  std::vector<ConvDef> convs;
  std::vector<BnDef> bns;
  ParamSet ps;
  HeadDef head;
  bool has_head = false;
  Tensor out;    // module output (interior modules; serial mode) / AuxNet output
  Tensor r, seed;
  double* loss_acc = nullptr;  // [2]
  void* stats_region = nullptr;
  size_t stats_bytes = 0;
  void* dx_fallback = nullptr;
  bool interior = false;
  bool ran_fwd_bwd = false;
  // Weight gradients feed nothing but the update, so in the backward pass they leave the chain
  // dy -> BN' -> dx -> ... : each is enqueued on this second stream right after the kernel that wrote its dy
  // (one event per weight gradient), and the pass joins the stream back at its end.
  cudaStream_t side = nullptr;
  std::vector<cudaEvent_t> side_ev;
  cudaEvent_t side_done = nullptr;
};

struct Arena {
  uint8_t* base = nullptr;
  size_t off = 0;
  void* alloc(size_t bytes) {
    off = align_up(off, 256);
    void* p = base + off;
    off += bytes;
    return p;
  }
};

struct RunCtx {
  cudaStream_t st = nullptr;
  const void* x = nullptr;
  const void* xnext = nullptr;
  const void* kappa = nullptr;
  void* dx = nullptr;
  const int32_t* labels = nullptr;
  const void* images = nullptr;
  void* const* xout = nullptr;
  float rho = 0.f;
  float* loss_out = nullptr;
  bool serial = false;       // layer-serial mode: interior modules produce `out`, no local loss
  cudaEvent_t loss_wait = nullptr;  // recorded when x_{k+1} is ready: awaited just before the local loss
  int plan_id = 0;           // time line: module k, or LP_AUX(k)
  int phase = 0;             // time line: LP_PHASE_*
};

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

struct Device {
  bool ready = false;
  int sm_count = 148;
  EncodeTiledFn encode = nullptr;
  // kernel attributes are per device: set on the first launch of each kernel family on that device
  bool conv_attr = false, wgrad_attr = false, wgrad_halo_attr = false, conv2_attr = false;
  int max_pairs = 0;   // CTA pairs of conv_tc2_kernel that can be resident at once (0: not usable)
  int init() {
    if (ready) return LP_OK;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return LP_ERR_CUDA;
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, dev) != cudaSuccess) return LP_ERR_CUDA;
    sm_count = prop.multiProcessorCount;
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q) != cudaSuccess || !fn)
      return LP_ERR_CUDA;
    encode = (EncodeTiledFn)fn;
    if (prop.major != 10) return LP_ERR_UNSUPPORTED;  // the kernels are built for sm_100a only
    ready = true;
    return LP_OK;
  }
};
// One record per device ordinal; the current device's record is looked up at every use.  The mutex
// covers first-use initialisation from several host threads.
static const int kMaxDevices = 64;
static Device g_devices[kMaxDevices];
static std::mutex g_devices_mutex;
static inline Device& cur_dev() {
  int d = 0;
  if (cudaGetDevice(&d) != cudaSuccess || d < 0 || d >= kMaxDevices) d = 0;
  return g_devices[d];
}
static inline int init_cur_dev() {
  std::lock_guard<std::mutex> lock(g_devices_mutex);
  return cur_dev().init();
}

// Per-operation time line: a pair of events around every operation of every plan, on the stream
// the operation runs on.  Events do not serialise the streams; they cannot be recorded into a graph.
struct TimelineRec {
  cudaEvent_t a = nullptr, b = nullptr;
  int plan = 0, op_type = 0, phase = 0;
  double bytes = 0.0;
};
struct Timeline {
  bool enabled = false;
  cudaEvent_t base = nullptr;
  bool base_recorded = false;
  std::vector<TimelineRec> recs;
  size_t used = 0;
};

struct ConvProfile {
  bool enabled = false;
  std::vector<std::pair<cudaEvent_t, cudaEvent_t>> events;
  std::vector<double> flops;
  size_t used = 0;
};

}  // namespace lp

using namespace lp;

struct lp_handle {
  NetDef net;
  int dtype = LP_F32;
  std::vector<Plan> modules, auxs;
  int* dev_err = nullptr;
  std::vector<cudaStream_t> streams;
  std::vector<cudaEvent_t> done;
  cudaEvent_t fork = nullptr;
  cudaStream_t aux_stream = nullptr;
  std::vector<cudaEvent_t> aux_done;  // aux_done[k]: x_{k+1} has been produced
  cudaEvent_t aux_end = nullptr;
  int64_t launches = 0;
  ConvProfile prof;
  Timeline tl;
  int conv_impl = LP_CONV_IMPL_AUTO;
  bool concurrent = false;   // set while a call enqueues the K modules on their own streams
  uint8_t* ws = nullptr;
  size_t ws_bytes = 0;
  int32_t* zero_labels = nullptr;  // N zeros, for forward passes that only want logits
  std::vector<cudaGraphExec_t> graphs;
  int64_t launches_at_capture = 0;
  std::vector<int64_t> graph_launches;  // kernels recorded in each graph
};

namespace lp {

#define LP_CUDA_OK(expr)                         \
  do {                                           \
    cudaError_t e__ = (expr);                    \
    if (e__ != cudaSuccess) return LP_ERR_CUDA;  \
  } while (0)

static inline int grid_for(long long work_items, int threads, int sm_count, int per_sm = 8) {
  long long blocks = (work_items + threads - 1) / threads;
  long long cap = (long long)sm_count * per_sm;
  if (blocks > cap) blocks = cap;
  if (blocks < 1) blocks = 1;
  return (int)blocks;
}

// block size that is a multiple of the number of 16-byte channel groups
static inline int threads_for_channels(int C, int dtype) {
  const int V = dtype == LP_F32 ? 4 : 8;
  const int CV = C / V;
  if (CV >= 256) return CV <= 1024 ? CV : 0;
  return CV * (256 / CV);
}

// ---------------------------------------------------------------------------------------------
// tensor-core convolution launch (forward / input gradient share one kernel)
// ---------------------------------------------------------------------------------------------
struct TcGemmSpec {
  const bf16* act; int aN, aH, aW, aC;
  const bf16* wmat; int w_rows; long long w_K;
  int in_step;
  int OHl, OWl;
  int ntaps; int dh[16], dw[16], widx[16];
  bf16* out; const bf16* addend; int out_H, out_W, out_C, os, oo_h, oo_w;
  double* stats;
  // local loss fused into the epilogue (interior module's last convolution); x_next == nullptr: off
  const bf16* x_next; const bf16* kappa; bf16* r_out; bf16* seed_out; float rho; double* loss_acc;
  int epilogue;          // 0: default (staged where a residual operand exists), 1: direct, 2: staged wherever it applies
  int two_cta;           // 1: 3x3 stride-1 convolutions take the CTA-pair kernel where it applies
  // reduction pass of a batch-norm backward fused into the epilogue; bwd_x == nullptr: off
  const bf16* bwd_x; BnArgs bwd_bn; float* bwd_dgamma; float* bwd_dbeta; int bwd_relu;
  // tile classes (see ConvTcParams): n_cls > 1 for the parity classes of a stride-2 input gradient in one launch;
  // the taps of class i are dh/dw/widx[cls_tap0[i] .. +cls_ntaps[i]), its output offset (cls_oo_h[i], cls_oo_w[i])
  int n_cls; int cls_ntaps[4], cls_tap0[4], cls_oo_h[4], cls_oo_w[4];
};

static void pick_pixel_box(int OWl, int OHl, int Nimg, int& BW, int& BH, int& BNI) {
  BW = std::min(OWl, 128);
  int bh = std::max(1, 128 / BW);
  bh = std::min(bh, OHl);
  const int th = (OHl + bh - 1) / bh;
  BH = (OHl + th - 1) / th;
  int bn = std::max(1, 128 / (BW * BH));
  bn = std::min(bn, Nimg);
  const int tn = (Nimg + bn - 1) / bn;
  BNI = (Nimg + tn - 1) / tn;
}

// K chunk (channels per pipeline stage).  Every stage costs a fixed amount (barrier round trip,
// TMA and MMA issue) worth roughly 48 channels of tensor work, so fewer, larger chunks win even
// when the last chunk of a tap is partly zero fill (160 channels: 3 chunks of 64, not 5 of 32).
static int pick_kc(int Cin) {
  int best = 16, best_cost = 1 << 30;
  for (int kc : {64, 32, 16}) {
    const int cost = (Cin + kc - 1) / kc * (kc + 48);
    if (cost < best_cost) { best_cost = cost; best = kc; }
  }
  return best;
}

static void pick_n_tile(int Cout, int& n_tile, int& n_tiles) {
  int best_nt = 0, best_tile = 0, best_waste = 1 << 30;
  const int lo = (Cout + 255) / 256;
  for (int nt = lo; nt <= lo + 3; ++nt) {
    int tile = (Cout + nt - 1) / nt;
    tile = (tile + 15) / 16 * 16;
    if (tile > 256) continue;
    const int waste = nt * tile - Cout;
    if (waste < best_waste) { best_waste = waste; best_nt = nt; best_tile = tile; }
  }
  n_tile = best_tile;
  n_tiles = best_nt;
}

static int encode_act_map(CUtensorMap* m, const void* base, int N, int H, int W, int C, int boxC, int BW, int BH,
                          int BNI, int step, int row_bytes) {
  cuuint64_t dims[4] = {(cuuint64_t)C, (cuuint64_t)W, (cuuint64_t)H, (cuuint64_t)N};
  cuuint64_t strides[3] = {(cuuint64_t)C * 2, (cuuint64_t)W * C * 2, (cuuint64_t)H * W * C * 2};
  cuuint32_t box[4] = {(cuuint32_t)boxC, (cuuint32_t)((BW - 1) * step + 1), (cuuint32_t)((BH - 1) * step + 1),
                       (cuuint32_t)BNI};
  cuuint32_t es[4] = {1, (cuuint32_t)step, (cuuint32_t)step, 1};
  const CUtensorMapSwizzle sw = row_bytes == 128 ? CU_TENSOR_MAP_SWIZZLE_128B
                                : row_bytes == 64 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_32B;
  CUresult r = cur_dev().encode(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, es,
                            CU_TENSOR_MAP_INTERLEAVE_NONE, sw, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? LP_OK : LP_ERR_CUDA;
}

static int encode_mat_map(CUtensorMap* m, const void* base, long long K, int rows, int boxK, int boxRows,
                          int row_bytes) {
  cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)K * 2};
  cuuint32_t box[2] = {(cuuint32_t)boxK, (cuuint32_t)boxRows};
  cuuint32_t es[2] = {1, 1};
  const CUtensorMapSwizzle sw = row_bytes == 128 ? CU_TENSOR_MAP_SWIZZLE_128B
                                : row_bytes == 64 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_32B;
  CUresult r = cur_dev().encode(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, es,
                            CU_TENSOR_MAP_INTERLEAVE_NONE, sw, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? LP_OK : LP_ERR_CUDA;
}

// Tensor map of an NHWC bf16 tensor for the staged epilogue: boxes of 32 channels x one pixel tile, 64-byte
// swizzled rows; `wnh` selects the dimension order (C, W, image, H) of the halo-mode tiles.
static int encode_tile32_map(CUtensorMap* m, const void* base, int N, int H, int W, int C, int BW, int BH, int BNI,
                             bool wnh) {
  cuuint64_t dims[4] = {(cuuint64_t)C, (cuuint64_t)W, (cuuint64_t)(wnh ? N : H), (cuuint64_t)(wnh ? H : N)};
  cuuint64_t strides[3] = {(cuuint64_t)C * 2, (cuuint64_t)(wnh ? (size_t)H * W * C * 2 : (size_t)W * C * 2),
                           (cuuint64_t)(wnh ? (size_t)W * C * 2 : (size_t)H * W * C * 2)};
  cuuint32_t box[4] = {32, (cuuint32_t)BW, (cuuint32_t)(wnh ? BNI : BH), (cuuint32_t)(wnh ? BH : BNI)};
  cuuint32_t es[4] = {1, 1, 1, 1};
  CUresult r = cur_dev().encode(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, es,
                                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? LP_OK : LP_ERR_CUDA;
}

static const size_t kTcMinSmem = 120 * 1024;   // more than half an SM: one CTA (and one TMEM owner) per SM
static const size_t kTcMaxSmem = 220 * 1024;
// A convolution of fewer FLOPs than this (and at most 64 channels) cannot fill the machine whatever its launch
// shape: a few microseconds of fixed cost dominate.  While several modules are enqueued side by side such
// launches are sized to share the SMs with the other modules' kernels instead of taking them whole.
static const double kSmallConvFlops = 4e9;
static const size_t kTcThinSmem = 100 * 1024;  // two CTAs of the few-channel instantiation (or other kernels) per SM

// Halo mode (one activation box per K chunk serves all nine taps, see conv_tc.cuh): a 3x3 stride-1
// tap set, 64-channel K chunks and an output width that is a multiple of 8.
#ifndef LP_CONV_MAX_NB
#define LP_CONV_MAX_NB 8   // weight stages in flight (halo mode), as far as shared memory allows
#endif
#ifndef LP_CONV_MAX_ITEMS_PER_STAGE
#define LP_CONV_MAX_ITEMS_PER_STAGE 16   // (tap, chunk) items per pipeline stage of the plain mode, at most
#endif
#ifndef LP_CONV2_TAPS_PER_STAGE
#define LP_CONV2_TAPS_PER_STAGE 3  // the same for the CTA-pair kernel (a stage holds each CTA's half of the taps' weights)
#endif
#ifndef LP_CONV_TAPS_PER_STAGE
#define LP_CONV_TAPS_PER_STAGE 16  // taps per weight stage (halo mode), at most: as many as leave three stages
#endif
static const int kHaloBoxW = 10;   // 8-pixel tile width plus one halo pixel on each side

// Halo mode: the taps form a full R x R grid of whole-pixel offsets (3x3 convolutions; the 4x4 grid of a
// space-to-depth stem), stride 1.  R: grid size; dw0, dh0: offset of the first tap; tapw[dy*R + dx]: weight index.
static bool pick_halo_box_r(const TcGemmSpec& s, int& BW, int& BH, int& BNI, int& R, int& dw0, int& dh0, int tapw[16]) {
  R = s.ntaps == 9 ? 3 : (s.ntaps == 16 ? 4 : 0);
  // tiles are 8 pixels wide; a width that is not a multiple of 8 leaves the last tile column ragged (rows past the
  // image read zero fill and are masked in the epilogue): taken where at most an eighth of the columns is wasted
  // (7, 14, 28, ...), since the alternative is nine shifted boxes per K chunk instead of one
  const int tiles_w8 = (s.OWl + 7) / 8;
  if (!R || s.in_step != 1 || s.os != 1 || s.OWl * 8 < 7 * 8 * tiles_w8) return false;
  dw0 = dh0 = 1 << 20;
  for (int i = 0; i < s.ntaps; ++i) { dw0 = std::min(dw0, s.dw[i]); dh0 = std::min(dh0, s.dh[i]); }
  bool seen[16] = {};
  for (int i = 0; i < s.ntaps; ++i) {
    const int dx = s.dw[i] - dw0, dy = s.dh[i] - dh0;
    if (dx < 0 || dx >= R || dy < 0 || dy >= R || seen[dy * R + dx]) return false;
    seen[dy * R + dx] = true;
    tapw[dy * R + dx] = s.widx[i];
  }
  BW = 8;
  if (8 * s.OHl <= 64) {
    BH = s.OHl;
    BNI = std::min(s.aN, 128 / (8 * BH));
  } else {
    BNI = 1;
    BH = std::min(s.OHl, 16);
    const int th = (s.OHl + BH - 1) / BH;
    BH = (s.OHl + th - 1) / th;
  }
  return BH >= 2 && 8 * BH * BNI >= 96;
}
static bool pick_halo_box(const TcGemmSpec& s, int& BW, int& BH, int& BNI, int tapw3[3][3]) {
  int R, dw0, dh0, tapw[16];
  if (!pick_halo_box_r(s, BW, BH, BNI, R, dw0, dh0, tapw) || R != 3 || dw0 != -1 || dh0 != -1) return false;
  for (int dy = 0; dy < 3; ++dy)
    for (int dx = 0; dx < 3; ++dx) tapw3[dx][dy] = tapw[dy * 3 + dx];
  return true;
}

static int encode_act_map_halo(CUtensorMap* m, const void* base, int N, int H, int W, int C, int boxC, int boxW, int BH,
                               int BNI, int row_bytes, int halo = 2) {
  // dimension order (C, W, image, H): the image row is the slowest coordinate of the box
  cuuint64_t dims[4] = {(cuuint64_t)C, (cuuint64_t)W, (cuuint64_t)N, (cuuint64_t)H};
  cuuint64_t strides[3] = {(cuuint64_t)C * 2, (cuuint64_t)H * W * C * 2, (cuuint64_t)W * C * 2};
  cuuint32_t box[4] = {(cuuint32_t)boxC, (cuuint32_t)boxW, (cuuint32_t)BNI, (cuuint32_t)(BH + halo)};
  cuuint32_t es[4] = {1, 1, 1, 1};
  const CUtensorMapSwizzle sw = row_bytes == 128 ? CU_TENSOR_MAP_SWIZZLE_128B
                                : row_bytes == 64 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_32B;
  CUresult r = cur_dev().encode(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, es,
                            CU_TENSOR_MAP_INTERLEAVE_NONE, sw, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? LP_OK : LP_ERR_CUDA;
}

// Launch with a cluster of two CTAs and programmatic stream serialisation allowed.
template <typename... KArgs, typename... Args>
static inline cudaError_t launch_pdl_pair(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                                          Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = LP_PDL;
  attr[1].id = cudaLaunchAttributeClusterDimension;
  attr[1].val.clusterDim.x = 2;
  attr[1].val.clusterDim.y = 1;
  attr[1].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// 3x3 stride-1 convolutions with 64-channel K chunks on CTA pairs (conv_tc2.cuh).  Returns LP_ERR_UNSUPPORTED
// when the shape is not one this kernel takes (the caller then uses the one-CTA kernel).
static int launch_conv_tc2(lp_handle* h, const TcGemmSpec& s, int* dev_err, cudaStream_t st) {
  Device& D = cur_dev();
  tc::ConvTcParams p;
  memset(&p, 0, sizeof(p));
  p.Nimg = s.aN; p.OHl = s.OHl; p.OWl = s.OWl;
  int tapw3[3][3];
  if (s.x_next || s.os != 1 || s.oo_h || s.oo_w || pick_kc(s.aC) != 64 || !pick_halo_box(s, p.BW, p.BH, p.BNI, tapw3))
    return LP_ERR_UNSUPPORTED;
  p.halo = 1;
  p.tiles_w = (s.OWl + p.BW - 1) / p.BW;
  p.tiles_h = (s.OHl + p.BH - 1) / p.BH;
  p.m_tiles = p.tiles_w * p.tiles_h * ((s.aN + p.BNI - 1) / p.BNI);
  pick_n_tile(s.w_rows, p.n_tile_cols, p.n_tiles);
  if (p.n_tile_cols % 16 || p.n_tile_cols < 32) return LP_ERR_UNSUPPORTED;
  p.total_tiles = p.m_tiles * p.n_tiles;
  if (p.m_tiles < 4) return LP_ERR_UNSUPPORTED;     // too few pixel tiles to form units
  p.in_step = 1;
  p.out_H = s.out_H; p.out_W = s.out_W; p.out_C = s.out_C;
  p.os = 1;
  p.Cout = s.w_rows;
  p.ntaps = 9;
  p.Cin = s.aC;
  p.KC = 64;
  p.chunks = (s.aC + 63) / 64;
  p.nk_last = (s.aC - (p.chunks - 1) * 64 + 15) / 16;
  const int row_bytes = 128;
  const int n_half = p.n_tile_cols / 2;
  const uint32_t b_half = (uint32_t)align_up((size_t)n_half * row_bytes, 1024);
  const size_t tail = tc::kTailBytes + (s.stats ? sizeof(tc::TcStatScratch) : 0) + 1024;
  p.tx_b = (uint32_t)(n_half * row_bytes);
  p.acc_stride = (p.n_tile_cols + 31) / 32 * 32;
  p.nslots = std::min(tc::kMaxSlots, tc::kTmemCols / p.acc_stride);
  if (p.nslots < 2) return LP_ERR_UNSUPPORTED;
  const int halo_rows = kHaloBoxW * p.BNI * (p.BH + 2);
  p.a_halo_bytes = (uint32_t)align_up((size_t)halo_rows * row_bytes, 1024);
  for (int dy = 0; dy < 3; ++dy)
    for (int dx = 0; dx < 3; ++dx) {
      p.tap_widx9[dy * 3 + dx] = tapw3[dx][dy];
      p.tap_off9[dy * 3 + dx] = (uint32_t)((dy * kHaloBoxW * p.BNI + dx) * row_bytes);
    }
  p.desc_hi_a = tc::smem_desc_hi(16, kHaloBoxW * row_bytes, tc::swizzle_code_for_row_bytes(row_bytes));
  p.desc_hi = tc::smem_desc_hi(16, 8 * row_bytes, tc::swizzle_code_for_row_bytes(row_bytes));
  p.tx_a = (uint32_t)(halo_rows * row_bytes);
  p.nA = 2;
  p.mpair = 2;
  p.a_stage_bytes = 2 * p.a_halo_bytes;
  const size_t a_bytes = (size_t)p.nA * p.a_stage_bytes;
  if (a_bytes + 3 * (size_t)b_half + tail > kTcMaxSmem) return LP_ERR_UNSUPPORTED;
  // taps per weight stage: as many (of at most LP_CONV2_TAPS_PER_STAGE) as leave three stages, as in the one-CTA kernel
  p.b_tile_bytes = b_half;
  p.tps = 1;
  for (int tps = LP_CONV2_TAPS_PER_STAGE; tps > 1; --tps)
    if ((kTcMaxSmem - tail - a_bytes) / ((size_t)tps * b_half) >= 3) { p.tps = tps; break; }
  p.b_stage_bytes = p.tps * b_half;
  p.nB = (int)std::min<size_t>((kTcMaxSmem - tail - a_bytes) / p.b_stage_bytes, tc::kMaxStages);
  p.b_ring_offset = (uint32_t)a_bytes;
  p.tail_offset = p.b_ring_offset + p.nB * p.b_stage_bytes;
  p.stage_offset = p.tail_offset;
  p.idesc = tc::instr_desc_bf16(256, p.n_tile_cols, 0, 0);
  p.out = s.out; p.addend = s.addend; p.stats = s.stats; p.err = dev_err;
  p.wide32 = (s.out_C % 16 == 0 && s.w_rows % 16 == 0 && p.n_tile_cols % 16 == 0 &&
              (reinterpret_cast<uintptr_t>(s.out) & 31) == 0 &&
              (!s.addend || (reinterpret_cast<uintptr_t>(s.addend) & 31) == 0)) ? 1 : 0;
  CUtensorMap tmA, tmB;
  int rc = encode_act_map_halo(&tmA, s.act, s.aN, s.aH, s.aW, s.aC, 64, kHaloBoxW, p.BH, p.BNI, row_bytes);
  if (rc != LP_OK) return rc;
  rc = encode_mat_map(&tmB, s.wmat, s.w_K, s.w_rows, 64, n_half, row_bytes);
  if (rc != LP_OK) return rc;
  const size_t smem = std::max((size_t)p.tail_offset + tail, kTcMinSmem);
  if (!D.conv2_attr) {
    LP_CUDA_OK(cudaFuncSetAttribute(tc::conv_tc2_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kTcMaxSmem));
    LP_CUDA_OK(cudaFuncSetAttribute(tc::conv_tc2_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kTcMaxSmem));
    // how many CTA pairs fit the device at once (persistent kernel: never more pairs than that)
    cudaLaunchConfig_t q = {};
    q.gridDim = dim3(2 * D.sm_count);
    q.blockDim = dim3(tc::kConvThreads);
    q.dynamicSmemBytes = kTcMaxSmem;
    cudaLaunchAttribute qa[1];
    qa[0].id = cudaLaunchAttributeClusterDimension;
    qa[0].val.clusterDim.x = 2; qa[0].val.clusterDim.y = 1; qa[0].val.clusterDim.z = 1;
    q.attrs = qa;
    q.numAttrs = 1;
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, tc::conv_tc2_kernel<false>, &q) != cudaSuccess) { cudaGetLastError(); n = 0; }
    D.max_pairs = n;
    D.conv2_attr = true;
  }
  if (D.max_pairs < 1) return LP_ERR_UNSUPPORTED;
  // persistent CTA pairs over contiguous tile ranges; side by side with other modules the smallest number of
  // pairs whose busiest one has no more units of four tiles (see launch_conv_tc)
  int pairs = std::max(1, std::min(D.max_pairs, p.total_tiles / 2));
  // a pair whose tile range crosses a channel-tile boundary works on two short units instead of one: with
  // several channel tiles, a number of pairs that the channel tiles divide keeps every range inside one
  if (p.n_tiles > 1 && pairs >= p.n_tiles) pairs = pairs / p.n_tiles * p.n_tiles;
  if (h && h->concurrent) {
    int per = (p.total_tiles + pairs - 1) / pairs;
    per = (per + 3) / 4 * 4;
    pairs = (p.total_tiles + per - 1) / per;
  }
  cudaError_t le;
  const dim3 g3(2 * pairs), b3(tc::kConvThreads);
  if (s.addend) le = launch_pdl_pair(tc::conv_tc2_kernel<true>, g3, b3, smem, st, tmA, tmB, p);
  else le = launch_pdl_pair(tc::conv_tc2_kernel<false>, g3, b3, smem, st, tmA, tmB, p);
  LP_CUDA_OK(le);
  if (h) h->launches++;
  LP_CUDA_OK(cudaGetLastError());
  return LP_OK;
}

static int launch_conv_tc(lp_handle* h, const TcGemmSpec& s, int* dev_err, cudaStream_t st, bool allow_thin = true) {
  const bool bnbwd = s.bwd_x != nullptr;
  if (bnbwd && (s.stats || s.x_next)) return LP_ERR_UNSUPPORTED;
  if (s.two_cta && !bnbwd) {
    const int rc2 = launch_conv_tc2(h, s, dev_err, st);
    if (rc2 != LP_ERR_UNSUPPORTED) return rc2;
  }
  tc::ConvTcParams p;
  memset(&p, 0, sizeof(p));
  p.Nimg = s.aN; p.OHl = s.OHl; p.OWl = s.OWl;
  int tapw[16], halo_R = 3;
  // (any K chunk width: the row-shifted operand descriptors only need the swizzle to be a function of the
  // shared-memory address, which holds for 32-, 64- and 128-byte rows alike)
  p.halo = (s.n_cls <= 1 && pick_halo_box_r(s, p.BW, p.BH, p.BNI, halo_R, p.halo_dw0, p.halo_dh0, tapw)) ? 1 : 0;
  const int halo_w = 8 + halo_R - 1;   // box width: the 8-pixel tile plus the taps' reach
  if (!p.halo) pick_pixel_box(s.OWl, s.OHl, s.aN, p.BW, p.BH, p.BNI);
  p.tiles_w = (s.OWl + p.BW - 1) / p.BW;
  p.tiles_h = (s.OHl + p.BH - 1) / p.BH;
  const int tiles_n = (s.aN + p.BNI - 1) / p.BNI;
  p.m_tiles = p.tiles_w * p.tiles_h * tiles_n;
  pick_n_tile(s.w_rows, p.n_tile_cols, p.n_tiles);
  p.n_cls = std::max(1, s.n_cls);
  int max_cls_taps = s.ntaps;
  if (s.n_cls > 1) {
    max_cls_taps = 0;
    for (int i = 0; i < s.n_cls; ++i) {
      p.cls_ntaps[i] = s.cls_ntaps[i]; p.cls_tap0[i] = s.cls_tap0[i];
      p.cls_oo_h[i] = s.cls_oo_h[i]; p.cls_oo_w[i] = s.cls_oo_w[i];
      max_cls_taps = std::max(max_cls_taps, s.cls_ntaps[i]);
    }
  } else {
    p.cls_ntaps[0] = s.ntaps; p.cls_tap0[0] = 0; p.cls_oo_h[0] = s.oo_h; p.cls_oo_w[0] = s.oo_w;
  }
  p.total_tiles = p.m_tiles * p.n_tiles * p.n_cls;
  p.in_step = s.in_step;
  p.out_H = s.out_H; p.out_W = s.out_W; p.out_C = s.out_C;
  p.os = s.os; p.oo_h = s.oo_h; p.oo_w = s.oo_w;
  p.Cout = s.w_rows;
  p.ntaps = s.ntaps;
  for (int i = 0; i < s.ntaps; ++i) { p.tap_dh[i] = s.dh[i]; p.tap_dw[i] = s.dw[i]; p.tap_w[i] = s.widx[i]; }
  p.Cin = s.aC;
  p.KC = pick_kc(s.aC);
  p.chunks = (s.aC + p.KC - 1) / p.KC;
  p.nk_last = (s.aC - (p.chunks - 1) * p.KC + 15) / 16;
  const int row_bytes = p.KC * 2;
  p.a_region_bytes = (uint32_t)align_up((size_t)128 * row_bytes, 1024);
  const uint32_t b_region = (uint32_t)align_up((size_t)p.n_tile_cols * row_bytes, 1024);
  // Staged epilogue (output tile through shared memory, TMA stores, TMA-loaded residual): where the output
  // grid is the logical grid, the channel tile is a multiple of 32 and the tensors start on 16-byte boundaries.
  const bool staged0 = !bnbwd && (s.epilogue == 2 || (s.epilogue == 0 && s.addend != nullptr)) && !s.x_next && s.os == 1 && s.oo_h == 0 && s.oo_w == 0 &&
                      p.n_tile_cols % 32 == 0 && s.out_C % 8 == 0 && tc::kEpiThreads == 128 &&
                      (reinterpret_cast<uintptr_t>(s.out) & 15) == 0 &&
                      (!s.addend || (reinterpret_cast<uintptr_t>(s.addend) & 15) == 0);
  // Layers of few channels, while the modules are enqueued side by side: the two-per-SM instantiation with
  // half an SM's shared memory at most and tensor memory sized to need, so that kernels of several modules share
  // the SMs (each such kernel is bound by latency: a few hundred MFLOP and a few MB per launch).
  const bool thin = allow_thin && h && h->concurrent && !bnbwd && !s.x_next && p.n_tile_cols <= 64 &&
                    2.0 * s.aN * s.OHl * s.OWl * (double)s.w_rows * s.ntaps * s.aC < kSmallConvFlops;
  const bool staged = staged0 && !thin;
  const size_t max_smem = thin ? kTcThinSmem : kTcMaxSmem;
  const size_t stage_bytes = staged ? (size_t)(p.n_tile_cols / 32) * tc::kStageGroupBytes : 0;
  // the direct epilogue's statistics scratch is only there when statistics are asked for
  const size_t tail = tc::kTailBytes + ((staged || !(s.stats || bnbwd)) ? 0 : sizeof(tc::TcStatScratch)) +
                      (bnbwd ? sizeof(tc::TcBnBwdScratch) : 0) + stage_bytes + 1024;
  p.tx_b = (uint32_t)(p.n_tile_cols * row_bytes);
  p.acc_stride = (p.n_tile_cols + 31) / 32 * 32;
  p.nslots = std::min(tc::kMaxSlots, (thin ? 256 : tc::kTmemCols) / p.acc_stride);
  p.tmem_cols = tc::kTmemCols;
  if (thin) {
    p.tmem_cols = 32;
    while (p.tmem_cols < p.nslots * p.acc_stride) p.tmem_cols *= 2;
  }
  if (p.halo) {
    // activation ring: three boxes deep if at least three weight stages still fit, else two
    const int halo_rows = halo_w * p.BNI * (p.BH + halo_R - 1);
    p.a_halo_bytes = (uint32_t)align_up((size_t)halo_rows * row_bytes, 1024);
    for (int dy = 0; dy < halo_R; ++dy)
      for (int dx = 0; dx < halo_R; ++dx) {
        p.tap_widx9[dy * halo_R + dx] = tapw[dy * halo_R + dx];
        p.tap_off9[dy * halo_R + dx] = (uint32_t)((dy * halo_w * p.BNI + dx) * row_bytes);
      }
    // 8-row groups of the operand are one box row (halo_w pixels) apart
    p.desc_hi_a = tc::smem_desc_hi(16, halo_w * row_bytes, tc::swizzle_code_for_row_bytes(row_bytes));
    p.b_tile_bytes = b_region;
    p.tx_a = (uint32_t)(halo_rows * row_bytes);
    const size_t avail = max_smem - tail;
    // two activation stages (each lasts all nine taps), the rest of shared memory for weights: stages of
    // as many taps as leave three of them (all nine for layers of 16 or 32 channels, two at 160)
    bool fits = false;
    p.nA = 2;
    for (int pair = (p.m_tiles >= 2 && 2 * p.total_tiles >= 3 * std::min(p.total_tiles, cur_dev().sm_count)) ? 2 : 1;
         pair >= 1 && !fits; --pair) {
      const size_t a_bytes = (size_t)p.nA * pair * p.a_halo_bytes;
      if (a_bytes >= avail) continue;
      for (int tps = std::min(LP_CONV_TAPS_PER_STAGE, s.ntaps); tps >= 1 && !fits; --tps) {
        const int nb = (int)std::min<size_t>((avail - a_bytes) / ((size_t)tps * b_region), LP_CONV_MAX_NB);
        if (nb >= 3) { p.mpair = pair; p.nB = nb; p.tps = tps; fits = true; }
      }
    }
    p.b_stage_bytes = p.tps * b_region;
    if (fits) {
      p.a_stage_bytes = p.mpair * p.a_halo_bytes;
      p.b_ring_offset = p.nA * p.a_stage_bytes;
      p.stage_offset = p.b_ring_offset + p.nB * p.b_stage_bytes;
      p.tail_offset = p.stage_offset + (uint32_t)stage_bytes;
    } else {
      p.halo = 0;
      pick_pixel_box(s.OWl, s.OHl, s.aN, p.BW, p.BH, p.BNI);
      p.tiles_w = (s.OWl + p.BW - 1) / p.BW;
      p.tiles_h = (s.OHl + p.BH - 1) / p.BH;
      p.m_tiles = p.tiles_w * p.tiles_h * ((s.aN + p.BNI - 1) / p.BNI);
      p.total_tiles = p.m_tiles * p.n_tiles * p.n_cls;
    }
  }
  if (!p.halo) {
    // two pixel tiles per weight tile wherever a CTA has at least two tiles and three stages still fit
    p.mpair = 1;
    if (p.m_tiles >= 2 && 2 * p.total_tiles >= 3 * std::min(p.total_tiles, cur_dev().sm_count) &&
        (max_smem - tail) / (2 * p.a_region_bytes + b_region) >= 3)
      p.mpair = 2;
    p.b_offset = p.mpair * p.a_region_bytes;
    p.item_bytes = p.b_offset + b_region;
    p.tx_a = (uint32_t)(p.BW * p.BH * p.BNI * row_bytes);
    // Items (one tap of one K chunk) per pipeline stage: as many as leave three stages, spread evenly over the
    // stages of a tile.  Layers with few channels (16 or 32: an item is one or two instructions) then pay the
    // fixed cost of a stage once per several taps; wide layers keep one item per stage.
    {
      const int kiters = max_cls_taps * p.chunks;   // (of the class with the most taps)
      int ips = (int)std::min<size_t>((size_t)std::min(kiters, LP_CONV_MAX_ITEMS_PER_STAGE), (max_smem - tail) / 3 / p.item_bytes);
      ips = std::max(ips, 1);
      const int n_st = (kiters + ips - 1) / ips;
      p.ips = (kiters + n_st - 1) / n_st;
    }
    p.stage_bytes = p.ips * p.item_bytes;
    int stages = (int)((max_smem - tail) / p.stage_bytes);
    stages = std::min(stages, tc::kMaxStages);
    if (stages < 2) return thin ? launch_conv_tc(h, s, dev_err, st, false) : LP_ERR_UNSUPPORTED;
    p.stages = stages;
    p.stage_offset = (uint32_t)(stages * p.stage_bytes);
    p.tail_offset = p.stage_offset + (uint32_t)stage_bytes;
  }
  p.fd_tiles_w = tc::make_fastdiv(p.tiles_w); p.fd_tiles_h = tc::make_fastdiv(p.tiles_h);
  p.fd_m_tiles = tc::make_fastdiv(p.m_tiles); p.fd_n_tiles = tc::make_fastdiv(p.n_tiles);
  p.fd_chunks = tc::make_fastdiv(p.chunks);
  p.idesc = tc::instr_desc_bf16(128, p.n_tile_cols, 0, 0);
  p.desc_hi = tc::smem_desc_hi(16, 8 * row_bytes, tc::swizzle_code_for_row_bytes(row_bytes));
  p.out = s.out; p.addend = s.addend; p.stats = s.stats; p.err = dev_err;
  p.x_next = s.x_next; p.kappa = s.kappa; p.r_out = s.r_out; p.seed_out = s.seed_out; p.rho = s.rho;
  p.loss_acc = s.loss_acc;
  p.bwd_x = s.bwd_x; p.bwd_bn = s.bwd_bn; p.bwd_dgamma = s.bwd_dgamma; p.bwd_dbeta = s.bwd_dbeta; p.bwd_relu = s.bwd_relu;
  // 32-byte epilogue accesses: rows and channel-group offsets are multiples of 32 bytes when the channel
  // count is a multiple of 16 and the tensors start on a 32-byte boundary (caller buffers need only 16)
  p.wide32 = (s.out_C % 16 == 0 && s.w_rows % 16 == 0 && p.n_tile_cols % 16 == 0 &&
              (reinterpret_cast<uintptr_t>(s.out) & 31) == 0 &&
              (!s.addend || (reinterpret_cast<uintptr_t>(s.addend) & 31) == 0)) ? 1 : 0;
  CUtensorMap tmA, tmB;
  int rc = p.halo ? encode_act_map_halo(&tmA, s.act, s.aN, s.aH, s.aW, s.aC, p.KC, halo_w, p.BH, p.BNI, row_bytes, halo_R - 1)
                  : encode_act_map(&tmA, s.act, s.aN, s.aH, s.aW, s.aC, p.KC, p.BW, p.BH, p.BNI, s.in_step, row_bytes);
  if (rc != LP_OK) return rc;
  rc = encode_mat_map(&tmB, s.wmat, s.w_K, s.w_rows, p.KC, p.n_tile_cols, row_bytes);
  if (rc != LP_OK) return rc;
  CUtensorMap tmOut, tmAdd;
  memset(&tmOut, 0, sizeof(tmOut));
  memset(&tmAdd, 0, sizeof(tmAdd));
  if (staged) {
    rc = encode_tile32_map(&tmOut, s.out, s.aN, s.out_H, s.out_W, s.out_C, p.BW, p.BH, p.BNI, p.halo != 0);
    if (rc != LP_OK) return rc;
    if (s.addend) {
      rc = encode_tile32_map(&tmAdd, s.addend, s.aN, s.out_H, s.out_W, s.out_C, p.BW, p.BH, p.BNI, p.halo != 0);
      if (rc != LP_OK) return rc;
    }
  }
  size_t smem = (size_t)p.tail_offset + (tail - stage_bytes);
  if (!thin) smem = std::max(smem, kTcMinSmem);
  bool& attr_set = cur_dev().conv_attr;
  if (!attr_set) {
    LP_CUDA_OK(cudaFuncSetAttribute(tc::conv_tc_kernel<false, false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                    (int)kTcMaxSmem));
    LP_CUDA_OK(cudaFuncSetAttribute(tc::conv_tc_kernel<false, true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                    (int)kTcMaxSmem));
    LP_CUDA_OK(cudaFuncSetAttribute(tc::conv_tc_kernel<true, true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                    (int)kTcMaxSmem));
    LP_CUDA_OK(cudaFuncSetAttribute(tc::conv_tc_kernel<false, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                    (int)kTcMaxSmem));
    LP_CUDA_OK(cudaFuncSetAttribute(tc::conv_tc_kernel<false, true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                    (int)kTcMaxSmem));
    LP_CUDA_OK(cudaFuncSetAttribute(tc::conv_tc_kernel<false, false, false, false, 2>,
                                    cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kTcThinSmem));
    LP_CUDA_OK(cudaFuncSetAttribute(tc::conv_tc_kernel<false, true, false, false, 2>,
                                    cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kTcThinSmem));
    LP_CUDA_OK(cudaFuncSetAttribute(tc::conv_tc_kernel<false, false, false, true>,
                                    cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kTcMaxSmem));
    LP_CUDA_OK(cudaFuncSetAttribute(tc::conv_tc_kernel<false, true, false, true>,
                                    cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kTcMaxSmem));
    attr_set = true;
  }
  // Persistent CTAs walk contiguous tile ranges; the launch takes about as long as the CTA with the most
  // units (pairs of tiles).  While the K modules are enqueued side by side, the smallest grid with that
  // same maximum is used (1024 tiles: 128 CTAs of four pairs instead of 148 of three pairs and a single
  // tile): the freed SMs go to the kernels of the other modules' streams and the freed power to the
  // clock (step 5.21 -> 5.07 ms).  A module running alone keeps one CTA per SM, which is a few per
  // cent faster for the launch itself.
  int grid = std::min(p.total_tiles, cur_dev().sm_count);
  if (h && h->concurrent) {
    int per = (p.total_tiles + grid - 1) / grid;
    if (p.mpair == 2) per = (per + 1) / 2 * 2;
    grid = (p.total_tiles + per - 1) / per;
  }
  if (s.x_next && !s.addend) return LP_ERR_UNSUPPORTED;   // the fused loss belongs to a convolution with a shortcut
  cudaError_t le;
  const dim3 g3(grid), b3(tc::kConvThreads);
  if (thin && s.addend) le = launch_pdl(tc::conv_tc_kernel<false, true, false, false, 2>, g3, b3, smem, st, tmA, tmB, tmOut, tmAdd, p);
  else if (thin) le = launch_pdl(tc::conv_tc_kernel<false, false, false, false, 2>, g3, b3, smem, st, tmA, tmB, tmOut, tmAdd, p);
  else if (bnbwd && s.addend) le = launch_pdl(tc::conv_tc_kernel<false, true, false, true>, g3, b3, smem, st, tmA, tmB, tmOut, tmAdd, p);
  else if (bnbwd) le = launch_pdl(tc::conv_tc_kernel<false, false, false, true>, g3, b3, smem, st, tmA, tmB, tmOut, tmAdd, p);
  else if (s.x_next) le = launch_pdl(tc::conv_tc_kernel<true, true, false>, g3, b3, smem, st, tmA, tmB, tmOut, tmAdd, p);
  else if (staged && s.addend) le = launch_pdl(tc::conv_tc_kernel<false, true, true>, g3, b3, smem, st, tmA, tmB, tmOut, tmAdd, p);
  else if (staged) le = launch_pdl(tc::conv_tc_kernel<false, false, true>, g3, b3, smem, st, tmA, tmB, tmOut, tmAdd, p);
  else if (s.addend) le = launch_pdl(tc::conv_tc_kernel<false, true, false>, g3, b3, smem, st, tmA, tmB, tmOut, tmAdd, p);
  else le = launch_pdl(tc::conv_tc_kernel<false, false, false>, g3, b3, smem, st, tmA, tmB, tmOut, tmAdd, p);
  LP_CUDA_OK(le);
  if (h) h->launches++;
  LP_CUDA_OK(cudaGetLastError());
  return LP_OK;
}

static bool tc_fwd_ok(const ConvDef& c) {
  return c.cin % 8 == 0 && c.cout % 8 == 0 && (c.R == 1 || c.R == 3) && (c.stride == 1 || c.stride == 2);
}
static bool tc_dgrad_ok(const ConvDef& c) {
  return tc_fwd_ok(c) && (c.stride == 1 || (c.H % 2 == 0 && c.W % 2 == 0));
}
// A stride-2 input gradient runs as one launch per parity class of the input pixels; a class that no
// filter tap reaches (1x1 filters) is not written by any epilogue.
static bool dgrad_has_empty_class(const ConvDef& c) {
  for (int ph = 0; ph < c.stride; ++ph) {
    int cnt = 0;
    for (int r = 0; r < c.R; ++r) cnt += ((ph + c.pad - r) % c.stride == 0) ? 1 : 0;
    if (cnt == 0) return true;
  }
  return false;
}
static bool tc_wgrad_ok(const ConvDef& c) {
  return c.cin % 8 == 0 && c.cout % 8 == 0 && (c.R == 1 || c.R == 3) && (c.stride == 1 || c.stride == 2);
}

static bool s2d_stem_ok(const ConvDef& c) {
  return c.R == 7 && c.stride == 2 && c.pad == 3 && c.cin >= 1 && c.cin <= 4 && c.cout % 8 == 0 && c.H % 2 == 0 &&
         c.W % 2 == 0 && c.H >= 8 && c.W >= 8;
}

// Local loss of an interior module computed by the epilogue of the module's last convolution.
struct LossFuse {
  const void* x_next; const void* kappa; void* r_out; void* seed_out; float rho; double* acc;
};

// Reduction pass of the batch-norm backward that consumes an input gradient, taken by the epilogue
// of the convolution that writes it.
struct BnBwdFuse {
  const void* x; BnArgs bn; float* dgamma; float* dbeta; int relu;
};

struct ProfScope {
  lp_handle* h; cudaStream_t st; double flops; bool on = false; size_t idx = 0;
  ProfScope(lp_handle* h_, cudaStream_t st_, double fl) : h(h_), st(st_), flops(fl) {
    if (!h || !h->prof.enabled) return;
    ConvProfile& pr = h->prof;
    if (pr.used == pr.events.size()) {
      cudaEvent_t a, b;
      if (cudaEventCreate(&a) != cudaSuccess || cudaEventCreate(&b) != cudaSuccess) return;
      pr.events.push_back({a, b});
      pr.flops.push_back(0.0);
    }
    idx = pr.used++;
    pr.flops[idx] = flops;
    cudaEventRecord(pr.events[idx].first, st);
    on = true;
  }
  ~ProfScope() {
    if (on) cudaEventRecord(h->prof.events[idx].second, st);
  }
};

// Output channels per thread of the few-input-channel kernels: the largest of 64, 32, 16, 8 that
// divides C_out (0: not eligible).
static int fewch_cpt(int cout, int dtype) {
  (void)dtype;
  for (int c : {64, 32, 16, 8})
    if (cout % c == 0) return c;
  return 0;
}

// y = conv(x, w) [+ addend]; optional per-channel statistics of y
static int conv_forward(lp_handle* h, int dtype, int impl, const ConvDef& c, int N, const void* x, void* y,
                        const void* addend, double* stats, bool* stats_done, int* dev_err, cudaStream_t st,
                        const LossFuse* loss = nullptr) {
  if (stats_done) *stats_done = false;
  if (c.s2d) {
    // 7x7 / stride-2 stem: regroup the image, then a 4x4 stride-1 tensor-core convolution over 16 channels
    const int H2 = c.H / 2, W2 = c.W / 2;
    const long long pix = (long long)N * H2 * W2;
    s2d_input_kernel<bf16><<<grid_for(pix, 256, cur_dev().sm_count, 8), 256, 0, st>>>((const bf16*)x, c.xs, N, c.H, c.W, c.cin);
    if (h) h->launches++;
    LP_CUDA_OK(cudaGetLastError());
    TcGemmSpec s;
    memset(&s, 0, sizeof(s));
    s.act = c.xs; s.aN = N; s.aH = H2; s.aW = W2; s.aC = 16;
    s.wmat = c.wf; s.w_rows = c.cout; s.w_K = 256;
    s.in_step = 1; s.OHl = c.OH; s.OWl = c.OW;
    s.ntaps = 16;
    for (int i = 0; i < 16; ++i) { s.dh[i] = i / 4 - 2; s.dw[i] = i % 4 - 2; s.widx[i] = i; }
    s.out = (bf16*)y; s.addend = (const bf16*)addend;
    s.out_H = c.OH; s.out_W = c.OW; s.out_C = c.cout; s.os = 1;
    s.stats = stats;
    s.epilogue = (impl & LP_CONV_DIRECT_EPILOGUE) ? 1 : ((impl & LP_CONV_STAGED_EPILOGUE) ? 2 : 0);
    if (stats_done) *stats_done = stats != nullptr;
    ProfScope ps(h, st, 2.0 * N * c.OH * c.OW * (double)c.cout * c.R * c.R * c.cin);
    return launch_conv_tc(h, s, dev_err, st);
  }
  const bool use_tc = dtype == LP_BF16 && (impl & 15) != LP_CONV_IMPL_SIMT && !(impl & 16) && tc_fwd_ok(c) && c.wf;
  if ((impl & 15) == LP_CONV_IMPL_TENSOR && !use_tc) return LP_ERR_UNSUPPORTED;
  if (loss && !use_tc) return LP_ERR_UNSUPPORTED;  // the planner fuses the loss only into tensor-core convolutions
  if (use_tc) {
    TcGemmSpec s;
    memset(&s, 0, sizeof(s));
    s.act = (const bf16*)x; s.aN = N; s.aH = c.H; s.aW = c.W; s.aC = c.cin;
    s.wmat = c.wf; s.w_rows = c.cout; s.w_K = (long long)c.R * c.R * c.cin;
    s.in_step = c.stride; s.OHl = c.OH; s.OWl = c.OW;
    s.ntaps = c.R * c.R;
    for (int r = 0; r < c.R; ++r)
      for (int q = 0; q < c.R; ++q) {
        s.dh[r * c.R + q] = r - c.pad; s.dw[r * c.R + q] = q - c.pad; s.widx[r * c.R + q] = r * c.R + q;
      }
    s.out = (bf16*)y; s.addend = (const bf16*)addend;
    s.out_H = c.OH; s.out_W = c.OW; s.out_C = c.cout; s.os = 1; s.oo_h = s.oo_w = 0;
    s.stats = stats;
    s.epilogue = (impl & LP_CONV_DIRECT_EPILOGUE) ? 1 : ((impl & LP_CONV_STAGED_EPILOGUE) ? 2 : 0);
    s.two_cta = (impl & LP_CONV_TWO_CTA) ? 1 : 0;
    if (loss) {
      s.x_next = (const bf16*)loss->x_next; s.kappa = (const bf16*)loss->kappa; s.r_out = (bf16*)loss->r_out;
      s.seed_out = (bf16*)loss->seed_out; s.rho = loss->rho; s.loss_acc = loss->acc;
    }
    if (stats_done) *stats_done = stats != nullptr;
    ProfScope ps(h, st, 2.0 * N * c.OH * c.OW * (double)c.cout * c.R * c.R * c.cin);
    return launch_conv_tc(h, s, dev_err, st);
  }
  if (c.cout % 4) return LP_ERR_UNSUPPORTED;
  ConvGeom g{N, c.H, c.W, c.cin, c.OH, c.OW, c.cout, c.R, c.R, c.stride, c.pad};
  const size_t few_smem = (size_t)c.R * c.R * c.cin * c.cout * 4;
  const int few_cpt = fewch_cpt(c.cout, dtype);
  if (c.cin <= 4 && !addend && few_cpt && few_smem <= 48 * 1024) {
    // stems and the first AuxNet convolution: filter bank in shared memory
    const long long items = (long long)N * c.OH * c.OW * (c.cout / few_cpt);
    const int fgrid = grid_for(items, 256, cur_dev().sm_count, 8);
#define LP_FEWCH_FWD(CPT)                                                                                      \
    if (dtype == LP_F32)                                                                                       \
      conv_fwd_fewch_kernel<float, CPT><<<fgrid, 256, few_smem, st>>>((const float*)x, c.w, (float*)y, g);       \
    else                                                                                                       \
      conv_fwd_fewch_kernel<bf16, CPT><<<fgrid, 256, few_smem, st>>>((const bf16*)x, c.w, (bf16*)y, g)
    switch (few_cpt) {
      case 64: LP_FEWCH_FWD(64); break;
      case 32: LP_FEWCH_FWD(32); break;
      case 16: LP_FEWCH_FWD(16); break;
      default: LP_FEWCH_FWD(8); break;
    }
#undef LP_FEWCH_FWD
    if (h) h->launches++;
    LP_CUDA_OK(cudaGetLastError());
    return LP_OK;
  }
  const long long work = (long long)N * c.OH * c.OW * (c.cout / 4);
  const int grid = grid_for(work, 128, cur_dev().sm_count, 16);
  if (dtype == LP_F32)
    conv_fwd_simt_kernel<float><<<grid, 128, 0, st>>>((const float*)x, c.w, (const float*)addend, (float*)y, g);
  else
    conv_fwd_simt_kernel<bf16><<<grid, 128, 0, st>>>((const bf16*)x, c.w, (const bf16*)addend, (bf16*)y, g);
  if (h) h->launches++;
  LP_CUDA_OK(cudaGetLastError());
  return LP_OK;
}

// dx = conv^T(dy, w) [+ addend]   (addend may alias dx)
static int conv_dgrad(lp_handle* h, int dtype, int impl, const ConvDef& c, int N, const void* dy, void* dx,
                      const void* addend, int* dev_err, cudaStream_t st, const BnBwdFuse* bnf = nullptr) {
  const bool use_tc = dtype == LP_BF16 && (impl & 15) != LP_CONV_IMPL_SIMT && !(impl & 32) && tc_dgrad_ok(c) && c.wt;
  if ((impl & 15) == LP_CONV_IMPL_TENSOR && !use_tc) return LP_ERR_UNSUPPORTED;
  if (bnf && (!use_tc || dgrad_has_empty_class(c))) return LP_ERR_UNSUPPORTED;  // the planner fuses only where every pixel passes an epilogue
  if (use_tc) {
    const int st2 = c.stride;
    const int classes = st2 * st2;
    // parity classes with no contributing tap leave dx = addend (or zero)
    bool any_empty = false;
    for (int ph = 0; ph < st2; ++ph) {
      int cnt = 0;
      for (int r = 0; r < c.R; ++r) cnt += ((ph + c.pad - r) % st2 == 0) ? 1 : 0;
      if (cnt == 0) any_empty = true;
    }
    if (any_empty) {
      if (addend && addend != dx) return LP_ERR_UNSUPPORTED;
      if (!addend) LP_CUDA_OK(cudaMemsetAsync(dx, 0, (size_t)N * c.H * c.W * c.cin * 2, st));
    }
    ProfScope ps(h, st, 2.0 * N * c.OH * c.OW * (double)c.cout * c.R * c.R * c.cin);
    if (st2 == 2 && !any_empty && c.H % 2 == 0 && c.W % 2 == 0 && c.R * c.R <= 16) {
      // every parity class has the same logical grid (H/2 x W/2) and only its taps and its offset into dx differ:
      // one launch walks the four classes (tile classes of the kernel) instead of four quarter-size launches
      TcGemmSpec s;
      memset(&s, 0, sizeof(s));
      s.act = (const bf16*)dy; s.aN = N; s.aH = c.OH; s.aW = c.OW; s.aC = c.cout;
      s.wmat = c.wt; s.w_rows = c.cin; s.w_K = (long long)c.R * c.R * c.cout;
      s.in_step = 1;
      s.OHl = c.H / 2; s.OWl = c.W / 2;
      s.n_cls = 4;
      for (int cls = 0; cls < 4; ++cls) {
        const int ph = cls / 2, pw = cls % 2;
        s.cls_tap0[cls] = s.ntaps; s.cls_oo_h[cls] = ph; s.cls_oo_w[cls] = pw;
        for (int r = 0; r < c.R; ++r) {
          if ((ph + c.pad - r) % 2) continue;
          for (int q = 0; q < c.R; ++q) {
            if ((pw + c.pad - q) % 2) continue;
            s.dh[s.ntaps] = (ph + c.pad - r) / 2;
            s.dw[s.ntaps] = (pw + c.pad - q) / 2;
            s.widx[s.ntaps] = r * c.R + q;
            s.ntaps++;
          }
        }
        s.cls_ntaps[cls] = s.ntaps - s.cls_tap0[cls];
      }
      s.out = (bf16*)dx; s.addend = (const bf16*)addend;
      s.out_H = c.H; s.out_W = c.W; s.out_C = c.cin; s.os = 2; s.oo_h = 0; s.oo_w = 0;
      s.epilogue = 1;   // (the staged epilogue needs the output grid to be the logical grid)
      if (bnf) {
        s.bwd_x = (const bf16*)bnf->x; s.bwd_bn = bnf->bn; s.bwd_dgamma = bnf->dgamma; s.bwd_dbeta = bnf->dbeta;
        s.bwd_relu = bnf->relu;
      }
      return launch_conv_tc(h, s, dev_err, st);
    }
    for (int cls = 0; cls < classes; ++cls) {
      const int ph = cls / st2, pw = cls % st2;
      TcGemmSpec s;
      memset(&s, 0, sizeof(s));
      s.act = (const bf16*)dy; s.aN = N; s.aH = c.OH; s.aW = c.OW; s.aC = c.cout;
      s.wmat = c.wt; s.w_rows = c.cin; s.w_K = (long long)c.R * c.R * c.cout;
      s.in_step = 1;
      s.OHl = (c.H - ph + st2 - 1) / st2; s.OWl = (c.W - pw + st2 - 1) / st2;
      s.ntaps = 0;
      for (int r = 0; r < c.R; ++r) {
        if ((ph + c.pad - r) % st2) continue;
        for (int q = 0; q < c.R; ++q) {
          if ((pw + c.pad - q) % st2) continue;
          s.dh[s.ntaps] = (ph + c.pad - r) / st2;
          s.dw[s.ntaps] = (pw + c.pad - q) / st2;
          s.widx[s.ntaps] = r * c.R + q;
          s.ntaps++;
        }
      }
      if (s.ntaps == 0 || s.OHl <= 0 || s.OWl <= 0) continue;
      s.out = (bf16*)dx; s.addend = (const bf16*)addend;
      s.out_H = c.H; s.out_W = c.W; s.out_C = c.cin; s.os = st2; s.oo_h = ph; s.oo_w = pw;
      s.stats = nullptr;
      s.epilogue = (impl & LP_CONV_DIRECT_EPILOGUE) ? 1 : ((impl & LP_CONV_STAGED_EPILOGUE) ? 2 : 0);
      s.two_cta = (impl & LP_CONV_TWO_CTA) ? 1 : 0;
      if (bnf) {
        s.bwd_x = (const bf16*)bnf->x; s.bwd_bn = bnf->bn; s.bwd_dgamma = bnf->dgamma; s.bwd_dbeta = bnf->dbeta;
        s.bwd_relu = bnf->relu;
      }
      int rc = launch_conv_tc(h, s, dev_err, st);
      if (rc != LP_OK) return rc;
    }
    return LP_OK;
  }
  if (c.cin % 4) return LP_ERR_UNSUPPORTED;
  ConvGeom g{N, c.H, c.W, c.cin, c.OH, c.OW, c.cout, c.R, c.R, c.stride, c.pad};
  const long long work = (long long)N * c.H * c.W * (c.cin / 4);
  const int grid = grid_for(work, 128, cur_dev().sm_count, 16);
  if (dtype == LP_F32)
    conv_dgrad_simt_kernel<float><<<grid, 128, 0, st>>>((const float*)dy, c.w, (const float*)addend, (float*)dx, g);
  else
    conv_dgrad_simt_kernel<bf16><<<grid, 128, 0, st>>>((const bf16*)dy, c.w, (const bf16*)addend, (bf16*)dx, g);
  if (h) h->launches++;
  LP_CUDA_OK(cudaGetLastError());
  return LP_OK;
}

// dw += x (*) dy     (dw zeroed by the caller beforehand)
static int conv_wgrad(lp_handle* h, int dtype, int impl, const ConvDef& c, int N, const void* x, const void* dy,
                      float* dw, int* dev_err, cudaStream_t st) {
  if (c.s2d) {
    // weight gradient of the regrouped 4x4 convolution (x is the image: its regrouped copy was kept by the
    // forward pass), then the real filter positions are picked out of it
    LP_CUDA_OK(cudaMemsetAsync(c.dws, 0, (size_t)c.cout * 256 * 4, st));
    Device& D = cur_dev();
    {
      ProfScope ps(h, st, 2.0 * N * c.OH * c.OW * (double)c.cout * c.R * c.R * c.cin);
      int rc = launch_wgrad_tc(D.encode, D.sm_count, &D.wgrad_attr, &D.wgrad_halo_attr, c.xs, (const bf16*)dy, c.dws, N, c.H / 2,
                               c.W / 2, 16, c.OH, c.OW, c.cout, 4, 1, 2, dev_err, st);
      if (h) h->launches++;
      if (rc != LP_OK) return rc;
    }
    const int total = c.cout * 49 * c.cin;
    s2d_unpack_wgrad_kernel<<<grid_for(total, 256, D.sm_count, 8), 256, 0, st>>>(c.dws, dw, c.cout, c.cin);
    if (h) h->launches++;
    LP_CUDA_OK(cudaGetLastError());
    return LP_OK;
  }
  const bool use_tc = dtype == LP_BF16 && (impl & 15) != LP_CONV_IMPL_SIMT && !(impl & 64) && tc_wgrad_ok(c);
  if ((impl & 15) == LP_CONV_IMPL_TENSOR && !use_tc) return LP_ERR_UNSUPPORTED;
  if (use_tc) {
    ProfScope ps(h, st, 2.0 * N * c.OH * c.OW * (double)c.cout * c.R * c.R * c.cin);
    Device& D = cur_dev();
    // small layers of modules that run side by side share the SMs (see kSmallConvFlops)
    const bool shared_sm = h && h->concurrent && c.cin <= 64 && c.cout <= 64 &&
                           2.0 * N * c.OH * c.OW * (double)c.cout * c.R * c.R * c.cin < kSmallConvFlops;
    int rc = launch_wgrad_tc(D.encode, D.sm_count, &D.wgrad_attr, &D.wgrad_halo_attr, (const bf16*)x, (const bf16*)dy, dw, N,
                             c.H, c.W, c.cin, c.OH, c.OW, c.cout, c.R, c.stride, c.pad, dev_err, st, shared_sm);
    if (h) h->launches++;
    return rc;
  }
  ConvGeom g{N, c.H, c.W, c.cin, c.OH, c.OW, c.cout, c.R, c.R, c.stride, c.pad};
  const int n_out = c.cout * c.R * c.R * c.cin;
  const long long npix = (long long)N * c.OH * c.OW;
  const int few_cpt = fewch_cpt(c.cout, dtype);
  if (c.cin <= 4 && few_cpt) {
    const int npairs = c.R * c.R * c.cin * (c.cout / few_cpt);
    if (npairs <= 256) {
      const int pair_threads = (npairs + 31) / 32 * 32;
      int lanes = 256 / pair_threads;   // pixel lanes, as many as 48 KB of reduction scratch allow
      while (lanes > 1 && (size_t)lanes * pair_threads * few_cpt * 4 > 48 * 1024) --lanes;
      const int threads = lanes * pair_threads;
      const size_t red_bytes = lanes > 1 ? (size_t)threads * few_cpt * 4 : 0;
      const long long blocks = std::min<long long>((npix + 63) / 64, 6LL * cur_dev().sm_count);
      const long long ppb = (npix + blocks - 1) / blocks;
      const int fgrid = (int)((npix + ppb - 1) / ppb);
#define LP_FEWCH_WGRAD(CPT)                                                                                    \
      if (dtype == LP_F32)                                                                                     \
        conv_wgrad_fewch_kernel<float, CPT><<<fgrid, threads, red_bytes, st>>>((const float*)x, (const float*)dy, dw, \
                                                                               g, pair_threads, ppb);          \
      else                                                                                                     \
        conv_wgrad_fewch_kernel<bf16, CPT><<<fgrid, threads, red_bytes, st>>>((const bf16*)x, (const bf16*)dy, dw, g, \
                                                                              pair_threads, ppb)
      switch (few_cpt) {
        case 64: LP_FEWCH_WGRAD(64); break;
        case 32: LP_FEWCH_WGRAD(32); break;
        case 16: LP_FEWCH_WGRAD(16); break;
        default: LP_FEWCH_WGRAD(8); break;
      }
#undef LP_FEWCH_WGRAD
      if (h) h->launches++;
      LP_CUDA_OK(cudaGetLastError());
      return LP_OK;
    }
  }
  int chunk = 256;
  while ((npix + chunk - 1) / chunk > 4096) chunk *= 2;
  dim3 grid((n_out + 127) / 128, (unsigned)((npix + chunk - 1) / chunk));
  if (dtype == LP_F32)
    conv_wgrad_simt_kernel<float><<<grid, 128, 0, st>>>((const float*)x, (const float*)dy, dw, g, chunk);
  else
    conv_wgrad_simt_kernel<bf16><<<grid, 128, 0, st>>>((const bf16*)x, (const bf16*)dy, dw, g, chunk);
  if (h) h->launches++;
  LP_CUDA_OK(cudaGetLastError());
  return LP_OK;
}

// ---------------------------------------------------------------------------------------------
// planner
// ---------------------------------------------------------------------------------------------
struct Planner {
  const NetDef& net;
  Arena& A;
  int dtype;
  int impl;
  Planner(const NetDef& n, Arena& a) : net(n), A(a), dtype(n.d.dtype), impl(n.d.conv_impl & 15) {}

  Tensor new_tensor(int n, int h, int w, int c) {
    Tensor t;
    t.n = n; t.h = h; t.w = w; t.c = c;
    t.p = A.alloc((size_t)t.elems() * esize(dtype));
    return t;
  }
  static Tensor like(const Tensor& s, void* p) {
    Tensor t = s;
    t.p = p; t.ext = EXT_NONE;
    return t;
  }

  void alloc_params(Plan& P, int which) {
    uint64_t total = 0;
    net.layout(which, P.ps.layout, &total);
    P.ps.n = (size_t)total;
    P.ps.p = (float*)A.alloc(total * 4);
    P.ps.g = (float*)A.alloc(total * 4);
    P.ps.m = (float*)A.alloc(total * 4);
  }
  const lp_param_entry* find(const Plan& P, const std::string& name) const {
    for (const auto& e : P.ps.layout)
      if (name == e.name) return &e;
    return nullptr;
  }
  int add_conv(Plan& P, const std::string& wname, int cin, int cout, int R, int stride, int pad, int H, int W,
               bool need_dgrad) {
    ConvDef c;
    c.cin = cin; c.cout = cout; c.R = R; c.stride = stride; c.pad = pad; c.H = H; c.W = W;
    c.OH = conv_out(H, R, stride, pad); c.OW = conv_out(W, R, stride, pad);
    const lp_param_entry* e = find(P, wname);
    c.w = P.ps.p + e->offset;
    c.gw = P.ps.g + e->offset;
    c.need_dgrad = need_dgrad;
    if (dtype == LP_BF16 && impl != LP_CONV_IMPL_SIMT && tc_fwd_ok(c)) {
      const size_t n = (size_t)cout * R * R * cin;
      c.wf = (bf16*)A.alloc(n * 2);
      if (need_dgrad && tc_dgrad_ok(c)) c.wt = (bf16*)A.alloc(n * 2);
      PackEntry pe;
      pe.w = c.w; pe.wf = c.wf; pe.wt = c.wt; pe.cout = cout; pe.taps = R * R; pe.cin = cin;
      pe.begin = P.ps.pack_total;
      pe.tile_begin = P.ps.pack_tiles;
      pe.tile64_begin = P.ps.pack_tiles64;
      P.ps.pack_tiles64 += (long long)R * R * ((cin + 63) / 64) * ((cout + 63) / 64);
      if (e->offset % 4 != 0 || cin % 4 != 0 || cout % 2 != 0) P.ps.pack64_ok = false;
      P.ps.pack_total += (long long)n;
      P.ps.pack_tiles += (long long)R * R * ((cin + 31) / 32) * ((cout + 31) / 32);
      P.ps.host_pack.push_back(pe);
    } else if (dtype == LP_BF16 && impl != LP_CONV_IMPL_SIMT && !(net.d.conv_impl & 16) && !(net.d.conv_impl & 64) &&
               !need_dgrad && s2d_stem_ok(c)) {
      c.s2d = true;
      c.wf = (bf16*)A.alloc((size_t)cout * 256 * 2);
      c.dws = (float*)A.alloc((size_t)cout * 256 * 4);
      c.xs = (bf16*)A.alloc((size_t)net.d.N * (H / 2) * (W / 2) * 16 * 2);
    }
    P.convs.push_back(c);
    return (int)P.convs.size() - 1;
  }
  int add_bn(Plan& P, const std::string& prefix, int C, long long count) {
    BnDef b;
    b.C = C; b.count = count;
    const lp_param_entry* g = find(P, prefix + ".g");
    const lp_param_entry* be = find(P, prefix + ".b");
    b.gamma = P.ps.p + g->offset; b.beta = P.ps.p + be->offset;
    b.dgamma = P.ps.g + g->offset; b.dbeta = P.ps.g + be->offset;
    P.bns.push_back(b);
    return (int)P.bns.size() - 1;
  }
  void finish_stats(Plan& P) {
    size_t total = 0;
    for (auto& b : P.bns) total += (size_t)2 * b.C;
    P.stats_bytes = total * sizeof(double);
    double* base = (double*)A.alloc(std::max<size_t>(P.stats_bytes, 16));
    P.stats_region = base;
    size_t off = 0;
    for (auto& b : P.bns) { b.stats = base + off; off += (size_t)2 * b.C; }
    P.loss_acc = (double*)A.alloc(2 * sizeof(double));
    if (!P.ps.host_pack.empty()) {
      P.ps.dev_pack = (PackEntry*)A.alloc(P.ps.host_pack.size() * sizeof(PackEntry));
      // complement of the packed entries in [0, n), cut into ranges of at most 16384 elements
      std::vector<std::pair<long long, long long>> packed;
      for (const PackEntry& e : P.ps.host_pack)
        packed.push_back({(long long)(e.w - P.ps.p), (long long)(e.w - P.ps.p) + (long long)e.cout * e.taps * e.cin});
      std::sort(packed.begin(), packed.end());
      long long pos = 0;
      auto add = [&](long long a, long long b) {
        for (long long q = a; q < b; q += 16384) P.ps.host_ranges.push_back({q, (int)std::min<long long>(16384, b - q)});
      };
      for (const auto& pr : packed) { add(pos, pr.first); pos = pr.second; }
      add(pos, (long long)P.ps.n);
      if (!P.ps.host_ranges.empty()) P.ps.dev_ranges = (SgdRange*)A.alloc(P.ps.host_ranges.size() * sizeof(SgdRange));
    }
  }

  bool conv_fuses_stats(const ConvDef& c) const {
    return dtype == LP_BF16 && impl != LP_CONV_IMPL_SIMT && !(net.d.conv_impl & 16) && (tc_fwd_ok(c) || c.s2d) && c.wf;
  }
  Tensor emit_conv(Plan& P, std::vector<Op>& ops, const Tensor& in, int conv, const Tensor* addend, int stats_bn) {
    const ConvDef& c = P.convs[conv];
    Tensor out = new_tensor(in.n, c.OH, c.OW, c.cout);
    Op op;
    op.type = OP_CONV_FWD; op.in = in; op.out = out; op.conv = conv;
    if (addend) op.addend = *addend;
    const bool fused = stats_bn >= 0 && conv_fuses_stats(c);
    op.stats_bn = fused ? stats_bn : -1;
    ops.push_back(op);
    if (stats_bn >= 0 && !fused) emit_stats(ops, out, stats_bn);
    return out;
  }
  void emit_stats(std::vector<Op>& ops, const Tensor& t, int bn) {
    Op op;
    op.type = OP_BN_STATS; op.in = t; op.bn = bn;
    ops.push_back(op);
  }
  Tensor emit_bn_apply(std::vector<Op>& ops, const Tensor& x, int bn, const Tensor* x2, int bn2, const Tensor* addend,
                       int relu) {
    Tensor out = new_tensor(x.n, x.h, x.w, x.c);
    Op op;
    op.type = OP_BN_APPLY; op.in = x; op.bn = bn; op.relu = relu; op.out = out;
    if (x2) { op.in2 = *x2; op.bn2 = bn2; }
    if (addend) op.addend = *addend;
    ops.push_back(op);
    return out;
  }
  // backward of y = bn(x) (dy optionally masked by a stored post-ReLU tensor); returns dx
  bool dgrad_fuses_bn_bwd(const ConvDef& c) const {
    return (net.d.conv_impl & LP_CONV_BN_REDUCE_IN_EPILOGUE) && dtype == LP_BF16 && impl != LP_CONV_IMPL_SIMT &&
           !(net.d.conv_impl & 32) && tc_dgrad_ok(c) && c.wt && !dgrad_has_empty_class(c);
  }
  Tensor emit_bn_bwd(Plan& P, std::vector<Op>& ops, const Tensor& dy, const Tensor& x, const Tensor* mask, int bn,
                     const Tensor* addend, const Tensor* out_override = nullptr) {
    Tensor out = out_override ? *out_override : new_tensor(x.n, x.h, x.w, x.c);
    Op op;
    op.type = OP_BN_BWD; op.in = dy; op.in2 = x; op.bn = bn; op.out = out;
    // On request (LP_CONV_BN_REDUCE_IN_EPILOGUE): where the last kernel to write dy is a tensor-core input
    // gradient, its epilogue takes this batch norm's reduction pass (one such consumer per convolution).
    for (int i = (int)ops.size() - 1; i >= 0; --i) {
      Op& w = ops[i];
      if (!(w.out.p == dy.p && w.out.ext == dy.ext) || !w.out.defined()) continue;
      if (w.type == OP_CONV_DGRAD && w.bwd_bn < 0 && dgrad_fuses_bn_bwd(P.convs[w.conv])) {
        w.bwd_bn = bn; w.bwd_x = x; w.bwd_relu = mask ? 1 : 0;
        op.reduce_fused = 1;
      }
      break;
    }
    if (mask) op.mask = *mask;
    if (addend) op.addend = *addend;
    ops.push_back(op);
    return out;
  }
  void emit_wgrad(std::vector<Op>& ops, const Tensor& x, const Tensor& dy, int conv) {
    Op op;
    op.type = OP_CONV_WGRAD; op.in = x; op.in2 = dy; op.conv = conv;
    ops.push_back(op);
  }
  Tensor emit_dgrad(Plan& P, std::vector<Op>& ops, const Tensor& dy, int conv, const Tensor* addend,
                    const Tensor* out_override) {
    const ConvDef& c = P.convs[conv];
    Tensor out = out_override ? *out_override : new_tensor(dy.n, c.H, c.W, c.cin);
    Op op;
    op.type = OP_CONV_DGRAD; op.in = dy; op.conv = conv; op.out = out;
    if (addend) op.addend = *addend;
    ops.push_back(op);
    return out;
  }

  struct BlockRec {
    int bi;
    Tensor x, y1, a1, y2, ys, o;  // saved activations (o: pre-activated input, pre-act blocks)
    Tensor a2, y3;                // bottleneck blocks: second activation, third convolution output
    int c1, c2, cs, bn1, bn2, bns;
    int c3 = -1, bn3 = -1;
  };

  void build_module(Plan& P, int k) {
    const lp_net_desc& d = net.d;
    const bool post = d.block_kind != LP_PREACT;
    const bool bott = d.block_kind == LP_BOTTLENECK;
    const bool last = k == net.K - 1;
    P.interior = !last;
    alloc_params(P, k);
    const Shape4 in_shape = net.boundary[k];
    Tensor x;
    x.ext = EXT_X; x.n = in_shape.n; x.h = in_shape.h; x.w = in_shape.w; x.c = in_shape.c;

    // ---- register convolutions and batch norms (so that a producer knows its consumer's BN) ----
    int stem_conv = -1, stem_bn = -1;
    if (k == 0) {
      stem_conv = add_conv(P, "stem.conv.w", d.C_in, d.stem_channels, net.stem_R, net.stem_stride, net.stem_pad, d.H,
                           d.W, false);
      if (post) stem_bn = add_bn(P, "stem.bn", d.stem_channels, (long long)d.N * net.stem_h * net.stem_w);
    }
    std::vector<BlockRec> recs;
    for (int bi = net.mod_begin[k]; bi < net.mod_end[k]; ++bi) {
      const BlockDef& b = net.blocks[bi];
      const std::string q = "block" + std::to_string(bi);
      BlockRec r;
      r.bi = bi; r.cs = -1; r.bns = -1;
      const bool need_dx1 = true;  // every block input is either x_k (dx_k exported) or an internal tensor
      if (bott) {
        r.c1 = add_conv(P, q + ".conv1.w", b.cin, b.mid, 1, 1, 0, b.hin, b.win, need_dx1);
        r.c2 = add_conv(P, q + ".conv2.w", b.mid, b.mid, 3, b.stride, 1, b.hin, b.win, true);
        r.c3 = add_conv(P, q + ".conv3.w", b.mid, b.cout, 1, 1, 0, b.hout, b.wout, true);
      } else {
        r.c1 = add_conv(P, q + ".conv1.w", b.cin, b.cout, 3, b.stride, 1, b.hin, b.win, need_dx1);
        r.c2 = add_conv(P, q + ".conv2.w", b.cout, b.cout, 3, 1, 1, b.hout, b.wout, true);
      }
      if (b.proj) r.cs = add_conv(P, q + ".sc.w", b.cin, b.cout, 1, b.stride, 0, b.hin, b.win, true);
      if (bott) {
        const long long cnt = (long long)d.N * b.hout * b.wout;
        r.bn1 = add_bn(P, q + ".bn1", b.mid, (long long)d.N * b.hin * b.win);
        r.bn2 = add_bn(P, q + ".bn2", b.mid, cnt);
        r.bn3 = add_bn(P, q + ".bn3", b.cout, cnt);
        if (b.proj) r.bns = add_bn(P, q + ".bns", b.cout, cnt);
      } else if (post) {
        const long long cnt = (long long)d.N * b.hout * b.wout;
        r.bn1 = add_bn(P, q + ".bn1", b.cout, cnt);
        r.bn2 = add_bn(P, q + ".bn2", b.cout, cnt);
        if (b.proj) r.bns = add_bn(P, q + ".bns", b.cout, cnt);
      } else {
        r.bn1 = add_bn(P, q + ".bn1", b.cin, (long long)d.N * b.hin * b.win);
        r.bn2 = add_bn(P, q + ".bn2", b.cout, (long long)d.N * b.hout * b.wout);
      }
      recs.push_back(r);
    }
    int head_bn = -1;
    const BlockDef& lastb = net.blocks[net.mod_end[k] - 1];
    if (last) {
      P.has_head = true;
      if (!post) head_bn = add_bn(P, "head.bn", lastb.cout, (long long)d.N * lastb.hout * lastb.wout);
      HeadDef& hd = P.head;
      hd.C = lastb.cout; hd.classes = d.num_classes; hd.HW = lastb.hout * lastb.wout; hd.N = d.N;
      const lp_param_entry* w = find(P, "head.fc.w");
      const lp_param_entry* b = find(P, "head.fc.b");
      hd.W = P.ps.p + w->offset; hd.b = P.ps.p + b->offset;
      hd.dW = P.ps.g + w->offset; hd.db = P.ps.g + b->offset;
      hd.pooled = (float*)A.alloc((size_t)d.N * hd.C * 4);
      hd.logits = (float*)A.alloc((size_t)d.N * hd.classes * 4);
      hd.dlogits = (float*)A.alloc((size_t)d.N * hd.classes * 4);
    }
    finish_stats(P);

    // ---- forward ----
    std::vector<Op>& F = P.fwd;
    Tensor cur = x;
    Tensor stem_y, stem_a, stem_pool_out;
    uint8_t* pool_arg = nullptr;
    if (k == 0) {
      const int first_bn1 = !post ? recs[0].bn1 : -1;
      stem_y = emit_conv(P, F, x, stem_conv, nullptr, post ? stem_bn : first_bn1);
      cur = stem_y;
      if (post) {
        stem_a = emit_bn_apply(F, stem_y, stem_bn, nullptr, -1, nullptr, 1);
        cur = stem_a;
        if (net.stem_pool) {
          stem_pool_out = new_tensor(d.N, net.body_h, net.body_w, d.stem_channels);
          pool_arg = (uint8_t*)A.alloc((size_t)stem_pool_out.elems());
          Op op;
          op.type = OP_MAXPOOL_FWD; op.in = stem_a; op.out = stem_pool_out; op.arg = pool_arg;
          F.push_back(op);
          cur = stem_pool_out;
        }
      }
    } else if (!post) {
      emit_stats(F, x, recs[0].bn1);  // statistics of the module input for the first pre-activation
    }
    const Shape4 out_shape = last ? Shape4{d.N, lastb.hout, lastb.wout, lastb.cout} : net.boundary[k + 1];
    if (!last) {
      P.out = new_tensor(out_shape.n, out_shape.h, out_shape.w, out_shape.c);
      P.r = new_tensor(out_shape.n, out_shape.h, out_shape.w, out_shape.c);
      P.seed = new_tensor(out_shape.n, out_shape.h, out_shape.w, out_shape.c);
    }
    for (size_t i = 0; i < recs.size(); ++i) {
      BlockRec& r = recs[i];
      const BlockDef& b = net.blocks[r.bi];
      const bool final_block = i + 1 == recs.size();
      r.x = cur;
      if (post) {
        r.y1 = emit_conv(P, F, cur, r.c1, nullptr, r.bn1);
        r.a1 = emit_bn_apply(F, r.y1, r.bn1, nullptr, -1, nullptr, 1);
        r.y2 = emit_conv(P, F, r.a1, r.c2, nullptr, r.bn2);
        if (bott) {
          r.a2 = emit_bn_apply(F, r.y2, r.bn2, nullptr, -1, nullptr, 1);
          r.y3 = emit_conv(P, F, r.a2, r.c3, nullptr, r.bn3);
        }
        const Tensor& ylast = bott ? r.y3 : r.y2;   // the branch's last convolution and its batch norm
        const int bnlast = bott ? r.bn3 : r.bn2;
        if (b.proj) r.ys = emit_conv(P, F, cur, r.cs, nullptr, r.bns);
        if (final_block && !last) {
          Op op;
          op.type = OP_OUT_LOSS; op.in = ylast; op.bn = bnlast; op.out = P.out;
          if (b.proj) { op.in2 = r.ys; op.bn2 = r.bns; } else { op.addend = cur; }
          F.push_back(op);
          cur = P.out;
        } else {
          cur = b.proj ? emit_bn_apply(F, ylast, bnlast, &r.ys, r.bns, nullptr, 0)
                       : emit_bn_apply(F, ylast, bnlast, nullptr, -1, &cur, 0);
        }
      } else {
        r.o = emit_bn_apply(F, cur, r.bn1, nullptr, -1, nullptr, 1);
        r.y1 = emit_conv(P, F, r.o, r.c1, nullptr, r.bn2);
        r.a1 = emit_bn_apply(F, r.y1, r.bn2, nullptr, -1, nullptr, 1);
        Tensor sc = cur;
        if (b.proj) { r.ys = emit_conv(P, F, r.o, r.cs, nullptr, -1); sc = r.ys; }
        const int next_bn = !final_block ? recs[i + 1].bn1 : (last ? head_bn : -1);
        Tensor out = emit_conv(P, F, r.a1, r.c2, &sc, next_bn);
        if (final_block && !last) {
          // The module output is this convolution's accumulator plus the shortcut: on request its
          // epilogue also takes the residual against x_{k+1}, the loss sums and the terminal adjoint.
          const bool fuse = (net.d.conv_impl & LP_CONV_LOSS_IN_EPILOGUE) && conv_fuses_stats(P.convs[r.c2]);
          if (fuse) F.back().fuse_loss = 1;
          Op op;
          op.fuse_loss = fuse ? 1 : 0;
          op.type = OP_OUT_LOSS; op.addend = out; op.out = P.out;  // in undefined: output already final
          F.push_back(op);
          P.out = like(P.out, out.p);  // layer-serial mode reads the conv output directly
          cur = out;
        } else {
          cur = out;
        }
      }
    }
    Tensor head_o;
    if (last) {
      Tensor hin = cur;
      if (!post) { head_o = emit_bn_apply(F, cur, head_bn, nullptr, -1, nullptr, 1); hin = head_o; }
      Op op;
      op.type = OP_HEAD_FWD; op.in = hin;
      F.push_back(op);
    }

    // ---- backward ----
    std::vector<Op>& Bw = P.bwd;
    Tensor dcur;
    if (last) {
      Tensor dh = new_tensor(d.N, lastb.hout, lastb.wout, lastb.cout);
      Op op;
      op.type = OP_HEAD_BWD; op.out = dh;
      Bw.push_back(op);
      dcur = dh;
      if (!post) dcur = emit_bn_bwd(P, Bw, dh, cur, &head_o, head_bn, nullptr);
    } else {
      dcur = P.seed;
    }
    Tensor dx_ext;  // gradient with respect to x_k goes to the caller's buffer
    dx_ext.ext = EXT_DX; dx_ext.n = in_shape.n; dx_ext.h = in_shape.h; dx_ext.w = in_shape.w; dx_ext.c = in_shape.c;
    if (k > 0) {
      P.dx_fallback = A.alloc((size_t)dx_ext.elems() * esize(dtype));
      dx_ext.p = P.dx_fallback;
    }
    for (int i = (int)recs.size() - 1; i >= 0; --i) {
      BlockRec& r = recs[i];
      const BlockDef& b = net.blocks[r.bi];
      const bool first_of_module = i == 0 && k > 0;  // its input is x_k: dx goes to the caller
      const Tensor* dx_target = first_of_module ? &dx_ext : nullptr;
      if (post) {
        Tensor dy2;
        if (bott) {
          Tensor dy3 = emit_bn_bwd(P, Bw, dcur, r.y3, nullptr, r.bn3, nullptr);
          emit_wgrad(Bw, r.a2, dy3, r.c3);
          Tensor da2 = emit_dgrad(P, Bw, dy3, r.c3, nullptr, nullptr);
          dy2 = emit_bn_bwd(P, Bw, da2, r.y2, &r.a2, r.bn2, nullptr);
        } else {
          dy2 = emit_bn_bwd(P, Bw, dcur, r.y2, nullptr, r.bn2, nullptr);
        }
        emit_wgrad(Bw, r.a1, dy2, r.c2);
        Tensor da1 = emit_dgrad(P, Bw, dy2, r.c2, nullptr, nullptr);
        Tensor dy1 = emit_bn_bwd(P, Bw, da1, r.y1, &r.a1, r.bn1, nullptr);
        emit_wgrad(Bw, r.x, dy1, r.c1);
        if (b.proj) {
          Tensor dys = emit_bn_bwd(P, Bw, dcur, r.ys, nullptr, r.bns, nullptr);
          emit_wgrad(Bw, r.x, dys, r.cs);
          Tensor dx = emit_dgrad(P, Bw, dy1, r.c1, nullptr, dx_target);
          dcur = emit_dgrad(P, Bw, dys, r.cs, &dx, &dx);
        } else {
          dcur = emit_dgrad(P, Bw, dy1, r.c1, &dcur, dx_target);
        }
      } else {
        emit_wgrad(Bw, r.a1, dcur, r.c2);
        Tensor da1 = emit_dgrad(P, Bw, dcur, r.c2, nullptr, nullptr);
        Tensor dy1 = emit_bn_bwd(P, Bw, da1, r.y1, &r.a1, r.bn2, nullptr);
        emit_wgrad(Bw, r.o, dy1, r.c1);
        Tensor dO = emit_dgrad(P, Bw, dy1, r.c1, nullptr, nullptr);
        if (b.proj) {
          emit_wgrad(Bw, r.o, dcur, r.cs);
          dO = emit_dgrad(P, Bw, dcur, r.cs, &dO, &dO);
        }
        dcur = emit_bn_bwd(P, Bw, dO, r.x, &r.o, r.bn1, b.proj ? nullptr : &dcur, dx_target);
      }
    }
    if (k == 0) {
      Tensor dstem = dcur;
      if (post) {
        if (net.stem_pool) {
          Tensor dpool = new_tensor(stem_a.n, stem_a.h, stem_a.w, stem_a.c);
          Op op;
          op.type = OP_MAXPOOL_BWD; op.in = dcur; op.out = dpool; op.arg = pool_arg;
          Bw.push_back(op);
          dstem = dpool;
        }
        dstem = emit_bn_bwd(P, Bw, dstem, stem_y, &stem_a, stem_bn, nullptr);
      }
      emit_wgrad(Bw, x, dstem, stem_conv);
    }
  }

  // AuxNet_k of the serial chain: x_k (the images for k = 0) -> x_{k+1}
  void build_aux(Plan& P, int k) {
    Tensor x;
    x.ext = k == 0 ? EXT_IMAGES : EXT_XOUT0 + (k - 1);
    const Shape4 s = net.boundary[k];
    x.n = s.n; x.h = s.h; x.w = s.w; x.c = s.c;
    build_aux_unit(P, k, k, x, true, nullptr);
  }
  // Stack k of the recursive form: units j = 0..k-1, the first fed by the images, the last writing x_k;
  // in the backward pass unit j+1 hands the adjoint of its input to unit j as its seed.
  void build_reaux_stack(std::vector<Plan>& plans, int k) {
    Tensor cur;
    cur.ext = EXT_IMAGES;
    const Shape4 s0 = net.boundary[0];
    cur.n = s0.n; cur.h = s0.h; cur.w = s0.w; cur.c = s0.c;
    for (int j = 0; j < k; ++j) {
      Plan& P = plans[NetDef::reaux_index(k, j)];
      const Tensor* dx_out = j > 0 ? &plans[NetDef::reaux_index(k, j - 1)].seed : nullptr;
      build_aux_unit(P, NetDef::reaux_index(k, j), j, cur, false, dx_out, j == k - 1 ? k - 1 : -1);
      cur = P.out;
    }
  }
  // One AuxNet-shaped unit (architecture of AuxNet_j) as plan number `idx`.  out_slot >= 0: the output
  // is the caller's x_{out_slot+1}; otherwise it stays in the workspace.  dx_out: where the adjoint of
  // the unit's input goes (nullptr: not needed).
  void build_aux_unit(Plan& P, int idx, int j, const Tensor& x, bool chain, const Tensor* dx_out, int out_slot = -1) {
    alloc_params(P, LP_AUX(idx));
    const int k = j;
    if (chain) out_slot = k;
    const auto& cv = net.aux[k];
    const Shape4 s = net.boundary[k];
    std::vector<int> ci, bi;
    for (size_t i = 0; i < cv.size(); ++i) {
      const std::string id = std::to_string(i + 1);
      // the distillation step back-propagates through the second convolution into the first
      ci.push_back(add_conv(P, "conv" + id + ".w", cv[i].cin, cv[i].cout, 3, cv[i].stride, 1, cv[i].hin, cv[i].win,
                            i > 0 || dx_out != nullptr));
      bi.push_back(add_bn(P, "bn" + id, cv[i].cout, (long long)s.n * cv[i].hout * cv[i].wout));
    }
    finish_stats(P);
    Tensor cur = x;
    std::vector<Tensor> ins, ys, acts;
    for (size_t i = 0; i < cv.size(); ++i) {
      ins.push_back(cur);
      Tensor y = emit_conv(P, P.fwd, cur, ci[i], nullptr, bi[i]);
      ys.push_back(y);
      const bool final_conv = i + 1 == cv.size();
      Tensor out;
      Op op;
      op.type = OP_BN_APPLY; op.in = y; op.bn = bi[i]; op.relu = final_conv ? 0 : 1;
      if (final_conv && out_slot >= 0) {
        const Shape4 o = net.boundary[k + 1];
        out.ext = EXT_XOUT0 + out_slot; out.n = o.n; out.h = o.h; out.w = o.w; out.c = o.c;
      } else {
        out = new_tensor(y.n, y.h, y.w, y.c);
      }
      op.out = out;
      P.fwd.push_back(op);
      acts.push_back(out);
      cur = out;
    }
    P.out = cur;
    // backward of the distillation loss ||x_{k+1}^{new} - AuxNet_k(x_k)||^2, seeded in P.seed
    const Shape4 o = net.boundary[k + 1];
    P.seed = new_tensor(o.n, o.h, o.w, o.c);
    Tensor d = P.seed;
    for (int i = (int)cv.size() - 1; i >= 0; --i) {
      const bool relu_after = i + 1 < (int)cv.size();
      Tensor dy = emit_bn_bwd(P, P.bwd, d, ys[i], relu_after ? &acts[i] : nullptr, bi[i], nullptr);
      emit_wgrad(P.bwd, ins[i], dy, ci[i]);
      if (i > 0) d = emit_dgrad(P, P.bwd, dy, ci[i], nullptr, nullptr);
      else if (dx_out) emit_dgrad(P, P.bwd, dy, ci[i], nullptr, dx_out);
    }
  }
};

// ---------------------------------------------------------------------------------------------
// executor
// ---------------------------------------------------------------------------------------------
static inline void* resolve(const Tensor& t, const RunCtx& c) {
  switch (t.ext) {
    case EXT_NONE: return t.p;
    case EXT_X: return const_cast<void*>(c.x);
    case EXT_XNEXT: return const_cast<void*>(c.xnext);
    case EXT_KAPPA: return const_cast<void*>(c.kappa);
    case EXT_DX: return c.dx ? c.dx : t.p;
    case EXT_IMAGES: return const_cast<void*>(c.images);
    default: return c.xout ? c.xout[t.ext - EXT_XOUT0] : nullptr;
  }
}

static BnArgs bn_args(const BnDef& b, float eps) {
  BnArgs a;
  a.stats = b.stats; a.gamma = b.gamma; a.beta = b.beta; a.inv_count = 1.0 / (double)b.count; a.eps = eps;
  return a;
}

template <typename T>
static int run_op_t(lp_handle* h, Plan& P, const Op& op, const RunCtx& c) {
  const int dtype = h->dtype;
  const float eps = h->net.d.bn_eps;
  cudaStream_t st = c.st;
  constexpr int V = VecT<T>::N;
  switch (op.type) {
    case OP_CONV_FWD: {
      const ConvDef& cv = P.convs[op.conv];
      double* stats = op.stats_bn >= 0 ? P.bns[op.stats_bn].stats : nullptr;
      const void* addend = op.addend.defined() ? resolve(op.addend, c) : nullptr;
      bool done = false;
      if (op.fuse_loss && !c.serial) {
        if (c.loss_wait) LP_CUDA_OK(cudaStreamWaitEvent(st, c.loss_wait, 0));   // x_{k+1} must exist
        LossFuse lf{c.xnext, c.kappa, P.r.p, P.seed.p, c.rho, P.loss_acc};
        return conv_forward(h, dtype, h->conv_impl, cv, op.in.n, resolve(op.in, c), resolve(op.out, c), addend, stats,
                            &done, h->dev_err, st, &lf);
      }
      return conv_forward(h, dtype, h->conv_impl, cv, op.in.n, resolve(op.in, c), resolve(op.out, c), addend, stats,
                          &done, h->dev_err, st);
    }
    case OP_CONV_DGRAD: {
      const ConvDef& cv = P.convs[op.conv];
      const void* addend = op.addend.defined() ? resolve(op.addend, c) : nullptr;
      BnBwdFuse bf;
      const BnBwdFuse* bfp = nullptr;
      if (op.bwd_bn >= 0) {
        const BnDef& b = P.bns[op.bwd_bn];
        bf.x = resolve(op.bwd_x, c); bf.bn = bn_args(b, eps); bf.dgamma = b.dgamma; bf.dbeta = b.dbeta; bf.relu = op.bwd_relu;
        bfp = &bf;
      }
      return conv_dgrad(h, dtype, h->conv_impl, cv, op.in.n, resolve(op.in, c), resolve(op.out, c), addend, h->dev_err,
                        st, bfp);
    }
    case OP_CONV_WGRAD: {
      const ConvDef& cv = P.convs[op.conv];
      return conv_wgrad(h, dtype, h->conv_impl, cv, op.in.n, resolve(op.in, c), resolve(op.in2, c), cv.gw, h->dev_err,
                        st);
    }
    case OP_BN_STATS: {
      const BnDef& b = P.bns[op.bn];
      const int threads = threads_for_channels(b.C, dtype);
      if (!threads) return LP_ERR_UNSUPPORTED;
      const long long vecs = op.in.elems() / V;
      const int grid = grid_for(vecs, threads * 8, cur_dev().sm_count, 4);
      LP_CUDA_OK(launch_pdl(bn_stats_kernel<T>, dim3(grid), dim3(threads), (size_t)threads * 2 * V * 4, st,
                            (const T*)resolve(op.in, c), vecs, b.C, b.stats));
      h->launches++;
      break;
    }
    case OP_BN_APPLY: {
      const BnDef& b = P.bns[op.bn];
      const int threads = threads_for_channels(b.C, dtype);
      if (!threads) return LP_ERR_UNSUPPORTED;
      const long long vecs = op.in.elems() / V;
      // one wave of blocks: as many per SM as the variant's register cap keeps resident (a second, partial
      // wave cost a fifth of these kernels' time)
      const int per_sm = op.in2.defined() ? 2 : (op.addend.defined() ? 3 : 4);
      const int grid = grid_for(vecs, threads * 4, cur_dev().sm_count, per_sm);
      BnArgs A = bn_args(b, eps), B2 = A;
      const T* x2 = nullptr;
      if (op.in2.defined()) { x2 = (const T*)resolve(op.in2, c); B2 = bn_args(P.bns[op.bn2], eps); }
      const T* addend = op.addend.defined() ? (const T*)resolve(op.addend, c) : nullptr;
      launch_bn_apply<T>(grid, threads, st, (const T*)resolve(op.in, c), A, x2, B2, addend, (T*)resolve(op.out, c), vecs,
                         b.C, op.relu);
      h->launches++;
      break;
    }
    case OP_OUT_LOSS: {
      if (c.loss_wait && !c.serial) LP_CUDA_OK(cudaStreamWaitEvent(st, c.loss_wait, 0));
      const int C = op.out.c;
      const int threads = threads_for_channels(C, dtype);
      if (!threads) return LP_ERR_UNSUPPORTED;
      const long long vecs = op.out.elems() / V;
      const int grid = grid_for(vecs, threads * 4, cur_dev().sm_count, 8);
      BnArgs A, B2;
      memset(&A, 0, sizeof(A));
      memset(&B2, 0, sizeof(B2));
      const T* x = nullptr; const T* x2 = nullptr;
      if (op.in.defined()) { x = (const T*)resolve(op.in, c); A = bn_args(P.bns[op.bn], eps); }
      if (op.in2.defined()) { x2 = (const T*)resolve(op.in2, c); B2 = bn_args(P.bns[op.bn2], eps); }
      const T* addend = op.addend.defined() ? (const T*)resolve(op.addend, c) : nullptr;
      if (op.fuse_loss && !c.serial) {   // sums, residual and seed came from the last convolution's epilogue
        loss_finalize_kernel<<<1, 1, 0, st>>>(P.loss_acc, c.rho, c.loss_out);
        h->launches++;
        break;
      }
      if (c.serial) {
        if (!x) break;  // the producing convolution already wrote the module output
        launch_bn_apply<T>(grid, threads, st, x, A, x2, B2, addend, (T*)P.out.p, vecs, C, 0);
        h->launches++;
        break;
      }
      module_out_loss_kernel<T><<<grid, threads, 0, st>>>(x, A, x2, B2, addend, (const T*)c.xnext, (const T*)c.kappa,
                                                          c.rho, (T*)P.r.p, (T*)P.seed.p, P.loss_acc, vecs, C);
      loss_finalize_kernel<<<1, 1, 0, st>>>(P.loss_acc, c.rho, c.loss_out);
      h->launches += 2;
      break;
    }
    case OP_BN_BWD: {
      const BnDef& b = P.bns[op.bn];
      const int threads = threads_for_channels(b.C, dtype);
      if (!threads) return LP_ERR_UNSUPPORTED;
      const long long vecs = op.in2.elems() / V;
      BnArgs A = bn_args(b, eps);
      const int mask = op.mask.defined() ? 1 : 0;  // a ReLU followed this BN in the forward pass
      const T* addend = op.addend.defined() ? (const T*)resolve(op.addend, c) : nullptr;
      if (!op.reduce_fused) {   // (otherwise the convolution that wrote dy has left the two sums in dgamma, dbeta)
        const int grid_r = grid_for(vecs, threads * 8, cur_dev().sm_count, 2);   // one wave: two blocks stay resident per SM
        LP_CUDA_OK(launch_pdl(bn_bwd_reduce_kernel<T>, dim3(grid_r), dim3(threads), (size_t)threads * 2 * V * 4, st,
                              (const T*)resolve(op.in, c), (const T*)resolve(op.in2, c), mask, A, b.dgamma, b.dbeta, vecs, b.C));
        h->launches++;
      }
      const int grid_a = grid_for(vecs, threads * 4, cur_dev().sm_count, 2);
      LP_CUDA_OK(launch_pdl(bn_bwd_apply_kernel<T>, dim3(grid_a), dim3(threads), 0, st, (const T*)resolve(op.in, c),
                            (const T*)resolve(op.in2, c), mask, A, (const float*)b.dgamma, (const float*)b.dbeta, addend,
                            (T*)resolve(op.out, c), vecs, b.C));
      h->launches++;
      break;
    }
    case OP_MAXPOOL_FWD: {
      if (op.out.c % V) return LP_ERR_UNSUPPORTED;
      const long long total = op.out.elems() / V;
      maxpool_fwd_kernel<T><<<grid_for(total, 256, cur_dev().sm_count, 16), 256, 0, st>>>(
          (const T*)resolve(op.in, c), (T*)resolve(op.out, c), op.arg, op.in.n, op.in.h, op.in.w, op.in.c, op.out.h,
          op.out.w);
      h->launches++;
      break;
    }
    case OP_MAXPOOL_BWD: {
      if (op.out.c % V) return LP_ERR_UNSUPPORTED;
      const long long total = op.out.elems() / V;
      maxpool_bwd_kernel<T><<<grid_for(total, 256, cur_dev().sm_count, 16), 256, 0, st>>>(
          (const T*)resolve(op.in, c), op.arg, (T*)resolve(op.out, c), op.out.n, op.out.h, op.out.w, op.out.c, op.in.h,
          op.in.w);
      h->launches++;
      break;
    }
    case OP_HEAD_FWD: {
      HeadDef& hd = P.head;
      const int32_t* labels = c.labels ? c.labels : h->zero_labels;  // logits-only runs use label 0
      if (hd.classes <= 128 && (size_t)(hd.C + hd.classes) * 4 <= 40 * 1024) {
        head_fused_kernel<T><<<hd.N, 256, (size_t)(hd.C + hd.classes) * 4, st>>>(
            (const T*)resolve(op.in, c), hd.W, hd.b, labels, hd.pooled, hd.logits, hd.dlogits, P.loss_acc, hd.N, hd.HW, hd.C,
            hd.classes);
        h->launches++;
        if (c.loss_out) {
          ce_finalize_kernel<<<1, 1, 0, st>>>(P.loss_acc, c.loss_out);
          h->launches++;
        }
        break;
      }
      avgpool_kernel<T><<<hd.N, 256, 0, st>>>((const T*)resolve(op.in, c), hd.pooled, hd.HW, hd.C);
      h->launches++;
      head_logits_kernel<<<dim3((hd.classes + 3) / 4, (hd.N + 7) / 8), 128, 0, st>>>(hd.pooled, hd.W, hd.b, hd.logits, hd.N,
                                                                                     hd.C, hd.classes);
      head_fwd_kernel<<<hd.N, 128, (size_t)(hd.classes + 32) * 4, st>>>(labels, hd.logits, hd.dlogits, P.loss_acc, hd.N,
                                                                        hd.classes);
      h->launches += 2;
      if (c.loss_out) {
        ce_finalize_kernel<<<1, 1, 0, st>>>(P.loss_acc, c.loss_out);
        h->launches++;
      }
      break;
    }
    case OP_HEAD_BWD: {
      HeadDef& hd = P.head;
      const long long total = (long long)hd.classes * hd.C;
      head_bwd_w_kernel<<<grid_for(total, 128, cur_dev().sm_count, 16), 128, 0, st>>>(hd.dlogits, hd.pooled, hd.dW, hd.db,
                                                                                  hd.N, hd.C, hd.classes);
      head_bwd_x_kernel<T><<<dim3(hd.N, (hd.C + 255) / 256), 256, 0, st>>>(hd.dlogits, hd.W, (T*)resolve(op.out, c), hd.HW,
                                                                           hd.C, hd.classes);
      h->launches += 2;
      break;
    }
    default:
      return LP_ERR_UNSUPPORTED;
  }
  LP_CUDA_OK(cudaGetLastError());
  return LP_OK;
}

struct TimelineScope {
  lp_handle* h; cudaStream_t st; TimelineRec* r = nullptr;
  TimelineScope(lp_handle* h_, cudaStream_t st_, int plan, int op_type, int phase, double bytes = 0.0) : h(h_), st(st_) {
    if (!h || !h->tl.enabled) return;
    Timeline& tl = h->tl;
    if (tl.used == tl.recs.size()) {
      TimelineRec n;
      if (cudaEventCreate(&n.a) != cudaSuccess || cudaEventCreate(&n.b) != cudaSuccess) return;
      tl.recs.push_back(n);
    }
    r = &tl.recs[tl.used++];
    r->plan = plan; r->op_type = op_type; r->phase = phase; r->bytes = bytes;
    cudaEventRecord(r->a, st);
  }
  ~TimelineScope() {
    if (r) cudaEventRecord(r->b, st);
  }
};

// Algorithmic global-memory traffic of one operation: every operand read once, every result written once.
static double op_bytes(const lp_handle* h, const Plan& P, const Op& op) {
  const double e = (double)esize(h->dtype);
  auto sz = [&](const Tensor& t) { return t.defined() ? (double)t.elems() * e : 0.0; };
  switch (op.type) {
    case OP_CONV_FWD: {
      const ConvDef& c = P.convs[op.conv];
      return sz(op.in) + sz(op.out) + sz(op.addend) + (double)c.cout * c.R * c.R * c.cin * e;
    }
    case OP_CONV_DGRAD: {
      const ConvDef& c = P.convs[op.conv];
      return sz(op.in) + sz(op.out) + sz(op.addend) + (op.bwd_bn >= 0 ? sz(op.bwd_x) : 0.0) +
             (double)c.cout * c.R * c.R * c.cin * e;
    }
    case OP_CONV_WGRAD: {
      const ConvDef& c = P.convs[op.conv];
      return sz(op.in) + sz(op.in2) + (double)c.cout * c.R * c.R * c.cin * 4.0;
    }
    case OP_BN_STATS: return sz(op.in);
    case OP_BN_APPLY: return sz(op.in) + sz(op.in2) + sz(op.addend) + sz(op.out);
    case OP_OUT_LOSS:   // operands of the output, x_next, [kappa,] residual and terminal adjoint
      return op.fuse_loss ? 0.0 : sz(op.in) + sz(op.in2) + sz(op.addend) + 3.0 * sz(op.out);
    case OP_BN_BWD:     // reduction pass (dy, x; not where a convolution took it) and apply pass (dy, x, [addend] -> dx)
      return (op.reduce_fused ? 1.0 : 2.0) * (sz(op.in) + sz(op.in2)) + sz(op.addend) + sz(op.out);
    case OP_MAXPOOL_FWD: return sz(op.in) + sz(op.out) + (double)op.out.elems();
    case OP_MAXPOOL_BWD: return sz(op.in) + sz(op.out) + (double)op.in.elems();
    case OP_HEAD_FWD: return sz(op.in);
    case OP_HEAD_BWD: return sz(op.out);
    default: return 0.0;
  }
}

static int run_ops(lp_handle* h, Plan& P, const std::vector<Op>& ops, const RunCtx& c) {
  // (per-operation timing wants one stream: the time line and the convolution profile keep everything in order)
  const bool use_side = P.side && !h->tl.enabled && !h->prof.enabled;
  size_t nside = 0;
  int rc = LP_OK;
  for (const Op& op : ops) {
    if (use_side && op.type == OP_CONV_WGRAD && nside < P.side_ev.size()) {
      if (cudaEventRecord(P.side_ev[nside], c.st) != cudaSuccess ||
          cudaStreamWaitEvent(P.side, P.side_ev[nside], 0) != cudaSuccess) { rc = LP_ERR_CUDA; break; }
      ++nside;
      RunCtx c2 = c;
      c2.st = P.side;
      rc = h->dtype == LP_F32 ? run_op_t<float>(h, P, op, c2) : run_op_t<bf16>(h, P, op, c2);
    } else {
      TimelineScope ts(h, c.st, c.plan_id, (int)op.type, c.phase, h->tl.enabled ? op_bytes(h, P, op) : 0.0);
      rc = h->dtype == LP_F32 ? run_op_t<float>(h, P, op, c) : run_op_t<bf16>(h, P, op, c);
    }
    if (rc != LP_OK) break;
  }
  // joined whatever happened: a stream left unjoined would invalidate a capture in progress
  if (nside && (cudaEventRecord(P.side_done, P.side) != cudaSuccess || cudaStreamWaitEvent(c.st, P.side_done, 0) != cudaSuccess))
    if (rc == LP_OK) rc = LP_ERR_CUDA;
  return rc;
}

static int zero_forward_state(Plan& P, cudaStream_t st) {
  if (P.stats_bytes) LP_CUDA_OK(cudaMemsetAsync(P.stats_region, 0, P.stats_bytes, st));
  LP_CUDA_OK(cudaMemsetAsync(P.loss_acc, 0, 2 * sizeof(double), st));
  return LP_OK;
}

// bf16 copies of the regrouped stem weights (space-to-depth stems), after every change of the master weights
static int pack_s2d_weights(lp_handle* h, Plan& P, cudaStream_t st) {
  for (const ConvDef& c : P.convs) {
    if (!c.s2d) continue;
    s2d_pack_weights_kernel<<<grid_for((long long)c.cout * 256, 256, cur_dev().sm_count, 8), 256, 0, st>>>(c.w, c.wf, c.cout,
                                                                                                          c.cin);
    h->launches++;
    LP_CUDA_OK(cudaGetLastError());
  }
  return LP_OK;
}

static int pack_weights(lp_handle* h, Plan& P, cudaStream_t st) {
  {
    int rc = pack_s2d_weights(h, P, st);
    if (rc != LP_OK) return rc;
  }
  if (P.ps.host_pack.empty()) return LP_OK;
  pack_weights_tiled_kernel<<<(unsigned)P.ps.pack_tiles, dim3(32, 8), 0, st>>>(P.ps.dev_pack,
                                                                              (int)P.ps.host_pack.size());
  h->launches++;
  LP_CUDA_OK(cudaGetLastError());
  return LP_OK;
}

// theta <- theta - lr*(g + wd*theta [momentum]) and, for the tensor-core path, fresh bf16 copies of
// the convolution weights: one fused pass over the packed weights plus a small one over the rest.
static int sgd_update_inner(lp_handle* h, Plan& P, float lr, float momentum, float weight_decay, cudaStream_t st);
static int sgd_update(lp_handle* h, Plan& P, float lr, float momentum, float weight_decay, cudaStream_t st) {
  int rc = sgd_update_inner(h, P, lr, momentum, weight_decay, st);
  if (rc != LP_OK) return rc;
  return pack_s2d_weights(h, P, st);
}
static int sgd_update_inner(lp_handle* h, Plan& P, float lr, float momentum, float weight_decay, cudaStream_t st) {
  float* mom = momentum != 0.f ? P.ps.m : nullptr;
  if (P.ps.host_pack.empty()) {
    sgd_kernel<<<grid_for((long long)P.ps.n, 256, cur_dev().sm_count, 8), 256, 0, st>>>(P.ps.p, P.ps.g, P.ps.m,
                                                                                    (long long)P.ps.n, lr, momentum,
                                                                                    weight_decay);
    h->launches++;
    LP_CUDA_OK(cudaGetLastError());
    return LP_OK;
  }
  const bool blobs16 = ((reinterpret_cast<uintptr_t>(P.ps.p) | reinterpret_cast<uintptr_t>(P.ps.g) |
                         reinterpret_cast<uintptr_t>(P.ps.m)) & 15) == 0;
  if (!(P.ps.pack64_ok && blobs16)) {
    // a weight tensor off the 16-byte grid of the blobs: the plain update over everything, then the copies
    sgd_kernel<<<grid_for((long long)P.ps.n, 256, cur_dev().sm_count, 8), 256, 0, st>>>(P.ps.p, P.ps.g, P.ps.m,
                                                                                    (long long)P.ps.n, lr, momentum,
                                                                                    weight_decay);
    h->launches++;
    LP_CUDA_OK(cudaGetLastError());
    pack_weights_tiled_kernel<<<(unsigned)P.ps.pack_tiles, dim3(32, 8), 0, st>>>(P.ps.dev_pack,
                                                                                (int)P.ps.host_pack.size());
    h->launches++;
    LP_CUDA_OK(cudaGetLastError());
    return LP_OK;
  }
  if (!P.ps.host_ranges.empty()) {
    sgd_ranges_kernel<<<(unsigned)P.ps.host_ranges.size(), 256, 0, st>>>(P.ps.dev_ranges, P.ps.p, P.ps.g, mom, lr,
                                                                         momentum, weight_decay);
    h->launches++;
  }
  sgd_pack_tiled64_kernel<<<(unsigned)P.ps.pack_tiles64, 256, 0, st>>>(P.ps.dev_pack, (int)P.ps.host_pack.size(), P.ps.p,
                                                                       P.ps.g, mom, lr, momentum, weight_decay);
  h->launches++;
  LP_CUDA_OK(cudaGetLastError());
  return LP_OK;
}

static bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }

static int module_fwd_bwd(lp_handle* h, int k, const void* x_k, const void* x_next_or_labels, const void* lambda_k,
                          float rho, float* loss_out, void* dx_k, cudaStream_t st, cudaEvent_t loss_wait = nullptr) {
  Plan& P = h->modules[k];
  const bool last = k == h->net.K - 1;
  RunCtx c;
  c.st = st; c.x = x_k; c.rho = rho; c.loss_out = loss_out; c.dx = dx_k; c.loss_wait = loss_wait;
  if (last) c.labels = (const int32_t*)x_next_or_labels;
  else { c.xnext = x_next_or_labels; c.kappa = lambda_k; }
  int rc = zero_forward_state(P, st);
  if (rc != LP_OK) return rc;
  LP_CUDA_OK(cudaMemsetAsync(P.ps.g, 0, P.ps.n * 4, st));
  c.plan_id = k;
  c.phase = LP_PHASE_FORWARD;
  rc = run_ops(h, P, P.fwd, c);
  if (rc != LP_OK) return rc;
  c.phase = LP_PHASE_BACKWARD;
  rc = run_ops(h, P, P.bwd, c);
  if (rc != LP_OK) return rc;
  P.ps.grads_fresh = true;
  P.ran_fwd_bwd = true;
  return LP_OK;
}

}  // namespace lp

// =============================================================================================
// C ABI
// =============================================================================================
extern "C" {

const char* lp_status_string(int s) {
  switch (s) {
    case LP_OK: return "ok";
    case LP_ERR_NULL: return "null pointer";
    case LP_ERR_BAD_DESC: return "bad network descriptor";
    case LP_ERR_BAD_INDEX: return "index out of range";
    case LP_ERR_ALIGN: return "pointer not 16-byte aligned";
    case LP_ERR_WORKSPACE: return "workspace too small or misaligned";
    case LP_ERR_ORDER: return "call order violated";
    case LP_ERR_DEVICE_TIMEOUT: return "device-side wait timed out";
    case LP_ERR_CUDA: return "CUDA error";
    case LP_ERR_SIZE: return "size mismatch";
    case LP_ERR_UNSUPPORTED: return "unsupported";
    default: return "unknown status";
  }
}

int lp_validate_desc(const lp_net_desc* desc) {
  NetDef n;
  return n.build(desc);
}

static int plan_all(const NetDef& net, Arena& A, std::vector<Plan>* modules, std::vector<Plan>* auxs, int** dev_err,
                    int32_t** zero_labels) {
  Planner pl(net, A);
  *dev_err = (int*)A.alloc(256);
  *zero_labels = (int32_t*)A.alloc((size_t)net.d.N * 4);
  modules->resize(net.K);
  for (int k = 0; k < net.K; ++k) pl.build_module((*modules)[k], k);
  auxs->resize(net.n_aux_plans());
  if (net.d.aux_recursive) {
    for (int k = 1; k < net.K; ++k) pl.build_reaux_stack(*auxs, k);
  } else {
    for (int k = 0; k + 1 < net.K; ++k) pl.build_aux((*auxs)[k], k);
  }
  return LP_OK;
}

size_t lp_workspace_bytes(const lp_net_desc* desc) {
  NetDef net;
  if (net.build(desc) != LP_OK) return 0;
  Arena A;
  std::vector<Plan> m, a;
  int* e = nullptr;
  int32_t* z = nullptr;
  plan_all(net, A, &m, &a, &e, &z);
  return align_up(A.off, 256) + 256;
}

int lp_param_layout(const lp_net_desc* desc, int which, lp_param_entry* entries, int max_entries, int* n_entries) {
  NetDef net;
  int rc = net.build(desc);
  if (rc != LP_OK) return rc;
  std::vector<lp_param_entry> L;
  rc = net.layout(which, L, nullptr);
  if (rc != LP_OK) return rc;
  if (n_entries) *n_entries = (int)L.size();
  if (entries)
    for (int i = 0; i < (int)L.size() && i < max_entries; ++i) entries[i] = L[i];
  return LP_OK;
}

int lp_boundary_shape_desc(const lp_net_desc* desc, int k, int shape[4]) {
  NetDef net;
  int rc = net.build(desc);
  if (rc != LP_OK) return rc;
  if (!shape) return LP_ERR_NULL;
  if (k < 0 || k >= net.K) return LP_ERR_BAD_INDEX;
  shape[0] = net.boundary[k].n; shape[1] = net.boundary[k].h; shape[2] = net.boundary[k].w; shape[3] = net.boundary[k].c;
  return LP_OK;
}

int lp_create(const lp_net_desc* desc, void* dev_workspace, size_t bytes, lp_handle** out) {
  if (!desc || !dev_workspace || !out) return LP_ERR_NULL;
  *out = nullptr;
  NetDef net;
  int rc = net.build(desc);
  if (rc != LP_OK) return rc;
  if (reinterpret_cast<uintptr_t>(dev_workspace) & 255) return LP_ERR_WORKSPACE;
  const size_t need = lp_workspace_bytes(desc);
  if (bytes < need) return LP_ERR_WORKSPACE;
  rc = init_cur_dev();
  if (rc != LP_OK) return rc;
  lp_handle* h = new lp_handle();
  h->net = net;
  h->dtype = net.d.dtype;
  h->conv_impl = net.d.conv_impl;
  h->ws = (uint8_t*)dev_workspace;
  h->ws_bytes = bytes;
  Arena A;
  A.base = h->ws;
  plan_all(h->net, A, &h->modules, &h->auxs, &h->dev_err, &h->zero_labels);
  if (cudaMemset(dev_workspace, 0, need) != cudaSuccess) { delete h; return LP_ERR_CUDA; }
  auto upload = [&](Plan& P) -> int {
    if (P.ps.host_pack.empty()) return LP_OK;
    LP_CUDA_OK(cudaMemcpy(P.ps.dev_pack, P.ps.host_pack.data(), P.ps.host_pack.size() * sizeof(PackEntry),
                          cudaMemcpyHostToDevice));
    if (!P.ps.host_ranges.empty())
      LP_CUDA_OK(cudaMemcpy(P.ps.dev_ranges, P.ps.host_ranges.data(), P.ps.host_ranges.size() * sizeof(SgdRange),
                            cudaMemcpyHostToDevice));
    return LP_OK;
  };
  for (auto& P : h->modules) if ((rc = upload(P)) != LP_OK) { delete h; return rc; }
  for (auto& P : h->auxs) if ((rc = upload(P)) != LP_OK) { delete h; return rc; }
  h->streams.resize(net.K);
  h->done.resize(net.K);
  for (int k = 0; k < net.K; ++k) {
    if (cudaStreamCreateWithFlags(&h->streams[k], cudaStreamNonBlocking) != cudaSuccess ||
        cudaEventCreateWithFlags(&h->done[k], cudaEventDisableTiming) != cudaSuccess) {
      delete h;
      return LP_ERR_CUDA;
    }
  }
  if (!(net.d.conv_impl & LP_CONV_WGRAD_IN_CHAIN)) {
    for (auto& P : h->modules) {
      size_t n_wgrad = 0;
      for (const Op& op : P.bwd) n_wgrad += op.type == OP_CONV_WGRAD ? 1 : 0;
      if (!n_wgrad) continue;
      if (cudaStreamCreateWithFlags(&P.side, cudaStreamNonBlocking) != cudaSuccess ||
          cudaEventCreateWithFlags(&P.side_done, cudaEventDisableTiming) != cudaSuccess) { delete h; return LP_ERR_CUDA; }
      P.side_ev.assign(n_wgrad, nullptr);
      for (auto& e : P.side_ev)
        if (cudaEventCreateWithFlags(&e, cudaEventDisableTiming) != cudaSuccess) { delete h; return LP_ERR_CUDA; }
    }
  }
  if (cudaEventCreateWithFlags(&h->fork, cudaEventDisableTiming) != cudaSuccess) { delete h; return LP_ERR_CUDA; }
  if (cudaStreamCreateWithFlags(&h->aux_stream, cudaStreamNonBlocking) != cudaSuccess ||
      cudaEventCreateWithFlags(&h->aux_end, cudaEventDisableTiming) != cudaSuccess) { delete h; return LP_ERR_CUDA; }
  h->aux_done.resize(net.K > 1 ? net.K - 1 : 0);
  for (auto& e : h->aux_done)
    if (cudaEventCreateWithFlags(&e, cudaEventDisableTiming) != cudaSuccess) { delete h; return LP_ERR_CUDA; }
  *out = h;
  return LP_OK;
}

int lp_destroy(lp_handle* h) {
  if (!h) return LP_ERR_NULL;
  cudaDeviceSynchronize();
  for (auto s : h->streams) if (s) cudaStreamDestroy(s);
  for (auto e : h->done) if (e) cudaEventDestroy(e);
  if (h->fork) cudaEventDestroy(h->fork);
  if (h->aux_stream) cudaStreamDestroy(h->aux_stream);
  if (h->aux_end) cudaEventDestroy(h->aux_end);
  for (auto e : h->aux_done) if (e) cudaEventDestroy(e);
  for (auto& pr : h->prof.events) { cudaEventDestroy(pr.first); cudaEventDestroy(pr.second); }
  for (auto& r : h->tl.recs) { if (r.a) cudaEventDestroy(r.a); if (r.b) cudaEventDestroy(r.b); }
  for (auto g : h->graphs) cudaGraphExecDestroy(g);
  for (auto& P : h->modules) {
    if (P.side) cudaStreamDestroy(P.side);
    if (P.side_done) cudaEventDestroy(P.side_done);
    for (auto e : P.side_ev) if (e) cudaEventDestroy(e);
  }
  delete h;
  return LP_OK;
}

static Plan* plan_for(lp_handle* h, int which) {
  if (which >= LP_AUX(0)) {
    const int k = which - LP_AUX(0);
    if (k < 0 || k >= (int)h->auxs.size()) return nullptr;
    return &h->auxs[k];
  }
  if (which < 0 || which >= (int)h->modules.size()) return nullptr;
  return &h->modules[which];
}

int lp_param_count(lp_handle* h, int which, size_t* n) {
  if (!h || !n) return LP_ERR_NULL;
  Plan* P = plan_for(h, which);
  if (!P) return LP_ERR_BAD_INDEX;
  *n = P->ps.n;
  return LP_OK;
}

int lp_set_params(lp_handle* h, int which, const float* host, size_t n) {
  if (!h || !host) return LP_ERR_NULL;
  Plan* P = plan_for(h, which);
  if (!P) return LP_ERR_BAD_INDEX;
  if (n != P->ps.n) return LP_ERR_SIZE;
  LP_CUDA_OK(cudaMemcpy(P->ps.p, host, n * 4, cudaMemcpyHostToDevice));
  int rc = pack_weights(h, *P, nullptr);
  if (rc != LP_OK) return rc;
  LP_CUDA_OK(cudaDeviceSynchronize());
  return LP_OK;
}

int lp_get_params(lp_handle* h, int which, float* host, size_t n) {
  if (!h || !host) return LP_ERR_NULL;
  Plan* P = plan_for(h, which);
  if (!P) return LP_ERR_BAD_INDEX;
  if (n != P->ps.n) return LP_ERR_SIZE;
  LP_CUDA_OK(cudaDeviceSynchronize());
  LP_CUDA_OK(cudaMemcpy(host, P->ps.p, n * 4, cudaMemcpyDeviceToHost));
  return LP_OK;
}

int lp_get_grads(lp_handle* h, int which, float* host, size_t n) {
  if (!h || !host) return LP_ERR_NULL;
  Plan* P = plan_for(h, which);
  if (!P) return LP_ERR_BAD_INDEX;
  if (n != P->ps.n) return LP_ERR_SIZE;
  LP_CUDA_OK(cudaDeviceSynchronize());
  LP_CUDA_OK(cudaMemcpy(host, P->ps.g, n * 4, cudaMemcpyDeviceToHost));
  return LP_OK;
}

int lp_boundary_shape(lp_handle* h, int k, int shape[4]) {
  if (!h || !shape) return LP_ERR_NULL;
  if (k < 0 || k >= h->net.K) return LP_ERR_BAD_INDEX;
  const Shape4& s = h->net.boundary[k];
  shape[0] = s.n; shape[1] = s.h; shape[2] = s.w; shape[3] = s.c;
  return LP_OK;
}

static int aux_plan_forward(lp_handle* h, int idx, RunCtx& c) {
  int rc = zero_forward_state(h->auxs[idx], c.st);
  if (rc != LP_OK) return rc;
  c.plan_id = LP_AUX(idx); c.phase = LP_PHASE_AUX_FORWARD;
  return run_ops(h, h->auxs[idx], h->auxs[idx].fwd, c);
}

int lp_auxnet_forward(lp_handle* h, const void* images, void* const* x_out, void* stream) {
  if (!h || !images) return LP_ERR_NULL;
  const int K = h->net.K;
  if (K > 1 && !x_out) return LP_ERR_NULL;
  if (!aligned16(images)) return LP_ERR_ALIGN;
  for (int k = 0; k + 1 < K; ++k) {
    if (!x_out[k]) return LP_ERR_NULL;
    if (!aligned16(x_out[k])) return LP_ERR_ALIGN;
  }
  RunCtx c;
  c.st = (cudaStream_t)stream; c.images = images; c.xout = x_out;
  for (size_t i = 0; i < h->auxs.size(); ++i) {   // chain order, or stack by stack (units in order)
    int rc = aux_plan_forward(h, (int)i, c);
    if (rc != LP_OK) return rc;
  }
  return LP_OK;
}

static int check_module_args(lp_handle* h, int k, const void* x_k, const void* x_next_or_labels, const void* lambda_k,
                             float* loss_out, void* dx_k) {
  if (!h || !x_k || !x_next_or_labels || !loss_out) return LP_ERR_NULL;
  if (k < 0 || k >= h->net.K) return LP_ERR_BAD_INDEX;
  if (!aligned16(x_k) || !aligned16(x_next_or_labels) || (lambda_k && !aligned16(lambda_k)) ||
      (dx_k && !aligned16(dx_k)) || (reinterpret_cast<uintptr_t>(loss_out) & 3))
    return LP_ERR_ALIGN;
  return LP_OK;
}

int lp_module_fwd_bwd(lp_handle* h, int k, const void* x_k, const void* x_next_or_labels, const void* lambda_k,
                      float rho, float* loss_out, void* dx_k, void* stream) {
  int rc = check_module_args(h, k, x_k, x_next_or_labels, lambda_k, loss_out, dx_k);
  if (rc != LP_OK) return rc;
  return module_fwd_bwd(h, k, x_k, x_next_or_labels, lambda_k, rho, loss_out, dx_k, (cudaStream_t)stream);
}

// Marks the handle while the modules are being enqueued side by side (convolution grids then leave SMs
// to the other streams, see launch_conv_tc).
struct ConcurrentScope {
  lp_handle* h;
  explicit ConcurrentScope(lp_handle* h_) : h(h_) { h->concurrent = true; }
  ~ConcurrentScope() { h->concurrent = false; }
};

int lp_modules_fwd_bwd_all(lp_handle* h, const void* const* x, const int32_t* labels, const void* const* lambdas,
                           float rho, float* loss_out, void* const* dx, void* stream) {
  if (!h || !x || !labels || !loss_out) return LP_ERR_NULL;
  const int K = h->net.K;
  for (int k = 0; k < K; ++k) {
    const void* tgt = k == K - 1 ? (const void*)labels : x[k + 1];
    int rc = check_module_args(h, k, x[k], tgt, (lambdas && k < K - 1) ? lambdas[k] : nullptr, loss_out + 2 * k,
                               dx ? dx[k] : nullptr);
    if (rc != LP_OK) return rc;
  }
  cudaStream_t st = (cudaStream_t)stream;
  ConcurrentScope concurrent(h);
  LP_CUDA_OK(cudaEventRecord(h->fork, st));
  // heaviest modules first is not needed: all K are enqueued before any can finish
  // A failure part-way still joins every stream that was forked back into the caller's (a stream left
  // unjoined would invalidate a capture in progress); the first error is what the call returns.
  int first_err = LP_OK;
  int forked = 0;
  for (int k = 0; k < K && first_err == LP_OK; ++k) {
    if (cudaStreamWaitEvent(h->streams[k], h->fork, 0) != cudaSuccess) { first_err = LP_ERR_CUDA; break; }
    forked = k + 1;
    const void* tgt = k == K - 1 ? (const void*)labels : x[k + 1];
    first_err = module_fwd_bwd(h, k, x[k], tgt, (lambdas && k < K - 1) ? lambdas[k] : nullptr, rho, loss_out + 2 * k,
                               dx ? dx[k] : nullptr, h->streams[k]);
  }
  for (int k = 0; k < forked; ++k) {
    if (cudaEventRecord(h->done[k], h->streams[k]) != cudaSuccess || cudaStreamWaitEvent(st, h->done[k], 0) != cudaSuccess)
      if (first_err == LP_OK) first_err = LP_ERR_CUDA;
  }
  return first_err;
}

static int update_module(lp_handle* h, int k, float lr, float momentum, float weight_decay, float kappa_step,
                         void* lambda_inout, cudaStream_t st) {
  Plan& P = h->modules[k];
  // parameters read and written, gradients read, both bf16 copies of the packed weights written
  TimelineScope ts(h, st, k, LP_OP_UPDATE, LP_PHASE_UPDATE, 12.0 * (double)P.ps.n + 4.0 * (double)P.ps.pack_total);
  int rc = sgd_update(h, P, lr, momentum, weight_decay, st);
  if (rc != LP_OK) return rc;
  P.ps.grads_fresh = false;
  if (lambda_inout && k + 1 < h->net.K) {
    const long long n = P.r.elems();
    if (h->dtype == LP_F32)
      kappa_update_kernel<float><<<grid_for(n / 4, 256, cur_dev().sm_count, 8), 256, 0, st>>>(
          (float*)lambda_inout, (const float*)P.r.p, kappa_step, n / 4);
    else
      kappa_update_kernel<bf16><<<grid_for(n / 8, 256, cur_dev().sm_count, 8), 256, 0, st>>>(
          (bf16*)lambda_inout, (const bf16*)P.r.p, kappa_step, n / 8);
    h->launches++;
    LP_CUDA_OK(cudaGetLastError());
  }
  return LP_OK;
}

int lp_step(lp_handle* h, float lr, float momentum, float weight_decay, float kappa_step, void* const* lambdas_inout,
            void* stream) {
  if (!h) return LP_ERR_NULL;
  cudaStream_t st = (cudaStream_t)stream;
  bool any = false;
  for (auto& P : h->modules) any = any || P.ps.grads_fresh;
  if (!any) return LP_ERR_ORDER;
  const int K = h->net.K;
  if (lambdas_inout)
    for (int k = 0; k + 1 < K; ++k)
      if (lambdas_inout[k] && !aligned16(lambdas_inout[k])) return LP_ERR_ALIGN;
  for (int k = 0; k < K; ++k) {
    if (!h->modules[k].ps.grads_fresh) continue;
    int rc = update_module(h, k, lr, momentum, weight_decay, kappa_step,
                           (lambdas_inout && k + 1 < K) ? lambdas_inout[k] : nullptr, st);
    if (rc != LP_OK) return rc;
  }
  return LP_OK;
}

int lp_layer_parallel_step(lp_handle* h, const void* images, void* const* x_out, const int32_t* labels,
                           void* const* lambdas_inout, float rho, float* loss_out, void* const* dx, float lr,
                           float momentum, float weight_decay, float kappa_step, void* stream) {
  if (!h || !images || !labels || !loss_out) return LP_ERR_NULL;
  const int K = h->net.K;
  if (K > 1 && !x_out) return LP_ERR_NULL;
  if (!aligned16(images)) return LP_ERR_ALIGN;
  for (int k = 0; k + 1 < K; ++k) {
    if (!x_out[k]) return LP_ERR_NULL;
    if (!aligned16(x_out[k]) || (lambdas_inout && lambdas_inout[k] && !aligned16(lambdas_inout[k])) ||
        (dx && dx[k + 1] && !aligned16(dx[k + 1])))
      return LP_ERR_ALIGN;
  }
  cudaStream_t st = (cudaStream_t)stream;
  ConcurrentScope concurrent(h);
  LP_CUDA_OK(cudaEventRecord(h->fork, st));
  // Streams forked from the caller's so far; whatever happens below, each is joined back before the
  // call returns (a stream left unjoined would invalidate a capture in progress).
  bool aux_forked = false;
  std::vector<bool> forked(K, false);
  auto fork = [&](cudaStream_t s, bool* flag) -> int {
    if (*flag) return LP_OK;
    LP_CUDA_OK(cudaStreamWaitEvent(s, h->fork, 0));
    *flag = true;
    return LP_OK;
  };
  auto fork_module = [&](int k) -> int {
    bool f = forked[k];
    int rc = fork(h->streams[k], &f);
    forked[k] = f;
    return rc;
  };
  auto enqueue = [&]() -> int {
    int rc = fork(h->aux_stream, &aux_forked);
    if (rc != LP_OK) return rc;
    if (h->net.d.aux_recursive) {
      // recursive form: stack k needs the images only and runs on module k's stream, right before the
      // module it feeds; aux_done[k-1] marks x_k for module k-1's local loss
      for (int k = 1; k < K; ++k) {
        cudaStream_t sk = h->streams[k];
        if ((rc = fork_module(k)) != LP_OK) return rc;
        RunCtx c;
        c.st = sk; c.images = images; c.xout = x_out;
        for (int j = 0; j < k; ++j)
          if ((rc = aux_plan_forward(h, NetDef::reaux_index(k, j), c)) != LP_OK) return rc;
        LP_CUDA_OK(cudaEventRecord(h->aux_done[k - 1], sk));
      }
    } else {
      // AuxNet chain on its own stream; aux_done[k] marks x_{k+1}
      RunCtx c;
      c.st = h->aux_stream; c.images = images; c.xout = x_out;
      for (int k = 0; k + 1 < K; ++k) {
        if ((rc = aux_plan_forward(h, k, c)) != LP_OK) return rc;
        LP_CUDA_OK(cudaEventRecord(h->aux_done[k], h->aux_stream));
      }
    }
    // module k starts as soon as x_k exists, takes its local loss as soon as x_{k+1} exists, and
    // updates its own parameters right after its own backward pass
    for (int k = 0; k < K; ++k) {
      cudaStream_t sk = h->streams[k];
      if ((rc = fork_module(k)) != LP_OK) return rc;
      if (k > 0) LP_CUDA_OK(cudaStreamWaitEvent(sk, h->aux_done[k - 1], 0));
      const bool last = k == K - 1;
      const void* xk = k == 0 ? images : x_out[k - 1];
      const void* tgt = last ? (const void*)labels : (const void*)x_out[k];
      void* lam = (lambdas_inout && !last) ? lambdas_inout[k] : nullptr;
      rc = module_fwd_bwd(h, k, xk, tgt, lam, rho, loss_out + 2 * k, dx ? dx[k] : nullptr, sk,
                          last ? nullptr : h->aux_done[k]);
      if (rc != LP_OK) return rc;
      rc = update_module(h, k, lr, momentum, weight_decay, kappa_step, lam, sk);
      if (rc != LP_OK) return rc;
    }
    return LP_OK;
  };
  int first_err = enqueue();
  if (aux_forked) {
    if (cudaEventRecord(h->aux_end, h->aux_stream) != cudaSuccess || cudaStreamWaitEvent(st, h->aux_end, 0) != cudaSuccess)
      if (first_err == LP_OK) first_err = LP_ERR_CUDA;
  }
  for (int k = 0; k < K; ++k) {
    if (!forked[k]) continue;
    if (cudaEventRecord(h->done[k], h->streams[k]) != cudaSuccess || cudaStreamWaitEvent(st, h->done[k], 0) != cudaSuccess)
      if (first_err == LP_OK) first_err = LP_ERR_CUDA;
  }
  return first_err;
}

int lp_auxnet_distill(lp_handle* h, const void* images, void* const* x, const void* const* dx, float lr_lambda,
                      float lr_aux, void* const* x_new, float* loss_out, void* stream) {
  if (!h || !images || !x || !dx || !loss_out) return LP_ERR_NULL;
  const int K = h->net.K;
  if (!aligned16(images)) return LP_ERR_ALIGN;
  for (int k = 1; k < K; ++k) {
    if (!x[k - 1] || !dx[k]) return LP_ERR_NULL;
    if (!aligned16(x[k - 1]) || !aligned16(dx[k]) || (x_new && x_new[k - 1] && !aligned16(x_new[k - 1]))) return LP_ERR_ALIGN;
    if (!h->modules[k - 1].ran_fwd_bwd) return LP_ERR_ORDER;  // its terminal adjoint is the other half of g_k
  }
  cudaStream_t st = (cudaStream_t)stream;
  RunCtx c;
  c.st = st; c.images = images; c.xout = x;
  const bool rec = h->net.d.aux_recursive != 0;
  for (int k = 1; k < K; ++k) {
    // the network that produced x_k: AuxNet_{k-1}, or the last unit of stack k
    const int last_idx = rec ? NetDef::reaux_index(k, k - 1) : k - 1;
    const int first_idx = rec ? NetDef::reaux_index(k, 0) : k - 1;
    Plan& A = h->auxs[last_idx];
    const long long n = A.seed.elems();
    LP_CUDA_OK(cudaMemsetAsync(A.loss_acc, 0, 2 * sizeof(double), st));
    for (int i = first_idx; i <= last_idx; ++i) LP_CUDA_OK(cudaMemsetAsync(h->auxs[i].ps.g, 0, h->auxs[i].ps.n * 4, st));
    void* xn = x_new ? x_new[k - 1] : nullptr;
    if (h->dtype == LP_F32)
      distill_seed_kernel<float><<<grid_for(n / 4, 256, cur_dev().sm_count, 8), 256, 0, st>>>(
          (const float*)x[k - 1], (const float*)dx[k], (const float*)h->modules[k - 1].seed.p, lr_lambda,
          (float*)xn, (float*)A.seed.p, A.loss_acc, n / 4);
    else
      distill_seed_kernel<bf16><<<grid_for(n / 8, 256, cur_dev().sm_count, 8), 256, 0, st>>>(
          (const bf16*)x[k - 1], (const bf16*)dx[k], (const bf16*)h->modules[k - 1].seed.p, lr_lambda, (bf16*)xn,
          (bf16*)A.seed.p, A.loss_acc, n / 8);
    distill_loss_kernel<<<1, 1, 0, st>>>(A.loss_acc, loss_out + (k - 1));
    h->launches += 2;
    LP_CUDA_OK(cudaGetLastError());
    // back through the units (one in the chain form), each followed by its own SGD step
    for (int i = last_idx; i >= first_idx; --i) {
      Plan& U = h->auxs[i];
      c.plan_id = LP_AUX(i); c.phase = LP_PHASE_DISTILL;
      int rc = run_ops(h, U, U.bwd, c);
      if (rc != LP_OK) return rc;
    }
    for (int i = first_idx; i <= last_idx; ++i) {
      TimelineScope ts(h, st, LP_AUX(i), LP_OP_UPDATE, LP_PHASE_DISTILL);
      int rc = sgd_update(h, h->auxs[i], lr_aux, 0.f, 0.f, st);
      if (rc != LP_OK) return rc;
    }
  }
  return LP_OK;
}

int lp_aux_correct(lp_handle* h, void* const* x_inout, const void* const* dx, float lr_lambda, float* norm_out,
                   void* stream) {
  if (!h || !x_inout || !dx) return LP_ERR_NULL;
  const int K = h->net.K;
  for (int k = 1; k < K; ++k) {
    if (!x_inout[k - 1] || !dx[k]) return LP_ERR_NULL;
    if (!aligned16(x_inout[k - 1]) || !aligned16(dx[k])) return LP_ERR_ALIGN;
    if (!h->modules[k - 1].ran_fwd_bwd) return LP_ERR_ORDER;
  }
  cudaStream_t st = (cudaStream_t)stream;
  for (int k = 1; k < K; ++k) {
    Plan& A = h->auxs[k - 1];   // only its loss accumulator is used
    const long long n = h->modules[k - 1].seed.elems();
    TimelineScope ts(h, st, LP_AUX(k - 1), LP_OP_UPDATE, LP_PHASE_DISTILL);
    LP_CUDA_OK(cudaMemsetAsync(A.loss_acc, 0, 2 * sizeof(double), st));
    if (h->dtype == LP_F32)
      distill_seed_kernel<float><<<grid_for(n / 4, 256, cur_dev().sm_count, 8), 256, 0, st>>>(
          (const float*)x_inout[k - 1], (const float*)dx[k], (const float*)h->modules[k - 1].seed.p, lr_lambda,
          (float*)x_inout[k - 1], nullptr, A.loss_acc, n / 4);
    else
      distill_seed_kernel<bf16><<<grid_for(n / 8, 256, cur_dev().sm_count, 8), 256, 0, st>>>(
          (const bf16*)x_inout[k - 1], (const bf16*)dx[k], (const bf16*)h->modules[k - 1].seed.p, lr_lambda,
          (bf16*)x_inout[k - 1], nullptr, A.loss_acc, n / 8);
    h->launches++;
    if (norm_out) {
      distill_loss_kernel<<<1, 1, 0, st>>>(A.loss_acc, norm_out + (k - 1));
      h->launches++;
    }
    LP_CUDA_OK(cudaGetLastError());
  }
  return LP_OK;
}

static int serial_forward(lp_handle* h, const void* images, const int32_t* labels, float* loss_out, cudaStream_t st) {
  const int K = h->net.K;
  const void* x = images;
  for (int k = 0; k < K; ++k) {
    Plan& P = h->modules[k];
    RunCtx c;
    c.st = st; c.x = x; c.serial = true; c.labels = labels; c.loss_out = loss_out;
    int rc = zero_forward_state(P, st);
    if (rc != LP_OK) return rc;
    c.plan_id = k; c.phase = LP_PHASE_FORWARD;
    rc = run_ops(h, P, P.fwd, c);
    if (rc != LP_OK) return rc;
    x = P.out.p;
  }
  return LP_OK;
}

int lp_forward_serial(lp_handle* h, const void* images, float* logits, void* stream) {
  if (!h || !images || !logits) return LP_ERR_NULL;
  if (!aligned16(images)) return LP_ERR_ALIGN;
  cudaStream_t st = (cudaStream_t)stream;
  Plan& L = h->modules[h->net.K - 1];
  int rc = serial_forward(h, images, nullptr, nullptr, st);
  if (rc != LP_OK) return rc;
  LP_CUDA_OK(cudaMemcpyAsync(logits, L.head.logits, (size_t)h->net.d.N * h->net.d.num_classes * 4,
                             cudaMemcpyDeviceToDevice, st));
  return LP_OK;
}

int lp_serial_fwd_bwd(lp_handle* h, const void* images, const int32_t* labels, float* loss_out, void* stream) {
  if (!h || !images || !labels || !loss_out) return LP_ERR_NULL;
  if (!aligned16(images)) return LP_ERR_ALIGN;
  cudaStream_t st = (cudaStream_t)stream;
  const int K = h->net.K;
  for (int k = 0; k < K; ++k) LP_CUDA_OK(cudaMemsetAsync(h->modules[k].ps.g, 0, h->modules[k].ps.n * 4, st));
  int rc = serial_forward(h, images, labels, loss_out, st);
  if (rc != LP_OK) return rc;
  for (int k = K - 1; k >= 0; --k) {
    Plan& P = h->modules[k];
    RunCtx c;
    c.st = st; c.serial = true; c.labels = labels;
    c.x = k == 0 ? images : h->modules[k - 1].out.p;
    c.dx = k > 0 ? h->modules[k - 1].seed.p : nullptr;  // adjoint handed to the previous module
    c.plan_id = k; c.phase = LP_PHASE_BACKWARD;
    rc = run_ops(h, P, P.bwd, c);
    if (rc != LP_OK) return rc;
    P.ps.grads_fresh = true;
  }
  return LP_OK;
}

int lp_get_residual(lp_handle* h, int k, void* r_dst, void* seed_dst, void* stream) {
  if (!h) return LP_ERR_NULL;
  if (k < 0 || k >= h->net.K - 1) return LP_ERR_BAD_INDEX;
  Plan& P = h->modules[k];
  if (!P.ran_fwd_bwd) return LP_ERR_ORDER;
  const size_t bytes = (size_t)P.r.elems() * esize(h->dtype);
  cudaStream_t st = (cudaStream_t)stream;
  if (r_dst) LP_CUDA_OK(cudaMemcpyAsync(r_dst, P.r.p, bytes, cudaMemcpyDeviceToDevice, st));
  if (seed_dst) LP_CUDA_OK(cudaMemcpyAsync(seed_dst, P.seed.p, bytes, cudaMemcpyDeviceToDevice, st));
  return LP_OK;
}

int lp_last_device_status(lp_handle* h, void* stream) {
  if (!h) return LP_ERR_NULL;
  if (cudaStreamSynchronize((cudaStream_t)stream) != cudaSuccess) return LP_ERR_CUDA;
  if (cudaDeviceSynchronize() != cudaSuccess) return LP_ERR_CUDA;
  int e = 0;
  if (cudaMemcpy(&e, h->dev_err, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) return LP_ERR_CUDA;
  if (e) {
    cudaMemset(h->dev_err, 0, sizeof(int));
    return LP_ERR_DEVICE_TIMEOUT;
  }
  return LP_OK;
}

int lp_selftest_bounded_wait(lp_handle* h, double limit_ms, double* waited_ms, void* stream) {
  if (!h) return LP_ERR_NULL;
  if (!(limit_ms > 0.0) || limit_ms > 100.0) return LP_ERR_SIZE;
  int dev = 0, khz = 0;
  LP_CUDA_OK(cudaGetDevice(&dev));
  LP_CUDA_OK(cudaDeviceGetAttribute(&khz, cudaDevAttrClockRate, dev));
  const long long limit_cycles = (long long)(limit_ms * (double)khz);
  cudaStream_t st = (cudaStream_t)stream;
  long long* waited = reinterpret_cast<long long*>(h->dev_err + 2);   // the error word's 256-byte slot
  tc::bounded_wait_selftest_kernel<<<1, 32, 0, st>>>(limit_cycles, h->dev_err, waited);
  h->launches++;
  LP_CUDA_OK(cudaGetLastError());
  if (waited_ms) {
    LP_CUDA_OK(cudaStreamSynchronize(st));
    long long w = 0;
    LP_CUDA_OK(cudaMemcpy(&w, waited, sizeof(w), cudaMemcpyDeviceToHost));
    *waited_ms = (double)w / (double)khz;
  }
  return LP_OK;
}

int64_t lp_launch_count(lp_handle* h, int reset) {
  if (!h) return 0;
  const int64_t v = h->launches;
  if (reset) h->launches = 0;
  return v;
}

int lp_conv_profile(lp_handle* h, int enable, double* ms, double* flops, int64_t* launches) {
  if (!h) return LP_ERR_NULL;
  ConvProfile& pr = h->prof;
  if (ms || flops || launches) {
    LP_CUDA_OK(cudaDeviceSynchronize());
    double t = 0, f = 0;
    for (size_t i = 0; i < pr.used; ++i) {
      float e = 0;
      if (cudaEventElapsedTime(&e, pr.events[i].first, pr.events[i].second) == cudaSuccess) t += e;
      f += pr.flops[i];
    }
    if (ms) *ms = t;
    if (flops) *flops = f;
    if (launches) *launches = (int64_t)pr.used;
  }
  pr.used = 0;
  pr.enabled = enable != 0;
  return LP_OK;
}

int lp_timeline(lp_handle* h, int enable, int max_records, lp_timeline_record* records, int* n_records) {
  if (!h) return LP_ERR_NULL;
  Timeline& tl = h->tl;
  if (records || n_records) {
    LP_CUDA_OK(cudaDeviceSynchronize());
    int n = 0;
    // times are relative to the earliest start among the records
    std::vector<float> t0(tl.used, 0.f), t1(tl.used, 0.f);
    size_t first = 0;
    for (size_t i = 1; i < tl.used; ++i) {
      float d = 0.f;
      if (cudaEventElapsedTime(&d, tl.recs[first].a, tl.recs[i].a) == cudaSuccess && d < 0.f) first = i;
    }
    for (size_t i = 0; i < tl.used; ++i) {
      if (cudaEventElapsedTime(&t0[i], tl.recs[first].a, tl.recs[i].a) != cudaSuccess) return LP_ERR_CUDA;
      if (cudaEventElapsedTime(&t1[i], tl.recs[first].a, tl.recs[i].b) != cudaSuccess) return LP_ERR_CUDA;
      if (records && n < max_records) {
        records[n].plan = tl.recs[i].plan; records[n].op = tl.recs[i].op_type; records[n].phase = tl.recs[i].phase;
        records[n].start_ms = t0[i]; records[n].end_ms = t1[i]; records[n].bytes = tl.recs[i].bytes;
      }
      ++n;
    }
    if (n_records) *n_records = n;
  }
  tl.used = 0;
  tl.enabled = enable != 0;
  return LP_OK;
}

int lp_graph_begin(lp_handle* h, void* stream) {
  if (!h) return LP_ERR_NULL;
  if (h->graphs.size() >= 8) return LP_ERR_UNSUPPORTED;
  if (h->prof.enabled || h->tl.enabled) return LP_ERR_ORDER;
  h->launches_at_capture = h->launches;
  LP_CUDA_OK(cudaStreamBeginCapture((cudaStream_t)stream, cudaStreamCaptureModeRelaxed));
  return LP_OK;
}

int lp_graph_end(lp_handle* h, void* stream, int* graph_id) {
  if (!h || !graph_id) return LP_ERR_NULL;
  cudaGraph_t g = nullptr;
  LP_CUDA_OK(cudaStreamEndCapture((cudaStream_t)stream, &g));
  cudaGraphExec_t exec = nullptr;
  cudaError_t e = cudaGraphInstantiate(&exec, g, 0);
  cudaGraphDestroy(g);
  if (e != cudaSuccess) return LP_ERR_CUDA;
  h->graphs.push_back(exec);
  h->graph_launches.push_back(h->launches - h->launches_at_capture);
  h->launches = h->launches_at_capture;  // recording launched nothing
  *graph_id = (int)h->graphs.size() - 1;
  return LP_OK;
}

int lp_graph_launch(lp_handle* h, int graph_id, void* stream) {
  if (!h) return LP_ERR_NULL;
  if (graph_id < 0 || graph_id >= (int)h->graphs.size()) return LP_ERR_BAD_INDEX;
  LP_CUDA_OK(cudaGraphLaunch(h->graphs[graph_id], (cudaStream_t)stream));
  h->launches += h->graph_launches[graph_id];
  for (auto& P : h->modules) { P.ran_fwd_bwd = true; }
  return LP_OK;
}

size_t lp_conv2d_scratch_bytes(int Cin, int Cout, int R) {
  const size_t n = (size_t)Cin * Cout * R * R;
  return align_up(n * 2, 256) * 2 + 256 + 1024;
}

int lp_conv2d(int op, int dtype, int impl, int N, int H, int W, int Cin, int Cout, int R, int stride, int pad,
              const void* a, const void* b, void* out, double* stats, void* scratch, size_t scratch_bytes,
              float* elapsed_ms, void* stream) {
  if (!a || !b || !out || !scratch) return LP_ERR_NULL;
  if (N < 1 || H < 1 || W < 1 || Cin < 1 || Cout < 1 || R < 1 || stride < 1 || pad < 0) return LP_ERR_SIZE;
  if (scratch_bytes < lp_conv2d_scratch_bytes(Cin, Cout, R)) return LP_ERR_WORKSPACE;
  if (!aligned16(a) || !aligned16(b) || !aligned16(out) || (reinterpret_cast<uintptr_t>(scratch) & 255)) return LP_ERR_ALIGN;
  int rc = init_cur_dev();
  if (rc != LP_OK) return rc;
  cudaStream_t st = (cudaStream_t)stream;
  ConvDef c;
  c.cin = Cin; c.cout = Cout; c.R = R; c.stride = stride; c.pad = pad; c.H = H; c.W = W;
  c.OH = conv_out(H, R, stride, pad); c.OW = conv_out(W, R, stride, pad);
  if (c.OH < 1 || c.OW < 1) return LP_ERR_SIZE;
  const size_t n = (size_t)Cin * Cout * R * R;
  uint8_t* sp = (uint8_t*)scratch;
  int* dev_err = (int*)sp;
  c.wf = (bf16*)(sp + 256);
  c.wt = (bf16*)(sp + 256 + align_up(n * 2, 256));
  LP_CUDA_OK(cudaMemsetAsync(dev_err, 0, 4, st));
  if (op != LP_CONV_WGRAD) {
    c.w = (float*)b;
    if (dtype == LP_BF16 && impl != LP_CONV_IMPL_SIMT) {
      // pack on the fly: one-entry table placed after the two weight copies is not available on the
      // device, so build it in pinned-free fashion: the table lives in the scratch tail
      PackEntry pe;
      pe.w = c.w; pe.wf = c.wf; pe.wt = c.wt; pe.cout = Cout; pe.taps = R * R; pe.cin = Cin; pe.begin = 0; pe.tile_begin = 0; pe.tile64_begin = 0;
      PackEntry* dpe = (PackEntry*)(sp + 256 + 2 * align_up(n * 2, 256));
      LP_CUDA_OK(cudaMemcpyAsync(dpe, &pe, sizeof(pe), cudaMemcpyHostToDevice, st));
      LP_CUDA_OK(cudaStreamSynchronize(st));
      pack_weights_kernel<<<grid_for((long long)n, 256, cur_dev().sm_count, 8), 256, 0, st>>>(dpe, 1, (long long)n);
      LP_CUDA_OK(cudaGetLastError());
    } else {
      c.wf = nullptr; c.wt = nullptr;
    }
  }
  cudaEvent_t e0 = nullptr, e1 = nullptr;
  if (elapsed_ms) {
    LP_CUDA_OK(cudaEventCreate(&e0));
    LP_CUDA_OK(cudaEventCreate(&e1));
  }
  if (op == LP_CONV_WGRAD) LP_CUDA_OK(cudaMemsetAsync(out, 0, n * 4, st));
  if (op == LP_CONV_FWD && stats) LP_CUDA_OK(cudaMemsetAsync(stats, 0, (size_t)2 * Cout * 8, st));
  if (e0) LP_CUDA_OK(cudaEventRecord(e0, st));
  if (op == LP_CONV_FWD) {
    bool done = false;
    rc = conv_forward(nullptr, dtype, impl, c, N, a, out, nullptr, stats, &done, dev_err, st);
    if (rc == LP_OK && stats && !done) {
      const int threads = threads_for_channels(Cout, dtype);
      const long long elems = (long long)N * c.OH * c.OW * Cout;
      if (!threads) rc = LP_ERR_UNSUPPORTED;
      else if (dtype == LP_F32)
        bn_stats_kernel<float><<<grid_for(elems / 4, threads * 8, cur_dev().sm_count, 4), threads, (size_t)threads * 8 * 4, st>>>(
            (const float*)out, elems / 4, Cout, stats);
      else
        bn_stats_kernel<bf16><<<grid_for(elems / 8, threads * 8, cur_dev().sm_count, 4), threads, (size_t)threads * 16 * 4, st>>>(
            (const bf16*)out, elems / 8, Cout, stats);
    }
  } else if (op == LP_CONV_DGRAD) {
    rc = conv_dgrad(nullptr, dtype, impl, c, N, a, out, nullptr, dev_err, st);
  } else if (op == LP_CONV_WGRAD) {
    rc = conv_wgrad(nullptr, dtype, impl, c, N, a, b, (float*)out, dev_err, st);
  } else {
    rc = LP_ERR_UNSUPPORTED;
  }
  if (e1) LP_CUDA_OK(cudaEventRecord(e1, st));
  if (rc != LP_OK) {
    if (e0) { cudaEventDestroy(e0); cudaEventDestroy(e1); }
    return rc;
  }
  LP_CUDA_OK(cudaStreamSynchronize(st));
  if (elapsed_ms) {
    cudaEventElapsedTime(elapsed_ms, e0, e1);
    cudaEventDestroy(e0);
    cudaEventDestroy(e1);
  }
  int e = 0;
  LP_CUDA_OK(cudaMemcpy(&e, dev_err, 4, cudaMemcpyDeviceToHost));
  return e ? LP_ERR_DEVICE_TIMEOUT : LP_OK;
}

// ---------------------------------------------------------------------------------------------
// Forward convolution without any caller- or library-side allocation: the scratch that lp_conv2d
// takes from its caller lives in this fixed device array instead.  In host code the array's name
// is only a handle: its device address is looked up once per device with cudaGetSymbolAddress.
// ---------------------------------------------------------------------------------------------
static __device__ __align__(256) unsigned char g_noalloc_scratch[LP_NOALLOC_SCRATCH_BYTES];
static void* g_noalloc_ptr[64] = {nullptr};

int lp_conv2d_fwd_noalloc(int N, int H, int W, int Cin, int Cout, int R, int stride, int pad, const void* x,
                          const float* w, void* y, void* stream) {
  if (!x || !w || !y) return LP_ERR_NULL;
  if (N < 1 || H < 1 || W < 1 || Cin < 1 || Cout < 1 || R < 1 || stride < 1 || pad < 0) return LP_ERR_SIZE;
  if (!aligned16(x) || !aligned16(w) || !aligned16(y)) return LP_ERR_ALIGN;
  const size_t n = (size_t)Cin * Cout * R * R;
  const size_t need = 256 + align_up(n * 2, 256) + 256;  // error word | bf16 weights | one-entry table
  if (need > (size_t)LP_NOALLOC_SCRATCH_BYTES) return LP_ERR_SIZE;
  int rc = init_cur_dev();
  if (rc != LP_OK) return rc;
  int dev = 0;
  LP_CUDA_OK(cudaGetDevice(&dev));
  if (dev < 0 || dev >= 64) return LP_ERR_UNSUPPORTED;
  if (!g_noalloc_ptr[dev]) {  // set-up, once per device, with that device current
    void* ptr = nullptr;
    if (cudaGetSymbolAddress((void**)&ptr, g_noalloc_scratch) != cudaSuccess || !ptr) return LP_ERR_CUDA;
    g_noalloc_ptr[dev] = ptr;
  }
  uint8_t* sp = (uint8_t*)g_noalloc_ptr[dev];
  cudaStream_t st = (cudaStream_t)stream;
  ConvDef c;
  c.cin = Cin; c.cout = Cout; c.R = R; c.stride = stride; c.pad = pad; c.H = H; c.W = W;
  c.OH = conv_out(H, R, stride, pad); c.OW = conv_out(W, R, stride, pad);
  if (c.OH < 1 || c.OW < 1) return LP_ERR_SIZE;
  if (!tc_fwd_ok(c)) return LP_ERR_UNSUPPORTED;
  int* dev_err = (int*)sp;
  c.w = const_cast<float*>(w);
  c.wf = (bf16*)(sp + 256);
  c.wt = nullptr;
  PackEntry pe;
  pe.w = c.w; pe.wf = c.wf; pe.wt = nullptr; pe.cout = Cout; pe.taps = R * R; pe.cin = Cin; pe.begin = 0; pe.tile_begin = 0; pe.tile64_begin = 0;
  PackEntry* dpe = (PackEntry*)(sp + 256 + align_up(n * 2, 256));
  LP_CUDA_OK(cudaMemsetAsync(dev_err, 0, 4, st));  // the only word that must start at zero
  LP_CUDA_OK(cudaMemcpyAsync(dpe, &pe, sizeof(pe), cudaMemcpyHostToDevice, st));
  LP_CUDA_OK(cudaStreamSynchronize(st));
  pack_weights_kernel<<<grid_for((long long)n, 256, cur_dev().sm_count, 8), 256, 0, st>>>(dpe, 1, (long long)n);
  LP_CUDA_OK(cudaGetLastError());
  bool done = false;
  rc = conv_forward(nullptr, LP_BF16, LP_CONV_IMPL_TENSOR, c, N, x, y, nullptr, nullptr, &done, dev_err, st);
  if (rc != LP_OK) return rc;
  LP_CUDA_OK(cudaStreamSynchronize(st));
  int e = 0;
  LP_CUDA_OK(cudaMemcpy(&e, dev_err, 4, cudaMemcpyDeviceToHost));
  return e ? LP_ERR_DEVICE_TIMEOUT : LP_OK;
}

}  // extern "C"
