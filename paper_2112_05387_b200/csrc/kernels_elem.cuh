// Elementwise and reduction kernels of the step: batch-norm statistics / apply / backward, ReLU,
// residual add, penalty / augmented-Lagrangian loss and terminal adjoint, pooling, head, updates.
// All tensors are NHWC; every thread moves 16 bytes per access and keeps a fixed channel group,
// so per-channel scale/shift live in registers (block size is a multiple of C / VEC).
#pragma once
#include "common.cuh"

namespace lp {

// The constants of V consecutive channels c0..c0+V-1 (V = 4 or 8, c0 a multiple of V): mean,
// 1/sqrt(var+eps), gamma, beta.  16-byte loads wherever the pointers allow: every thread of every
// block runs this prologue, and scalar loads at a stride of V channels between neighbouring
// threads (32 sectors per warp instruction, 4*V instructions) took longer than the pass itself.
template <int V>
__device__ __forceinline__ void bn_load_consts(const BnArgs& a, int C, int c0, float (&mean)[V], float (&rstd)[V],
                                               float (&gamma)[V], float (&beta)[V]) {
  double s1[V], s2[V];
  if ((reinterpret_cast<uintptr_t>(a.stats) & 15) == 0 && (C & 1) == 0) {
#pragma unroll
    for (int j = 0; j < V; j += 2) {
      const double2 u = *reinterpret_cast<const double2*>(a.stats + c0 + j);
      const double2 w = *reinterpret_cast<const double2*>(a.stats + C + c0 + j);
      s1[j] = u.x; s1[j + 1] = u.y; s2[j] = w.x; s2[j + 1] = w.y;
    }
  } else {
#pragma unroll
    for (int j = 0; j < V; ++j) { s1[j] = a.stats[c0 + j]; s2[j] = a.stats[C + c0 + j]; }
  }
  if (((reinterpret_cast<uintptr_t>(a.gamma + c0) | reinterpret_cast<uintptr_t>(a.beta + c0)) & 15) == 0) {
#pragma unroll
    for (int j = 0; j < V; j += 4) {
      const float4 g = *reinterpret_cast<const float4*>(a.gamma + c0 + j);
      const float4 b = *reinterpret_cast<const float4*>(a.beta + c0 + j);
      gamma[j] = g.x; gamma[j + 1] = g.y; gamma[j + 2] = g.z; gamma[j + 3] = g.w;
      beta[j] = b.x; beta[j + 1] = b.y; beta[j + 2] = b.z; beta[j + 3] = b.w;
    }
  } else {
#pragma unroll
    for (int j = 0; j < V; ++j) { gamma[j] = a.gamma[c0 + j]; beta[j] = a.beta[c0 + j]; }
  }
#pragma unroll
  for (int j = 0; j < V; ++j) bn_mean_rstd(s1[j], s2[j], a.inv_count, a.eps, mean[j], rstd[j]);
}

// Block-level tail of the per-channel reductions.  Every thread holds V sums of each of two kinds (a, b) for its
// fixed channel group (threadIdx.x % CV).  block_channel_partials() leaves partial sums in shared memory and
// returns how many there are per channel; block_channel_sum() adds them up for one (kind, channel) column.
// Where the channel groups line up with the lanes of a warp (CV divides 32), lanes of the same group are first
// added by shuffles, which leaves blockDim/32 partial sums per channel instead of blockDim/CV (8 instead of 120
// at 16 channels: that serial loop took longer than the pass over a small tensor).
template <int V>
__device__ __forceinline__ int block_channel_partials(float (&a)[V], float (&b)[V], float* sm, int C) {
  const int CV = C / V;
  if (CV <= 32 && (32 % CV) == 0 && (blockDim.x & 31) == 0) {
#pragma unroll
    for (int j = 0; j < V; ++j) {
      for (int o = CV; o < 32; o <<= 1) {
        a[j] += __shfl_xor_sync(0xffffffffu, a[j], o);
        b[j] += __shfl_xor_sync(0xffffffffu, b[j], o);
      }
    }
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    if (lane < CV) {
#pragma unroll
      for (int j = 0; j < V; ++j) {
        sm[(w * CV + lane) * 2 * V + j] = a[j];
        sm[(w * CV + lane) * 2 * V + V + j] = b[j];
      }
    }
    __syncthreads();
    return (int)(blockDim.x >> 5);
  }
#pragma unroll
  for (int j = 0; j < V; ++j) {
    sm[threadIdx.x * 2 * V + j] = a[j];
    sm[threadIdx.x * 2 * V + V + j] = b[j];
  }
  __syncthreads();
  return (int)blockDim.x / CV;
}
// kind 0: the a sums, kind 1: the b sums; c: channel.  Partial p of channel group g sits at row p*CV + g.
template <int V>
__device__ __forceinline__ float block_channel_sum(const float* sm, int C, int n_partials, int kind, int c) {
  const int CV = C / V;
  const int g = c / V, j = c % V;
  float acc = 0.f;
  for (int p = 0; p < n_partials; ++p) acc += sm[(p * CV + g) * 2 * V + kind * V + j];
  return acc;
}

// ---------------------------------------------------------------------------------------
// per-channel sum / sum of squares  ->  stats[2C] (double atomics, one per block and channel)
// ---------------------------------------------------------------------------------------
template <typename T>
__global__ void bn_stats_kernel(const T* __restrict__ x, long long total_vecs, int C, double* __restrict__ stats) {
  pdl_wait();
  pdl_launch_dependents();
  constexpr int V = VecT<T>::N;
  extern __shared__ float sm[];  // [blockDim][2*V]
  float s[V], q[V];
#pragma unroll
  for (int j = 0; j < V; ++j) s[j] = q[j] = 0.f;
  const long long stride = (long long)gridDim.x * blockDim.x;
  constexpr int U = 4;   // loads of a trip issued before the first use (see bn_apply_kernel)
  for (long long i0 = (long long)blockIdx.x * blockDim.x + threadIdx.x; i0 < total_vecs; i0 += U * stride) {
    uint4 rf[U];
#pragma unroll
    for (int u = 0; u < U; ++u)
      if (i0 + u * stride < total_vecs) rf[u] = ld_raw(x + (i0 + u * stride) * V);
#pragma unroll
    for (int u = 0; u < U; ++u) {
      if (i0 + u * stride >= total_vecs) break;
      float f[V];
      cvt_raw(rf[u], f);
#pragma unroll
      for (int j = 0; j < V; ++j) {
        s[j] += f[j];
        q[j] += f[j] * f[j];
      }
    }
  }
  // thread t < 2*C sums one (moment, channel) column of the block's partial sums
  const int n_partials = block_channel_partials<V>(s, q, sm, C);
  for (int t = threadIdx.x; t < 2 * C; t += blockDim.x)
    atomicAdd(&stats[t], (double)block_channel_sum<V>(sm, C, n_partials, t / C, t % C));
}

// ---------------------------------------------------------------------------------------
// out = [relu]( bnA(x) [+ bnB(x2)] [+ addend] )
// ---------------------------------------------------------------------------------------
// X2 / ADD select at compile time whether a second normalised input and a plain addend exist, so
// that the common one-input form keeps few enough registers for four 256-thread blocks per SM.
template <typename T, bool X2, bool ADD>
__global__ void __launch_bounds__(256, X2 ? 2 : (ADD ? 3 : 4))
bn_apply_kernel(const T* __restrict__ x, BnArgs A, const T* __restrict__ x2, BnArgs B,
                const T* __restrict__ addend, T* __restrict__ out, long long total_vecs, int C, int relu) {
  pdl_wait();
  pdl_launch_dependents();
  constexpr int V = VecT<T>::N;
  const int CV = C / V;
  const int c0 = (threadIdx.x % CV) * V;
  float sa[V], ta[V], sb[X2 ? V : 1], tb[X2 ? V : 1];
  {
    float mean[V], rstd[V], gamma[V], beta[V];
    bn_load_consts<V>(A, C, c0, mean, rstd, gamma, beta);
#pragma unroll
    for (int j = 0; j < V; ++j) {
      sa[j] = gamma[j] * rstd[j];
      ta[j] = beta[j] - mean[j] * sa[j];
    }
    if (X2) {
      bn_load_consts<V>(B, C, c0, mean, rstd, gamma, beta);
#pragma unroll
      for (int j = 0; j < V; ++j) {
        sb[X2 ? j : 0] = gamma[j] * rstd[j];
        tb[X2 ? j : 0] = beta[j] - mean[j] * sb[X2 ? j : 0];
      }
    }
  }
  const long long stride = (long long)gridDim.x * blockDim.x;
  // U vectors per thread and trip, all loads issued before the first use: with one 16-byte load
  // per thread a grid that fills the machine keeps only a few MB in flight, less than the
  // bandwidth-latency product of the memory system
  constexpr int U = 4;
  for (long long i0 = (long long)blockIdx.x * blockDim.x + threadIdx.x; i0 < total_vecs; i0 += U * stride) {
    uint4 rf[U], rg[X2 ? U : 1], ra[ADD ? U : 1];
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const long long i = i0 + u * stride;
      if (i < total_vecs) {
        rf[u] = ld_raw(x + i * V);
        if (X2) rg[X2 ? u : 0] = ld_raw(x2 + i * V);
        if (ADD) ra[ADD ? u : 0] = ld_raw(addend + i * V);
      }
    }
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const long long i = i0 + u * stride;
      if (i >= total_vecs) break;
      float f[V], y[V];
      cvt_raw(rf[u], f);
#pragma unroll
      for (int j = 0; j < V; ++j) y[j] = fmaf(f[j], sa[j], ta[j]);
      if (X2) {
        cvt_raw(rg[X2 ? u : 0], f);
#pragma unroll
        for (int j = 0; j < V; ++j) y[j] += f[j] * sb[X2 ? j : 0] + tb[X2 ? j : 0];
      }
      if (ADD) {
        cvt_raw(ra[ADD ? u : 0], f);
#pragma unroll
        for (int j = 0; j < V; ++j) y[j] += f[j];
      }
      if (relu) {
#pragma unroll
        for (int j = 0; j < V; ++j) y[j] = y[j] > 0.f ? y[j] : 0.f;
      }
      stv(out + i * V, y);
    }
  }
}

template <typename T>
void launch_bn_apply(int grid, int threads, cudaStream_t st, const T* x, const BnArgs& A, const T* x2, const BnArgs& B,
                     const T* addend, T* out, long long total_vecs, int C, int relu) {
  if (x2 && addend) launch_pdl(bn_apply_kernel<T, true, true>, dim3(grid), dim3(threads), 0, st, x, A, x2, B, addend, out, total_vecs, C, relu);
  else if (x2) launch_pdl(bn_apply_kernel<T, true, false>, dim3(grid), dim3(threads), 0, st, x, A, x2, B, addend, out, total_vecs, C, relu);
  else if (addend) launch_pdl(bn_apply_kernel<T, false, true>, dim3(grid), dim3(threads), 0, st, x, A, x2, B, addend, out, total_vecs, C, relu);
  else launch_pdl(bn_apply_kernel<T, false, false>, dim3(grid), dim3(threads), 0, st, x, A, x2, B, addend, out, total_vecs, C, relu);
}

// ---------------------------------------------------------------------------------------
// Interior local loss, fused into the kernel that produces the module output:
//   out = bnA(x) [+ bnB(x2)] [+ addend];  r = out - x_next;  seed = rho*r + kappa
// writes r and seed, accumulates sum r^2 and sum kappa*r (double atomics, one pair per block).
// With x == nullptr the output is taken from `addend` alone (already final).
// ---------------------------------------------------------------------------------------
template <typename T>
__global__ void module_out_loss_kernel(const T* __restrict__ x, BnArgs A, const T* __restrict__ x2, BnArgs B,
                                       const T* __restrict__ addend, const T* __restrict__ x_next,
                                       const T* __restrict__ kappa, float rho, T* __restrict__ r_out,
                                       T* __restrict__ seed_out, double* __restrict__ acc,
                                       long long total_vecs, int C) {
  constexpr int V = VecT<T>::N;
  const int CV = C / V;
  const int c0 = (threadIdx.x % CV) * V;
  float sa[V], ta[V], sb[V], tb[V];
#pragma unroll
  for (int j = 0; j < V; ++j) sa[j] = ta[j] = sb[j] = tb[j] = 0.f;
  {
    float mean[V], rstd[V], gamma[V], beta[V];
    if (x) {
      bn_load_consts<V>(A, C, c0, mean, rstd, gamma, beta);
#pragma unroll
      for (int j = 0; j < V; ++j) {
        sa[j] = gamma[j] * rstd[j];
        ta[j] = beta[j] - mean[j] * sa[j];
      }
    }
    if (x2) {
      bn_load_consts<V>(B, C, c0, mean, rstd, gamma, beta);
#pragma unroll
      for (int j = 0; j < V; ++j) {
        sb[j] = gamma[j] * rstd[j];
        tb[j] = beta[j] - mean[j] * sb[j];
      }
    }
  }
  float sum_rr = 0.f, sum_kr = 0.f;
  const long long stride = (long long)gridDim.x * blockDim.x;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total_vecs; i += stride) {
    float f[V], y[V], k[V];
#pragma unroll
    for (int j = 0; j < V; ++j) y[j] = 0.f;
    if (x) {
      ldv(x + i * V, f);
#pragma unroll
      for (int j = 0; j < V; ++j) y[j] = f[j] * sa[j] + ta[j];
    }
    if (x2) {
      ldv(x2 + i * V, f);
#pragma unroll
      for (int j = 0; j < V; ++j) y[j] += f[j] * sb[j] + tb[j];
    }
    if (addend) {
      ldv(addend + i * V, f);
#pragma unroll
      for (int j = 0; j < V; ++j) y[j] += f[j];
    }
    ldv(x_next + i * V, f);
#pragma unroll
    for (int j = 0; j < V; ++j) {
      y[j] -= f[j];  // r
      sum_rr += y[j] * y[j];
    }
    stv(r_out + i * V, y);
    if (kappa) {
      ldv(kappa + i * V, k);
#pragma unroll
      for (int j = 0; j < V; ++j) {
        sum_kr += k[j] * y[j];
        y[j] = rho * y[j] + k[j];
      }
    } else {
#pragma unroll
      for (int j = 0; j < V; ++j) y[j] = rho * y[j];
    }
    stv(seed_out + i * V, y);
  }
  // Block sums through shared memory: the block size follows the channel count (240 threads for 160, 320
  // or 640 bf16 channels), so the last warp may be partial and full-mask shuffles are not available to it.
  __shared__ float red[2][1024];
  red[0][threadIdx.x] = sum_rr;
  red[1][threadIdx.x] = sum_kr;
  __syncthreads();
  if (threadIdx.x < 32) {
    float a = 0.f, b = 0.f;
    for (int t = threadIdx.x; t < (int)blockDim.x; t += 32) {
      a += red[0][t];
      b += red[1][t];
    }
    a = warp_sum(a);   // warp 0 is always complete: block sizes are at least 32
    b = warp_sum(b);
    if (threadIdx.x == 0) {
      atomicAdd(&acc[0], (double)a);
      atomicAdd(&acc[1], (double)b);
    }
  }
}

__global__ void loss_finalize_kernel(const double* __restrict__ acc, float rho, float* __restrict__ loss_out) {
  loss_out[0] = (float)(0.5 * (double)rho * acc[0] + acc[1]);
  loss_out[1] = (float)acc[0];
}

// ---------------------------------------------------------------------------------------
// BN backward.  dy_m = dy * [bn(x) > 0] when a ReLU followed the normalisation (relu_mask): the
// mask is recomputed from x with the forward kernel's own expression instead of being read back.
//   reduce: dbeta += sum dy_m ; dgamma += sum dy_m * xhat
//   apply : dx = gamma*rstd*(dy_m - dbeta/M - xhat*dgamma/M) [+ addend]
// ---------------------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(256, 2)
bn_bwd_reduce_kernel(const T* __restrict__ dy, const T* __restrict__ x, int relu_mask,
                                     BnArgs A, float* __restrict__ dgamma, float* __restrict__ dbeta,
                                     long long total_vecs, int C) {
  pdl_wait();
  pdl_launch_dependents();
  constexpr int V = VecT<T>::N;
  extern __shared__ float sm[];
  const int CV = C / V;
  const int c0 = (threadIdx.x % CV) * V;
  float mean[V], rstd[V], sb[V], sg[V], sa[V], ta[V];
  {
    float gamma[V], beta[V];
    bn_load_consts<V>(A, C, c0, mean, rstd, gamma, beta);
#pragma unroll
    for (int j = 0; j < V; ++j) {
      sa[j] = gamma[j] * rstd[j];
      ta[j] = beta[j] - mean[j] * sa[j];
      sb[j] = sg[j] = 0.f;
    }
  }
  const long long stride = (long long)gridDim.x * blockDim.x;
  constexpr int U = 4;
  for (long long i0 = (long long)blockIdx.x * blockDim.x + threadIdx.x; i0 < total_vecs; i0 += U * stride) {
    uint4 rd[U], rx[U];
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const long long i = i0 + u * stride;
      if (i < total_vecs) {
        rd[u] = ld_raw(dy + i * V);
        rx[u] = ld_raw(x + i * V);
      }
    }
#pragma unroll
    for (int u = 0; u < U; ++u) {
      if (i0 + u * stride >= total_vecs) break;
      float d[V], f[V];
      cvt_raw(rd[u], d);
      cvt_raw(rx[u], f);
      if (relu_mask) {
#pragma unroll
        for (int j = 0; j < V; ++j) d[j] = fmaf(f[j], sa[j], ta[j]) > 0.f ? d[j] : 0.f;
      }
#pragma unroll
      for (int j = 0; j < V; ++j) {
        sb[j] += d[j];
        sg[j] += d[j] * (f[j] - mean[j]) * rstd[j];
      }
    }
  }
  const int n_partials = block_channel_partials<V>(sb, sg, sm, C);
  for (int t = threadIdx.x; t < 2 * C; t += blockDim.x) {
    const float acc = block_channel_sum<V>(sm, C, n_partials, t / C, t % C);
    atomicAdd(t / C ? &dgamma[t % C] : &dbeta[t % C], acc);
  }
}

template <typename T>
__global__ void __launch_bounds__(256, 2)
bn_bwd_apply_kernel(const T* __restrict__ dy, const T* __restrict__ x, int relu_mask, BnArgs A,
                    const float* __restrict__ dgamma, const float* __restrict__ dbeta,
                    const T* __restrict__ addend, T* __restrict__ out, long long total_vecs, int C) {
  pdl_wait();
  pdl_launch_dependents();
  constexpr int V = VecT<T>::N;
  const int CV = C / V;
  const int c0 = (threadIdx.x % CV) * V;
  // dx = sc*(dy_m - mb - xhat*mg) = sc*dy_m + a2*x + a3   with xhat = (x - mean)*rstd
  float sc[V], ta[V], a2[V], a3[V];
  const float invM = (float)A.inv_count;
  {
    float mean[V], rstd[V], gamma[V], beta[V];
    bn_load_consts<V>(A, C, c0, mean, rstd, gamma, beta);
    const bool vec = ((reinterpret_cast<uintptr_t>(dbeta + c0) | reinterpret_cast<uintptr_t>(dgamma + c0)) & 15) == 0;
#pragma unroll
    for (int j = 0; j < V; j += 4) {
      float4 b, g;
      if (vec) {
        b = *reinterpret_cast<const float4*>(dbeta + c0 + j);
        g = *reinterpret_cast<const float4*>(dgamma + c0 + j);
      } else {
        b = make_float4(dbeta[c0 + j], dbeta[c0 + j + 1], dbeta[c0 + j + 2], dbeta[c0 + j + 3]);
        g = make_float4(dgamma[c0 + j], dgamma[c0 + j + 1], dgamma[c0 + j + 2], dgamma[c0 + j + 3]);
      }
      const float mb[4] = {b.x * invM, b.y * invM, b.z * invM, b.w * invM};
      const float mg[4] = {g.x * invM, g.y * invM, g.z * invM, g.w * invM};
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        sc[j + q] = gamma[j + q] * rstd[j + q];
        ta[j + q] = beta[j + q] - mean[j + q] * sc[j + q];
        a2[j + q] = -sc[j + q] * rstd[j + q] * mg[q];
        a3[j + q] = -sc[j + q] * mb[q] - a2[j + q] * mean[j + q];
      }
    }
  }
  const long long stride = (long long)gridDim.x * blockDim.x;
  constexpr int U = 4;
  for (long long i0 = (long long)blockIdx.x * blockDim.x + threadIdx.x; i0 < total_vecs; i0 += U * stride) {
    uint4 rd[U], rx[U], ra[U];
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const long long i = i0 + u * stride;
      if (i < total_vecs) {
        rd[u] = ld_raw(dy + i * V);
        rx[u] = ld_raw(x + i * V);
        if (addend) ra[u] = ld_raw(addend + i * V);
      }
    }
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const long long i = i0 + u * stride;
      if (i >= total_vecs) break;
      float d[V], f[V], o[V];
      cvt_raw(rd[u], d);
      cvt_raw(rx[u], f);
      if (relu_mask) {
#pragma unroll
        for (int j = 0; j < V; ++j) d[j] = fmaf(f[j], sc[j], ta[j]) > 0.f ? d[j] : 0.f;
      }
#pragma unroll
      for (int j = 0; j < V; ++j) o[j] = fmaf(sc[j], d[j], fmaf(a2[j], f[j], a3[j]));
      if (addend) {
        cvt_raw(ra[u], f);
#pragma unroll
        for (int j = 0; j < V; ++j) o[j] += f[j];
      }
      stv(out + i * V, o);
    }
  }
}

// out = a + b
template <typename T>
__global__ void add_kernel(const T* __restrict__ a, const T* __restrict__ b, T* __restrict__ out, long long total_vecs) {
  constexpr int V = VecT<T>::N;
  const long long stride = (long long)gridDim.x * blockDim.x;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total_vecs; i += stride) {
    float f[V], g[V];
    ldv(a + i * V, f);
    ldv(b + i * V, g);
#pragma unroll
    for (int j = 0; j < V; ++j) f[j] += g[j];
    stv(out + i * V, f);
  }
}

// ---------------------------------------------------------------------------------------
// 3x3 / stride 2 / pad 1 max-pool; the first maximum in (r,s) scan order wins (stored as 0..8).
// ---------------------------------------------------------------------------------------
// A thread handles VecT<T>::N consecutive channels of one pixel (16-byte accesses; C is a multiple of that).
template <typename T>
__global__ void maxpool_fwd_kernel(const T* __restrict__ x, T* __restrict__ y, uint8_t* __restrict__ arg, int N,
                                   int H, int W, int C, int OH, int OW) {
  constexpr int V = VecT<T>::N;
  const int CV = C / V;
  const long long total = (long long)N * OH * OW * CV;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total;
       i += (long long)gridDim.x * blockDim.x) {
    const int cg = (int)(i % CV);
    long long p = i / CV;
    const int ow = (int)(p % OW);
    p /= OW;
    const int oh = (int)(p % OH);
    const int n = (int)(p / OH);
    float best[V];
    int ba[V];
#pragma unroll
    for (int j = 0; j < V; ++j) { best[j] = -INFINITY; ba[j] = 0; }
    for (int r = 0; r < 3; ++r) {
      const int ih = oh * 2 + r - 1;
      if (ih < 0 || ih >= H) continue;
      for (int s = 0; s < 3; ++s) {
        const int iw = ow * 2 + s - 1;
        if (iw < 0 || iw >= W) continue;
        float v[V];
        ldv(x + (((long long)n * H + ih) * W + iw) * C + cg * V, v);
#pragma unroll
        for (int j = 0; j < V; ++j)
          if (v[j] > best[j]) { best[j] = v[j]; ba[j] = r * 3 + s; }
      }
    }
    stv(y + i * V, best);
    uint8_t* ap = arg + i * V;
#pragma unroll
    for (int j = 0; j < V; j += 4)
      *reinterpret_cast<uint32_t*>(ap + j) = (uint32_t)ba[j] | ((uint32_t)ba[j + 1] << 8) | ((uint32_t)ba[j + 2] << 16) |
                                             ((uint32_t)ba[j + 3] << 24);
  }
}

template <typename T>
__global__ void maxpool_bwd_kernel(const T* __restrict__ dy, const uint8_t* __restrict__ arg, T* __restrict__ dx,
                                   int N, int H, int W, int C, int OH, int OW) {
  constexpr int V = VecT<T>::N;
  const int CV = C / V;
  const long long total = (long long)N * H * W * CV;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total;
       i += (long long)gridDim.x * blockDim.x) {
    const int cg = (int)(i % CV);
    long long p = i / CV;
    const int iw = (int)(p % W);
    p /= W;
    const int ih = (int)(p % H);
    const int n = (int)(p / H);
    float acc[V];
#pragma unroll
    for (int j = 0; j < V; ++j) acc[j] = 0.f;
    for (int r = 0; r < 3; ++r) {
      const int t = ih + 1 - r;
      if (t < 0 || (t & 1)) continue;
      const int oh = t >> 1;
      if (oh >= OH) continue;
      for (int s = 0; s < 3; ++s) {
        const int u = iw + 1 - s;
        if (u < 0 || (u & 1)) continue;
        const int ow = u >> 1;
        if (ow >= OW) continue;
        const long long o = ((((long long)n * OH + oh) * OW + ow) * CV + cg) * V;
        float d[V];
        ldv(dy + o, d);
        const uint8_t* ap = arg + o;
        const int want = r * 3 + s;
#pragma unroll
        for (int j = 0; j < V; j += 4) {
          const uint32_t a4 = *reinterpret_cast<const uint32_t*>(ap + j);
#pragma unroll
          for (int q = 0; q < 4; ++q)
            if ((int)((a4 >> (8 * q)) & 255u) == want) acc[j + q] += d[j + q];
        }
      }
    }
    stv(dx + i * V, acc);
  }
}

// ---------------------------------------------------------------------------------------
// head: global average pool, linear + softmax cross-entropy (mean over the batch), backward
// ---------------------------------------------------------------------------------------
template <typename T>
__global__ void avgpool_kernel(const T* __restrict__ x, float* __restrict__ pooled, int HW, int C) {
  // grid: N blocks; thread c-strided
  const int n = blockIdx.x;
  for (int c = threadIdx.x; c < C; c += blockDim.x) {
    float acc = 0.f;
    const T* p = x + (long long)n * HW * C + c;
    for (int i = 0; i < HW; ++i) acc += to_f(p[(long long)i * C]);
    pooled[(long long)n * C + c] = acc / (float)HW;
  }
}

// logits[n][j] = bias[j] + sum_c W[j][c] * pooled[n][c].  One warp per class and tile of 8 samples: the
// weight row is read once (coalesced) for the eight dot products.
__global__ void __launch_bounds__(128)
head_logits_kernel(const float* __restrict__ pooled, const float* __restrict__ Wt, const float* __restrict__ bias,
                   float* __restrict__ logits, int N, int C, int classes) {
  const int lane = threadIdx.x & 31;
  const int j = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const int n0 = blockIdx.y * 8;
  if (j >= classes) return;
  float acc[8];
#pragma unroll
  for (int s = 0; s < 8; ++s) acc[s] = 0.f;
  const float* w = Wt + (long long)j * C;
  for (int c = lane; c < C; c += 32) {
    const float wv = w[c];
#pragma unroll
    for (int s = 0; s < 8; ++s)
      if (n0 + s < N) acc[s] += wv * pooled[(long long)(n0 + s) * C + c];
  }
#pragma unroll
  for (int s = 0; s < 8; ++s) {
    const float v = warp_sum(acc[s]);
    if (lane == 0 && n0 + s < N) logits[(long long)(n0 + s) * classes + j] = v + bias[j];
  }
}

// one block per sample; softmax of the logits, loss (atomic mean), dlogits = (softmax - onehot)/N
__global__ void head_fwd_kernel(const int32_t* __restrict__ labels, const float* __restrict__ logits,
                                float* __restrict__ dlogits, double* __restrict__ loss_acc, int N, int classes) {
  extern __shared__ float sh[];  // [classes] logits, then reduction scratch [32]
  float* lg = sh;
  float* red = sh + classes;
  const int n = blockIdx.x;
  for (int j = threadIdx.x; j < classes; j += blockDim.x) lg[j] = logits[(long long)n * classes + j];
  __syncthreads();
  float mx = -INFINITY;
  for (int j = threadIdx.x; j < classes; j += blockDim.x) mx = fmaxf(mx, lg[j]);
  for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = mx;
  __syncthreads();
  mx = -INFINITY;
  for (int i = 0; i < (blockDim.x + 31) / 32; ++i) mx = fmaxf(mx, red[i]);
  __syncthreads();
  float se = 0.f;
  for (int j = threadIdx.x; j < classes; j += blockDim.x) se += __expf(lg[j] - mx);
  se = warp_sum(se);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = se;
  __syncthreads();
  se = 0.f;
  for (int i = 0; i < (blockDim.x + 31) / 32; ++i) se += red[i];
  const float lse = logf(se) + mx;
  const int lab = labels[n];
  for (int j = threadIdx.x; j < classes; j += blockDim.x) {
    const float p = __expf(lg[j] - lse);
    dlogits[(long long)n * classes + j] = (p - (j == lab ? 1.f : 0.f)) / (float)N;
  }
  if (threadIdx.x == 0) atomicAdd(loss_acc, (double)(lse - lg[lab]) / (double)N);
}

// Heads of few classes (at most 128: the CIFAR-shaped networks) in one launch, one block of 256 threads per
// sample: the average pool (kept in shared memory and written out for the backward pass), the logits (one warp
// per class, the same summation order as head_logits_kernel) and, by the first warp, softmax, loss and dlogits.
// Three dependent launches of a few microseconds of work each become one on the last module's chain.
template <typename T>
__global__ void __launch_bounds__(256)
head_fused_kernel(const T* __restrict__ x, const float* __restrict__ Wt, const float* __restrict__ bias,
                  const int32_t* __restrict__ labels, float* __restrict__ pooled, float* __restrict__ logits,
                  float* __restrict__ dlogits, double* __restrict__ loss_acc, int N, int HW, int C, int classes) {
  extern __shared__ float sh[];  // [C] pooled, then [classes] logits
  float* sp = sh;
  float* lg = sh + C;
  const int n = blockIdx.x;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  for (int c = threadIdx.x; c < C; c += blockDim.x) {
    float acc = 0.f;
    const T* p = x + (long long)n * HW * C + c;
    for (int i = 0; i < HW; ++i) acc += to_f(p[(long long)i * C]);
    const float v = acc / (float)HW;
    pooled[(long long)n * C + c] = v;
    sp[c] = v;
  }
  __syncthreads();
  for (int j = warp; j < classes; j += (int)(blockDim.x >> 5)) {
    const float* w = Wt + (long long)j * C;
    float acc = 0.f;
    for (int c = lane; c < C; c += 32) acc += w[c] * sp[c];
    acc = warp_sum(acc);
    if (lane == 0) {
      const float v = acc + bias[j];
      lg[j] = v;
      logits[(long long)n * classes + j] = v;
    }
  }
  __syncthreads();
  if (warp != 0) return;
  float mx = -INFINITY;
  for (int j = lane; j < classes; j += 32) mx = fmaxf(mx, lg[j]);
  for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
  float se = 0.f;
  for (int j = lane; j < classes; j += 32) se += __expf(lg[j] - mx);
  se = warp_sum(se);
  const float lse = logf(se) + mx;
  const int lab = labels[n];
  for (int j = lane; j < classes; j += 32) {
    const float pj = __expf(lg[j] - lse);
    dlogits[(long long)n * classes + j] = (pj - (j == lab ? 1.f : 0.f)) / (float)N;
  }
  if (lane == 0) atomicAdd(loss_acc, (double)(lse - lg[lab]) / (double)N);
}

__global__ void ce_finalize_kernel(const double* __restrict__ acc, float* __restrict__ loss_out) {
  loss_out[0] = (float)acc[0];
  loss_out[1] = 0.f;
}

// dW[j][c] = sum_n dlogits[n][j]*pooled[n][c]; db[j] = sum_n dlogits[n][j]
__global__ void head_bwd_w_kernel(const float* __restrict__ dlogits, const float* __restrict__ pooled,
                                  float* __restrict__ dW, float* __restrict__ db, int N, int C, int classes) {
  const long long total = (long long)classes * C;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total;
       i += (long long)gridDim.x * blockDim.x) {
    const int j = (int)(i / C), c = (int)(i % C);
    float acc = 0.f;
    for (int n = 0; n < N; ++n) acc += dlogits[(long long)n * classes + j] * pooled[(long long)n * C + c];
    dW[i] = acc;
    if (c == 0) {
      float b = 0.f;
      for (int n = 0; n < N; ++n) b += dlogits[(long long)n * classes + j];
      db[j] = b;
    }
  }
}

// d[n,h,w,c] = (sum_j dlogits[n][j] W[j][c]) / HW, broadcast over the pixels
template <typename T>
__global__ void head_bwd_x_kernel(const float* __restrict__ dlogits, const float* __restrict__ Wt, T* __restrict__ d,
                                  int HW, int C, int classes) {
  const int n = blockIdx.x;
  const int c = blockIdx.y * blockDim.x + threadIdx.x;   // grid.y covers the channels
  if (c >= C) return;
  const float* dl = dlogits + (long long)n * classes;
  float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
  int j = 0;
  for (; j + 4 <= classes; j += 4) {
    a0 += dl[j] * Wt[(long long)j * C + c];
    a1 += dl[j + 1] * Wt[(long long)(j + 1) * C + c];
    a2 += dl[j + 2] * Wt[(long long)(j + 2) * C + c];
    a3 += dl[j + 3] * Wt[(long long)(j + 3) * C + c];
  }
  for (; j < classes; ++j) a0 += dl[j] * Wt[(long long)j * C + c];
  const float acc = ((a0 + a1) + (a2 + a3)) / (float)HW;
  T v;
  from_f(v, acc);
  T* p = d + (long long)n * HW * C + c;
  for (int i = 0; i < HW; ++i) p[(long long)i * C] = v;
}

// ---------------------------------------------------------------------------------------
// updates
// ---------------------------------------------------------------------------------------
__global__ void sgd_kernel(float* __restrict__ p, const float* __restrict__ g, float* __restrict__ mom, long long n,
                           float lr, float momentum, float wd) {
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x) {
    float gi = g[i] + wd * p[i];
    if (momentum != 0.f) {
      gi = momentum * mom[i] + gi;
      mom[i] = gi;
    }
    p[i] -= lr * gi;
  }
}

template <typename T>
__global__ void kappa_update_kernel(T* __restrict__ kappa, const T* __restrict__ r, float c, long long total_vecs) {
  constexpr int V = VecT<T>::N;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total_vecs;
       i += (long long)gridDim.x * blockDim.x) {
    float k[V], f[V];
    ldv(kappa + i * V, k);
    ldv(r + i * V, f);
#pragma unroll
    for (int j = 0; j < V; ++j) k[j] += c * f[j];
    stv(kappa + i * V, k);
  }
}

// Correction of an auxiliary variable and seed of the AuxNet distillation:
//   g = dx_k - seed_{k-1};  x_new = x_k - lr*g (optional output);  d = 2*(x_k - x_new) = 2*lr*g;
//   acc[0] += sum (lr*g)^2   (the distillation loss ||x_new - AuxNet(x_{k-1})||^2 before the update)
template <typename T>
__global__ void distill_seed_kernel(const T* xk, const T* __restrict__ dxk, const T* __restrict__ seed_prev,
                                    float lr, T* x_new /* may alias xk */, T* __restrict__ d_out /* nullable */, double* __restrict__ acc,
                                    long long total_vecs) {
  constexpr int V = VecT<T>::N;
  float sum = 0.f;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total_vecs;
       i += (long long)gridDim.x * blockDim.x) {
    float a[V], b[V], x[V];
    ldv(dxk + i * V, a);
    ldv(seed_prev + i * V, b);
#pragma unroll
    for (int j = 0; j < V; ++j) {
      a[j] = lr * (a[j] - b[j]);
      sum += a[j] * a[j];
    }
    if (x_new) {
      ldv(xk + i * V, x);
#pragma unroll
      for (int j = 0; j < V; ++j) x[j] -= a[j];
      stv(x_new + i * V, x);
    }
    if (d_out) {
#pragma unroll
      for (int j = 0; j < V; ++j) a[j] *= 2.f;
      stv(d_out + i * V, a);
    }
  }
  __shared__ float red[32];
  sum = warp_sum(sum);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = sum;
  __syncthreads();
  if (threadIdx.x < 32) {
    float v = threadIdx.x < (blockDim.x + 31) / 32 ? red[threadIdx.x] : 0.f;
    v = warp_sum(v);
    if (threadIdx.x == 0) atomicAdd(&acc[0], (double)v);
  }
}

__global__ void distill_loss_kernel(const double* __restrict__ acc, float* __restrict__ loss_out) {
  loss_out[0] = (float)acc[0];
}

// bf16 operand copies of one convolution's fp32 master weights w[co][t][ci]:
//   wf[co][t*Cin + ci]  (forward B operand, K-major)      wt[ci][t*Cout + co]  (dgrad B operand)
struct PackEntry {
  const float* w;
  bf16* wf;
  bf16* wt;  // may be null
  int cout, taps, cin;
  long long begin;       // first flat element index handled for this entry
  long long tile_begin;  // first 32x32 tile index of this entry (tiled kernel)
  long long tile64_begin;  // first 64x64 tile index of this entry (sgd_pack_tiled64_kernel)
};

__global__ void pack_weights_kernel(const PackEntry* __restrict__ tab, int n_entries, long long total) {
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total;
       i += (long long)gridDim.x * blockDim.x) {
    int lo = 0, hi = n_entries - 1;
    while (lo < hi) {
      const int mid = (lo + hi + 1) >> 1;
      if (tab[mid].begin <= i) lo = mid; else hi = mid - 1;
    }
    const PackEntry e = tab[lo];
    const long long j = i - e.begin;
    const float v = e.w[j];
    const bf16 b = __float2bfloat16_rn(v);
    e.wf[j] = b;
    if (e.wt) {
      const int ci = (int)(j % e.cin);
      const long long q = j / e.cin;
      const int t = (int)(q % e.taps);
      const int co = (int)(q / e.taps);
      e.wt[((long long)ci * e.taps + t) * e.cout + co] = b;
    }
  }
}

// Same copies, one 32 (c_out) x 32 (c_in) tile of one tap per block: reads and both writes are
// coalesced (the transposed copy goes through shared memory).  blockDim = (32, 8).
__global__ void pack_weights_tiled_kernel(const PackEntry* __restrict__ tab, int n_entries) {
  __shared__ float tile[32][33];
  const long long b = blockIdx.x;
  int lo = 0, hi = n_entries - 1;
  while (lo < hi) {
    const int mid = (lo + hi + 1) >> 1;
    if (tab[mid].tile_begin <= b) lo = mid; else hi = mid - 1;
  }
  const PackEntry e = tab[lo];
  const int tiles_ci = (e.cin + 31) >> 5, tiles_co = (e.cout + 31) >> 5;
  int r = (int)(b - e.tile_begin);
  const int ci0 = (r % tiles_ci) << 5;
  r /= tiles_ci;
  const int co0 = (r % tiles_co) << 5;
  const int t = r / tiles_co;
  const int tx = threadIdx.x, ty = threadIdx.y;
  for (int i = ty; i < 32; i += 8) {
    const int co = co0 + i, ci = ci0 + tx;
    float v = 0.f;
    if (co < e.cout && ci < e.cin) {
      const long long j = ((long long)co * e.taps + t) * e.cin + ci;
      v = e.w[j];
      e.wf[j] = __float2bfloat16_rn(v);
    }
    tile[i][tx] = v;
  }
  if (!e.wt) return;
  __syncthreads();
  for (int i = ty; i < 32; i += 8) {
    const int ci = ci0 + i, co = co0 + tx;
    if (co < e.cout && ci < e.cin) e.wt[((long long)ci * e.taps + t) * e.cout + co] = __float2bfloat16_rn(tile[tx][i]);
  }
}

// The update and the weight copies in one pass over the packed convolution weights:
//   w <- w - lr*(g + wd*w [momentum])   then the two bf16 copies of the new w, as above,
// on 64 (c_out) x 64 (c_in) tiles of one tap with 16-byte accesses: a thread holds four float4 pieces of the
// parameters and of the gradients (128 bytes of loads in flight), the K-major copy leaves in 8-byte pieces and
// the transposed one, through shared memory, in 128-byte rows of 64 output channels.  `p_base` / `g_base` /
// `m_base` are the parameter, gradient and momentum blobs the entries point into (m_base may be null when
// momentum is 0).  Requires c_in % 4 == 0, c_out % 2 == 0 and 16-byte aligned weight tensors inside the blobs
// (checked when the table is built; otherwise the plain update and pack_weights_tiled_kernel run instead).
// blockDim = 256.
__global__ void __launch_bounds__(256)
sgd_pack_tiled64_kernel(const PackEntry* __restrict__ tab, int n_entries, float* __restrict__ p_base,
                        const float* __restrict__ g_base, float* __restrict__ m_base, float lr, float momentum, float wd) {
  __shared__ float tile[64][65];
  const long long b = blockIdx.x;
  int lo = 0, hi = n_entries - 1;
  while (lo < hi) {
    const int mid = (lo + hi + 1) >> 1;
    if (tab[mid].tile64_begin <= b) lo = mid; else hi = mid - 1;
  }
  const PackEntry e = tab[lo];
  const long long base = e.w - p_base;
  const int tiles_ci = (e.cin + 63) >> 6, tiles_co = (e.cout + 63) >> 6;
  int r = (int)(b - e.tile64_begin);
  const int ci0 = (r % tiles_ci) << 6;
  r /= tiles_ci;
  const int co0 = (r % tiles_co) << 6;
  const int t = r / tiles_co;
  const int tid = threadIdx.x;
  const int cx = (tid & 15) << 2, ry = tid >> 4;   // four input channels of one of 16 rows per pass
  const int ci = ci0 + cx;
  float4 pv[4], gv[4], mv[4];
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    const int co = co0 + ry + 16 * q;
    pv[q] = gv[q] = mv[q] = make_float4(0.f, 0.f, 0.f, 0.f);
    if (co < e.cout && ci < e.cin) {
      const long long j = base + ((long long)co * e.taps + t) * e.cin + ci;
      pv[q] = *reinterpret_cast<const float4*>(p_base + j);
      gv[q] = *reinterpret_cast<const float4*>(g_base + j);
      if (momentum != 0.f) mv[q] = *reinterpret_cast<const float4*>(m_base + j);
    }
  }
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    const int row = ry + 16 * q;
    const int co = co0 + row;
    float v[4] = {0.f, 0.f, 0.f, 0.f};
    if (co < e.cout && ci < e.cin) {
      const long long j = ((long long)co * e.taps + t) * e.cin + ci;
      const float pw[4] = {pv[q].x, pv[q].y, pv[q].z, pv[q].w};
      const float gw[4] = {gv[q].x, gv[q].y, gv[q].z, gv[q].w};
      const float mw[4] = {mv[q].x, mv[q].y, mv[q].z, mv[q].w};
      float gi[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        gi[u] = gw[u] + wd * pw[u];
        if (momentum != 0.f) gi[u] = momentum * mw[u] + gi[u];
        v[u] = pw[u] - lr * gi[u];
      }
      if (momentum != 0.f) *reinterpret_cast<float4*>(m_base + base + j) = make_float4(gi[0], gi[1], gi[2], gi[3]);
      *reinterpret_cast<float4*>(p_base + base + j) = make_float4(v[0], v[1], v[2], v[3]);
      const __nv_bfloat162 lo2 = __floats2bfloat162_rn(v[0], v[1]), hi2 = __floats2bfloat162_rn(v[2], v[3]);
      uint2 pk;
      pk.x = *reinterpret_cast<const uint32_t*>(&lo2);
      pk.y = *reinterpret_cast<const uint32_t*>(&hi2);
      *reinterpret_cast<uint2*>(e.wf + j) = pk;
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) tile[row][cx + u] = v[u];
  }
  if (!e.wt) return;
  __syncthreads();
  const int warp = tid >> 5, lane = tid & 31;
  const int co = co0 + 2 * lane;
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const int cil = warp + 8 * i;
    const int ci2 = ci0 + cil;
    if (ci2 < e.cin && co < e.cout) {
      const __nv_bfloat162 v2 = __floats2bfloat162_rn(tile[2 * lane][cil], tile[2 * lane + 1][cil]);
      *reinterpret_cast<__nv_bfloat162*>(e.wt + ((long long)ci2 * e.taps + t) * e.cout + co) = v2;
    }
  }
}

// ---------------------------------------------------------------------------------------
// 7x7 / stride 2 / pad 3 stem convolution on the tensor cores by space-to-depth.
// The image x[N][H][W][C] (C <= 4, H and W even) is regrouped as xs[N][H/2][W/2][16]: channel (by*2 + bx)*C + c of
// pixel (i, j) is x[2i + by][2j + bx][c] (channels 4C..15 are zero).  Since input row 2*oh + r - 3 = 2*(oh + a) + by
// with a = floor((r - 3) / 2) in {-2..1}, the convolution becomes a 4x4 stride-1 convolution over xs with taps
// a_h, a_w in {-2..1} (tap index (a_h + 2)*4 + (a_w + 2)) and weights
//   ws[co][tap][(by*2 + bx)*C + c] = w[co][2*a_h + by + 3][2*a_w + bx + 3][c]   (zero where that row or column is not 0..6).
// ---------------------------------------------------------------------------------------
template <typename T>
__global__ void s2d_input_kernel(const T* __restrict__ x, bf16* __restrict__ xs, int N, int H, int W, int C) {
  const int OH = H >> 1, OW = W >> 1;
  const long long total = (long long)N * OH * OW;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (long long)gridDim.x * blockDim.x) {
    const int ow = (int)(i % OW);
    long long q = i / OW;
    const int oh = (int)(q % OH);
    const int n = (int)(q / OH);
    float v[16];
#pragma unroll
    for (int j = 0; j < 16; ++j) v[j] = 0.f;
    for (int by = 0; by < 2; ++by)
      for (int bx = 0; bx < 2; ++bx) {
        const T* px = x + (((long long)n * H + 2 * oh + by) * W + 2 * ow + bx) * C;
        for (int c = 0; c < C; ++c) v[(by * 2 + bx) * C + c] = to_f(px[c]);
      }
    uint4 lo, hi;
    lo.x = pack_bf16x2(v[0], v[1]); lo.y = pack_bf16x2(v[2], v[3]); lo.z = pack_bf16x2(v[4], v[5]); lo.w = pack_bf16x2(v[6], v[7]);
    hi.x = pack_bf16x2(v[8], v[9]); hi.y = pack_bf16x2(v[10], v[11]); hi.z = pack_bf16x2(v[12], v[13]); hi.w = pack_bf16x2(v[14], v[15]);
    uint4* dst = reinterpret_cast<uint4*>(xs + i * 16);
    dst[0] = lo;
    dst[1] = hi;
  }
}

// ws[co][16 taps][16 channels] (bf16) from w[co][7][7][C] (fp32)
__global__ void s2d_pack_weights_kernel(const float* __restrict__ w, bf16* __restrict__ ws, int Cout, int C) {
  const int total = Cout * 256;
  for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < total; i += gridDim.x * blockDim.x) {
    const int ch = i & 15, tap = (i >> 4) & 15, co = i >> 8;
    float v = 0.f;
    if (ch < 4 * C) {
      const int blk = ch / C, c = ch % C;
      const int by = blk >> 1, bx = blk & 1;
      const int r = 2 * ((tap >> 2) - 2) + by + 3, q = 2 * ((tap & 3) - 2) + bx + 3;
      if (r >= 0 && r < 7 && q >= 0 && q < 7) v = w[(((long long)co * 7 + r) * 7 + q) * C + c];
    }
    ws[i] = __float2bfloat16_rn(v);
  }
}

// gw[co][7][7][C] = the entries of dws[co][16 taps][16 channels] that correspond to real filter positions
__global__ void s2d_unpack_wgrad_kernel(const float* __restrict__ dws, float* __restrict__ gw, int Cout, int C) {
  const int total = Cout * 49 * C;
  for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < total; i += gridDim.x * blockDim.x) {
    const int c = i % C;
    int t = i / C;
    const int q = t % 7;
    t /= 7;
    const int r = t % 7, co = t / 7;
    const int by = (r + 1) & 1, bx = (q + 1) & 1;            // r - 3 = 2a + by with by in {0, 1}
    const int ah = (r - 3 - by) / 2, aw = (q - 3 - bx) / 2;   // exact: the numerators are even
    const int tap = (ah + 2) * 4 + (aw + 2);
    gw[i] = dws[((long long)co * 16 + tap) * 16 + (by * 2 + bx) * C + c];
  }
}

// Plain update of the parameters that have no packed copy (normalisation, head, convolutions on
// the CUDA-core path): one block per range of the blob.
struct SgdRange {
  long long begin;
  int count;
};
__global__ void sgd_ranges_kernel(const SgdRange* __restrict__ ranges, float* __restrict__ p,
                                  const float* __restrict__ g, float* __restrict__ mom, float lr, float momentum,
                                  float wd) {
  const SgdRange r = ranges[blockIdx.x];
  for (int i = threadIdx.x; i < r.count; i += blockDim.x) {
    const long long j = r.begin + i;
    float gi = g[j] + wd * p[j];
    if (momentum != 0.f) {
      gi = momentum * mom[j] + gi;
      mom[j] = gi;
    }
    p[j] -= lr * gi;
  }
}

}  // namespace lp
