// Direct (CUDA-core) convolution kernels: any filter size, stride, padding and channel count.
// They carry the fp32 workload (tensor cores have no true-fp32 mode) and the few bf16 shapes
// the tensor-core path does not take (3-channel stems).  fp32 accumulation throughout;
// weights are the fp32 masters w[co][r][s][ci], rounded to the activation type as they are read
// so that both convolution paths of a bf16 network contract the same operands.
#pragma once
#include "common.cuh"

namespace lp {

struct ConvGeom {
  int N, H, W, Cin;      // input
  int OH, OW, Cout;      // output
  int R, S, stride, pad;
};

// y[n,oh,ow,co..co+3] = sum_{r,s,ci} w[co][r][s][ci] * x[n, oh*st+r-p, ow*st+s-p, ci]  (+ addend)
template <typename T>
__global__ void conv_fwd_simt_kernel(const T* __restrict__ x, const float* __restrict__ w, const T* __restrict__ addend,
                                     T* __restrict__ y, ConvGeom g) {
  const int CG = g.Cout >> 2;
  const long long total = (long long)g.N * g.OH * g.OW * CG;
  const long long tap_stride = (long long)g.R * g.S * g.Cin;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total;
       i += (long long)gridDim.x * blockDim.x) {
    const int co = (int)(i % CG) * 4;
    long long p = i / CG;
    const int ow = (int)(p % g.OW);
    long long q = p / g.OW;
    const int oh = (int)(q % g.OH);
    const int n = (int)(q / g.OH);
    float acc[4] = {0.f, 0.f, 0.f, 0.f};
    for (int r = 0; r < g.R; ++r) {
      const int ih = oh * g.stride + r - g.pad;
      if (ih < 0 || ih >= g.H) continue;
      for (int s = 0; s < g.S; ++s) {
        const int iw = ow * g.stride + s - g.pad;
        if (iw < 0 || iw >= g.W) continue;
        const T* xp = x + (((long long)n * g.H + ih) * g.W + iw) * g.Cin;
        const float* wp = w + ((long long)co * g.R * g.S + (r * g.S + s)) * g.Cin;
        for (int ci = 0; ci < g.Cin; ++ci) {
          const float xv = to_f(xp[ci]);
#pragma unroll
          for (int j = 0; j < 4; ++j) acc[j] += xv * round_storage<T>(__ldg(wp + j * tap_stride + ci));
        }
      }
    }
    const long long o = p * g.Cout + co;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      float v = acc[j];
      if (addend) v += to_f(addend[o + j]);
      from_f(y[o + j], v);
    }
  }
}

// dx[n,ih,iw,ci..ci+3] = sum_{r,s,co : (ih+p-r) % st == 0 ...} dy[n,(ih+p-r)/st,(iw+p-s)/st,co] * w[co][r][s][ci]
template <typename T>
__global__ void conv_dgrad_simt_kernel(const T* __restrict__ dy, const float* __restrict__ w,
                                       const T* __restrict__ addend, T* __restrict__ dx, ConvGeom g) {
  const int CG = g.Cin >> 2;
  const long long total = (long long)g.N * g.H * g.W * CG;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total;
       i += (long long)gridDim.x * blockDim.x) {
    const int ci = (int)(i % CG) * 4;
    long long p = i / CG;
    const int iw = (int)(p % g.W);
    long long q = p / g.W;
    const int ih = (int)(q % g.H);
    const int n = (int)(q / g.H);
    float acc[4] = {0.f, 0.f, 0.f, 0.f};
    for (int r = 0; r < g.R; ++r) {
      const int th = ih + g.pad - r;
      if (th < 0 || th % g.stride) continue;
      const int oh = th / g.stride;
      if (oh >= g.OH) continue;
      for (int s = 0; s < g.S; ++s) {
        const int tw = iw + g.pad - s;
        if (tw < 0 || tw % g.stride) continue;
        const int ow = tw / g.stride;
        if (ow >= g.OW) continue;
        const T* dp = dy + (((long long)n * g.OH + oh) * g.OW + ow) * g.Cout;
        const float* wp = w + (long long)(r * g.S + s) * g.Cin + ci;
        for (int co = 0; co < g.Cout; ++co) {
          const float d = to_f(dp[co]);
          const float4 wv = __ldg(reinterpret_cast<const float4*>(wp + (long long)co * g.R * g.S * g.Cin));
          acc[0] += d * round_storage<T>(wv.x);
          acc[1] += d * round_storage<T>(wv.y);
          acc[2] += d * round_storage<T>(wv.z);
          acc[3] += d * round_storage<T>(wv.w);
        }
      }
    }
    const long long o = p * g.Cin + ci;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      float v = acc[j];
      if (addend) v += to_f(addend[o + j]);
      from_f(dx[o + j], v);
    }
  }
}

// dw[co][r][s][ci] += sum over the block's pixel chunk of dy[n,oh,ow,co] * x[n,oh*st+r-p,ow*st+s-p,ci]
// grid.x: chunks of output elements, grid.y: pixel chunks; dw must be zero before the launch.
template <typename T>
__global__ void conv_wgrad_simt_kernel(const T* __restrict__ x, const T* __restrict__ dy, float* __restrict__ dw,
                                       ConvGeom g, int pixels_per_chunk) {
  const int n_out = g.Cout * g.R * g.S * g.Cin;
  const int o = blockIdx.x * blockDim.x + threadIdx.x;
  if (o >= n_out) return;
  const int ci = o % g.Cin;
  int t = o / g.Cin;
  const int s = t % g.S;
  t /= g.S;
  const int r = t % g.R;
  const int co = t / g.R;
  const long long npix = (long long)g.N * g.OH * g.OW;
  long long p0 = (long long)blockIdx.y * pixels_per_chunk;
  long long p1 = p0 + pixels_per_chunk;
  if (p1 > npix) p1 = npix;
  int ow = (int)(p0 % g.OW);
  long long q = p0 / g.OW;
  int oh = (int)(q % g.OH);
  int n = (int)(q / g.OH);
  float acc = 0.f;
  for (long long p = p0; p < p1; ++p) {
    const int ih = oh * g.stride + r - g.pad, iw = ow * g.stride + s - g.pad;
    if (ih >= 0 && ih < g.H && iw >= 0 && iw < g.W)
      acc += to_f(dy[p * g.Cout + co]) * to_f(x[(((long long)n * g.H + ih) * g.W + iw) * g.Cin + ci]);
    if (++ow == g.OW) {
      ow = 0;
      if (++oh == g.OH) {
        oh = 0;
        ++n;
      }
    }
  }
  atomicAdd(&dw[o], acc);
}

// ---------------------------------------------------------------------------------------------
// Few input channels (the 3-channel stems and the first AuxNet convolution): K = R*S*Cin is tiny,
// so the whole filter bank fits in shared memory.  A thread produces CPT output channels of one
// pixel: one activation load and CPT/4 broadcast reads of the filter bank feed CPT multiply-adds.
// Same operands as the generic kernels (weights rounded to the activation type, fp32 accumulation).
// ---------------------------------------------------------------------------------------------
template <typename T, int CPT>
__global__ void __launch_bounds__(256)
conv_fwd_fewch_kernel(const T* __restrict__ x, const float* __restrict__ w, T* __restrict__ y, ConvGeom g) {
  constexpr int V = VecT<T>::N;
  extern __shared__ float ws[];            // [K][Cout], K = R*S*Cin
  const int K = g.R * g.S * g.Cin;
  for (int i = threadIdx.x; i < K * g.Cout; i += blockDim.x) {
    const int k = i / g.Cout, co = i % g.Cout;
    ws[i] = round_storage<T>(w[(long long)co * K + k]);
  }
  __syncthreads();
  const int CG = g.Cout / CPT;
  const long long total = (long long)g.N * g.OH * g.OW * CG;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total;
       i += (long long)gridDim.x * blockDim.x) {
    const int cg = (int)(i % CG);
    const long long p = i / CG;
    const int ow = (int)(p % g.OW);
    const long long q = p / g.OW;
    const int oh = (int)(q % g.OH);
    const int n = (int)(q / g.OH);
    float acc[CPT];
#pragma unroll
    for (int j = 0; j < CPT; ++j) acc[j] = 0.f;
    for (int r = 0; r < g.R; ++r) {
      const int ih = oh * g.stride + r - g.pad;
      if (ih < 0 || ih >= g.H) continue;
      for (int s = 0; s < g.S; ++s) {
        const int iw = ow * g.stride + s - g.pad;
        if (iw < 0 || iw >= g.W) continue;
        const T* xp = x + (((long long)n * g.H + ih) * g.W + iw) * g.Cin;
        const float* wr = ws + (r * g.S + s) * g.Cin * g.Cout + cg * CPT;
        for (int ci = 0; ci < g.Cin; ++ci) {
          const float xv = to_f(xp[ci]);
#pragma unroll
          for (int j4 = 0; j4 < CPT; j4 += 4) {
            const float4 wv = *reinterpret_cast<const float4*>(wr + ci * g.Cout + j4);
            acc[j4] += xv * wv.x; acc[j4 + 1] += xv * wv.y; acc[j4 + 2] += xv * wv.z; acc[j4 + 3] += xv * wv.w;
          }
        }
      }
    }
#pragma unroll
    for (int j = 0; j < CPT; j += V) stv(y + p * g.Cout + cg * CPT + j, *reinterpret_cast<float(*)[V]>(&acc[j]));
  }
}

// Weight gradient for few input channels.  A thread owns one filter position k = (r, s, ci) and
// CPT output channels, and walks the pixels of its block's range: per pixel one activation load
// and CPT/V 16-byte loads of dy (the same for every thread of a channel group) feed CPT
// multiply-adds.  With few (k, group) pairs the block's threads also split into pixel lanes, summed
// through shared memory (threads * CPT floats, dynamic) before one atomic add per output.
// dw must be zero before the launch.
template <typename T, int CPT>
__global__ void __launch_bounds__(256)
conv_wgrad_fewch_kernel(const T* __restrict__ x, const T* __restrict__ dy, float* __restrict__ dw, ConvGeom g,
                        int pair_threads, long long pixels_per_block) {
  constexpr int V = VecT<T>::N;
  extern __shared__ float red[];
  const int K = g.R * g.S * g.Cin;
  const int CG = g.Cout / CPT;
  const int npairs = K * CG;
  const int PL = blockDim.x / pair_threads;          // pixel lanes
  const int pl = threadIdx.x / pair_threads, pt = threadIdx.x % pair_threads;
  const bool live = pt < npairs;
  const int k = live ? pt / CG : 0, cg = live ? pt % CG : 0;
  const int ci = k % g.Cin, fs = (k / g.Cin) % g.S, fr = k / (g.Cin * g.S);
  float acc[CPT];
#pragma unroll
  for (int j = 0; j < CPT; ++j) acc[j] = 0.f;
  const long long npix = (long long)g.N * g.OH * g.OW;
  const long long p0 = (long long)blockIdx.x * pixels_per_block;
  long long p1 = p0 + pixels_per_block;
  if (p1 > npix) p1 = npix;
  if (live && p0 + pl < p1) {
    long long p = p0 + pl;
    int ow = (int)(p % g.OW);
    long long t = p / g.OW;
    int oh = (int)(t % g.OH);
    int n = (int)(t / g.OH);
    for (; p < p1; p += PL) {
      const int ih = oh * g.stride + fr - g.pad, iw = ow * g.stride + fs - g.pad;
      if (ih >= 0 && ih < g.H && iw >= 0 && iw < g.W) {
        const float xv = to_f(x[(((long long)n * g.H + ih) * g.W + iw) * g.Cin + ci]);
        const T* dp = dy + p * g.Cout + cg * CPT;
#pragma unroll
        for (int j = 0; j < CPT; j += V) {
          float f[V];
          ldv(dp + j, f);
#pragma unroll
          for (int u = 0; u < V; ++u) acc[j + u] += xv * f[u];
        }
      }
      ow += PL;
      while (ow >= g.OW) {
        ow -= g.OW;
        if (++oh == g.OH) { oh = 0; ++n; }
      }
    }
  }
  if (PL > 1) {
#pragma unroll
    for (int j = 0; j < CPT; ++j) red[threadIdx.x * CPT + j] = acc[j];
    __syncthreads();
    if (pl == 0)
      for (int l = 1; l < PL; ++l)
#pragma unroll
        for (int j = 0; j < CPT; ++j) acc[j] += red[(l * pair_threads + pt) * CPT + j];
  }
  if (pl == 0 && live) {
#pragma unroll
    for (int j = 0; j < CPT; ++j) atomicAdd(&dw[(long long)(cg * CPT + j) * K + k], acc[j]);
  }
}

}  // namespace lp
