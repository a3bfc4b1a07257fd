// Shared device helpers: 16-byte vector access for fp32 / bf16 activations.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace lp {

typedef __nv_bfloat16 bf16;

template <typename T>
struct VecT;
template <>
struct VecT<float> {
  static constexpr int N = 4;
};
template <>
struct VecT<bf16> {
  static constexpr int N = 8;
};

// Load / store VecT<T>::N consecutive elements (16 bytes) as floats.
__device__ __forceinline__ void ldv(const float* p, float (&f)[4]) {
  float4 v = *reinterpret_cast<const float4*>(p);
  f[0] = v.x; f[1] = v.y; f[2] = v.z; f[3] = v.w;
}
__device__ __forceinline__ void ldv(const bf16* p, float (&f)[8]) {
  uint4 v = *reinterpret_cast<const uint4*>(p);
  const uint32_t u[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    f[2 * i] = __uint_as_float(u[i] << 16);
    f[2 * i + 1] = __uint_as_float(u[i] & 0xFFFF0000u);
  }
}
// The same in two steps: a raw 16-byte load now, the conversion when the values are needed, so
// that several loads can be in flight per thread without holding their unpacked values.
template <typename T>
__device__ __forceinline__ uint4 ld_raw(const T* p) { return *reinterpret_cast<const uint4*>(p); }
__device__ __forceinline__ void cvt_raw(const uint4& v, float (&f)[4]) {
  f[0] = __uint_as_float(v.x); f[1] = __uint_as_float(v.y); f[2] = __uint_as_float(v.z); f[3] = __uint_as_float(v.w);
}
__device__ __forceinline__ void cvt_raw(const uint4& v, float (&f)[8]) {
  const uint32_t u[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    f[2 * i] = __uint_as_float(u[i] << 16);
    f[2 * i + 1] = __uint_as_float(u[i] & 0xFFFF0000u);
  }
}
__device__ __forceinline__ void stv(float* p, const float (&f)[4]) {
  *reinterpret_cast<float4*>(p) = make_float4(f[0], f[1], f[2], f[3]);
}
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&h);
}
__device__ __forceinline__ void stv(bf16* p, const float (&f)[8]) {
  uint4 v;
  v.x = pack_bf16x2(f[0], f[1]);
  v.y = pack_bf16x2(f[2], f[3]);
  v.z = pack_bf16x2(f[4], f[5]);
  v.w = pack_bf16x2(f[6], f[7]);
  *reinterpret_cast<uint4*>(p) = v;
}
__device__ __forceinline__ float to_f(float v) { return v; }
__device__ __forceinline__ float to_f(bf16 v) { return __bfloat162float(v); }
__device__ __forceinline__ void from_f(float& d, float v) { d = v; }
__device__ __forceinline__ void from_f(bf16& d, float v) { d = __float2bfloat16_rn(v); }

// Value a store of `v` in type T would leave in memory, as float (storage rounding).
template <typename T>
__device__ __forceinline__ float round_storage(float v) {
  T t;
  from_f(t, v);
  return to_f(t);
}

// Training-mode batch norm of one tensor: per-channel sums of the batch and the affine parameters.
struct BnArgs {
  const double* stats;  // [2*C]: per-channel sum, sum of squares
  const float* gamma;
  const float* beta;
  double inv_count;     // 1 / (N*H*W)
  float eps;
};

// Mean and 1/sqrt(var + eps) of one channel from its sums.  Every kernel that normalises, or that
// recomputes a ReLU mask from a normalised value, goes through this function, so that all of them
// see the same two numbers.
__device__ __forceinline__ void bn_mean_rstd(double s1, double s2, double inv_count, float eps, float& mean, float& rstd) {
  const double m = s1 * inv_count;
  const double var = fma(-m, m, s2 * inv_count);
  mean = (float)m;
  const float v = fmaxf((float)var, 0.f) + eps;
  float r = rsqrtf(v);
  r = r * fmaf(-0.5f * v * r, r, 1.5f);
  rstd = r;
}


// Programmatic dependent launch.  A kernel launched with the programmatic-serialisation attribute
// may start while the kernel before it in the stream is still draining: everything up to
// pdl_wait() (barrier set-up, tensor-memory allocation, constants) overlaps that tail; pdl_wait()
// returns once the preceding grid has completed and its memory is visible, so nothing that depends
// on it may come earlier.  Every such kernel executes it unconditionally, which also keeps the
// stream order transitive.  pdl_launch_dependents() lets the NEXT kernel begin its own prologue as
// soon as this grid's blocks have all passed that point and resources free up.  Launched without
// the attribute both are no-ops.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// Host side: launch with programmatic stream serialisation allowed (see pdl_wait).
#ifndef LP_PDL
#define LP_PDL 1
#endif
template <typename... KArgs, typename... Args>
static inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                                     Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = LP_PDL;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

}  // namespace lp
