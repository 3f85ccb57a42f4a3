// Small device helpers shared by the kernels; every one is generic over the
// arithmetic type R (float or double).
#pragma once
#include <cuda_runtime.h>
#include <math_constants.h>
#include <stdint.h>

template <typename R>
struct __align__(16) Vec4 {
  R x, y, z, w;
};

__device__ __forceinline__ Vec4<float> ldg4(const float *p) {
  float4 v = __ldg(reinterpret_cast<const float4 *>(p));
  return Vec4<float>{v.x, v.y, v.z, v.w};
}
__device__ __forceinline__ Vec4<double> ldg4(const double *p) {
  double2 a = __ldg(reinterpret_cast<const double2 *>(p));
  double2 b = __ldg(reinterpret_cast<const double2 *>(p) + 1);
  return Vec4<double>{a.x, a.y, b.x, b.y};
}

template <typename R>
__device__ __forceinline__ R warp_sum(R v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
template <typename R>
__device__ __forceinline__ R bi_max(R a, R b) { return a > b ? a : b; }
template <typename R>
__device__ __forceinline__ R warp_max(R v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = bi_max(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}

template <typename R> __device__ __forceinline__ R bi_inf();
template <> __device__ __forceinline__ float bi_inf<float>() { return CUDART_INF_F; }
template <> __device__ __forceinline__ double bi_inf<double>() { return CUDART_INF; }

__device__ __forceinline__ float bi_exp(float x) { return expf(x); }
__device__ __forceinline__ double bi_exp(double x) { return exp(x); }
__device__ __forceinline__ float bi_log(float x) { return logf(x); }
__device__ __forceinline__ double bi_log(double x) { return log(x); }

// index into [0, hi); out-of-range values are clamped and flagged, never trapped
__device__ __forceinline__ int clamp_flag(int v, int hi, uint32_t *status, uint32_t flag) {
  if (v < 0 || v >= hi) {
    atomicOr(status, flag);
    v = v < 0 ? 0 : hi - 1;
  }
  return v;
}
