// A measurement aid, not part of the inference path: the rate at which this GPU
// issues dependent-free multiply-adds, so that a benchmark can quote achieved
// arithmetic against a peak measured in the same run.
#include <cuda_runtime.h>

#include "bi.h"

namespace {

// 8 independent chains per thread, operands that repeat (the rate the pipe reaches at best)
template <typename R>
__global__ void __launch_bounds__(256) bi_probe_fma_kernel(R *out, int iters) {
  R a[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) a[i] = (R)(threadIdx.x * 1e-3) + (R)i;
  const R m = (R)1.0000001, c = (R)1e-9;
  for (int q = 0; q < iters; ++q) {
#pragma unroll
    for (int i = 0; i < 8; ++i) a[i] = fma(a[i], m, c);
  }
  R s = (R)0;
#pragma unroll
  for (int i = 0; i < 8; ++i) s += a[i];
  if (s == (R)-1) out[0] = s;   // never true: keeps the chains alive without a store per thread
}

template <typename R>
int probe(double *tflops, cudaStream_t stream) {
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return BI_ERR_CUDA;
  if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return BI_ERR_CUDA;
  R *out = nullptr;
  if (cudaMalloc(&out, sizeof(R)) != cudaSuccess) return BI_ERR_ALLOC;
  cudaEvent_t e0, e1;
  cudaEventCreate(&e0);
  cudaEventCreate(&e1);
  const int grid = sms * 8, iters = 1 << 14;
  bi_probe_fma_kernel<R><<<grid, 256, 0, stream>>>(out, iters);   // warm-up
  cudaEventRecord(e0, stream);
  bi_probe_fma_kernel<R><<<grid, 256, 0, stream>>>(out, iters);
  cudaEventRecord(e1, stream);
  float ms = 0.f;
  const cudaError_t err = cudaEventSynchronize(e1);
  if (err == cudaSuccess) cudaEventElapsedTime(&ms, e0, e1);
  cudaEventDestroy(e0);
  cudaEventDestroy(e1);
  cudaFree(out);
  if (err != cudaSuccess || ms <= 0.f) return BI_ERR_CUDA;
  *tflops = 2.0 * 8.0 * iters * 256.0 * grid / (ms * 1e-3) / 1e12;
  return BI_OK;
}

}  // namespace

extern "C" int bi_probe_fma(int arith, double *tflops, void *cuda_stream) {
  if (!tflops || (arith != BI_ARITH_F64 && arith != BI_ARITH_F32)) return BI_ERR_INVALID_ARG;
  return arith == BI_ARITH_F64 ? probe<double>(tflops, (cudaStream_t)cuda_stream)
                               : probe<float>(tflops, (cudaStream_t)cuda_stream);
}
