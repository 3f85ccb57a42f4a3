// Benchmark-side measurement aid (built and loaded by bench.py; no part of the
// library): the rate at which this GPU issues dependent-free multiply-adds, so
// that the benchmark can quote achieved arithmetic against a peak measured in
// the same run.
#include <cuda_runtime.h>

enum { PROBE_OK = 0, PROBE_ERR = -1 };

namespace {

// 8 independent chains per thread, operands that repeat (the rate the pipe reaches at best)
template <typename R>
__global__ void __launch_bounds__(256) bench_probe_fma_kernel(R *out, int iters) {
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
  if (cudaGetDevice(&dev) != cudaSuccess) return PROBE_ERR;
  if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return PROBE_ERR;
  R *out = nullptr;
  if (cudaMalloc(&out, sizeof(R)) != cudaSuccess) return PROBE_ERR;
  cudaEvent_t e0, e1;
  cudaEventCreate(&e0);
  cudaEventCreate(&e1);
  const int grid = sms * 8, iters = 1 << 14;
  bench_probe_fma_kernel<R><<<grid, 256, 0, stream>>>(out, iters);   // warm-up
  cudaEventRecord(e0, stream);
  bench_probe_fma_kernel<R><<<grid, 256, 0, stream>>>(out, iters);
  cudaEventRecord(e1, stream);
  float ms = 0.f;
  const cudaError_t err = cudaEventSynchronize(e1);
  if (err == cudaSuccess) cudaEventElapsedTime(&ms, e0, e1);
  cudaEventDestroy(e0);
  cudaEventDestroy(e1);
  cudaFree(out);
  if (err != cudaSuccess || ms <= 0.f) return PROBE_ERR;
  *tflops = 2.0 * 8.0 * iters * 256.0 * grid / (ms * 1e-3) / 1e12;
  return PROBE_OK;
}

}  // namespace

// float64 != 0: the float64 pipe, else the float32 pipe; *tflops (HOST) receives the measured rate
extern "C" int bench_probe_fma(int float64, double *tflops, void *cuda_stream) {
  if (!tflops) return PROBE_ERR;
  return float64 ? probe<double>(tflops, (cudaStream_t)cuda_stream) : probe<float>(tflops, (cudaStream_t)cuda_stream);
}
