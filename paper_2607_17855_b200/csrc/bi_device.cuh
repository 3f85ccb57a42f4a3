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
// Branch-free exp for softmax arguments (x <= about 0 after the shift; exact
// zero below -700, where the true value is below 1e-304).  The library exp()
// carries special-case branches, which keep the compiler from interleaving
// the independent exponentials of a sweep; this one is straight-line code, so
// three of them overlap.  Cody-Waite reduction by ln 2 (two constants), degree
// 13 Taylor polynomial split into even and odd halves, scaling through the
// exponent field.  Measured against exp() over [-700, 50]: within 3.2e-16
// relative (about 1.4 ulp).
__device__ __forceinline__ double bi_exp_inline(double x) {
  const double L2E = 1.4426950408889634074, LN2H = 6.93147180369123816490e-01, LN2L = 1.90821492927058770002e-10;
  const double MAGIC = 6755399441055744.0;  // 1.5 * 2^52: adding it rounds to the nearest integer
  double t = fma(x, L2E, MAGIC);
  const int k = __double2loint(t);
  const double kd = t - MAGIC;
  double r = fma(kd, -LN2H, x);
  r = fma(kd, -LN2L, r);
  const double r2 = r * r;
  double E = 1.0 / 479001600.0;
  E = fma(E, r2, 1.0 / 3628800.0);
  E = fma(E, r2, 1.0 / 40320.0);
  E = fma(E, r2, 1.0 / 720.0);
  E = fma(E, r2, 1.0 / 24.0);
  E = fma(E, r2, 0.5);
  E = fma(E, r2, 1.0);
  double O = 1.0 / 6227020800.0;
  O = fma(O, r2, 1.0 / 39916800.0);
  O = fma(O, r2, 1.0 / 362880.0);
  O = fma(O, r2, 1.0 / 5040.0);
  O = fma(O, r2, 1.0 / 120.0);
  O = fma(O, r2, 1.0 / 6.0);
  O = fma(O, r2, 1.0);
  const double p = fma(O, r, E);
  const double res = __hiloint2double(__double2hiint(p) + (k << 20), __double2loint(p));
  return x < -700.0 ? 0.0 : res;
}
__device__ __forceinline__ float bi_exp_inline(float x) { return expf(x); }

// The same with a 32-entry table of 2^(j/32) (in shared memory: tab): the reduced
// argument is then below ln2/64 and a degree-6 polynomial suffices, 13 FP64
// operations instead of 19.  exp(x) = 2^(k>>5) * tab[k&31] * exp(r),
// k = round(x * 32/ln2), r = x - k ln2/32.  Same range and accuracy.
__device__ __forceinline__ double bi_exp_tab(double x, const double *tab) {
  const double K32 = 46.166241308446828384, LH = 6.93147180369123816490e-01 / 32.0, LL = 1.90821492927058770002e-10 / 32.0;
  const double MAGIC = 6755399441055744.0;
  double t = fma(x, K32, MAGIC);
  const int k = __double2loint(t);
  const double kd = t - MAGIC;
  double r = fma(kd, -LH, x);
  r = fma(kd, -LL, r);
  const double T = tab[k & 31];
  const double r2 = r * r;
  const double a = fma(r, 1.0 / 6.0, 0.5);
  double b = fma(r, 1.0 / 120.0, 1.0 / 24.0);
  b = fma(r2, 1.0 / 720.0, b);
  const double c = fma(r2, b, a);
  const double p = fma(r2, c, r);
  const double res = fma(T, p, T);
  const double out = __hiloint2double(__double2hiint(res) + ((k >> 5) << 20), __double2loint(res));
  return x < -700.0 ? 0.0 : out;
}
__device__ __forceinline__ float bi_exp_tab(float x, const float *) { return expf(x); }
// fills tab[0..32) with 2^(j/32); call with at least 32 threads, then synchronise them
__device__ __forceinline__ void bi_exp_tab_init(double *tab, int lane) {
  if (lane < 32) tab[lane] = exp2((double)lane / 32.0);
}
__device__ __forceinline__ void bi_exp_tab_init(float *, int) {}

// The argument reduction and the minimax coefficients Lg1..Lg7 (and the two-part ln 2 shared with the
// exponentials above) are those of FreeBSD's msun / fdlibm e_log.c:
//   Copyright (C) 1993 by Sun Microsystems, Inc. All rights reserved.
//   Developed at SunSoft, a Sun Microsystems, Inc. business.
//   Permission to use, copy, modify, and distribute this software is freely granted,
//   provided that this notice is preserved.
// ---- table-driven exp and log in float64, for kernels whose pace is set by FP64 instructions ----
// Tables in shared memory, filled by the block (bi_fast_tabs_init, then a block-wide barrier).
//   exp: x = k ln2/512 + r with k = round(x 512/ln 2), |r| <= ln2/1024; exp(x) = 2^(k >> 9) *
//        2^((k & 511)/512) * (1 + r + r^2/2 + r^3/6): 7 operations, within 1e-14 relative.  k ln2/512 is
//        exact inside the fused multiply-add, so one constant serves the reduction (error |x| 1.1e-16).
//   log: x = 2^k m, m in [1, 2); c_j = 1 + (j + 1/2)/128 for the j-th of 128 mantissa intervals;
//        ln x = k ln 2 + ln c_j + log1p(r), r = m / c_j - 1, |r| <= 1/256, log1p to the fifth power:
//        9 operations (25 for the table-free form below), absolute error below 1e-15 for the
//        probabilities and normalisers it is used on (|k| <= 54).
constexpr int BI_EXP_TAB = 512, BI_EXP_BITS = 9, BI_LOG_TAB = 128;
__device__ __forceinline__ void bi_fast_tabs_init(double *exp_tab, double2 *log_tab, int tid, int nthreads) {
  for (int j = tid; j < BI_EXP_TAB; j += nthreads) exp_tab[j] = exp2((double)j * (1.0 / BI_EXP_TAB));
  for (int j = tid; j < BI_LOG_TAB; j += nthreads) {
    const double c = 1.0 + ((double)j + 0.5) * (1.0 / BI_LOG_TAB);
    log_tab[j] = make_double2(1.0 / c, log(c));
  }
}
__device__ __forceinline__ void bi_fast_tabs_init(float *, float2 *, int, int) {}
// exact zero below -700 (the true value is below 1e-304)
__device__ __forceinline__ double bi_exp_fast(double x, const double *__restrict__ tab) {
  const double KL = 738.6598609351493, LK = 0.0013538030870311431, MAGIC = 6755399441055744.0;
  const double t = fma(x, KL, MAGIC);
  const int k = __double2loint(t);
  const double kd = t - MAGIC;
  const double r = fma(kd, -LK, x);
  const double T = tab[k & (BI_EXP_TAB - 1)];
  const double a = fma(r, 1.0 / 6.0, 0.5);
  const double r2 = r * r;
  const double p = fma(r2, a, r);
  const double res = fma(T, p, T);
  const double out = __hiloint2double(__double2hiint(res) + ((k >> BI_EXP_BITS) << 20), __double2loint(res));
  return x < -700.0 ? 0.0 : out;
}
__device__ __forceinline__ float bi_exp_fast(float x, const float *) { return expf(x); }
// x a positive normal double
__device__ __forceinline__ double bi_log_fast(double x, const double2 *__restrict__ tab) {
  const int hx = __double2hiint(x);
  const int k = (hx >> 20) - 1023;
  const double2 cj = tab[(hx >> 13) & (BI_LOG_TAB - 1)];
  const double m = __hiloint2double((hx & 0x000fffff) | 0x3ff00000, __double2loint(x));
  const double r = fma(m, cj.x, -1.0);
  const double r2 = r * r;
  const double a = fma(r, 1.0 / 3.0, -0.5);
  const double b = fma(r, 0.2, -0.25);
  const double c = fma(r2, b, a);
  const double p = fma(r2, c, r);
  return fma((double)k, 0.69314718055994530942, cj.y) + p;
}
__device__ __forceinline__ float bi_log_fast(float x, const float2 *) { return logf(x); }

// Branch-free natural log of a positive normal double (the messages take logs
// of probabilities clamped at 1e-16 and of sums of exponentials: never zero,
// subnormal, infinite or NaN).  Same motive as bi_exp_inline: the six logs of
// an MMP sweep are independent, and straight-line code lets them overlap
// (measured: 860 cycles for six against 1590 with log()).  Classic scheme:
// x = 2^k m with m in [sqrt(1/2), sqrt(2)), f = m - 1, s = f / (2 + f),
// log m = f - f^2/2 + s (f^2/2 + R(s^2)) with a degree-7 minimax R.  Measured
// against log() over [1e-16, 40]: within 2.3e-16 relative.
__device__ __forceinline__ double bi_log_inline(double x) {
  const double ln2_hi = 6.93147180369123816490e-01, ln2_lo = 1.90821492927058770002e-10;
  const double Lg1 = 6.666666666666735130e-01, Lg2 = 3.999999999940941908e-01, Lg3 = 2.857142874366239149e-01,
               Lg4 = 2.222219843214978396e-01, Lg5 = 1.818357216161805012e-01, Lg6 = 1.531383769920937332e-01,
               Lg7 = 1.479819860511658591e-01;
  int hx = __double2hiint(x);
  const int lx = __double2loint(x);
  int k = (hx >> 20) - 1023;
  hx &= 0x000fffff;
  const int i = (hx + 0x95f64) & 0x100000;  // mantissa above sqrt(2): halve it
  k += i >> 20;
  const double m = __hiloint2double(hx | (i ^ 0x3ff00000), lx);
  const double f = m - 1.0;
  const double d = 2.0 + f;
  double y;
  asm("rcp.approx.ftz.f64 %0, %1;" : "=d"(y) : "d"(d));
  double e = fma(-d, y, 1.0);
  y = fma(y, e, y);
  e = fma(-d, y, 1.0);
  y = fma(y, e, y);
  const double s = f * y;
  const double z = s * s, w = z * z;
  const double t1 = w * fma(w, fma(w, Lg6, Lg4), Lg2);
  const double t2 = z * fma(w, fma(w, fma(w, Lg7, Lg5), Lg3), Lg1);
  const double hfsq = 0.5 * f * f;
  const double dk = (double)k;
  return dk * ln2_hi - ((hfsq - (s * (hfsq + (t2 + t1)) + dk * ln2_lo)) - f);
}
__device__ __forceinline__ float bi_log_inline(float x) { return logf(x); }

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

// ---- bulk asynchronous copy, global -> shared, completed on an mbarrier ----
// (the copy engine's untiled form: cp.async.bulk; both addresses 16-byte
// aligned, the size a multiple of 16 bytes, no multicast)
__device__ __forceinline__ uint32_t bi_smem_addr(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void bi_mbar_init(unsigned long long *bar, int arrivals) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bi_smem_addr(bar)), "r"(arrivals) : "memory");
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}

// one thread: announce `bytes` on the barrier (its one arrival) and start the copy
__device__ __forceinline__ void bi_bulk_load(void *dst_smem, const void *src_global, uint32_t bytes,
                                             unsigned long long *bar) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bi_smem_addr(bar)), "r"(bytes)
               : "memory");
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                   bi_smem_addr(dst_smem)),
               "l"(src_global), "r"(bytes), "r"(bi_smem_addr(bar))
               : "memory");
}

// the announcement alone: `bytes` expected on the barrier, and this thread's arrival (a testing aid uses
// it without the copy, to make the bounded wait below run out)
__device__ __forceinline__ void bi_mbar_expect(unsigned long long *bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bi_smem_addr(bar)), "r"(bytes)
               : "memory");
}

// Waits for the barrier's phase of the given parity with a bounded number of
// probes; false when the limit ran out (the caller raises a status flag and
// leaves: nothing here spins without an end).
__device__ __forceinline__ bool bi_mbar_wait(unsigned long long *bar, uint32_t parity, int limit = 1 << 18) {
  for (int i = 0; i < limit; ++i) {
    uint32_t done;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(done)
        : "r"(bi_smem_addr(bar)), "r"(parity)
        : "memory");
    if (done) return true;
  }
  return false;
}
