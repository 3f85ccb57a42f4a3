// Float64 register-tile filtering kernel for single-group rank-3 models whose
// first packed axis fits the lanes of a unit one to one (SB == 1) and whose
// other two axes are no longer than that lane count.
//
// Same data distribution as tile3.cuh: a unit is one agent, lane a of the unit
// holds L[a][.][.] (the step's summed slice) in registers, four units per warp.
// One Jacobi sweep (Section IV marginalisation, then the softmax of Section
// III-A) is
//   V[b] = sum_c L[b][c] e_c[c],  W[c] = sum_b e_b[b] L[b][c]        2 NB NC multiply-adds, in-lane
//   message to a: sum_b V[b] e_b[b]                                  in-lane
//   messages to b and c: sum_a e_a V_a[b], sum_a e_a W_a[c]          across the unit's lanes
//   three exponentials per lane, new e's to every lane, their sums, one reciprocal.
// Measured on B200 with single-purpose programs, the costs that shape the
// kernel: an FP64 instruction occupies its pipe 2.2 cycles per warp; a warp's
// shuffles or shared-memory instructions issue at most one per 4-5 cycles
// (3 with two warps on the scheduler) whatever their width, and a warp issues
// in order, so the count of such instructions matters as much as the FP64
// count, not the bytes they move.  Hence:
//  * the cross-lane sums go through one shared-memory transpose of (V[j], W[j])
//    pairs: 8 16-byte stores and 8 16-byte loads per lane, no selects, against
//    28 shuffles and 52 selects for a butterfly;
//  * the new e's are exchanged through shared memory (3 stores, 11 16-byte
//    broadcast loads; a broadcast load costs one wavefront) and their sums are
//    taken in-lane from the loaded copies;
//  * exp through a 512-entry table of 2^(j/512) and a cubic: 7 FP64
//    operations.  The softmax shift is the largest binary exponent among the
//    logits, found with one integer warp reduction on the rounded arguments and
//    applied by integer arithmetic on the exponent field, so it costs no FP64
//    operation and is never stale: every e lies in [0, 2);
//  * per step, the slice comes from a table pre-summed over every outcome
//    combination when the model has one (one gather, no additions), and the
//    transition rows are read as 16-byte vectors.  (Staging the next step's
//    slice in shared memory with a bulk asynchronous copy issued a step ahead,
//    and a copy of the transition matrices in shared memory, were measured and
//    changed nothing: with two warps per scheduler a step's head already runs
//    under the other warp's sweeps.)
#pragma once
#include "bi_internal.h"
#include "tile3.cuh"
#include "tile3_common.cuh"

namespace tile3_f64 {


constexpr int EXP_TAB = 512;   // entries of the 2^(j/512) table
constexpr int EXP_BITS = 9;

// exp(x) = 2^(k >> 9) * m with k = round(x * 512 / ln 2) and the mantissa part
// m = 2^((k & 511)/512) * exp(r) in [1, 2], r = x - k ln2/512, |r| <= ln2/1024:
// the cubic 1 + r + r^2/2 + r^3/6 is then within 9e-15 relative.  The product
// k * (ln2/512) is exact inside the fused multiply-add, so one constant suffices
// for the reduction (error |x| * 1.1e-16 from the constant's own rounding).
__device__ __forceinline__ double exp_mant(double x, const double *__restrict__ tab, int &k) {
  const double KL = 738.6598609351493,        // 512 / ln 2
               LK = 0.0013538030870311431,    // ln 2 / 512
               MAGIC = 6755399441055744.0;     // 1.5 * 2^52: adding it rounds to the nearest integer
  const double t = fma(x, KL, MAGIC);
  k = __double2loint(t);
  const double kd = t - MAGIC;
  const double r = fma(kd, -LK, x);
  const double T = tab[k & (EXP_TAB - 1)];
  const double a = fma(r, 1.0 / 6.0, 0.5);
  const double r2 = r * r;
  const double p = fma(r2, a, r);
  return fma(T, p, T);
}
// m * 2^d for d <= 0 (0 below 2^-1000: the true value is then far below any belief that matters)
__device__ __forceinline__ double exp_scale(double m, int d) {
  const double v = __hiloint2double(__double2hiint(m) + (d << 20), __double2loint(m));
  return d < -1000 ? 0.0 : v;
}

// Largest k over the warp (one instruction, warp-uniform result) or over the lanes of a unit (shuffle
// steps; with one lane mask per unit the reduction intrinsic compiles to a loop over the units).  The
// warp-wide form shifts every unit by the same exponent: safe while three factors' sums cannot
// underflow together, which the caller checks from the number of modalities.
template <int NL, bool UNITMAX>
__device__ __forceinline__ int max_k(int k) {
  if constexpr (!UNITMAX || NL == 32) return __reduce_max_sync(0xffffffffu, k);
  else {
#pragma unroll
    for (int d = NL / 2; d >= 1; d >>= 1) k = max(k, __shfl_xor_sync(0xffffffffu, k, d));
    return k;
  }
}

// reciprocal of a normal double to about 1e-13 relative: hardware seed and one Newton step with a
// correction term (the scale of a likelihood message: an error of that size moves a logit by 1e-11)
__device__ __forceinline__ double rcp_fast(double x) {
  double y;
  asm("rcp.approx.ftz.f64 %0, %1;" : "=d"(y) : "d"(x));
  const double e = fma(-x, y, 1.0);
  const double e2 = fma(e, e, e);
  return fma(y, e2, y);
}

__device__ __forceinline__ void lds2(const double *p, double &x, double &y) {
  const double2 v = *reinterpret_cast<const double2 *>(p);
  x = v.x;
  y = v.y;
}
__device__ __forceinline__ void sts2(double *p, double x, double y) { *reinterpret_cast<double2 *>(p) = make_double2(x, y); }

// sum_r row[r] q[r]: row in global memory (16-byte aligned) and q in shared memory (offset q_off
// elements into a 16-byte aligned array), read as 16-byte vectors where alignment allows
template <int N>
__device__ __forceinline__ double row_dot(const double *row, const double *qbase, int q_off) {
  double s0 = 0.0, s1 = 0.0;
  const double *q = qbase + q_off;
#pragma unroll
  for (int r = 0; r + 1 < N; r += 2) {
    const double2 m = __ldg(reinterpret_cast<const double2 *>(row + r));
    double q0, q1;
    if ((q_off & 1) == 0) lds2(q + r, q0, q1);
    else { q0 = q[r]; q1 = q[r + 1]; }
    s0 = fma(m.x, q0, s0);
    s1 = fma(m.y, q1, s1);
  }
  if (N & 1) s0 = fma(__ldg(row + N - 1), q[N - 1], s0);
  return s0 + s1;
}

template <int NA_, int NB_, int NC_>
struct Geo {
  static constexpr int NA = NA_, NB = NB_, NC = NC_;
  static constexpr int LPU = Pow2Ceil<NA>::v;       // lanes per unit
  static constexpr int UPW = 32 / LPU;
  static constexpr int NBP = (NB + 1) & ~1;         // e_b padded to whole 16-byte vectors
  static constexpr int NCP = (NC + 3) & ~3;         // the slice's padded last axis
  static constexpr int NP = NBP > NCP ? NBP : NCP;  // (V, W) pairs per transpose row
  static constexpr int TPR = 2 * NP + 2;            // row stride: 16 bytes more than a multiple of 128
  static constexpr int SE_A = 0, SE_B = LPU, SE_C = LPU + NBP, SE = LPU + NBP + NCP;   // exchange area layout
  static constexpr int P_TILE = LPU * NB * NCP;
  static constexpr int NV = NB * NCP / 2;           // 16-byte vectors of a lane's part of the slice
  static_assert(NB <= LPU && NC <= LPU, "b and c must fit the unit's lanes");
};

// Per-step state of one lane and the sweep.  Everything is indexed with compile-time constants once
// inlined, so the members live in registers.
template <class G>
struct Sweep {
  using R = double;
  static constexpr int NA = G::NA, NB = G::NB, NC = G::NC, LPU = G::LPU, NBP = G::NBP, NCP = G::NCP;

  R L[NB][NCP];              // this lane's part of the step's summed slice
  R eav[LPU], eb[NBP], ec[NCP];   // current iterate, unnormalised, every lane's copy
  R ea;                      // this lane's own e_a
  R sa, sb, sc;              // 1 / (z z) of the other two factors
  R za, zb, zc;              // sums of the e's
  R lpa, lpb, lpc;           // ln prior of the owned logits
  R xa, xb, xc;              // latest logits of the owned states
  R o_eb, o_ec;              // this lane's own e_b, e_c
  int Ma, Mb, Mc;            // binary exponents the e's are relative to
  int u;
  bool a_ok, b_ok, c_ok;
  const R *tab;
  R *tp, *se;                // this unit's transpose and exchange areas

  __device__ __forceinline__ void start() {   // uniform beliefs: every e = 1
    ea = a_ok ? 1.0 : 0.0;
#pragma unroll
    for (int r = 0; r < LPU; ++r) eav[r] = r < NA ? 1.0 : 0.0;
#pragma unroll
    for (int b = 0; b < NBP; ++b) eb[b] = b < NB ? 1.0 : 0.0;
#pragma unroll
    for (int c = 0; c < NCP; ++c) ec[c] = c < NC ? 1.0 : 0.0;
    sa = 1.0 / (NB * NC); sb = 1.0 / (NA * NC); sc = 1.0 / (NA * NB);
    za = NA; zb = NB; zc = NC;
    xa = xb = xc = 0.0;
    o_eb = b_ok ? 1.0 : 0.0;
    o_ec = c_ok ? 1.0 : 0.0;
    Ma = Mb = Mc = 0;
  }

  // DAMPED: the logits take a step of size lam from the previous iterate's (oml = 1 - lam; the
  // uniform start's logits are a constant, taken as 0); a separate instantiation, so that the plain
  // sweep carries none of it.
  template <bool UNITMAX, bool DAMPED>
  __device__ __forceinline__ void sweep(R lam, R oml) {
    const R pxa = xa, pxb = xb, pxc = xc;
    R V[G::NP], W[G::NP];
#pragma unroll
    for (int j = 0; j < G::NP; ++j) V[j] = W[j] = 0.0;
#pragma unroll
    for (int c = 0; c < NCP; ++c)
#pragma unroll
      for (int b = 0; b < NB; ++b) V[b] = fma(L[b][c], ec[c], V[b]);
#pragma unroll
    for (int b = 0; b < NB; ++b)
#pragma unroll
      for (int c = 0; c < NCP; ++c) W[c] = fma(eb[b], L[b][c], W[c]);
    // ---- transpose: lane r writes row r of (V[j], W[j]) pairs, lane u reads pair u of every row
    R *row = tp + u * G::TPR;
#pragma unroll
    for (int j = 0; j < G::NP; ++j) sts2(row + 2 * j, V[j], W[j]);
    R la0 = 0.0, la1 = 0.0;
#pragma unroll
    for (int b = 0; b < NB; ++b) {
      if (b & 1) la1 = fma(V[b], eb[b], la1);
      else la0 = fma(V[b], eb[b], la0);
    }
    xa = fma(la0 + la1, sa, lpa);
    if (DAMPED) xa = fma(lam, xa, oml * pxa);
    __syncwarp();
    R b0 = 0.0, b1 = 0.0, c0 = 0.0, c1 = 0.0;
#pragma unroll
    for (int r = 0; r < LPU; ++r) {
      R vb, vc;
      lds2(tp + r * G::TPR + 2 * u, vb, vc);
      if (r & 1) { b1 = fma(eav[r], vb, b1); c1 = fma(eav[r], vc, c1); }
      else { b0 = fma(eav[r], vb, b0); c0 = fma(eav[r], vc, c0); }
    }
    xb = fma(b0 + b1, sb, lpb);
    xc = fma(c0 + c1, sc, lpc);
    if (DAMPED) {
      xb = fma(lam, xb, oml * pxb);
      xc = fma(lam, xc, oml * pxc);
    }
    // ---- softmax numerators relative to the largest binary exponent
    int ka, kb, kc;
    const R ma = exp_mant(xa, tab, ka);
    const R mb = exp_mant(xb, tab, kb);
    const R mc = exp_mant(xc, tab, kc);
    Ma = max_k<LPU, UNITMAX>(a_ok ? ka : INT_MIN) >> EXP_BITS;
    Mb = max_k<LPU, UNITMAX>(b_ok ? kb : INT_MIN) >> EXP_BITS;
    Mc = max_k<LPU, UNITMAX>(c_ok ? kc : INT_MIN) >> EXP_BITS;
    ea = a_ok ? exp_scale(ma, (ka >> EXP_BITS) - Ma) : 0.0;
    o_eb = b_ok ? exp_scale(mb, (kb >> EXP_BITS) - Mb) : 0.0;
    o_ec = c_ok ? exp_scale(mc, (kc >> EXP_BITS) - Mc) : 0.0;
    // ---- exchange: every lane gets every e
    se[G::SE_A + u] = ea;
    if (u < NBP) se[G::SE_B + u] = o_eb;
    if (u < NCP) se[G::SE_C + u] = o_ec;
    __syncwarp();
#pragma unroll
    for (int r = 0; r < LPU; r += 2) lds2(se + G::SE_A + r, eav[r], eav[r + 1]);
#pragma unroll
    for (int b = 0; b < NBP; b += 2) lds2(se + G::SE_B + b, eb[b], eb[b + 1]);
#pragma unroll
    for (int c = 0; c < NCP; c += 2) lds2(se + G::SE_C + c, ec[c], ec[c + 1]);
    za = tree_sum<R, LPU>(eav);
    zb = tree_sum<R, NBP>(eb);
    zc = tree_sum<R, NCP>(ec);
    const R rinv = rcp_fast(za * zb * zc);
    sa = rinv * za;
    sb = rinv * zb;
    sc = rinv * zc;
  }
};

template <int NA, int NB, int NC, bool DAMPED>
__global__ void __launch_bounds__(32) bi_tile3_filter_f64_kernel(const Tile3Params p) {
  using R = double;
  using G = Geo<NA, NB, NC>;
  using SW = Sweep<G>;
  constexpr int LPU = G::LPU, UPW = G::UPW, NCP = G::NCP, NV = G::NV;
  __shared__ __align__(16) R exp_tab[EXP_TAB];
  __shared__ __align__(16) R sm_q[UPW][(NA + NB + NC + 1) & ~1];   // final beliefs of the previous step
  __shared__ __align__(16) R sm_tp[UPW][LPU * G::TPR + 2];
  __shared__ __align__(16) R sm_se[UPW][G::SE];
  const int lane = threadIdx.x;
  for (int j = lane; j < EXP_TAB; j += 32) exp_tab[j] = exp2((double)j * (1.0 / EXP_TAB));
  // One warp-wide reduction finds the softmax shift of all the warp's agents at once, unless the model's
  // logits can lie too far apart for a common shift (many modalities, entries of A above 1, observation
  // vectors with the caller's weights): then every agent takes its own.
  const bool unit_shift = p.unit_shift != 0 || p.nmem > 5 || __ldg(p.status + 1) != 0;
  const int unit = lane / LPU, u = lane % LPU;
  int agent = blockIdx.x * UPW + unit;
  const bool live = agent < p.N;
  if (!live) agent = p.N - 1;   // keeps every warp-wide operation uniform; its stores are suppressed
  const int g = p.G == 1 ? 0 : agent;

  SW sw;
  sw.u = u;
  sw.tab = exp_tab;
  sw.tp = sm_tp[unit];
  sw.se = sm_se[unit];
  const int a = u, bi = u, ci = u;
  const bool a_ok = u < NA, b_ok = u < NB, c_ok = u < NC;
  sw.a_ok = a_ok; sw.b_ok = b_ok; sw.c_ok = c_ok;
  const int asafe = a_ok ? a : 0, bsafe = b_ok ? bi : 0, csafe = c_ok ? ci : 0;
  R *sq = sm_q[unit];
  for (int i = u; i < G::SE; i += LPU) sm_se[unit][i] = 0.0;
  __syncwarp();

  const size_t out_base = (size_t)agent * p.T;
  const bool from_prev = p.q_prev != nullptr || p.carry_in != nullptr;
  int u_next[3] = {0, 0, 0};
  if (from_prev) {
    if (p.carry_in) {   // the previous call's last belief at full precision
      const R *qp = (const R *)p.carry_in + (size_t)agent * p.S;
      if (a_ok) sq[a] = qp[p.off[0] + a];
      if (b_ok) sq[NA + bi] = qp[p.off[1] + bi];
      if (c_ok) sq[NA + NB + ci] = qp[p.off[2] + ci];
    } else {
      const float *qp = p.q_prev + (size_t)agent * p.S;
      if (a_ok) sq[a] = (R)__ldg(qp + p.off[0] + a);
      if (b_ok) sq[NA + bi] = (R)__ldg(qp + p.off[1] + bi);
      if (c_ok) sq[NA + NB + ci] = (R)__ldg(qp + p.off[2] + ci);
    }
    const int32_t *ap = p.act_prev + (size_t)agent * p.F;
    u_next[0] = __ldg(ap + p.fac[0]);
    u_next[1] = __ldg(ap + p.fac[1]);
    u_next[2] = __ldg(ap + p.fac[2]);
    __syncwarp();
  }
  // The outcome stream is read one step ahead (models with up to MAXC modalities, which covers every
  // model with a pre-summed table), so that its latency is hidden by the previous step's sweeps.
  constexpr int MAXC = 4;
  const bool ahead = p.nmem <= MAXC;
  int o_nx[MAXC] = {0, 0, 0, 0};
  auto load_outcomes = [&](int t) {
#pragma unroll
    for (int mi = 0; mi < MAXC; ++mi)
      if (mi < p.nmem) o_nx[mi] = __ldg(p.obs + (out_base + t) * p.M + p.modality[mi]);
  };
  if (ahead) load_outcomes(0);

  for (int t = 0; t < p.T; ++t) {
    // ---- the step's summed slice into registers: from the table pre-summed over every outcome
    // combination when the model has one, else the modalities' slices added here.  Out-of-range
    // outcomes are clamped and flagged.  (Lane-interleaved layout: 16-byte vector v of lane u at
    // (v * LPU + u) * 2.)
    int o_cur[MAXC];
#pragma unroll
    for (int mi = 0; mi < MAXC; ++mi)
      o_cur[mi] = mi < p.nmem ? clamp_flag(o_nx[mi], p.mcount[mi], p.status, BI_FLAG_OBS_RANGE) : 0;
    if (p.Lcomb) {
      int64_t idx = 0;
#pragma unroll
      for (int mi = 0; mi < MAXC; ++mi)
        if (mi < p.nmem) idx += (int64_t)o_cur[mi] * p.comb_mul[mi];
      const R *s0 = (const R *)p.Lcomb + ((size_t)g * p.ncomb + (size_t)idx) * p.P_tile + u * 2;
#pragma unroll
      for (int v = 0; v < NV; ++v) {
        R x[2];
        ldg_vec(s0 + v * LPU * 2, x);
        sw.L[(v * 2) / NCP][(v * 2) % NCP] = x[0];
        sw.L[(v * 2 + 1) / NCP][(v * 2 + 1) % NCP] = x[1];
      }
    } else {
#pragma unroll
      for (int b = 0; b < NB; ++b)
#pragma unroll
        for (int c = 0; c < NCP; ++c) sw.L[b][c] = 0.0;
      for (int mi = 0; mi < p.nmem; ++mi) {
        int o;
        if (ahead) {
          o = o_cur[0];
#pragma unroll
          for (int j = 1; j < MAXC; ++j) o = mi == j ? o_cur[j] : o;
        } else {
          o = clamp_flag(__ldg(p.obs + (out_base + t) * p.M + p.modality[mi]), p.mcount[mi], p.status,
                         BI_FLAG_OBS_RANGE);
        }
        const R *sp = (const R *)p.logA[mi] + ((size_t)g * p.mcount[mi] + (size_t)o) * p.P_tile + u * 2;
#pragma unroll
        for (int v = 0; v < NV; ++v) {
          R x[2];
          ldg_vec(sp + v * LPU * 2, x);
          sw.L[(v * 2) / NCP][(v * 2) % NCP] += x[0];
          sw.L[(v * 2 + 1) / NCP][(v * 2 + 1) % NCP] += x[1];
        }
      }
    }
    if (ahead && t + 1 < p.T) load_outcomes(t + 1);
    const int u_cur[3] = {u_next[0], u_next[1], u_next[2]};
    if (t + 1 < p.T) {
      const int32_t *an = p.act + ((size_t)agent * (p.T - 1) + t) * 3;
      u_next[0] = __ldg(an + p.fac[0]);
      u_next[1] = __ldg(an + p.fac[1]);
      u_next[2] = __ldg(an + p.fac[2]);
    }

    // ---- ln prior of the logits this lane owns: D, or B_u times the previous step's belief
    R lpa, lpb, lpc;
    if (t == 0 && !from_prev) {
      lpa = __ldg((const R *)p.logD[0] + (size_t)g * p.Dstride[0] + asafe);
      lpb = __ldg((const R *)p.logD[1] + (size_t)g * p.Dstride[1] + bsafe);
      lpc = __ldg((const R *)p.logD[2] + (size_t)g * p.Dstride[2] + csafe);
    } else {
      const int ua = clamp_flag(u_cur[0], p.U[0], p.status, BI_FLAG_ACT_RANGE);
      const int ub = clamp_flag(u_cur[1], p.U[1], p.status, BI_FLAG_ACT_RANGE);
      const int uc = clamp_flag(u_cur[2], p.U[2], p.status, BI_FLAG_ACT_RANGE);
      // forward matrices [next][previous], rows padded to a multiple of four: this lane's next state
      // is one row, read as 16-byte vectors
      const R *ra = (const R *)p.Bf[0] + (size_t)g * p.Bstride[0] + ((size_t)ua * NA + asafe) * p.np[0];
      const R *rb = (const R *)p.Bf[1] + (size_t)g * p.Bstride[1] + ((size_t)ub * NB + bsafe) * p.np[1];
      const R *rc = (const R *)p.Bf[2] + (size_t)g * p.Bstride[2] + ((size_t)uc * NC + csafe) * p.np[2];
      lpa = bi_log_inline(bi_max(row_dot<NA>(ra, sq, 0), (R)BI_EPS));
      lpb = bi_log_inline(bi_max(row_dot<NB>(rb, sq, NA), (R)BI_EPS));
      lpc = bi_log_inline(bi_max(row_dot<NC>(rc, sq, NA + NB), (R)BI_EPS));
    }
    sw.lpa = a_ok ? lpa : 0.0;
    sw.lpb = b_ok ? lpb : 0.0;
    sw.lpc = c_ok ? lpc : 0.0;

    sw.start();
    const R lam = (R)p.lambda, oml = 1.0 - lam;
    if (unit_shift) for (int k = 0; k < p.K; ++k) sw.template sweep<true, DAMPED>(lam, oml);
    else for (int k = 0; k < p.K; ++k) sw.template sweep<false, DAMPED>(lam, oml);

    // ---- final beliefs of the step: outputs, and the next step's prior input
    // (1/za = sc zb, 1/zb = sc za, 1/zc = sa zb)
    const R qa = sw.ea * (sw.sc * sw.zb);
    const R qb = sw.o_eb * (sw.sc * sw.za);
    const R qc = sw.o_ec * (sw.sa * sw.zb);
    if (a_ok) sq[a] = qa;
    if (b_ok) sq[NA + bi] = qb;
    if (c_ok) sq[NA + NB + ci] = qc;
    if (live) {
      float *qo = p.q_out + (out_base + t) * p.S;
      if (a_ok) qo[p.off[0] + a] = (float)qa;
      if (b_ok) qo[p.off[1] + bi] = (float)qb;
      if (c_ok) qo[p.off[2] + ci] = (float)qc;
      if (p.carry_out && t == p.T - 1) {
        R *co = (R *)p.carry_out + (size_t)agent * p.S;
        if (a_ok) co[p.off[0] + a] = qa;
        if (b_ok) co[p.off[1] + bi] = qb;
        if (c_ok) co[p.off[2] + ci] = qc;
      }
      if (p.logq_out) {
        const R LN2 = 0.69314718055994530942;
        float *lo = p.logq_out + (out_base + t) * p.S;
        if (a_ok) lo[p.off[0] + a] = (float)(sw.xa - ((R)sw.Ma * LN2 + bi_log(sw.za)));
        if (b_ok) lo[p.off[1] + bi] = (float)(sw.xb - ((R)sw.Mb * LN2 + bi_log(sw.zb)));
        if (c_ok) lo[p.off[2] + ci] = (float)(sw.xc - ((R)sw.Mc * LN2 + bi_log(sw.zc)));
      }
    }
    if (p.argmax_out) {
      const int ia = group_argmax<R, LPU, 1>(a_ok ? sw.xa : -bi_inf<R>(), a_ok ? a : 1 << 20);
      const int ib = group_argmax<R, LPU, 1>(b_ok ? sw.xb : -bi_inf<R>(), b_ok ? bi : 1 << 20);
      const int ic = group_argmax<R, LPU, 1>(c_ok ? sw.xc : -bi_inf<R>(), c_ok ? ci : 1 << 20);
      if (live && u == 0) {
        int32_t *ao = p.argmax_out + (out_base + t) * 3;
        ao[p.fac[0]] = ia;
        ao[p.fac[1]] = ib;
        ao[p.fac[2]] = ic;
      }
    }
    __syncwarp();
  }
}

}  // namespace tile3_f64
