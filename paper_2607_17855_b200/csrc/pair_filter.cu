// Filtering kernel for models whose factors are coupled at most in one pair: every modality depends
// on a single factor, except for the modalities of at most one dependency group over two factors
// (a, b).  (Of the 128 random structures of the randomised benchmark sweep, 77 are of this kind, and
// so is the smallest benchmark configuration.)  For such a model
//   * a factor outside the pair receives no message that depends on another factor's belief: its
//     logits are prior + its modalities' slices, the same in every iteration, so its belief is one
//     softmax per step (Section III-A's update reaches its fixed point at once);
//   * the pair's Jacobi sweep (Section IV marginalisation) is two matrix-vector products,
//     ell_a = L e_b / z_b and ell_b = L^T e_a / z_a with L the summed slice [n_a][n_b].
// One unit of LPU lanes serves an agent (LPU = the largest state count rounded up to a power of two),
// lane u owning state u of every factor; a warp holds 32 / LPU agents and nothing ever crosses a warp,
// so an iteration costs no block barrier: the CTA-per-agent kernel that served these models spends
// more than a microsecond per sweep on its three barriers, this one a few hundred cycles.  The summed
// slice lives in registers twice, as rows (lane a holds L[a][.]) and, from a transposed copy made at
// packing time, as columns (lane b holds L[.][b]), so both products are in-lane; the unnormalised
// beliefs are exchanged through shared memory and read as broadcast 16-byte pairs inside the product
// loops.  Float64 handles, plain (undamped) update.
#include "bi_internal.h"
#include "tile3_filter_f64.cuh"   // the table-driven exponential, the integer softmax shift, rcp_fast

namespace {

using tile3_f64::EXP_BITS;
using tile3_f64::EXP_TAB;
using tile3_f64::exp_mant;
using tile3_f64::exp_scale;
using tile3_f64::lds2;
using tile3_f64::max_k;
using tile3_f64::rcp_fast;
typedef double R;

struct PairParams {
  int32_t N, T, K, F, M, S, G;
  double lambda;   // damping step on the logits; 1 = the plain update
  int32_t n[BI_MAX_F], off[BI_MAX_F], npad[BI_MAX_F], U[BI_MAX_F];
  const R *Bf[BI_MAX_F], *logD[BI_MAX_F];   // forward matrices [u][next][previous (padded)], ln D
  int64_t Bstride[BI_MAX_F], Dstride[BI_MAX_F];
  // modalities that depend on one factor, ordered by factor: those of factor f are [r1_begin[f], r1_begin[f + 1])
  int32_t r1_begin[BI_MAX_F + 1];
  int32_t r1_mod[BI_MAX_M], r1_m[BI_MAX_M], r1_P[BI_MAX_M];
  const R *r1_logA[BI_MAX_M];
  int64_t r1_gstride[BI_MAX_M];
  // the pair (fa < 0: none): slices [m][na][npb] and their transposes [m][nb][npa]
  int32_t fa, fb, na, nb, npa, npb, n2;
  int32_t r2_mod[BI_MAX_M], r2_m[BI_MAX_M];
  const R *r2_logA[BI_MAX_M], *r2_logAT[BI_MAX_M];
  int64_t r2_gstride[BI_MAX_M], r2_gstrideT[BI_MAX_M];
  const int32_t *obs, *act, *act_prev;
  const float *q_prev;
  const R *carry_in;
  R *carry_out;
  float *q_out, *logq_out;
  int32_t *argmax_out;
  uint32_t *status;
};

template <int LPU>
__device__ __forceinline__ R unit_sum(R v) {
#pragma unroll
  for (int d = LPU / 2; d >= 1; d >>= 1) v += __shfl_xor_sync(0xffffffffu, v, d);
  return v;
}
// exact argmax over the unit: largest x, lowest index among equals
template <int LPU>
__device__ __forceinline__ int unit_argmax(R x, int idx) {
#pragma unroll
  for (int d = LPU / 2; d >= 1; d >>= 1) {
    const R xo = __shfl_xor_sync(0xffffffffu, x, d);
    const int io = __shfl_xor_sync(0xffffffffu, idx, d);
    if (xo > x || (xo == x && io < idx)) { x = xo; idx = io; }
  }
  return idx;
}

constexpr int WARPS = 4;

// WARPMAX: the pair's softmax shifts by the largest binary exponent of the whole warp (one reduction
// instruction) instead of the unit's (a shuffle per halving of the unit): every unit of the warp is then
// scaled by the same power of two, which is exact, and safe while a logit cannot differ from another
// agent's by more than the exponent range, which the caller checks from the number of modalities.
// DAMPED: every iteration takes a step of size lambda on the logits from the previous iterate's (the
// uniform start's logits are a constant, taken as 0); an instantiation of its own.
template <int LPU, bool WARPMAX, bool DAMPED>
__global__ void __launch_bounds__(WARPS * 32) bi_pair_filter_kernel(const PairParams p) {
  const R lam = p.lambda, oml = 1.0 - lam;
  // the normalisers come from the exchanged copies every lane reads anyway (additions in the shadow of the
  // products) instead of a shuffle sum at the end of the sweep's dependency chain (measured on the sweep's
  // 77 structures of this kind: 7.4 -> 7.0 ms with it for every unit size; config 1's call 65 -> 54 us)
  constexpr bool ZLOCAL = true;
  const bool unit_shift = __ldg(p.status + 1) != 0;   // entries of A above 1: no common shift (BiDev::status)
  constexpr int UPW = 32 / LPU;
  constexpr int QS = BI_MAX_F * LPU;                  // previous beliefs of one unit: [factor][state]
  __shared__ __align__(16) R exp_tab[EXP_TAB];
  __shared__ __align__(16) R sm_q[WARPS * UPW][QS];
  __shared__ __align__(16) R sm_e[WARPS * UPW][2 * LPU];   // e_a, e_b of the pair
  for (int j = threadIdx.x; j < EXP_TAB; j += blockDim.x) exp_tab[j] = exp2((double)j * (1.0 / EXP_TAB));
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int unit = lane / LPU, u = lane % LPU;
  int agent = (blockIdx.x * WARPS + warp) * UPW + unit;
  const bool live = agent < p.N;
  if (!live) agent = p.N - 1;   // keeps the warp's shuffles uniform; its stores are suppressed
  const int g = p.G == 1 ? 0 : agent;
  R *sq = sm_q[warp * UPW + unit], *se = sm_e[warp * UPW + unit];
  const bool from_prev = p.q_prev != nullptr || p.carry_in != nullptr;
  for (int f = 0; f < p.F; ++f) {
    R v = 0.0;
    if (from_prev && u < p.n[f])
      v = p.carry_in ? p.carry_in[(size_t)agent * p.S + p.off[f] + u] : (R)p.q_prev[(size_t)agent * p.S + p.off[f] + u];
    sq[f * LPU + u] = v;
  }
  __syncthreads();   // the table; every later exchange stays inside a warp

  const bool pair = p.fa >= 0;
  const bool a_ok = pair && u < p.na, b_ok = pair && u < p.nb;
  const size_t ob0 = (size_t)agent * p.T;
  for (int t = 0; t < p.T; ++t) {
    const int32_t *obs_t = p.obs + (ob0 + t) * p.M;
    R ca = 0.0, cb = 0.0;
    // ---- every factor: ln prior + the slices of its own modalities; outside the pair that is the
    // whole update, and the belief is final after one softmax
    for (int f = 0; f < p.F; ++f) {
      const int nf = p.n[f];
      const bool ok = u < nf;
      R c = 0.0;
      if (t == 0 && !from_prev) {
        if (ok) c = __ldg(p.logD[f] + (size_t)g * p.Dstride[f] + u);
      } else {
        const int ur = t == 0 ? __ldg(p.act_prev + (size_t)agent * p.F + f)
                              : __ldg(p.act + ((size_t)agent * (p.T - 1) + (t - 1)) * p.F + f);
        const int ua = clamp_flag(ur, p.U[f], p.status, BI_FLAG_ACT_RANGE);
        // forward matrix row of this lane's next state, [previous] padded to a multiple of four
        const R *row = p.Bf[f] + (size_t)g * p.Bstride[f] + ((size_t)ua * nf + (ok ? u : 0)) * p.npad[f];
        const R *qp = sq + f * LPU;
        R s0 = 0.0, s1 = 0.0;
        for (int r = 0; r < nf; r += 2) {   // (padding columns of the row and of the belief are zero)
          const double2 m = __ldg(reinterpret_cast<const double2 *>(row + r));
          R q0, q1;
          lds2(qp + r, q0, q1);
          s0 = fma(m.x, q0, s0);
          s1 = fma(m.y, q1, s1);
        }
        c = ok ? bi_log_inline(bi_max(s0 + s1, (R)BI_EPS)) : 0.0;
      }
      for (int j = p.r1_begin[f]; j < p.r1_begin[f + 1]; ++j) {
        const int o = clamp_flag(__ldg(obs_t + p.r1_mod[j]), p.r1_m[j], p.status, BI_FLAG_OBS_RANGE);
        if (ok) c += __ldg(p.r1_logA[j] + (size_t)g * p.r1_gstride[j] + (size_t)o * p.r1_P[j] + u);
      }
      if (pair && f == p.fa) { ca = c; continue; }
      if (pair && f == p.fb) { cb = c; continue; }
      if (DAMPED) {   // a factor outside the pair: its message does not change, its logits approach it
        R x = 0.0;
        for (int k = 0; k < p.K; ++k) x = fma(lam, c, oml * x);
        c = x;
      }
      int k;
      const R mant = exp_mant(c, exp_tab, k);
      const int M = max_k<LPU, true>(ok ? k : INT_MIN) >> EXP_BITS;
      const R e = ok ? exp_scale(mant, (k >> EXP_BITS) - M) : 0.0;
      const R z = unit_sum<LPU>(e);
      const R q = e * rcp_fast(z) * (2.0 - z * rcp_fast(z));   // one more Newton step: a belief to full precision
      __syncwarp();
      sq[f * LPU + u] = q;
      if (live && ok) {
        const size_t o = (ob0 + t) * p.S + p.off[f] + u;
        p.q_out[o] = (float)q;
        if (p.logq_out) p.logq_out[o] = (float)(c - ((R)M * 0.69314718055994530942 + bi_log(z)));
        if (p.carry_out && t == p.T - 1) p.carry_out[(size_t)agent * p.S + p.off[f] + u] = q;
      }
      if (p.argmax_out) {
        const int am = unit_argmax<LPU>(ok ? c : -bi_inf<R>(), ok ? u : 1 << 20);
        if (live && u == 0) p.argmax_out[(ob0 + t) * p.F + f] = am;
      }
      __syncwarp();
    }
    if (!pair) continue;

    // ---- the pair: the step's summed slice as rows (lane a) and as columns (lane b)
    R L[LPU], LT[LPU];
#pragma unroll
    for (int i = 0; i < LPU; ++i) L[i] = LT[i] = 0.0;
    for (int j = 0; j < p.n2; ++j) {
      const int o = clamp_flag(__ldg(obs_t + p.r2_mod[j]), p.r2_m[j], p.status, BI_FLAG_OBS_RANGE);
      const R *row = p.r2_logA[j] + (size_t)g * p.r2_gstride[j] + ((size_t)o * p.na + (a_ok ? u : 0)) * p.npb;
      const R *col = p.r2_logAT[j] + (size_t)g * p.r2_gstrideT[j] + ((size_t)o * p.nb + (b_ok ? u : 0)) * p.npa;
#pragma unroll
      for (int i = 0; i < LPU; i += 2) {
        if (i < p.npb) {
          const double2 x = __ldg(reinterpret_cast<const double2 *>(row + i));
          L[i] += x.x; L[i + 1] += x.y;
        }
        if (i < p.npa) {
          const double2 x = __ldg(reinterpret_cast<const double2 *>(col + i));
          LT[i] += x.x; LT[i + 1] += x.y;
        }
      }
    }
    // uniform start, unnormalised: e = 1 on the real states
    R ea = a_ok ? 1.0 : 0.0, eb = b_ok ? 1.0 : 0.0;
    R rza = 1.0 / p.na, rzb = 1.0 / p.nb, za = p.na, zb = p.nb, xa = 0.0, xb = 0.0;
    int Ma = 0, Mb = 0;
    __syncwarp();
    se[u] = ea;
    se[LPU + u] = eb;
    __syncwarp();
    for (int k = 0; k < p.K; ++k) {
      R v0 = 0.0, v1 = 0.0, w0 = 0.0, w1 = 0.0, sa0 = 0.0, sa1 = 0.0, sb0 = 0.0, sb1 = 0.0;
#pragma unroll
      for (int i = 0; i < LPU; i += 2) {
        R b0, b1, a0, a1;
        lds2(se + LPU + i, b0, b1);
        lds2(se + i, a0, a1);
        v0 = fma(L[i], b0, v0); v1 = fma(L[i + 1], b1, v1);
        w0 = fma(LT[i], a0, w0); w1 = fma(LT[i + 1], a1, w1);
        if (ZLOCAL) { sa0 += a0; sa1 += a1; sb0 += b0; sb1 += b1; }
      }
      if (ZLOCAL) {   // (one Newton step: 1e-13 relative on a message's scale; the final beliefs take two)
        za = sa0 + sa1; zb = sb0 + sb1;
        rza = rcp_fast(za); rzb = rcp_fast(zb);
      }
      if (DAMPED) {
        xa = fma(lam, fma(v0 + v1, rzb, ca), oml * xa);
        xb = fma(lam, fma(w0 + w1, rza, cb), oml * xb);
      } else {
        xa = fma(v0 + v1, rzb, ca);
        xb = fma(w0 + w1, rza, cb);
      }
      int ka, kb;
      const R ma = exp_mant(xa, exp_tab, ka);
      const R mb = exp_mant(xb, exp_tab, kb);
      if (WARPMAX && !unit_shift) {
        Ma = max_k<LPU, false>(a_ok ? ka : INT_MIN) >> EXP_BITS;
        Mb = max_k<LPU, false>(b_ok ? kb : INT_MIN) >> EXP_BITS;
      } else {
        Ma = max_k<LPU, true>(a_ok ? ka : INT_MIN) >> EXP_BITS;
        Mb = max_k<LPU, true>(b_ok ? kb : INT_MIN) >> EXP_BITS;
      }
      ea = a_ok ? exp_scale(ma, (ka >> EXP_BITS) - Ma) : 0.0;
      eb = b_ok ? exp_scale(mb, (kb >> EXP_BITS) - Mb) : 0.0;
      __syncwarp();          // every lane has read the previous iterate
      se[u] = ea;
      se[LPU + u] = eb;
      if (!ZLOCAL) {
        za = unit_sum<LPU>(ea);
        zb = unit_sum<LPU>(eb);
        rza = rcp_fast(za); rzb = rcp_fast(zb);
      }
      __syncwarp();
    }
    {   // the last iterate's normalisers, to full precision: they scale the step's beliefs
      za = unit_sum<LPU>(ea);
      zb = unit_sum<LPU>(eb);
      const R ra = rcp_fast(za), rb = rcp_fast(zb);
      rza = ra * (2.0 - za * ra);
      rzb = rb * (2.0 - zb * rb);
    }
    const R qa = ea * rza, qb = eb * rzb;
    sq[p.fa * LPU + u] = qa;
    sq[p.fb * LPU + u] = qb;
    if (live) {
      const size_t o = (ob0 + t) * p.S;
      if (a_ok) p.q_out[o + p.off[p.fa] + u] = (float)qa;
      if (b_ok) p.q_out[o + p.off[p.fb] + u] = (float)qb;
      if (p.logq_out) {
        const R LN2 = 0.69314718055994530942;
        if (a_ok) p.logq_out[o + p.off[p.fa] + u] = (float)(xa - ((R)Ma * LN2 + bi_log(za)));
        if (b_ok) p.logq_out[o + p.off[p.fb] + u] = (float)(xb - ((R)Mb * LN2 + bi_log(zb)));
      }
      if (p.carry_out && t == p.T - 1) {
        if (a_ok) p.carry_out[(size_t)agent * p.S + p.off[p.fa] + u] = qa;
        if (b_ok) p.carry_out[(size_t)agent * p.S + p.off[p.fb] + u] = qb;
      }
    }
    if (p.argmax_out) {
      const int ia = unit_argmax<LPU>(a_ok ? xa : -bi_inf<R>(), a_ok ? u : 1 << 20);
      const int ib = unit_argmax<LPU>(b_ok ? xb : -bi_inf<R>(), b_ok ? u : 1 << 20);
      if (live && u == 0) {
        p.argmax_out[(ob0 + t) * p.F + p.fa] = ia;
        p.argmax_out[(ob0 + t) * p.F + p.fb] = ib;
      }
    }
    __syncwarp();
  }
}

template <int LPU>
int launch(const PairParams &p, cudaStream_t stream) {
  constexpr int per_cta = WARPS * (32 / LPU);
  const int grid = (p.N + per_cta - 1) / per_cta;
  // (logits are sums of at most M + 1 terms of magnitude below 37: with few modalities two agents'
  // logits are within a few hundred binary exponents of each other)
  if (p.lambda != 1.0) {
    if (p.M <= 5) bi_pair_filter_kernel<LPU, true, true><<<grid, WARPS * 32, 0, stream>>>(p);
    else bi_pair_filter_kernel<LPU, false, true><<<grid, WARPS * 32, 0, stream>>>(p);
  } else if (p.M <= 5) bi_pair_filter_kernel<LPU, true, false><<<grid, WARPS * 32, 0, stream>>>(p);
  else bi_pair_filter_kernel<LPU, false, false><<<grid, WARPS * 32, 0, stream>>>(p);
  return cudaGetLastError() == cudaSuccess ? BI_OK : BI_ERR_CUDA;
}

}  // namespace

// Applicable to float64 handles, plain and damped updates, trivial B-dependencies and models whose groups
// over more than one factor number at most one, over exactly two factors; BI_ERR_UNSUPPORTED otherwise.
int bi_launch_pair_filter(const BiCall &c, bi_model *mut) {
  const bi_model *md = c.model;
  const BiDev &h = md->h;
  if (c.algo != BI_ALGO_FILTER || md->arith != BI_ARITH_F64 || h.has_bdep) return BI_ERR_UNSUPPORTED;
  if (!md->pair_ok) return BI_ERR_UNSUPPORTED;
  PairParams p;
  memset(&p, 0, sizeof(p));
  p.lambda = c.lambda;
  p.N = c.N; p.T = c.T; p.K = c.K; p.F = h.F; p.M = h.M; p.S = h.S; p.G = h.G;
  int nmax = 1;
  for (int f = 0; f < h.F; ++f) {
    p.n[f] = h.n[f]; p.off[f] = h.off[f]; p.npad[f] = h.npad[f]; p.U[f] = h.U[f];
    p.Bf[f] = (const R *)h.Bf[f]; p.logD[f] = (const R *)h.logD[f];
    p.Bstride[f] = h.Bstride[f]; p.Dstride[f] = h.Dstride[f];
    nmax = h.n[f] > nmax ? h.n[f] : nmax;
  }
  p.fa = p.fb = -1;
  // members by kind; the single-factor ones ordered by factor
  int n1 = 0;
  for (int f = 0; f < h.F; ++f) {
    p.r1_begin[f] = n1;
    for (int gi = 0; gi < h.ngroups; ++gi) {
      const BiGroup &gr = h.grp[gi];
      if (gr.rank != 1 || gr.axis[0] != f) continue;
      for (int mi = gr.mem_begin; mi < gr.mem_end; ++mi) {
        const BiMember &mm = h.mem[mi];
        p.r1_mod[n1] = mm.modality; p.r1_m[n1] = mm.m; p.r1_P[n1] = mm.P_pad;
        p.r1_logA[n1] = (const R *)mm.logA; p.r1_gstride[n1] = mm.gstride;
        ++n1;
      }
    }
  }
  p.r1_begin[h.F] = n1;
  for (int gi = 0; gi < h.ngroups; ++gi) {
    const BiGroup &gr = h.grp[gi];
    if (gr.rank != 2) continue;
    p.fa = gr.axis[0]; p.fb = gr.axis[1];
    p.na = gr.dim[0]; p.nb = gr.dim[1];
    p.npa = bi_pad4(p.na); p.npb = bi_pad4(p.nb);
    for (int mi = gr.mem_begin; mi < gr.mem_end; ++mi) {
      const BiMember &mm = h.mem[mi];
      const int j = p.n2++;
      p.r2_mod[j] = mm.modality; p.r2_m[j] = mm.m;
      p.r2_logA[j] = (const R *)mm.logA; p.r2_logAT[j] = (const R *)mm.logA_T;
      p.r2_gstride[j] = mm.gstride;
      p.r2_gstrideT[j] = mm.gstride ? (int64_t)mm.m * p.nb * p.npa : 0;
    }
  }
  p.obs = c.obs; p.act = c.act; p.act_prev = c.act_prev; p.q_prev = c.q_prev;
  p.carry_in = (const R *)c.carry_in; p.carry_out = (R *)c.carry_out;
  p.q_out = c.q_out; p.logq_out = c.logq_out; p.argmax_out = c.argmax_out; p.status = h.status;
  int rc;
  if (nmax <= 4) rc = launch<4>(p, c.stream);
  else if (nmax <= 8) rc = launch<8>(p, c.stream);
  else if (nmax <= 16) rc = launch<16>(p, c.stream);
  else rc = launch<32>(p, c.stream);
  if (rc == BI_OK) {
    mut->launches += 1;
    mut->last_kernel = "pair_filter_f64";
  }
  return rc;
}
