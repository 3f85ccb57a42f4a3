// Window kernel (VMP and MMP) for models whose dependency groups span at most two factors: every
// modality depends on a single factor or on a pair of factors (one pair, the models pair_filter.cu
// serves for filtering; or several: chains, triangles, separate pairs).
//
// One CTA per agent; a unit of LPU lanes owns one time step (LPU = the largest state count rounded up
// to a power of two, lane s owning state s of every factor), so the whole window iterates inside one
// launch with a block barrier per Jacobi iteration (Appendix A-2 runs the window's steps side by
// side; Section IV's transition messages read the neighbouring steps' previous iterate, which the
// units exchange through two belief buffers in shared memory).  Per iteration and factor a lane adds
//   * a constant found once per call: ln D (first step) and the slices of the factor's own modalities,
//   * the two transition messages: dot products of the neighbours' beliefs with one row of a
//     transposed transition matrix, read [summation index][own state] so that the unit's lanes read
//     consecutive addresses (the matrices of a shared model stay in L1),
//   * for every two-factor group the factor is in, a matrix-vector product with the step's summed
//     slice, staged once per call in shared memory (row-major with a padded row: a lane reads its row
//     for the group's first factor and its column for the second without bank conflicts; a model with
//     a single such group and units below 32 lanes keeps the row in registers),
// and takes the softmax over the unit's lanes (table-driven exponential, shift by the largest binary
// exponent).  Float64 handles, plain (undamped) update, trivial B-dependencies.
#include <algorithm>

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

struct PairWinParams {
  int32_t N, T, K, F, M, S, G, algo;
  double lambda;   // damping step on the logits; 1 = the plain update
  int32_t n[BI_MAX_F], off[BI_MAX_F], npad[BI_MAX_F], U[BI_MAX_F];
  // transition matrices read [summation index][own state]: past edge and future edge
  const R *Mp[BI_MAX_F], *Mf[BI_MAX_F], *logD[BI_MAX_F];
  int64_t Bstride[BI_MAX_F], Dstride[BI_MAX_F];
  int32_t r1_begin[BI_MAX_F + 1];
  int32_t r1_mod[BI_MAX_M], r1_m[BI_MAX_M], r1_P[BI_MAX_M];
  const R *r1_logA[BI_MAX_M];
  int64_t r1_gstride[BI_MAX_M];
  // the groups over two factors (ng of them; fa[0] < 0 when ng == 0): factors, sizes, and their member
  // modalities [g2_begin[j], g2_begin[j + 1]) of the r2 arrays; slices [m][na][npb]
  int32_t ng, fa[BI_MAX_GROUPS], fb[BI_MAX_GROUPS], na[BI_MAX_GROUPS], nb[BI_MAX_GROUPS], npb[BI_MAX_GROUPS];
  int32_t g2_begin[BI_MAX_GROUPS + 1];
  int32_t r2_mod[BI_MAX_M], r2_m[BI_MAX_M];
  const R *r2_logA[BI_MAX_M];
  int64_t r2_gstride[BI_MAX_M];
  const int32_t *obs, *act;
  const float *q_init;
  const R *lnprior;
  float *q_out, *logq_out;
  int32_t *argmax_out;
  uint32_t *status;
  int32_t units;   // step slots per CTA (whole warps)
  // staged slices of the two-factor groups: `nar` rows of `ls` entries each (the groups' largest first
  // axis; their largest padded second axis plus one: an odd stride, so rows and columns are both read
  // without bank conflicts), sized by the model and not by the lane count so that two CTAs fit an SM
  int32_t nar, ls;
};

template <int LPU>
__device__ __forceinline__ R unit_sum(R v) {
#pragma unroll
  for (int d = LPU / 2; d >= 1; d >>= 1) v += __shfl_xor_sync(0xffffffffu, v, d);
  return v;
}
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

// Both edges' dot products at once: dp = sum_r Mp[r][s] qp[r], df = sum_r Mf[r][s] qf[r], r < n.  Two
// summation indices per trip (the beliefs are read as 16-byte pairs), the trip unrolled twice so that
// eight matrix loads are in flight; pointers advance by additions only.
__device__ __forceinline__ void edge_dots(const R *__restrict__ mp, const R *__restrict__ mf, int stride,
                                          const R *qp, const R *qf, int n, R &dp, R &df) {
  R p0 = 0.0, p1 = 0.0, f0 = 0.0, f1 = 0.0;
  const int st2 = 2 * stride;
  int r = 0;
#pragma unroll 2
  for (; r + 1 < n; r += 2) {
    R x0, x1, y0, y1;
    lds2(qp + r, x0, x1);
    lds2(qf + r, y0, y1);
    p0 = fma(__ldg(mp), x0, p0); p1 = fma(__ldg(mp + stride), x1, p1);
    f0 = fma(__ldg(mf), y0, f0); f1 = fma(__ldg(mf + stride), y1, f1);
    mp += st2;
    mf += st2;
  }
  if (r < n) {
    p0 = fma(__ldg(mp), qp[r], p0);
    f0 = fma(__ldg(mf), qf[r], f0);
  }
  dp = p0 + p1;
  df = f0 + f1;
}

// MAXT: the most threads a launch of this instantiation has; windows of up to 320 threads get a
// register budget under which two CTAs share an SM.  DAMPED: every iteration takes a step of size
// lambda on the logits from the previous iterate's, kept in shared memory (the first from ln q of the
// starting belief; the uniform start's is a constant, taken as 0); instantiations of their own.
template <int LPU, int ALGO, int MAXT, bool DAMPED>
__global__ void __launch_bounds__(MAXT, MAXT <= 320 ? 2 : 1) bi_pair_window_kernel(const PairWinParams p) {
  const int LS = p.ls, NAR = p.nar;   // row stride and rows of a staged slice
  constexpr bool LREG = LPU < 32;   // the slice's row stays in registers for the iterations
  extern __shared__ __align__(16) unsigned char smem_raw[];
  R *exp_tab = reinterpret_cast<R *>(smem_raw);                 // [EXP_TAB]
  R *qb = exp_tab + EXP_TAB;                                    // [2][units + 2][F][LPU]; slot 0 and the last are never read as neighbours of a real edge
  const int slot_sz = p.F * LPU, buf_sz = (p.units + 2) * slot_sz;
  R *cst = qb + 2 * buf_sz;                                     // [units][F][LPU] constants of the logits
  R *xpv = cst + p.units * slot_sz;                             // DAMPED: [units][F][LPU] the previous iterate's logits
  R *Ls = xpv + (DAMPED ? p.units * slot_sz : 0);               // [units][ng][LPU][LS] the pair groups' summed slices, row-major
  const R lam = p.lambda, oml = 1.0 - lam;
  int32_t *aoff = reinterpret_cast<int32_t *>(Ls + (((size_t)p.units * p.ng * NAR * LS + 1) & ~(size_t)1));   // [units][F][2] matrix offsets of the two edges
  for (int j = threadIdx.x; j < EXP_TAB; j += blockDim.x) exp_tab[j] = exp2((double)j * (1.0 / EXP_TAB));

  const int agent = blockIdx.x, g = p.G == 1 ? 0 : agent;
  const int tl = threadIdx.x / LPU, s = threadIdx.x % LPU;
  const bool live = tl < p.T;
  const int t = live ? tl : p.T - 1;   // idle units shadow the last step; they store nothing
  const size_t ob = (size_t)agent * p.T + t;
  const int32_t *obs_t = p.obs + ob * p.M;
  const int NG = p.ng;

  // ---- once per call: constants, matrix offsets, the pair's slice, the starting beliefs
  for (int f = 0; f < p.F; ++f) {
    const int nf = p.n[f];
    const bool ok = s < nf;
    R c = 0.0;
    if (t == 0 && ok)
      c = p.lnprior ? p.lnprior[(size_t)agent * p.S + p.off[f] + s] : __ldg(p.logD[f] + (size_t)g * p.Dstride[f] + s);
    for (int j = p.r1_begin[f]; j < p.r1_begin[f + 1]; ++j) {
      const int o = clamp_flag(__ldg(obs_t + p.r1_mod[j]), p.r1_m[j], p.status, BI_FLAG_OBS_RANGE);
      if (ok) c += __ldg(p.r1_logA[j] + (size_t)g * p.r1_gstride[j] + (size_t)o * p.r1_P[j] + s);
    }
    R q0 = ok ? 1.0 / nf : 0.0;
    if (p.q_init && ok) q0 = (R)__ldg(p.q_init + ob * p.S + p.off[f] + s);
    {   // (idle units fill their slots too: nothing in shared memory stays unwritten)
      cst[(tl * p.F + f) * LPU + s] = c;
      qb[(tl + 1) * slot_sz + f * LPU + s] = q0;
      qb[buf_sz + (tl + 1) * slot_sz + f * LPU + s] = 0.0;
      if (DAMPED) xpv[(tl * p.F + f) * LPU + s] = (p.q_init && ok) ? bi_log(bi_max(q0, (R)BI_EPS)) : 0.0;
      if (s < 2) {
        int off = 0;
        const int tt = s == 0 ? t - 1 : t;   // the action that drives t-1 -> t, or t -> t+1
        if (tt >= 0 && tt < p.T - 1) {
          const int ua = clamp_flag(__ldg(p.act + ((size_t)agent * (p.T - 1) + tt) * p.F + f), p.U[f], p.status,
                                    BI_FLAG_ACT_RANGE);
          off = ua * nf * p.npad[f];
        }
        aoff[(tl * p.F + f) * 2 + s] = off;
      }
    }
  }
  // the groups' summed slices: lane s forms row s; a single group's row also stays in registers
  R L[LPU];
#pragma unroll
  for (int i = 0; i < LPU; ++i) L[i] = 0.0;
  for (int gj = 0; gj < NG; ++gj) {
    const bool a_ok = s < p.na[gj];
#pragma unroll
    for (int i = 0; i < LPU; ++i) L[i] = 0.0;
    for (int j = p.g2_begin[gj]; j < p.g2_begin[gj + 1]; ++j) {
      const int o = clamp_flag(__ldg(obs_t + p.r2_mod[j]), p.r2_m[j], p.status, BI_FLAG_OBS_RANGE);
      const R *row = p.r2_logA[j] + (size_t)g * p.r2_gstride[j] + ((size_t)o * p.na[gj] + (a_ok ? s : 0)) * p.npb[gj];
#pragma unroll
      for (int i = 0; i < LPU; i += 2) {
        if (i < p.npb[gj]) {
          const double2 x = __ldg(reinterpret_cast<const double2 *>(row + i));
          L[i] += x.x; L[i + 1] += x.y;
        }
      }
    }
#pragma unroll
    for (int i = 0; i < LPU; ++i) {
      if (!a_ok) L[i] = 0.0;
      if (s < NAR && i < LS) Ls[(((size_t)tl * NG + gj) * NAR + s) * LS + i] = L[i];
    }
  }
  // slots 0 and units + 1 (the neighbours of the window's ends): zeros, never weighted
  for (int i = threadIdx.x; i < slot_sz; i += blockDim.x) {
    qb[i] = qb[buf_sz + i] = 0.0;
    qb[(p.units + 1) * slot_sz + i] = qb[buf_sz + (p.units + 1) * slot_sz + i] = 0.0;
  }
  __syncthreads();

  const bool has_prev = t > 0, has_next = t + 1 < p.T;
  int cur = 0;
  for (int k = 0; k < p.K; ++k) {
    const R *qc = qb + cur * buf_sz + (tl + 1) * slot_sz;   // this step's beliefs, previous iterate
    R *qn = qb + (cur ^ 1) * buf_sz + (tl + 1) * slot_sz;
    const bool final = k == p.K - 1;
    for (int f = 0; f < p.F; ++f) {
      const int nf = p.n[f], np = p.npad[f];
      const bool ok = s < nf;
      const int sc = ok ? s : 0;
      R x = cst[(tl * p.F + f) * LPU + s];
      // transition messages (both evaluated; a window's ends discard theirs)
      {
        const int2 ao = *reinterpret_cast<const int2 *>(aoff + (tl * p.F + f) * 2);
        const R *mp = p.Mp[f] + (size_t)g * p.Bstride[f] + ao.x + sc;
        const R *mf = p.Mf[f] + (size_t)g * p.Bstride[f] + ao.y + sc;
        R dp, df;
        edge_dots(mp, mf, np, qc - slot_sz + f * LPU, qc + slot_sz + f * LPU, nf, dp, df);
        if (ALGO == BI_ALGO_MMP) {
          dp = 0.5 * bi_log_inline(bi_max(dp, (R)BI_EPS));
          df = 0.5 * bi_log_inline(bi_max(df, (R)BI_EPS));
        }
        x += (has_prev ? dp : 0.0) + (has_next ? df : 0.0);
      }
      for (int gj = 0; gj < NG; ++gj) {
        const R *Lg = Ls + ((size_t)tl * NG + gj) * NAR * LS;
        if (f == p.fa[gj]) {          // row s of the group's slice with the other factor's belief
          const R *qo = qc + p.fb[gj] * LPU;
          const R *rowp = Lg + (size_t)(s < NAR ? s : 0) * LS;   // (several groups, or 32-lane units: the row from the staged copy)
          const bool lreg = LREG && NG == 1;
          R v0 = 0.0, v1 = 0.0;
#pragma unroll
          for (int i = 0; i < LPU; i += 2) {
            if (i + 1 < LS) {   // (a row holds LS - 1 entries, an even count)
              R b0, b1;
              lds2(qo + i, b0, b1);
              v0 = fma(lreg ? L[i] : rowp[i], b0, v0); v1 = fma(lreg ? L[i + 1] : rowp[i + 1], b1, v1);
            }
          }
          x += v0 + v1;
        } else if (f == p.fb[gj]) {   // column s
          const R *qo = qc + p.fa[gj] * LPU;
          const R *col = Lg + (s < LS - 1 ? s : 0);
          R v0 = 0.0, v1 = 0.0;
#pragma unroll
          for (int i = 0; i < LPU; i += 2) {
            if (i < NAR) {      // (NAR rows, an even count)
              R a0, a1;
              lds2(qo + i, a0, a1);
              v0 = fma(col[i * LS], a0, v0); v1 = fma(col[(i + 1) * LS], a1, v1);
            }
          }
          x += v0 + v1;
        }
      }
      if (DAMPED) {
        R *xq = xpv + (tl * p.F + f) * LPU + s;   // (this thread's own entry)
        x = fma(lam, x, oml * *xq);
        *xq = x;
      }
      int kk;
      const R mant = exp_mant(ok ? x : 0.0, exp_tab, kk);
      const int Mx = max_k<LPU, true>(ok ? kk : INT_MIN) >> EXP_BITS;
      const R e = ok ? exp_scale(mant, (kk >> EXP_BITS) - Mx) : 0.0;
      const R z = unit_sum<LPU>(e);
      const R rz = rcp_fast(z);
      const R q = e * (rz * (2.0 - z * rz));   // a second Newton step: a belief to full precision
      qn[f * LPU + s] = q;
      if (final) {
        if (live && ok) {
          const size_t o = ob * p.S + p.off[f] + s;
          p.q_out[o] = (float)q;
          if (p.logq_out) p.logq_out[o] = (float)(x - ((R)Mx * 0.69314718055994530942 + bi_log(z)));
        }
        if (p.argmax_out) {
          const int am = unit_argmax<LPU>(ok ? x : -bi_inf<R>(), ok ? s : 1 << 20);
          if (live && s == 0) p.argmax_out[ob * p.F + f] = am;
        }
      }
    }
    __syncthreads();
    cur ^= 1;
  }
}

template <int LPU>
int launch(PairWinParams &p, const bi_model *md, cudaStream_t stream) {
  const int threads = ((p.T * LPU + 31) / 32) * 32;
  if (threads > 512) return BI_ERR_UNSUPPORTED;   // (the kernel's register budget is set for this)
  p.units = threads / LPU;
  const size_t slot = (size_t)p.F * LPU;
  const bool damped = p.lambda != 1.0;
  size_t elems = EXP_TAB + 2 * (p.units + 2) * slot + (damped ? 2 : 1) * p.units * slot + (((size_t)p.units * p.ng * p.nar * p.ls + 1) & ~(size_t)1);
  const size_t bytes = elems * sizeof(R) + (size_t)p.units * p.F * 2 * sizeof(int32_t) + 16;
  if (bytes > (size_t)md->max_smem_optin - 1024) return BI_ERR_UNSUPPORTED;
  void (*kern)(const PairWinParams);
  if (threads <= 320) {
    if (damped) kern = p.algo == BI_ALGO_VMP ? bi_pair_window_kernel<LPU, BI_ALGO_VMP, 320, true> : bi_pair_window_kernel<LPU, BI_ALGO_MMP, 320, true>;
    else kern = p.algo == BI_ALGO_VMP ? bi_pair_window_kernel<LPU, BI_ALGO_VMP, 320, false> : bi_pair_window_kernel<LPU, BI_ALGO_MMP, 320, false>;
  } else {
    if (damped) kern = p.algo == BI_ALGO_VMP ? bi_pair_window_kernel<LPU, BI_ALGO_VMP, 512, true> : bi_pair_window_kernel<LPU, BI_ALGO_MMP, 512, true>;
    else kern = p.algo == BI_ALGO_VMP ? bi_pair_window_kernel<LPU, BI_ALGO_VMP, 512, false> : bi_pair_window_kernel<LPU, BI_ALGO_MMP, 512, false>;
  }
  if (cudaFuncSetAttribute((const void *)kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes) != cudaSuccess) {
    cudaGetLastError();
    return BI_ERR_CUDA;
  }
  kern<<<p.N, threads, bytes, stream>>>(p);
  return cudaGetLastError() == cudaSuccess ? BI_OK : BI_ERR_CUDA;
}

}  // namespace

// Applicable to float64 handles, plain and damped updates, trivial B-dependencies, window calls (also warm
// starts and continued windows) on models with no group over more than two factors, and to windows
// whose steps and staged slices fit one CTA; BI_ERR_UNSUPPORTED otherwise.
int bi_launch_pair_window(const BiCall &c, bi_model *mut) {
  const bi_model *md = c.model;
  const BiDev &h = md->h;
  if (c.algo == BI_ALGO_FILTER || md->arith != BI_ARITH_F64 || h.has_bdep) return BI_ERR_UNSUPPORTED;
  if (!md->rank2_ok) return BI_ERR_UNSUPPORTED;
  PairWinParams p;
  memset(&p, 0, sizeof(p));
  p.lambda = c.lambda;
  p.N = c.N; p.T = c.T; p.K = c.K; p.F = h.F; p.M = h.M; p.S = h.S; p.G = h.G; p.algo = c.algo;
  int nmax = 1;
  for (int f = 0; f < h.F; ++f) {
    p.n[f] = h.n[f]; p.off[f] = h.off[f]; p.npad[f] = h.npad[f]; p.U[f] = h.U[f];
    p.Mp[f] = (const R *)(c.algo == BI_ALGO_VMP ? h.logBt[f] : h.BfT[f]);
    p.Mf[f] = (const R *)(c.algo == BI_ALGO_VMP ? h.logB[f] : h.BdagT[f]);
    p.logD[f] = (const R *)h.logD[f];
    p.Bstride[f] = h.Bstride[f]; p.Dstride[f] = h.Dstride[f];
    nmax = h.n[f] > nmax ? h.n[f] : nmax;
  }
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
  int n2 = 0;
  for (int gi = 0; gi < h.ngroups; ++gi) {
    const BiGroup &gr = h.grp[gi];
    if (gr.rank != 2) continue;
    const int gj = p.ng++;
    p.fa[gj] = gr.axis[0]; p.fb[gj] = gr.axis[1];
    p.na[gj] = gr.dim[0]; p.nb[gj] = gr.dim[1];
    p.npb[gj] = bi_pad4(gr.dim[1]);
    p.g2_begin[gj] = n2;
    for (int mi = gr.mem_begin; mi < gr.mem_end; ++mi) {
      const BiMember &mm = h.mem[mi];
      p.r2_mod[n2] = mm.modality; p.r2_m[n2] = mm.m;
      p.r2_logA[n2] = (const R *)mm.logA;
      p.r2_gstride[n2] = mm.gstride;
      ++n2;
    }
  }
  p.g2_begin[p.ng] = n2;
  p.nar = 2; p.ls = 3;
  for (int gj = 0; gj < p.ng; ++gj) {
    p.nar = std::max(p.nar, (p.na[gj] + 1) & ~1);
    p.ls = std::max(p.ls, p.npb[gj] + 1);
  }
  p.obs = c.obs; p.act = c.act; p.q_init = c.q_init; p.lnprior = (const R *)c.lnprior;
  p.q_out = c.q_out; p.logq_out = c.logq_out; p.argmax_out = c.argmax_out; p.status = h.status;
  int rc;
  if (nmax <= 4) rc = launch<4>(p, md, c.stream);
  else if (nmax <= 8) rc = launch<8>(p, md, c.stream);
  else if (nmax <= 16) rc = launch<16>(p, md, c.stream);
  else rc = launch<32>(p, md, c.stream);
  if (rc == BI_OK) {
    mut->launches += 1;
    mut->last_kernel = c.algo == BI_ALGO_VMP ? "pair_vmp_f64" : "pair_mmp_f64";
  }
  return rc;
}
