// Register-tile window kernels (VMP and MMP) for single-group rank-3 models.
//
// One thread-block cluster per agent.  Each CTA of the cluster owns a run of
// consecutive time steps; a group of LPU lanes owns one step.  The summed
// slices of all the CTA's steps are gathered from HBM once and stay in shared
// memory for every iteration (re-reading them would multiply the dominant HBM
// traffic by the iteration count).  Beliefs of neighbouring steps are exchanged
// through shared memory; at a CTA boundary the owning lanes also store their
// beliefs into the neighbouring CTA's halo slot through distributed shared
// memory, so every read in the iteration loop is a local shared-memory load
// (Appendix A-2 runs the window's steps in parallel; Section IV's transition
// messages need the neighbours' beliefs of the previous iterate).
#include <cooperative_groups.h>

#include <algorithm>
#include <type_traits>
#include <cstdlib>

#include "bi_internal.h"
#include "tile3.cuh"
#include "tile3_common.cuh"

namespace cg = cooperative_groups;

namespace {

struct WindowGeom {
  int32_t CS;       // CTAs per cluster (= per agent)
  int32_t Tc;       // time steps per CTA
  int32_t units;    // step slots per CTA (>= Tc; whole warps)
  int32_t off_q, off_se, off_B, off_tp;  // element offsets: belief buffers, gather area, transition matrices, transpose areas
};

// sum_r M[r][s] q[r] with two interleaved accumulators; M and q in shared memory
template <typename R, int N>
__device__ __forceinline__ R col_dot_smem(const R *col, int stride, const R *q) {
  R s0 = (R)0, s1 = (R)0;
#pragma unroll
  for (int r = 0; r + 1 < N; r += 2) {
    s0 = fma(col[r * stride], q[r], s0);
    s1 = fma(col[(r + 1) * stride], q[r + 1], s1);
  }
  if (N & 1) s0 = fma(col[(N - 1) * stride], q[N - 1], s0);
  return s0 + s1;
}

// the same with the column held in registers; the beliefs are read two at a time where their
// offset allows (broadcast loads: half the shared-memory wavefronts)
template <typename R, int N, bool PAIRS>
__device__ __forceinline__ R reg_dot_smem(const R (&col)[N], const R *q) {
  R s0 = (R)0, s1 = (R)0;
  if constexpr (PAIRS && sizeof(R) == 8) {
#pragma unroll
    for (int r = 0; r + 1 < N; r += 2) {
      const double2 x = *reinterpret_cast<const double2 *>(q + r);
      s0 = fma(col[r], x.x, s0);
      s1 = fma(col[r + 1], x.y, s1);
    }
  } else {
#pragma unroll
    for (int r = 0; r + 1 < N; r += 2) {
      s0 = fma(col[r], q[r], s0);
      s1 = fma(col[r + 1], q[r + 1], s1);
    }
  }
  if (N & 1) s0 = fma(col[N - 1], q[N - 1], s0);
  return s0 + s1;
}

// LREG: the step's summed slice lives in registers (small tiles); otherwise in
// shared memory (tiles too large for the register file).
template <typename R, int NA, int NB, int NC, int SB, bool LREG, int ALGO, bool STALE, bool CLUSTER, bool DAMPED>
__global__ void __launch_bounds__(320)
bi_tile3_window_kernel(const Tile3Params p, const WindowGeom geo) {
  using TT = Tile3<R, NA, NB, NC, SB>;
  constexpr int LPU = TT::LPU, NBL = TT::NBL, NCP = TT::NCP, NAP = TT::NAP, VE = TT::VE, NV = TT::NV;
  constexpr int PT = TT::P_TILE;
  constexpr int SQ = (NA + NB + NC + 1) & ~1;  // beliefs of one step, padded to 16 bytes
  extern __shared__ __align__(16) unsigned char smem_raw[];
  R *Ls = reinterpret_cast<R *>(smem_raw);   // [units][PT] summed slices
  // beliefs: two buffers of (units + 2) slots; slot 0 and slot units + 1 are the
  // halos holding the neighbouring CTAs' boundary steps
  R *qb = Ls + geo.off_q;
  R *seb = Ls + geo.off_se;                  // [units][NB + NCP] gathered e_b, e_c
  R *Bs = Ls + geo.off_B;                    // this agent's transition matrices, every action

  // tables of the fast exponential and logarithm (float64; synchronised with the staging below)
  using R2 = typename std::conditional<sizeof(R) == 8, double2, float2>::type;
  __shared__ __align__(16) R exp_tab[sizeof(R) == 8 ? BI_EXP_TAB : 2];
  __shared__ __align__(16) R2 log_tab[sizeof(R) == 8 ? BI_LOG_TAB : 1];
  bi_fast_tabs_init(exp_tab, log_tab, (int)threadIdx.x, (int)blockDim.x);
  int rank = 0;
  if (CLUSTER) rank = (int)cg::this_cluster().block_rank();
  const int agent = blockIdx.x / geo.CS;
  const int g = p.G == 1 ? 0 : agent;
  const int lane = threadIdx.x & 31;
  const int tl = threadIdx.x / LPU;        // step slot of this lane group
  const int t_raw = rank * geo.Tc + tl;
  const bool live = tl < geo.Tc && t_raw < p.T;
  const int t = live ? t_raw : p.T - 1;    // idle groups shadow the last step; their stores are suppressed
  const int T = p.T;

  TT t3;
  t3.init_lane(lane);
  t3.tp = Ls + geo.off_tp + (size_t)tl * TT::TP_UNIT;
  const int a = t3.a, bi = t3.bi, ci = t3.ci;
  const bool a_ok = t3.a_ok, b_ok = t3.b_ok, c_ok = t3.c_ok;
  const int bsafe = b_ok ? bi : 0, csafe = c_ok ? ci : 0, asafe = a_ok ? a : 0;
  R *se = seb + tl * (NB + NCP);
  R *Lt = Ls + (LREG ? 0 : (size_t)tl * PT);
  for (int i = t3.u; i < NB + NCP; i += LPU) se[i] = (R)0;

  // ---- gather the step's summed slice (one HBM read per slice) into registers or shared memory
  if (LREG) {
    const size_t ob = ((size_t)agent * T + t) * p.M;
    const R *slice[BI_MAX_M];
    for (int mi = 0; mi < p.nmem; ++mi) {
      int o = clamp_flag(__ldg(p.obs + ob + p.modality[mi]), p.mcount[mi], p.status, BI_FLAG_OBS_RANGE);
      slice[mi] = (const R *)p.logA[mi] + ((size_t)g * p.mcount[mi] + (size_t)o) * p.P_tile;
    }
    t3.load_slices(slice, p.nmem);
  } else if (p.cmask[0] != nullptr) {
    // Compressed slices (sparse per-agent models): per lane one 64-bit mask of the elements that are
    // not the floor ln 1e-16, and those values packed lane after lane; the HBM traffic of the gather
    // shrinks with the share of zeros in A.  This lane's values start at the slice's offset plus the
    // other lanes' counts before it (a scan over the unit's lanes).
    static_assert(NV * VE <= 64, "a lane's part of a slice must fit one mask");
    constexpr int MAXC = 4;   // the packing layer compresses groups of up to four modalities
    const size_t ob = ((size_t)agent * T + t) * p.M;
    const R flr = __ldg((const R *)p.floor_log);
    unsigned long long mk[MAXC];
    const R *vp[MAXC];
#pragma unroll
    for (int mi = 0; mi < MAXC; ++mi) {
      mk[mi] = 0ull;
      vp[mi] = nullptr;
      if (mi < p.nmem) {
        const int o = clamp_flag(__ldg(p.obs + ob + p.modality[mi]), p.mcount[mi], p.status, BI_FLAG_OBS_RANGE);
        const size_t sl = (size_t)g * p.mcount[mi] + (size_t)o;
        mk[mi] = __ldg(p.cmask[mi] + sl * LPU + t3.u);
        const int cnt = __popcll(mk[mi]);
        int incl = cnt;
#pragma unroll
        for (int d = 1; d < LPU; d <<= 1) {
          const int up = __shfl_up_sync(0xffffffffu, incl, d, LPU);
          if (t3.u >= d) incl += up;
        }
        vp[mi] = (const R *)p.cvals[mi] + __ldg(p.coff[mi] + sl) + (incl - cnt);
      }
    }
    constexpr int CH = NV % 12 == 0 ? 12 : (NV % 8 == 0 ? 8 : (NV % 6 == 0 ? 6 : NV));
    for (int v0 = 0; v0 < NV; v0 += CH) {
      R acc[CH][VE];
#pragma unroll
      for (int v = 0; v < CH; ++v)
#pragma unroll
        for (int i = 0; i < VE; ++i) acc[v][i] = (R)0;
#pragma unroll
      for (int mi = 0; mi < MAXC; ++mi) {
        if (mi < p.nmem) {
#pragma unroll
          for (int v = 0; v < CH; ++v)
#pragma unroll
            for (int i = 0; i < VE; ++i) {
              const bool bit = (mk[mi] & 1ull) != 0ull;
              mk[mi] >>= 1;
              acc[v][i] += bit ? __ldg(vp[mi]) : flr;
              vp[mi] += bit ? 1 : 0;
            }
        }
      }
#pragma unroll
      for (int v = 0; v < CH; ++v)
#pragma unroll
        for (int i = 0; i < VE; ++i) Lt[((v0 + v) * LPU + t3.u) * VE + i] = acc[v][i];
    }
  } else {
    const size_t ob = ((size_t)agent * T + t) * p.M;
    constexpr int CH = NV % 12 == 0 ? 12 : (NV % 8 == 0 ? 8 : (NV % 6 == 0 ? 6 : NV));  // vectors in flight per pass
    for (int v0 = 0; v0 < NV; v0 += CH) {
      R acc[CH][VE];
#pragma unroll
      for (int v = 0; v < CH; ++v)
#pragma unroll
        for (int i = 0; i < VE; ++i) acc[v][i] = (R)0;
      for (int mi = 0; mi < p.nmem; ++mi) {
        int o = clamp_flag(__ldg(p.obs + ob + p.modality[mi]), p.mcount[mi], p.status, BI_FLAG_OBS_RANGE);
        const R *sl = (const R *)p.logA[mi] + ((size_t)g * p.mcount[mi] + (size_t)o) * p.P_tile +
                      ((size_t)v0 * LPU + t3.u) * VE;
#pragma unroll
        for (int v = 0; v < CH; ++v) {
          R x[VE];
          ldg_vec(sl + v * LPU * VE, x);
#pragma unroll
          for (int i = 0; i < VE; ++i) acc[v][i] += x[i];
        }
      }
#pragma unroll
      for (int v = 0; v < CH; ++v)
#pragma unroll
        for (int i = 0; i < VE; ++i) Lt[((v0 + v) * LPU + t3.u) * VE + i] = acc[v][i];
    }
  }

  // ---- this agent's transition matrices, staged once; then the columns this
  // lane needs for its owned states on the step's two edges.  Transposed
  // layouts ([previous][next] for the past edge, [next][previous] for the
  // future edge): the lanes of a group read consecutive addresses.
  const R *pa0, *pa1, *pa2, *fu0, *fu1, *fu2;
  R dprior[3] = {0, 0, 0};
  {
    const int own[3] = {asafe, bsafe, csafe};
    const int nn[3] = {NA, NB, NC};
    const R *pa[3], *fu[3];
    int boff = 0;
#pragma unroll
    for (int j = 0; j < 3; ++j) {
      const int msz = p.U[j] * nn[j] * p.np[j];
      const R *Mp = (const R *)(ALGO == BI_ALGO_VMP ? p.logBt[j] : p.BfT[j]) + (size_t)g * p.Bstride[j];
      const R *Mf = (const R *)(ALGO == BI_ALGO_VMP ? p.logB[j] : p.BdagT[j]) + (size_t)g * p.Bstride[j];
      for (int i = threadIdx.x; i < msz; i += blockDim.x) {
        Bs[boff + i] = __ldg(Mp + i);
        Bs[boff + msz + i] = __ldg(Mf + i);
      }
      int up = 0, uf = 0;
      if (t == 0)
        dprior[j] = p.lnprior ? __ldg((const R *)p.lnprior + (size_t)agent * p.S + p.off[j] + own[j])
                              : __ldg((const R *)p.logD[j] + (size_t)g * p.Dstride[j] + own[j]);
      else up = clamp_flag(__ldg(p.act + ((size_t)agent * (T - 1) + (t - 1)) * 3 + p.fac[j]), p.U[j], p.status,
                           BI_FLAG_ACT_RANGE);
      if (t + 1 < T)
        uf = clamp_flag(__ldg(p.act + ((size_t)agent * (T - 1) + t) * 3 + p.fac[j]), p.U[j], p.status,
                        BI_FLAG_ACT_RANGE);
      pa[j] = Bs + boff + up * nn[j] * p.np[j] + own[j];
      fu[j] = Bs + boff + msz + uf * nn[j] * p.np[j] + own[j];
      boff += 2 * msz;
    }
    pa0 = pa[0]; pa1 = pa[1]; pa2 = pa[2];
    fu0 = fu[0]; fu1 = fu[1]; fu2 = fu[2];
  }

  // ---- belief slots: own step at slot tl + 1; neighbours at tl and tl + 2
  const int bufsz = (geo.units + 2) * SQ;
  R *q_cur = qb + (size_t)(tl + 1) * SQ;   // this step, buffer 0
  R *q_nxt = q_cur + bufsz;                // this step, buffer 1
  // remote halo slots this group also feeds (same offsets in the neighbour CTA)
  R *r_prev_cur = nullptr, *r_prev_nxt = nullptr, *r_next_cur = nullptr, *r_next_nxt = nullptr;
  if (CLUSTER) {
    cg::cluster_group cl = cg::this_cluster();
    if (live && tl == 0 && rank > 0) {
      R *rb = cl.map_shared_rank(qb, rank - 1);
      r_prev_cur = rb + (size_t)(geo.Tc + 1) * SQ;  // the previous CTA's "next" halo
      r_prev_nxt = r_prev_cur + bufsz;
    }
    if (live && tl == geo.Tc - 1 && rank + 1 < geo.CS) {
      R *rb = cl.map_shared_rank(qb, rank + 1);
      r_next_cur = rb;                              // the next CTA's "previous" halo
      r_next_nxt = rb + bufsz;
    }
  }
  // uniform start (every slot, halos included: neighbours start uniform too)
  for (int i = threadIdx.x; i < (geo.units + 2) * SQ; i += blockDim.x) {
    const int s = i % SQ;
    qb[i] = s < NA ? (R)1 / (R)NA : s < NA + NB ? (R)1 / (R)NB : s < NA + NB + NC ? (R)1 / (R)NC : (R)0;
  }
  t3.set_uniform();
  R pxa = 0, pxb = 0, pxc = 0;   // previous iterate's logits (uniform start: a constant, taken as 0)
  const R lam = (R)p.lambda, oml = (R)1 - lam;
  if (p.q_init) {
    // Warm start: every slot that stands for a real step (halos included) takes that step's
    // given beliefs; this lane group then holds them as e with normalisers of 1.
    __syncthreads();
    for (int i = threadIdx.x; i < (geo.units + 2) * SQ; i += blockDim.x) {
      const int slot = i / SQ, s = i % SQ, ts = rank * geo.Tc + slot - 1;
      if (ts < 0 || ts >= T || s >= NA + NB + NC) continue;
      const int j = s < NA ? 0 : s < NA + NB ? 1 : 2;
      const int sj = s - (j == 0 ? 0 : j == 1 ? NA : NA + NB);
      qb[i] = (R)__ldg(p.q_init + ((size_t)agent * T + ts) * p.S + p.off[j] + sj);
    }
    __syncthreads();
    const R *qs = qb + (size_t)(tl + 1) * SQ;   // this group's own step (idle groups shadow a valid slot's layout)
    t3.ea = a_ok ? qs[asafe] : (R)0;
#pragma unroll
    for (int bl = 0; bl < TT::NBL; ++bl) t3.eb[bl] = qs[NA + t3.bh * TT::NBL + bl];
#pragma unroll
    for (int c = 0; c < TT::NCP; ++c) t3.ec[c] = c < NC ? qs[NA + NB + c] : (R)0;
    t3.sa = t3.sb = t3.sc = (R)1;
    // the damped update starts from the logarithms of the given beliefs
    if (DAMPED) pxa = a_ok ? bi_log(bi_max(qs[asafe], (R)BI_EPS)) : (R)0;
    if (DAMPED) pxb = b_ok ? bi_log(bi_max(qs[NA + bsafe], (R)BI_EPS)) : (R)0;
    if (DAMPED) pxc = c_ok ? bi_log(bi_max(qs[NA + NB + csafe], (R)BI_EPS)) : (R)0;
  }
  // With the slices in shared memory the register file has room for the transition-matrix column
  // of each owned state (for the one edge this lane evaluates): they do not change between
  // iterations, and reading them from shared memory again every time was a third of the
  // kernel's shared-memory traffic.
  constexpr int NPA_ = (NA + 3) & ~3, NPB_ = (NB + 3) & ~3, NPC_ = (NC + 3) & ~3;
  constexpr bool DUPA_ = SB >= 2, DUPB_ = !TT::TP && TT::SHB >= 1;
  // (the a and b columns: with the c column as well the kernel spills at the 168 registers a
  // ten-warp CTA may use, and measured slower)
  constexpr bool BRA = !LREG && DUPA_, BRB = !LREG && DUPB_, BRC = false;
  R bca[BRA ? NA : 1], bcb[BRB ? NB : 1], bcc[BRC ? NC : 1];
  if (BRA || BRB || BRC) {
    __syncthreads();
    if (BRA) {
      const R *col = (t3.u & 1) ? fu0 : pa0;
#pragma unroll
      for (int r = 0; r < (BRA ? NA : 1); ++r) bca[r] = col[r * NPA_];
    }
    if (BRB) {
      const R *col = (a & 1) ? fu1 : pa1;
#pragma unroll
      for (int r = 0; r < (BRB ? NB : 1); ++r) bcb[r] = col[r * NPB_];
    }
    if (BRC) {
      const R *col = (t3.u & 1) ? fu2 : pa2;
#pragma unroll
      for (int r = 0; r < (BRC ? NC : 1); ++r) bcc[r] = col[r * NPC_];
    }
  }
  // The barrier between iterations is split: a CTA arrives as soon as its beliefs are published and
  // waits only when it needs its neighbours', with the contraction (own data only) in between.
  // (A launch without a cluster attribute is a cluster of one CTA, so the same barrier serves both.)
  // Only the warps that store into a neighbouring CTA's halo need the arrival to release at cluster
  // scope; for the others every store before it is to this CTA's own shared memory, so a fence at
  // CTA scope and a relaxed arrival give the same ordering without the wider fence's latency.
  // (The wait keeps its acquire: it orders the halo reads after the neighbours' stores.)
  const bool remote_writer =
      CLUSTER && __any_sync(0xffffffffu, r_prev_cur != nullptr || r_next_cur != nullptr) != 0;
  auto arrive = [&]() {
    if (remote_writer) asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    else asm volatile("fence.acq_rel.cta;\n\tbarrier.cluster.arrive.relaxed.aligned;" ::: "memory");
  };
  auto wait = [&]() { asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory"); };
  arrive();

  R xa = 0, xb = 0, xc = 0, za = 1, zb = 1, zc = 1, rinv = 1;
  float ma = 0.f, mb = 0.f, mc = 0.f, pma = 0.f, pmb = 0.f, pmc = 0.f;
  for (int k = 0; k < p.K; ++k) {
    // likelihood messages from this step's own beliefs, while the other CTAs finish publishing theirs
    if (LREG) t3.messages(xa, xb, xc);
    else t3.messages_smem(Lt, xa, xb, xc);
    wait();
    // Transition messages from the previous iterate of the neighbouring steps.
    // Both edges are evaluated without branches (a window's first and last
    // step read their halo slot, which always holds valid beliefs, and discard
    // the result).
    // Where a state is owned by two or more lanes of the group (more lanes than
    // states), one of them evaluates the past edge and its neighbour the future
    // edge at the same time, and a shuffle adds the two: half the dot products
    // and half the logarithms per lane.
    R ta, tb, tc;
    {
      // row strides of the staged matrices: each factor's padded state count, known at compile time
      constexpr int NPA = (NA + 3) & ~3, NPB = (NB + 3) & ~3, NPC = (NC + 3) & ~3;
      const R *qp = q_cur - SQ, *qn = q_cur + SQ;
      const bool has_prev = t > 0, has_next = t + 1 < T;
      auto edge = [&](R dot, bool future, R prior) -> R {
        const R v = ALGO == BI_ALGO_MMP ? (R)0.5 * bi_log_fast(bi_max(dot, (R)BI_EPS), log_tab) : dot;
        return future ? (has_next ? v : (R)0) : (has_prev ? v : prior);
      };
      constexpr bool DUPA = SB >= 2, DUPB = !TT::TP && TT::SHB >= 1, DUPC = !TT::TP && TT::SHC >= 1;
      if (DUPA) {
        const bool fut = (t3.u & 1) != 0;   // u = a * SB + bh: the lowest bit tells the two apart
        const R dot = BRA ? reg_dot_smem<R, BRA ? NA : 1, true>(bca, fut ? qn : qp)
                          : col_dot_smem<R, NA>(fut ? fu0 : pa0, NPA, fut ? qn : qp);
        const R v = edge(dot, fut, dprior[0]);
        ta = v + __shfl_xor_sync(0xffffffffu, v, 1);
      } else {
        ta = edge(col_dot_smem<R, NA>(pa0, NPA, qp), false, dprior[0]) +
             edge(col_dot_smem<R, NA>(fu0, NPA, qn), true, (R)0);
      }
      if (DUPB) {
        const bool fut = (a & 1) != 0;      // duplicates of a b owner differ in the low bits of a
        const R dot = BRB ? reg_dot_smem<R, BRB ? NB : 1, NA % 2 == 0>(bcb, (fut ? qn : qp) + NA)
                          : col_dot_smem<R, NB>(fut ? fu1 : pa1, NPB, (fut ? qn : qp) + NA);
        const R v = edge(dot, fut, dprior[1]);
        tb = v + __shfl_xor_sync(0xffffffffu, v, SB);
      } else {
        tb = edge(col_dot_smem<R, NB>(pa1, NPB, qp + NA), false, dprior[1]) +
             edge(col_dot_smem<R, NB>(fu1, NPB, qn + NA), true, (R)0);
      }
      if (DUPC) {
        const bool fut = (t3.u & 1) != 0;   // duplicates of a c owner differ in the low bits of u
        const R dot = BRC ? reg_dot_smem<R, BRC ? NC : 1, (NA + NB) % 2 == 0>(bcc, (fut ? qn : qp) + NA + NB)
                          : col_dot_smem<R, NC>(fut ? fu2 : pa2, NPC, (fut ? qn : qp) + NA + NB);
        const R v = edge(dot, fut, dprior[2]);
        tc = v + __shfl_xor_sync(0xffffffffu, v, 1);
      } else {
        tc = edge(col_dot_smem<R, NC>(pa2, NPC, qp + NA + NB), false, dprior[2]) +
             edge(col_dot_smem<R, NC>(fu2, NPC, qn + NA + NB), true, (R)0);
      }
    }
    xa = a_ok ? xa + ta : -bi_inf<R>();
    xb = b_ok ? xb + tb : -bi_inf<R>();
    xc = c_ok ? xc + tc : -bi_inf<R>();
    if (DAMPED) {   // damped step on the logits (a shift per factor does not matter)
      xa = a_ok ? fma(lam, xa, oml * pxa) : xa;
      xb = b_ok ? fma(lam, xb, oml * pxb) : xb;
      xc = c_ok ? fma(lam, xc, oml * pxc) : xc;
      pxa = a_ok ? xa : (R)0; pxb = b_ok ? xb : (R)0; pxc = c_ok ? xc : (R)0;
    }
    const float cma = group_max_f<NAP, SB>((float)xa);
    const float cmb = group_max_f<LPU, 1>((float)xb);
    const float cmc = group_max_f<LPU, 1>((float)xc);
    if (!STALE || k == 0) { ma = cma; mb = cmb; mc = cmc; }
    else { ma = pma; mb = pmb; mc = pmc; }
    pma = cma; pmb = cmb; pmc = cmc;
    const R ean = a_ok ? bi_exp_fast(xa - (R)ma, exp_tab) : (R)0;
    const R ebn = b_ok ? bi_exp_fast(xb - (R)mb, exp_tab) : (R)0;
    const R ecn = c_ok ? bi_exp_fast(xc - (R)mc, exp_tab) : (R)0;
    __syncwarp();
    if (t3.own_b) se[bi] = ebn;
    if (t3.own_c) se[NB + ci] = ecn;
    za = group_sum<R, NAP, SB>(ean);
    __syncwarp();
    t3.ea = ean;
    if constexpr (sizeof(R) == 8 && NBL % 2 == 0 && NB % 2 == 0) {   // 16-byte broadcast loads
#pragma unroll
      for (int bl = 0; bl < NBL; bl += 2) {
        const double2 x = *reinterpret_cast<const double2 *>(se + t3.bh * NBL + bl);
        t3.eb[bl] = x.x; t3.eb[bl + 1] = x.y;
      }
#pragma unroll
      for (int c = 0; c < NCP; c += 2) {
        const double2 x = *reinterpret_cast<const double2 *>(se + NB + c);
        t3.ec[c] = x.x; t3.ec[c + 1] = x.y;
      }
    } else {
#pragma unroll
      for (int bl = 0; bl < NBL; ++bl) t3.eb[bl] = se[t3.bh * NBL + bl];
#pragma unroll
      for (int c = 0; c < NCP; ++c) t3.ec[c] = se[NB + c];
    }
    zb = group_sum<R, SB, 1>(tree_sum<R, NBL>(t3.eb));
    zc = tree_sum<R, NCP>(t3.ec);
    rinv = bi_rcp(za * zb * zc);
    t3.sa = rinv * za;
    t3.sb = rinv * zb;
    t3.sc = rinv * zc;
    // normalised beliefs for the neighbours' next iteration
    const R qa = ean * (rinv * zb * zc), qbv = ebn * (rinv * za * zc), qc = ecn * (rinv * za * zb);
    // (idle groups do not publish: the slot after a CTA's last step is a halo)
    if (live && t3.own_a) q_nxt[a] = qa;
    if (live && t3.own_b) q_nxt[NA + bi] = qbv;
    if (live && t3.own_c) q_nxt[NA + NB + ci] = qc;
    if (CLUSTER) {
      if (r_prev_nxt) {
        if (t3.own_a) r_prev_nxt[a] = qa;
        if (t3.own_b) r_prev_nxt[NA + bi] = qbv;
        if (t3.own_c) r_prev_nxt[NA + NB + ci] = qc;
      }
      if (r_next_nxt) {
        if (t3.own_a) r_next_nxt[a] = qa;
        if (t3.own_b) r_next_nxt[NA + bi] = qbv;
        if (t3.own_c) r_next_nxt[NA + NB + ci] = qc;
      }
    }
    if (k == p.K - 1) {
      const size_t ob = (size_t)agent * T + t;
      if (live) {
        float *qo = p.q_out + ob * p.S;
        if (t3.own_a) qo[p.off[0] + a] = (float)qa;
        if (t3.own_b) qo[p.off[1] + bi] = (float)qbv;
        if (t3.own_c) qo[p.off[2] + ci] = (float)qc;
        if (p.logq_out) {
          float *lo = p.logq_out + ob * p.S;
          if (t3.own_a) lo[p.off[0] + a] = (float)(xa - (R)ma - bi_log(za));
          if (t3.own_b) lo[p.off[1] + bi] = (float)(xb - (R)mb - bi_log(zb));
          if (t3.own_c) lo[p.off[2] + ci] = (float)(xc - (R)mc - bi_log(zc));
        }
      }
      if (p.argmax_out) {
        const int ia = group_argmax<R, NAP, SB>(xa, a_ok ? a : 1 << 20);
        const int ib = group_argmax<R, LPU, 1>(xb, b_ok ? bi : 1 << 20);
        const int ic = group_argmax<R, LPU, 1>(xc, c_ok ? ci : 1 << 20);
        if (live && t3.u == 0) {
          int32_t *ao = p.argmax_out + ob * 3;
          ao[p.fac[0]] = ia;
          ao[p.fac[1]] = ib;
          ao[p.fac[2]] = ic;
        }
      }
    }
    // swap the belief buffers (pointers stay in registers)
    { R *tmp = q_cur; q_cur = q_nxt; q_nxt = tmp; }
    { R *tmp = r_prev_cur; r_prev_cur = r_prev_nxt; r_prev_nxt = tmp; }
    { R *tmp = r_next_cur; r_next_cur = r_next_nxt; r_next_nxt = tmp; }
    arrive();
  }
  wait();   // nobody leaves while a neighbour may still write into its halo
}

template <typename R, int NA, int NB, int NC, int SB, bool LREG, int ALGO>
int launch_window(const Tile3Params &p, int smem_budget, cudaStream_t stream) {
  using TT = Tile3<R, NA, NB, NC, SB>;
  constexpr int SQ = (NA + NB + NC + 1) & ~1;
  constexpr int UPW = TT::UPW;
  WindowGeom geo;
  size_t bytes = 0;
  int threads = 0;
  bool found = false;
  // transition matrices (both directions, every action) are staged in shared memory
  size_t bsz = 0;
  {
    const int nn[3] = {NA, NB, NC};
    for (int j = 0; j < 3; ++j) bsz += 2 * (size_t)p.U[j] * nn[j] * p.np[j];
  }
  if (bsz * sizeof(R) > 48 * 1024) return BI_ERR_UNSUPPORTED;
  // Fewest CTAs per agent whose share of the window fits; a larger cluster is
  // preferred when it lets several CTAs share an SM (more warps in flight to
  // hide the per-iteration barrier).
  const bool stale = sizeof(R) == 8 && p.nmem <= 12;
  // (a damped call is a separate instantiation, so that the plain update carries none of it)
  auto pick = [&](bool cl) -> const void * {
#define BI_WIN_KERN(ST, CL, DA) ((const void *)bi_tile3_window_kernel<R, NA, NB, NC, SB, LREG, ALGO, ST, CL, DA>)
    if (p.lambda != 1.0) return cl ? BI_WIN_KERN(false, true, true) : BI_WIN_KERN(false, false, true);
    if (stale) return cl ? BI_WIN_KERN(true, true, false) : BI_WIN_KERN(true, false, false);
    return cl ? BI_WIN_KERN(false, true, false) : BI_WIN_KERN(false, false, false);
#undef BI_WIN_KERN
  };
  int best_cs = 0;
  double best_score = -1.0;
  for (int cs = 1; cs <= 8; cs *= 2) {
    const int Tc = (p.T + cs - 1) / cs;
    if (cs > 1 && Tc * (cs - 1) >= p.T) continue;  // an empty CTA: no gain over the smaller cluster
    const int warps = (Tc + UPW - 1) / UPW;
    const int units = warps * UPW;
    const size_t elems = (LREG ? 0 : (size_t)units * TT::P_TILE) + 2 * (size_t)(units + 2) * SQ +
                         (size_t)units * (NB + TT::NCP) + bsz + (TT::TP ? (size_t)units * TT::TP_UNIT : 0);
    const size_t b = elems * sizeof(R);
    if (warps * 32 > (320) || b > (size_t)smem_budget) continue;
    // CTAs that fit an SM together (shared memory and registers), as the runtime counts them
    const void *kf = pick(cs > 1);
    int per_sm = 0;
    if (cudaFuncSetAttribute(kf, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)b) != cudaSuccess ||
        cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kf, warps * 32, b) != cudaSuccess) {
      cudaGetLastError();
      continue;
    }
    per_sm = std::min(per_sm, 8);
    if (per_sm < 1) continue;
    // useful warps resident per SM, discounted by idle step slots
    const double score = (double)per_sm * warps * ((double)Tc / units) - 0.01 * cs;
    if (score > best_score) { best_score = score; best_cs = cs; }
  }
  if (best_cs == 0) return BI_ERR_UNSUPPORTED;
  {
    const int cs = best_cs;
    const int Tc = (p.T + cs - 1) / cs;
    const int warps = (Tc + UPW - 1) / UPW;
    const int units = warps * UPW;
    geo.CS = cs; geo.Tc = Tc; geo.units = units;
    geo.off_q = LREG ? 0 : units * TT::P_TILE;
    geo.off_se = geo.off_q + 2 * (units + 2) * SQ;
    geo.off_B = geo.off_se + units * (NB + TT::NCP);
    geo.off_tp = geo.off_B + (int)((bsz + 1) & ~(size_t)1);
    bytes = ((size_t)geo.off_tp + (TT::TP ? (size_t)units * TT::TP_UNIT : 0)) * sizeof(R);
    threads = warps * 32;
    found = true;
  }
  if (!found) return BI_ERR_UNSUPPORTED;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)(p.N * geo.CS));
  cfg.blockDim = dim3((unsigned)threads);
  cfg.dynamicSmemBytes = bytes;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = (unsigned)geo.CS;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = geo.CS > 1 ? 1 : 0;
  const void *kern = pick(geo.CS > 1);
  void *args[2] = {(void *)&p, (void *)&geo};
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
  if (e == cudaSuccess) e = cudaLaunchKernelExC(&cfg, kern, args);
  if (e != cudaSuccess) {
    cudaGetLastError();
    return BI_ERR_CUDA;
  }
  return BI_OK;
}

template <typename R, int ALGO>
int dispatch_window(const Tile3Params &p, int na, int nb, int nc, int budget, cudaStream_t stream) {
#define X(A, B, C, S, LS) \
  if (na == A && nb == B && nc == C) return launch_window<R, A, B, C, S, !(LS), ALGO>(p, budget, stream);
  BI_TILE3_SHAPES(X)
#undef X
  return BI_ERR_UNSUPPORTED;
}

}  // namespace

int bi_launch_tile3_window(const BiCall &c, bi_model *mut) {
  const bi_model *md = c.model;
  if (c.algo == BI_ALGO_FILTER || md->tile_sb <= 0) return BI_ERR_UNSUPPORTED;
  const BiGroup &g = md->h.grp[0];
  Tile3Params p;
  bi_tile3_fill_params(c, p);
  const int budget = md->max_smem_optin - 1024 - 6400;   // (the kernel's static tables)
  int rc;
  const bool f64 = md->arith == BI_ARITH_F64;
  if (c.algo == BI_ALGO_VMP)
    rc = f64 ? dispatch_window<double, BI_ALGO_VMP>(p, g.dim[0], g.dim[1], g.dim[2], budget, c.stream)
             : dispatch_window<float, BI_ALGO_VMP>(p, g.dim[0], g.dim[1], g.dim[2], budget, c.stream);
  else
    rc = f64 ? dispatch_window<double, BI_ALGO_MMP>(p, g.dim[0], g.dim[1], g.dim[2], budget, c.stream)
             : dispatch_window<float, BI_ALGO_MMP>(p, g.dim[0], g.dim[1], g.dim[2], budget, c.stream);
  if (rc == BI_OK) {
    mut->launches += 1;
    mut->last_kernel = c.algo == BI_ALGO_VMP ? (f64 ? "tile3_vmp_f64" : "tile3_vmp_f32")
                                             : (f64 ? "tile3_mmp_f64" : "tile3_mmp_f32");
  }
  return rc;
}
