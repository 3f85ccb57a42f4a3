// The register-tile filtering kernel and its launch templates, shared by the
// two translation units that instantiate it: the plain update and the damped
// one are compiled apart, so that neither's code placement depends on the other.
#pragma once
#include "bi_internal.h"
#include "tile3.cuh"
#include "tile3_common.cuh"

namespace tile3_filter {


// DAMPED: the update takes a step of size p.lambda on the logits (a separate instantiation, so that
// the plain update carries none of it)
template <typename R, int NA, int NB, int NC, int SB, bool LSMEM, bool STALE, bool DAMPED>
__global__ void __launch_bounds__(32) bi_tile3_filter_kernel(const Tile3Params p) {
  using TT = Tile3<R, NA, NB, NC, SB>;
  constexpr int LPU = TT::LPU, UPW = TT::UPW, NBL = TT::NBL, NCP = TT::NCP, NAP = TT::NAP;
  __shared__ __align__(16) R sm_e[UPW][NB + NCP + NAP];  // gathered e_b, e_c, e_a of the current iterate
  __shared__ __align__(16) R sm_q[UPW][NA + NB + NC];  // final beliefs of the previous step
  __shared__ __align__(16) R sm_L[LSMEM ? UPW : 1][LSMEM ? TT::P_TILE : 2];  // large tiles: the step's slice
  __shared__ __align__(16) R sm_tp[UPW][TT::TP ? TT::TP_UNIT : 2];           // transpose area of the b / c sums

  __shared__ R exp_tab[32];   // 2^(j/32) for the table-driven exponential
  bi_exp_tab_init(exp_tab, (int)threadIdx.x);
  const int lane = threadIdx.x;
  const int unit = lane / LPU;
  int agent = blockIdx.x * UPW + unit;
  const bool live = agent < p.N;
  if (!live) agent = p.N - 1;  // keeps every shuffle warp-uniform; its stores are suppressed
  const int g = p.G == 1 ? 0 : agent;

  TT t3;
  t3.init_lane(lane);
  t3.tp = sm_tp[unit];
  const int a = t3.a, bi = t3.bi, ci = t3.ci;
  const bool a_ok = t3.a_ok, b_ok = t3.b_ok, c_ok = t3.c_ok;
  const int bsafe = b_ok ? bi : 0, csafe = c_ok ? ci : 0, asafe = a_ok ? a : 0;
  R *se = sm_e[unit], *sq = sm_q[unit];
  for (int i = t3.u; i < NB + NCP + NAP; i += LPU) se[i] = (R)0;
  __syncwarp();

  const size_t out_base = (size_t)agent * p.T;
  // The index streams are read one step ahead: their DRAM latency then overlaps
  // the previous step's iterations instead of heading every step's chain.
  int o_next[BI_MAX_M], u_next[3] = {0, 0, 0};
  for (int mi = 0; mi < p.nmem; ++mi) o_next[mi] = __ldg(p.obs + out_base * p.M + p.modality[mi]);
  // Continued filtering: the belief of the step before the window takes the
  // place of "the previous step's final belief", and its action that of u_{t-1}.
  const bool from_prev = p.q_prev != nullptr || p.carry_in != nullptr;
  if (from_prev) {
    if (p.carry_in) {   // the previous call's last belief at full precision
      const R *qp = (const R *)p.carry_in + (size_t)agent * p.S;
      if (t3.own_a) sq[a] = qp[p.off[0] + a];
      if (t3.own_b) sq[NA + bi] = qp[p.off[1] + bi];
      if (t3.own_c) sq[NA + NB + ci] = qp[p.off[2] + ci];
    } else {
      const float *qp = p.q_prev + (size_t)agent * p.S;
      if (t3.own_a) sq[a] = (R)__ldg(qp + p.off[0] + a);
      if (t3.own_b) sq[NA + bi] = (R)__ldg(qp + p.off[1] + bi);
      if (t3.own_c) sq[NA + NB + ci] = (R)__ldg(qp + p.off[2] + ci);
    }
    const int32_t *ap = p.act_prev + (size_t)agent * p.F;
    u_next[0] = __ldg(ap + p.fac[0]);
    u_next[1] = __ldg(ap + p.fac[1]);
    u_next[2] = __ldg(ap + p.fac[2]);
    __syncwarp();
  }
  for (int t = 0; t < p.T; ++t) {
    // ---- the step's summed slice: one gather of every modality's observed slice
    const R *slice[BI_MAX_M];
    for (int mi = 0; mi < p.nmem; ++mi) {
      int o = clamp_flag(o_next[mi], p.mcount[mi], p.status, BI_FLAG_OBS_RANGE);
      slice[mi] = (const R *)p.logA[mi] + ((size_t)g * p.mcount[mi] + (size_t)o) * p.P_tile;
    }
    const int u_cur[3] = {u_next[0], u_next[1], u_next[2]};
    if (t + 1 < p.T) {
      for (int mi = 0; mi < p.nmem; ++mi) o_next[mi] = __ldg(p.obs + (out_base + t + 1) * p.M + p.modality[mi]);
      const int32_t *an = p.act + ((size_t)agent * (p.T - 1) + t) * 3;
      u_next[0] = __ldg(an + p.fac[0]);
      u_next[1] = __ldg(an + p.fac[1]);
      u_next[2] = __ldg(an + p.fac[2]);
    }
    if (LSMEM) t3.load_slices_smem(slice, p.nmem, sm_L[LSMEM ? unit : 0]);
    else t3.load_slices(slice, p.nmem);

    // ---- ln prior of the logits this lane owns: D, or B_u times the previous step's belief
    R lpa, lpb, lpc;
    if (t == 0 && !from_prev) {
      lpa = __ldg((const R *)p.logD[0] + (size_t)g * p.Dstride[0] + asafe);
      lpb = __ldg((const R *)p.logD[1] + (size_t)g * p.Dstride[1] + bsafe);
      lpc = __ldg((const R *)p.logD[2] + (size_t)g * p.Dstride[2] + csafe);
    } else {
      int ua = clamp_flag(u_cur[0], p.U[0], p.status, BI_FLAG_ACT_RANGE);
      int ub = clamp_flag(u_cur[1], p.U[1], p.status, BI_FLAG_ACT_RANGE);
      int uc = clamp_flag(u_cur[2], p.U[2], p.status, BI_FLAG_ACT_RANGE);
      // transposed forward matrices [previous][next]: the lanes of a unit read consecutive next states
      const R *ta = (const R *)p.BfT[0] + (size_t)g * p.Bstride[0] + (size_t)ua * NA * p.np[0] + asafe;
      const R *tb = (const R *)p.BfT[1] + (size_t)g * p.Bstride[1] + (size_t)ub * NB * p.np[1] + bsafe;
      const R *tc = (const R *)p.BfT[2] + (size_t)g * p.Bstride[2] + (size_t)uc * NC * p.np[2] + csafe;
      lpa = bi_log_inline(bi_max(col_dot<R, NA>(ta, p.np[0], sq), (R)BI_EPS));
      lpb = bi_log_inline(bi_max(col_dot<R, NB>(tb, p.np[1], sq + NA), (R)BI_EPS));
      lpc = bi_log_inline(bi_max(col_dot<R, NC>(tc, p.np[2], sq + NA + NB), (R)BI_EPS));
    }
    __syncwarp();

    t3.set_uniform();
    R xa = 0, xb = 0, xc = 0;
    R pxa = 0, pxb = 0, pxc = 0;   // previous iterate's logits (the uniform start: a constant, taken as 0)
    const R lam = (R)p.lambda, oml = (R)1 - lam;
    // za: sum of the current iterate's e_a over the unit; with the transpose
    // area in use every lane holds all e_a (read back from shared memory) and
    // sums them itself, otherwise the lanes sum theirs with shuffles
    R eav[TT::TP ? NAP : 1];
#pragma unroll
    for (int r = 0; r < (TT::TP ? NAP : 1); ++r) eav[r] = r < NA ? (R)1 : (R)0;
    R za_sh = (R)NA;
    // softmax shifts in use
    float ma = STALE ? group_max_f<NAP, SB>(a_ok ? (float)lpa : -CUDART_INF_F) : 0.f;
    float mb = STALE ? group_max_f<LPU, 1>(b_ok ? (float)lpb : -CUDART_INF_F) : 0.f;
    float mc = STALE ? group_max_f<LPU, 1>(c_ok ? (float)lpc : -CUDART_INF_F) : 0.f;
    for (int k = 0; k < p.K; ++k) {
      // The normalisers of the current iterate head the loop body, in one
      // straight-line block with the contraction: their reciprocal is needed
      // only when the messages are scaled, so its dependency chain runs under
      // the contraction's multiply-adds instead of ahead of them.
      {
        const R za = TT::TP ? tree_sum<R, TT::TP ? NAP : 1>(eav) : za_sh;
        const R zb = group_sum<R, SB, 1>(tree_sum<R, NBL>(t3.eb));
        const R zc = tree_sum<R, NCP>(t3.ec);
        const R rinv = bi_rcp(za * zb * zc);
        t3.sa = rinv * za;
        t3.sb = rinv * zb;
        t3.sc = rinv * zc;
      }
      if (LSMEM) t3.messages_smem(sm_L[LSMEM ? unit : 0], xa, xb, xc, TT::TP ? eav : nullptr);
      else t3.messages(xa, xb, xc, TT::TP ? eav : nullptr);
      xa = a_ok ? xa + lpa : -bi_inf<R>();
      xb = b_ok ? xb + lpb : -bi_inf<R>();
      xc = c_ok ? xc + lpc : -bi_inf<R>();
      if (DAMPED) {   // damped step on the logits (a shift per factor does not matter)
        xa = a_ok ? fma(lam, xa, oml * pxa) : xa;
        xb = b_ok ? fma(lam, xb, oml * pxb) : xb;
        xc = c_ok ? fma(lam, xc, oml * pxc) : xc;
        pxa = a_ok ? xa : (R)0; pxb = b_ok ? xb : (R)0; pxc = c_ok ? xc : (R)0;
      }
      // Softmax is invariant to the shift; any shift that keeps the exponents
      // in range is exact.  With STALE the shift is the previous iterate's
      // maximum (the prior's maximum at the first iterate: the likelihood
      // message is <= 0 and bounded below by nmem * ln(1e-16)), so the max
      // reduction sits after the exponentials in program order and its
      // shuffles no longer delay them (a warp issues in order).
      if (!STALE) {
        ma = group_max_f<NAP, SB>((float)xa);
        mb = group_max_f<LPU, 1>((float)xb);
        mc = group_max_f<LPU, 1>((float)xc);
      }
      const R ean = a_ok ? bi_exp_tab(xa - (R)ma, exp_tab) : (R)0;
      const R ebn = b_ok ? bi_exp_tab(xb - (R)mb, exp_tab) : (R)0;
      const R ecn = c_ok ? bi_exp_tab(xc - (R)mc, exp_tab) : (R)0;
      if (t3.own_b) se[bi] = ebn;
      if (t3.own_c) se[NB + ci] = ecn;
      if (TT::TP && t3.own_a) se[NB + NCP + a] = ean;
      if (!TT::TP) za_sh = group_sum<R, NAP, SB>(ean);
      __syncwarp();
      t3.ea = ean;
#pragma unroll
      for (int bl = 0; bl < NBL; ++bl) t3.eb[bl] = se[t3.bh * NBL + bl];
#pragma unroll
      for (int c = 0; c < NCP; ++c) t3.ec[c] = se[NB + c];
      if (TT::TP) {
#pragma unroll
        for (int r = 0; r < NAP; ++r) eav[r] = se[NB + NCP + r];
      }
      if (STALE && k + 1 < p.K) {
        ma = group_max_f<NAP, SB>((float)xa);
        mb = group_max_f<LPU, 1>((float)xb);
        mc = group_max_f<LPU, 1>((float)xc);
      }
      __syncwarp();
    }
    // normalisers of the last iterate
    const R za = TT::TP ? tree_sum<R, TT::TP ? NAP : 1>(eav) : za_sh;
    const R zb = group_sum<R, SB, 1>(tree_sum<R, NBL>(t3.eb));
    const R zc = tree_sum<R, NCP>(t3.ec);
    const R rinv = bi_rcp(za * zb * zc);

    // ---- final beliefs of the step: outputs, and the next step's prior input
    const R qa = t3.ea * (rinv * zb * zc);
    const R qb = (b_ok ? se[bsafe] : (R)0) * (rinv * za * zc);
    const R qc = (c_ok ? se[NB + csafe] : (R)0) * (rinv * za * zb);
    if (t3.own_a) sq[a] = qa;
    if (t3.own_b) sq[NA + bi] = qb;
    if (t3.own_c) sq[NA + NB + ci] = qc;
    float *qo = p.q_out + (out_base + t) * p.S;
    if (live) {
      if (t3.own_a) qo[p.off[0] + a] = (float)qa;
      if (t3.own_b) qo[p.off[1] + bi] = (float)qb;
      if (t3.own_c) qo[p.off[2] + ci] = (float)qc;
      if (p.carry_out && t == p.T - 1) {
        R *co = (R *)p.carry_out + (size_t)agent * p.S;
        if (t3.own_a) co[p.off[0] + a] = qa;
        if (t3.own_b) co[p.off[1] + bi] = qb;
        if (t3.own_c) co[p.off[2] + ci] = qc;
      }
      if (p.logq_out) {
        float *lo = p.logq_out + (out_base + t) * p.S;
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
        int32_t *ao = p.argmax_out + (out_base + t) * 3;
        ao[p.fac[0]] = ia;
        ao[p.fac[1]] = ib;
        ao[p.fac[2]] = ic;
      }
    }
    __syncwarp();
  }
}

template <typename R, int NA, int NB, int NC, int SB, bool LSMEM, bool DAMPED>
int launch_filter(const Tile3Params &p, cudaStream_t stream) {
  using TT = Tile3<R, NA, NB, NC, SB>;
  const int grid = (p.N + TT::UPW - 1) / TT::UPW;
  // shifts may lag one iterate only where the exponent range has room for the
  // largest possible move of a logit: float64 and at most 12 modalities
  if (DAMPED)
    bi_tile3_filter_kernel<R, NA, NB, NC, SB, LSMEM, false, true><<<grid, 32, 0, stream>>>(p);
  else if (sizeof(R) == 8 && p.nmem <= 12)
    bi_tile3_filter_kernel<R, NA, NB, NC, SB, LSMEM, true, false><<<grid, 32, 0, stream>>>(p);
  else
    bi_tile3_filter_kernel<R, NA, NB, NC, SB, LSMEM, false, false><<<grid, 32, 0, stream>>>(p);
  return cudaGetLastError() == cudaSuccess ? BI_OK : BI_ERR_CUDA;
}

template <typename R, bool DAMPED>
int dispatch_filter(const Tile3Params &p, int na, int nb, int nc, cudaStream_t stream) {
#define X(A, B, C, S, LS) \
  if (na == A && nb == B && nc == C) return launch_filter<R, A, B, C, S, LS, DAMPED>(p, stream);
  BI_TILE3_SHAPES(X)
#undef X
  return BI_ERR_UNSUPPORTED;
}


}  // namespace tile3_filter
