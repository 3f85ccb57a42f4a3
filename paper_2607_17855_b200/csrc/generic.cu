// Generic kernels: any model within the BI_MAX_* limits, any of the three
// algorithms, either arithmetic.  One CTA per agent; the whole time recursion /
// window and the whole iteration loop run inside one launch (the launch
// overhead of looping small contractions is one of the costs Section III-C
// names).
//
// Likelihood messages (Section IV, marginalisation): a dependency group's
// summed slice L[s_0..s_{k-1}] is contracted one axis at a time, last axis
// first.  A level with leading multi-index r and last index c computes
//   V[r]       = sum_c L[r,c] q_last[c]                (input of the next level)
//   ell_last[c] += (prod_j q_j[r_j]) * L[r,c]          (message to the last axis)
// so all k messages cost about 2 P multiply-adds instead of k P.
#include "bi_internal.h"
#include "bi_device.cuh"

namespace {

struct GenSmem {  // element offsets (units of R) into dynamic shared memory
  int q0, q1, lpri, ell, Lst, V0, V1, red, obs, total_bytes;
  int xp;      // damped calls: previous logits, Tq steps; -1 otherwise
  int Tq;      // belief steps kept (1 for filtering, T for windows)
  int staged;  // summed slices staged in shared memory
};

// Sum over a group's members of their slices for the observed outcomes.
template <typename R>
struct GlobalSliceLoader {
  const R *ptr[BI_MAX_M];
  int nmem, npad;
  __device__ __forceinline__ Vec4<R> operator()(int r, int c4) const {
    Vec4<R> acc = ldg4(ptr[0] + (size_t)r * npad + 4 * c4);
    for (int i = 1; i < nmem; ++i) {
      Vec4<R> x = ldg4(ptr[i] + (size_t)r * npad + 4 * c4);
      acc.x += x.x; acc.y += x.y; acc.z += x.z; acc.w += x.w;
    }
    return acc;
  }
};
template <typename R>
struct SmemLoader {
  const R *base;
  int npad;
  __device__ __forceinline__ Vec4<R> operator()(int r, int c4) const {
    return *reinterpret_cast<const Vec4<R> *>(base + r * npad + 4 * c4);
  }
};

// Adds acc[c], summed over the CTA, to dst[c] for c < n.  Fixed order: the
// result does not depend on scheduling.
template <typename R>
__device__ __forceinline__ void block_accumulate(const R (&acc)[32], int n, R *dst, R *red,
                                                 bool warp_has_rows, int nwarps_with_rows) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  if (warp_has_rows) {
#pragma unroll
    for (int c = 0; c < 32; ++c) {
      if (c < n) {
        R s = warp_sum(acc[c]);
        if (lane == 0) red[warp * 32 + c] = s;
      }
    }
  }
  __syncthreads();
  if ((int)threadIdx.x < n) {
    R s = dst[threadIdx.x];
    for (int w = 0; w < nwarps_with_rows; ++w) s += red[w * 32 + threadIdx.x];
    dst[threadIdx.x] = s;
  }
  __syncthreads();
}

template <typename R, class LD>
__device__ __forceinline__ void peel_level(const BiLevel &lv, const LD &ld, const R *qt, R *Vout,
                                           R *ell, R *red) {
  R acc[32];
#pragma unroll
  for (int c = 0; c < 32; ++c) acc[c] = (R)0;
  const int NT = blockDim.x;
  const int npad4 = lv.last_npad4;
  const Vec4<R> *q4 = reinterpret_cast<const Vec4<R> *>(qt + lv.last_qoff);
  const int ndig = lv.ndig;
  for (int r = threadIdx.x; r < lv.nrows; r += NT) {
    uint32_t rem = (uint32_t)r;
    R w = (R)1;
    int lastdig = 0, hi = 0;
#pragma unroll
    for (int i = 3; i >= 0; --i) {
      if (i < ndig) {
        uint32_t qd = __umulhi(rem, lv.magic[i]);
        int dg = (int)(rem - qd * (uint32_t)lv.dim[i]);
        rem = qd;
        w *= qt[lv.qoff[i] + dg];
        if (i == ndig - 1) { lastdig = dg; hi = (int)qd; }
      }
    }
    R v = (R)0;
#pragma unroll
    for (int c4 = 0; c4 < 8; ++c4) {
      if (c4 < npad4) {
        Vec4<R> x = ld(r, c4);
        Vec4<R> qq = q4[c4];
        v = fma(x.x, qq.x, v); v = fma(x.y, qq.y, v);
        v = fma(x.z, qq.z, v); v = fma(x.w, qq.w, v);
        acc[4 * c4 + 0] = fma(w, x.x, acc[4 * c4 + 0]);
        acc[4 * c4 + 1] = fma(w, x.y, acc[4 * c4 + 1]);
        acc[4 * c4 + 2] = fma(w, x.z, acc[4 * c4 + 2]);
        acc[4 * c4 + 3] = fma(w, x.w, acc[4 * c4 + 3]);
      }
    }
    Vout[hi * lv.out_npad + lastdig] = v;
  }
  const int warp = threadIdx.x >> 5;
  const int nwr = min((lv.nrows + 31) >> 5, (int)(blockDim.x >> 5));
  block_accumulate(acc, lv.last_n, ell + lv.last_qoff, red, warp < nwr, nwr);
}

// All likelihood messages of one group at one time step, added into ell.
template <typename R, class LD>
__device__ __forceinline__ void contract_group(const BiGroup &g, const LD &first, const R *qt, R *ell,
                                               R *V0, R *V1, R *red) {
  if (g.rank == 1) {
    if ((int)threadIdx.x < g.first_n) {
      // rank-1 slice: it is the message itself
      Vec4<R> x = first(0, threadIdx.x >> 2);
      const int k = threadIdx.x & 3;
      R xv = k == 0 ? x.x : k == 1 ? x.y : k == 2 ? x.z : x.w;
      ell[g.first_qoff + threadIdx.x] += xv;
    }
    __syncthreads();
    return;
  }
  peel_level<R>(g.lev[0], first, qt, V0, ell, red);
  R *vin = V0, *vout = V1;
  for (int l = 1; l + 1 < g.rank; ++l) {
    SmemLoader<R> sl{vin, g.lev[l].last_npad4 * 4};
    peel_level<R>(g.lev[l], sl, qt, vout, ell, red);
    R *t = vin; vin = vout; vout = t;
  }
  if ((int)threadIdx.x < g.first_n) ell[g.first_qoff + threadIdx.x] += vin[threadIdx.x];
  __syncthreads();
}

// softmax of every factor of one step: x = ell (already holding all messages);
// writes the next beliefs (padded layout) and, if final, the outputs.
template <typename R>
__device__ __forceinline__ void softmax_step(const BiDev &md, const R *ell, R *qn, bool final,
                                             float *q_out, float *logq_out, int32_t *argmax_out,
                                             R *xp = nullptr, R lam = (R)1) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = blockDim.x >> 5;
  for (int f = warp; f < md.F; f += nw) {
    const int n = md.n[f], op = md.offp[f];
    R x = lane < n ? ell[op + lane] : -bi_inf<R>();
    if (xp && lane < n) {   // damped step on the logits; xp: the previous iterate's
      x = fma(lam, x, ((R)1 - lam) * xp[op + lane]);
      xp[op + lane] = x;
    }
    R mx = warp_max(x);
    R e = lane < n ? bi_exp(x - mx) : (R)0;
    R z = warp_sum(e);
    R q = e / z;
    if (lane < md.npad[f]) qn[op + lane] = lane < n ? q : (R)0;
    if (final) {
      if (lane < n) {
        q_out[md.off[f] + lane] = (float)q;
        if (logq_out) logq_out[md.off[f] + lane] = (float)(x - mx - bi_log(z));
      }
      if (argmax_out) {
        unsigned b = __ballot_sync(0xffffffffu, lane < n && x == mx);
        if (lane == 0) argmax_out[f] = __ffs(b) - 1;
      }
    }
  }
}

template <typename R>
__device__ __forceinline__ void set_uniform(const BiDev &md, R *q, int count_steps) {
  for (int idx = threadIdx.x; idx < count_steps * md.Sp; idx += blockDim.x) {
    int p = idx % md.Sp, f = 0;
    while (f + 1 < md.F && p >= md.offp[f + 1]) ++f;
    q[idx] = (p - md.offp[f]) < md.n[f] ? (R)1 / (R)md.n[f] : (R)0;
  }
}

template <typename R>
__device__ __forceinline__ void stage_step(const BiDev &md, int g, const int32_t *obs_t, R *dst) {
  for (int gi = 0; gi < md.ngroups; ++gi) {
    const BiGroup &gr = md.grp[gi];
    for (int e = threadIdx.x; e < gr.P_pad; e += blockDim.x) {
      R v = (R)0;
      for (int mi = gr.mem_begin; mi < gr.mem_end; ++mi) {
        const BiMember &mm = md.mem[mi];
        v += __ldg((const R *)mm.logA + (size_t)g * mm.gstride + (size_t)obs_t[mm.modality] * mm.P_pad + e);
      }
      dst[gr.L_off + e] = v;
    }
  }
}

template <typename R, bool STAGED>
__device__ __forceinline__ void all_groups(const BiDev &md, int g, const int32_t *obs_t, const R *Lst_t,
                                           const R *qt, R *ell, R *V0, R *V1, R *red) {
  for (int gi = 0; gi < md.ngroups; ++gi) {
    const BiGroup &gr = md.grp[gi];
    const int npad = gr.rank > 1 ? gr.lev[0].last_npad4 * 4 : bi_pad4(gr.first_n);
    if (STAGED) {
      SmemLoader<R> ld{Lst_t + gr.L_off, npad};
      contract_group<R>(gr, ld, qt, ell, V0, V1, red);
    } else {
      GlobalSliceLoader<R> ld;
      ld.nmem = gr.mem_end - gr.mem_begin;
      ld.npad = npad;
      for (int mi = gr.mem_begin; mi < gr.mem_end; ++mi) {
        const BiMember &mm = md.mem[mi];
        ld.ptr[mi - gr.mem_begin] =
            (const R *)mm.logA + (size_t)g * mm.gstride + (size_t)obs_t[mm.modality] * mm.P_pad;
      }
      contract_group<R>(gr, ld, qt, ell, V0, V1, red);
    }
  }
}

// ---- transition tensors with several parents (non-trivial B-dependencies) ----
// One warp per output value, lanes over the joint states of the parents; sums in a fixed order.
// X: the tensor's rows for one model and action, [n_f][PB]; q: one step's beliefs (padded layout).

// sum_{parents} X[s_next][parents] prod_j q_{parent_j}[s_j]
template <typename R>
__device__ R bdep_expect(const BiDev &md, int f, const R *__restrict__ Xrow, const R *q, int lane) {
  const int k = md.bdep_len[f], PB = md.PB[f];
  R acc = (R)0;
  for (int e = lane; e < PB; e += 32) {
    int rem = e;
    R w = (R)1;
    for (int j = k - 1; j >= 0; --j) {
      const int gq = md.bdep[f][j], nj = md.n[gq];
      const int d = rem % nj;
      rem /= nj;
      w *= q[md.offp[gq] + d];
    }
    acc = fma(Xrow[e], w, acc);
  }
  return warp_sum(acc);
}

// VMP future message to state s of factor f0 at a step: over every factor h whose transition reads f0,
// sum_{s'} qn_h[s'] sum_{parents with s_f0 = s} ln B_h[s'][parents] prod_{other parents} q[...];
// act_t: the actions taken at this step
template <typename R>
__device__ R bdep_future(const BiDev &md, int g, int f0, int s, const R *q, const R *qn,
                         const int32_t *__restrict__ act_t, int lane) {
  R acc = (R)0;
  for (int h = 0; h < md.F; ++h) {
    const int k = md.bdep_len[h];
    int pos = -1;
    for (int j = 0; j < k; ++j)
      if (md.bdep[h][j] == f0) pos = j;
    if (pos < 0) continue;
    const int nh = md.n[h], PB = md.PB[h];
    const int u = clamp_flag(act_t[h], md.U[h], md.status, BI_FLAG_ACT_RANGE);
    const R *X = (const R *)md.logBfull[h] + (size_t)g * md.Bfull_stride[h] + (size_t)u * nh * PB;
    const int others = PB / md.n[f0];
    for (int i = lane; i < nh * others; i += 32) {
      const int sn = i / others;
      int rem = i - sn * others, e = 0, stride = 1;
      R w = (R)1;
      for (int j = k - 1; j >= 0; --j) {
        const int gq = md.bdep[h][j], nj = md.n[gq];
        int d;
        if (j == pos) d = s;
        else {
          d = rem % nj;
          rem /= nj;
          w *= q[md.offp[gq] + d];
        }
        e += d * stride;
        stride *= nj;
      }
      acc = fma(qn[md.offp[h] + sn] * w, X[(size_t)sn * PB + e], acc);
    }
  }
  return warp_sum(acc);
}

template <typename R, int ALGO, bool STAGED>
__global__ void __launch_bounds__(256)
bi_generic_kernel(const BiDev *__restrict__ mdp, int N, int T, const int32_t *__restrict__ obs,
                  const int32_t *__restrict__ act, const float *q_prev, const int32_t *__restrict__ act_prev,
                  const void *carry_in, void *carry_out, const float *__restrict__ q_init, const void *__restrict__ lnprior, double lambda, int K,
                  float *q_out, float *__restrict__ logq_out, int32_t *__restrict__ argmax_out, GenSmem sm) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  R *smem = reinterpret_cast<R *>(smem_raw);
  const BiDev &md = *mdp;
  const int a = blockIdx.x;
  const int g = md.G == 1 ? 0 : a;
  const int tid = threadIdx.x, NT = blockDim.x;
  const int S = md.S, Sp = md.Sp, F = md.F, M = md.M;
  R *q0 = smem + sm.q0, *q1 = smem + sm.q1, *lpri = smem + sm.lpri, *ell = smem + sm.ell;
  R *xpb = sm.xp >= 0 ? smem + sm.xp : nullptr;   // previous logits (damped calls)
  R *Lst = smem + sm.Lst, *V0 = smem + sm.V0, *V1 = smem + sm.V1, *red = smem + sm.red;
  int32_t *obs_s = reinterpret_cast<int32_t *>(smem + sm.obs);

  // observed outcomes, clamped into range, for the whole call
  for (int i = tid; i < T * M; i += NT)
    obs_s[i] = clamp_flag(obs[(size_t)a * T * M + i], md.m[i % M], md.status, BI_FLAG_OBS_RANGE);
  for (int i = tid; i < 2 * sm.Tq * Sp; i += NT) q0[i] = (R)0;  // q0 and q1 are adjacent
  for (int i = tid; i < sm.red - sm.V0; i += NT) V0[i] = (R)0;  // V0 and V1 are adjacent
  __syncthreads();

  float *q_a = q_out + (size_t)a * T * S;
  float *lq_a = logq_out ? logq_out + (size_t)a * T * S : nullptr;
  int32_t *am_a = argmax_out ? argmax_out + (size_t)a * T * F : nullptr;

  if (ALGO == BI_ALGO_FILTER) {
    R *cur = q0, *nxt = q1;
    const bool from_prev = q_prev != nullptr || carry_in != nullptr;
    if (from_prev) {  // continued filtering: the belief of the step before the window
      for (int idx = tid; idx < Sp; idx += NT) {
        int f = 0;
        while (f + 1 < F && idx >= md.offp[f + 1]) ++f;
        const int s = idx - md.offp[f];
        const size_t src = (size_t)a * S + md.off[f] + s;
        cur[idx] = s < md.n[f] ? (carry_in ? ((const R *)carry_in)[src] : (R)q_prev[src]) : (R)0;
      }
      __syncthreads();
    }
    for (int t = 0; t < T; ++t) {
      // ln prior: D at the first step, else B_u q_{t-1} (cur still holds step t-1)
      if (md.has_bdep) {   // transition tensors with several parents: a warp per state
        for (int idx = tid >> 5; idx < Sp; idx += NT >> 5) {
          int f = 0;
          while (f + 1 < F && idx >= md.offp[f + 1]) ++f;
          const int s = idx - md.offp[f], n = md.n[f];
          R lp = (R)0;
          if (s < n) {
            if (t == 0 && !from_prev) {
              lp = ((const R *)md.logD[f])[(size_t)g * md.Dstride[f] + s];
            } else {
              const int ur = t == 0 ? act_prev[(size_t)a * F + f] : act[((size_t)a * (T - 1) + (t - 1)) * F + f];
              const int u = clamp_flag(ur, md.U[f], md.status, BI_FLAG_ACT_RANGE);
              const R *row = (const R *)md.Bfull[f] + (size_t)g * md.Bfull_stride[f] + ((size_t)u * n + s) * md.PB[f];
              lp = bi_log(bi_max(bdep_expect<R>(md, f, row, cur, tid & 31), (R)BI_EPS));
            }
          }
          if ((tid & 31) == 0) lpri[idx] = lp;
        }
      } else
      for (int idx = tid; idx < Sp; idx += NT) {
        int f = 0;
        while (f + 1 < F && idx >= md.offp[f + 1]) ++f;
        const int s = idx - md.offp[f], n = md.n[f];
        R lp = (R)0;
        if (s < n) {
          if (t == 0 && !from_prev) {
            lp = ((const R *)md.logD[f])[(size_t)g * md.Dstride[f] + s];
          } else {
            const int ur = t == 0 ? act_prev[(size_t)a * F + f] : act[((size_t)a * (T - 1) + (t - 1)) * F + f];
            int u = clamp_flag(ur, md.U[f], md.status, BI_FLAG_ACT_RANGE);
            const R *row = (const R *)md.Bf[f] + (size_t)g * md.Bstride[f] + ((size_t)u * n + s) * md.npad[f];
            R p = (R)0;
            for (int r = 0; r < n; ++r) p = fma(row[r], cur[md.offp[f] + r], p);
            lp = bi_log(bi_max(p, (R)BI_EPS));
          }
        }
        lpri[idx] = lp;
      }
      if (STAGED) stage_step<R>(md, g, obs_s + t * M, Lst);
      __syncthreads();
      set_uniform<R>(md, cur, 1);
      if (xpb)
        for (int idx = tid; idx < Sp; idx += NT) xpb[idx] = (R)0;   // logits of the uniform start: a constant
      __syncthreads();
      for (int k = 0; k < K; ++k) {
        for (int idx = tid; idx < Sp; idx += NT) ell[idx] = lpri[idx];
        __syncthreads();
        all_groups<R, STAGED>(md, g, obs_s + t * M, Lst, cur, ell, V0, V1, red);
        softmax_step<R>(md, ell, nxt, k == K - 1, q_a + (size_t)t * S, lq_a ? lq_a + (size_t)t * S : nullptr,
                        am_a ? am_a + (size_t)t * F : nullptr, xpb, (R)lambda);
        __syncthreads();
        R *tmp = cur; cur = nxt; nxt = tmp;
      }
    }
    if (carry_out) {   // the last step's belief at full precision, for a call that continues this one
      for (int idx = tid; idx < Sp; idx += NT) {
        int f = 0;
        while (f + 1 < F && idx >= md.offp[f + 1]) ++f;
        const int s = idx - md.offp[f];
        if (s < md.n[f]) ((R *)carry_out)[(size_t)a * S + md.off[f] + s] = cur[idx];
      }
    }
  } else {
    // ---- window algorithms: beliefs of all T steps, Jacobi over (t, f)
    R *cur = q0, *nxt = q1;
    set_uniform<R>(md, cur, T);
    if (q_init) {  // warm start: the given beliefs replace the uniform ones (pad entries stay zero)
      for (int idx = tid; idx < T * Sp; idx += NT) {
        int p = idx % Sp, f = 0;
        while (f + 1 < F && p >= md.offp[f + 1]) ++f;
        const int s = p - md.offp[f];
        if (s < md.n[f]) cur[idx] = (R)q_init[((size_t)a * T + idx / Sp) * S + md.off[f] + s];
      }
    }
    if (xpb) {   // damped calls start from the logarithms of the starting beliefs (uniform: a constant)
      __syncthreads();
      for (int idx = tid; idx < T * Sp; idx += NT) {
        int p = idx % Sp, f = 0;
        while (f + 1 < F && p >= md.offp[f + 1]) ++f;
        xpb[idx] = (q_init && p - md.offp[f] < md.n[f]) ? bi_log(bi_max(cur[idx], (R)BI_EPS)) : (R)0;
      }
    }
    if (STAGED)
      for (int t = 0; t < T; ++t) stage_step<R>(md, g, obs_s + t * M, Lst + (size_t)t * md.Ltot);
    __syncthreads();
    for (int k = 0; k < K; ++k) {
      for (int t = 0; t < T; ++t) {
        const R *qt = cur + t * Sp;
        // transition messages (Section IV: low-rank contractions of B with the
        // neighbouring steps' beliefs)
        if (md.has_bdep) {   // transition tensors with several parents (VMP only): a warp per state
          for (int idx = tid >> 5; idx < Sp; idx += NT >> 5) {
            int f = 0;
            while (f + 1 < F && idx >= md.offp[f + 1]) ++f;
            const int s = idx - md.offp[f], n = md.n[f];
            R msg = (R)0;
            if (s < n) {
              if (t == 0) {
                msg = ((const R *)md.logD[f])[(size_t)g * md.Dstride[f] + s];
              } else {
                const int u = clamp_flag(act[((size_t)a * (T - 1) + (t - 1)) * F + f], md.U[f], md.status, BI_FLAG_ACT_RANGE);
                const R *row = (const R *)md.logBfull[f] + (size_t)g * md.Bfull_stride[f] + ((size_t)u * n + s) * md.PB[f];
                msg = bdep_expect<R>(md, f, row, cur + (t - 1) * Sp, tid & 31);
              }
              if (t + 1 < T)
                msg += bdep_future<R>(md, g, f, s, qt, cur + (t + 1) * Sp, act + ((size_t)a * (T - 1) + t) * F, tid & 31);
            }
            if ((tid & 31) == 0) ell[idx] = msg;
          }
        } else
        for (int idx = tid; idx < Sp; idx += NT) {
          int f = 0;
          while (f + 1 < F && idx >= md.offp[f + 1]) ++f;
          const int s = idx - md.offp[f], n = md.n[f], np = md.npad[f];
          R msg = (R)0;
          if (s < n) {
            if (t == 0) {
              msg = lnprior ? ((const R *)lnprior)[(size_t)a * S + md.off[f] + s]
                            : ((const R *)md.logD[f])[(size_t)g * md.Dstride[f] + s];
            } else {
              int u = clamp_flag(act[((size_t)a * (T - 1) + (t - 1)) * F + f], md.U[f], md.status, BI_FLAG_ACT_RANGE);
              const R *qp = cur + (t - 1) * Sp + md.offp[f];
              size_t ro = (size_t)g * md.Bstride[f] + ((size_t)u * n + s) * np;
              const R *row = (ALGO == BI_ALGO_VMP ? (const R *)md.logB[f] : (const R *)md.Bf[f]) + ro;
              R p = (R)0;
              for (int r = 0; r < n; ++r) p = fma(row[r], qp[r], p);
              msg = ALGO == BI_ALGO_VMP ? p : (R)0.5 * bi_log(bi_max(p, (R)BI_EPS));
            }
            if (t + 1 < T) {
              int u = clamp_flag(act[((size_t)a * (T - 1) + t) * F + f], md.U[f], md.status, BI_FLAG_ACT_RANGE);
              const R *qn = cur + (t + 1) * Sp + md.offp[f];
              size_t ro = (size_t)g * md.Bstride[f] + ((size_t)u * n + s) * np;
              const R *row = (ALGO == BI_ALGO_VMP ? (const R *)md.logBt[f] : (const R *)md.Bdag[f]) + ro;
              R p = (R)0;
              for (int r = 0; r < n; ++r) p = fma(row[r], qn[r], p);
              msg += ALGO == BI_ALGO_VMP ? p : (R)0.5 * bi_log(bi_max(p, (R)BI_EPS));
            }
          }
          ell[idx] = msg;
        }
        __syncthreads();
        all_groups<R, STAGED>(md, g, obs_s + t * M, Lst + (size_t)t * md.Ltot, qt, ell, V0, V1, red);
        softmax_step<R>(md, ell, nxt + t * Sp, k == K - 1, q_a + (size_t)t * S,
                        lq_a ? lq_a + (size_t)t * S : nullptr, am_a ? am_a + (size_t)t * F : nullptr,
                        xpb ? xpb + t * Sp : nullptr, (R)lambda);
        __syncthreads();
      }
      R *tmp = cur; cur = nxt; nxt = tmp;
    }
  }
}

template <typename R>
int launch_generic_t(const BiCall &c, bi_model *mut) {
  const bi_model *md = c.model;
  const BiDev &h = md->h;
  const bool window = c.algo != BI_ALGO_FILTER;
  int NT = 32;
  while (NT < md->rows_max && NT < 256) NT <<= 1;
  const int nwarps = NT / 32;
  GenSmem sm;
  sm.Tq = window ? c.T : 1;
  int o = 0;
  sm.q0 = o; o += sm.Tq * h.Sp;
  sm.q1 = o; o += sm.Tq * h.Sp;
  sm.lpri = o; o += h.Sp;
  sm.ell = o; o += h.Sp;
  sm.V0 = o; o += bi_pad4(md->V0max);
  sm.V1 = o; o += bi_pad4(md->V1max);
  sm.red = o; o += nwarps * 32;
  sm.obs = o; o += bi_pad4(c.T * h.M + 1);
  sm.xp = c.lambda != 1.0 ? o : -1;
  if (c.lambda != 1.0) o += sm.Tq * h.Sp;
  const size_t budget = (size_t)md->max_smem_optin - 1024;
  const size_t stage = (size_t)(window ? c.T : 1) * h.Ltot;
  sm.staged = stage > 0 && ((size_t)o + stage) * sizeof(R) <= budget;
  sm.Lst = o;
  if (sm.staged) o += (int)stage;
  sm.total_bytes = (int)(o * sizeof(R));
  if ((size_t)sm.total_bytes > budget) return BI_ERR_UNSUPPORTED;

  using KernelT = void (*)(const BiDev *, int, int, const int32_t *, const int32_t *, const float *,
                           const int32_t *, const void *, void *, const float *, const void *, double, int, float *,
                           float *, int32_t *, GenSmem);
  KernelT kern = nullptr;
  const char *name = "";
  const bool f64 = sizeof(R) == 8;
  if (c.algo == BI_ALGO_FILTER) {
    kern = sm.staged ? bi_generic_kernel<R, BI_ALGO_FILTER, true> : bi_generic_kernel<R, BI_ALGO_FILTER, false>;
    name = f64 ? (sm.staged ? "generic_filter_staged_f64" : "generic_filter_global_f64")
               : (sm.staged ? "generic_filter_staged_f32" : "generic_filter_global_f32");
  } else if (c.algo == BI_ALGO_VMP) {
    kern = sm.staged ? bi_generic_kernel<R, BI_ALGO_VMP, true> : bi_generic_kernel<R, BI_ALGO_VMP, false>;
    name = f64 ? (sm.staged ? "generic_vmp_staged_f64" : "generic_vmp_global_f64")
               : (sm.staged ? "generic_vmp_staged_f32" : "generic_vmp_global_f32");
  } else {
    kern = sm.staged ? bi_generic_kernel<R, BI_ALGO_MMP, true> : bi_generic_kernel<R, BI_ALGO_MMP, false>;
    name = f64 ? (sm.staged ? "generic_mmp_staged_f64" : "generic_mmp_global_f64")
               : (sm.staged ? "generic_mmp_staged_f32" : "generic_mmp_global_f32");
  }
  if (cudaFuncSetAttribute((const void *)kern, cudaFuncAttributeMaxDynamicSharedMemorySize, sm.total_bytes) !=
      cudaSuccess)
    return BI_ERR_CUDA;
  kern<<<c.N, NT, sm.total_bytes, c.stream>>>(md->d, c.N, c.T, c.obs, c.act, c.q_prev, c.act_prev, c.carry_in,
                                               c.carry_out, c.q_init, c.lnprior, c.lambda, c.K, c.q_out, c.logq_out, c.argmax_out, sm);
  if (cudaGetLastError() != cudaSuccess) return BI_ERR_CUDA;
  mut->launches += 1;
  mut->last_kernel = name;
  return BI_OK;
}

}  // namespace

int bi_launch_generic(const BiCall &c, bi_model *mut) {
  return c.model->arith == BI_ARITH_F64 ? launch_generic_t<double>(c, mut) : launch_generic_t<float>(c, mut);
}
