// Variational filtering with one CTA per agent, for batches too small to fill
// the machine with one warp per agent and models whose groups do not fit a
// compiled tile.
//
// The time recursion and the iteration loop run inside one launch (Section
// III-C names the launch overhead of looping small contractions as a cost).
// Per step the summed slices of every dependency group are staged in shared
// memory once.  One Jacobi iteration (Section IV, marginalisation) is three
// phases with one CTA barrier after each:
//
//   A  the first contraction level of every group of rank 3 or more, its rows
//      dealt round all the CTA's threads: V[r] = sum_c L[r,c] q_last[c] for the next level, and the
//      per-warp partial sums of (prod_j q_j[r_j]) L[r,c] for the message to the
//      last axis;
//   B  one warp per group of rank 4 or more takes that group down to its last
//      two axes (these levels are small) and writes their messages to the
//      group's own message row;
//   C  one warp per factor: log-prior, the per-warp partial sums of the classes
//      that end in this factor, the messages from groups of rank 2 and 3 (what
//      is left of them is a matrix of at most 32 x 32 over their first two
//      axes: the factor's warp sums its rows or columns itself), rank-1 slices
//      and phase B's rows, all in a fixed order; softmax, next beliefs (and the
//      outputs after the last iteration).  What a factor adds up is a list of
//      operations over shared memory, built once per launch, so that an iteration
//      reads one 16-byte descriptor per operation instead of following the model's
//      description; float64 calls take the softmax of every iteration but the last
//      with the table-driven exponential and an integer reduction for the shift.
// Models without a group of rank 3 or more skip phase A, models without one of rank 4 or
// more phase B, each with its barrier.
//
// Sums are taken in a fixed order: results do not depend on scheduling.
#include <algorithm>
#include <cstdlib>

#include "bi_internal.h"
#include "tile3.cuh"
#include "tile3_filter_f64.cuh"

namespace {

struct CtaGeom {   // element offsets (units of R) into dynamic shared memory
  int desc, q0, q1, lpri, xp, ellg, part, obs;
  int Lst[BI_MAX_GROUPS];    // per group: its staged slice, rows `lstride` apart
  int lstride[BI_MAX_GROUPS];
  int V[BI_MAX_GROUPS][2];   // per group: the two buffers its levels alternate between
  int vtot_begin, vtot_end;  // the range holding every V buffer (zeroed once: pad columns stay zero)
  // Groups of rank >= 3 whose last axis is the same factor form a class: a thread adds their
  // column sums in registers and the warp reduces once per class.  order[] lists those groups
  // class by class; class c is order[cls_begin[c] .. cls_begin[c + 1]).
  int ncls, order[BI_MAX_GROUPS], cls_begin[BI_MAX_GROUPS + 1], cls_pv[BI_MAX_GROUPS];
  int row_start[BI_MAX_GROUPS];   // thread that takes the group's row 0 (rows go round the CTA's threads)
  int cls_wmask[BI_MAX_GROUPS];   // warps that hold rows of the class
  // what phase C adds up for factor f, as bit masks: classes whose last axis is f, groups of rank 2
  // or 3 whose first / second axis is f (a matrix contracted by the factor's own warp), rank-1
  // groups on f (the slice is the message), groups of rank >= 4 that contain f (finished by phase B)
  unsigned f_cls[BI_MAX_F], f_m0[BI_MAX_F], f_m1[BI_MAX_F], f_r1[BI_MAX_F], f_deep[BI_MAX_F];
  // the matrix over a group's first two axes that phase C contracts: a rank-2 group's staged slice, a
  // rank-3 group's first partial tensor; its offset, row stride and the level that describes it
  int mat_off[BI_MAX_GROUPS], mat_ls[BI_MAX_GROUPS], mat_lev[BI_MAX_GROUPS];
  int deep;                       // any group of rank >= 4: phase B and its barrier are needed
  int ops, maxops, nops, exptab;  // phase C's operation lists [F][maxops] (16 bytes each), their lengths, the exp table
  int prior_tps;                  // threads that share one state when the prior is formed (1, 2 or 4)
  int wpar, wpar_cap;             // models with several parents per transition: the parents' outer product of one factor
  int total_bytes;
};

template <typename R>
__device__ __forceinline__ Vec4<R> lds4(const R *p) {
  return *reinterpret_cast<const Vec4<R> *>(p);
}

// Rows r0, r0 + step, ... of one level: writes V, accumulates the column sums in acc.
template <typename R, int PV>
__device__ __forceinline__ void peel_rows(const BiLevel &lv, const R *L, int lstride, const R *qt, R *Vout,
                                          int ostride, int r0, int step, R (&acc)[PV]) {
  const int npad4 = lv.last_npad4, ndig = lv.ndig, nrows = lv.nrows;
  uint32_t magic[4], dim[4];
  const R *qd[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    magic[i] = i < ndig ? lv.magic[i] : 0u;
    dim[i] = i < ndig ? (uint32_t)lv.dim[i] : 1u;
    qd[i] = qt + (i < ndig ? lv.qoff[i] : 0);
  }
  const R *q4 = qt + lv.last_qoff;
  for (int r = r0; r < nrows; r += step) {
    uint32_t rem = (uint32_t)r;
    R w = (R)1;
    int lastdig = 0, hi = 0;
#pragma unroll
    for (int i = 3; i >= 0; --i) {
      if (i < ndig) {
        const uint32_t qq = __umulhi(rem, magic[i]);
        const int dg = (int)(rem - qq * dim[i]);
        rem = qq;
        w *= qd[i][dg];
        if (i == ndig - 1) { lastdig = dg; hi = (int)qq; }
      }
    }
    R v0 = (R)0, v1 = (R)0;
#pragma unroll
    for (int c4 = 0; c4 < PV / 4; ++c4) {
      if (c4 < npad4) {
        const Vec4<R> x = lds4(L + r * lstride + 4 * c4);
        const Vec4<R> qq = lds4(q4 + 4 * c4);
        v0 = fma(x.x, qq.x, v0); v1 = fma(x.y, qq.y, v1);
        v0 = fma(x.z, qq.z, v0); v1 = fma(x.w, qq.w, v1);
        acc[4 * c4 + 0] = fma(w, x.x, acc[4 * c4 + 0]);
        acc[4 * c4 + 1] = fma(w, x.y, acc[4 * c4 + 1]);
        acc[4 * c4 + 2] = fma(w, x.z, acc[4 * c4 + 2]);
        acc[4 * c4 + 3] = fma(w, x.w, acc[4 * c4 + 3]);
      }
    }
    Vout[hi * ostride + lastdig] = v0 + v1;
  }
}

// phase A for one class of groups: this thread's rows of their first levels; the warp's column sums go to part_w[c]
template <typename R, int PV>
__device__ __forceinline__ void first_levels(const BiDev &md, const CtaGeom &sm, int cls, R *smem, const R *qt,
                                             R *part_w, int lane) {
  R acc[PV];
#pragma unroll
  for (int c = 0; c < PV; ++c) acc[c] = (R)0;
  const int NT = blockDim.x;
  for (int i = sm.cls_begin[cls]; i < sm.cls_begin[cls + 1]; ++i) {
    const int gi = sm.order[i];
    const BiLevel &lv = md.grp[gi].lev[0];
    int r0 = (int)threadIdx.x - sm.row_start[gi];
    if (r0 < 0) r0 += NT;
    peel_rows<R, PV>(lv, smem + sm.Lst[gi], sm.lstride[gi], qt, smem + sm.V[gi][0], bi_row_stride(lv.out_npad, (int)sizeof(R)), r0, NT,
                     acc);
  }
  const R tot = reduce_scatter<R, PV, 32, 1>(acc, lane);
  constexpr int SH = 5 - Log2<PV>::v;
  if ((lane & ((1 << SH) - 1)) == 0) part_w[lane >> SH] = tot;
}

// phase B for one deeper level, by one warp: message entries are written (each level feeds another factor)
template <typename R, int PV>
__device__ __forceinline__ void deeper_level(const BiLevel &lv, const R *L, const R *qt, R *Vout, R *ell_g, int lane) {
  R acc[PV];
#pragma unroll
  for (int c = 0; c < PV; ++c) acc[c] = (R)0;
  peel_rows<R, PV>(lv, L, bi_row_stride(lv.last_npad4 * 4, (int)sizeof(R)), qt, Vout, bi_row_stride(lv.out_npad, (int)sizeof(R)), lane, 32, acc);
  const R tot = reduce_scatter<R, PV, 32, 1>(acc, lane);
  constexpr int SH = 5 - Log2<PV>::v;
  const int idx = lane >> SH;
  if ((lane & ((1 << SH) - 1)) == 0 && idx < lv.last_n) ell_g[lv.last_qoff + idx] = tot;
  __syncwarp();
}

// The last level of a group, by one warp: a matrix L[r][c] over the group's first two axes (at most
// 32 x 32).  Both of its results are plain loops, one lane per row and one lane per column, with no
// cross-lane sums: vec[r] = sum_c L[r][c] q1[c] (the message to the first axis) and
// msg[c] = sum_r q0[r] L[r][c] (the message to the second).
template <typename R>
__device__ __forceinline__ void last_level(const BiLevel &lv, const R *L, const R *qt, R *ell_g, int first_qoff,
                                           int lane) {
  const int lstride = bi_row_stride(lv.last_npad4 * 4, (int)sizeof(R));
  const int nrows = lv.nrows, npad4 = lv.last_npad4, n1 = lv.last_n;
  const R *q0 = qt + lv.qoff[0], *q1 = qt + lv.last_qoff;
  if (lane < nrows) {
    R v0 = (R)0, v1 = (R)0;
    for (int c4 = 0; c4 < npad4; ++c4) {
      const Vec4<R> x = lds4(L + lane * lstride + 4 * c4);
      const Vec4<R> qq = lds4(q1 + 4 * c4);
      v0 = fma(x.x, qq.x, v0); v1 = fma(x.y, qq.y, v1);
      v0 = fma(x.z, qq.z, v0); v1 = fma(x.w, qq.w, v1);
    }
    ell_g[first_qoff + lane] = v0 + v1;
  }
  if (lane < n1) {
    R m0 = (R)0, m1 = (R)0;
    int r = 0;
    for (; r + 1 < nrows; r += 2) {
      m0 = fma(q0[r], L[r * lstride + lane], m0);
      m1 = fma(q0[r + 1], L[(r + 1) * lstride + lane], m1);
    }
    if (r < nrows) m0 = fma(q0[r], L[r * lstride + lane], m0);
    ell_g[lv.last_qoff + lane] = m0 + m1;
  }
  __syncwarp();
}

// Phase C's operations.  ROW: this lane's row of a matrix against a belief vector, sum_c L[lane][c] q[c]
// (count = padded columns / 4); COL: this lane's column, sum_r q[r] L[r][lane] (count = rows); ADD:
// sum_i base[i * stride + lane] (count terms: per-warp partial sums, a rank-1 slice, phase B's row).
enum { CTA_OP_ROW = 0, CTA_OP_COL = 1, CTA_OP_ADD = 2 };

template <typename R>
__device__ __forceinline__ R op_row_dot(const R *row, const R *q, int npad4) {
  R v0 = (R)0, v1 = (R)0, v2 = (R)0, v3 = (R)0;
  int c4 = 0;
  for (; c4 + 1 < npad4; c4 += 2) {   // loads of two vectors first, then four independent chains
    const Vec4<R> x = lds4(row + 4 * c4), y = lds4(row + 4 * c4 + 4);
    const Vec4<R> qx = lds4(q + 4 * c4), qy = lds4(q + 4 * c4 + 4);
    v0 = fma(x.x, qx.x, v0); v1 = fma(x.y, qx.y, v1); v2 = fma(x.z, qx.z, v2); v3 = fma(x.w, qx.w, v3);
    v0 = fma(y.x, qy.x, v0); v1 = fma(y.y, qy.y, v1); v2 = fma(y.z, qy.z, v2); v3 = fma(y.w, qy.w, v3);
  }
  if (c4 < npad4) {
    const Vec4<R> x = lds4(row + 4 * c4);
    const Vec4<R> qx = lds4(q + 4 * c4);
    v0 = fma(x.x, qx.x, v0); v1 = fma(x.y, qx.y, v1); v2 = fma(x.z, qx.z, v2); v3 = fma(x.w, qx.w, v3);
  }
  return (v0 + v1) + (v2 + v3);
}
template <typename R>
__device__ __forceinline__ R op_col_dot(const R *col, int ls, const R *q, int nrows) {
  R m0 = (R)0, m1 = (R)0, m2 = (R)0, m3 = (R)0;
  int r = 0;
  for (; r + 3 < nrows; r += 4) {
    const Vec4<R> w = lds4(q + r);
    const R a = col[r * ls], b = col[(r + 1) * ls], c = col[(r + 2) * ls], d = col[(r + 3) * ls];
    m0 = fma(w.x, a, m0); m1 = fma(w.y, b, m1); m2 = fma(w.z, c, m2); m3 = fma(w.w, d, m3);
  }
  for (; r < nrows; ++r) m0 = fma(q[r], col[r * ls], m0);
  return (m0 + m1) + (m2 + m3);
}

// sum over the warp of values that are zero in lanes n and above
template <typename R>
__device__ __forceinline__ R warp_sum_first(R v, int n) {
  if (n > 16) v += __shfl_xor_sync(0xffffffffu, v, 16);
  if (n > 8) v += __shfl_xor_sync(0xffffffffu, v, 8);
  if (n > 4) v += __shfl_xor_sync(0xffffffffu, v, 4);
  v += __shfl_xor_sync(0xffffffffu, v, 2);
  v += __shfl_xor_sync(0xffffffffu, v, 1);
  return v;
}

// Non-trivial B-dependencies (a transition that reads several factors' previous states): the prior of
// state s_next is sum_{parents} X[s_next][parents] prod_j q_{parent_j}[s_j], summed by a warp in a fixed
// order.  It is the only place where such a model differs from a plain one in filtering: the prior is
// formed once per step, outside the iteration.
template <typename R>
__device__ R cta_bdep_expect(const BiDev &md, int f, const R *__restrict__ Xrow, const R *q, int lane) {
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
    acc = fma(__ldg(Xrow + e), w, acc);
  }
  return warp_sum(acc);
}

template <typename R>
__global__ void __launch_bounds__(256, 2)
bi_cta_filter_kernel(const BiDev *__restrict__ mdp, int T, const int32_t *__restrict__ obs,
                     const int32_t *__restrict__ act, const float *q_prev,
                     const int32_t *__restrict__ act_prev, const void *carry_in, void *carry_out, double lambda,
                     int K, float *q_out, float *__restrict__ logq_out, int32_t *__restrict__ argmax_out,
                     const CtaGeom sm) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  R *smem = reinterpret_cast<R *>(smem_raw);
  {  // the model's description, read from shared memory from here on
    const int4 *s = reinterpret_cast<const int4 *>(mdp);
    int4 *d = reinterpret_cast<int4 *>(smem + sm.desc);
    for (int i = threadIdx.x; i < (int)(sizeof(BiDev) / sizeof(int4)); i += blockDim.x) d[i] = __ldg(s + i);
    __syncthreads();
  }
  const BiDev &md = *reinterpret_cast<const BiDev *>(smem + sm.desc);
  const int a = blockIdx.x, g = md.G == 1 ? 0 : a;
  const int tid = threadIdx.x, NT = blockDim.x, lane = tid & 31, warp = tid >> 5, NW = NT >> 5;
  const int S = md.S, Sp = md.Sp, F = md.F, M = md.M, NG = md.ngroups;
  R *cur = smem + sm.q0, *nxt = smem + sm.q1, *lpri = smem + sm.lpri;
  R *xp = sm.xp >= 0 ? smem + sm.xp : nullptr;   // previous logits (damped calls)
  R *ellg = smem + sm.ellg;                      // [NG][Sp] the groups' messages
  R *part = smem + sm.part;                      // [classes][NW][32] per-warp column sums of the first levels
  int32_t *obs_s = reinterpret_cast<int32_t *>(smem + sm.obs);
  const R lam = (R)lambda;

  for (int i = tid; i < T * M; i += NT)
    obs_s[i] = clamp_flag(__ldg(obs + (size_t)a * T * M + i), md.m[i % M], md.status, BI_FLAG_OBS_RANGE);
  for (int i = tid; i < 2 * Sp; i += NT) cur[i] = (R)0;   // q0 and q1 are adjacent
  for (int i = tid; i < NG * Sp; i += NT) ellg[i] = (R)0;  // entries of factors outside a group stay zero
  for (int i = sm.vtot_begin + tid; i < sm.vtot_end; i += NT) smem[i] = (R)0;
  int4 *ops = reinterpret_cast<int4 *>(smem + sm.ops);     // [F][maxops]
  int32_t *nops = reinterpret_cast<int32_t *>(smem + sm.nops);
  if (tid < F) {   // what phase C adds up for factor tid, in the order it is added
    const int f = tid;
    int4 *o = ops + f * sm.maxops;
    int c = 0;
    for (unsigned mk = sm.f_cls[f]; mk; mk &= mk - 1) {   // per-warp partial sums: one operation per run of warps
      const int cls = __ffs(mk) - 1;
      const unsigned wm = (unsigned)sm.cls_wmask[cls];
      for (int w = 0; w < NW;) {
        if (!((wm >> w) & 1)) { ++w; continue; }
        int e = w;
        while (e < NW && ((wm >> e) & 1)) ++e;
        o[c++] = make_int4(CTA_OP_ADD | ((e - w) << 8), sm.part + (cls * NW + w) * 32, 32, 0);
        w = e;
      }
    }
    for (unsigned mk = sm.f_m0[f]; mk; mk &= mk - 1) {   // groups of rank 2 or 3 with f as first axis
      const int gi = __ffs(mk) - 1;
      const BiLevel &lv = md.grp[gi].lev[sm.mat_lev[gi]];
      o[c++] = make_int4(CTA_OP_ROW | (lv.last_npad4 << 8), sm.mat_off[gi], sm.mat_ls[gi], lv.last_qoff);
    }
    for (unsigned mk = sm.f_m1[f]; mk; mk &= mk - 1) {   // ... and as second axis
      const int gi = __ffs(mk) - 1;
      const BiLevel &lv = md.grp[gi].lev[sm.mat_lev[gi]];
      o[c++] = make_int4(CTA_OP_COL | (lv.nrows << 8), sm.mat_off[gi], sm.mat_ls[gi], lv.qoff[0]);
    }
    for (unsigned mk = sm.f_r1[f]; mk; mk &= mk - 1) o[c++] = make_int4(CTA_OP_ADD | (1 << 8), sm.Lst[__ffs(mk) - 1], 0, 0);
    for (unsigned mk = sm.f_deep[f]; mk; mk &= mk - 1)
      o[c++] = make_int4(CTA_OP_ADD | (1 << 8), sm.ellg + (__ffs(mk) - 1) * Sp + md.offp[f], 0, 0);
    nops[f] = c;
  }
  const double *exp_tab = nullptr;
  if constexpr (sizeof(R) == 8) {
    double *tab = reinterpret_cast<double *>(smem + sm.exptab);
    for (int j = tid; j < tile3_f64::EXP_TAB; j += NT) tab[j] = exp2((double)j * (1.0 / tile3_f64::EXP_TAB));
    exp_tab = tab;
  }
  __syncthreads();
  const bool from_prev = q_prev != nullptr || carry_in != nullptr;
  if (from_prev) {  // continued filtering: the belief of the step before the first
    for (int idx = tid; idx < Sp; idx += NT) {
      int f = 0;
      while (f + 1 < F && idx >= md.offp[f + 1]) ++f;
      const int s = idx - md.offp[f];
      const size_t src = (size_t)a * S + md.off[f] + s;
      cur[idx] = s < md.n[f] ? (carry_in ? ((const R *)carry_in)[src] : (R)q_prev[src]) : (R)0;   // (q_prev may alias q_out: plain load)
    }
    __syncthreads();
  }

  for (int t = 0; t < T; ++t) {
    // ln prior: D at the first step, else B_u q_{t-1} (cur still holds step t-1)
    if (md.has_bdep && (t > 0 || from_prev)) {
      // The expectation of the transition tensor under the parents' beliefs.  The parents' outer product
      // is the same for every next state of a factor: formed once per factor in shared memory (when it
      // fits), then a warp per state sums its row against it, lane by lane in a fixed order.
      R *wpar = smem + sm.wpar;
      for (int f = 0; f < F; ++f) {
        const int n = md.n[f], PB = md.PB[f], k = md.bdep_len[f];
        const int ur = t == 0 ? __ldg(act_prev + (size_t)a * F + f) : __ldg(act + ((size_t)a * (T - 1) + (t - 1)) * F + f);
        const int u = clamp_flag(ur, md.U[f], md.status, BI_FLAG_ACT_RANGE);
        const R *Xu = (const R *)md.Bfull[f] + (size_t)g * md.Bfull_stride[f] + (size_t)u * n * PB;
        const bool shared_w = PB <= sm.wpar_cap;
        if (shared_w) {
          for (int e = tid; e < PB; e += NT) {
            int rem = e;
            R w = (R)1;
            for (int j = k - 1; j >= 0; --j) {
              const int gq = md.bdep[f][j], nj = md.n[gq];
              const int d = rem % nj;
              rem /= nj;
              w *= cur[md.offp[gq] + d];
            }
            wpar[e] = w;
          }
          __syncthreads();
        }
        for (int s = warp; s < n; s += NW) {
          const R *row = Xu + (size_t)s * PB;
          R ex;
          if (shared_w) {
            R acc = (R)0;
            int e = lane;
            for (; e + 96 < PB; e += 128) {   // four loads in flight, one accumulator: the order of the plain loop
              const R x0 = __ldg(row + e), x1 = __ldg(row + e + 32), x2 = __ldg(row + e + 64), x3 = __ldg(row + e + 96);
              acc = fma(x0, wpar[e], acc);
              acc = fma(x1, wpar[e + 32], acc);
              acc = fma(x2, wpar[e + 64], acc);
              acc = fma(x3, wpar[e + 96], acc);
            }
            for (; e < PB; e += 32) acc = fma(__ldg(row + e), wpar[e], acc);
            ex = warp_sum(acc);
          } else {
            ex = cta_bdep_expect<R>(md, f, row, cur, lane);
          }
          if (lane == 0) lpri[md.offp[f] + s] = bi_log(bi_max(ex, (R)BI_EPS));
        }
        for (int s = n + tid; s < md.npad[f]; s += NT) lpri[md.offp[f] + s] = (R)0;
        if (shared_w) __syncthreads();   // (the next factor overwrites the product)
      }
    } else if (t == 0 && !from_prev) {
      for (int idx = tid; idx < Sp; idx += NT) {
        int f = 0;
        while (f + 1 < F && idx >= md.offp[f + 1]) ++f;
        const int s = idx - md.offp[f];
        lpri[idx] = s < md.n[f] ? __ldg((const R *)md.logD[f] + (size_t)g * md.Dstride[f] + s) : (R)0;
      }
    } else {
      // tps threads of one warp share a state: each takes every tps-th term of the row's product with
      // the previous belief (its loads are all in flight together), then the partial sums are added
      const int tps = sm.prior_tps, per = NT / tps, sub = tid % tps;
      for (int base = 0; base < Sp; base += per) {
        const int idx = base + tid / tps;
        int f = 0;
        while (f + 1 < F && idx >= md.offp[f + 1]) ++f;
        const int s = idx - md.offp[f], n = md.n[f];
        const bool live = idx < Sp && s < n;
        R p0 = (R)0, p1 = (R)0;
        if (live) {
          const int ur = t == 0 ? __ldg(act_prev + (size_t)a * F + f)
                                : __ldg(act + ((size_t)a * (T - 1) + (t - 1)) * F + f);
          const int u = clamp_flag(ur, md.U[f], md.status, BI_FLAG_ACT_RANGE);
          const R *row = (const R *)md.Bf[f] + (size_t)g * md.Bstride[f] + ((size_t)u * n + s) * md.npad[f];
          const R *qf = cur + md.offp[f];
          int r = sub;
#pragma unroll 4
          for (; r + tps < n; r += 2 * tps) {
            p0 = fma(__ldg(row + r), qf[r], p0);
            p1 = fma(__ldg(row + r + tps), qf[r + tps], p1);
          }
          if (r < n) p0 = fma(__ldg(row + r), qf[r], p0);
        }
        R pr = p0 + p1;
        for (int d = 1; d < tps; d <<= 1) pr += __shfl_xor_sync(0xffffffffu, pr, d);
        if (idx < Sp && sub == 0) lpri[idx] = live ? bi_log(bi_max(pr, (R)BI_EPS)) : (R)0;
      }
    }
    // the step's summed slices, rows at their padded stride
    for (int gi = 0; gi < NG; ++gi) {
      const BiGroup &gr = md.grp[gi];
      const int nm = gr.mem_end - gr.mem_begin;
      const R *src[BI_MAX_M];
      for (int mi = 0; mi < nm; ++mi) {
        const BiMember &mm = md.mem[gr.mem_begin + mi];
        src[mi] = (const R *)mm.logA + (size_t)g * mm.gstride + (size_t)obs_s[t * M + mm.modality] * mm.P_pad;
      }
      const int npad4 = gr.rank > 1 ? gr.lev[0].last_npad4 : bi_pad4(gr.first_n) / 4;
      R *dst = smem + sm.Lst[gi];
      const int ls = sm.lstride[gi];
      for (int e4 = tid; e4 < gr.P_pad / 4; e4 += NT) {
        Vec4<R> v = ldg4(src[0] + 4 * e4);
        for (int mi = 1; mi < nm; ++mi) {
          const Vec4<R> x = ldg4(src[mi] + 4 * e4);
          v.x += x.x; v.y += x.y; v.z += x.z; v.w += x.w;
        }
        const int row = e4 / npad4, c4 = e4 - row * npad4;
        *reinterpret_cast<Vec4<R> *>(dst + row * ls + 4 * c4) = v;
      }
    }
    __syncthreads();
    // uniform start
    for (int idx = tid; idx < Sp; idx += NT) {
      int f = 0;
      while (f + 1 < F && idx >= md.offp[f + 1]) ++f;
      cur[idx] = (idx - md.offp[f]) < md.n[f] ? (R)1 / (R)md.n[f] : (R)0;
      if (xp) xp[idx] = (R)0;   // logits of the uniform start: a constant
    }
    __syncthreads();

    for (int k = 0; k < K; ++k) {
      // ---- A: first levels of the groups of rank >= 3, all threads
      for (int cls = 0; cls < sm.ncls; ++cls) {
        if (!((sm.cls_wmask[cls] >> warp) & 1)) continue;   // none of the class' rows fall to this warp
        R *pw = part + ((size_t)cls * NW + warp) * 32;
        switch (sm.cls_pv[cls]) {
          case 4: first_levels<R, 4>(md, sm, cls, smem, cur, pw, lane); break;
          case 8: first_levels<R, 8>(md, sm, cls, smem, cur, pw, lane); break;
          case 16: first_levels<R, 16>(md, sm, cls, smem, cur, pw, lane); break;
          default: first_levels<R, 32>(md, sm, cls, smem, cur, pw, lane); break;
        }
      }
      if (sm.ncls) __syncthreads();
      // ---- B: one warp per group of rank >= 4
      if (sm.deep) {
        for (int gi = warp; gi < NG; gi += NW) {
          const BiGroup &gr = md.grp[gi];
          if (gr.rank < 4) continue;
          R *eg = ellg + (size_t)gi * Sp;
          int bin = 0;
          for (int l = 1; l + 2 < gr.rank; ++l) {
            const BiLevel &lv = gr.lev[l];
            const R *L = smem + sm.V[gi][bin];
            R *Vout = smem + sm.V[gi][bin ^ 1];
            switch (lv.last_pv) {
              case 4: deeper_level<R, 4>(lv, L, cur, Vout, eg, lane); break;
              case 8: deeper_level<R, 8>(lv, L, cur, Vout, eg, lane); break;
              case 16: deeper_level<R, 16>(lv, L, cur, Vout, eg, lane); break;
              default: deeper_level<R, 32>(lv, L, cur, Vout, eg, lane); break;
            }
            bin ^= 1;
          }
          last_level<R>(gr.lev[gr.rank - 2], smem + sm.V[gi][bin], cur, eg, gr.first_qoff, lane);
        }
        __syncthreads();
      }
      // ---- C: one warp per factor
      const bool final = k == K - 1;
      for (int f = warp; f < F; f += NW) {
        const int n = md.n[f], op = md.offp[f];
        R x = -bi_inf<R>();
        if (lane < n) {
          R x0 = lpri[op + lane], x1 = (R)0;
          const int4 *o = ops + f * sm.maxops;
          const int no = nops[f];
          for (int j = 0; j < no; ++j) {
            const int4 e = o[j];
            const int cnt = e.x >> 8;
            const R *base = smem + e.y;
            switch (e.x & 255) {
              case CTA_OP_ROW: x0 += op_row_dot<R>(base + lane * e.z, cur + e.w, cnt); break;
              case CTA_OP_COL: x1 += op_col_dot<R>(base + lane, e.z, cur + e.w, cnt); break;
              default: {
                R s0 = base[lane];
                for (int i = 1; i < cnt; ++i) s0 += base[i * e.z + lane];
                x1 += s0;
              }
            }
          }
          x = x0 + x1;
          if (xp) {   // damped step on the logits; xp: the previous iterate's
            x = fma(lam, x, ((R)1 - lam) * xp[op + lane]);
            xp[op + lane] = x;
          }
        }
        R mx, e, z, q;
        bool fast = false;
        if constexpr (sizeof(R) == 8) fast = !final;
        if (fast) {
          // every iteration but the last: exponentials relative to the largest binary exponent among the
          // logits (one integer reduction; every e lies in [0, 2)) and a reciprocal good to 1e-13
          if constexpr (sizeof(R) == 8) {
            int kx;
            const double mant = tile3_f64::exp_mant(lane < n ? x : 0.0, exp_tab, kx);
            const int km = __reduce_max_sync(0xffffffffu, lane < n ? kx : INT_MIN);
            e = lane < n ? tile3_f64::exp_scale(mant, (kx >> tile3_f64::EXP_BITS) - (km >> tile3_f64::EXP_BITS)) : 0.0;
            z = warp_sum_first(e, n);
            q = e * tile3_f64::rcp_fast(z);
          }
          mx = (R)0;
        } else {
          mx = warp_max(x);
          e = lane < n ? bi_exp_inline(x - mx) : (R)0;
          z = warp_sum(e);
          q = e * bi_rcp(z);
        }
        if (lane < md.npad[f]) nxt[op + lane] = lane < n ? q : (R)0;
        if (final) {
          const size_t ob = (size_t)a * T + t;
          if (lane < n) {
            q_out[ob * S + md.off[f] + lane] = (float)q;
            if (logq_out) logq_out[ob * S + md.off[f] + lane] = (float)(x - mx - bi_log(z));
          }
          if (argmax_out) {
            const unsigned b = __ballot_sync(0xffffffffu, lane < n && x == mx);
            if (lane == 0) argmax_out[ob * F + f] = __ffs(b) - 1;
          }
        }
      }
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
}

template <typename R>
int launch_cta_filter_t(const BiCall &c, bi_model *mut) {
  const bi_model *md = c.model;
  const BiDev &h = md->h;
  // Threads per CTA: enough for the largest first level's rows, and more when the batch leaves the
  // SMs room (two 8-warp CTAs fill an SM's registers; with more agents per SM smaller CTAs let more
  // of them be resident).  Measured on the 128 random structures: 256 threads for every structure
  // took the sum of times from 61 to 54 ms at 256 agents and from 133 to 204 ms at 1024.
  int NT = c.N <= 2 * md->sm_count ? 256 : c.N <= 4 * md->sm_count ? 128 : 64;
  while (NT < md->rows_max && NT < 256) NT <<= 1;
  const int NW = NT / 32;
  CtaGeom sm;
  int o = 0;
  sm.desc = o; o += (int)((sizeof(BiDev) + sizeof(R) - 1) / sizeof(R));
  o = (o + 3) & ~3;
  sm.q0 = o; o += h.Sp;
  sm.q1 = o; o += h.Sp;
  sm.lpri = o; o += h.Sp;
  sm.xp = c.lambda != 1.0 ? o : -1;
  if (c.lambda != 1.0) o += h.Sp;
  sm.ellg = o; o += h.ngroups * h.Sp;
  // classes of rank >= 3 groups by the factor of their last axis
  sm.ncls = 0;
  {
    bool taken[BI_MAX_GROUPS] = {};
    int pos = 0, start = 0;
    for (int gi = 0; gi < h.ngroups; ++gi) {
      if (taken[gi] || h.grp[gi].rank < 3) continue;
      sm.cls_begin[sm.ncls] = pos;
      sm.cls_pv[sm.ncls] = h.grp[gi].lev[0].last_pv;
      sm.cls_wmask[sm.ncls] = 0;
      for (int gj = gi; gj < h.ngroups; ++gj) {
        if (taken[gj] || h.grp[gj].rank < 3 || h.grp[gj].lev[0].last_qoff != h.grp[gi].lev[0].last_qoff) continue;
        taken[gj] = true;
        sm.order[pos++] = gj;
        // rows go round the CTA's threads from where the previous group's ended (a whole warp on)
        sm.row_start[gj] = start % NT;
        const int nr = h.grp[gj].lev[0].nrows;
        for (int w = 0; w < NW; ++w) {
          int first = w * 32 - sm.row_start[gj];   // the row of this warp's first thread
          if (first < 0) first += NT;
          if (nr >= NT || first < nr || first + 31 >= NT) sm.cls_wmask[sm.ncls] |= 1 << w;
        }
        start = (start + nr + 31) & ~31;
      }
      ++sm.ncls;
    }
    sm.cls_begin[sm.ncls] = pos;
  }
  sm.deep = 0;
  for (int f = 0; f < BI_MAX_F; ++f) sm.f_cls[f] = sm.f_m0[f] = sm.f_m1[f] = sm.f_r1[f] = sm.f_deep[f] = 0;
  for (int f = 0; f < h.F; ++f) {
    for (int cls = 0; cls < sm.ncls; ++cls)
      if (h.grp[sm.order[sm.cls_begin[cls]]].lev[0].last_qoff == h.offp[f]) sm.f_cls[f] |= 1u << cls;
    for (int gi = 0; gi < h.ngroups; ++gi) {
      const BiGroup &g = h.grp[gi];
      if (g.rank == 1) {
        if (g.first_qoff == h.offp[f]) sm.f_r1[f] |= 1u << gi;
      } else if (g.rank <= 3) {
        if (g.axis[0] == f) sm.f_m0[f] |= 1u << gi;
        if (g.axis[1] == f) sm.f_m1[f] |= 1u << gi;
      } else {
        sm.deep = 1;
        // every axis but the last is finished by phase B (the last axis' message comes from the class)
        for (int j = 0; j + 1 < g.rank; ++j)
          if (g.axis[j] == f) sm.f_deep[f] |= 1u << gi;
      }
    }
  }
  sm.part = o; o += std::max(1, sm.ncls) * NW * 32;
  {  // phase C's operation lists: the longest decides the row length
    sm.maxops = 1;
    for (int f = 0; f < h.F; ++f) {
      int c = __builtin_popcount(sm.f_m0[f]) + __builtin_popcount(sm.f_m1[f]) + __builtin_popcount(sm.f_r1[f]) +
              __builtin_popcount(sm.f_deep[f]);
      for (int cls = 0; cls < sm.ncls; ++cls) {
        if (!((sm.f_cls[f] >> cls) & 1)) continue;
        const unsigned wm = (unsigned)sm.cls_wmask[cls];
        for (int w = 0; w < NW; ++w) c += ((wm >> w) & 1) && (w == 0 || !((wm >> (w - 1)) & 1));
      }
      sm.maxops = std::max(sm.maxops, c);
    }
    o = (o + 3) & ~3;
    sm.ops = o; o += (int)((size_t)h.F * sm.maxops * 16 / sizeof(R));
    sm.nops = o; o += bi_pad4(h.F);
    sm.exptab = o;
    if (sizeof(R) == 8) o += tile3_f64::EXP_TAB;
  }
  sm.vtot_begin = o;
  for (int gi = 0; gi < BI_MAX_GROUPS; ++gi) sm.V[gi][0] = sm.V[gi][1] = o;
  for (int gi = 0; gi < h.ngroups; ++gi) {
    const BiGroup &g = h.grp[gi];
    int need[2] = {4, 4};
    for (int l = 0; l + 1 < g.rank; ++l) {
      const BiLevel &lv = g.lev[l];
      const int out = (lv.nrows / lv.dim[lv.ndig - 1]) * bi_row_stride(lv.out_npad, (int)sizeof(R));
      need[l & 1] = std::max(need[l & 1], out);
    }
    sm.V[gi][0] = o; o += bi_pad4(need[0]);
    sm.V[gi][1] = o; o += bi_pad4(need[1]);
  }
  sm.vtot_end = o;
  sm.obs = o; o += bi_pad4(c.T * h.M + 1);
  for (int gi = 0; gi < BI_MAX_GROUPS; ++gi) { sm.Lst[gi] = o; sm.lstride[gi] = 4; }
  for (int gi = 0; gi < h.ngroups; ++gi) {
    const BiGroup &g = h.grp[gi];
    const int npad = g.rank > 1 ? g.lev[0].last_npad4 * 4 : bi_pad4(g.first_n);
    const int rows = g.P_pad / npad;
    sm.lstride[gi] = bi_row_stride(npad, (int)sizeof(R));
    sm.Lst[gi] = o;
    o += bi_pad4(rows * sm.lstride[gi]);
  }
  for (int gi = 0; gi < BI_MAX_GROUPS; ++gi) sm.mat_off[gi] = sm.mat_ls[gi] = sm.mat_lev[gi] = 0;
  for (int gi = 0; gi < h.ngroups; ++gi) {
    const BiGroup &g = h.grp[gi];
    if (g.rank == 2) {
      sm.mat_off[gi] = sm.Lst[gi]; sm.mat_ls[gi] = sm.lstride[gi]; sm.mat_lev[gi] = 0;
    } else if (g.rank == 3) {   // the first level's output: rows at the padded stride of its last axis
      sm.mat_off[gi] = sm.V[gi][0];
      sm.mat_ls[gi] = bi_row_stride(g.lev[0].out_npad, (int)sizeof(R));
      sm.mat_lev[gi] = 1;
    }
  }
  sm.prior_tps = 4 * h.Sp <= NT ? 4 : 2 * h.Sp <= NT ? 2 : 1;
  sm.wpar = o;
  sm.wpar_cap = 0;
  if (h.has_bdep) {
    for (int f = 0; f < h.F; ++f) sm.wpar_cap = std::max(sm.wpar_cap, (int)h.PB[f]);
    sm.wpar_cap = std::min(bi_pad4(sm.wpar_cap), 4096);
    o += sm.wpar_cap;
  }
  sm.total_bytes = (int)((size_t)o * sizeof(R));
  if ((size_t)o * sizeof(R) > (size_t)md->max_smem_optin - 1024) return BI_ERR_UNSUPPORTED;

  auto kern = bi_cta_filter_kernel<R>;
  if (cudaFuncSetAttribute((const void *)kern, cudaFuncAttributeMaxDynamicSharedMemorySize, sm.total_bytes) !=
      cudaSuccess)
    return BI_ERR_CUDA;
  kern<<<c.N, NT, sm.total_bytes, c.stream>>>(md->d, c.T, c.obs, c.act, c.q_prev, c.act_prev, c.carry_in, c.carry_out, c.lambda, c.K, c.q_out,
                                               c.logq_out, c.argmax_out, sm);
  if (cudaGetLastError() != cudaSuccess) return BI_ERR_CUDA;
  mut->launches += 1;
  mut->last_kernel = sizeof(R) == 8 ? "cta_filter_f64" : "cta_filter_f32";
  return BI_OK;
}

}  // namespace

int bi_launch_cta_filter(const BiCall &c, bi_model *mut) {
  if (c.algo != BI_ALGO_FILTER) return BI_ERR_UNSUPPORTED;
  return c.model->arith == BI_ARITH_F64 ? launch_cta_filter_t<double>(c, mut) : launch_cta_filter_t<float>(c, mut);
}
