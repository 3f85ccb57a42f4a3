// Generic kernels, one warp per (agent, time step): any model within the
// BI_MAX_* limits, any of the three algorithms, either arithmetic.
//
// A warp owns one agent at one time step.  Filtering: the warp walks the
// agent's steps in order.  Windows: a CTA owns one agent, its warps share the
// steps, and one barrier per iteration publishes the beliefs (Jacobi over
// steps: Appendix A-2 runs the window's steps side by side).  Inside a sweep
// only the warp synchronises.
//
// Likelihood messages (Section IV, marginalisation) of a dependency group are
// contracted one axis at a time, last axis first.  A level with leading
// multi-index r (rows, spread over the lanes) and last index c computes
//   V[r]        = sum_c L[r,c] q_last[c]            (input of the next level)
//   ell_last[c] += (prod_j q_j[r_j]) * L[r,c]       (message to the last axis)
// so the k messages of a group cost about 2 P multiply-adds, not k P.  Each
// lane keeps its partial ell_last in registers; a transposing butterfly
// (reduce-scatter) sums them over the warp.  The slice L is read from the
// packed model through L1/L2 (summed over the group's modalities on the fly).
#include <algorithm>

#include "bi_internal.h"
#include "tile3.cuh"

namespace {

struct WarpSmem {       // element offsets (units of R) into dynamic shared memory after the descriptor copy
  int q;                // window: [2][T][Sp] beliefs shared by the CTA; filtering: unused
  int warp0, per_warp;  // per-warp scratch: ell | lpri | q0 | q1 | V0 | V1 | slice pointers
  int o_ell, o_lpri, o_q0, o_q1, o_V0, o_V1, o_sl;
  int obs;              // window: [T][M] clamped observations (ints, offset in units of R)
  int md_bytes;         // bytes reserved for the model descriptor copy
  int total_bytes;
  int W;                // warps per CTA
  int o_xp;             // filtering, damped calls: per-warp previous logits [Sp]; -1 otherwise
  int o_Y;              // window, models with B-dependencies: per-warp [sum_h PB_h] next-belief-weighted tensors; -1 otherwise
  int xp;               // window, damped calls: [T][Sp] previous logits shared by the CTA; -1 otherwise
  // window, models with B-dependencies of at most four parents: per-warp [sum_f PB_f] products of the
  // parents' previous beliefs, and the CTA's table [sum_f PB_f] of the belief entries each product takes
  // (one byte per parent: its padded belief offset); -1 otherwise
  int o_W, dtab;
};

template <typename R>
struct GlobalRows {     // sum over a group's members of their observed slices
  const R *const *sl;   // per-warp table of slice pointers (shared memory)
  int m0, m1, npad;
  __device__ __forceinline__ Vec4<R> operator()(int r, int c4) const {
    Vec4<R> acc = ldg4(sl[m0] + (size_t)r * npad + 4 * c4);
    for (int i = m0 + 1; i < m1; ++i) {
      Vec4<R> x = ldg4(sl[i] + (size_t)r * npad + 4 * c4);
      acc.x += x.x; acc.y += x.y; acc.z += x.z; acc.w += x.w;
    }
    return acc;
  }
};
template <typename R>
struct SmemRows {
  const R *base;
  int npad;
  __device__ __forceinline__ Vec4<R> operator()(int r, int c4) const {
    return *reinterpret_cast<const Vec4<R> *>(base + r * npad + 4 * c4);
  }
};

template <typename R, int PV, class LD>
__device__ __forceinline__ void peel_level_warp(const BiLevel &lv, const LD &ld, const R *qt, R *Vout,
                                                R *ell, int lane) {
  R acc[PV];
#pragma unroll
  for (int c = 0; c < PV; ++c) acc[c] = (R)0;
  // the level's description is read into registers once: it lives in shared
  // memory, and the stores below would otherwise force a reload per row
  const int npad4 = lv.last_npad4, ndig = lv.ndig, nrows = lv.nrows;
  const int onp = bi_row_stride(lv.out_npad, (int)sizeof(R));   // rows of the partial tensor at a conflict-free stride
  uint32_t magic[4], dim[4];
  const R *qd_base[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    magic[i] = i < ndig ? lv.magic[i] : 0u;
    dim[i] = i < ndig ? (uint32_t)lv.dim[i] : 1u;
    qd_base[i] = qt + (i < ndig ? lv.qoff[i] : 0);
  }
  const Vec4<R> *q4 = reinterpret_cast<const Vec4<R> *>(qt + lv.last_qoff);
  for (int r = lane; r < nrows; r += 32) {
    uint32_t rem = (uint32_t)r;
    R w = (R)1;
    int lastdig = 0, hi = 0;
#pragma unroll
    for (int i = 3; i >= 0; --i) {
      if (i < ndig) {
        uint32_t qd = __umulhi(rem, magic[i]);
        int dg = (int)(rem - qd * dim[i]);
        rem = qd;
        w *= qd_base[i][dg];
        if (i == ndig - 1) { lastdig = dg; hi = (int)qd; }
      }
    }
    R v0 = (R)0, v1 = (R)0;
#pragma unroll
    for (int c4 = 0; c4 < PV / 4; ++c4) {
      if (c4 < npad4) {
        Vec4<R> x = ld(r, c4);
        Vec4<R> qq = q4[c4];
        v0 = fma(x.x, qq.x, v0); v1 = fma(x.y, qq.y, v1);
        v0 = fma(x.z, qq.z, v0); v1 = fma(x.w, qq.w, v1);
        acc[4 * c4 + 0] = fma(w, x.x, acc[4 * c4 + 0]);
        acc[4 * c4 + 1] = fma(w, x.y, acc[4 * c4 + 1]);
        acc[4 * c4 + 2] = fma(w, x.z, acc[4 * c4 + 2]);
        acc[4 * c4 + 3] = fma(w, x.w, acc[4 * c4 + 3]);
      }
    }
    Vout[hi * onp + lastdig] = v0 + v1;
  }
  const R tot = reduce_scatter<R, PV, 32, 1>(acc, lane);
  constexpr int SH = 5 - Log2<PV>::v;
  const int idx = lane >> SH;
  if ((lane & ((1 << SH) - 1)) == 0 && idx < lv.last_n) ell[lv.last_qoff + idx] += tot;
  __syncwarp();
}

template <typename R, class LD>
__device__ __forceinline__ void peel_dispatch(const BiLevel &lv, const LD &ld, const R *qt, R *Vout, R *ell,
                                              int lane) {
  switch (lv.last_pv) {
    case 4: peel_level_warp<R, 4>(lv, ld, qt, Vout, ell, lane); break;
    case 8: peel_level_warp<R, 8>(lv, ld, qt, Vout, ell, lane); break;
    case 16: peel_level_warp<R, 16>(lv, ld, qt, Vout, ell, lane); break;
    default: peel_level_warp<R, 32>(lv, ld, qt, Vout, ell, lane); break;
  }
}

// every group's likelihood messages of one (agent, step), added into ell
template <typename R>
__device__ __forceinline__ void likelihood_warp(const BiDev &md, const R *const *sl, const R *qt, R *ell,
                                                R *V0, R *V1, int lane) {
  for (int gi = 0; gi < md.ngroups; ++gi) {
    const BiGroup &gr = md.grp[gi];
    GlobalRows<R> first{sl, gr.mem_begin, gr.mem_end,
                        gr.rank > 1 ? gr.lev[0].last_npad4 * 4 : bi_pad4(gr.first_n)};
    if (gr.rank == 1) {
      if (lane < gr.first_n) {
        Vec4<R> x = first(0, lane >> 2);
        const int k = lane & 3;
        ell[gr.first_qoff + lane] += k == 0 ? x.x : k == 1 ? x.y : k == 2 ? x.z : x.w;
      }
      __syncwarp();
      continue;
    }
    peel_dispatch<R>(gr.lev[0], first, qt, V0, ell, lane);
    R *vin = V0, *vout = V1;
    for (int l = 1; l + 1 < gr.rank; ++l) {
      SmemRows<R> rows{vin, bi_row_stride(gr.lev[l].last_npad4 * 4, (int)sizeof(R))};
      peel_dispatch<R>(gr.lev[l], rows, qt, vout, ell, lane);
      R *t = vin; vin = vout; vout = t;
    }
    if (lane < gr.first_n) ell[gr.first_qoff + lane] += vin[lane];
    __syncwarp();
  }
}

// slice pointers of one (agent, step): sl[mi] for every packed member
template <typename R>
__device__ __forceinline__ void slice_table(const BiDev &md, int g, const int32_t *obs_t, bool clamp,
                                            const R **sl, int lane) {
  if (lane < md.nmem) {
    const BiMember &mm = md.mem[lane];
    int o = obs_t[mm.modality];
    if (clamp) o = clamp_flag(o, mm.m, md.status, BI_FLAG_OBS_RANGE);
    sl[lane] = (const R *)mm.logA + (size_t)g * mm.gstride + (size_t)o * mm.P_pad;
  }
  __syncwarp();
}

// reductions over the NW lanes that hold a factor's states (NW: the power of two at or above n, at
// least 4): a small factor needs two or three shuffle steps, not five
template <int NW, typename T>
__device__ __forceinline__ T group_sum_w(T v) {
#pragma unroll
  for (int o = NW / 2; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
template <int NW, typename T>
__device__ __forceinline__ T group_max_w(T v) {
#pragma unroll
  for (int o = NW / 2; o > 0; o >>= 1) v = bi_max(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}

template <typename R, int NW>
__device__ __forceinline__ void softmax_factor(const BiDev &md, int f, const R *ell, R *qn, bool final, float *q_out,
                                               float *logq_out, int32_t *argmax_out, int lane, R *xp, R lam) {
  const int n = md.n[f], op = md.offp[f];
  R x = lane < n ? ell[op + lane] : -bi_inf<R>();
  if (xp && lane < n) {   // damped step on the logits; xp: the previous iterate's
    x = fma(lam, x, ((R)1 - lam) * xp[op + lane]);
    xp[op + lane] = x;
  }
  // the shift only has to be close to the maximum (softmax is shift
  // invariant): a float reduction halves the shuffles of a double one
  R mx = final ? group_max_w<NW>(x) : (R)group_max_w<NW>((float)x);
  R e = lane < n ? bi_exp_inline(x - mx) : (R)0;
  R z = group_sum_w<NW>(e);
  R q = e * bi_rcp(z);
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

// softmax of every factor of one step from the logits in ell
template <typename R>
__device__ __forceinline__ void softmax_warp(const BiDev &md, const R *ell, R *qn, bool final, float *q_out,
                                             float *logq_out, int32_t *argmax_out, int lane, R *xp = nullptr,
                                             R lam = (R)1) {
  for (int f = 0; f < md.F; ++f) {
    const int n = md.n[f];
    if (n <= 4) softmax_factor<R, 4>(md, f, ell, qn, final, q_out, logq_out, argmax_out, lane, xp, lam);
    else if (n <= 8) softmax_factor<R, 8>(md, f, ell, qn, final, q_out, logq_out, argmax_out, lane, xp, lam);
    else if (n <= 16) softmax_factor<R, 16>(md, f, ell, qn, final, q_out, logq_out, argmax_out, lane, xp, lam);
    else softmax_factor<R, 32>(md, f, ell, qn, final, q_out, logq_out, argmax_out, lane, xp, lam);
  }
  __syncwarp();
}

// sum_r M[r][s] q[r] for this lane's state s (M stored [r][s], rows npad apart)
template <typename R>
__device__ __forceinline__ R col_dot_rt(const R *__restrict__ col, int npad, const R *q, int n) {
  R s0 = (R)0, s1 = (R)0;
  int r = 0;
  for (; r + 1 < n; r += 2) {
    s0 = fma(__ldg(col + (size_t)r * npad), q[r], s0);
    s1 = fma(__ldg(col + (size_t)(r + 1) * npad), q[r + 1], s1);
  }
  if (r < n) s0 = fma(__ldg(col + (size_t)r * npad), q[r], s0);
  return s0 + s1;
}

// Non-trivial B-dependencies (VMP only): the two transition messages of one state, summed by its lane.
// The parents' state combinations are walked with an odometer (last parent fastest, the order the
// tensor is stored in) and running prefix products of their beliefs, so a step costs one multiply
// per digit that changed and no division.
// Past: sum_{parents} ln B_f[s][parents] prod_j q_{t-1, parent_j}[s_j].
template <typename R>
__device__ R bdep_past_lane(const BiDev &md, int f, const R *__restrict__ Xrow, const R *qprev) {
  const int k = md.bdep_len[f], PB = md.PB[f];
  int dig[BI_MAX_RANK], nj[BI_MAX_RANK], op[BI_MAX_RANK];
  R wp[BI_MAX_RANK];   // wp[j] = prod_{i <= j} q_{parent_i}[dig_i]
#pragma unroll
  for (int j = 0; j < BI_MAX_RANK; ++j) {
    dig[j] = 0;
    nj[j] = j < k ? md.n[md.bdep[f][j]] : 1;
    op[j] = j < k ? md.offp[md.bdep[f][j]] : 0;
    wp[j] = (R)1;
  }
#pragma unroll
  for (int j = 0; j < BI_MAX_RANK; ++j)
    if (j < k) wp[j] = (j > 0 ? wp[j > 0 ? j - 1 : 0] : (R)1) * qprev[op[j]];
  R acc = (R)0;
  for (int e = 0; e < PB; ++e) {
    R w = wp[0];
#pragma unroll
    for (int j = 1; j < BI_MAX_RANK; ++j) w = j == k - 1 ? wp[j] : w;
    acc = fma(__ldg(Xrow + e), w, acc);
    // next combination: increment from the last parent, carrying
    int lo = k;   // lowest digit index that changed
    bool carry = true;
#pragma unroll
    for (int j = BI_MAX_RANK - 1; j >= 0; --j) {
      if (j < k && carry) {
        dig[j] += 1;
        if (dig[j] == nj[j]) dig[j] = 0; else carry = false;
        lo = j;
      }
    }
#pragma unroll
    for (int j = 0; j < BI_MAX_RANK; ++j)
      if (j < k && j >= lo) wp[j] = (j > 0 ? wp[j > 0 ? j - 1 : 0] : (R)1) * qprev[op[j] + dig[j]];
  }
  return acc;
}
// The same with the parents' products already formed (W: one entry per parent combination).
template <typename R>
__device__ __forceinline__ R bdep_past_dot(const R *__restrict__ Xrow, const R *W, int PB) {
  R a0 = (R)0, a1 = (R)0;
  int e = 0;
#pragma unroll 2
  for (; e + 1 < PB; e += 2) {
    a0 = fma(__ldg(Xrow + e), W[e], a0);
    a1 = fma(__ldg(Xrow + e + 1), W[e + 1], a1);
  }
  if (e < PB) a0 = fma(__ldg(Xrow + e), W[e], a0);
  return a0 + a1;
}
// Future, to state s of factor f0: over every factor h whose transition reads f0,
// sum_{s'} q_{t+1,h}[s'] sum_{parents with s_f0 = s} ln B_h[s'][parents] prod_{other parents} q_t[...];
// act_t: the actions taken at this step.  The other parents' combinations are walked the same way.
// Y: for every factor h in turn, Y_h[parents] = sum_{s'} q_{t+1,h}[s'] ln B_h[s'][parents], formed by the warp
// before its lanes call this (bdep_weighted_tensors).
template <typename R>
__device__ void bdep_weighted_tensors(const BiDev &md, int g, const R *qn, const int32_t *__restrict__ act_t, R *Y,
                                      int lane) {
  int yo = 0;
  for (int h = 0; h < md.F; ++h) {
    const int nh = md.n[h], PB = md.PB[h];
    const int u = clamp_flag(act_t[h], md.U[h], md.status, BI_FLAG_ACT_RANGE);
    const R *X = (const R *)md.logBfull[h] + (size_t)g * md.Bfull_stride[h] + (size_t)u * nh * PB;
    for (int e = lane; e < PB; e += 32) {   // (consecutive lanes read consecutive entries of a tensor row)
      R acc = (R)0;
      for (int sn = 0; sn < nh; ++sn) acc = fma(qn[md.offp[h] + sn], __ldg(X + (size_t)sn * PB + e), acc);
      Y[yo + e] = acc;
    }
    yo += PB;
  }
}
template <typename R>
__device__ R bdep_future_lane(const BiDev &md, int f0, int s, const R *q, const R *Y) {
  R acc = (R)0;
  int yo = 0;
  for (int h = 0; h < md.F; yo += md.PB[h], ++h) {
    const int k = md.bdep_len[h];
    int pos = -1;
    for (int j = 0; j < k; ++j)
      if (md.bdep[h][j] == f0) pos = j;
    if (pos < 0) continue;
    const int PB = md.PB[h];
    const R *Yh = Y + yo;
    if (k == 1) {   // the factor's own previous state only: the weighted tensor's entry is the message
      acc += Yh[s];
      continue;
    }
    if (k == 2) {   // one other parent: a strided dot product with its belief, no odometer
      const int go = md.bdep[h][1 - pos], no = md.n[go];
      const R *qo = q + md.offp[go];
      // parents in list order, last fastest: entry (d0, d1) sits at d0 * n1 + d1
      const int n1 = md.n[md.bdep[h][1]];
      const R *y = Yh + (pos == 0 ? s * n1 : s);
      const int st = pos == 0 ? 1 : n1;
      R a0 = (R)0, a1 = (R)0;
      int i = 0;
      for (; i + 1 < no; i += 2) {
        a0 = fma(qo[i], y[i * st], a0);
        a1 = fma(qo[i + 1], y[(i + 1) * st], a1);
      }
      if (i < no) a0 = fma(qo[i], y[i * st], a0);
      acc += a0 + a1;
      continue;
    }
    const int others = PB / md.n[f0];
    int dig[BI_MAX_RANK], nj[BI_MAX_RANK], op[BI_MAX_RANK], str[BI_MAX_RANK];
    int stride = 1;
#pragma unroll
    for (int j = BI_MAX_RANK - 1; j >= 0; --j) {
      dig[j] = 0;
      nj[j] = j < k ? md.n[md.bdep[h][j]] : 1;
      op[j] = j < k ? md.offp[md.bdep[h][j]] : 0;
      str[j] = stride;           // element stride of parent j in the tensor's parent index
      if (j < k) stride *= nj[j];
    }
    int e = 0;                   // parent index of the current combination (own digit fixed at s)
#pragma unroll
    for (int j = 0; j < BI_MAX_RANK; ++j)
      if (j == pos) { dig[j] = s; e += s * str[j]; }
    for (int i = 0; i < others; ++i) {
      R w = (R)1;
#pragma unroll
      for (int j = 0; j < BI_MAX_RANK; ++j)
        if (j < k && j != pos) w *= q[op[j] + dig[j]];
      acc = fma(w, Yh[e], acc);
      bool carry = true;
#pragma unroll
      for (int j = BI_MAX_RANK - 1; j >= 0; --j) {
        if (j < k && j != pos && carry) {
          dig[j] += 1;
          e += str[j];
          if (dig[j] == nj[j]) { dig[j] = 0; e -= nj[j] * str[j]; } else carry = false;
        }
      }
    }
  }
  return acc;
}

static_assert(sizeof(BiDev) % sizeof(int4) == 0, "descriptor is copied as 16-byte vectors");
__device__ __forceinline__ void copy_descriptor(const BiDev *src, void *dst) {
  const int4 *s = reinterpret_cast<const int4 *>(src);
  int4 *d = reinterpret_cast<int4 *>(dst);
  for (int i = threadIdx.x; i < (int)(sizeof(BiDev) / sizeof(int4)); i += blockDim.x) d[i] = __ldg(s + i);
  __syncthreads();
}

template <typename R>
__global__ void __launch_bounds__(512)
bi_warp_filter_kernel(const BiDev *__restrict__ mdp, int N, int T, const int32_t *__restrict__ obs,
                      const int32_t *__restrict__ act, const float *q_prev, const int32_t *__restrict__ act_prev,
                      const void *carry_in, void *carry_out, double lambda, int K, float *q_out,
                      float *__restrict__ logq_out, int32_t *__restrict__ argmax_out, WarpSmem sm) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  copy_descriptor(mdp, smem_raw);
  const BiDev &md = *reinterpret_cast<const BiDev *>(smem_raw);
  R *base = reinterpret_cast<R *>(smem_raw + sm.md_bytes);
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int a = blockIdx.x * sm.W + warp;
  if (a >= N) return;  // whole warps leave; nothing below synchronises the CTA
  const int g = md.G == 1 ? 0 : a;
  const int S = md.S, Sp = md.Sp, F = md.F, M = md.M;
  R *wb = base + sm.warp0 + (size_t)warp * sm.per_warp;
  R *ell = wb + sm.o_ell, *lpri = wb + sm.o_lpri, *cur = wb + sm.o_q0, *nxt = wb + sm.o_q1;
  R *V0 = wb + sm.o_V0, *V1 = wb + sm.o_V1;
  const R **sl = reinterpret_cast<const R **>(wb + sm.o_sl);
  R *xpw = sm.o_xp >= 0 ? wb + sm.o_xp : nullptr;
  for (int i = lane; i < sm.o_sl - sm.o_q0; i += 32) cur[i] = (R)0;  // q0, q1, V0, V1 are adjacent
  __syncwarp();
  const bool from_prev = q_prev != nullptr || carry_in != nullptr;
  if (from_prev) {  // continued filtering: the belief of the step before the window
    for (int idx = lane; idx < Sp; idx += 32) {
      int f = 0;
      while (f + 1 < F && idx >= md.offp[f + 1]) ++f;
      const int s = idx - md.offp[f];
      const size_t src = (size_t)a * S + md.off[f] + s;
      if (s < md.n[f]) cur[idx] = carry_in ? ((const R *)carry_in)[src] : (R)q_prev[src];
    }
    __syncwarp();
  }

  float *q_a = q_out + (size_t)a * T * S;
  float *lq_a = logq_out ? logq_out + (size_t)a * T * S : nullptr;
  int32_t *am_a = argmax_out ? argmax_out + (size_t)a * T * F : nullptr;
  for (int t = 0; t < T; ++t) {
    // ln prior: D at the first step, else B_u q_{t-1} (cur still holds step t-1's final belief)
    for (int idx = lane; idx < Sp; idx += 32) {
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
          const R *col = (const R *)md.BfT[f] + (size_t)g * md.Bstride[f] + (size_t)u * n * md.npad[f] + s;
          lp = bi_log_inline(bi_max(col_dot_rt<R>(col, md.npad[f], cur + md.offp[f], n), (R)BI_EPS));
        }
      }
      lpri[idx] = lp;
    }
    slice_table<R>(md, g, obs + ((size_t)a * T + t) * M, true, sl, lane);
    for (int idx = lane; idx < Sp; idx += 32) {
      int f = 0;
      while (f + 1 < F && idx >= md.offp[f + 1]) ++f;
      cur[idx] = (idx - md.offp[f]) < md.n[f] ? (R)1 / (R)md.n[f] : (R)0;
      if (xpw) xpw[idx] = (R)0;   // logits of the uniform start: a constant
    }
    __syncwarp();
    for (int k = 0; k < K; ++k) {
      for (int idx = lane; idx < Sp; idx += 32) ell[idx] = lpri[idx];
      __syncwarp();
      likelihood_warp<R>(md, sl, cur, ell, V0, V1, lane);
      softmax_warp<R>(md, ell, nxt, k == K - 1, q_a + (size_t)t * S, lq_a ? lq_a + (size_t)t * S : nullptr,
                      am_a ? am_a + (size_t)t * F : nullptr, lane, xpw, (R)lambda);
      R *tmp = cur; cur = nxt; nxt = tmp;
    }
  }
  if (carry_out) {   // the last step's belief at full precision, for a call that continues this one
    __syncwarp();
    for (int idx = lane; idx < Sp; idx += 32) {
      int f = 0;
      while (f + 1 < F && idx >= md.offp[f + 1]) ++f;
      const int s = idx - md.offp[f];
      if (s < md.n[f]) ((R *)carry_out)[(size_t)a * S + md.off[f] + s] = cur[idx];
    }
  }
}

template <typename R, int ALGO>
__global__ void __launch_bounds__(512)
bi_warp_window_kernel(const BiDev *__restrict__ mdp, int N, int T, const int32_t *__restrict__ obs,
                      const int32_t *__restrict__ act, const float *__restrict__ q_init,
                      const void *__restrict__ lnprior, double lambda, int K, float *__restrict__ q_out,
                      float *__restrict__ logq_out, int32_t *__restrict__ argmax_out, WarpSmem sm) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  copy_descriptor(mdp, smem_raw);
  const BiDev &md = *reinterpret_cast<const BiDev *>(smem_raw);
  R *base = reinterpret_cast<R *>(smem_raw + sm.md_bytes);
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, W = sm.W;
  const int a = blockIdx.x;
  const int g = md.G == 1 ? 0 : a;
  const int S = md.S, Sp = md.Sp, F = md.F, M = md.M;
  R *qb = base + sm.q;
  int32_t *obs_s = reinterpret_cast<int32_t *>(base + sm.obs);
  R *wb = base + sm.warp0 + (size_t)warp * sm.per_warp;
  R *ell = wb + sm.o_ell, *V0 = wb + sm.o_V0, *V1 = wb + sm.o_V1;
  const R **sl = reinterpret_cast<const R **>(wb + sm.o_sl);
  for (int i = lane; i < sm.o_sl - sm.o_V0; i += 32) V0[i] = (R)0;  // V0 and V1 are adjacent
  for (int i = threadIdx.x; i < T * M; i += blockDim.x)
    obs_s[i] = clamp_flag(obs[(size_t)a * T * M + i], md.m[i % M], md.status, BI_FLAG_OBS_RANGE);
  if (sm.dtab >= 0) {   // which belief entries the product of a parent combination takes (once per launch)
    uint32_t *dt = reinterpret_cast<uint32_t *>(base + sm.dtab);
    int yo = 0;
    for (int f = 0; f < F; ++f) {
      const int PB = md.PB[f], k = md.bdep_len[f];
      for (int e = threadIdx.x; e < PB; e += blockDim.x) {
        int rem = e;
        uint32_t pack = 0;
        for (int j = k - 1; j >= 0; --j) {
          const int gq = md.bdep[f][j], nj = md.n[gq];
          pack |= (uint32_t)(md.offp[gq] + rem % nj) << (8 * j);
          rem /= nj;
        }
        dt[yo + e] = pack;
      }
      yo += PB;
    }
  }
  for (int i = threadIdx.x; i < 2 * T * Sp; i += blockDim.x) {
    const int pidx = i % Sp;
    int f = 0;
    while (f + 1 < F && pidx >= md.offp[f + 1]) ++f;
    const int s = pidx - md.offp[f];
    R v = (R)0;
    if (s < md.n[f])
      v = (q_init && i < T * Sp) ? (R)q_init[((size_t)a * T + i / Sp) * S + md.off[f] + s] : (R)1 / (R)md.n[f];
    qb[i] = v;
    if (sm.xp >= 0 && i < T * Sp)   // damped calls: logits of the start (uniform: a constant)
      (base + sm.xp)[i] = (q_init && s < md.n[f]) ? bi_log(bi_max(v, (R)BI_EPS)) : (R)0;
  }
  __syncthreads();

  float *q_a = q_out + (size_t)a * T * S;
  float *lq_a = logq_out ? logq_out + (size_t)a * T * S : nullptr;
  int32_t *am_a = argmax_out ? argmax_out + (size_t)a * T * F : nullptr;
  R *cur = qb, *nxt = qb + (size_t)T * Sp;
  for (int k = 0; k < K; ++k) {
    for (int t = warp; t < T; t += W) {
      const R *qt = cur + (size_t)t * Sp;
      slice_table<R>(md, g, obs_s + t * M, false, sl, lane);
      if (sm.o_Y >= 0 && t + 1 < T) {
        bdep_weighted_tensors<R>(md, g, cur + (size_t)(t + 1) * Sp, act + ((size_t)a * (T - 1) + t) * F, wb + sm.o_Y, lane);
        __syncwarp();
      }
      if (sm.o_W >= 0 && t > 0) {   // the parents' products under the previous step's beliefs, for every factor
        const R *qp = cur + (size_t)(t - 1) * Sp;
        const uint32_t *dt = reinterpret_cast<const uint32_t *>(base + sm.dtab);
        R *Wv = wb + sm.o_W;
        int yo = 0;
        for (int f = 0; f < F; ++f) {
          const int PB = md.PB[f], k = md.bdep_len[f];
          for (int e = lane; e < PB; e += 32) {
            const uint32_t d = dt[yo + e];
            R w = qp[d & 255u];
            if (k > 1) w *= qp[(d >> 8) & 255u];
            if (k > 2) w *= qp[(d >> 16) & 255u];
            if (k > 3) w *= qp[d >> 24];
            Wv[yo + e] = w;
          }
          yo += PB;
        }
        __syncwarp();
      }
      // transition messages (Section IV): low-rank contractions of B with the
      // neighbouring steps' beliefs of the previous iterate; transposed layouts
      // so that consecutive lanes read consecutive addresses
      for (int idx = lane; idx < Sp; idx += 32) {
        int f = 0;
        while (f + 1 < F && idx >= md.offp[f + 1]) ++f;
        const int s = idx - md.offp[f], n = md.n[f], np = md.npad[f];
        R msg = (R)0;
        if (s < n) {
          if (t == 0) {
            msg = lnprior ? ((const R *)lnprior)[(size_t)a * S + md.off[f] + s]
                          : ((const R *)md.logD[f])[(size_t)g * md.Dstride[f] + s];
          } else if (md.has_bdep) {
            const int u = clamp_flag(act[((size_t)a * (T - 1) + (t - 1)) * F + f], md.U[f], md.status, BI_FLAG_ACT_RANGE);
            const R *row = (const R *)md.logBfull[f] + (size_t)g * md.Bfull_stride[f] + ((size_t)u * n + s) * md.PB[f];
            if (sm.o_W >= 0) {
              int yo = 0;
              for (int j = 0; j < f; ++j) yo += md.PB[j];
              msg = bdep_past_dot<R>(row, wb + sm.o_W + yo, md.PB[f]);
            } else {
              msg = bdep_past_lane<R>(md, f, row, cur + (size_t)(t - 1) * Sp);
            }
          } else {
            int u = clamp_flag(act[((size_t)a * (T - 1) + (t - 1)) * F + f], md.U[f], md.status, BI_FLAG_ACT_RANGE);
            const R *M0 = (const R *)(ALGO == BI_ALGO_VMP ? md.logBt[f] : md.BfT[f]);  // [previous][next]
            const R *col = M0 + (size_t)g * md.Bstride[f] + (size_t)u * n * np + s;
            R v = col_dot_rt<R>(col, np, cur + (size_t)(t - 1) * Sp + md.offp[f], n);
            msg = ALGO == BI_ALGO_VMP ? v : (R)0.5 * bi_log_inline(bi_max(v, (R)BI_EPS));
          }
          if (t + 1 < T && md.has_bdep) {
            msg += bdep_future_lane<R>(md, f, s, qt, wb + sm.o_Y);
          } else if (t + 1 < T) {
            int u = clamp_flag(act[((size_t)a * (T - 1) + t) * F + f], md.U[f], md.status, BI_FLAG_ACT_RANGE);
            const R *M1 = (const R *)(ALGO == BI_ALGO_VMP ? md.logB[f] : md.BdagT[f]);  // [next][previous]
            const R *col = M1 + (size_t)g * md.Bstride[f] + (size_t)u * n * np + s;
            R v = col_dot_rt<R>(col, np, cur + (size_t)(t + 1) * Sp + md.offp[f], n);
            msg += ALGO == BI_ALGO_VMP ? v : (R)0.5 * bi_log_inline(bi_max(v, (R)BI_EPS));
          }
        }
        ell[idx] = msg;
      }
      __syncwarp();
      likelihood_warp<R>(md, sl, qt, ell, V0, V1, lane);
      softmax_warp<R>(md, ell, nxt + (size_t)t * Sp, k == K - 1, q_a + (size_t)t * S,
                      lq_a ? lq_a + (size_t)t * S : nullptr, am_a ? am_a + (size_t)t * F : nullptr, lane,
                      sm.xp >= 0 ? base + sm.xp + (size_t)t * Sp : nullptr, (R)lambda);
    }
    __syncthreads();
    R *tmp = cur; cur = nxt; nxt = tmp;
  }
}

template <typename R>
int launch_warp_t(const BiCall &c, bi_model *mut) {
  const bi_model *md = c.model;
  const BiDev &h = md->h;
  const bool window = c.algo != BI_ALGO_FILTER;
  WarpSmem sm;
  sm.md_bytes = (int)((sizeof(BiDev) + 15) & ~(size_t)15);
  int o = 0;
  sm.o_ell = o; o += h.Sp;
  sm.o_lpri = o; o += window ? 0 : h.Sp;
  sm.o_q0 = o; o += window ? 0 : h.Sp;
  sm.o_q1 = o; o += window ? 0 : h.Sp;
  // the two buffers the levels' partial tensors alternate between, rows at their padded strides
  int v0 = 4, v1 = 4;
  for (int gi = 0; gi < h.ngroups; ++gi)
    for (int l = 0; l + 1 < h.grp[gi].rank; ++l) {
      const BiLevel &lv = h.grp[gi].lev[l];
      const int out = (lv.nrows / lv.dim[lv.ndig - 1]) * bi_row_stride(lv.out_npad, (int)sizeof(R));
      (l % 2 == 0 ? v0 : v1) = std::max(l % 2 == 0 ? v0 : v1, out);
    }
  sm.o_V0 = o; o += bi_pad4(v0);
  sm.o_V1 = o; o += bi_pad4(v1);
  sm.o_sl = o; o += (int)(BI_MAX_M * sizeof(void *) / sizeof(R));
  const bool damped = c.lambda != 1.0;
  sm.o_xp = (!window && damped) ? o : -1;
  if (!window && damped) o += h.Sp;
  sm.o_Y = -1;
  sm.o_W = -1;
  sm.dtab = -1;
  int ysum = 0;
  bool four = true;   // (a table entry holds four parents' offsets)
  if (window && h.has_bdep) {
    for (int f = 0; f < h.F; ++f) {
      ysum += h.PB[f];
      four = four && h.bdep_len[f] <= 4;
    }
    sm.o_Y = o;
    o += bi_pad4(ysum);
    if (four && ysum <= 4096) {
      sm.o_W = o;
      o += bi_pad4(ysum);
    }
  }
  sm.per_warp = o;
  const size_t budget = 100 * 1024;  // at least two CTAs per SM
  size_t shared_elems = 0;
  if (window) {
    sm.q = 0;
    shared_elems = 2 * (size_t)c.T * h.Sp;
    sm.obs = (int)shared_elems;
    shared_elems += (size_t)bi_pad4((int)(((size_t)c.T * h.M * sizeof(int32_t) + sizeof(R) - 1) / sizeof(R)) + 1);
    sm.xp = damped ? (int)shared_elems : -1;
    if (damped) shared_elems += (size_t)c.T * h.Sp;
    if (sm.o_W >= 0) {
      sm.dtab = (int)shared_elems;
      shared_elems += (size_t)bi_pad4((int)(((size_t)ysum * sizeof(uint32_t) + sizeof(R) - 1) / sizeof(R)));
    }
  } else {
    sm.xp = -1;
    sm.q = 0;
    sm.obs = 0;
  }
  sm.warp0 = (int)shared_elems;
  auto bytes_for = [&](int w) { return (size_t)sm.md_bytes + (shared_elems + (size_t)w * sm.per_warp) * sizeof(R); };
  // warps per CTA: the count that keeps the most useful warps resident per SM
  // (registers: 128 per thread; shared memory: 227 KB; steps per warp rounded up)
  int W = 1;
  if (window) {
    double best = -1.0;
    for (int w = 1; w <= 16 && w <= c.T; ++w) {
      const size_t b = bytes_for(w);
      if (b > (size_t)md->max_smem_optin - 1024) break;
      const int rounds = (c.T + w - 1) / w;
      const int by_regs = 65536 / (128 * 32 * w), by_smem = (int)((size_t)(227 * 1024) / (b + 1024));
      const int blocks = std::min(std::min(by_regs, by_smem), 32);
      const double score = (double)blocks * w * ((double)c.T / (rounds * w));
      if (score > best + 1e-9) { best = score; W = w; }
    }
  } else {
    W = 4;
    while (W > 1 && bytes_for(W) > budget) --W;
  }
  if (bytes_for(W) > (size_t)md->max_smem_optin - 1024) return BI_ERR_UNSUPPORTED;
  sm.W = W;
  sm.total_bytes = (int)bytes_for(W);
  const bool f64 = sizeof(R) == 8;
  const char *name;
  cudaError_t e;
  if (!window) {
    auto kern = bi_warp_filter_kernel<R>;
    e = cudaFuncSetAttribute((const void *)kern, cudaFuncAttributeMaxDynamicSharedMemorySize, sm.total_bytes);
    if (e != cudaSuccess) return BI_ERR_CUDA;
    kern<<<(c.N + W - 1) / W, W * 32, sm.total_bytes, c.stream>>>(md->d, c.N, c.T, c.obs, c.act, c.q_prev,
                                                                   c.act_prev, c.carry_in, c.carry_out, c.lambda, c.K,
                                                                   c.q_out, c.logq_out, c.argmax_out, sm);
    name = f64 ? "warp_filter_f64" : "warp_filter_f32";
  } else if (c.algo == BI_ALGO_VMP) {
    auto kern = bi_warp_window_kernel<R, BI_ALGO_VMP>;
    e = cudaFuncSetAttribute((const void *)kern, cudaFuncAttributeMaxDynamicSharedMemorySize, sm.total_bytes);
    if (e != cudaSuccess) return BI_ERR_CUDA;
    kern<<<c.N, W * 32, sm.total_bytes, c.stream>>>(md->d, c.N, c.T, c.obs, c.act, c.q_init, c.lnprior, c.lambda, c.K,
                                                    c.q_out, c.logq_out, c.argmax_out, sm);
    name = f64 ? "warp_vmp_f64" : "warp_vmp_f32";
  } else {
    auto kern = bi_warp_window_kernel<R, BI_ALGO_MMP>;
    e = cudaFuncSetAttribute((const void *)kern, cudaFuncAttributeMaxDynamicSharedMemorySize, sm.total_bytes);
    if (e != cudaSuccess) return BI_ERR_CUDA;
    kern<<<c.N, W * 32, sm.total_bytes, c.stream>>>(md->d, c.N, c.T, c.obs, c.act, c.q_init, c.lnprior, c.lambda, c.K,
                                                    c.q_out, c.logq_out, c.argmax_out, sm);
    name = f64 ? "warp_mmp_f64" : "warp_mmp_f32";
  }
  if (cudaGetLastError() != cudaSuccess) return BI_ERR_CUDA;
  mut->launches += 1;
  mut->last_kernel = name;
  return BI_OK;
}

}  // namespace

// BI_ERR_UNSUPPORTED when a single warp's scratch does not fit in shared memory
int bi_launch_warp(const BiCall &c, bi_model *mut) {
  return c.model->arith == BI_ARITH_F64 ? launch_warp_t<double>(c, mut) : launch_warp_t<float>(c, mut);
}
