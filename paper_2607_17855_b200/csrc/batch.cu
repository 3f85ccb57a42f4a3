// Batched window kernels (VMP / MMP) for agents that share one model.
//
// With a shared model, every (agent, step) whose observation of modality i is
// the same outcome o contracts the SAME slice ln A_i[o] against its own
// beliefs.  The calls are therefore organised iteration by iteration over all
// agents at once: (agent, step) units are bucketed by observed outcome per
// modality (once per call), and in each iteration a CTA stages one slice in
// shared memory and 128 units of that bucket contract against it, one thread
// per unit with every accumulator in registers.  A slice row is then one
// broadcast shared-memory load for the whole warp, the row's index arithmetic
// is shared by all units, and the leave-one-out messages of all the group's
// factors (Section IV, marginalisation) come out of a single pass over the
// slice.  A second kernel per iteration adds the transition messages and takes
// the softmax per unit (Jacobi over steps and factors, Appendix A-2).
//
// Compiled for the dependency-group shapes in BI_BATCH_SHAPES; other models use
// the warp-per-step kernels.
#include <algorithm>
#include <cstring>

#include "bi_internal.h"
#include "tile3.cuh"

namespace {

constexpr int kTU = 128;   // most units per contraction CTA (the call picks 32, 64 or 128)

// packed dims of the compiled group shapes: rank, then the axis sizes (last axis unpadded)
#define BI_BATCH_SHAPES(X) \
  X(0, 4, 10, 10, 6, 8)    \
  X(1, 3, 10, 6, 8, 0)     \
  X(2, 2, 10, 8, 0, 0)     \
  X(3, 2, 10, 10, 0, 0)    \
  X(4, 3, 3, 2, 4, 0)      \
  X(5, 2, 5, 3, 0, 0)

struct BatchMember {
  const void *logA;        // packed [m][P_pad]
  int32_t m, P_pad, modality, shape, rank;
  int32_t offp[4];         // padded belief offsets of the group's axes, packed order
  int32_t task0;           // first task slot of this member
};

struct BatchParams {
  BatchMember mem[BI_MAX_M];
  int32_t nmem;            // members of rank >= 2
  int32_t NU, Sp, ntask, tu;   // tu: units per contraction CTA
  const int32_t *perm;     // [nmem][NU] unit ids ordered by observed outcome
  const int4 *task;        // [ntask] (outcome, first position, count, unused)
  void *ellp;              // [nmem][NU][Sp] partial likelihood messages
  void *qbuf;              // [2][NU][Sp] beliefs
};

// ---- one unit against one slice: every message of the group in one pass ----
// L: the slice in shared memory, rows of NCP; q / out: this unit's beliefs and
// message area (padded layout); o0..: offsets of the axes' factors.

template <typename R, int N1, int NC>
__device__ __forceinline__ void contract2(const R *__restrict__ L, const R *__restrict__ q, R *__restrict__ out,
                                          const int32_t *o) {
  constexpr int NCP = (NC + 3) & ~3;
  R qc[NC], accc[NC];
#pragma unroll
  for (int c = 0; c < NC; ++c) { qc[c] = q[o[1] + c]; accc[c] = (R)0; }
  for (int s1 = 0; s1 < N1; ++s1) {
    const R q1 = q[o[0] + s1];
    const R *row = L + s1 * NCP;
    R v0 = (R)0, v1 = (R)0;
#pragma unroll
    for (int c = 0; c < NC; ++c) {
      const R x = row[c];
      if (c & 1) v1 = fma(x, qc[c], v1); else v0 = fma(x, qc[c], v0);
      accc[c] = fma(q1, x, accc[c]);
    }
    out[o[0] + s1] = v0 + v1;
  }
#pragma unroll
  for (int c = 0; c < NC; ++c) out[o[1] + c] = accc[c];
}

template <typename R, int N1, int N2, int NC>
__device__ __forceinline__ void contract3(const R *__restrict__ L, const R *__restrict__ q, R *__restrict__ out,
                                          const int32_t *o) {
  constexpr int NCP = (NC + 3) & ~3;
  R q2[N2], qc[NC], acc2[N2], accc[NC];
#pragma unroll
  for (int i = 0; i < N2; ++i) { q2[i] = q[o[1] + i]; acc2[i] = (R)0; }
#pragma unroll
  for (int c = 0; c < NC; ++c) { qc[c] = q[o[2] + c]; accc[c] = (R)0; }
  for (int s1 = 0; s1 < N1; ++s1) {
    const R q1 = q[o[0] + s1];
    R a1 = (R)0;
#pragma unroll
    for (int s2 = 0; s2 < N2; ++s2) {
      const R *row = L + (s1 * N2 + s2) * NCP;
      const R w = q1 * q2[s2];
      R v0 = (R)0, v1 = (R)0;
#pragma unroll
      for (int c = 0; c < NC; ++c) {
        const R x = row[c];
        if (c & 1) v1 = fma(x, qc[c], v1); else v0 = fma(x, qc[c], v0);
        accc[c] = fma(w, x, accc[c]);
      }
      const R v = v0 + v1;
      acc2[s2] = fma(q1, v, acc2[s2]);
      a1 = fma(q2[s2], v, a1);
    }
    out[o[0] + s1] = a1;
  }
#pragma unroll
  for (int i = 0; i < N2; ++i) out[o[1] + i] = acc2[i];
#pragma unroll
  for (int c = 0; c < NC; ++c) out[o[2] + c] = accc[c];
}

template <typename R, int N1, int N2, int N3, int NC>
__device__ __forceinline__ void contract4(const R *__restrict__ L, const R *__restrict__ q, R *__restrict__ out,
                                          const int32_t *o) {
  constexpr int NCP = (NC + 3) & ~3;
  R q2[N2], q3[N3], qc[NC], acc2[N2], acc3[N3], accc[NC];
#pragma unroll
  for (int i = 0; i < N2; ++i) { q2[i] = q[o[1] + i]; acc2[i] = (R)0; }
#pragma unroll
  for (int i = 0; i < N3; ++i) { q3[i] = q[o[2] + i]; acc3[i] = (R)0; }
#pragma unroll
  for (int c = 0; c < NC; ++c) { qc[c] = q[o[3] + c]; accc[c] = (R)0; }
  for (int s1 = 0; s1 < N1; ++s1) {
    const R q1 = q[o[0] + s1];
    R a1 = (R)0;
#pragma unroll
    for (int s2 = 0; s2 < N2; ++s2) {
      const R w12 = q1 * q2[s2];
      R v2 = (R)0;
#pragma unroll
      for (int s3 = 0; s3 < N3; ++s3) {
        const R *row = L + ((s1 * N2 + s2) * N3 + s3) * NCP;
        const R w = w12 * q3[s3];
        R v0 = (R)0, v1 = (R)0;
#pragma unroll
        for (int c = 0; c < NC; ++c) {
          const R x = row[c];
          if (c & 1) v1 = fma(x, qc[c], v1); else v0 = fma(x, qc[c], v0);
          accc[c] = fma(w, x, accc[c]);
        }
        const R v = v0 + v1;
        acc3[s3] = fma(w12, v, acc3[s3]);
        v2 = fma(q3[s3], v, v2);
      }
      acc2[s2] = fma(q1, v2, acc2[s2]);
      a1 = fma(q2[s2], v2, a1);
    }
    out[o[0] + s1] = a1;
  }
#pragma unroll
  for (int i = 0; i < N2; ++i) out[o[1] + i] = acc2[i];
#pragma unroll
  for (int i = 0; i < N3; ++i) out[o[2] + i] = acc3[i];
#pragma unroll
  for (int c = 0; c < NC; ++c) out[o[3] + c] = accc[c];
}

template <typename R, int RANK, int D0, int D1, int D2, int D3>
__device__ __forceinline__ void contract_shape(const R *L, const R *q, R *out, const int32_t *o) {
  if constexpr (RANK == 2) contract2<R, D0, D1>(L, q, out, o);
  else if constexpr (RANK == 3) contract3<R, D0, D1, D2>(L, q, out, o);
  else contract4<R, D0, D1, D2, D3>(L, q, out, o);
}

// ---- bucket the units of one modality by observed outcome (once per call) ----
// One CTA per member.  Writes perm[mi][*] (unit ids grouped by outcome) and the
// member's task slots: chunks of at most kTU units of one outcome.
__global__ void __launch_bounds__(1024)
bi_batch_bucket_kernel(BatchParams P, const int32_t *__restrict__ obs, int M, uint32_t *status,
                       int32_t *perm, int4 *task) {
  extern __shared__ int32_t sh[];       // count[m] | cursor[m]
  const BatchMember &mm = P.mem[blockIdx.x];
  const int m = mm.m, NU = P.NU;
  int32_t *count = sh, *cursor = sh + m;
  for (int i = threadIdx.x; i < m; i += blockDim.x) count[i] = 0;
  __syncthreads();
  for (int u = threadIdx.x; u < NU; u += blockDim.x) {
    const int o = clamp_flag(obs[(size_t)u * M + mm.modality], m, status, BI_FLAG_OBS_RANGE);
    atomicAdd(&count[o], 1);
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    int pos = 0, slot = mm.task0;
    const int tu = P.tu;
    const int slot_end = mm.task0 + (NU + tu - 1) / tu + m;
    for (int o = 0; o < m; ++o) {
      cursor[o] = pos;
      for (int b = 0; b < count[o]; b += tu) task[slot++] = make_int4(o, pos + b, min(tu, count[o] - b), 0);
      pos += count[o];
    }
    for (; slot < slot_end; ++slot) task[slot] = make_int4(0, 0, 0, 0);
  }
  __syncthreads();
  int32_t *pm = perm + (size_t)blockIdx.x * NU;
  for (int u = threadIdx.x; u < NU; u += blockDim.x) {
    int o = obs[(size_t)u * M + mm.modality];
    o = o < 0 ? 0 : (o >= m ? m - 1 : o);
    pm[atomicAdd(&cursor[o], 1)] = u;
  }
}

// ---- contraction: one task = one slice, up to kTU units, one thread per unit ----
template <typename R>
__global__ void __launch_bounds__(kTU)
bi_batch_contract_kernel(BatchParams P, int cur) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  R *L = reinterpret_cast<R *>(smem_raw);
  int mi = 0;
  while (mi + 1 < P.nmem && (int)blockIdx.x >= P.mem[mi + 1].task0) ++mi;
  const BatchMember &mm = P.mem[mi];
  const int4 tk = P.task[blockIdx.x];
  if (tk.z == 0) return;
  {  // stage the slice of outcome tk.x
    const R *src = (const R *)mm.logA + (size_t)tk.x * mm.P_pad;
    for (int i = threadIdx.x * 4; i < mm.P_pad; i += blockDim.x * 4) {
      Vec4<R> v = ldg4(src + i);
      *reinterpret_cast<Vec4<R> *>(L + i) = v;
    }
  }
  __syncthreads();
  if ((int)threadIdx.x >= tk.z) return;
  const int unit = P.perm[(size_t)mi * P.NU + tk.y + threadIdx.x];
  const R *q = (const R *)P.qbuf + ((size_t)cur * P.NU + unit) * P.Sp;
  R *out = (R *)P.ellp + ((size_t)mi * P.NU + unit) * P.Sp;
  switch (mm.shape) {
#define X(ID, RANK, D0, D1, D2, D3) \
  case ID: contract_shape<R, RANK, D0, D1, D2, D3>(L, q, out, mm.offp); break;
    BI_BATCH_SHAPES(X)
#undef X
    default: break;
  }
}

// ---- per unit: sum the partial messages, add rank-1 slices and transition messages, softmax ----
struct UpdateArgs {
  const int32_t *obs, *act;
  float *q_out, *logq_out;
  int32_t *argmax_out;
  int32_t T, cur, final;
  uint32_t fmask[BI_MAX_F];   // members (rank >= 2) whose group contains factor f
  uint32_t r1mask[BI_MAX_F];  // descriptor members (modalities) that depend on factor f alone
};

template <typename R>
__device__ __forceinline__ R col_dot_g(const R *__restrict__ col, int npad, const R *__restrict__ q, int n) {
  R s0 = (R)0, s1 = (R)0;
  int r = 0;
  for (; r + 1 < n; r += 2) {
    s0 = fma(__ldg(col + (size_t)r * npad), q[r], s0);
    s1 = fma(__ldg(col + (size_t)(r + 1) * npad), q[r + 1], s1);
  }
  if (r < n) s0 = fma(__ldg(col + (size_t)r * npad), q[r], s0);
  return s0 + s1;
}

// LW lanes per unit (the smallest power of two that holds the largest factor),
// one lane per state: for each factor in turn the lanes gather the partial
// messages, add the single-factor slices and the two transition messages, and
// normalise with shuffles inside the lane group.
struct FactorInfo {
  int32_t n, np, op, off, U;
  uint32_t fmask, r1mask;
  int32_t pad_;
};

template <int LW, typename R>
__device__ __forceinline__ R lane_group_sum(R v) {
#pragma unroll
  for (int o = LW / 2; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
template <int LW, typename R>
__device__ __forceinline__ R lane_group_max(R v) {
#pragma unroll
  for (int o = LW / 2; o > 0; o >>= 1) v = bi_max(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}

template <typename R, int ALGO, int LW>
__global__ void __launch_bounds__(128)
bi_batch_update_kernel(const BiDev *__restrict__ mdp, BatchParams P, UpdateArgs A) {
  __shared__ FactorInfo fi[BI_MAX_F];
  const BiDev &md = *mdp;
  constexpr int UPB = 128 / LW;   // units per CTA
  const int F = md.F, Sp = md.Sp, S = md.S, M = md.M, T = A.T, NU = P.NU;
  if ((int)threadIdx.x < F) {
    const int f = threadIdx.x;
    FactorInfo x;
    x.n = md.n[f]; x.np = md.npad[f]; x.op = md.offp[f]; x.off = md.off[f]; x.U = md.U[f];
    x.fmask = A.fmask[f]; x.r1mask = A.r1mask[f]; x.pad_ = 0;
    fi[f] = x;
  }
  __syncthreads();
  const int sub = threadIdx.x / LW, s = threadIdx.x % LW;
  int unit = blockIdx.x * UPB + sub;
  const bool live = unit < NU;    // dead groups shadow the last unit so that whole warps reach the shuffles
  if (!live) unit = NU - 1;
  const int a = unit / T, t = unit - a * T;
  const R *qc = (const R *)P.qbuf + (size_t)A.cur * NU * Sp;
  R *qn = (R *)P.qbuf + ((size_t)(A.cur ^ 1) * NU + unit) * Sp;
  const int32_t *ob = A.obs + (size_t)unit * M;
  // acp[f]: action into step t (t > 0); acp[F + f]: action out of it (t + 1 < T)
  const int32_t *acp = A.act + ((ptrdiff_t)a * (T - 1) + (t - 1)) * F;
  for (int f = 0; f < F; ++f) {
    const FactorInfo I = fi[f];
    const int n = I.n, np = I.np, op = I.op;
    R x = -bi_inf<R>();
    if (s < n) {
      x = (R)0;
      for (uint32_t mk = I.fmask; mk; mk &= mk - 1) {
        const int j = __ffs(mk) - 1;
        x += ((const R *)P.ellp)[((size_t)j * NU + unit) * Sp + op + s];
      }
      for (uint32_t mk = I.r1mask; mk; mk &= mk - 1) {   // single-factor modalities: the slice is the message
        const BiMember &mm = md.mem[__ffs(mk) - 1];
        const int o = clamp_flag(ob[mm.modality], mm.m, md.status, BI_FLAG_OBS_RANGE);
        x += __ldg((const R *)mm.logA + (size_t)o * mm.P_pad + s);
      }
      if (t == 0) {
        x += ((const R *)md.logD[f])[s];
      } else {
        const int u = clamp_flag(acp[f], I.U, md.status, BI_FLAG_ACT_RANGE);
        const R *M0 = (const R *)(ALGO == BI_ALGO_VMP ? md.logBt[f] : md.BfT[f]);   // [previous][next]
        const R v = col_dot_g<R>(M0 + (size_t)u * n * np + s, np, qc + (size_t)(unit - 1) * Sp + op, n);
        x += ALGO == BI_ALGO_VMP ? v : (R)0.5 * bi_log_inline(bi_max(v, (R)BI_EPS));
      }
      if (t + 1 < T) {
        const int u = clamp_flag(acp[F + f], I.U, md.status, BI_FLAG_ACT_RANGE);
        const R *M1 = (const R *)(ALGO == BI_ALGO_VMP ? md.logB[f] : md.BdagT[f]);   // [next][previous]
        const R v = col_dot_g<R>(M1 + (size_t)u * n * np + s, np, qc + (size_t)(unit + 1) * Sp + op, n);
        x += ALGO == BI_ALGO_VMP ? v : (R)0.5 * bi_log_inline(bi_max(v, (R)BI_EPS));
      }
    }
    // any shift near the maximum keeps the exponentials in range; the last iterate takes the exact one
    const R mx = A.final ? lane_group_max<LW>(x) : (R)lane_group_max<LW>((float)x);
    const R e = s < n ? bi_exp_inline(x - mx) : (R)0;
    const R z = lane_group_sum<LW>(e);
    const R q = e * bi_rcp(z);
    if (live && s < np) qn[op + s] = q;
    if (A.final) {
      if (live && s < n) {
        A.q_out[(size_t)unit * S + I.off + s] = (float)q;
        if (A.logq_out) A.logq_out[(size_t)unit * S + I.off + s] = (float)(x - mx - bi_log(z));
      }
      if (A.argmax_out) {
        unsigned b = __ballot_sync(0xffffffffu, s < n && x == mx);
        if (LW < 32) b = (b >> ((threadIdx.x & 31) - s)) & ((1u << (LW & 31)) - 1u);
        if (live && s == 0) A.argmax_out[(size_t)unit * F + f] = __ffs(b) - 1;
      }
    }
  }
}

template <typename R>
__global__ void bi_batch_init_kernel(const BiDev *__restrict__ mdp, R *q, int NU) {
  const BiDev &md = *mdp;
  const size_t total = (size_t)NU * md.Sp;
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
    const int p = (int)(i % md.Sp);
    int f = 0;
    while (f + 1 < md.F && p >= md.offp[f + 1]) ++f;
    q[i] = (p - md.offp[f]) < md.n[f] ? (R)1 / (R)md.n[f] : (R)0;
  }
}

int shape_of(const BiGroup &g) {
  const int d[4] = {g.rank > 0 ? g.dim[0] : 0, g.rank > 1 ? g.dim[1] : 0, g.rank > 2 ? g.dim[2] : 0,
                    g.rank > 3 ? g.dim[3] : 0};
#define X(ID, RANK, D0, D1, D2, D3) \
  if (g.rank == RANK && d[0] == D0 && d[1] == D1 && d[2] == D2 && d[3] == D3) return ID;
  BI_BATCH_SHAPES(X)
#undef X
  return -1;
}

size_t up256(size_t x) { return (x + 255) & ~(size_t)255; }

template <typename R>
int launch_batch_t(const BiCall &c, bi_model *mut) {
  const bi_model *md = c.model;
  const BiDev &h = md->h;
  const int NU = c.N * c.T;
  BatchParams P;
  memset(&P, 0, sizeof(P));
  // units per contraction CTA: small enough that the heaviest member alone gives every SM a CTA
  int tu = kTU;
  while (tu > 32 && NU / tu < md->sm_count) tu >>= 1;
  P.tu = tu;
  UpdateArgs A;
  memset(&A, 0, sizeof(A));
  // members of rank >= 2, largest slices first (their tasks are the longest)
  int order[BI_MAX_M], cnt = 0;
  for (int gi = 0; gi < h.ngroups; ++gi) {
    const BiGroup &g = h.grp[gi];
    if (g.rank < 2) continue;
    if (g.rank > 4 || shape_of(g) < 0) return BI_ERR_UNSUPPORTED;
    for (int mi = g.mem_begin; mi < g.mem_end; ++mi) order[cnt++] = mi;
  }
  if (cnt == 0) return BI_ERR_UNSUPPORTED;
  std::sort(order, order + cnt, [&](int x, int y) { return h.mem[x].P_pad > h.mem[y].P_pad; });
  size_t max_slice = 0;
  int max_m = 1, ntask = 0;
  for (int j = 0; j < cnt; ++j) {
    const BiMember &mm = h.mem[order[j]];
    int gi = 0;
    while (!(order[j] >= h.grp[gi].mem_begin && order[j] < h.grp[gi].mem_end)) ++gi;
    const BiGroup &g = h.grp[gi];
    BatchMember &bm = P.mem[j];
    bm.logA = mm.logA; bm.m = mm.m; bm.P_pad = mm.P_pad; bm.modality = mm.modality;
    bm.shape = shape_of(g); bm.rank = g.rank;
    for (int k = 0; k < g.rank; ++k) {
      bm.offp[k] = h.offp[g.axis[k]];
      A.fmask[g.axis[k]] |= 1u << j;
    }
    bm.task0 = ntask;
    ntask += (NU + tu - 1) / tu + mm.m;
    max_slice = std::max(max_slice, (size_t)mm.P_pad * sizeof(R));
    max_m = std::max(max_m, mm.m);
  }
  if (max_slice > (size_t)md->max_smem_optin - 1024 || max_m > 4096) return BI_ERR_UNSUPPORTED;
  P.nmem = cnt; P.NU = NU; P.Sp = h.Sp; P.ntask = ntask;

  // ---- workspace (stream-ordered; kept in the handle and grown on demand)
  const size_t b_perm = up256((size_t)cnt * NU * sizeof(int32_t));
  const size_t b_task = up256((size_t)ntask * sizeof(int4));
  const size_t b_ellp = up256((size_t)cnt * NU * h.Sp * sizeof(R));
  const size_t b_q = up256(2 * (size_t)NU * h.Sp * sizeof(R));
  const size_t need = b_perm + b_task + b_ellp + b_q;
  if (mut->ws_bytes < need) {
    if (mut->ws && cudaFreeAsync(mut->ws, c.stream) != cudaSuccess) return BI_ERR_CUDA;
    mut->ws = nullptr;
    mut->ws_bytes = 0;
    void *pnew = nullptr;
    if (cudaMallocAsync(&pnew, need, c.stream) != cudaSuccess) {
      cudaGetLastError();
      return BI_ERR_ALLOC;
    }
    mut->ws = pnew;
    mut->ws_bytes = need;
  }
  unsigned char *w = static_cast<unsigned char *>(mut->ws);
  int32_t *perm = reinterpret_cast<int32_t *>(w);
  int4 *task = reinterpret_cast<int4 *>(w + b_perm);
  P.perm = perm;
  P.task = task;
  P.ellp = w + b_perm + b_task;
  P.qbuf = w + b_perm + b_task + b_ellp;
  A.obs = c.obs; A.act = c.act; A.q_out = c.q_out; A.logq_out = c.logq_out; A.argmax_out = c.argmax_out;
  A.T = c.T;

  bi_batch_init_kernel<R><<<256, 256, 0, c.stream>>>(md->d, (R *)P.qbuf, NU);
  bi_batch_bucket_kernel<<<cnt, 1024, 2 * max_m * sizeof(int32_t), c.stream>>>(P, c.obs, h.M, h.status, perm, task);
  auto contract = bi_batch_contract_kernel<R>;
  if (cudaFuncSetAttribute((const void *)contract, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)max_slice) !=
      cudaSuccess)
    return BI_ERR_CUDA;
  for (int gi = 0; gi < h.ngroups; ++gi) {
    const BiGroup &g = h.grp[gi];
    if (g.rank != 1) continue;
    for (int mi = g.mem_begin; mi < g.mem_end; ++mi) A.r1mask[g.axis[0]] |= 1u << mi;
  }
  int nmax = 1;
  for (int f = 0; f < h.F; ++f) nmax = std::max(nmax, (int)h.n[f]);
  const int lw = nmax <= 8 ? 8 : nmax <= 16 ? 16 : 32, upb = 128 / lw;
  void (*update)(const BiDev *, BatchParams, UpdateArgs);
  if (c.algo == BI_ALGO_VMP)
    update = lw == 8 ? bi_batch_update_kernel<R, BI_ALGO_VMP, 8>
                     : lw == 16 ? bi_batch_update_kernel<R, BI_ALGO_VMP, 16> : bi_batch_update_kernel<R, BI_ALGO_VMP, 32>;
  else
    update = lw == 8 ? bi_batch_update_kernel<R, BI_ALGO_MMP, 8>
                     : lw == 16 ? bi_batch_update_kernel<R, BI_ALGO_MMP, 16> : bi_batch_update_kernel<R, BI_ALGO_MMP, 32>;
  for (int k = 0; k < c.K; ++k) {
    const int cur = k & 1;
    contract<<<ntask, tu, max_slice, c.stream>>>(P, cur);
    A.cur = cur;
    A.final = (k == c.K - 1);
    update<<<(NU + upb - 1) / upb, 128, 0, c.stream>>>(md->d, P, A);
  }
  if (cudaGetLastError() != cudaSuccess) return BI_ERR_CUDA;
  mut->launches += 2 + 2 * c.K;
  const bool f64 = sizeof(R) == 8;
  mut->last_kernel = c.algo == BI_ALGO_VMP ? (f64 ? "batch_vmp_f64" : "batch_vmp_f32")
                                           : (f64 ? "batch_mmp_f64" : "batch_mmp_f32");
  return BI_OK;
}

}  // namespace

// Applies to window calls on a shared model with enough (agent, step) units to
// fill the machine and whose dependency groups all have a compiled shape.
int bi_launch_batch(const BiCall &c, bi_model *mut) {
  const bi_model *md = c.model;
  if (c.algo == BI_ALGO_FILTER || md->h.G != 1) return BI_ERR_UNSUPPORTED;
  if ((long long)c.N * c.T < 2048) return BI_ERR_UNSUPPORTED;
  return md->arith == BI_ARITH_F64 ? launch_batch_t<double>(c, mut) : launch_batch_t<float>(c, mut);
}
