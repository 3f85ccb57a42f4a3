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
// The contraction has two forms: fully unrolled code for the dependency-group
// shapes in BI_BATCH_SHAPES (every accumulator in registers), and a form for any
// shape of rank 2..5 that is compiled only for the padded size of the last axis
// (its accumulators in registers, those of the outer axes in per-thread columns
// of shared memory, the outer loops an odometer shared by the whole CTA).
#include <algorithm>
#include <cstring>

#include <type_traits>

#include "bi_internal.h"
#include "tile3.cuh"

namespace {

// Programmatic dependent launch: the iteration loop queues its kernels so that the next one may be
// scheduled while the previous one drains.  A kernel first does what needs none of its
// predecessor's results (its task, the slice copy, index loads), then waits for the predecessor to
// complete (bi_grid_wait; a no-op when launched without the attribute) and only then lets its own
// successor be scheduled: when a kernel starts, everything before its predecessor is complete.
__device__ __forceinline__ void bi_grid_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void bi_grid_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;"); }

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
  int32_t offp[BI_MAX_RANK];   // padded belief offsets of the group's axes, packed order
  int32_t dim[BI_MAX_RANK];    // axis sizes, packed order (last one unpadded)
  int32_t ooff[BI_MAX_RANK];   // start of each outer axis in the per-thread shared-memory columns
  int32_t ncp, rows;       // padded last axis; rows = product of the outer axes
  int64_t gstride;         // elements per agent's model (per-agent models), 0 when shared
  int32_t task0;           // first task slot of this member
  int32_t split;           // unrolled forms: threads per unit (1, 2 or 4), each taking a range of the first axis
};

struct BatchParams {
  BatchMember mem[BI_MAX_M];
  int32_t nmem;            // members of rank >= 2
  int32_t NU, Sp, ntask, tu;   // tu: units per contraction CTA
  int32_t sc_off;          // unrolled forms: element offset of the split tasks' scratch columns behind the slice
  int32_t lbuf, so_max;    // any-shape form: elements of the slice staging buffer; most outer states of a member
  const int32_t *perm;     // [nmem][NU] unit ids ordered by observed outcome
  const int4 *task;        // [ntask] (outcome, first position, count, unused)
  void *ellp;              // [nmem][NU][Sp] partial likelihood messages
  void *qbuf;              // [2][NU][Sp] beliefs
  uint32_t *status;        // the handle's status word
  const int32_t *obs;      // [NU][M] (per-agent models: every unit reads its own slice)
  int32_t M, T;
  int32_t drop_copy;       // testing aid: the contraction announces its slice copy and does not issue it
};

// ---- one unit against one slice: every message of the group in one pass ----
// L: the slice in shared memory, rows of NCP; q / out: this unit's beliefs and
// message area (padded layout); o0..: offsets of the axes' factors.

// SPLIT > 1: the threads of `SPLIT` different warps share a unit, each taking a range of the first
// axis (part = which); a thread writes the first axis' messages of its range, and its partial messages
// of the other axes to the scratch columns sc[i * nt + tid], which the caller adds in a fixed order.
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

template <typename R, int N1, int N2, int NC, int SPLIT = 1>
__device__ __forceinline__ void contract3(const R *__restrict__ L, const R *__restrict__ q, R *__restrict__ out,
                                          const int32_t *o, int part = 0, bool wr = true, R *sc = nullptr, int nt = 0) {
  const int sa = part * N1 / SPLIT, sb = (part + 1) * N1 / SPLIT;
  constexpr int NCP = (NC + 3) & ~3;
  R q2[N2], qc[NC], acc2[N2], accc[NC];
#pragma unroll
  for (int i = 0; i < N2; ++i) { q2[i] = q[o[1] + i]; acc2[i] = (R)0; }
#pragma unroll
  for (int c = 0; c < NC; ++c) { qc[c] = q[o[2] + c]; accc[c] = (R)0; }
  R q1n = q[o[0] + sa];   // (the first axis' belief is read one index ahead: its latency hides under the rows)
  for (int s1 = sa; s1 < sb; ++s1) {
    const R q1 = q1n;
    if (s1 + 1 < sb) q1n = q[o[0] + s1 + 1];
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
    if (wr) out[o[0] + s1] = a1;
  }
#pragma unroll
  for (int i = 0; i < N2; ++i) {
    if (SPLIT > 1) sc[i * nt] = acc2[i];
    else out[o[1] + i] = acc2[i];
  }
#pragma unroll
  for (int c = 0; c < NC; ++c) {
    if (SPLIT > 1) sc[(N2 + c) * nt] = accc[c];
    else out[o[2] + c] = accc[c];
  }
}

template <typename R, int N1, int N2, int N3, int NC, int SPLIT = 1>
__device__ __forceinline__ void contract4(const R *__restrict__ L, const R *__restrict__ q, R *__restrict__ out,
                                          const int32_t *o, int part = 0, bool wr = true, R *sc = nullptr, int nt = 0) {
  const int sa = part * N1 / SPLIT, sb = (part + 1) * N1 / SPLIT;
  constexpr int NCP = (NC + 3) & ~3;
  R q2[N2], q3[N3], qc[NC], acc2[N2], acc3[N3], accc[NC];
#pragma unroll
  for (int i = 0; i < N2; ++i) { q2[i] = q[o[1] + i]; acc2[i] = (R)0; }
#pragma unroll
  for (int i = 0; i < N3; ++i) { q3[i] = q[o[2] + i]; acc3[i] = (R)0; }
#pragma unroll
  for (int c = 0; c < NC; ++c) { qc[c] = q[o[3] + c]; accc[c] = (R)0; }
  R q1n = q[o[0] + sa];   // (read one index ahead, as above)
  for (int s1 = sa; s1 < sb; ++s1) {
    const R q1 = q1n;
    if (s1 + 1 < sb) q1n = q[o[0] + s1 + 1];
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
    if (wr) out[o[0] + s1] = a1;
  }
#pragma unroll
  for (int i = 0; i < N2; ++i) {
    if (SPLIT > 1) sc[i * nt] = acc2[i];
    else out[o[1] + i] = acc2[i];
  }
#pragma unroll
  for (int i = 0; i < N3; ++i) {
    if (SPLIT > 1) sc[(N2 + i) * nt] = acc3[i];
    else out[o[2] + i] = acc3[i];
  }
#pragma unroll
  for (int c = 0; c < NC; ++c) {
    if (SPLIT > 1) sc[(N2 + N3 + c) * nt] = accc[c];
    else out[o[3] + c] = accc[c];
  }
}

template <typename R, int RANK, int D0, int D1, int D2, int D3>
__device__ __forceinline__ void contract_shape(const R *L, const R *q, R *out, const int32_t *o, int split, int part,
                                               bool wr, R *sc, int nt) {
  if constexpr (RANK == 2) contract2<R, D0, D1>(L, q, out, o);
  else if constexpr (RANK == 3) {
    if (split == 1) contract3<R, D0, D1, D2>(L, q, out, o);
    else contract3<R, D0, D1, D2, 2>(L, q, out, o, part, wr, sc, nt);
  } else {
    if (split == 1) contract4<R, D0, D1, D2, D3>(L, q, out, o);
    else if (split == 2) contract4<R, D0, D1, D2, D3, 2>(L, q, out, o, part, wr, sc, nt);
    else contract4<R, D0, D1, D2, D3, 4>(L, q, out, o, part, wr, sc, nt);
  }
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
    const int tu = P.tu / mm.split;
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

// Per-agent models: no two units share a slice, so the "buckets" are just runs of consecutive units.
__global__ void bi_batch_identity_tasks_kernel(BatchParams P, int32_t *perm, int4 *task) {
  const int mi = blockIdx.y, NU = P.NU, tu = P.tu;
  const int nchunk = (NU + tu - 1) / tu;
  for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < NU; i += gridDim.x * blockDim.x)
    perm[(size_t)mi * NU + i] = i;
  for (int k = blockIdx.x * blockDim.x + threadIdx.x; k < nchunk + P.mem[mi].m; k += gridDim.x * blockDim.x)
    task[P.mem[mi].task0 + k] = k < nchunk ? make_int4(0, k * tu, min(tu, NU - k * tu), 0) : make_int4(0, 0, 0, 0);
}

// ---- contraction: one task = one slice, up to kTU units, one thread per unit ----
template <typename R>
__global__ void __launch_bounds__(kTU)
bi_batch_contract_kernel(BatchParams P, int cur, int first) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  R *L = reinterpret_cast<R *>(smem_raw);
  if (first) {   // the tasks were written by the kernel just before this one
    bi_grid_wait();
    bi_grid_launch_dependents();
  }
  int mi = 0;
  while (mi + 1 < P.nmem && (int)blockIdx.x >= P.mem[mi + 1].task0) ++mi;
  const BatchMember &mm = P.mem[mi];
  const int4 tk = P.task[blockIdx.x];
  if (tk.z == 0) {   // an unused task slot (an exiting CTA counts as having released its dependents)
    return;
  }
  // stage the slice of outcome tk.x: one bulk asynchronous copy, global -> shared, issued by one
  // thread; the others meanwhile look up their unit
  __shared__ __align__(8) unsigned long long bar;
  if (threadIdx.x == 0) bi_mbar_init(&bar, 1);
  __syncthreads();
  if (threadIdx.x == 0) {
    if (P.drop_copy) bi_mbar_expect(&bar, (uint32_t)(mm.P_pad * sizeof(R)));   // (testing aid: the copy never comes)
    else bi_bulk_load(L, (const R *)mm.logA + (size_t)tk.x * mm.P_pad, (uint32_t)(mm.P_pad * sizeof(R)), &bar);
  }
  // (a heavy member's units are shared by `split` threads, one in each of `split` groups of warps: a
  // warp's threads then still read the same slice row, a broadcast)
  const int upt = (int)blockDim.x / mm.split;   // units per task of this member
  const int ut = (int)threadIdx.x % upt, part = (int)threadIdx.x / upt;
  const bool has_unit = ut < tk.z;
  const int unit = has_unit ? P.perm[(size_t)mi * P.NU + tk.y + ut] : 0;
  const R *q = (const R *)P.qbuf + ((size_t)cur * P.NU + unit) * P.Sp;
  R *out = (R *)P.ellp + ((size_t)mi * P.NU + unit) * P.Sp;
  if (!first) {   // beliefs of the previous update, and the right to overwrite the messages it read
    bi_grid_wait();
    bi_grid_launch_dependents();
  }
  // a copy that does not arrive within the probe limit: the block reports it and leaves (nothing of
  // its own is in flight then; the call's outputs are invalid)
  if (!bi_mbar_wait(&bar, 0, P.drop_copy ? 256 : 1 << 18)) {
    if (threadIdx.x == 0) atomicOr(P.status, BI_FLAG_COPY_TIMEOUT);
    return;
  }
  // (in a split task the threads without a unit stay for the barrier below; they contract unit 0's
  // beliefs and write nothing)
  if (!has_unit && mm.split == 1) return;
  R *sc = L + P.sc_off + threadIdx.x;   // scratch columns behind the slice
  switch (mm.shape) {
#define X(ID, RANK, D0, D1, D2, D3) \
  case ID: contract_shape<R, RANK, D0, D1, D2, D3>(L, q, out, mm.offp, mm.split, part, has_unit, sc, (int)blockDim.x); break;
    BI_BATCH_SHAPES(X)
#undef X
    default: break;
  }
  if (mm.split > 1) {   // add the parts' partial messages of the axes after the first, part 0 first
    __syncthreads();
    if (part == 0 && has_unit) {
      const R *col = L + P.sc_off + ut;
      int idx = 0;
      for (int j = 1; j < mm.rank; ++j)
        for (int i = 0; i < mm.dim[j]; ++i, ++idx) {
          R sum = col[(size_t)idx * blockDim.x];
          for (int pp = 1; pp < mm.split; ++pp) sum += col[(size_t)idx * blockDim.x + pp * upt];
          out[mm.offp[j] + i] = sum;
        }
    }
  }
}

// ---- contraction for any shape: compiled for the padded last axis only ----
// Same arithmetic as the unrolled forms.  For a row of the slice (all outer
// indices fixed) v = sum_c L[row][c] q_c[c] and acc_c[c] += W L[row][c], with W
// the product of the outer beliefs.  v then climbs the outer axes from the
// innermost: at axis j the message accumulator of index s_j receives
// (product of the beliefs of axes before j) * v, the running sum p_{j-1}
// receives q_j[s_j] * v, and when s_j was the axis' last index that sum becomes
// the value handed to axis j - 1.  The indices are an odometer that is the same
// for every thread of a warp, so its branches are uniform and a slice row is a
// broadcast load.  qs / as: per-thread columns (state-major, thread-minor: no
// bank conflicts) holding the outer axes' beliefs and message accumulators.
//
// Small batches do not have enough units to fill the machine with one thread
// per unit, so a CTA is tu units x rs row splits: split r contracts the rows of
// a contiguous range of the first axis' indices for the same tu units, and the
// partial messages of the splits are added through shared memory at the end
// (fixed order: deterministic).
// PERUNIT (per-agent models): nothing is shared between units, so nothing is staged; every thread
// reads the rows of its own unit's slice straight from global memory (consecutive rows of one
// thread share cache lines, so L1 serves most of the loads).
template <typename R, int NCP, bool PERUNIT>
__device__ __forceinline__ void contract_rt(const BatchMember &mm, const R *__restrict__ slice, R *Lbuf, int lbuf,
                                            R *qs, R *as, int *unit_s, const BatchParams &P, int cur, int4 tk,
                                            int mi) {
  const int tid = threadIdx.x, nt = blockDim.x, tu = P.tu, rs = nt / tu;
  const int u = tid % tu, r = tid / tu;
  const bool has_unit = u < tk.z;
  const int unit = has_unit ? P.perm[(size_t)mi * P.NU + tk.y + u] : 0;
  if (r == 0) unit_s[u] = unit;
  const R *q = (const R *)P.qbuf + ((size_t)cur * P.NU + unit) * P.Sp;
  const int K1 = mm.rank - 1, NC = mm.dim[K1];
  R qc[NCP], accc[NCP];
#pragma unroll
  for (int c = 0; c < NCP; ++c) {
    qc[c] = (has_unit && c < NC) ? q[mm.offp[K1] + c] : (R)0;
    accc[c] = (R)0;
  }
  // (the outer axes' beliefs once per unit: the splits of a unit read the same column)
  for (int j = 0; j < K1; ++j)
    for (int sj = 0; sj < mm.dim[j]; ++sj) {
      if (r == 0) qs[(mm.ooff[j] + sj) * tu + u] = has_unit ? q[mm.offp[j] + sj] : (R)0;
      as[(mm.ooff[j] + sj) * nt + tid] = (R)0;
    }
  __syncthreads();
  // this split's range of the first axis, and of rows
  const int d0 = mm.dim[0], rps = mm.rows / d0;
  const int s0a = (int)((long long)r * d0 / rs), s0b = (int)((long long)(r + 1) * d0 / rs);
  const int row_a = s0a * rps, row_b = s0b * rps;
  const int most = ((d0 + rs - 1) / rs) * rps;   // rows of the largest split: the common trip count
  int dig[4] = {s0a < d0 ? s0a : 0, 0, 0, 0};
  R p[4] = {(R)0, (R)0, (R)0, (R)0}, Wp[4] = {(R)1, (R)1, (R)1, (R)1};
#pragma unroll
  for (int lv = 0; lv < 4; ++lv)
    if (lv < K1) Wp[lv] = (lv > 0 ? Wp[lv > 0 ? lv - 1 : 0] : (R)1) * qs[(mm.ooff[lv] + dig[lv]) * tu + u];
  const int lrows = PERUNIT ? most : lbuf / rs / NCP;   // rows of one split's staging area (PERUNIT: all at once)
  R *Lr = Lbuf + (size_t)r * (PERUNIT ? 0 : lrows) * NCP;
  __shared__ __align__(8) unsigned long long bar[8];   // one per split
  if (!PERUNIT && tid < rs) bi_mbar_init(&bar[tid], 1);
  uint32_t phase = 0;
  bool failed = false;
  const R *mine = nullptr;   // PERUNIT: this unit's slice
  if (PERUNIT && has_unit) {
    const int o = clamp_flag(P.obs[(size_t)unit * P.M + mm.modality], mm.m, P.status, BI_FLAG_OBS_RANGE);
    mine = (const R *)mm.logA + (size_t)(unit / P.T) * mm.gstride + (size_t)o * mm.P_pad;
  }
  for (int c0 = 0; c0 < most; c0 += lrows) {
    const int ra = row_a + c0;
    const int nr = max(0, min(lrows, row_b - ra));
    if (!PERUNIT) __syncthreads();   // the previous rows are consumed
    if (!PERUNIT && nr > 0) {
      // this split's rows: one bulk asynchronous copy issued by the split's first thread
      if (u == 0) bi_bulk_load(Lr, slice + (size_t)ra * NCP, (uint32_t)(nr * NCP * sizeof(R)), &bar[r]);
      if (!bi_mbar_wait(&bar[r], phase)) {
        if (u == 0) atomicOr(P.status, BI_FLAG_COPY_TIMEOUT);
        failed = true;
      }
      phase ^= 1u;
    }
    if (!has_unit || failed) continue;
    for (int rr = 0; rr < nr; ++rr) {
      constexpr int VE = 16 / (int)sizeof(R);
      const R *row = PERUNIT ? mine + (size_t)(ra + rr) * NCP : Lr + rr * NCP;
      const R wf = K1 == 1 ? Wp[0] : K1 == 2 ? Wp[1] : K1 == 3 ? Wp[2] : Wp[3];
      R v0 = (R)0, v1 = (R)0;
#pragma unroll
      for (int cc = 0; cc < NCP; cc += VE) {
        R x[VE];
        if (PERUNIT) ldg_vec(row + cc, x);
        else lds_vec(row + cc, x);
#pragma unroll
        for (int i = 0; i < VE; ++i) {
          if (i & 1) v1 = fma(x[i], qc[cc + i], v1);
          else v0 = fma(x[i], qc[cc + i], v0);
          accc[cc + i] = fma(wf, x[i], accc[cc + i]);
        }
      }
      R val = v0 + v1;
      bool act = true;
      int top = K1;
#pragma unroll
      for (int lv = 3; lv >= 0; --lv) {
        if (lv < K1 && act) {
          const int sj = dig[lv];
          const int idx = (mm.ooff[lv] + sj) * nt + tid;
          const R wprev = lv > 0 ? Wp[lv > 0 ? lv - 1 : 0] : (R)1;
          as[idx] = fma(wprev, val, as[idx]);
          if (lv > 0) p[lv > 0 ? lv - 1 : 0] = fma(qs[(mm.ooff[lv] + sj) * tu + u], val, p[lv > 0 ? lv - 1 : 0]);
          if (sj + 1 == mm.dim[lv]) {
            dig[lv] = 0;
            if (lv > 0) {
              val = p[lv > 0 ? lv - 1 : 0];
              p[lv > 0 ? lv - 1 : 0] = (R)0;
            }
          } else {
            dig[lv] = sj + 1;
            act = false;
          }
          top = lv;
        }
      }
      // prefix products of the outer beliefs, from the first axis whose index changed
#pragma unroll
      for (int lv = 0; lv < 4; ++lv)
        if (lv < K1 && lv >= top)
          Wp[lv] = (lv > 0 ? Wp[lv > 0 ? lv - 1 : 0] : (R)1) * qs[(mm.ooff[lv] + dig[lv]) * tu + u];
    }
  }
  // ---- add the splits' partial messages and write them out: the outer axes' from the accumulator
  // columns, then the last axis' through the same columns (they are free by then)
  __syncthreads();
  const int so = mm.ooff[K1];   // outer states of this member
  for (int i = tid; i < so * tu; i += nt) {
    const int uu = i % tu, st = i / tu;
    if (uu >= tk.z) continue;
    const R *col = as + (size_t)st * nt + uu;
    R sum = col[0];
    for (int k = 1; k < rs; ++k) sum += col[k * tu];
    int j = 0;
    while (j + 1 < K1 && st >= mm.ooff[j + 1]) ++j;
    ((R *)P.ellp)[((size_t)mi * P.NU + unit_s[uu]) * P.Sp + mm.offp[j] + (st - mm.ooff[j])] = sum;
  }
  __syncthreads();
#pragma unroll
  for (int c = 0; c < NCP; ++c) as[c * nt + tid] = accc[c];
  __syncthreads();
  for (int i = tid; i < NC * tu; i += nt) {
    const int uu = i % tu, st = i / tu;
    if (uu >= tk.z) continue;
    const R *col = as + (size_t)st * nt + uu;
    R sum = col[0];
    for (int k = 1; k < rs; ++k) sum += col[k * tu];
    ((R *)P.ellp)[((size_t)mi * P.NU + unit_s[uu]) * P.Sp + mm.offp[K1] + st] = sum;
  }
}

// NCPMAX: the largest padded last axis among the model's members.  The forms for longer last axes
// hold that many beliefs and accumulators in registers; a model that needs none of them gets a kernel
// with half the registers, two CTAs of which share an SM.
template <typename R, bool PERUNIT, int NCPMAX>
__global__ void __launch_bounds__(256, NCPMAX <= 16 ? 2 : 1)
bi_batch_contract_rt_kernel(BatchParams P, int cur, int first) {
  // (this form reads beliefs from its first instruction on, so it waits at once)
  bi_grid_wait();
  bi_grid_launch_dependents();
  (void)first;
  extern __shared__ __align__(16) unsigned char smem_raw[];
  R *Lbuf = reinterpret_cast<R *>(smem_raw);
  R *qs = Lbuf + P.lbuf;                                   // [so_max][tu] beliefs of the outer axes, per unit
  R *as = qs + (size_t)P.so_max * P.tu;                     // [so_max][threads] message accumulators, per thread
  int *unit_s = reinterpret_cast<int *>(as + (size_t)P.so_max * blockDim.x);
  int mi = 0;
  while (mi + 1 < P.nmem && (int)blockIdx.x >= P.mem[mi + 1].task0) ++mi;
  const BatchMember &mm = P.mem[mi];
  const int4 tk = P.task[blockIdx.x];
  if (tk.z == 0) return;
  const R *slice = (const R *)mm.logA + (size_t)tk.x * mm.P_pad;
  switch (mm.ncp) {
    case 4: contract_rt<R, 4, PERUNIT>(mm, slice, Lbuf, P.lbuf, qs, as, unit_s, P, cur, tk, mi); break;
    case 8: contract_rt<R, 8, PERUNIT>(mm, slice, Lbuf, P.lbuf, qs, as, unit_s, P, cur, tk, mi); break;
    case 12: contract_rt<R, 12, PERUNIT>(mm, slice, Lbuf, P.lbuf, qs, as, unit_s, P, cur, tk, mi); break;
    case 16: contract_rt<R, 16, PERUNIT>(mm, slice, Lbuf, P.lbuf, qs, as, unit_s, P, cur, tk, mi); break;
    case 20: if constexpr (NCPMAX > 16) contract_rt<R, 20, PERUNIT>(mm, slice, Lbuf, P.lbuf, qs, as, unit_s, P, cur, tk, mi); break;
    case 24: if constexpr (NCPMAX > 16) contract_rt<R, 24, PERUNIT>(mm, slice, Lbuf, P.lbuf, qs, as, unit_s, P, cur, tk, mi); break;
    case 28: if constexpr (NCPMAX > 16) contract_rt<R, 28, PERUNIT>(mm, slice, Lbuf, P.lbuf, qs, as, unit_s, P, cur, tk, mi); break;
    case 32: if constexpr (NCPMAX > 16) contract_rt<R, 32, PERUNIT>(mm, slice, Lbuf, P.lbuf, qs, as, unit_s, P, cur, tk, mi); break;
    default: break;
  }
}

// ---- per unit: sum the partial messages, add rank-1 slices and transition messages, softmax ----
struct UpdateArgs {
  const int32_t *obs, *act;
  float *q_out, *logq_out;
  int32_t *argmax_out;
  int32_t T, cur, final;
  const void *lnprior;        // [N][S] log-priors used in the place of ln D at a window's first step, or NULL
  double lambda;              // damping step; 1 = plain update
  void *xprev;                // [NU][Sp] previous iterate's logits (damped calls only), or NULL
  int32_t first;              // first iteration of the call
  const float *q_init;        // warm start (for the first damped step's ln q), or NULL
  uint32_t fmask[BI_MAX_F];   // members (rank >= 2) whose group contains factor f
  uint32_t r1mask[BI_MAX_F];  // descriptor members (modalities) that depend on factor f alone
};

// Both transition messages' dot products at once: dp = sum_r Mp[r][s] qp[r] and df = sum_r Mf[r][s] qf[r],
// r < n, the matrices read [summation index][own state] from global memory (L1), the beliefs as pairs
// from shared memory (their padding entries are zero); pointers advance by additions only.
template <typename R>
__device__ __forceinline__ void edge_dots_g(const R *__restrict__ mp, const R *__restrict__ mf, int npad,
                                            const R *qp, const R *qf, int n, R &dp, R &df) {
  using V2 = typename std::conditional<sizeof(R) == 8, double2, float2>::type;
  R p0 = (R)0, p1 = (R)0, f0 = (R)0, f1 = (R)0;
  const int st2 = 2 * npad;
  int r = 0;
#pragma unroll 2
  for (; r + 1 < n; r += 2) {
    const V2 x = *reinterpret_cast<const V2 *>(qp + r), y = *reinterpret_cast<const V2 *>(qf + r);
    p0 = fma(__ldg(mp), x.x, p0); p1 = fma(__ldg(mp + npad), x.y, p1);
    f0 = fma(__ldg(mf), y.x, f0); f1 = fma(__ldg(mf + npad), y.y, f1);
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

// A first pass gathers, with loads that do not depend on one another (one position of the unit's
// state vector per lane and trip), everything that comes from L2: the sum of the partial messages,
// the single-factor slices, the first step's log-prior, and the two neighbouring steps' beliefs, into
// the unit's part of shared memory.  The per-factor pass then reads shared memory and the transition
// matrices (L1) only.  (With the L2 reads inside the per-factor loop every factor paid several
// dependent round trips: 35 us per launch on 20 480 units, `long_scoreboard` 8.9 stall cycles per issue.)
// FW (small batches, 32 lanes per unit): a CTA is one unit and one warp per factor, so the factors are
// updated side by side instead of one after the other: with a few thousand units the kernel is a chain
// of latencies per unit, not a matter of throughput.
// FINAL: the call's last iteration (the only one that writes outputs); DAMPED: the damped update.  Both
// are instantiations of their own: the plain iteration in between runs sixteen times a call and is
// bound by instruction issue, so it carries none of their code.
template <typename R, int ALGO, int LW, bool FW, bool FINAL, bool DAMPED>
__global__ void __launch_bounds__(FW ? 32 * BI_MAX_F : 128)
bi_batch_update_kernel(const BiDev *__restrict__ mdp, BatchParams P, UpdateArgs A) {
  static_assert(!FW || LW == 32, "a warp per factor needs a whole warp per unit");
  __shared__ FactorInfo fi[BI_MAX_F];
  __shared__ unsigned char pfac[BI_MAX_F * 32];   // factor of each padded state position
  extern __shared__ __align__(16) unsigned char upd_smem[];
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
  for (int p = threadIdx.x; p < Sp; p += blockDim.x) {
    int f = 0;
    while (f + 1 < F && p >= md.offp[f + 1]) ++f;
    pfac[p] = (unsigned char)f;
  }
  __syncthreads();
  bi_grid_wait();   // the contraction's messages (and, for the beliefs, everything before it)
  bi_grid_launch_dependents();
  const int sub = FW ? 0 : threadIdx.x / LW, s = threadIdx.x % LW;
  int unit = FW ? (int)blockIdx.x : blockIdx.x * UPB + sub;
  const bool live = unit < NU;    // dead groups shadow the last unit so that whole warps reach the shuffles
  if (!live) unit = NU - 1;
  const int a = unit / T, t = unit - a * T;
  const int g = md.G == 1 ? 0 : a;   // per-agent models: this agent's matrices and slices
  const R *qc = (const R *)P.qbuf + (size_t)A.cur * NU * Sp;
  R *qn = (R *)P.qbuf + ((size_t)(A.cur ^ 1) * NU + unit) * Sp;
  const int32_t *ob = A.obs + (size_t)unit * M;
  // acp[f]: action into step t (t > 0); acp[F + f]: action out of it (t + 1 < T)
  const int32_t *acp = A.act + ((ptrdiff_t)a * (T - 1) + (t - 1)) * F;
  R *base = reinterpret_cast<R *>(upd_smem) + (size_t)sub * 3 * Sp;   // [Sp] logit constants, [Sp] q(t-1), [Sp] q(t+1)
  R *qprev = base + Sp, *qnext = base + 2 * Sp;
  for (int p = FW ? (int)threadIdx.x : s; p < Sp; p += FW ? (int)blockDim.x : LW) {
    const int f = pfac[p];
    const FactorInfo I = fi[f];
    const int sl = p - I.op;
    R x = (R)0;
    if (sl < I.n) {
      const R *ep = (const R *)P.ellp + (size_t)unit * Sp + p;   // member j's entry: NU * Sp elements further per j
      const size_t mstride = (size_t)NU * Sp;
      for (uint32_t mk = I.fmask; mk; mk &= mk - 1) x += ep[(__ffs(mk) - 1) * mstride];
      for (uint32_t mk = I.r1mask; mk; mk &= mk - 1) {   // single-factor modalities: the slice is the message
        const BiMember &mm = md.mem[__ffs(mk) - 1];
        const int o = clamp_flag(ob[mm.modality], mm.m, md.status, BI_FLAG_OBS_RANGE);
        x += __ldg((const R *)mm.logA + (size_t)g * mm.gstride + (size_t)o * mm.P_pad + sl);
      }
      if (t == 0)
        x += A.lnprior ? ((const R *)A.lnprior)[(size_t)a * S + I.off + sl]
                       : ((const R *)md.logD[f])[(size_t)g * md.Dstride[f] + sl];
    }
    base[p] = x;
    qprev[p] = t > 0 ? qc[(size_t)(unit - 1) * Sp + p] : (R)0;
    qnext[p] = t + 1 < T ? qc[(size_t)(unit + 1) * Sp + p] : (R)0;
  }
  if (FW) __syncthreads();
  else __syncwarp();
  for (int f = FW ? (int)(threadIdx.x >> 5) : 0; f < F; f += FW ? BI_MAX_F : 1) {
    const FactorInfo I = fi[f];
    const int n = I.n, np = I.np, op = I.op;
    R x = -bi_inf<R>();
    if (s < n) {
      x = base[op + s];
      // both edges are evaluated (a window's end reads zeros and discards the result)
      const int up = t > 0 ? clamp_flag(acp[f], I.U, md.status, BI_FLAG_ACT_RANGE) : 0;
      const int uf = t + 1 < T ? clamp_flag(acp[F + f], I.U, md.status, BI_FLAG_ACT_RANGE) : 0;
      const R *M0 = (const R *)(ALGO == BI_ALGO_VMP ? md.logBt[f] : md.BfT[f]);   // [previous][next]
      const R *M1 = (const R *)(ALGO == BI_ALGO_VMP ? md.logB[f] : md.BdagT[f]);   // [next][previous]
      const size_t mo = (size_t)g * md.Bstride[f] + s;
      R dp, df;
      edge_dots_g<R>(M0 + mo + up * n * np, M1 + mo + uf * n * np, np, qprev + op, qnext + op, n, dp, df);
      if (ALGO == BI_ALGO_MMP) {
        dp = (R)0.5 * bi_log_inline(bi_max(dp, (R)BI_EPS));
        df = (R)0.5 * bi_log_inline(bi_max(df, (R)BI_EPS));
      }
      x += (t > 0 ? dp : (R)0) + (t + 1 < T ? df : (R)0);
    }
    if (DAMPED) {
      // damped step on the logits; the first one starts from ln q of the starting belief (uniform: a
      // constant, taken as 0)
      R *xp = (R *)A.xprev + (size_t)unit * Sp + op;
      if (s < n) {
        R prev = (R)0;
        if (!A.first) prev = xp[s];
        else if (A.q_init) prev = bi_log(bi_max((R)A.q_init[(size_t)unit * S + I.off + s], (R)BI_EPS));
        x = fma((R)A.lambda, x, ((R)1 - (R)A.lambda) * prev);
        if (live) xp[s] = x;
      }
    }
    // any shift near the maximum keeps the exponentials in range; the last iterate takes the exact one
    const R mx = FINAL ? lane_group_max<LW>(x) : (R)lane_group_max<LW>((float)x);
    const R e = s < n ? bi_exp_inline(x - mx) : (R)0;
    const R z = lane_group_sum<LW>(e);
    const R q = e * bi_rcp(z);
    if (live && s < np) qn[op + s] = q;
    if (FINAL) {
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
__global__ void bi_batch_init_kernel(const BiDev *__restrict__ mdp, R *q, int NU, const float *__restrict__ q_init) {
  const BiDev &md = *mdp;
  const size_t total = (size_t)NU * md.Sp;
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
    const int p = (int)(i % md.Sp);
    int f = 0;
    while (f + 1 < md.F && p >= md.offp[f + 1]) ++f;
    const int s = p - md.offp[f];
    R v = (R)0;
    if (s < md.n[f]) v = q_init ? (R)q_init[(i / md.Sp) * md.S + md.off[f] + s] : (R)1 / (R)md.n[f];
    q[i] = v;
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
  const bool per_unit = h.G != 1;   // per-agent models: every unit contracts its own slice
  bool any_shape = per_unit;        // (also set when some group has no unrolled form)
  for (int gi = 0; gi < h.ngroups; ++gi) {
    const BiGroup &g = h.grp[gi];
    if (g.rank < 2) continue;
    if (g.rank > BI_MAX_RANK) return BI_ERR_UNSUPPORTED;
    if (shape_of(g) < 0) any_shape = true;
    for (int mi = g.mem_begin; mi < g.mem_end; ++mi) order[cnt++] = mi;
  }
  // (cnt == 0: every modality depends on a single factor; the update kernel alone does the work)
  std::sort(order, order + cnt, [&](int x, int y) { return h.mem[x].P_pad > h.mem[y].P_pad; });
  size_t max_slice = 0;
  int max_m = 1, so_max = 1, ncp_max = 4;
  for (int j = 0; j < cnt; ++j) {
    const BiMember &mm = h.mem[order[j]];
    int gi = 0;
    while (!(order[j] >= h.grp[gi].mem_begin && order[j] < h.grp[gi].mem_end)) ++gi;
    const BiGroup &g = h.grp[gi];
    BatchMember &bm = P.mem[j];
    bm.logA = mm.logA; bm.m = mm.m; bm.P_pad = mm.P_pad; bm.modality = mm.modality;
    bm.gstride = mm.gstride;
    bm.shape = shape_of(g); bm.rank = g.rank;
    int so = 0, rows = 1;
    for (int k = 0; k < g.rank; ++k) {
      bm.offp[k] = h.offp[g.axis[k]];
      bm.dim[k] = g.dim[k];
      bm.ooff[k] = so;
      if (k + 1 < g.rank) { so += g.dim[k]; rows *= g.dim[k]; }
      A.fmask[g.axis[k]] |= 1u << j;
    }
    bm.ncp = bi_pad4(g.dim[g.rank - 1]);
    bm.rows = rows;
    bm.split = 1;
    if ((long long)rows * bm.ncp != mm.P_pad || bm.ncp > 32) return BI_ERR_UNSUPPORTED;
    so_max = std::max(so_max, so);
    ncp_max = std::max(ncp_max, (int)bm.ncp);
    max_slice = std::max(max_slice, (size_t)mm.P_pad * sizeof(R));
    max_m = std::max(max_m, mm.m);
  }
  if (max_m > 4096) return BI_ERR_UNSUPPORTED;
  // shared memory and shape of a contraction CTA
  size_t csmem = max_slice;
  int rs = 1;
  if (any_shape) {
    // row splits: enough warps for about two per scheduler when the batch is small
    if (tu == 32) rs = NU <= 32 * 4 * md->sm_count ? 8 : 4;
    else if (tu == 64) rs = 2;
    // a column per unit (beliefs) and one per thread (message accumulators; at least 32 rows: they also
    // carry the last axis' partial messages to the final sum) for every outer state, and a staging area
    // of whole rows per split: 48 KB at most, and less when that lets a second CTA share the SM (the
    // kernel's loops are chains of shared-memory round trips: with one CTA of eight warps per SM it
    // issued on 29 % of the cycles); fewer splits, then fewer units, when even that does not fit
    P.so_max = std::max(so_max, 32);
    for (;;) {
      const size_t cols = ((size_t)P.so_max * tu + (size_t)P.so_max * tu * rs) * sizeof(R) + (size_t)tu * sizeof(int);
      size_t stage = std::min<size_t>(max_slice, 48 * 1024);
      const size_t half_sm = ((size_t)md->max_smem_optin + 1024) / 2 - 1024 - 1024;   // two CTAs, their reserved 1 KB each
      if (ncp_max <= 16 && cols + stage > half_sm && cols + 8 * 1024 <= half_sm) stage = half_sm - cols;
      P.lbuf = (int)(stage / sizeof(R));
      P.lbuf = std::max(P.lbuf / (32 * rs) * (32 * rs), 32 * rs);
      csmem = cols + (size_t)P.lbuf * sizeof(R);
      if (csmem <= (size_t)md->max_smem_optin - 1024) break;
      if (rs > 1) rs >>= 1;
      else if (tu > 32) tu >>= 1;
      else break;
    }
    P.tu = tu;
  }
  if (csmem > (size_t)md->max_smem_optin - 1024) return BI_ERR_UNSUPPORTED;
  // Unrolled forms: a member whose contraction is several thousand multiply-adds per unit is shared by
  // two threads per unit (halves of the first axis, in different warps), so that the schedulers that
  // get one more of its warps than the rest do not set the time.  (Measured on a rank-4 group of 4800
  // entries, 20 480 units: 1.32 ms per call unsplit, 1.23 ms in halves, 1.27 ms in quarters; lanes of one
  // warp sharing a unit, which turns the slice rows' broadcast loads into four different rows, 2.3 ms.)
  if (!any_shape)
    for (int j = 0; j < cnt; ++j) {
      BatchMember &bm = P.mem[j];
      const long long fm = 2LL * bm.P_pad;
      int sp = fm >= 4000 ? 2 : 1;
      if (bm.rank == 3 && sp > 2) sp = 2;
      if (bm.rank < 3) sp = 1;
      while (sp > 1 && (bm.dim[0] < sp || (tu / sp) % 32 != 0)) sp >>= 1;   // (whole warps per part)
      bm.split = sp;
      if (sp > 1) {
        int ns = 0;
        for (int k = 1; k < bm.rank; ++k) ns += bm.dim[k];
        P.sc_off = (int)((max_slice / sizeof(R) + 1) & ~(size_t)1);
        csmem = std::max(csmem, ((size_t)P.sc_off + (size_t)ns * tu) * sizeof(R));
      }
    }
  if (csmem > (size_t)md->max_smem_optin - 1024) return BI_ERR_UNSUPPORTED;
  int ntask = 0;
  for (int j = 0; j < cnt; ++j) {
    P.mem[j].task0 = ntask;
    const int tum = tu / P.mem[j].split;
    ntask += (NU + tum - 1) / tum + P.mem[j].m;
  }
  P.nmem = cnt; P.NU = NU; P.Sp = h.Sp; P.ntask = ntask;

  // ---- workspace (stream-ordered; kept in the handle and grown on demand)
  const size_t b_perm = up256((size_t)cnt * NU * sizeof(int32_t));
  const size_t b_task = up256((size_t)ntask * sizeof(int4));
  const size_t b_ellp = up256((size_t)cnt * NU * h.Sp * sizeof(R));
  const size_t b_q = up256(2 * (size_t)NU * h.Sp * sizeof(R));
  const size_t b_x = c.lambda != 1.0 ? up256((size_t)NU * h.Sp * sizeof(R)) : 0;
  const size_t need = b_perm + b_task + b_ellp + b_q + b_x;
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
  P.status = h.status;
  P.drop_copy = 0;
  if (mut->test_drop_copy > 0) {   // testing aid: this many calls lose their copies
    P.drop_copy = 1;
    mut->test_drop_copy -= 1;
  }
  P.obs = c.obs; P.M = h.M; P.T = c.T;
  A.obs = c.obs; A.act = c.act; A.q_out = c.q_out; A.logq_out = c.logq_out; A.argmax_out = c.argmax_out;
  A.T = c.T;
  A.lnprior = c.lnprior;
  A.lambda = c.lambda;
  A.xprev = b_x ? w + b_perm + b_task + b_ellp + b_q : nullptr;
  A.q_init = c.q_init;

  bi_batch_init_kernel<R><<<256, 256, 0, c.stream>>>(md->d, (R *)P.qbuf, NU, c.q_init);
  if (cnt > 0 && per_unit)
    bi_batch_identity_tasks_kernel<<<dim3(64, cnt), 256, 0, c.stream>>>(P, perm, task);
  else if (cnt > 0)
    bi_batch_bucket_kernel<<<cnt, 1024, 2 * max_m * sizeof(int32_t), c.stream>>>(P, c.obs, h.M, h.status, perm, task);
  void (*contract)(BatchParams, int, int) =
      per_unit    ? (ncp_max <= 16 ? bi_batch_contract_rt_kernel<R, true, 16> : bi_batch_contract_rt_kernel<R, true, 32>)
      : any_shape ? (ncp_max <= 16 ? bi_batch_contract_rt_kernel<R, false, 16> : bi_batch_contract_rt_kernel<R, false, 32>)
                  : bi_batch_contract_kernel<R>;
  if (cudaFuncSetAttribute((const void *)contract, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)csmem) !=
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
  typedef void (*UpdateKernel)(const BiDev *, BatchParams, UpdateArgs);
  const bool fw = lw == 32 && NU <= 64 * md->sm_count;   // a few thousand units: a warp per factor (see the kernel)
  const bool damped = A.xprev != nullptr;
  auto pick = [&](bool fin) -> UpdateKernel {
#define BI_UPD(AL, LWV, FWV) \
    (fin ? (damped ? (UpdateKernel)bi_batch_update_kernel<R, AL, LWV, FWV, true, true>   \
                   : (UpdateKernel)bi_batch_update_kernel<R, AL, LWV, FWV, true, false>) \
         : (damped ? (UpdateKernel)bi_batch_update_kernel<R, AL, LWV, FWV, false, true>  \
                   : (UpdateKernel)bi_batch_update_kernel<R, AL, LWV, FWV, false, false>))
    if (c.algo == BI_ALGO_VMP)
      return fw ? BI_UPD(BI_ALGO_VMP, 32, true)
                : lw == 8 ? BI_UPD(BI_ALGO_VMP, 8, false) : lw == 16 ? BI_UPD(BI_ALGO_VMP, 16, false) : BI_UPD(BI_ALGO_VMP, 32, false);
    return fw ? BI_UPD(BI_ALGO_MMP, 32, true)
              : lw == 8 ? BI_UPD(BI_ALGO_MMP, 8, false) : lw == 16 ? BI_UPD(BI_ALGO_MMP, 16, false) : BI_UPD(BI_ALGO_MMP, 32, false);
#undef BI_UPD
  };
  const UpdateKernel update_mid = pick(false), update_last = pick(true);
  // every launch of the loop may be scheduled while its predecessor drains (see bi_grid_wait)
  cudaLaunchAttribute pdl[1];
  pdl[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  pdl[0].val.programmaticStreamSerializationAllowed = 1;
  for (int k = 0; k < c.K; ++k) {
    const int cur = k & 1;
    A.cur = cur;
    A.final = (k == c.K - 1);
    A.first = (k == 0);
    cudaLaunchConfig_t cfg = {};
    cfg.stream = c.stream;
    cfg.attrs = pdl;
    cfg.numAttrs = 1;
    if (cnt > 0) {
      cfg.gridDim = dim3((unsigned)ntask);
      cfg.blockDim = dim3((unsigned)(tu * rs));
      cfg.dynamicSmemBytes = csmem;
      if (cudaLaunchKernelEx(&cfg, contract, P, cur, (int)(k == 0)) != cudaSuccess) return BI_ERR_CUDA;
    }
    cfg.gridDim = dim3((unsigned)(fw ? NU : (NU + upb - 1) / upb));
    cfg.blockDim = dim3((unsigned)(fw ? 32 * h.F : 128));
    cfg.dynamicSmemBytes = (size_t)(fw ? 1 : upb) * 3 * h.Sp * sizeof(R);
    if (cudaLaunchKernelEx(&cfg, A.final ? update_last : update_mid, (const BiDev *)md->d, P, A) != cudaSuccess)
      return BI_ERR_CUDA;
  }
  if (cudaGetLastError() != cudaSuccess) return BI_ERR_CUDA;
  mut->launches += cnt > 0 ? 2 + 2 * c.K : 1 + c.K;
  const bool f64 = sizeof(R) == 8;
  mut->last_kernel = c.algo == BI_ALGO_VMP ? (f64 ? "batch_vmp_f64" : "batch_vmp_f32")
                                           : (f64 ? "batch_mmp_f64" : "batch_mmp_f32");
  return BI_OK;
}

}  // namespace

int bi_batch_shape(int rank, const int *dim) {
  BiGroup g;
  memset(&g, 0, sizeof(g));
  g.rank = rank;
  for (int k = 0; k < rank && k < BI_MAX_RANK; ++k) g.dim[k] = dim[k];
  return rank >= 2 && rank <= 4 ? shape_of(g) : -1;
}

// Applies to window calls with enough (agent, step) units to fill the machine.  Shared models
// bucket the units by observed outcome and share a staged slice; per-agent models run the
// any-shape contraction with every unit reading its own slice.
int bi_launch_batch(const BiCall &c, bi_model *mut) {
  const bi_model *md = c.model;
  if (c.algo == BI_ALGO_FILTER) return BI_ERR_UNSUPPORTED;
  if (md->h.G != 1) {
    // per-agent models: the slices are re-read every iteration, which pays only while they stay in L2
    // (measured on config 3's model with per-step slices: faster than the warp-per-step kernels at
    // 112 MB of slices, slower at 224 MB)
    double bytes = 0;
    for (int gi = 0; gi < md->h.ngroups; ++gi)
      if (md->h.grp[gi].rank >= 2) bytes += (double)md->h.grp[gi].P_pad * (md->h.grp[gi].mem_end - md->h.grp[gi].mem_begin);
    bytes *= (double)c.N * c.T * (md->arith == BI_ARITH_F64 ? 8 : 4);
    if (bytes > 120e6) return BI_ERR_UNSUPPORTED;
  }
  if ((long long)c.N * c.T < 2048) return BI_ERR_UNSUPPORTED;   // too few units to fill the machine this way
  return md->arith == BI_ARITH_F64 ? launch_batch_t<double>(c, mut) : launch_batch_t<float>(c, mut);
}
