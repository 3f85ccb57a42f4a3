// Observations given as categorical vectors (Section III-B) instead of indices.
//
// The log-likelihood term of a modality is then the contraction over its
// observation axis, log(A_i) . o^i (Section III-C), and everything after it is
// unchanged.  So the call first forms, for every (agent, step) and dependency
// group, the group's slice  sum_{i in group} sum_o o^i[o] ln A_i[o, .]  in the
// layouts the inference kernels read, and then runs those kernels on a shadow
// model in which every group has one modality with T "outcomes" per agent: the
// slices just formed, selected by the step index.  Forming the slices is a
// dense product (observation vectors times ln A): float64 handles take it on
// the FP64 tensor instruction, float32 handles on scalar multiply-adds.
#include <algorithm>
#include <cstring>

#include "bi_device.cuh"
#include "bi_internal.h"

namespace {

constexpr int kTT = 16;   // steps accumulated per pass over a modality's outcomes
constexpr int kTTP = kTT + 4;   // row stride of the staged vectors (an outcome's kTT weights; padded against bank conflicts when staging)

struct SoftMember {
  const void *src;     // ln A of one modality in the layout being produced: [G][m][P]
  int64_t gstride;     // elements per model (0 when the model is shared)
  int32_t m, moff;     // outcomes; offset of the modality's block in an observation vector
};

struct SoftJob {
  SoftMember mem[BI_MAX_M];
  int32_t nmem, P, T, Mtot;
  const float *soft;   // [N][T][Mtot]
  void *dst;           // [N][T][P]
};

// kEPT slice elements of one agent per thread; a modality's outcomes are read
// once per block of kTT steps and weighted into kTT accumulators per element
// (four steps' weights are one broadcast shared-memory load for 4 kEPT multiply-adds).
// The vectors are converted to the arithmetic type once, when they are staged.
// One block of KT steps (nt of them real) starting at step t0.
template <typename R, int kEPT, int KT>
__device__ __forceinline__ void soft_block(const SoftJob &J, R *w_s, int a, int e0, R *dst, int t0, int nt) {
  __syncthreads();
  for (int i = threadIdx.x; i < KT * J.Mtot; i += blockDim.x) {   // (consecutive threads read consecutive floats)
    const int tt = i / J.Mtot, o = i - tt * J.Mtot;
    w_s[o * kTTP + tt] = tt < nt ? (R)J.soft[((size_t)a * J.T + t0) * J.Mtot + i] : (R)0;
  }
  __syncthreads();
  R acc[kEPT][KT];
#pragma unroll
  for (int j = 0; j < kEPT; ++j)
#pragma unroll
    for (int tt = 0; tt < KT; ++tt) acc[j][tt] = (R)0;
  for (int mi = 0; mi < J.nmem; ++mi) {
    const SoftMember &mm = J.mem[mi];
    const R *src = (const R *)mm.src + (size_t)a * mm.gstride;
    for (int o = 0; o < mm.m; ++o) {
      R la[kEPT];
#pragma unroll
      for (int j = 0; j < kEPT; ++j) {
        const int e = e0 + j * 128;
        la[j] = e < J.P ? __ldg(src + (size_t)o * J.P + e) : (R)0;
      }
      const Vec4<R> *wo = reinterpret_cast<const Vec4<R> *>(w_s + (size_t)(mm.moff + o) * kTTP);
#pragma unroll
      for (int t4 = 0; t4 < KT / 4; ++t4) {
        const Vec4<R> wv = wo[t4];
#pragma unroll
        for (int j = 0; j < kEPT; ++j) {
          acc[j][4 * t4 + 0] = fma(wv.x, la[j], acc[j][4 * t4 + 0]);
          acc[j][4 * t4 + 1] = fma(wv.y, la[j], acc[j][4 * t4 + 1]);
          acc[j][4 * t4 + 2] = fma(wv.z, la[j], acc[j][4 * t4 + 2]);
          acc[j][4 * t4 + 3] = fma(wv.w, la[j], acc[j][4 * t4 + 3]);
        }
      }
    }
  }
#pragma unroll
  for (int j = 0; j < kEPT; ++j) {
    const int e = e0 + j * 128;
    if (e < J.P) {
#pragma unroll
      for (int tt = 0; tt < KT; ++tt)
        if (tt < nt) dst[(size_t)(t0 + tt) * J.P + e] = acc[j][tt];
    }
  }
}

// Whole blocks of kTT steps, then the rest in the shortest block (a multiple of four steps) that holds it.
template <typename R, int kEPT>
__global__ void __launch_bounds__(128, kEPT * sizeof(R) <= 24 ? 4 : 3) bi_soft_slices_kernel(const SoftJob J) {
  extern __shared__ __align__(16) unsigned char w_raw[];
  R *w_s = reinterpret_cast<R *>(w_raw);   // [Mtot][kTTP] this agent's vectors for the current steps, outcome-major
  const int a = blockIdx.y;
  const int e0 = blockIdx.x * (kEPT * 128) + threadIdx.x;   // elements e0 + j * 128
  R *dst = (R *)J.dst + (size_t)a * J.T * J.P;
  int t0 = 0;
  for (; t0 + kTT <= J.T; t0 += kTT) soft_block<R, kEPT, kTT>(J, w_s, a, e0, dst, t0, kTT);
  const int rem = J.T - t0;
  if (rem > 12) soft_block<R, kEPT, 16>(J, w_s, a, e0, dst, t0, rem);
  else if (rem > 8) soft_block<R, kEPT, 12>(J, w_s, a, e0, dst, t0, rem);
  else if (rem > 4) soft_block<R, kEPT, 8>(J, w_s, a, e0, dst, t0, rem);
  else if (rem > 0) soft_block<R, kEPT, 4>(J, w_s, a, e0, dst, t0, rem);
}

// ---- the same slices on the FP64 tensor path ----
// Per agent the slices of a group are the product W S: W[t][k] the observation vectors' entries of
// the group's modalities (T x K, K = the sum of their outcome counts), S[k][e] the rows ln A_i[o, .]
// in the layout being produced (K x P).  A warp owns blocks of 32 columns and takes a block of up to
// 32 steps at a time: 16 accumulator tiles of 8 x 8, each k-step of four outcomes one S fragment per
// 8 columns (read once, used for every 8 steps) and one W fragment per 8 steps from shared memory.
// The m8n8k4 instruction issues once per 16 cycles and scheduler for 256 multiply-adds, so the FP64
// pipe is fed by a sixteenth of the issue slots the scalar form needs.
__device__ __forceinline__ void bi_dmma(double &c0, double &c1, double a, double b) {
  asm("mma.sync.aligned.m8n8k4.row.col.f64.f64.f64.f64 {%0,%1}, {%2}, {%3}, {%0,%1};"
               : "+d"(c0), "+d"(c1)
               : "d"(a), "d"(b));
}

constexpr int kMmaSteps = 32;   // steps per block (four tiles of 8)
constexpr int kMmaCols = 384;   // columns per CTA (four warps, three blocks of 32 columns each)

template <int MT>
__device__ __forceinline__ void soft_mma_block(const SoftJob &J, const double *Ws, int KS, const double *const *srow,
                                               int KP, double *dst, int t0, int nt, int c_begin, int c_end) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, gid = lane >> 2, tig = lane & 3;
  for (int n0 = c_begin + 32 * warp; n0 < c_end; n0 += 32 * 4) {
    double acc[MT][4][2];
#pragma unroll
    for (int m = 0; m < MT; ++m)
#pragma unroll
      for (int j = 0; j < 4; ++j) acc[m][j][0] = acc[m][j][1] = 0.0;
#pragma unroll 2
    for (int ks = 0; ks < KP; ks += 4) {
      const double *rp = srow[ks + tig];
      double b[4], av[MT];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int col = n0 + 8 * j + gid;
        b[j] = col < J.P ? __ldg(rp + col) : 0.0;
      }
#pragma unroll
      for (int m = 0; m < MT; ++m) av[m] = Ws[(8 * m + gid) * KS + ks + tig];
#pragma unroll
      for (int m = 0; m < MT; ++m)
#pragma unroll
        for (int j = 0; j < 4; ++j) bi_dmma(acc[m][j][0], acc[m][j][1], av[m], b[j]);
    }
#pragma unroll
    for (int m = 0; m < MT; ++m) {
      const int tt = 8 * m + gid;
      if (tt >= nt) continue;
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int col = n0 + 8 * j + 2 * tig;   // (P is a multiple of 4: a pair never straddles its end)
        if (col < J.P)
          *reinterpret_cast<double2 *>(dst + (size_t)(t0 + tt) * J.P + col) = make_double2(acc[m][j][0], acc[m][j][1]);
      }
    }
  }
}

__global__ void __launch_bounds__(128, 4) bi_soft_slices_mma_kernel(const SoftJob J, int Kg, int KP) {
  extern __shared__ __align__(16) unsigned char w_raw[];
  const int KS = KP + 2;                                        // row stride of the staged vectors
  double *Ws = reinterpret_cast<double *>(w_raw);              // [kMmaSteps][KS]
  const double **srow = reinterpret_cast<const double **>(Ws + kMmaSteps * KS);   // [KP] rows of S
  int32_t *sidx = reinterpret_cast<int32_t *>(srow + KP);      // [KP] their entries in an observation vector
  const int a = blockIdx.y;
  const int c_begin = blockIdx.x * kMmaCols, c_end = min(J.P, c_begin + kMmaCols);
  for (int k = threadIdx.x; k < KP; k += blockDim.x) {
    int mi = 0, o = k < Kg ? k : 0;   // (the padding rows point at the first row; their weights are zero)
    while (o >= J.mem[mi].m) { o -= J.mem[mi].m; ++mi; }
    srow[k] = (const double *)J.mem[mi].src + (size_t)a * J.mem[mi].gstride + (size_t)o * J.P;
    sidx[k] = J.mem[mi].moff + o;
  }
  double *dst = (double *)J.dst + (size_t)a * J.T * J.P;
  for (int t0 = 0; t0 < J.T; t0 += kMmaSteps) {
    const int nt = min(kMmaSteps, J.T - t0);
    __syncthreads();   // (the table above; the previous block's readers)
    for (int i = threadIdx.x; i < kMmaSteps * KP; i += blockDim.x) {
      const int tt = i / KP, k = i - tt * KP;
      Ws[tt * KS + k] = (tt < nt && k < Kg) ? (double)J.soft[((size_t)a * J.T + t0 + tt) * J.Mtot + sidx[k]] : 0.0;
    }
    __syncthreads();
    if (nt > 24) soft_mma_block<4>(J, Ws, KS, srow, KP, dst, t0, nt, c_begin, c_end);
    else if (nt > 16) soft_mma_block<3>(J, Ws, KS, srow, KP, dst, t0, nt, c_begin, c_end);
    else if (nt > 8) soft_mma_block<2>(J, Ws, KS, srow, KP, dst, t0, nt, c_begin, c_end);
    else soft_mma_block<1>(J, Ws, KS, srow, KP, dst, t0, nt, c_begin, c_end);
  }
}

__global__ void bi_soft_step_index_kernel(int32_t *obs, int N, int T, int M) {
  const size_t total = (size_t)N * T * M;
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x)
    obs[i] = (int32_t)((i / M) % T);
}

size_t up256(size_t x) { return (x + 255) & ~(size_t)255; }

template <typename R>
int run_soft_t(const bi_model *model, int algo, int N, int T, const float *obs_soft, const int32_t *act, int iters,
               float *q_out, float *logq_out, int32_t *argmax_out, cudaStream_t stream) {
  bi_model *mut = const_cast<bi_model *>(model);
  const BiDev &h = model->h;
  int moff[BI_MAX_M], Mtot = 0;
  for (int i = 0; i < h.M; ++i) { moff[i] = Mtot; Mtot += h.m[i]; }
  if ((size_t)kTTP * Mtot * sizeof(R) > 96 * 1024) return BI_ERR_UNSUPPORTED;
  const bool tile = model->tile_sb > 0;
  const size_t NT = (size_t)N * T;

  // ---- workspace: per group the packed slices (and the lane-interleaved ones of a tile model),
  // the step-index "observations", the shadow descriptor
  size_t off_pack[BI_MAX_GROUPS], off_tile = 0, need = 0;
  for (int k = 0; k < h.ngroups; ++k) {
    off_pack[k] = need;
    need += up256(NT * h.grp[k].P_pad * sizeof(R));
  }
  if (tile) { off_tile = need; need += up256(NT * model->tile_P * sizeof(R)); }
  // a filtering call on a model the pair filtering kernel serves: that kernel also reads the pair's
  // slices with the two axes exchanged, so those are formed too (from the handle's transposed copies)
  int kpair = -1;
  size_t off_packT = 0, PT = 0;
  if (algo == BI_ALGO_FILTER && model->pair_ok && sizeof(R) == 8)
    for (int k = 0; k < h.ngroups; ++k)
      if (h.grp[k].rank == 2 && h.mem[h.grp[k].mem_begin].logA_T) kpair = k;
  if (kpair >= 0) {
    PT = (size_t)h.grp[kpair].dim[1] * bi_pad4(h.grp[kpair].dim[0]);
    off_packT = need;
    need += up256(NT * PT * sizeof(R));
  }
  const size_t off_obs = need;
  need += up256(NT * h.ngroups * sizeof(int32_t));
  const size_t off_desc = need;
  need += up256(sizeof(BiDev));
  if (mut->ws_soft_bytes < need) {
    if (mut->ws_soft && cudaFreeAsync(mut->ws_soft, stream) != cudaSuccess) return BI_ERR_CUDA;
    mut->ws_soft = nullptr;
    mut->ws_soft_bytes = 0;
    void *pnew = nullptr;
    if (cudaMallocAsync(&pnew, need, stream) != cudaSuccess) {
      cudaGetLastError();
      return BI_ERR_ALLOC;
    }
    mut->ws_soft = pnew;
    mut->ws_soft_bytes = need;
  }
  unsigned char *w = static_cast<unsigned char *>(mut->ws_soft);

  // ---- the slices.  A register-tile model's kernels read only the lane-interleaved layout, so
  // that one is formed first; the packed layout follows only if those kernels decline the call.
  const size_t wsmem = (size_t)kTTP * Mtot * sizeof(R);
  void (*kerns[4])(const SoftJob) = {bi_soft_slices_kernel<R, 1>, bi_soft_slices_kernel<R, 2>,
                                     bi_soft_slices_kernel<R, 3>, bi_soft_slices_kernel<R, 4>};
  for (auto kf : kerns)
    if (cudaFuncSetAttribute((const void *)kf, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)wsmem) != cudaSuccess)
      return BI_ERR_CUDA;
  int launches = 0;
  // layout 0: every group's packed slices; 1: the lane-interleaved slices of a tile model; 2: the
  // pair's slices with the axes exchanged
  auto form = [&](int layout) {
    for (int k = layout == 2 ? kpair : 0; k < (layout == 1 ? 1 : layout == 2 ? kpair + 1 : h.ngroups); ++k) {
      const BiGroup &g = h.grp[k];
      SoftJob J;
      memset(&J, 0, sizeof(J));
      J.nmem = g.mem_end - g.mem_begin;
      J.P = layout == 1 ? model->tile_P : layout == 2 ? (int)PT : g.P_pad;
      J.T = T; J.Mtot = Mtot; J.soft = obs_soft;
      J.dst = w + (layout == 1 ? off_tile : layout == 2 ? off_packT : off_pack[k]);
      for (int i = 0; i < J.nmem; ++i) {
        const BiMember &mm = h.mem[g.mem_begin + i];
        J.mem[i].src = layout == 1 ? mm.logA_tile : layout == 2 ? mm.logA_T : mm.logA;
        J.mem[i].gstride = h.G == 1 ? 0 : (int64_t)mm.m * J.P;
        J.mem[i].m = mm.m;
        J.mem[i].moff = moff[mm.modality];
      }
      int Kg = 0;
      for (int i = 0; i < J.nmem; ++i) Kg += J.mem[i].m;
      const int KP = (Kg + 3) & ~3;
      const size_t msmem = ((size_t)kMmaSteps * (KP + 2) + KP) * sizeof(double) + (size_t)KP * sizeof(int32_t);
      if (sizeof(R) == 8 && msmem <= 48 * 1024) {   // float64: the tensor form
        bi_soft_slices_mma_kernel<<<dim3((J.P + kMmaCols - 1) / kMmaCols, N), 128, msmem, stream>>>(J, Kg, KP);
      } else {
        // elements per thread: 4 for large slices, else just enough to cover the slice with one CTA
        const int ept = J.P >= 512 ? 4 : (J.P + 127) / 128;
        kerns[ept - 1]<<<dim3((J.P + ept * 128 - 1) / (ept * 128), N), 128, wsmem, stream>>>(J);
      }
      ++launches;
    }
  };
  form(tile ? 1 : 0);
  if (kpair >= 0) form(2);
  int32_t *obs_idx = reinterpret_cast<int32_t *>(w + off_obs);
  bi_soft_step_index_kernel<<<256, 256, 0, stream>>>(obs_idx, N, T, h.ngroups);
  ++launches;
  if (cudaGetLastError() != cudaSuccess) return BI_ERR_CUDA;

  // ---- the shadow model: one modality per group, T outcomes per agent, selected by the step index
  bi_model sh = *model;
  sh.h.G = N;
  sh.h.M = h.ngroups;
  sh.h.nmem = h.ngroups;
  for (int k = 0; k < h.ngroups; ++k) {
    BiGroup &g = sh.h.grp[k];
    g.mem_begin = k;
    g.mem_end = k + 1;
    BiMember &mm = sh.h.mem[k];
    mm.logA = w + off_pack[k];
    mm.logA_tile = tile && k == 0 ? w + off_tile : nullptr;
    mm.logA_T = k == kpair ? w + off_packT : nullptr;
    mm.cmask = nullptr; mm.cvals = nullptr; mm.coff = nullptr;   // (the slices formed above are dense)
    mm.gstride = (int64_t)T * g.P_pad;
    mm.m = T;
    mm.modality = k;
    mm.P_pad = g.P_pad;
    sh.h.m[k] = T;
  }
  // (a group of one modality is its own pre-summed table: the shadow's T per-agent slices)
  sh.soft_shadow = 1;
  sh.pair_ok = kpair >= 0 || (model->pair_ok && sizeof(R) == 8 && algo == BI_ALGO_FILTER);
  // (the pair filtering kernel needs the transposed slices formed above, or no pair at all; the pair
  // window kernel reads rows only)
  sh.tile_comb = tile ? w + off_tile : nullptr;
  sh.tile_ncomb = T;
  sh.tile_comb_mul[0] = 1;
  sh.d = reinterpret_cast<BiDev *>(w + off_desc);
  // (the shadow borrows the handle's batched-path workspace and hands it back below)
  if (cudaMemcpyAsync(sh.d, &sh.h, sizeof(BiDev), cudaMemcpyHostToDevice, stream) != cudaSuccess) return BI_ERR_CUDA;

  BiCall c;
  c.carry_in = nullptr; c.carry_out = nullptr;
  c.model = &sh; c.algo = algo; c.N = N; c.T = T; c.K = iters;
  c.obs = obs_idx; c.act = act; c.q_prev = nullptr; c.act_prev = nullptr; c.q_init = nullptr; c.lnprior = nullptr; c.lambda = model->damping;
  c.q_out = q_out; c.logq_out = logq_out; c.argmax_out = argmax_out;
  c.stream = stream;
  const int64_t before = sh.launches;
  int rc;
  if (tile) {
    rc = bi_launch_tile3(c, &sh);
    if (rc == BI_ERR_UNSUPPORTED) rc = bi_launch_tile3_window(c, &sh);
    if (rc == BI_ERR_UNSUPPORTED) {
      form(0);
      if (cudaGetLastError() != cudaSuccess) return BI_ERR_CUDA;
      rc = bi_launch_warp(c, &sh);
      if (rc == BI_ERR_UNSUPPORTED) rc = bi_launch_generic(c, &sh);
    }
  } else {
    rc = bi_dispatch(c, &sh);
  }
  mut->ws = sh.ws;
  mut->ws_bytes = sh.ws_bytes;
  mut->launches += launches + (sh.launches - before);
  mut->last_kernel = sh.last_kernel;
  return rc;
}

}  // namespace

int bi_run_soft(const bi_model *model, int algo, int N, int T, const float *obs_soft, const int32_t *act, int iters,
                float *q_out, float *logq_out, int32_t *argmax_out, cudaStream_t stream) {
  return model->arith == BI_ARITH_F64
             ? run_soft_t<double>(model, algo, N, T, obs_soft, act, iters, q_out, logq_out, argmax_out, stream)
             : run_soft_t<float>(model, algo, N, T, obs_soft, act, iters, q_out, logq_out, argmax_out, stream);
}
