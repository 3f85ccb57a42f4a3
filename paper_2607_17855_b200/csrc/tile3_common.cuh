// Shared by the register-tile filtering and window kernels: the parameter block
// and its filling from a call, the compiled shape table, small device helpers.
#pragma once
#include "bi_internal.h"
#include "tile3.cuh"

// compiled tile shapes: packed dims (a, b, c), the lanes along b, and whether the
// filtering kernel keeps the step's slice in shared memory (large tiles) or registers
#define BI_TILE3_SHAPES(X) X(8, 6, 8, 1, false) X(16, 12, 8, 2, true) X(3, 2, 4, 1, false) X(10, 6, 8, 1, true)


struct Tile3Params {
  const void *logA[BI_MAX_M];
  int64_t gstride[BI_MAX_M];
  int32_t modality[BI_MAX_M], mcount[BI_MAX_M];
  int32_t nmem, P_tile;
  const unsigned long long *cmask[BI_MAX_M];   // compressed slices (BiMember), all NULL when the model has none
  const void *cvals[BI_MAX_M];
  const long long *coff[BI_MAX_M];
  const void *floor_log;     // device scalar ln 1e-16
  const void *Lcomb;        // the group's slices pre-summed for every outcome combination [G][ncomb][P_tile], or NULL
  int32_t ncomb, comb_mul[BI_MAX_M];   // combination index = sum_i outcome_i * comb_mul[i]
  int32_t fac[3];   // factor ids of the axes a, b, c
  int32_t off[3];   // offsets of those factors in an output belief vector
  int32_t np[3];    // padded row length of their transition matrices
  int32_t U[3];
  const void *Bf[3], *logB[3], *logBt[3], *Bdag[3], *BfT[3], *BdagT[3], *logD[3];
  int64_t Bstride[3], Dstride[3];
  int32_t N, T, K, M, S, G;
  const int32_t *obs, *act;
  const float *q_prev;       // filtering continued from these beliefs [N][S], or NULL
  const int32_t *act_prev;   // [N][F] with q_prev
  const void *carry_in;      // as BiCall
  void *carry_out;
  const float *q_init;       // window algorithms: starting beliefs [N][T][S], or NULL
  const void *lnprior;       // window algorithms: [N][S] log-priors used in the place of ln D, or NULL
  int32_t F;
  float *q_out, *logq_out;
  int32_t *argmax_out;
  uint32_t *status;
  double lambda;             // damping step (1 = plain update)
  int32_t unit_shift;        // softmax shifts per agent even where a warp-wide one would do (see BiDev::status)
};

// sum_r M[r][s] q[r] for this lane's s: col points at M[0][s], rows are `stride` apart
template <typename R, int N>
__device__ __forceinline__ R col_dot(const R *__restrict__ col, int stride, const R *q) {
  R x[N];
#pragma unroll
  for (int r = 0; r < N; ++r) x[r] = __ldg(col + r * stride) * q[r];
  return tree_sum<R, N>(x);
}


// the same for a matrix that may live in shared or global memory
template <typename R, int N>
__device__ __forceinline__ R col_dot_any(const R *col, int stride, const R *q) {
  R x[N];
#pragma unroll
  for (int r = 0; r < N; ++r) x[r] = col[r * stride] * q[r];
  return tree_sum<R, N>(x);
}

static inline void bi_tile3_fill_params(const BiCall &c, Tile3Params &p) {
  const bi_model *md = c.model;
  const BiDev &h = md->h;
  const BiGroup &g = h.grp[0];
  p.nmem = g.mem_end - g.mem_begin;
  p.floor_log = md->tile_floor;
  p.unit_shift = md->soft_shadow;
  p.Lcomb = md->tile_comb;
  p.ncomb = md->tile_ncomb;
  for (int i = 0; i < p.nmem; ++i) p.comb_mul[i] = md->tile_comb_mul[i];
  p.P_tile = md->tile_P;
  for (int i = 0; i < p.nmem; ++i) {
    const BiMember &mm = h.mem[g.mem_begin + i];
    p.logA[i] = mm.logA_tile;
    p.gstride[i] = mm.gstride;
    p.modality[i] = mm.modality;
    p.mcount[i] = mm.m;
    const bool comp = md->use_compressed != 0;
    p.cmask[i] = comp ? mm.cmask : nullptr; p.cvals[i] = comp ? mm.cvals : nullptr; p.coff[i] = comp ? mm.coff : nullptr;
  }
  for (int j = 0; j < 3; ++j) {
    const int f = g.axis[j];
    p.fac[j] = f;
    p.off[j] = h.off[f];
    p.np[j] = h.npad[f];
    p.U[j] = h.U[f];
    p.Bf[j] = h.Bf[f]; p.logB[j] = h.logB[f]; p.logBt[j] = h.logBt[f]; p.Bdag[j] = h.Bdag[f];
    p.BfT[j] = h.BfT[f]; p.BdagT[j] = h.BdagT[f];
    p.logD[j] = h.logD[f];
    p.Bstride[j] = h.Bstride[f];
    p.Dstride[j] = h.Dstride[f];
  }
  p.N = c.N; p.T = c.T; p.K = c.K; p.M = h.M; p.S = h.S; p.G = h.G;
  p.obs = c.obs; p.act = c.act; p.q_out = c.q_out; p.logq_out = c.logq_out;
  p.q_prev = c.q_prev; p.act_prev = c.act_prev; p.carry_in = c.carry_in; p.carry_out = c.carry_out; p.q_init = c.q_init; p.lnprior = c.lnprior; p.lambda = c.lambda; p.F = c.model->h.F;
  p.argmax_out = c.argmax_out; p.status = h.status;
}
