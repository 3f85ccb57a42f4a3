// Host side of the library: argument validation, the packing layer
// (bi_model_create) and the dispatcher behind bi_filter / bi_vmp / bi_mmp.
#include <algorithm>
#include <cstdio>
#include <cstring>
#include <new>
#include <vector>

#include "bi_device.cuh"
#include "bi_internal.h"

namespace {

#define BI_CUDA_TRY(expr)                      \
  do {                                         \
    cudaError_t e_ = (expr);                   \
    if (e_ != cudaSuccess) return BI_ERR_CUDA; \
  } while (0)

// ------------------------------------------------------------------ pack kernels

struct PackA {
  const float *src;  // [G][m][n_dep0]...[n_dep(k-1)]
  void *dst;         // [G][m][P_pad], R
  int64_t total;     // G * m * P_pad
  int32_t P, P_pad, rank;
  int32_t dim[BI_MAX_RANK];      // packed axis sizes
  int64_t sstride[BI_MAX_RANK];  // source stride of each packed axis
  int32_t npad;                  // padded size of the last packed axis (rank > 0)
  uint32_t *wide;                // set to 1 when an entry exceeds 1 (see BiDev::status)
};

// ln(max(A, eps)) in float64, rounded once; outcome slices contiguous, axes in
// the group's packed order, last axis padded with zeros.
template <typename R>
__global__ void bi_pack_A_kernel(PackA p) {
  int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (e >= p.total) return;
  int64_t go = e / p.P_pad;  // g * m + o
  int32_t idx = (int32_t)(e - go * p.P_pad);
  R out = (R)0;
  if (p.rank == 0) {
    // every axis has a single state: the slice is one number (padded to 4)
    if (idx == 0) {
      const float v = p.src[go * p.P];
      if (v > 1.0f) atomicOr(p.wide, 1u);
      out = (R)log(fmax((double)v, 1e-16));
    }
  } else {
    int32_t last = idx % p.npad, rest = idx / p.npad;
    if (last < p.dim[p.rank - 1]) {
      int64_t s = go * p.P + (int64_t)last * p.sstride[p.rank - 1];
      for (int j = p.rank - 2; j >= 0; --j) {
        int32_t dg = rest % p.dim[j];
        rest /= p.dim[j];
        s += (int64_t)dg * p.sstride[j];
      }
      const float v = p.src[s];
      if (v > 1.0f) atomicOr(p.wide, 1u);
      out = (R)log(fmax((double)v, 1e-16));
    }
  }
  ((R *)p.dst)[e] = out;
}

// B[g][s_next][s_prev][u] -> four [g][u][row][npad] matrices
template <typename R>
__global__ void bi_pack_B_kernel(const float *__restrict__ B, int G, int n, int npad, int U,
                                 R *Bf, R *logB, R *logBt, R *Bdag, R *BfT, R *BdagT) {
  int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  int64_t total = (int64_t)G * U * n * npad;
  if (e >= total) return;
  int c = (int)(e % npad);
  int64_t r1 = e / npad;
  int r = (int)(r1 % n);
  int64_t r2 = r1 / n;
  int u = (int)(r2 % U);
  int64_t g = r2 / U;
  R f = 0, lf = 0, lt = 0, bd = 0, ft = 0, bdt = 0;
  if (c < n) {
    const float *Bg = B + g * (int64_t)n * n * U;
    // forward: row = next state, column = previous state
    double b = (double)Bg[((int64_t)r * n + c) * U + u];
    f = (R)b;
    lf = (R)log(fmax(b, 1e-16));
    // transposed: row = previous state, column = next state
    double bt = (double)Bg[((int64_t)c * n + r) * U + u];
    lt = (R)log(fmax(bt, 1e-16));
    double rowsum = 0.0;
    for (int sp = 0; sp < n; ++sp) rowsum += (double)Bg[((int64_t)c * n + sp) * U + u];
    bd = (R)(rowsum > 0.0 ? bt / rowsum : 1.0 / n);
    ft = (R)bt;
    // row = next state r, column = previous state c, normalised over the previous states
    double rs2 = 0.0;
    for (int sp = 0; sp < n; ++sp) rs2 += (double)Bg[((int64_t)r * n + sp) * U + u];
    bdt = (R)(rs2 > 0.0 ? b / rs2 : 1.0 / n);
  }
  Bf[e] = f;
  logB[e] = lf;
  logBt[e] = lt;
  Bdag[e] = bd;
  BfT[e] = ft;
  BdagT[e] = bdt;
}

// Lane-interleaved slice layout of the register-tile kernels: within one
// outcome's slice, 16-byte vector v of lane u (u = a * SB + b / NBL) sits at
// (v * LPU + u) * VE, so one warp load instruction reads whole cache lines.
struct PackTile {
  const float *src;
  void *dst;
  int64_t total;    // G * m * P_tile
  int32_t P, P_tile, NA, NB, NC, NCP, NAP, SB, NBL, VE;
  int64_t sstride[3];
};

template <typename R>
__global__ void bi_pack_tile_kernel(PackTile p) {
  int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (e >= p.total) return;
  int64_t go = e / p.P_tile;
  int32_t idx = (int32_t)(e - go * p.P_tile);
  const int LPU = p.NAP * p.SB;
  int within = idx % p.VE, t = idx / p.VE;
  int u = t % LPU, v = t / LPU;
  int j = v * p.VE + within;
  int bl = j / p.NCP, c = j % p.NCP;
  int a = u / p.SB, b = (u % p.SB) * p.NBL + bl;
  R out = (R)0;
  if (a < p.NA && c < p.NC) {
    int64_t s = go * p.P + a * p.sstride[0] + b * p.sstride[1] + c * p.sstride[2];
    out = (R)log(fmax((double)p.src[s], 1e-16));
  }
  ((R *)p.dst)[e] = out;
}

// ---- compressed lane-interleaved slices (sparse per-agent models) ----
// A slice in the lane-interleaved layout: 16-byte vector v of lane u at (v * LPU + u) * VE, so lane u's
// local element i = v * VE + w sits at ((i / VE) * LPU + u) * VE + i % VE.
template <typename R>
__global__ void bi_floor_log_kernel(R *out) { out[0] = (R)log(fmax(0.0, 1e-16)); }

// masks[slice][u]: bit i set when lane u's i-th element differs from the floor; counts[slice]: set bits
template <typename R>
__global__ void bi_compress_count_kernel(const R *__restrict__ tile, int64_t nslices, int P_tile, int LPU, int VE,
                                         const R *__restrict__ flr, unsigned long long *masks, int32_t *counts) {
  const int64_t sl = (int64_t)blockIdx.x * (blockDim.x / 32) + threadIdx.x / 32;
  const int lane = threadIdx.x & 31;
  if (sl >= nslices) return;
  const R f = flr[0];
  const int nloc = P_tile / LPU;
  int total = 0;
  for (int u = lane; u < LPU; u += 32) {
    unsigned long long m = 0ull;
    for (int i = 0; i < nloc; ++i)
      if (tile[sl * P_tile + ((size_t)(i / VE) * LPU + u) * VE + i % VE] != f) m |= 1ull << i;
    masks[sl * LPU + u] = m;
    total += __popcll(m);
  }
  for (int o = 16; o > 0; o >>= 1) total += __shfl_xor_sync(0xffffffffu, total, o);
  if (lane == 0) counts[sl] = total;
}
// the values that are not the floor, lane after lane, at the slice's offset
template <typename R>
__global__ void bi_compress_fill_kernel(const R *__restrict__ tile, int64_t nslices, int P_tile, int LPU, int VE,
                                        const unsigned long long *__restrict__ masks,
                                        const long long *__restrict__ off, R *vals) {
  const int64_t sl = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (sl >= nslices) return;
  long long o = off[sl];
  const int nloc = P_tile / LPU;
  for (int u = 0; u < LPU; ++u) {
    unsigned long long m = masks[sl * LPU + u];
    for (int i = 0; i < nloc; ++i, m >>= 1)
      if (m & 1ull) vals[o++] = tile[sl * P_tile + ((size_t)(i / VE) * LPU + u) * VE + i % VE];
  }
}

// Pre-summed slices of a register-tile group: out[g][combo][e] = sum over the group's members, in
// member order (the order the kernels add them in), of that member's slice for its outcome in combo.
struct PackComb {
  const void *src[4];
  int32_t m[4], mul[4];
  int32_t nmem, ncomb, P_tile;
  int64_t total;   // G * ncomb * P_tile
  void *dst;
};
template <typename R>
__global__ void bi_pack_comb_kernel(PackComb p) {
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= p.total) return;
  const int e = (int)(i % p.P_tile);
  const int64_t gc = i / p.P_tile;
  int combo = (int)(gc % p.ncomb);
  const int64_t g = gc / p.ncomb;
  R acc = (R)0;
  for (int mi = 0; mi < p.nmem; ++mi) {
    const int o = combo / p.mul[mi];
    combo -= o * p.mul[mi];
    acc += ((const R *)p.src[mi])[((size_t)g * p.m[mi] + o) * p.P_tile + e];
  }
  ((R *)p.dst)[i] = acc;
}

// transition tensors with B-dependencies: source [G][n][PB][U] -> [G][U][n][PB], plain and clamped log
template <typename R>
__global__ void bi_pack_Bfull_kernel(const float *__restrict__ B, int64_t total, int n, int64_t PB, int U, R *Bfull,
                                     R *logBfull) {
  const int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (e >= total) return;
  const int64_t par = e % PB;
  int64_t r = e / PB;
  const int sn = (int)(r % n);
  r /= n;
  const int u = (int)(r % U);
  const int64_t g = r / U;
  const float v = B[((g * n + sn) * PB + par) * U + u];
  Bfull[e] = (R)v;
  logBfull[e] = (R)log(fmax((double)v, 1e-16));
}

template <typename R>
__global__ void bi_pack_D_kernel(const float *__restrict__ D, int G, int n, int npad, R *logD) {
  int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (e >= (int64_t)G * npad) return;
  int c = (int)(e % npad);
  int64_t g = e / npad;
  logD[e] = c < n ? (R)log(fmax((double)D[g * n + c], 1e-16)) : (R)0;
}

// ------------------------------------------------------------------ helpers

int dev_alloc(bi_model *md, void **p, size_t bytes) {
  if (bytes == 0) bytes = 16;
  if (md->nalloc >= (int)(sizeof(md->allocs) / sizeof(md->allocs[0]))) return BI_ERR_ALLOC;
  cudaError_t e = cudaMalloc(p, bytes);
  if (e != cudaSuccess) {
    cudaGetLastError();
    return BI_ERR_ALLOC;
  }
  md->allocs[md->nalloc++] = *p;
  return BI_OK;
}

void free_all(bi_model *md) {
  for (int i = 0; i < md->nalloc; ++i) cudaFree(md->allocs[i]);
  md->nalloc = 0;
}

uint32_t magic_for(int d) {  // d >= 2
  return (uint32_t)(((1ull << 32) + (uint64_t)d - 1) / (uint64_t)d);
}

int validate_desc(const bi_model_desc *d) {
  if (!d || !d->n || !d->U || !d->B || !d->D) return BI_ERR_INVALID_ARG;
  if (d->F < 1 || d->M < 0 || d->G < 1) return BI_ERR_INVALID_ARG;
  if (d->M > 0 && (!d->m || !d->dep_len || !d->dep || !d->A)) return BI_ERR_INVALID_ARG;
  if (d->F > BI_MAX_F || d->M > BI_MAX_M) return BI_ERR_UNSUPPORTED;
  for (int f = 0; f < d->F; ++f) {
    if (d->n[f] < 1 || d->U[f] < 1) return BI_ERR_INVALID_ARG;
    if (d->n[f] > BI_MAX_N) return BI_ERR_UNSUPPORTED;
    if (!d->B[f] || !d->D[f]) return BI_ERR_INVALID_ARG;
  }
  int o = 0;
  for (int i = 0; i < d->M; ++i) {
    if (d->m[i] < 1 || d->dep_len[i] < 1) return BI_ERR_INVALID_ARG;
    if (d->dep_len[i] > BI_MAX_RANK) return BI_ERR_UNSUPPORTED;
    if (!d->A[i]) return BI_ERR_INVALID_ARG;
    uint32_t seen = 0;
    for (int j = 0; j < d->dep_len[i]; ++j) {
      int f = d->dep[o + j];
      if (f < 0 || f >= d->F) return BI_ERR_INVALID_ARG;
      if (seen & (1u << f)) return BI_ERR_SHAPE;
      seen |= 1u << f;
    }
    o += d->dep_len[i];
  }
  return BI_OK;
}

}  // namespace

// ------------------------------------------------------------------ public API

extern "C" int bi_model_create(const bi_model_desc *desc, void *cuda_stream, bi_model_t **out) {
  return bi_model_create_arith(desc, BI_ARITH_F64, cuda_stream, out);
}

extern "C" int bi_model_arith(const bi_model_t *model) { return model ? model->arith : BI_ERR_INVALID_ARG; }

extern "C" int bi_model_set_compressed(bi_model_t *model, int on) {
  if (!model) return BI_ERR_INVALID_ARG;
  if (on && model->slice_bytes_compressed == 0) return BI_ERR_UNSUPPORTED;
  model->use_compressed = on ? 1 : 0;
  return BI_OK;
}

extern "C" int bi_model_slice_bytes(const bi_model_t *model, int64_t *dense, int64_t *compressed) {
  if (!model || !dense || !compressed) return BI_ERR_INVALID_ARG;
  *dense = model->slice_bytes_dense;
  *compressed = model->slice_bytes_compressed;
  return BI_OK;
}

static int create_impl(const bi_model_desc *desc, int arith, const int32_t *bdep_len, const int32_t *bdep,
                       void *cuda_stream, bi_model_t **out);

extern "C" int bi_model_create_arith(const bi_model_desc *desc, int arith, void *cuda_stream, bi_model_t **out) {
  return create_impl(desc, arith, nullptr, nullptr, cuda_stream, out);
}

extern "C" int bi_model_create_bdep(const bi_model_desc *desc, const int32_t *bdep_len, const int32_t *bdep, int arith,
                                    void *cuda_stream, bi_model_t **out) {
  if (!bdep_len || !bdep) return BI_ERR_INVALID_ARG;
  return create_impl(desc, arith, bdep_len, bdep, cuda_stream, out);
}

static int create_impl(const bi_model_desc *desc, int arith, const int32_t *bdep_len, const int32_t *bdep,
                       void *cuda_stream, bi_model_t **out) {
  if (!out) return BI_ERR_INVALID_ARG;
  *out = nullptr;
  if (arith != BI_ARITH_F64 && arith != BI_ARITH_F32) return BI_ERR_INVALID_ARG;
  const size_t esz = arith == BI_ARITH_F64 ? 8 : 4;
  int rc = validate_desc(desc);
  if (rc != BI_OK) return rc;
  if (bdep_len) {   // B-dependency lists: in range, no repeats, tensors of bounded size
    int o = 0;
    for (int f = 0; f < desc->F; ++f) {
      if (bdep_len[f] < 1) return BI_ERR_INVALID_ARG;
      if (bdep_len[f] > BI_MAX_RANK) return BI_ERR_UNSUPPORTED;
      uint32_t seen = 0;
      double entries = (double)desc->n[f] * desc->U[f];
      for (int j = 0; j < bdep_len[f]; ++j) {
        const int gq = bdep[o + j];
        if (gq < 0 || gq >= desc->F) return BI_ERR_INVALID_ARG;
        if (seen & (1u << gq)) return BI_ERR_SHAPE;
        seen |= 1u << gq;
        entries *= desc->n[gq];
      }
      if (entries > (double)(1 << 20)) return BI_ERR_UNSUPPORTED;
      o += bdep_len[f];
    }
  }
  cudaStream_t stream = (cudaStream_t)cuda_stream;

  bi_model *md = new (std::nothrow) bi_model();
  if (!md) return BI_ERR_ALLOC;
  memset(md, 0, sizeof(*md));
  md->damping = 1.0;
  if (const char *e = getenv("BI_TEST_NO_COMPRESS")) md->test_no_compress = atoi(e) != 0;
  if (const char *e = getenv("BI_TEST_DROP_COPY")) md->test_drop_copy = atoi(e) > 0 ? atoi(e) : 0;   // testing aids,
  if (const char *e = getenv("BI_TEST_FAMILY")) {                                                  // read here only
    md->test_family = !strcmp(e, "warp") ? BI_FAMILY_WARP : !strcmp(e, "generic") ? BI_FAMILY_GENERIC
                      : !strcmp(e, "cta") ? BI_FAMILY_CTA : !strcmp(e, "batch") ? BI_FAMILY_BATCH : BI_FAMILY_ANY;
  }
  md->last_kernel = "";
  md->arith = arith;
  if (cudaGetDevice(&md->device) != cudaSuccess) {
    delete md;
    return BI_ERR_CUDA;
  }
  cudaDeviceGetAttribute(&md->sm_count, cudaDevAttrMultiProcessorCount, md->device);
  cudaDeviceGetAttribute(&md->max_smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, md->device);

  BiDev &h = md->h;
  const int F = desc->F, M = desc->M, G = desc->G;
  h.F = F; h.M = M; h.G = G;
  int S = 0, Sp = 0;
  for (int f = 0; f < F; ++f) {
    h.n[f] = desc->n[f];
    h.npad[f] = bi_pad4(desc->n[f]);
    h.U[f] = desc->U[f];
    h.off[f] = S;
    h.offp[f] = Sp;
    S += h.n[f];
    Sp += h.npad[f];
  }
  h.S = S; h.Sp = Sp;
  for (int i = 0; i < M; ++i) h.m[i] = desc->m[i];

  // ---- group modalities by dependency set (axes with a single state dropped)
  struct Tmp { uint32_t mask; };
  std::vector<uint32_t> gmask;
  std::vector<std::vector<int>> gmembers;
  {
    int o = 0;
    for (int i = 0; i < M; ++i) {
      uint32_t mask = 0;
      for (int j = 0; j < desc->dep_len[i]; ++j) {
        int f = desc->dep[o + j];
        if (desc->n[f] > 1) mask |= 1u << f;
      }
      o += desc->dep_len[i];
      if (mask == 0) continue;  // a constant over every multi-state factor: no message
      size_t gi = 0;
      for (; gi < gmask.size(); ++gi)
        if (gmask[gi] == mask) break;
      if (gi == gmask.size()) {
        gmask.push_back(mask);
        gmembers.emplace_back();
      }
      gmembers[gi].push_back(i);
    }
  }
  h.ngroups = (int)gmask.size();
  int nmem = 0, Ltot = 0, V0 = 4, V1 = 4, rows_max = 1;
  std::vector<int> dep_off(M + 1, 0);
  for (int i = 0; i < M; ++i) dep_off[i + 1] = dep_off[i] + desc->dep_len[i];

  for (int gi = 0; gi < h.ngroups; ++gi) {
    BiGroup &g = h.grp[gi];
    std::vector<int> axes;
    for (int f = 0; f < F; ++f)
      if (gmask[gi] & (1u << f)) axes.push_back(f);
    int k = (int)axes.size();
    // the contracted-first (last, padded) axis: least padding, then the smallest
    int best = 0;
    for (int j = 1; j < k; ++j) {
      int nb = h.n[axes[best]], nj = h.n[axes[j]];
      long vb = (long)bi_pad4(nb) * nj, vj = (long)bi_pad4(nj) * nb;  // compare pad(nb)/nb vs pad(nj)/nj
      if (vj < vb || (vj == vb && nj < nb)) best = j;
    }
    // Orders with unrolled kernels (the register tiles, the batched shapes) are kept as they are.
    // For every other group of rank 3 or more the largest of the remaining axes goes first: the
    // batched contraction splits a small batch's work along the first axis.
    {
      std::vector<int> trial(axes);
      int lf = trial[best];
      trial.erase(trial.begin() + best);
      trial.push_back(lf);
      int d[BI_MAX_RANK] = {0, 0, 0, 0, 0};
      for (int j = 0; j < k && j < BI_MAX_RANK; ++j) d[j] = h.n[trial[j]];
      const bool unrolled = (k == 3 && bi_tile3_shape(d[0], d[1], d[2]) > 0) || bi_batch_shape(k, d) >= 0;
      if (!unrolled && k >= 3) {
        // largest outer axis first (stable otherwise)
        int first = -1;
        for (int j = 0; j < k; ++j)
          if (j != best && (first < 0 || h.n[axes[j]] > h.n[axes[first]])) first = j;
        const int ff = axes[first], lf2 = axes[best];
        std::vector<int> rest;
        for (int j = 0; j < k; ++j)
          if (j != first && j != best) rest.push_back(axes[j]);
        axes.clear();
        axes.push_back(ff);
        for (int f2 : rest) axes.push_back(f2);
        axes.push_back(lf2);
        best = k - 1;
      }
    }
    int lastf = axes[best];
    axes.erase(axes.begin() + best);
    axes.push_back(lastf);
    g.rank = k;
    int P_pad = 1;
    for (int j = 0; j < k; ++j) {
      g.axis[j] = axes[j];
      g.dim[j] = h.n[axes[j]];
      P_pad *= (j == k - 1) ? bi_pad4(g.dim[j]) : g.dim[j];
    }
    g.P_pad = P_pad;
    g.L_off = Ltot;
    Ltot += P_pad;
    g.first_qoff = h.offp[axes[0]];
    g.first_n = h.n[axes[0]];
    // levels: lev[l] contracts axis[k-1-l]; it has k-1-l leading axes
    for (int l = 0; l + 1 < k; ++l) {
      BiLevel &lv = g.lev[l];
      int last = k - 1 - l;
      lv.ndig = last;
      lv.nrows = 1;
      for (int j = 0; j < last; ++j) {
        lv.dim[j] = g.dim[j];
        lv.magic[j] = magic_for(g.dim[j]);
        lv.qoff[j] = h.offp[g.axis[j]];
        lv.nrows *= g.dim[j];
      }
      lv.last_n = g.dim[last];
      lv.last_npad4 = bi_pad4(g.dim[last]) / 4;
      lv.last_qoff = h.offp[g.axis[last]];
      lv.out_npad = bi_pad4(g.dim[last - 1]);
      lv.last_pv = 4;
      while (lv.last_pv < lv.last_n) lv.last_pv <<= 1;
      int out_floats = (lv.nrows / g.dim[last - 1]) * lv.out_npad;
      if (l % 2 == 0) V0 = std::max(V0, out_floats); else V1 = std::max(V1, out_floats);
      if (l == 0) rows_max = std::max(rows_max, lv.nrows);
    }
    g.mem_begin = nmem;
    for (int i : gmembers[gi]) {
      BiMember &mm = h.mem[nmem++];
      mm.modality = i;
      mm.m = desc->m[i];
      mm.P_pad = P_pad;
      mm.gstride = (G == 1) ? 0 : (int64_t)mm.m * P_pad;
    }
    g.mem_end = nmem;
  }
  h.nmem = nmem;
  h.Ltot = Ltot;
  md->V0max = V0; md->V1max = V1; md->rows_max = rows_max;

  // a register-tile shape applies when the model is one rank-3 group over exactly its factors
  md->tile_sb = 0;
  if (!bdep_len && h.ngroups == 1 && F == 3 && h.grp[0].rank == 3)
    md->tile_sb = bi_tile3_shape(h.grp[0].dim[0], h.grp[0].dim[1], h.grp[0].dim[2]);

  // at most one group over two factors, none over more: the pair filtering kernel's models
  {
    int r2 = 0, deep = 0;
    for (int gi = 0; gi < h.ngroups; ++gi) {
      if (h.grp[gi].rank == 2) ++r2;
      if (h.grp[gi].rank > 2) ++deep;
    }
    md->pair_ok = !bdep_len && deep == 0 && r2 <= 1;
    md->rank2_ok = !bdep_len && deep == 0;   // any number of groups over two factors: the pair window kernel's models
  }

  // ---- allocate and pack
  rc = dev_alloc(md, (void **)&h.status, 2 * sizeof(uint32_t));   // the flags, and the wide-range mark
  if (rc == BI_OK && cudaMemsetAsync(h.status, 0, 2 * sizeof(uint32_t), stream) != cudaSuccess) rc = BI_ERR_CUDA;
  for (int gi = 0; gi < h.ngroups && rc == BI_OK; ++gi) {
    BiGroup &g = h.grp[gi];
    for (int mi = g.mem_begin; mi < g.mem_end && rc == BI_OK; ++mi) {
      BiMember &mm = h.mem[mi];
      int i = mm.modality;
      void *dst = nullptr;
      size_t count = (size_t)G * mm.m * g.P_pad;
      rc = dev_alloc(md, &dst, count * esz);
      if (rc != BI_OK) break;
      mm.logA = dst;
      PackA p;
      memset(&p, 0, sizeof(p));
      p.src = desc->A[i];
      p.dst = dst;
      p.wide = h.status + 1;
      p.total = (int64_t)count;
      p.P_pad = g.P_pad;
      p.rank = g.rank;
      // source strides of every factor axis in A_i's own order
      int ki = desc->dep_len[i];
      int64_t sstr[BI_MAX_RANK];
      int64_t acc = 1;
      for (int j = ki - 1; j >= 0; --j) {
        sstr[j] = acc;
        acc *= desc->n[desc->dep[dep_off[i] + j]];
      }
      p.P = (int32_t)acc;
      for (int j = 0; j < g.rank; ++j) {
        p.dim[j] = g.dim[j];
        for (int jj = 0; jj < ki; ++jj)
          if (desc->dep[dep_off[i] + jj] == g.axis[j]) p.sstride[j] = sstr[jj];
      }
      p.npad = g.rank > 0 ? bi_pad4(g.dim[g.rank - 1]) : 4;
      int threads = 256;
      int64_t blocks = (p.total + threads - 1) / threads;
      if (arith == BI_ARITH_F64) bi_pack_A_kernel<double><<<(unsigned)blocks, threads, 0, stream>>>(p);
      else bi_pack_A_kernel<float><<<(unsigned)blocks, threads, 0, stream>>>(p);
      if (cudaGetLastError() != cudaSuccess) rc = BI_ERR_CUDA;
      if (rc == BI_OK && md->pair_ok && g.rank == 2 && arith == BI_ARITH_F64) {
        // the same slices with the two axes exchanged, for the pair filtering kernel's column copy
        PackA t = p;
        const size_t tcount = (size_t)G * mm.m * g.dim[1] * bi_pad4(g.dim[0]);
        void *tdst = nullptr;
        rc = dev_alloc(md, &tdst, tcount * esz);
        if (rc != BI_OK) break;
        t.dst = tdst;
        t.total = (int64_t)tcount;
        t.P_pad = g.dim[1] * bi_pad4(g.dim[0]);
        t.dim[0] = g.dim[1]; t.dim[1] = g.dim[0];
        t.sstride[0] = p.sstride[1]; t.sstride[1] = p.sstride[0];
        t.npad = bi_pad4(g.dim[0]);
        bi_pack_A_kernel<double><<<(unsigned)((t.total + threads - 1) / threads), threads, 0, stream>>>(t);
        if (cudaGetLastError() != cudaSuccess) rc = BI_ERR_CUDA;
        mm.logA_T = tdst;
      }
      if (rc == BI_OK && md->tile_sb > 0) {
        PackTile q;
        memset(&q, 0, sizeof(q));
        q.src = desc->A[i];
        q.P = p.P;
        q.NA = g.dim[0]; q.NB = g.dim[1]; q.NC = g.dim[2];
        q.NCP = bi_pad4(q.NC);
        q.NAP = 1;
        while (q.NAP < q.NA) q.NAP <<= 1;
        q.SB = md->tile_sb;
        q.NBL = q.NB / q.SB;
        q.VE = (int)(16 / esz);
        q.P_tile = q.NAP * q.NB * q.NCP;
        md->tile_P = q.P_tile;
        for (int j = 0; j < 3; ++j) q.sstride[j] = p.sstride[j];
        q.total = (int64_t)G * mm.m * q.P_tile;
        void *td = nullptr;
        rc = dev_alloc(md, &td, (size_t)q.total * esz);
        if (rc != BI_OK) break;
        q.dst = td;
        mm.logA_tile = td;
        int64_t tb = (q.total + threads - 1) / threads;
        if (arith == BI_ARITH_F64) bi_pack_tile_kernel<double><<<(unsigned)tb, threads, 0, stream>>>(q);
        else bi_pack_tile_kernel<float><<<(unsigned)tb, threads, 0, stream>>>(q);
        if (cudaGetLastError() != cudaSuccess) rc = BI_ERR_CUDA;
      }
    }
  }
  // register-tile models: the pre-summed table over every outcome combination, while it stays small
  // enough to live in L2 beside everything else (at most 4 modalities, at most 8 MiB)
  md->tile_comb = nullptr;
  md->tile_ncomb = 0;
  if (rc == BI_OK && md->tile_sb == 1 && arith == BI_ARITH_F64) {   // (read by the float64 filtering kernel only)
    const BiGroup &g0 = h.grp[0];
    const int nm = g0.mem_end - g0.mem_begin;
    double ncomb = 1.0;
    for (int mi = g0.mem_begin; mi < g0.mem_end; ++mi) ncomb *= h.mem[mi].m;
    const double bytes = ncomb * (double)G * md->tile_P * (double)esz;
    if (nm == 1) {
      md->tile_comb = const_cast<void *>(h.mem[g0.mem_begin].logA_tile);
      md->tile_ncomb = h.mem[g0.mem_begin].m;
      md->tile_comb_mul[0] = 1;
    } else if (nm <= 4 && bytes <= 8.0 * 1024 * 1024) {
      PackComb q;
      memset(&q, 0, sizeof(q));
      q.nmem = nm;
      q.ncomb = (int)ncomb;
      q.P_tile = md->tile_P;
      int mul = 1;
      for (int j = nm - 1; j >= 0; --j) {
        const BiMember &mm = h.mem[g0.mem_begin + j];
        q.src[j] = mm.logA_tile;
        q.m[j] = mm.m;
        q.mul[j] = mul;
        md->tile_comb_mul[j] = mul;
        mul *= mm.m;
      }
      q.total = (int64_t)G * q.ncomb * q.P_tile;
      void *td = nullptr;
      rc = dev_alloc(md, &td, (size_t)q.total * esz);
      if (rc == BI_OK) {
        q.dst = td;
        const int threads = 256;
        const int64_t tb = (q.total + threads - 1) / threads;
        if (arith == BI_ARITH_F64) bi_pack_comb_kernel<double><<<(unsigned)tb, threads, 0, stream>>>(q);
        else bi_pack_comb_kernel<float><<<(unsigned)tb, threads, 0, stream>>>(q);
        if (cudaGetLastError() != cudaSuccess) rc = BI_ERR_CUDA;
        md->tile_comb = td;
        md->tile_ncomb = q.ncomb;
      }
    }
  }
  // Per-agent register-tile models whose slices are mostly the floor ln 1e-16 (sparse A): a compressed
  // copy of the lane-interleaved slices for the window kernels' gather (a mask per lane and the other
  // values).  Sizing it needs the counts on the host, so making such a handle synchronises the stream.
  md->slice_bytes_dense = md->slice_bytes_compressed = 0;
  if (rc == BI_OK && md->tile_sb > 0) {
    void *fl = nullptr;
    rc = dev_alloc(md, &fl, 16);
    if (rc == BI_OK) {
      md->tile_floor = fl;
      if (arith == BI_ARITH_F64) bi_floor_log_kernel<double><<<1, 1, 0, stream>>>((double *)fl);
      else bi_floor_log_kernel<float><<<1, 1, 0, stream>>>((float *)fl);
      if (cudaGetLastError() != cudaSuccess) rc = BI_ERR_CUDA;
    }
  }
  if (rc == BI_OK && md->tile_sb > 0 && G > 1 && !md->test_no_compress) {
    const BiGroup &g0 = h.grp[0];
    const int nm = g0.mem_end - g0.mem_begin;
    int NAP = 1;
    while (NAP < g0.dim[0]) NAP <<= 1;
    const int LPU = NAP * md->tile_sb, VE = (int)(16 / esz), P_tile = md->tile_P;
    if (nm <= 4 && P_tile / LPU <= 64) {
      std::vector<unsigned long long *> masks(nm, nullptr);
      std::vector<std::vector<long long>> offs(nm);
      long long dense = 0, comp = 0;
      // pass 1: masks and counts of every member; offsets on the host
      for (int j = 0; j < nm && rc == BI_OK; ++j) {
        const BiMember &mm = h.mem[g0.mem_begin + j];
        const int64_t ns = (int64_t)G * mm.m;
        int32_t *cnt = nullptr;
        if (cudaMalloc(&masks[j], (size_t)ns * LPU * 8) != cudaSuccess || cudaMalloc(&cnt, (size_t)ns * 4) != cudaSuccess) {
          cudaGetLastError();
          if (cnt) cudaFree(cnt);
          rc = BI_ERR_ALLOC;
          break;
        }
        const unsigned blocks = (unsigned)((ns + 7) / 8);
        if (arith == BI_ARITH_F64)
          bi_compress_count_kernel<double><<<blocks, 256, 0, stream>>>((const double *)mm.logA_tile, ns, P_tile, LPU, VE,
                                                                       (const double *)md->tile_floor, masks[j], cnt);
        else
          bi_compress_count_kernel<float><<<blocks, 256, 0, stream>>>((const float *)mm.logA_tile, ns, P_tile, LPU, VE,
                                                                      (const float *)md->tile_floor, masks[j], cnt);
        std::vector<int32_t> hc((size_t)ns);
        if (cudaMemcpyAsync(hc.data(), cnt, (size_t)ns * 4, cudaMemcpyDeviceToHost, stream) != cudaSuccess ||
            cudaStreamSynchronize(stream) != cudaSuccess)
          rc = BI_ERR_CUDA;
        cudaFree(cnt);
        offs[j].assign((size_t)ns + 1, 0);
        for (int64_t i = 0; i < ns; ++i) offs[j][(size_t)i + 1] = offs[j][(size_t)i] + hc[(size_t)i];
        dense += ns * (long long)P_tile * (long long)esz;
        comp += offs[j][(size_t)ns] * (long long)esz + ns * (long long)LPU * 8 + (ns + 1) * 8;
      }
      // worth it when the compressed form is under 60 % of the dense one
      if (rc == BI_OK && comp * 10 < dense * 6) {
        for (int j = 0; j < nm && rc == BI_OK; ++j) {
          BiMember &mm = h.mem[g0.mem_begin + j];
          const int64_t ns = (int64_t)G * mm.m;
          void *dv = nullptr, *doff = nullptr, *dm = nullptr;
          if ((rc = dev_alloc(md, &dv, (size_t)offs[j][(size_t)ns] * esz)) != BI_OK) break;
          if ((rc = dev_alloc(md, &doff, (size_t)(ns + 1) * 8)) != BI_OK) break;
          if ((rc = dev_alloc(md, &dm, (size_t)ns * LPU * 8)) != BI_OK) break;
          if (cudaMemcpyAsync(doff, offs[j].data(), (size_t)(ns + 1) * 8, cudaMemcpyHostToDevice, stream) != cudaSuccess ||
              cudaMemcpyAsync(dm, masks[j], (size_t)ns * LPU * 8, cudaMemcpyDeviceToDevice, stream) != cudaSuccess) {
            rc = BI_ERR_CUDA;
            break;
          }
          const unsigned blocks = (unsigned)((ns + 127) / 128);
          if (arith == BI_ARITH_F64)
            bi_compress_fill_kernel<double><<<blocks, 128, 0, stream>>>((const double *)mm.logA_tile, ns, P_tile, LPU, VE,
                                                                        (const unsigned long long *)dm,
                                                                        (const long long *)doff, (double *)dv);
          else
            bi_compress_fill_kernel<float><<<blocks, 128, 0, stream>>>((const float *)mm.logA_tile, ns, P_tile, LPU, VE,
                                                                       (const unsigned long long *)dm,
                                                                       (const long long *)doff, (float *)dv);
          if (cudaGetLastError() != cudaSuccess) rc = BI_ERR_CUDA;
          // (the host offsets must outlive their asynchronous copy)
          if (rc == BI_OK && cudaStreamSynchronize(stream) != cudaSuccess) rc = BI_ERR_CUDA;
          mm.cmask = (const unsigned long long *)dm;
          mm.cvals = dv;
          mm.coff = (const long long *)doff;
        }
        md->slice_bytes_dense = dense;
        md->slice_bytes_compressed = comp;
      }
      cudaStreamSynchronize(stream);
      for (int j = 0; j < nm; ++j)
        if (masks[j]) cudaFree(masks[j]);
    }
  }
  h.has_bdep = bdep_len ? 1 : 0;
  for (int f = 0, bo = 0; f < F && rc == BI_OK && bdep_len; ++f) {
    // transition tensors of a model with B-dependencies (and ln D; the per-factor matrix forms are not made)
    h.bdep_len[f] = bdep_len[f];
    int64_t PB = 1;
    for (int j = 0; j < bdep_len[f]; ++j) {
      h.bdep[f][j] = bdep[bo + j];
      PB *= h.n[bdep[bo + j]];
    }
    bo += bdep_len[f];
    h.PB[f] = (int32_t)PB;
    const int n = h.n[f], npad = h.npad[f], U = h.U[f];
    const int64_t total = (int64_t)G * U * n * PB;
    void *bfull, *lbfull, *ld;
    if ((rc = dev_alloc(md, &bfull, (size_t)total * esz)) != BI_OK) break;
    if ((rc = dev_alloc(md, &lbfull, (size_t)total * esz)) != BI_OK) break;
    if ((rc = dev_alloc(md, &ld, (size_t)G * npad * esz)) != BI_OK) break;
    h.Bfull[f] = bfull; h.logBfull[f] = lbfull; h.logD[f] = ld;
    h.Bfull_stride[f] = (G == 1) ? 0 : (int64_t)U * n * PB;
    h.Dstride[f] = (G == 1) ? 0 : npad;
    const int threads = 256;
    const unsigned gb = (unsigned)((total + threads - 1) / threads);
    const unsigned gd = (unsigned)(((size_t)G * npad + threads - 1) / threads);
    if (arith == BI_ARITH_F64) {
      bi_pack_Bfull_kernel<double><<<gb, threads, 0, stream>>>(desc->B[f], total, n, PB, U, (double *)bfull, (double *)lbfull);
      bi_pack_D_kernel<double><<<gd, threads, 0, stream>>>(desc->D[f], G, n, npad, (double *)ld);
    } else {
      bi_pack_Bfull_kernel<float><<<gb, threads, 0, stream>>>(desc->B[f], total, n, PB, U, (float *)bfull, (float *)lbfull);
      bi_pack_D_kernel<float><<<gd, threads, 0, stream>>>(desc->D[f], G, n, npad, (float *)ld);
    }
    if (cudaGetLastError() != cudaSuccess) rc = BI_ERR_CUDA;
  }
  for (int f = 0; f < F && rc == BI_OK && !bdep_len; ++f) {
    int n = h.n[f], npad = h.npad[f], U = h.U[f];
    size_t count = (size_t)G * U * n * npad;
    void *bf, *lb, *lt, *bd, *ld, *bft, *bdt;
    if ((rc = dev_alloc(md, &bf, count * esz)) != BI_OK) break;
    if ((rc = dev_alloc(md, &lb, count * esz)) != BI_OK) break;
    if ((rc = dev_alloc(md, &lt, count * esz)) != BI_OK) break;
    if ((rc = dev_alloc(md, &bd, count * esz)) != BI_OK) break;
    if ((rc = dev_alloc(md, &ld, (size_t)G * npad * esz)) != BI_OK) break;
    if ((rc = dev_alloc(md, &bft, count * esz)) != BI_OK) break;
    if ((rc = dev_alloc(md, &bdt, count * esz)) != BI_OK) break;
    h.BfT[f] = bft; h.BdagT[f] = bdt;
    h.Bf[f] = bf; h.logB[f] = lb; h.logBt[f] = lt; h.Bdag[f] = bd; h.logD[f] = ld;
    h.Bstride[f] = (G == 1) ? 0 : (int64_t)U * n * npad;
    h.Dstride[f] = (G == 1) ? 0 : npad;
    int threads = 256;
    unsigned gb = (unsigned)((count + threads - 1) / threads);
    unsigned gd = (unsigned)(((size_t)G * npad + threads - 1) / threads);
    if (arith == BI_ARITH_F64) {
      bi_pack_B_kernel<double><<<gb, threads, 0, stream>>>(desc->B[f], G, n, npad, U, (double *)bf,
                                                           (double *)lb, (double *)lt, (double *)bd,
                                                           (double *)bft, (double *)bdt);
      bi_pack_D_kernel<double><<<gd, threads, 0, stream>>>(desc->D[f], G, n, npad, (double *)ld);
    } else {
      bi_pack_B_kernel<float><<<gb, threads, 0, stream>>>(desc->B[f], G, n, npad, U, (float *)bf,
                                                          (float *)lb, (float *)lt, (float *)bd,
                                                          (float *)bft, (float *)bdt);
      bi_pack_D_kernel<float><<<gd, threads, 0, stream>>>(desc->D[f], G, n, npad, (float *)ld);
    }
    if (cudaGetLastError() != cudaSuccess) rc = BI_ERR_CUDA;
  }
  if (rc == BI_OK) rc = dev_alloc(md, (void **)&md->d, sizeof(BiDev));
  if (rc == BI_OK) {
    // the host copy outlives the asynchronous copy: it is a member of the handle
    if (cudaMemcpyAsync(md->d, &md->h, sizeof(BiDev), cudaMemcpyHostToDevice, stream) != cudaSuccess)
      rc = BI_ERR_CUDA;
  }
  if (rc != BI_OK) {
    cudaStreamSynchronize(stream);
    free_all(md);
    delete md;
    return rc;
  }
  *out = md;
  return BI_OK;
}

extern "C" int bi_model_destroy(bi_model_t *model) {
  if (!model) return BI_OK;
  cudaError_t e = cudaDeviceSynchronize();
  if (model->ws) cudaFree(model->ws);
  if (model->ws_soft) cudaFree(model->ws_soft);
  if (model->ws_prior) cudaFree(model->ws_prior);
  if (model->carry) cudaFree(model->carry);
  free_all(model);
  delete model;
  return e == cudaSuccess ? BI_OK : BI_ERR_CUDA;
}

// ln max(B_u q_prev, eps) for every agent and state: the prior a continued window starts from
template <typename R>
__global__ void bi_predictive_prior_kernel(const BiDev *__restrict__ mdp, int N, const float *__restrict__ q_prev,
                                           const int32_t *__restrict__ act_prev, R *__restrict__ out) {
  const BiDev &md = *mdp;
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= N * md.S) return;
  const int a = i / md.S, p = i - a * md.S;
  int f = 0;
  while (f + 1 < md.F && p >= md.off[f + 1]) ++f;
  const int s = p - md.off[f], n = md.n[f], np = md.npad[f];
  const int g = md.G == 1 ? 0 : a;
  const int u = clamp_flag(act_prev[(size_t)a * md.F + f], md.U[f], md.status, BI_FLAG_ACT_RANGE);
  const R *row = (const R *)md.Bf[f] + (size_t)g * md.Bstride[f] + ((size_t)u * n + s) * np;   // [next][previous]
  R acc = (R)0;
  for (int r = 0; r < n; ++r) acc = fma(row[r], (R)q_prev[(size_t)a * md.S + md.off[f] + r], acc);
  out[i] = bi_log(bi_max(acc, (R)BI_EPS));
}

int bi_dispatch(const BiCall &c, bi_model *mut) {
  if (c.model->h.has_bdep) {
    // Transition tensors with several parents.  In filtering they enter only the prior, formed once per
    // step, which the CTA-per-agent filtering kernel computes; window calls (VMP) need them in every
    // message: the warp-per-step kernel's lanes sum them, the general kernel where that one does not fit.
    int rc = BI_ERR_UNSUPPORTED;
    if (c.model->test_family == BI_FAMILY_ANY)
      rc = c.algo == BI_ALGO_FILTER ? bi_launch_cta_filter(c, mut) : bi_launch_warp(c, mut);
    return rc == BI_ERR_UNSUPPORTED ? bi_launch_generic(c, mut) : rc;
  }
  const int only = c.model->test_family;   // testing aid: start at the named family
  int rc = BI_ERR_UNSUPPORTED;
  if (only == BI_FAMILY_ANY) {
    rc = bi_launch_tile3(c, mut);
    if (rc == BI_ERR_UNSUPPORTED) rc = bi_launch_tile3_window(c, mut);
    if (rc == BI_ERR_UNSUPPORTED) rc = bi_launch_pair_filter(c, mut);
    if (rc == BI_ERR_UNSUPPORTED) rc = bi_launch_pair_window(c, mut);
    if (rc == BI_ERR_UNSUPPORTED) rc = bi_launch_batch(c, mut);
    // Filtering exposes one unit per agent, so a CTA per agent keeps more of the machine busy than
    // a warp per agent, and its staged slices and per-factor warps pay at every batch size measured
    // on the 128 random structures (sum of times, CTA against warp kernel): 44 against 99 ms at 256
    // agents, 109 against 160 ms at 1024, 207 against 224 ms at 2048, 406 against 434 ms at 4096,
    // 784 against 846 ms at 8192.  The warp kernel serves the models whose slices do not fit in
    // shared memory.
    if (rc == BI_ERR_UNSUPPORTED && c.algo == BI_ALGO_FILTER) rc = bi_launch_cta_filter(c, mut);
  }
  if (only == BI_FAMILY_CTA && c.algo == BI_ALGO_FILTER) rc = bi_launch_cta_filter(c, mut);
  if (only == BI_FAMILY_BATCH) {   // the batched window kernels and what follows them
    rc = bi_launch_batch(c, mut);
    if (rc == BI_ERR_UNSUPPORTED && c.algo == BI_ALGO_FILTER) rc = bi_launch_cta_filter(c, mut);
  }
  if (rc == BI_ERR_UNSUPPORTED && only != BI_FAMILY_GENERIC) rc = bi_launch_warp(c, mut);
  if (rc == BI_ERR_UNSUPPORTED) rc = bi_launch_generic(c, mut);
  return rc;
}

static int run_call(const bi_model_t *model, int algo, int32_t N, int32_t T, const int32_t *obs,
                    const int32_t *act, int32_t iters, float *q_out, float *logq_out,
                    int32_t *argmax_out, void *cuda_stream, const float *q_prev = nullptr,
                    const int32_t *act_prev = nullptr, const float *q_init = nullptr, bool from_carry = false) {
  if (!model || N < 0 || T < 1 || iters < 1) return BI_ERR_INVALID_ARG;
  if (N == 0) return BI_OK;
  if (!q_out || (model->h.M > 0 && !obs) || (T > 1 && !act)) return BI_ERR_INVALID_ARG;
  if (model->h.G != 1 && model->h.G != N) return BI_ERR_SHAPE;
  if (algo != BI_ALGO_FILTER && T > BI_MAX_T) return BI_ERR_UNSUPPORTED;
  if (model->h.has_bdep && (algo == BI_ALGO_MMP || (algo != BI_ALGO_FILTER && q_prev))) return BI_ERR_UNSUPPORTED;
  BiCall c;
  c.model = model; c.algo = algo; c.N = N; c.T = T; c.K = iters;
  c.obs = obs; c.act = act; c.q_out = q_out; c.logq_out = logq_out; c.argmax_out = argmax_out;
  c.q_prev = q_prev; c.act_prev = act_prev; c.q_init = q_init; c.lnprior = nullptr;
  c.carry_in = nullptr; c.carry_out = nullptr;
  c.lambda = model->damping;
  c.stream = (cudaStream_t)cuda_stream;
  if (algo != BI_ALGO_FILTER && q_prev) {
    // window continued from a belief: ln(B_u q_prev) per agent, once, in the place of ln D
    bi_model *mh = const_cast<bi_model *>(model);
    const size_t need = (size_t)N * model->h.S * (model->arith == BI_ARITH_F64 ? 8 : 4);
    if (mh->ws_prior_bytes < need) {
      if (mh->ws_prior && cudaFreeAsync(mh->ws_prior, c.stream) != cudaSuccess) return BI_ERR_CUDA;
      mh->ws_prior = nullptr;
      mh->ws_prior_bytes = 0;
      void *pnew = nullptr;
      if (cudaMallocAsync(&pnew, need, c.stream) != cudaSuccess) {
        cudaGetLastError();
        return BI_ERR_ALLOC;
      }
      mh->ws_prior = pnew;
      mh->ws_prior_bytes = need;
    }
    const int total = N * model->h.S;
    if (model->arith == BI_ARITH_F64)
      bi_predictive_prior_kernel<double><<<(total + 255) / 256, 256, 0, c.stream>>>(model->d, N, q_prev, act_prev,
                                                                                   (double *)mh->ws_prior);
    else
      bi_predictive_prior_kernel<float><<<(total + 255) / 256, 256, 0, c.stream>>>(model->d, N, q_prev, act_prev,
                                                                                  (float *)mh->ws_prior);
    if (cudaGetLastError() != cudaSuccess) return BI_ERR_CUDA;
    mh->launches += 1;
    c.lnprior = mh->ws_prior;
    c.q_prev = nullptr;
    c.act_prev = nullptr;
  }
  c.stream = (cudaStream_t)cuda_stream;
  if (algo == BI_ALGO_FILTER) {
    // every filtering call leaves its last belief, in the handle's arithmetic, for bi_filter_continue
    bi_model *mh = const_cast<bi_model *>(model);
    if (from_carry && mh->carry_N != N) return BI_ERR_INVALID_ARG;
    const size_t need = (size_t)N * model->h.S * (model->arith == BI_ARITH_F64 ? 8 : 4);
    if (mh->carry_bytes < need) {   // (never while continuing: the carried belief has this size)
      if (mh->carry && cudaFreeAsync(mh->carry, c.stream) != cudaSuccess) return BI_ERR_CUDA;
      mh->carry = nullptr;
      mh->carry_bytes = 0;
      mh->carry_N = 0;
      void *pnew = nullptr;
      if (cudaMallocAsync(&pnew, need, c.stream) != cudaSuccess) {
        cudaGetLastError();
        return BI_ERR_ALLOC;
      }
      mh->carry = pnew;
      mh->carry_bytes = need;
    }
    c.carry_in = from_carry ? mh->carry : nullptr;
    c.carry_out = mh->carry;
    const int rc = bi_dispatch(c, mh);
    mh->carry_N = rc == BI_OK ? N : 0;
    return rc;
  }
  return bi_dispatch(c, const_cast<bi_model *>(model));
}

static int run_soft(const bi_model_t *model, int algo, int32_t N, int32_t T, const float *obs_soft,
                    const int32_t *act, int32_t iters, float *q_out, float *logq_out, int32_t *argmax_out,
                    void *cuda_stream) {
  if (!model || N < 0 || T < 1 || iters < 1) return BI_ERR_INVALID_ARG;
  if (N == 0) return BI_OK;
  if (!q_out || (model->h.M > 0 && !obs_soft) || (T > 1 && !act)) return BI_ERR_INVALID_ARG;
  if (model->h.G != 1 && model->h.G != N) return BI_ERR_SHAPE;
  if (algo != BI_ALGO_FILTER && T > BI_MAX_T) return BI_ERR_UNSUPPORTED;
  if (model->h.has_bdep) return BI_ERR_UNSUPPORTED;
  return bi_run_soft(model, algo, N, T, obs_soft, act, iters, q_out, logq_out, argmax_out,
                     (cudaStream_t)cuda_stream);
}

extern "C" int bi_filter_soft(const bi_model_t *model, int32_t N, int32_t T, const float *obs_soft,
                              const int32_t *act, int32_t iters, float *q_out, float *logq_out,
                              int32_t *argmax_out, void *cuda_stream) {
  return run_soft(model, BI_ALGO_FILTER, N, T, obs_soft, act, iters, q_out, logq_out, argmax_out, cuda_stream);
}

extern "C" int bi_vmp_soft(const bi_model_t *model, int32_t N, int32_t T, const float *obs_soft,
                           const int32_t *act, int32_t iters, float *q_out, float *logq_out,
                           int32_t *argmax_out, void *cuda_stream) {
  return run_soft(model, BI_ALGO_VMP, N, T, obs_soft, act, iters, q_out, logq_out, argmax_out, cuda_stream);
}

extern "C" int bi_mmp_soft(const bi_model_t *model, int32_t N, int32_t T, const float *obs_soft,
                           const int32_t *act, int32_t iters, float *q_out, float *logq_out,
                           int32_t *argmax_out, void *cuda_stream) {
  return run_soft(model, BI_ALGO_MMP, N, T, obs_soft, act, iters, q_out, logq_out, argmax_out, cuda_stream);
}

extern "C" int bi_filter(const bi_model_t *model, int32_t N, int32_t T, const int32_t *obs,
                         const int32_t *act, int32_t iters, float *q_out, float *logq_out,
                         int32_t *argmax_out, void *cuda_stream) {
  return run_call(model, BI_ALGO_FILTER, N, T, obs, act, iters, q_out, logq_out, argmax_out, cuda_stream);
}

extern "C" int bi_filter_from(const bi_model_t *model, int32_t N, int32_t T, const int32_t *obs,
                              const int32_t *act, const float *q_prev, const int32_t *act_prev,
                              int32_t iters, float *q_out, float *logq_out, int32_t *argmax_out,
                              void *cuda_stream) {
  if (!q_prev || !act_prev) return BI_ERR_INVALID_ARG;
  return run_call(model, BI_ALGO_FILTER, N, T, obs, act, iters, q_out, logq_out, argmax_out, cuda_stream, q_prev,
                  act_prev);
}

extern "C" int bi_filter_continue(const bi_model_t *model, int32_t N, int32_t T, const int32_t *obs,
                                  const int32_t *act, const int32_t *act_prev, int32_t iters, float *q_out,
                                  float *logq_out, int32_t *argmax_out, void *cuda_stream) {
  if (!model || !act_prev) return BI_ERR_INVALID_ARG;
  return run_call(model, BI_ALGO_FILTER, N, T, obs, act, iters, q_out, logq_out, argmax_out, cuda_stream, nullptr,
                  act_prev, nullptr, true);
}

extern "C" int bi_vmp(const bi_model_t *model, int32_t N, int32_t T, const int32_t *obs,
                      const int32_t *act, int32_t iters, float *q_out, float *logq_out,
                      int32_t *argmax_out, void *cuda_stream) {
  return run_call(model, BI_ALGO_VMP, N, T, obs, act, iters, q_out, logq_out, argmax_out, cuda_stream);
}

extern "C" int bi_mmp(const bi_model_t *model, int32_t N, int32_t T, const int32_t *obs,
                      const int32_t *act, int32_t iters, float *q_out, float *logq_out,
                      int32_t *argmax_out, void *cuda_stream) {
  return run_call(model, BI_ALGO_MMP, N, T, obs, act, iters, q_out, logq_out, argmax_out, cuda_stream);
}

extern "C" int bi_vmp_warm(const bi_model_t *model, int32_t N, int32_t T, const int32_t *obs,
                           const int32_t *act, const float *q_init, int32_t iters, float *q_out,
                           float *logq_out, int32_t *argmax_out, void *cuda_stream) {
  if (!q_init) return BI_ERR_INVALID_ARG;
  return run_call(model, BI_ALGO_VMP, N, T, obs, act, iters, q_out, logq_out, argmax_out, cuda_stream, nullptr,
                  nullptr, q_init);
}

extern "C" int bi_mmp_warm(const bi_model_t *model, int32_t N, int32_t T, const int32_t *obs,
                           const int32_t *act, const float *q_init, int32_t iters, float *q_out,
                           float *logq_out, int32_t *argmax_out, void *cuda_stream) {
  if (!q_init) return BI_ERR_INVALID_ARG;
  return run_call(model, BI_ALGO_MMP, N, T, obs, act, iters, q_out, logq_out, argmax_out, cuda_stream, nullptr,
                  nullptr, q_init);
}

extern "C" int bi_vmp_from(const bi_model_t *model, int32_t N, int32_t T, const int32_t *obs,
                           const int32_t *act, const float *q_prev, const int32_t *act_prev,
                           const float *q_init, int32_t iters, float *q_out, float *logq_out,
                           int32_t *argmax_out, void *cuda_stream) {
  if (!q_prev || !act_prev) return BI_ERR_INVALID_ARG;
  return run_call(model, BI_ALGO_VMP, N, T, obs, act, iters, q_out, logq_out, argmax_out, cuda_stream, q_prev,
                  act_prev, q_init);
}

extern "C" int bi_mmp_from(const bi_model_t *model, int32_t N, int32_t T, const int32_t *obs,
                           const int32_t *act, const float *q_prev, const int32_t *act_prev,
                           const float *q_init, int32_t iters, float *q_out, float *logq_out,
                           int32_t *argmax_out, void *cuda_stream) {
  if (!q_prev || !act_prev) return BI_ERR_INVALID_ARG;
  return run_call(model, BI_ALGO_MMP, N, T, obs, act, iters, q_out, logq_out, argmax_out, cuda_stream, q_prev,
                  act_prev, q_init);
}

extern "C" int bi_model_set_damping(bi_model_t *model, double lambda) {
  if (!model || !(lambda > 0.0 && lambda <= 1.0)) return BI_ERR_INVALID_ARG;
  model->damping = lambda;
  return BI_OK;
}

extern "C" int bi_status(const bi_model_t *model, void *cuda_stream, uint32_t *flags) {
  if (!model || !flags) return BI_ERR_INVALID_ARG;
  cudaStream_t s = (cudaStream_t)cuda_stream;
  uint32_t v = 0;
  BI_CUDA_TRY(cudaMemcpyAsync(&v, model->h.status, sizeof(v), cudaMemcpyDeviceToHost, s));
  BI_CUDA_TRY(cudaMemsetAsync(model->h.status, 0, sizeof(v), s));
  BI_CUDA_TRY(cudaStreamSynchronize(s));
  *flags = v;
  return BI_OK;
}

extern "C" const char *bi_last_kernel(const bi_model_t *model) { return model ? model->last_kernel : ""; }

extern "C" int64_t bi_launch_count(const bi_model_t *model) { return model ? model->launches : 0; }

extern "C" const char *bi_strerror(int code) {
  switch (code) {
    case BI_OK: return "ok";
    case BI_ERR_INVALID_ARG: return "invalid argument";
    case BI_ERR_SHAPE: return "shape mismatch";
    case BI_ERR_UNSUPPORTED: return "unsupported size or configuration";
    case BI_ERR_ALLOC: return "device allocation failed";
    case BI_ERR_CUDA: return "CUDA runtime error or no device";
    default: return "unknown error";
  }
}
