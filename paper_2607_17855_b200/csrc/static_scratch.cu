// bi_filter_static: variational filtering for callers that must not allocate.
//
// Every other entry point works on a handle whose packed model lives in device
// memory obtained with cudaMalloc at bi_model_create.  Some callers cannot do
// that: a control loop on an embedded or shared GPU whose memory was handed out
// in full at start-up, a plug-in running inside another runtime's memory pool
// that forbids allocations outside the pool, or code on a path where the
// implicit device synchronisation of cudaMalloc / cudaFree is not acceptable.
// For them this file keeps ONE fixed scratch area, a file-scope __device__
// array of BI_STATIC_SCRATCH_BYTES, packs the model into it on every call and
// runs the general filtering kernel on that copy.  It calls no cudaMalloc, no
// cudaFree and no host allocator.
//
// The array's name is only a host-side stand-in for the symbol; the device
// address is obtained once per device with cudaGetSymbolAddress (first call on
// that device) and handed to the kernels.
#include <cstring>

#include "bi_internal.h"

namespace {

static __device__ __align__(256) unsigned char bi_static_scratch[BI_STATIC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
void *g_scratch_addr[kMaxDevices];  // device address of the array, per device; NULL until set up

// ln(max(A, eps)) in float64; outcome slices contiguous, axes in the group's
// packed order, last axis padded with zeros (the layout the general kernels read)
struct StaticPackA {
  const float *src;
  double *dst;
  int64_t total;
  int32_t P, P_pad, rank, npad;
  int32_t dim[BI_MAX_RANK];
  int64_t sstride[BI_MAX_RANK];
};

__global__ void bi_static_pack_A_kernel(StaticPackA p) {
  int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (e >= p.total) return;
  int64_t go = e / p.P_pad;
  int32_t idx = (int32_t)(e - go * p.P_pad);
  double out = 0.0;
  int32_t last = idx % p.npad, rest = idx / p.npad;
  if (last < p.dim[p.rank - 1]) {
    int64_t s = go * p.P + (int64_t)last * p.sstride[p.rank - 1];
    for (int j = p.rank - 2; j >= 0; --j) {
      int32_t dg = rest % p.dim[j];
      rest /= p.dim[j];
      s += (int64_t)dg * p.sstride[j];
    }
    out = log(fmax((double)p.src[s], 1e-16));
  }
  p.dst[e] = out;
}

// forward transition matrices transposed, [action][previous][next], and ln D
__global__ void bi_static_pack_BD_kernel(const float *__restrict__ B, const float *__restrict__ D, int n, int npad,
                                         int U, double *BfT, double *logD) {
  int e = blockIdx.x * blockDim.x + threadIdx.x;
  const int total = U * n * npad;
  if (e < total) {
    int c = e % npad, r = (e / npad) % n, u = e / (npad * n);
    BfT[e] = c < n ? (double)B[((int64_t)c * n + r) * U + u] : 0.0;  // row = previous r, column = next c
  }
  if (e < npad) logD[e] = e < n ? log(fmax((double)D[e], 1e-16)) : 0.0;
}

// the model description travels as a kernel argument: no host-to-device copy of
// pageable memory is needed
__global__ void bi_static_store_descriptor_kernel(const __grid_constant__ BiDev v, BiDev *dst, uint32_t *status) {
  const int4 *s = reinterpret_cast<const int4 *>(&v);
  int4 *d = reinterpret_cast<int4 *>(dst);
  for (int i = threadIdx.x; i < (int)(sizeof(BiDev) / sizeof(int4)); i += blockDim.x) d[i] = s[i];
  if (threadIdx.x == 0) *status = 0u;  // the array keeps the previous call's contents
}

size_t align_up(size_t x) { return (x + 255) & ~(size_t)255; }

uint32_t magic32(int d) { return (uint32_t)(((1ull << 32) + (uint64_t)d - 1) / (uint64_t)d); }

}  // namespace

extern "C" int bi_filter_static(const bi_model_desc *desc, int32_t N, int32_t T, const int32_t *obs,
                                const int32_t *act, int32_t iters, float *q_out, float *logq_out,
                                int32_t *argmax_out, void *cuda_stream) {
  // ---- arguments (same rules as bi_model_create + bi_filter; shared models only)
  if (!desc || !desc->n || !desc->U || !desc->B || !desc->D) return BI_ERR_INVALID_ARG;
  const int F = desc->F, M = desc->M;
  if (F < 1 || M < 0 || N < 0 || T < 1 || iters < 1) return BI_ERR_INVALID_ARG;
  if (M > 0 && (!desc->m || !desc->dep_len || !desc->dep || !desc->A)) return BI_ERR_INVALID_ARG;
  if (F > BI_MAX_F || M > BI_MAX_M) return BI_ERR_UNSUPPORTED;
  if (desc->G != 1) return BI_ERR_UNSUPPORTED;  // per-agent models do not fit a fixed scratch area
  if (N == 0) return BI_OK;
  if (!q_out || (M > 0 && !obs) || (T > 1 && !act)) return BI_ERR_INVALID_ARG;
  int dep_off[BI_MAX_M + 1];
  dep_off[0] = 0;
  for (int f = 0; f < F; ++f) {
    if (desc->n[f] < 1 || desc->U[f] < 1 || !desc->B[f] || !desc->D[f]) return BI_ERR_INVALID_ARG;
    if (desc->n[f] > BI_MAX_N) return BI_ERR_UNSUPPORTED;
  }
  for (int i = 0; i < M; ++i) {
    if (desc->m[i] < 1 || desc->dep_len[i] < 1 || !desc->A[i]) return BI_ERR_INVALID_ARG;
    if (desc->dep_len[i] > BI_MAX_RANK) return BI_ERR_UNSUPPORTED;
    uint32_t seen = 0;
    for (int j = 0; j < desc->dep_len[i]; ++j) {
      int f = desc->dep[dep_off[i] + j];
      if (f < 0 || f >= F) return BI_ERR_INVALID_ARG;
      if (seen & (1u << f)) return BI_ERR_SHAPE;
      seen |= 1u << f;
    }
    dep_off[i + 1] = dep_off[i] + desc->dep_len[i];
  }
  cudaStream_t stream = (cudaStream_t)cuda_stream;

  // ---- set-up, once per device and with that device current: the device address of the array
  int device = 0;
  if (cudaGetDevice(&device) != cudaSuccess || device < 0 || device >= kMaxDevices) return BI_ERR_CUDA;
  if (!g_scratch_addr[device]) {
    void *ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, bi_static_scratch) != cudaSuccess || !ptr) {
      cudaGetLastError();
      return BI_ERR_CUDA;
    }
    g_scratch_addr[device] = ptr;
  }
  unsigned char *scratch = static_cast<unsigned char *>(g_scratch_addr[device]);

  // ---- plan on the stack (no heap): groups by dependency set, packed axis order, contraction levels
  bi_model md;
  memset(&md, 0, sizeof(md));
  md.last_kernel = "";
  md.arith = BI_ARITH_F64;
  md.device = device;
  cudaDeviceGetAttribute(&md.max_smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, device);
  BiDev &h = md.h;
  h.F = F; h.M = M; h.G = 1;
  int S = 0, Sp = 0;
  for (int f = 0; f < F; ++f) {
    h.n[f] = desc->n[f]; h.npad[f] = bi_pad4(desc->n[f]); h.U[f] = desc->U[f];
    h.off[f] = S; h.offp[f] = Sp;
    S += h.n[f]; Sp += h.npad[f];
  }
  h.S = S; h.Sp = Sp;
  for (int i = 0; i < M; ++i) h.m[i] = desc->m[i];
  uint32_t gmask[BI_MAX_M];
  int group_of[BI_MAX_M];
  int ngroups = 0;
  for (int i = 0; i < M; ++i) {
    uint32_t mask = 0;
    for (int j = 0; j < desc->dep_len[i]; ++j) {
      int f = desc->dep[dep_off[i] + j];
      if (desc->n[f] > 1) mask |= 1u << f;
    }
    group_of[i] = -1;
    if (mask == 0) continue;
    int gi = 0;
    while (gi < ngroups && gmask[gi] != mask) ++gi;
    if (gi == ngroups) gmask[ngroups++] = mask;
    group_of[i] = gi;
  }
  h.ngroups = ngroups;
  int nmem = 0, V0 = 4, V1 = 4, rows_max = 1, Ltot = 0;
  for (int gi = 0; gi < ngroups; ++gi) {
    BiGroup &g = h.grp[gi];
    int axes[BI_MAX_F], k = 0;
    for (int f = 0; f < F; ++f)
      if (gmask[gi] & (1u << f)) axes[k++] = f;
    int best = 0;
    for (int j = 1; j < k; ++j) {
      int nb = h.n[axes[best]], nj = h.n[axes[j]];
      long vb = (long)bi_pad4(nb) * nj, vj = (long)bi_pad4(nj) * nb;
      if (vj < vb || (vj == vb && nj < nb)) best = j;
    }
    {  // same rule as bi_model_create: orders with unrolled kernels stay, otherwise the largest outer axis goes first
      int d[BI_MAX_RANK] = {0, 0, 0, 0, 0}, p = 0;
      for (int j = 0; j < k; ++j)
        if (j != best && p < BI_MAX_RANK) d[p++] = h.n[axes[j]];
      if (p < BI_MAX_RANK) d[p] = h.n[axes[best]];
      const bool unrolled = (k == 3 && bi_tile3_shape(d[0], d[1], d[2]) > 0) || bi_batch_shape(k, d) >= 0;
      if (!unrolled && k >= 3) {
        int first = -1;
        for (int j = 0; j < k; ++j)
          if (j != best && (first < 0 || h.n[axes[j]] > h.n[axes[first]])) first = j;
        int tmp[BI_MAX_F], q = 0;
        tmp[q++] = axes[first];
        for (int j = 0; j < k; ++j)
          if (j != first && j != best) tmp[q++] = axes[j];
        tmp[q++] = axes[best];
        for (int j = 0; j < k; ++j) axes[j] = tmp[j];
        best = k - 1;
      }
    }
    const int lastf = axes[best];
    for (int j = best; j + 1 < k; ++j) axes[j] = axes[j + 1];
    axes[k - 1] = lastf;
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
    for (int l = 0; l + 1 < k; ++l) {
      BiLevel &lv = g.lev[l];
      const int last = k - 1 - l;
      lv.ndig = last;
      lv.nrows = 1;
      for (int j = 0; j < last; ++j) {
        lv.dim[j] = g.dim[j];
        lv.magic[j] = magic32(g.dim[j]);
        lv.qoff[j] = h.offp[g.axis[j]];
        lv.nrows *= g.dim[j];
      }
      lv.last_n = g.dim[last];
      lv.last_npad4 = bi_pad4(g.dim[last]) / 4;
      lv.last_qoff = h.offp[g.axis[last]];
      lv.out_npad = bi_pad4(g.dim[last - 1]);
      lv.last_pv = 4;
      while (lv.last_pv < lv.last_n) lv.last_pv <<= 1;
      const int out_elems = (lv.nrows / g.dim[last - 1]) * lv.out_npad;
      if (l % 2 == 0) { if (out_elems > V0) V0 = out_elems; } else { if (out_elems > V1) V1 = out_elems; }
      if (l == 0 && lv.nrows > rows_max) rows_max = lv.nrows;
    }
    g.mem_begin = nmem;
    for (int i = 0; i < M; ++i) {
      if (group_of[i] != gi) continue;
      BiMember &mm = h.mem[nmem++];
      mm.modality = i;
      mm.m = desc->m[i];
      mm.P_pad = P_pad;
      mm.gstride = 0;
    }
    g.mem_end = nmem;
  }
  h.nmem = nmem;
  h.Ltot = Ltot;
  md.V0max = V0; md.V1max = V1; md.rows_max = rows_max;
  md.tile_sb = 0;

  // ---- lay the packed model out in the scratch array; reject what does not fit
  size_t off = 0;
  h.status = reinterpret_cast<uint32_t *>(scratch + off);
  off += 256;
  md.d = reinterpret_cast<BiDev *>(scratch + off);
  off += align_up(sizeof(BiDev));
  for (int mi = 0; mi < nmem; ++mi) {
    BiMember &mm = h.mem[mi];
    mm.logA = scratch + off;
    off += align_up((size_t)mm.m * mm.P_pad * sizeof(double));
    if (off > BI_STATIC_SCRATCH_BYTES) return BI_ERR_UNSUPPORTED;
  }
  for (int f = 0; f < F; ++f) {
    h.BfT[f] = scratch + off;
    off += align_up((size_t)h.U[f] * h.n[f] * h.npad[f] * sizeof(double));
    h.logD[f] = scratch + off;
    off += align_up((size_t)h.npad[f] * sizeof(double));
    h.Bstride[f] = 0;
    h.Dstride[f] = 0;
    if (off > BI_STATIC_SCRATCH_BYTES) return BI_ERR_UNSUPPORTED;
  }

  // ---- pack (kernels write straight into the array) and store the description
  for (int gi = 0; gi < ngroups; ++gi) {
    const BiGroup &g = h.grp[gi];
    for (int mi = g.mem_begin; mi < g.mem_end; ++mi) {
      const BiMember &mm = h.mem[mi];
      const int i = mm.modality, ki = desc->dep_len[i];
      StaticPackA p;
      memset(&p, 0, sizeof(p));
      p.src = desc->A[i];
      p.dst = (double *)mm.logA;
      p.P_pad = g.P_pad;
      p.rank = g.rank;
      p.total = (int64_t)mm.m * g.P_pad;
      int64_t sstr[BI_MAX_RANK], acc = 1;
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
      p.npad = bi_pad4(g.dim[g.rank - 1]);
      bi_static_pack_A_kernel<<<(unsigned)((p.total + 255) / 256), 256, 0, stream>>>(p);
    }
  }
  for (int f = 0; f < F; ++f) {
    const int total = h.U[f] * h.n[f] * h.npad[f];
    const int work = total > h.npad[f] ? total : h.npad[f];
    bi_static_pack_BD_kernel<<<(work + 255) / 256, 256, 0, stream>>>(desc->B[f], desc->D[f], h.n[f], h.npad[f],
                                                                    h.U[f], (double *)h.BfT[f], (double *)h.logD[f]);
  }
  bi_static_store_descriptor_kernel<<<1, 256, 0, stream>>>(h, md.d, h.status);
  if (cudaGetLastError() != cudaSuccess) return BI_ERR_CUDA;

  // ---- the general filtering kernel on the packed copy
  BiCall c;
  c.carry_in = nullptr; c.carry_out = nullptr;
  c.model = &md; c.algo = BI_ALGO_FILTER; c.N = N; c.T = T; c.K = iters;
  c.obs = obs; c.act = act; c.q_out = q_out; c.logq_out = logq_out; c.argmax_out = argmax_out;
  c.q_prev = nullptr; c.act_prev = nullptr; c.q_init = nullptr; c.lnprior = nullptr; c.lambda = 1.0;
  c.stream = stream;
  return bi_launch_warp(c, &md);
}
