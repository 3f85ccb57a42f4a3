// Internal structures shared by the packing layer, the dispatcher and the
// kernels.  Nothing here is part of the public ABI.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "bi.h"

#define BI_EPS 1e-16
#define BI_MAX_GROUPS BI_MAX_M

enum { BI_ALGO_FILTER = 0, BI_ALGO_VMP = 1, BI_ALGO_MMP = 2 };
enum { BI_FAMILY_ANY = 0, BI_FAMILY_WARP = 1, BI_FAMILY_GENERIC = 2, BI_FAMILY_CTA = 3, BI_FAMILY_BATCH = 4 };

static __host__ __device__ inline int bi_pad4(int x) { return (x + 3) & ~3; }
// Row stride in shared memory for rows of npad elements (npad a multiple of 4, elements of esize
// bytes) read by one thread per row with 16-byte loads: an odd number of 16-byte units, or the lanes
// of a quarter warp fall on the same banks.
static __host__ __device__ inline int bi_row_stride(int npad, int esize) {
  const int per16 = 16 / esize;
  return ((npad / per16) % 2 == 1) ? npad : npad + per16;
}

// One contraction level of a dependency group.  The group's summed slice is a
// tensor with `ndig` leading axes and one last axis; the level contracts the
// last axis against its factor's belief (giving a tensor over the leading
// axes for the next level) and, weighted by the outer product of the leading
// beliefs, accumulates the likelihood message to the last axis' factor.
struct BiLevel {
  int32_t nrows;      // product of the leading axis sizes
  int32_t ndig;       // number of leading axes, 1..4
  int32_t dim[4];     // leading axis sizes, slowest first
  uint32_t magic[4];  // ceil(2^32 / dim) for exact division by multiply-high
  int32_t qoff[4];    // padded belief offset of each leading axis' factor
  int32_t last_n;     // size of the contracted axis
  int32_t last_npad4; // its padded size / 4
  int32_t last_qoff;  // padded belief offset of its factor
  int32_t out_npad;   // padded size of the output tensor's last axis
  int32_t last_pv;    // last_n rounded up to a power of two, at least 4
};

// Modalities with the same dependency *set* form one group: their slices add
// before any contraction, so they share one packed axis order.
struct BiGroup {
  int32_t rank;       // number of axes with more than one state
  int32_t axis[BI_MAX_RANK];  // factor ids in packed order (last = contracted first)
  int32_t dim[BI_MAX_RANK];
  int32_t P_pad;      // floats per packed slice (last axis padded to a multiple of 4)
  int32_t mem_begin, mem_end;  // members in BiDev::mem
  int32_t L_off;      // float offset of this group's summed slice in a staged step
  int32_t first_qoff, first_n; // axis[0]'s factor: receives the fully contracted vector
  BiLevel lev[BI_MAX_RANK - 1]; // lev[0] contracts axis[rank-1], lev[1] axis[rank-2], ...
};

struct BiMember {
  const void *logA;   // packed [G][m][P_pad], float or double (the handle's arithmetic)
  const void *logA_tile;  // lane-interleaved copy [G][m][P_tile] for the register-tile kernels, or NULL
  // Compressed form of the lane-interleaved copy for sparse per-agent models (or NULL): most entries
  // of such a slice are the floor ln 1e-16 (a zero of A), so a slice is stored as one 64-bit mask per
  // lane of a unit (bit i set: the lane's i-th element is not the floor) plus the other values, packed
  // lane after lane.  cmask: [G * m][LPU]; coff: [G * m + 1] element offsets into cvals.
  const void *logA_T;     // groups over two factors of pair models: the slices transposed, [G][m][dim1][pad4(dim0)], or NULL
  const unsigned long long *cmask;
  const void *cvals;
  const long long *coff;
  int64_t gstride;    // floats per model (0 when the model is shared)
  int32_t m, modality, P_pad, pad_;
};

// (16-byte aligned so that its size is a whole number of 16-byte vectors: kernels
// copy it into shared memory with vector loads)
struct alignas(16) BiDev {
  int32_t F, M, S, Sp, G, ngroups, nmem, Ltot;
  int32_t n[BI_MAX_F], npad[BI_MAX_F], off[BI_MAX_F], offp[BI_MAX_F], U[BI_MAX_F];
  int32_t m[BI_MAX_M];
  BiGroup grp[BI_MAX_GROUPS];
  BiMember mem[BI_MAX_M];
  // per factor, per model g, per action u: [n][npad] row-major, pad columns zero;
  // element type float or double (the handle's arithmetic)
  const void *Bf[BI_MAX_F];    // Bf[s_next][s_prev]    = B[s_next, s_prev, u]
  const void *logB[BI_MAX_F];  // ln of the same
  const void *logBt[BI_MAX_F]; // [s_prev][s_next]      = ln B[s_next, s_prev, u]
  const void *Bdag[BI_MAX_F];  // [s_prev][s_next]      = B[s_next, s_prev, u] / sum_r B[s_next, r, u]
  const void *BfT[BI_MAX_F];   // [s_prev][s_next]      = B[s_next, s_prev, u]
  const void *BdagT[BI_MAX_F]; // [s_next][s_prev]      = B[s_next, s_prev, u] / sum_r B[s_next, r, u]
  const void *logD[BI_MAX_F];  // [G][npad]
  int64_t Bstride[BI_MAX_F];    // floats per model in each B array (0 when shared)
  // Non-trivial B-dependencies (has_bdep != 0): factor f's transition reads the previous states of the
  // factors bdep[f][0..bdep_len[f]); PB[f] = product of their state counts.  The transition tensors,
  // per model g and action u: [n_f (next)][PB[f]] with the parents in list order, last fastest; the six
  // per-factor matrix forms above are not made for such a model.
  int32_t has_bdep, bdep_len[BI_MAX_F], bdep[BI_MAX_F][BI_MAX_RANK], PB[BI_MAX_F];
  const void *Bfull[BI_MAX_F];     // B[s_next, parents, u]
  const void *logBfull[BI_MAX_F];  // ln max(., 1e-16) of the same
  int64_t Bfull_stride[BI_MAX_F];  // elements per model (0 when shared)
  int64_t Dstride[BI_MAX_F];
  // status[0]: the BI_FLAG_* bits bi_status reports and clears.  status[1]: set when the model was packed
  // if an entry of A exceeds 1 (not a probability): kernels that shift several agents' softmaxes by one
  // common power of two then shift per agent, because such logits can lie too far apart for one shift.
  uint32_t *status;
};

// host-side handle
struct bi_model {
  BiDev h;          // host copy (device pointers inside)
  BiDev *d;         // device copy
  void *allocs[24 + 3 * BI_MAX_M + 10 * BI_MAX_F];  // status, descriptor, pre-summed table, 2 per modality, 7 per factor
  int nalloc;
  int arith;        // BI_ARITH_F64 or BI_ARITH_F32
  int device;
  int sm_count;
  int max_smem_optin;
  int tile_sb;      // > 0: a register-tile shape matches; lanes along b per (agent, step)
  int tile_P;       // elements per lane-interleaved slice
  int soft_shadow;  // this is the shadow model of a call with observation vectors (weights chosen by the caller)
  int rank2_ok;     // no group over more than two factors: the pair window kernel applies
  int pair_ok;      // at most one group over two factors and none over more: the pair filtering kernel applies
  const void *tile_floor;   // device scalar: ln 1e-16 in the arithmetic type, as the pack kernels compute it
  long long slice_bytes_dense, slice_bytes_compressed;   // per-agent tile models: bytes of the two forms (0: none)
  int test_no_compress;     // testing aid (BI_TEST_NO_COMPRESS, read when the handle is made)
  int use_compressed;       // window calls gather from the compressed form (bi_model_set_compressed)
  // Register-tile models with few outcome combinations: the group's slices pre-summed for every
  // combination, [G][tile_ncomb][tile_P] in the lane-interleaved layout (one gather per step instead of
  // one per modality and no additions); combination index = sum_i outcome_i * tile_comb_mul[i] over the
  // group's members.  NULL when the table would be too large.
  void *tile_comb;
  int tile_ncomb;
  int tile_comb_mul[BI_MAX_M];
  int V0max, V1max; // floats needed by the generic kernel's two intermediate buffers
  int rows_max;     // largest first-level row count over groups
  int64_t launches;
  const char *last_kernel;
  void *ws;         // workspace of the batched window path (stream-ordered allocation), or NULL
  size_t ws_bytes;
  void *ws_soft;    // workspace of the calls that take observation vectors, or NULL
  size_t ws_soft_bytes;
  void *ws_prior;   // predictive log-priors of continued window calls, or NULL
  size_t ws_prior_bytes;
  double damping;   // step of the update on log-beliefs, (0, 1]; 1 = the plain fixed-point map
  void *carry;      // last belief of the latest filtering call, [carry_N][S] in the arithmetic type, or NULL
  size_t carry_bytes;
  int carry_N;      // agents of that call (0: none yet)
  // Testing aid, read from the environment once, when the handle is made (BI_TEST_FAMILY = "batch", "cta", "warp"
  // or "generic"): calls skip the kernel families ahead of the named one, so that the general kernels can
  // be checked on inputs small enough for the oracle.  0 = normal dispatch.
  int test_family;
  // Testing aid (BI_TEST_DROP_COPY = n, read when the handle is made): the next n batched window calls
  // announce their slice copies without issuing them, so that the bounded wait on the copy runs out and
  // the status flag BI_FLAG_COPY_TIMEOUT is raised; nothing faults, nothing is left in flight.
  int test_drop_copy;
};

struct BiCall {
  const bi_model *model;
  int algo, N, T, K;
  const int32_t *obs, *act;
  const float *q_prev;       // filtering continued from a belief [N][S], or NULL
  const int32_t *act_prev;   // [N][F], with q_prev (or with carry_in)
  // Filtering calls: the last step's belief of every agent, [N][S] in the handle's arithmetic type.
  // carry_in (or NULL) takes the place of q_prev at full precision; carry_out (or NULL) receives this
  // call's last belief.  (A trajectory filtered in consecutive calls then equals the single call
  // bit for bit: nothing is rounded to float32 on the way.)
  const void *carry_in;
  void *carry_out;
  const float *q_init;       // window algorithms: starting beliefs [N][T][S], or NULL (uniform)
  double lambda;             // damping: ln q' = (1 - lambda) ln q + lambda (messages) + const; 1 = plain
  const void *lnprior;       // window algorithms continued from a belief: ln(B_u q_prev) per agent,
                             // [N][S] in the handle's arithmetic type, used in the place of ln D; or NULL
  float *q_out, *logq_out;
  int32_t *argmax_out;
  cudaStream_t stream;
};

// kernel families; each returns BI_OK, BI_ERR_UNSUPPORTED (not applicable to
// this model / call: the dispatcher tries the next one) or an error.
int bi_launch_generic(const BiCall &c, bi_model *mut);
int bi_launch_warp(const BiCall &c, bi_model *mut);
int bi_launch_cta_filter(const BiCall &c, bi_model *mut);   // filtering only; slices staged per step
int bi_launch_pair_filter(const BiCall &c, bi_model *mut);  // filtering only; models coupled in at most one pair of factors
int bi_launch_pair_window(const BiCall &c, bi_model *mut);  // window calls on the same models; a CTA per agent
int bi_launch_tile3(const BiCall &c, bi_model *mut);
int bi_launch_tile3_window(const BiCall &c, bi_model *mut);
int bi_launch_batch(const BiCall &c, bi_model *mut);
// tries the kernel families in order (the dispatcher behind every inference call)
int bi_dispatch(const BiCall &c, bi_model *mut);
// inference with observations given as categorical vectors [N][T][sum m_i]
int bi_run_soft(const bi_model *model, int algo, int N, int T, const float *obs_soft, const int32_t *act, int iters,
                float *q_out, float *logq_out, int32_t *argmax_out, cudaStream_t stream);
// id of the batched path's unrolled shape for packed dims (rank, then the axis sizes), or -1
int bi_batch_shape(int rank, const int *dim);
// SB of the compiled register-tile shape for packed dims (na, nb, nc), or 0
int bi_tile3_shape(int na, int nb, int nc);
