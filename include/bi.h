/*
 * bi -- batched mean-field belief updates for factorised discrete HMMs/POMDPs
 * on NVIDIA B200 (sm_100a).  C ABI; no C++ or framework types cross it.
 *
 * Model (Section III-B of the paper): M observation modalities, F hidden-state
 * factors with n_f states, one control per factor with U_f actions;
 *   p(o, s | u) = p(s_1) prod_{t>=2} p(s_t | s_{t-1}, u_{t-1}; B) prod_t p(o_t | s_t; A).
 * A_i = P(o^i | s^{dep(i)}) for an arbitrary dependency list dep(i);
 * B_f = P(s^f_{t+1} | s^f_t, u^f_t) (trivial B-dependencies only).
 *
 * Every inference entry point computes, for N independent agents, the
 * posterior marginals q_{t,f} of a fully factorised approximation by iterating
 * the generic coordinate update of Section III-A,
 *   log q(s^f) = E_{q(s^{\f})}[ log p(o, s) ] + const,
 * whose expensive part is the likelihood message (Section III-C log-likelihood
 * with the observed outcome selecting a slice of log A_i, then the
 * marginalisation of Section IV):
 *   ell_{t,f}[s] = sum_{i: f in dep(i)} sum_{s_dep(i) \ f}
 *                  ln A_i[o_{t,i}, s_dep(i)] prod_{g in dep(i), g != f} q_{t,g}[s_g].
 * Conventions the paper leaves open and this library fixes:
 *   - all (t, f) are updated simultaneously from the previous iterate (Jacobi;
 *     the paper maps the window's steps onto parallel threads, Appendix A-2);
 *   - beliefs start uniform; exactly `iters` iterations run, no early exit;
 *   - ln x means ln(max(x, 1e-16)).
 *
 * Pointers are marked HOST or DEVICE.  All arrays are dense, row-major.
 * Inference calls are asynchronous on the given CUDA stream (a cudaStream_t
 * passed as void*, NULL = default stream) and never synchronise; the caller
 * owns every pointer it passes.  Nothing in this library falls back to the
 * CPU: without a usable CUDA device every call fails with BI_ERR_CUDA.
 */
#ifndef BI_H
#define BI_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* compile-time limits; exceeding one returns BI_ERR_UNSUPPORTED */
#define BI_MAX_F 8      /* hidden-state factors              */
#define BI_MAX_M 16     /* observation modalities            */
#define BI_MAX_RANK 5   /* factors one modality may depend on */
#define BI_MAX_N 32     /* states per factor                 */
#define BI_MAX_T 64     /* steps per window call (bi_vmp / bi_mmp) */

enum {
  BI_OK = 0,
  BI_ERR_INVALID_ARG = -1, /* null pointer, non-positive count, bad dependency id   */
  BI_ERR_SHAPE = -2,       /* N / G mismatch, repeated factor in a dependency list  */
  BI_ERR_UNSUPPORTED = -3, /* a BI_MAX_* limit or the on-chip working set exceeded  */
  BI_ERR_ALLOC = -4,       /* device allocation failed                              */
  BI_ERR_CUDA = -5         /* a CUDA runtime call failed / no device                */
};

/*
 * Arithmetic of the inference kernels.  Inputs and outputs are float32 either
 * way.  The Jacobi fixed-point map is not contractive on sharp or sparse
 * models (beliefs can oscillate between iterations), so rounding errors are
 * amplified by factors that reach 1e3 on dense models and 1e9 on sparse ones
 * within 16 iterations; float32 arithmetic then cannot reproduce a float64
 * evaluation to 1e-5.  BI_ARITH_F64 (the default) carries logs, beliefs and
 * accumulations in float64; BI_ARITH_F32 is the fast mode, exact to float32
 * rounding per operation but not to 1e-5 on ill-conditioned agents.
 */
#define BI_ARITH_F64 0
#define BI_ARITH_F32 1

/* bits of the device status word read by bi_status */
#define BI_FLAG_OBS_RANGE 1u /* an observation index was outside [0, m_i): clamped */
#define BI_FLAG_ACT_RANGE 2u /* an action index was outside [0, U_f): clamped      */
#define BI_FLAG_COPY_TIMEOUT 4u /* an asynchronous copy inside a kernel did not complete within its
                                   probe limit: the CTA left early and the call's outputs are invalid */

typedef struct bi_model bi_model_t; /* opaque; owns the packed device copies */

/*
 * Description of a generative model (the tuple that defines a POMDP
 * configuration in Section V-A, plus action counts and the arrays).
 */
typedef struct {
  int32_t F, M;
  const int32_t *n;       /* HOST [F]  state counts, 1 <= n_f <= BI_MAX_N          */
  const int32_t *m;       /* HOST [M]  outcome counts, m_i >= 1                    */
  const int32_t *dep_len; /* HOST [M]  k_i, 1 <= k_i <= BI_MAX_RANK                */
  const int32_t *dep;     /* HOST [sum k_i] 0-based factor ids, no repeats within a
                             list; A_i's hidden axes follow this order             */
  const int32_t *U;       /* HOST [F]  action counts, U_f >= 1                     */
  int32_t G;              /* 1: one model shared by all agents; else one per agent */
  const float *const *A;  /* HOST array of M DEVICE pointers;
                             A[i]: [G][m_i][n_dep(i)[0]]...[n_dep(i)[k_i-1]]       */
  const float *const *B;  /* HOST array of F DEVICE pointers;
                             B[f]: [G][n_f next][n_f previous][U_f]                */
  const float *const *D;  /* HOST array of F DEVICE pointers; D[f]: [G][n_f]       */
} bi_model_desc;

/*
 * Pack a model for inference (the once-only initialisation step of Section
 * III-C: layout work happens here, never at inference time).  Computes
 * ln(max(A, 1e-16)) in float64 (rounded once to float32 in BI_ARITH_F32), stores each
 * outcome's slice contiguously with modalities of equal dependency set sharing
 * one axis order; B is re-laid per action as forward, log, log-transposed and
 * column-normalised-transposed matrices; D as ln D.  The packed copies live in
 * device memory owned by the handle; the caller's A, B, D may be released once
 * the stream's work has completed.  Returns BI_OK and *out, or an error code
 * with *out = NULL.
 */
int bi_model_create(const bi_model_desc *desc, void *cuda_stream, bi_model_t **out);

/* As bi_model_create (which uses BI_ARITH_F64) with the arithmetic chosen. */
int bi_model_create_arith(const bi_model_desc *desc, int arith, void *cuda_stream, bi_model_t **out);

/*
 * Storage of a per-agent model's observation slices in the layout the window kernels gather from
 * (HOST outputs, bytes): *dense as full slices, *compressed as the handle keeps them when most of A is
 * zero -- the paper's motive for sparse storage, Section III-D: its BCOO variants cut parameter counts
 * 14-fold without a speed-up, Section V-B.  Here a slice becomes one 64-bit mask per lane (which of the
 * lane's elements are not the floor ln 1e-16) plus those values; bi_vmp / bi_mmp read that form, so the
 * gather's HBM traffic shrinks with the share of zeros; the result is bit for bit that of the dense
 * form.  Made automatically by bi_model_create for per-agent register-tile models (G > 1, up to four
 * modalities) when it is under 60 % of the dense size; sizing it needs the non-zero counts on the
 * host, so creating such a handle synchronises the stream.  Both are 0 when the handle has no
 * compressed form.
 */
int bi_model_slice_bytes(const bi_model_t *model, int64_t *dense, int64_t *compressed);

/*
 * Chooses the form later bi_vmp / bi_mmp calls on this handle gather from: on != 0 the compressed
 * one (BI_ERR_UNSUPPORTED when the handle has none), 0 the dense one (the default).  Measured on a
 * B200 with 70 % zeros: a third of the bytes from HBM, but the calls are not bound by that gather,
 * and decoding costs about 5 % more time; the switch is for deployments where HBM traffic or
 * capacity is the scarcer resource.
 */
int bi_model_set_compressed(bi_model_t *model, int on);

/* BI_ARITH_* of a handle, or BI_ERR_INVALID_ARG for NULL. */
int bi_model_arith(const bi_model_t *model);

/* Synchronises the device, frees the packed copies and the handle's workspaces.  NULL is accepted. */
/*
 * A model whose transitions have non-trivial B-dependencies: factor f's next state depends on the
 * previous states of a list of factors, p(s^f_{t+1} | s^{bdep(f)}_t, u^f_t) (Section III-B restricts
 * itself to the trivial case bdep(f) = {f}; Section VI names the general case as the next step).
 *   bdep_len  HOST [F]: k_f >= 1, at most BI_MAX_RANK
 *   bdep      HOST [sum k_f]: 0-based factor ids, no repeats within a list (f itself need not be in it)
 *   desc->B[f] DEVICE [G][n_f next][n_{bdep(f)[0]}]...[n_{bdep(f)[k-1]}][U_f] row-major, at most 2^20
 *             entries per model; everything else of desc as for bi_model_create
 * The mean-field update of Section III-A then gives: filtering, prior of a step = the transition
 * tensor contracted with the previous step's beliefs of all its parents; VMP, past message = the
 * tensor of logarithms contracted likewise, future message to a factor = the sum, over the factors
 * whose transitions read it, of the log-tensor contracted with the next step's belief of that factor
 * and this step's beliefs of the other parents.  Such handles serve bi_filter, bi_filter_from,
 * bi_filter_continue, bi_vmp and bi_vmp_warm (the general kernel families; damping applies).  Marginal
 * message passing has no reversed transition for several parents: bi_mmp and its variants, the calls
 * with observation vectors and bi_vmp_from return BI_ERR_UNSUPPORTED on such a handle.
 * Errors as bi_model_create; BI_ERR_INVALID_ARG for a malformed list, BI_ERR_UNSUPPORTED beyond the limits.
 */
int bi_model_create_bdep(const bi_model_desc *desc, const int32_t *bdep_len, const int32_t *bdep, int arith,
                         void *cuda_stream, bi_model_t **out);

int bi_model_destroy(bi_model_t *model);

/*
 * Damped updates (optional; the paper's iteration is the plain one, lambda = 1).
 * Every later inference call on the handle replaces the update of a factor by
 *   ln q' = (1 - lambda) ln q + lambda (likelihood message + transition messages) + const,
 * a step of size lambda on the log-beliefs towards the plain update; ln q of a
 * starting belief is ln max(q, 1e-16).  The plain Jacobi map oscillates on many
 * models (see BI_ARITH_*); a step below 1 damps that and, with it, the
 * amplification of rounding errors.  0 < lambda <= 1, else BI_ERR_INVALID_ARG.
 */
int bi_model_set_damping(bi_model_t *model, double lambda);

/*
 * Threads and streams.  A handle may be used from any thread, but its inference
 * calls must not overlap on the GPU: the status word, the launch bookkeeping and
 * its workspaces (of the batched window path for shared models, of the calls that
 * take observation vectors and of the continued window calls; all obtained from the stream-ordered allocator
 * on first need, grown on demand and kept until bi_model_destroy) belong to the
 * handle.  Issue a handle's calls on one stream, or order the streams with
 * events; for concurrent inference on one model create one handle per stream.
 * All other calls allocate nothing.
 */

/*
 * Variational filtering by fixed-point iteration ("FPI", Sections I and IV).
 * For each agent and t = 1..T in order:
 *   prior_t = D (t = 1) or B_{u_{t-1}} q_{t-1} (final belief of step t-1),
 *   q <- uniform; repeat `iters` times, all factors at once:
 *   q_{t,f} <- softmax( ell_{t,f}(q) + ln prior_{t,f} ).
 *
 *   N, T      agents, time steps (N >= 0, T >= 1); if model G != 1 then N == G
 *   obs       DEVICE [N][T][M]   int32, 0 <= obs < m_i
 *   act       DEVICE [N][T-1][F] int32, 0 <= act < U_f; may be NULL when T == 1
 *   iters     K >= 1
 *   q_out     DEVICE [N][T][S] float32, S = sum n_f, factor f at offset sum_{g<f} n_g
 *   logq_out  DEVICE [N][T][S] float32 log-beliefs, or NULL
 *   argmax_out DEVICE [N][T][F] int32 most probable state (lowest index on ties), or NULL
 * Out-of-range indices are clamped and flagged in the status word; nothing traps.
 */
int bi_filter(const bi_model_t *model, int32_t N, int32_t T, const int32_t *obs,
              const int32_t *act, int32_t iters, float *q_out, float *logq_out,
              int32_t *argmax_out, void *cuda_stream);

/*
 * Variational message passing over one window of T steps (Sections I, IV and
 * Appendix A-2).  All (t, f) at once, `iters` times:
 *   q_{t,f} <- softmax( ell_{t,f}(q_t) + past + future ),
 *   past   = ln D_f (t = 1) or (ln B_{u_{t-1}}) q_{t-1,f},
 *   future = 0 (t = T) or (ln B_{u_t})^T q_{t+1,f}.
 * Arguments as bi_filter; T <= BI_MAX_T.
 */
int bi_vmp(const bi_model_t *model, int32_t N, int32_t T, const int32_t *obs,
           const int32_t *act, int32_t iters, float *q_out, float *logq_out,
           int32_t *argmax_out, void *cuda_stream);

/*
 * Marginal message passing over one window of T steps.  Same loop as bi_vmp with
 *   past   = ln D_f (t = 1) or 1/2 ln( B_{u_{t-1}} q_{t-1,f} ),
 *   future = 0 (t = T) or 1/2 ln( Bdag_{u_t} q_{t+1,f} ),
 * Bdag = transpose of B_u with each column renormalised (zero sum -> uniform).
 * The paper names the algorithm and cites its source without printing these
 * formulas; this is the library's stated reading of it.
 */
int bi_mmp(const bi_model_t *model, int32_t N, int32_t T, const int32_t *obs,
           const int32_t *act, int32_t iters, float *q_out, float *logq_out,
           int32_t *argmax_out, void *cuda_stream);

/*
 * Variational filtering continued from a known belief: the recursion of
 * bi_filter (Section III-B: prior of a step = B_u applied to the previous
 * step's belief) entered mid-stream.  For an agent that receives its
 * observations over time -- one call per tick, or per block of ticks -- and
 * for splitting a long trajectory into pieces whose results can be copied out
 * while the next piece runs.
 *   q_prev    DEVICE [N][S] float32: each agent's belief at the step before this
 *             window (normally the last step of the previous call's q_out)
 *   act_prev  DEVICE [N][F] int32: the action taken at that step, u in [0, U_f)
 *   others    as for bi_filter (act is [N][T-1][F]; may be NULL when T == 1)
 * The first step's prior is B_{act_prev} q_prev instead of D; everything else is
 * bi_filter.  Because q_prev carries float32 rounding, a split run equals the
 * uninterrupted one only up to that rounding (and to what the iteration makes of
 * it).  Each agent's q_prev row is read before that agent's outputs are written,
 * so with T == 1 q_prev and q_out may be the same buffer (an in-place tick).
 * Returns BI_ERR_INVALID_ARG when q_prev or act_prev is NULL.
 */
int bi_filter_from(const bi_model_t *model, int32_t N, int32_t T, const int32_t *obs,
                   const int32_t *act, const float *q_prev, const int32_t *act_prev,
                   int32_t iters, float *q_out, float *logq_out, int32_t *argmax_out,
                   void *cuda_stream);

/*
 * Variational filtering continued from the handle's own record of where the
 * previous filtering call on this handle stopped (the same recursion of Section
 * III-B entered mid-stream, as bi_filter_from).  Every bi_filter,
 * bi_filter_from and bi_filter_continue call leaves the last step's belief of
 * each of its N agents in a device buffer the handle owns, in the handle's
 * arithmetic (float64 by default), and this call starts from that buffer.
 * Nothing is rounded to float32 on the way, so a trajectory filtered as
 * consecutive blocks of steps -- the first with bi_filter, the rest with this
 * call -- gives bit for bit the beliefs of one bi_filter call over all the
 * steps, which bi_filter_from (float32 q_prev) cannot promise on models whose
 * iteration amplifies rounding.
 *   act_prev  DEVICE [N][F] int32: the action taken at the previous call's last step
 *   others    as for bi_filter (act is [N][T-1][F]; may be NULL when T == 1)
 * The calls must be issued in order on one stream (or otherwise ordered); N must
 * equal the previous filtering call's N, else BI_ERR_INVALID_ARG (also when
 * there was no previous call, or it failed).  Calls with observation vectors
 * (bi_filter_soft) and bi_filter_static neither read nor update the record.
 * The buffer is N * S elements, obtained from the stream-ordered allocator at
 * the first filtering call (and again when N grows), freed by bi_model_destroy.
 */
int bi_filter_continue(const bi_model_t *model, int32_t N, int32_t T, const int32_t *obs,
                       const int32_t *act, const int32_t *act_prev, int32_t iters, float *q_out,
                       float *logq_out, int32_t *argmax_out, void *cuda_stream);

/*
 * bi_vmp / bi_mmp started from given beliefs instead of the uniform ones: the
 * warm start of a sliding inference window (Section III-A: inference over a
 * horizon that advances with t), where the previous window's result, shifted by
 * one step, is the natural starting point.
 *   q_init    DEVICE [N][T][S] float32: the starting belief of every step, laid out
 *             like q_out; each factor's block is used as given (not renormalised).
 *             Must not overlap q_out.
 *   others    as for bi_vmp / bi_mmp
 * The iterates are the same Jacobi sweeps; only iterate 0 differs.
 */
int bi_vmp_warm(const bi_model_t *model, int32_t N, int32_t T, const int32_t *obs,
                const int32_t *act, const float *q_init, int32_t iters, float *q_out,
                float *logq_out, int32_t *argmax_out, void *cuda_stream);
int bi_mmp_warm(const bi_model_t *model, int32_t N, int32_t T, const int32_t *obs,
                const int32_t *act, const float *q_init, int32_t iters, float *q_out,
                float *logq_out, int32_t *argmax_out, void *cuda_stream);

/*
 * bi_vmp / bi_mmp over a window that continues a stream (the sliding inference
 * window of Section III-B: the current step together with the preceding h
 * steps).  As in bi_filter_from, q_prev [N][S] is each agent's belief at the
 * step before the window and act_prev [N][F] the action taken there; the first
 * step's past message is then ln(B_{act_prev} q_prev) at full weight, i.e. the
 * model's prior D is replaced, per agent, by the predictive prior.  q_init may
 * be NULL (uniform start) or DEVICE [N][T][S] as in bi_vmp_warm.  A small
 * [N][S] workspace is obtained from the stream-ordered allocator on first use.
 */
int bi_vmp_from(const bi_model_t *model, int32_t N, int32_t T, const int32_t *obs,
                const int32_t *act, const float *q_prev, const int32_t *act_prev,
                const float *q_init, int32_t iters, float *q_out, float *logq_out,
                int32_t *argmax_out, void *cuda_stream);
int bi_mmp_from(const bi_model_t *model, int32_t N, int32_t T, const int32_t *obs,
                const int32_t *act, const float *q_prev, const int32_t *act_prev,
                const float *q_init, int32_t iters, float *q_out, float *logq_out,
                int32_t *argmax_out, void *cuda_stream);

/*
 * The three algorithms with every observation given as categorical vectors
 * (Section III-B: an observation modality is represented as a categorical
 * probability vector of length m_i) instead of an index.  The log-likelihood
 * term of modality i at a step is then log(A_i) . o^i = sum_o o^i[o] ln A_i[o, .]
 * (Section III-C); a one-hot vector reproduces the index form.
 *   obs_soft  DEVICE [N][T][sum_i m_i] float32: per step the modalities' vectors one
 *             after the other, in modality order; used as weights as given (not
 *             checked or renormalised)
 *   others    as for bi_filter / bi_vmp / bi_mmp
 * The call first forms the weighted slices of every (agent, step) in a workspace
 * of N * T * (sum over dependency groups of the padded slice size) elements of
 * the handle's arithmetic type (twice that for register-tile models), obtained
 * from the stream-ordered allocator on first use and kept in the handle, then
 * runs the same inference kernels on them.  BI_ERR_ALLOC if the workspace cannot
 * be obtained; BI_ERR_UNSUPPORTED if sum_i m_i exceeds 768 (1536 in float32 arithmetic).
 */
int bi_filter_soft(const bi_model_t *model, int32_t N, int32_t T, const float *obs_soft,
                   const int32_t *act, int32_t iters, float *q_out, float *logq_out,
                   int32_t *argmax_out, void *cuda_stream);
int bi_vmp_soft(const bi_model_t *model, int32_t N, int32_t T, const float *obs_soft,
                const int32_t *act, int32_t iters, float *q_out, float *logq_out,
                int32_t *argmax_out, void *cuda_stream);
int bi_mmp_soft(const bi_model_t *model, int32_t N, int32_t T, const float *obs_soft,
                const int32_t *act, int32_t iters, float *q_out, float *logq_out,
                int32_t *argmax_out, void *cuda_stream);

/*
 * Variational filtering without any allocation.  (The paper has no counterpart
 * to this entry point: it is a deployment convenience of this library.)
 *
 * bi_model_create obtains device memory for the packed model, so it cannot be
 * used by callers that are not allowed to allocate: a control loop on a GPU
 * whose memory was handed out in full at start-up, a plug-in confined to
 * another runtime's memory pool, or any path that cannot tolerate the device
 * synchronisation cudaMalloc and cudaFree imply.  For them this call packs the
 * model into a fixed scratch array inside the library
 * (BI_STATIC_SCRATCH_BYTES of device memory per GPU that loads the library,
 * held until the process exits), runs the general filtering kernel on that
 * copy in float64 arithmetic and returns; it calls no cudaMalloc, no cudaFree
 * and no host allocator.
 *
 *   desc      as for bi_model_create; only shared models (G == 1)
 *   others    as for bi_filter
 * Results are identical to bi_filter on a handle made from the same desc when
 * that call runs the general kernel.  Returns BI_ERR_UNSUPPORTED if the packed
 * model (float64 logs of every A_i, transition matrices, priors) needs more
 * than BI_STATIC_SCRATCH_BYTES or the model is per-agent.
 * The first call on a device looks up the scratch array's device address; make
 * that first call outside any stream capture.  All calls share the one array,
 * which keeps the previous call's contents: every call re-packs the model and
 * clears its status word, and two calls whose GPU work overlaps (different
 * streams, different threads) race on it -- serialise them.  Out-of-range
 * indices are clamped as in bi_filter; no status word is reported.
 */
#define BI_STATIC_SCRATCH_BYTES (4u << 20)
int bi_filter_static(const bi_model_desc *desc, int32_t N, int32_t T, const int32_t *obs,
                     const int32_t *act, int32_t iters, float *q_out, float *logq_out,
                     int32_t *argmax_out, void *cuda_stream);


/* Synchronises the stream, returns the OR of BI_FLAG_* raised since the last
 * call in *flags (HOST) and clears them. */
int bi_status(const bi_model_t *model, void *cuda_stream, uint32_t *flags);

/* Name of the kernel family the dispatcher picked for the most recent
 * inference call on this handle ("" before the first call).  Static storage. */
const char *bi_last_kernel(const bi_model_t *model);

/* Number of kernel launches issued by inference calls on this handle so far. */
int64_t bi_launch_count(const bi_model_t *model);

/* Human-readable text for an error code.  Static storage. */
const char *bi_strerror(int code);

#ifdef __cplusplus
}
#endif
#endif /* BI_H */
