/*
 * CPU oracle for batched mean-field belief updates on factorised discrete
 * HMMs/POMDPs.  TEST INFRASTRUCTURE ONLY: the tests, the smoke check and the
 * benchmark's CPU-baseline leg call it; the CUDA library never does, and the
 * two share no code.
 *
 * Plain C, float64 arithmetic on float32 inputs widened exactly.  Nothing is
 * blocked, fused or reordered: every function below is the definition it cites
 * written as loops.
 *
 * Generative model (Section III-B): p(o,s|u) = p(s_1) prod_t p(s_t|s_{t-1},
 * u_{t-1}; B) prod_t p(o_t|s_t; A), with M observation modalities, F hidden
 * factors, one control per factor, arbitrary A-dependencies and trivial
 * B-dependencies.  Posterior approximation q(s) = prod_{t,f} q_{t,f}.
 *
 * Update (Section III-A, the generic mean-field coordinate update):
 *     log q(s^f) = E_{q(s^{\f})}[ log p(o, s) ] + const,
 * which for this model splits into a likelihood message (the log-likelihood
 * log(A_i).o^i of Section III-C marginalised over the other factors of each
 * modality's dependency list, Section IV) plus prior / transition messages.
 *
 * The paper names the three algorithms (FPI = variational filtering by fixed
 * point iteration, VMP, MMP) without printing their equations; the readings
 * taken here are:
 *   - schedule: Jacobi -- every (t, f) of iteration k+1 reads iteration k only
 *     (the paper maps the window's time steps onto parallel threads, App. A-2);
 *   - initial beliefs uniform (or a caller-supplied start, used by the tests);
 *   - exactly K iterations, no early exit;
 *   - log of a probability is ln(max(x, 1e-16));
 *   - filtering: prior_t = D (t = 1) or B_u q_{t-1} computed once per step
 *     outside the iteration (FPI itself only computes likelihood messages,
 *     Section IV); q <- softmax(lik + ln prior);
 *   - VMP: past = ln D (t = 1) or (ln B_u) q_{t-1}; future = (ln B_u)^T q_{t+1}
 *     (0 at the last step);
 *   - MMP: past = ln D (t = 1) or 1/2 ln(B_u q_{t-1}); future = 1/2 ln(Bdag_u
 *     q_{t+1}) (0 at the last step), Bdag = transpose of B_u with every column
 *     renormalised (a zero sum gives a uniform column).
 * Pins: filtering, VMP and the free-energy property are pinned by closed forms
 * and brute-force enumeration in the CPU tests.  MMP is pinned by a hand-worked
 * two-step window whose backward message varies over states, by a permutation
 * transition, by an unreachable-state case, and by a restatement of the update
 * from the model's definition (likelihood by enumeration, Bayes reversal of the
 * transition by conditioning an enumerated joint table).  What no test can
 * settle is whether this reading of "MMP" (1/2 weights, reversed transition
 * under a uniform prior, D at full weight) is the one the paper's authors ran:
 * Section IV names the algorithm and prints no equation.
 *
 * Non-trivial B-dependencies (the extension Section VI leaves as future work; Section III-B restricts
 * itself to the trivial case): factor f's transition may depend on the previous states of a list
 * bdep(f) of factors, p(s^f_{t+1} | s^{bdep(f)}_t, u^f_t) = B_f[s', s_bdep..., u].  The same mean-field
 * update (Section III-A) then gives
 *   - filtering: prior_t,f[s'] = sum_{s_par} B_f[s', s_par, u] prod_{g in bdep(f)} q_{t-1,g}[s_g];
 *   - VMP past message to (t, f): sum_{s_par} ln B_f[s', s_par, u_{t-1}] prod_g q_{t-1,g}[s_g];
 *     future message to (t, g): sum over the factors h with g in bdep(h) of
 *       sum_{s'} q_{t+1,h}[s'] sum_{s_par \ g} ln B_h[s', s_par, u_t] prod_{j in bdep(h), j != g} q_{t,j}[s_j];
 *   - MMP is not defined for them here (its reversed transition has no counterpart with several
 *     parents): such a call is rejected.
 *
 * Layouts (row-major):
 *   A[i]: [G][m_i][n_{dep(i)[0]}]...[n_{dep(i)[k-1]}]   float32
 *   B[f]: [G][n_f next][n_f prev][U_f]                   float32
 *         (with B-dependencies: [G][n_f next][n_{bdep(f)[0]}]...[n_{bdep(f)[k-1]}][U_f])
 *   D[f]: [G][n_f]                                       float32
 *   obs:  [N][T][M] int32     act: [N][T-1][F] int32
 *   q, logq: [N][T][S] float64 (factor f at offset sum_{g<f} n_g)
 *   argmax: [N][T][F] int32 (lowest index among exactly tied logits)
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define BI_REF_EPS 1e-16
#define BI_REF_MAXK 16

enum { ALGO_FILTER = 0, ALGO_VMP = 1, ALGO_MMP = 2 };

typedef struct {
    int F, M, G, S;
    const int32_t *n, *m, *dep_len, *dep, *U;
    const float *const *A;
    const float *const *B;
    const float *const *D;
    int *off;      /* [F] offset of factor f in a belief vector */
    int *dep_off;  /* [M] offset of modality i's list in dep     */
    int64_t *P;    /* [M] product of the sizes of the factors in dep(i) */
    int *moff;     /* [M] offset of modality i's block in a soft observation vector */
    int Mtot;      /* sum of m_i */
    int round32;   /* conditioning probe: round logs and beliefs to float32 */
    double lambda; /* damping of the log-belief update: 1 = the plain fixed-point map */
    /* B-dependencies: NULL = trivial (every factor depends on its own previous state) */
    const int32_t *bdep_len, *bdep;
    int *bdep_off;  /* [F] offset of factor f's list in bdep */
    int64_t *PB;    /* [F] product of the sizes of the factors in bdep(f) */
} model_t;

static double log_eps(double x, int round32)
{
    double v = log(x > BI_REF_EPS ? x : BI_REF_EPS);
    return round32 ? (double)(float)v : v;
}

/* B_{f,u}[s_next, s_prev] of model g */
static double B_at(const model_t *md, int g, int f, int u, int s_next, int s_prev)
{
    int nf = md->n[f], Uf = md->U[f];
    return (double)md->B[f][(((size_t)g * nf + s_next) * nf + s_prev) * Uf + u];
}

/* B_f[s_next, parents, u] of model g with B-dependencies; par is the row-major index of the parents'
 * states in bdep(f) order */
static double B_par(const model_t *md, int g, int f, int u, int s_next, int64_t par)
{
    int nf = md->n[f], Uf = md->U[f];
    return (double)md->B[f][((((size_t)g * nf + s_next) * (size_t)md->PB[f]) + (size_t)par) * Uf + u];
}

/* sum_{parents} X(B_f[s_next, parents, u]) prod_{g in bdep(f)} q_g[s_g], X = identity or the clamped log;
 * q is one step's belief vector [S] */
static double transition_expectation(const model_t *md, int g, int f, int u, int s_next, const double *q, int take_log)
{
    int k = md->bdep_len[f];
    const int32_t *d = md->bdep + md->bdep_off[f];
    int idx[BI_REF_MAXK];
    for (int j = 0; j < k; ++j) idx[j] = 0;
    double total = 0.0;
    for (int64_t e = 0; e < md->PB[f]; ++e) {
        double w = 1.0;
        for (int j = 0; j < k; ++j) w *= q[md->off[d[j]] + idx[j]];
        double b = B_par(md, g, f, u, s_next, e);
        total += (take_log ? log_eps(b, md->round32) : b) * w;
        for (int j = k - 1; j >= 0; --j) {
            if (++idx[j] < md->n[d[j]]) break;
            idx[j] = 0;
        }
    }
    return total;
}

/* VMP future message to factor f0 at a step, state s: over every factor h whose transition depends on f0,
 * sum_{s'} qn_h[s'] sum_{parents with s_f0 = s} ln B_h[s', parents, u_h] prod_{other parents} q_j[s_j];
 * q: this step's beliefs, qn: the next step's, act_t: the actions taken at this step [F] */
static double future_message_bdep(const model_t *md, int g, int f0, int s, const double *q, const double *qn,
                                  const int32_t *act_t)
{
    double total = 0.0;
    for (int h = 0; h < md->F; ++h) {
        int k = md->bdep_len[h], pos = -1;
        const int32_t *d = md->bdep + md->bdep_off[h];
        for (int j = 0; j < k; ++j) if (d[j] == f0) pos = j;
        if (pos < 0) continue;
        int idx[BI_REF_MAXK];
        for (int j = 0; j < k; ++j) idx[j] = 0;
        for (int64_t e = 0; e < md->PB[h]; ++e) {
            if (idx[pos] == s) {
                double w = 1.0;
                for (int j = 0; j < k; ++j) if (j != pos) w *= q[md->off[d[j]] + idx[j]];
                for (int sn = 0; sn < md->n[h]; ++sn)
                    total += qn[md->off[h] + sn] * log_eps(B_par(md, g, h, act_t[h], sn, e), md->round32) * w;
            }
            for (int j = k - 1; j >= 0; --j) {
                if (++idx[j] < md->n[d[j]]) break;
                idx[j] = 0;
            }
        }
    }
    return total;
}

/*
 * Likelihood message to every factor at one time step (Section III-C
 * log-likelihood with a one-hot observation, then the marginalisation of
 * Section IV):
 *   ell_f[s] = sum_{i: f in dep(i)} sum_{s_dep(i) \ f}
 *              ln A_i[o_i, s_dep(i) with s_f = s] * prod_{g in dep(i), g != f} q_g[s_g].
 * With soft_t (the step's observation given as one categorical vector per
 * modality, Section III-B; [Mtot] floats, modality blocks in order) the term
 * ln A_i[o_i, .] is the contraction over the observation axis of Section
 * III-C, log(A_i) . o^i = sum_o o^i[o] ln A_i[o, .]; obs_t is then unused.
 */
static void likelihood_messages(const model_t *md, int g, const int32_t *obs_t, const float *soft_t,
                                const double *q, double *ell)
{
    for (int s = 0; s < md->S; ++s) ell[s] = 0.0;
    for (int i = 0; i < md->M; ++i) {
        int k = md->dep_len[i];
        const int32_t *d = md->dep + md->dep_off[i];
        int64_t P = md->P[i];
        const float *slice = md->A[i] + ((size_t)g * md->m[i] + (size_t)(soft_t ? 0 : obs_t[i])) * (size_t)P;
        int idx[BI_REF_MAXK];
        for (int j = 0; j < k; ++j) idx[j] = 0;
        for (int64_t e = 0; e < P; ++e) {
            double la;
            if (soft_t) {
                la = 0.0;
                for (int o = 0; o < md->m[i]; ++o)
                    la += (double)soft_t[md->moff[i] + o] * log_eps((double)slice[(size_t)o * (size_t)P + e], md->round32);
            } else {
                la = log_eps((double)slice[e], md->round32);
            }
            for (int j = 0; j < k; ++j) {
                double w = 1.0;
                for (int jj = 0; jj < k; ++jj)
                    if (jj != j) w *= q[md->off[d[jj]] + idx[jj]];
                ell[md->off[d[j]] + idx[j]] += la * w;
            }
            /* next multi-index, last axis fastest */
            for (int j = k - 1; j >= 0; --j) {
                if (++idx[j] < md->n[d[j]]) break;
                idx[j] = 0;
            }
        }
    }
}

/* softmax of x[0..n) into q, log-softmax into lq (may be NULL), argmax (lowest index) */
static int softmax_vec(const double *x, int n, double *q, double *lq, int round32)
{
    double mx = x[0];
    int am = 0;
    for (int s = 1; s < n; ++s)
        if (x[s] > mx) { mx = x[s]; am = s; }
    double z = 0.0;
    for (int s = 0; s < n; ++s) z += exp(x[s] - mx);
    double lz = log(z);
    for (int s = 0; s < n; ++s) {
        double v = exp(x[s] - mx) / z;
        q[s] = round32 ? (double)(float)v : v;
        if (lq) lq[s] = x[s] - mx - lz;
    }
    return am;
}

static void set_initial(const model_t *md, const double *q_init, double *q)
{
    if (q_init) {
        memcpy(q, q_init, sizeof(double) * (size_t)md->S);
        return;
    }
    for (int f = 0; f < md->F; ++f)
        for (int s = 0; s < md->n[f]; ++s) q[md->off[f] + s] = 1.0 / md->n[f];
}

/* ---- variational filtering (FPI) for one agent ------------------------- */
/* q_prev / act_prev (both NULL, or both given): the belief of the step before the
 * window, [S], and the action taken at that step, [F]; the first step's prior is
 * then B_u q_prev, the same recursion as every later step, instead of D. */
static void filter_agent(const model_t *md, int g, int T, int K, const int32_t *obs, const float *soft,
                         const int32_t *act, const double *q_init, const double *q_prev,
                         const int32_t *act_prev, double *q_out,
                         double *lq_out, int32_t *am_out)
{
    int S = md->S, F = md->F;
    double *lprior = malloc(sizeof(double) * S), *ell = malloc(sizeof(double) * S);
    double *cur = malloc(sizeof(double) * S), *nxt = malloc(sizeof(double) * S);
    double *x = malloc(sizeof(double) * S), *lq = malloc(sizeof(double) * S);
    int32_t *am = malloc(sizeof(int32_t) * F);
    for (int t = 0; t < T; ++t) {
        /* prior: D at the first step, else B_u q_{t-1} with the previous step's final belief */
        for (int f = 0; f < F; ++f) {
            int nf = md->n[f], o = md->off[f];
            for (int s = 0; s < nf; ++s) {
                double p;
                if (t == 0 && !q_prev) {
                    p = (double)md->D[f][(size_t)g * nf + s];
                } else {
                    int u = t == 0 ? act_prev[f] : act[(size_t)(t - 1) * F + f];
                    const double *qp = t == 0 ? q_prev + o : q_out + (size_t)(t - 1) * S + o;
                    p = 0.0;
                    if (md->bdep_len) p = transition_expectation(md, g, f, u, s, qp - o, 0);
                    else for (int r = 0; r < nf; ++r) p += B_at(md, g, f, u, s, r) * qp[r];
                }
                lprior[o + s] = log_eps(p, md->round32);
            }
        }
        set_initial(md, q_init ? q_init + (size_t)t * S : NULL, cur);
        for (int s = 0; s < S; ++s) lq[s] = log_eps(cur[s], 0);
        for (int k = 0; k < K; ++k) {
            likelihood_messages(md, g, obs ? obs + (size_t)t * md->M : NULL,
                                soft ? soft + (size_t)t * md->Mtot : NULL, cur, ell);
            for (int f = 0; f < F; ++f) {
                int nf = md->n[f], o = md->off[f];
                /* damped update on log-beliefs: ln q' = (1 - lambda) ln q + lambda (message + ln prior) + const */
                for (int s = 0; s < nf; ++s)
                    x[o + s] = (1.0 - md->lambda) * lq[o + s] + md->lambda * (ell[o + s] + lprior[o + s]);
                am[f] = softmax_vec(x + o, nf, nxt + o, lq + o, md->round32);
            }
            double *tmp = cur; cur = nxt; nxt = tmp;
        }
        memcpy(q_out + (size_t)t * S, cur, sizeof(double) * S);
        if (lq_out) memcpy(lq_out + (size_t)t * S, lq, sizeof(double) * S);
        if (am_out) memcpy(am_out + (size_t)t * F, am, sizeof(int32_t) * F);
    }
    free(lprior); free(ell); free(cur); free(nxt); free(x); free(lq); free(am);
}

/* ---- VMP / MMP over one window for one agent --------------------------- */
/* q_prev / act_prev (both NULL, or both given): as for filter_agent, the belief of
 * the step before the window and the action taken there; the first step's past
 * message is then ln(B_u q_prev) at full weight, i.e. the window's prior D is
 * replaced by the predictive prior the filtering recursion would use. */
static void window_agent(const model_t *md, int algo, int g, int T, int K,
                         const int32_t *obs, const float *soft, const int32_t *act, const double *q_init,
                         const double *q_prev, const int32_t *act_prev,
                         double *q_out, double *lq_out, int32_t *am_out)
{
    int S = md->S, F = md->F;
    size_t TS = (size_t)T * S;
    double *cur = malloc(sizeof(double) * TS), *nxt = malloc(sizeof(double) * TS);
    double *lq = malloc(sizeof(double) * TS), *ell = malloc(sizeof(double) * S);
    double *x = malloc(sizeof(double) * S);
    int32_t *am = malloc(sizeof(int32_t) * (size_t)T * F);
    for (int t = 0; t < T; ++t) set_initial(md, q_init ? q_init + (size_t)t * S : NULL, cur + (size_t)t * S);
    for (size_t i = 0; i < TS; ++i) lq[i] = log_eps(cur[i], 0);
    for (int k = 0; k < K; ++k) {
        for (int t = 0; t < T; ++t) {
            const double *qt = cur + (size_t)t * S;
            likelihood_messages(md, g, obs ? obs + (size_t)t * md->M : NULL,
                                soft ? soft + (size_t)t * md->Mtot : NULL, qt, ell);
            for (int f = 0; f < F; ++f) {
                int nf = md->n[f], o = md->off[f];
                for (int s = 0; s < nf; ++s) {
                    double past, future = 0.0;
                    if (t == 0 && q_prev) {
                        double p = 0.0;
                        if (md->bdep_len) p = transition_expectation(md, g, f, act_prev[f], s, q_prev, 0);
                        else for (int r = 0; r < nf; ++r) p += B_at(md, g, f, act_prev[f], s, r) * q_prev[o + r];
                        past = log_eps(p, md->round32);
                    } else if (t == 0) {
                        past = log_eps((double)md->D[f][(size_t)g * nf + s], md->round32);
                    } else {
                        int u = act[(size_t)(t - 1) * F + f];
                        const double *qp = cur + (size_t)(t - 1) * S + o;
                        if (algo == ALGO_VMP && md->bdep_len) {
                            past = transition_expectation(md, g, f, u, s, qp - o, 1);
                        } else if (algo == ALGO_VMP) {
                            past = 0.0;
                            for (int r = 0; r < nf; ++r)
                                past += log_eps(B_at(md, g, f, u, s, r), md->round32) * qp[r];
                        } else {
                            double p = 0.0;
                            for (int r = 0; r < nf; ++r) p += B_at(md, g, f, u, s, r) * qp[r];
                            past = 0.5 * log_eps(p, md->round32);
                        }
                    }
                    if (t + 1 < T) {
                        int u = act[(size_t)t * F + f];
                        const double *qn = cur + (size_t)(t + 1) * S + o;
                        if (algo == ALGO_VMP && md->bdep_len) {
                            future = future_message_bdep(md, g, f, s, qt, qn - o, act + (size_t)t * F);
                        } else if (algo == ALGO_VMP) {
                            for (int r = 0; r < nf; ++r)
                                future += log_eps(B_at(md, g, f, u, r, s), md->round32) * qn[r];
                        } else {
                            /* Bdag_u[s, r] = B_u[r, s] / sum_{s'} B_u[r, s'] */
                            double p = 0.0;
                            for (int r = 0; r < nf; ++r) {
                                double rowsum = 0.0;
                                for (int sp = 0; sp < nf; ++sp) rowsum += B_at(md, g, f, u, r, sp);
                                double bd = rowsum > 0.0 ? B_at(md, g, f, u, r, s) / rowsum : 1.0 / nf;
                                p += bd * qn[r];
                            }
                            future = 0.5 * log_eps(p, md->round32);
                        }
                    }
                    x[o + s] = (1.0 - md->lambda) * lq[(size_t)t * S + o + s] + md->lambda * (ell[o + s] + past + future);
                }
                am[(size_t)t * F + f] = softmax_vec(x + o, nf, nxt + (size_t)t * S + o,
                                                    lq + (size_t)t * S + o, md->round32);
            }
        }
        double *tmp = cur; cur = nxt; nxt = tmp;
    }
    memcpy(q_out, cur, sizeof(double) * TS);
    if (lq_out) memcpy(lq_out, lq, sizeof(double) * TS);
    if (am_out) memcpy(am_out, am, sizeof(int32_t) * (size_t)T * F);
    free(cur); free(nxt); free(lq); free(ell); free(x); free(am);
}

/*
 * Run one algorithm over N agents.  q_init (may be NULL = uniform) is
 * [N][T][S]: the iteration's starting beliefs per step.  threads <= 0 uses the
 * OpenMP default; agents are independent, so threading is over agents only.
 * Returns 0, or a negative value for an invalid argument.
 */
static int run_impl(int algo, int F, int M, const int32_t *n, const int32_t *m,
                    const int32_t *dep_len, const int32_t *dep, const int32_t *U, int G,
                    const float *const *A, const float *const *B, const float *const *D,
                    int N, int T, const int32_t *obs, const float *obs_soft, const int32_t *act, int K,
                    const double *q_init, const double *q_prev, const int32_t *act_prev,
                    double *q_out, double *logq_out,
                    int32_t *argmax_out, int threads, int round32, double lambda,
                    const int32_t *bdep_len, const int32_t *bdep)
{
    if (algo < 0 || algo > 2 || F < 1 || M < 0 || N < 0 || T < 1 || K < 1) return -1;
    if ((bdep_len != NULL) != (bdep != NULL)) return -1;
    if (bdep_len && algo == ALGO_MMP) return -1;   /* not defined for several parents */
    if (!(lambda > 0.0 && lambda <= 1.0)) return -1;
    if ((q_prev != NULL) != (act_prev != NULL)) return -1;
    if (!(G == 1 || G == N)) return -1;
    model_t md;
    md.F = F; md.M = M; md.G = G; md.n = n; md.m = m; md.dep_len = dep_len; md.dep = dep;
    md.U = U; md.A = A; md.B = B; md.D = D; md.round32 = round32; md.lambda = lambda;
    md.bdep_len = bdep_len; md.bdep = bdep;
    md.bdep_off = malloc(sizeof(int) * F);
    md.PB = malloc(sizeof(int64_t) * F);
    md.off = malloc(sizeof(int) * F);
    md.dep_off = malloc(sizeof(int) * (M > 0 ? M : 1));
    md.P = malloc(sizeof(int64_t) * (M > 0 ? M : 1));
    md.moff = malloc(sizeof(int) * (M > 0 ? M : 1));
    md.Mtot = 0;
    for (int i = 0; i < M; ++i) { md.moff[i] = md.Mtot; md.Mtot += m[i]; }
    int S = 0;
    for (int f = 0; f < F; ++f) { md.off[f] = S; S += n[f]; }
    md.S = S;
    int o = 0, bad = 0;
    for (int i = 0; i < M; ++i) {
        md.dep_off[i] = o;
        if (dep_len[i] < 1 || dep_len[i] > BI_REF_MAXK) bad = 1;
        int64_t P = 1;
        for (int j = 0; j < dep_len[i] && !bad; ++j) {
            if (dep[o + j] < 0 || dep[o + j] >= F) { bad = 1; break; }
            P *= n[dep[o + j]];
        }
        md.P[i] = P;
        o += dep_len[i];
    }
    if (bdep_len) {
        int bo = 0;
        for (int f = 0; f < F && !bad; ++f) {
            md.bdep_off[f] = bo;
            if (bdep_len[f] < 1 || bdep_len[f] > BI_REF_MAXK) { bad = 1; break; }
            int64_t P = 1;
            for (int j = 0; j < bdep_len[f]; ++j) {
                if (bdep[bo + j] < 0 || bdep[bo + j] >= F) { bad = 1; break; }
                P *= n[bdep[bo + j]];
            }
            md.PB[f] = P;
            bo += bdep_len[f];
        }
    }
    if (bad) { free(md.off); free(md.dep_off); free(md.P); free(md.moff); free(md.bdep_off); free(md.PB); return -1; }
#ifdef _OPENMP
    if (threads > 0) omp_set_num_threads(threads);
#else
    (void)threads;
#endif
#pragma omp parallel for schedule(dynamic, 1)
    for (int a = 0; a < N; ++a) {
        int g = (G == 1) ? 0 : a;
        const int32_t *ob = obs ? obs + (size_t)a * T * M : NULL;
        const float *so = obs_soft ? obs_soft + (size_t)a * T * md.Mtot : NULL;
        const int32_t *ac = act ? act + (size_t)a * (T - 1) * F : NULL;
        const double *qi = q_init ? q_init + (size_t)a * T * S : NULL;
        double *qo = q_out + (size_t)a * T * S;
        double *lo = logq_out ? logq_out + (size_t)a * T * S : NULL;
        int32_t *ao = argmax_out ? argmax_out + (size_t)a * T * F : NULL;
        if (algo == ALGO_FILTER)
            filter_agent(&md, g, T, K, ob, so, ac, qi, q_prev ? q_prev + (size_t)a * S : NULL,
                         act_prev ? act_prev + (size_t)a * F : NULL, qo, lo, ao);
        else window_agent(&md, algo, g, T, K, ob, so, ac, qi, q_prev ? q_prev + (size_t)a * S : NULL,
                          act_prev ? act_prev + (size_t)a * F : NULL, qo, lo, ao);
    }
    free(md.off); free(md.dep_off); free(md.P); free(md.moff); free(md.bdep_off); free(md.PB);
    return 0;
}

int bi_ref_run(int algo, int F, int M, const int32_t *n, const int32_t *m,
               const int32_t *dep_len, const int32_t *dep, const int32_t *U, int G,
               const float *const *A, const float *const *B, const float *const *D,
               int N, int T, const int32_t *obs, const int32_t *act, int K,
               const double *q_init, double *q_out, double *logq_out,
               int32_t *argmax_out, int threads, int round32)
{
    return run_impl(algo, F, M, n, m, dep_len, dep, U, G, A, B, D, N, T, obs, NULL, act, K, q_init, NULL, NULL,
                    q_out, logq_out, argmax_out, threads, round32, 1.0, NULL, NULL);
}

/*
 * bi_ref_run with every observation given as categorical vectors instead of
 * indices: obs_soft is [N][T][sum_i m_i] float32, the modalities' blocks in
 * order (Section III-B: an observation modality is represented as a categorical
 * probability vector; Section III-C: the log-likelihood is log(A_i) . o^i).
 * A one-hot vector reproduces the index form.
 */
int bi_ref_run_soft(int algo, int F, int M, const int32_t *n, const int32_t *m,
                    const int32_t *dep_len, const int32_t *dep, const int32_t *U, int G,
                    const float *const *A, const float *const *B, const float *const *D,
                    int N, int T, const float *obs_soft, const int32_t *act, int K,
                    double *q_out, double *logq_out, int32_t *argmax_out, int threads)
{
    if (!obs_soft && M > 0) return -1;
    return run_impl(algo, F, M, n, m, dep_len, dep, U, G, A, B, D, N, T, NULL, obs_soft, act, K, NULL, NULL, NULL,
                    q_out, logq_out, argmax_out, threads, 0, 1.0, NULL, NULL);
}

/*
 * Filtering continued from a known belief: q_prev [N][S] is every agent's belief
 * at the step before the window and act_prev [N][F] the action taken there, so
 * the first step's prior is B_u q_prev (the recursion of Section III-B entered
 * mid-stream) instead of D.  Everything else as bi_ref_run with the filtering
 * algorithm.
 */
int bi_ref_filter_from(int F, int M, const int32_t *n, const int32_t *m,
                       const int32_t *dep_len, const int32_t *dep, const int32_t *U, int G,
                       const float *const *A, const float *const *B, const float *const *D,
                       int N, int T, const int32_t *obs, const int32_t *act, int K,
                       const double *q_prev, const int32_t *act_prev,
                       double *q_out, double *logq_out, int32_t *argmax_out, int threads)
{
    if (!q_prev || !act_prev) return -1;
    return run_impl(ALGO_FILTER, F, M, n, m, dep_len, dep, U, G, A, B, D, N, T, obs, NULL, act, K, NULL, q_prev,
                    act_prev, q_out, logq_out, argmax_out, threads, 0, 1.0, NULL, NULL);
}

/*
 * VMP / MMP over a window that continues a stream: as bi_ref_filter_from, the
 * first step's prior is B_u q_prev (at full weight, in the place of D); q_init
 * may be NULL (uniform start).
 */
int bi_ref_window_from(int algo, int F, int M, const int32_t *n, const int32_t *m,
                       const int32_t *dep_len, const int32_t *dep, const int32_t *U, int G,
                       const float *const *A, const float *const *B, const float *const *D,
                       int N, int T, const int32_t *obs, const int32_t *act, int K,
                       const double *q_init, const double *q_prev, const int32_t *act_prev,
                       double *q_out, double *logq_out, int32_t *argmax_out, int threads)
{
    if (!q_prev || !act_prev || (algo != ALGO_VMP && algo != ALGO_MMP)) return -1;
    return run_impl(algo, F, M, n, m, dep_len, dep, U, G, A, B, D, N, T, obs, NULL, act, K, q_init, q_prev,
                    act_prev, q_out, logq_out, argmax_out, threads, 0, 1.0, NULL, NULL);
}

/*
 * Every option at once, plus damping: the update becomes
 *   ln q' = (1 - lambda) ln q + lambda (likelihood message + transition messages) + const,
 * a step of size lambda on the log-beliefs towards the plain update (lambda = 1).
 * Unused options are NULL; obs_soft replaces obs when given.
 */
int bi_ref_run_opts(int algo, int F, int M, const int32_t *n, const int32_t *m,
                    const int32_t *dep_len, const int32_t *dep, const int32_t *U, int G,
                    const float *const *A, const float *const *B, const float *const *D,
                    int N, int T, const int32_t *obs, const float *obs_soft, const int32_t *act, int K,
                    const double *q_init, const double *q_prev, const int32_t *act_prev, double lambda,
                    double *q_out, double *logq_out, int32_t *argmax_out, int threads, int round32)
{
    return run_impl(algo, F, M, n, m, dep_len, dep, U, G, A, B, D, N, T, obs, obs_soft, act, K, q_init, q_prev,
                    act_prev, q_out, logq_out, argmax_out, threads, round32, lambda, NULL, NULL);
}

/*
 * Filtering or VMP on a model with B-dependencies: bdep_len [F] and bdep [sum] list, per factor, the
 * factors whose previous states its transition depends on (B[f] laid out [G][n_f][parents...][U_f]).
 * Other options as bi_ref_run_opts (no observation vectors, no damping).
 */
int bi_ref_run_bdep(int algo, int F, int M, const int32_t *n, const int32_t *m,
                    const int32_t *dep_len, const int32_t *dep, const int32_t *U, int G,
                    const float *const *A, const float *const *B, const float *const *D,
                    const int32_t *bdep_len, const int32_t *bdep,
                    int N, int T, const int32_t *obs, const int32_t *act, int K,
                    const double *q_init, const double *q_prev, const int32_t *act_prev,
                    double *q_out, double *logq_out, int32_t *argmax_out, int threads)
{
    if (!bdep_len || !bdep) return -1;
    return run_impl(algo, F, M, n, m, dep_len, dep, U, G, A, B, D, N, T, obs, NULL, act, K, q_init, q_prev,
                    act_prev, q_out, logq_out, argmax_out, threads, 0, 1.0, bdep_len, bdep);
}

/*
 * The same with the damped update of bi_ref_run_opts (lambda in (0, 1]; 1 = plain): the step on the
 * log-beliefs is taken after the messages are formed, in the code the plain model runs, so nothing
 * about it depends on how many parents a transition has.
 */
int bi_ref_run_bdep_damped(int algo, int F, int M, const int32_t *n, const int32_t *m,
                           const int32_t *dep_len, const int32_t *dep, const int32_t *U, int G,
                           const float *const *A, const float *const *B, const float *const *D,
                           const int32_t *bdep_len, const int32_t *bdep,
                           int N, int T, const int32_t *obs, const int32_t *act, int K,
                           const double *q_init, const double *q_prev, const int32_t *act_prev, double lambda,
                           double *q_out, double *logq_out, int32_t *argmax_out, int threads)
{
    if (!bdep_len || !bdep) return -1;
    return run_impl(algo, F, M, n, m, dep_len, dep, U, G, A, B, D, N, T, obs, NULL, act, K, q_init, q_prev,
                    act_prev, q_out, logq_out, argmax_out, threads, 0, lambda, bdep_len, bdep);
}

int bi_ref_max_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}
