"""Pins for the CPU oracle: closed forms, brute-force enumeration, invariants.

The oracle is the yardstick for the CUDA path, so it is checked here against
things that are not itself: hand-derived fixtures, the textbook HMM forward
recursion, enumeration of every joint trajectory of tiny models (the model's
definition, Section III-B, and the generic coordinate update, Section III-A),
and metamorphic properties (the paper's claim that padding / regrouping never
changes results).
"""
import itertools
import os

import numpy as np
import pytest

import oracle
from biwl import make_config, make_model, sample_streams
from bruteforce import TinyModel, hmm_forward, mmp_update_by_definition, reversed_transition
from conftest import read_golden


def tiny(seed, n, m, dep, U, T, *, sparsity=0.0, d_alpha=1.0, N=1):
    rng = np.random.default_rng(seed)
    A, B, D = make_model(rng, n, m, dep, U, 1, sparsity=sparsity, d_alpha=d_alpha)
    obs, act = sample_streams(rng, n, m, dep, U, 1, A, B, D, N, T)
    return dict(n=n, m=m, dep=dep, U=U, G=1, A=A, B=B, D=D, obs=obs, act=act)


def run(algo, w, K, **kw):
    return oracle.run(algo, w["n"], w["m"], w["dep"], w["U"], w["G"], w["A"], w["B"], w["D"],
                      w["obs"], w["act"], K, **kw)


def tm(w, a=0):
    return TinyModel(w["n"], w["m"], w["dep"], w["U"], w["A"], w["B"], w["D"], w["obs"][a], w["act"][a])


# ---- P1: single factor filtering is exact Bayes --------------------------------

def test_golden_two_state_hmm(golden_dir):
    g = read_golden(os.path.join(golden_dir, "hmm_two_state.txt"))
    A = [g["A"].reshape(1, 2, 2).astype(np.float32)]
    B = [g["B"].reshape(1, 2, 2, 1).astype(np.float32)]
    D = [g["D"].reshape(1, 2).astype(np.float32)]
    obs = g["obs"].astype(np.int32).reshape(1, 2, 1)
    act = np.zeros((1, 1, 1), np.int32)
    for K in (1, 2, 7):
        q, lq, am = oracle.run("filter", [2], [2], [[0]], [1], 1, A, B, D, obs, act, K)
        np.testing.assert_allclose(q[0, 0], g["q1"], atol=2e-7)
        np.testing.assert_allclose(q[0, 1], g["q2"], atol=2e-7)
        np.testing.assert_allclose(np.exp(lq), q, atol=1e-14)
        assert am.tolist() == [[[0], [1]]]


def test_golden_state_independent_transition(golden_dir):
    g = read_golden(os.path.join(golden_dir, "state_independent_transition.txt"))
    A = [g["A"].reshape(1, 2, 2).astype(np.float32)]
    B = [np.repeat(g["pi"].reshape(1, 2, 1, 1), 2, axis=2).astype(np.float32)]
    D = [g["D"].reshape(1, 2).astype(np.float32)]
    obs = g["obs"].astype(np.int32).reshape(1, 3, 1)
    act = np.zeros((1, 2, 1), np.int32)
    for K in (1, 3):
        qv, _, _ = oracle.run("vmp", [2], [2], [[0]], [1], 1, A, B, D, obs, act, K)
        qm, _, _ = oracle.run("mmp", [2], [2], [[0]], [1], 1, A, B, D, obs, act, K)
        for q, key in ((qv, "q_vmp"), (qm, "q_mmp")):
            np.testing.assert_allclose(q[0, 0], g["q_first"], atol=2e-7)
            np.testing.assert_allclose(q[0, 1], g[key], atol=2e-7)
            np.testing.assert_allclose(q[0, 2], g[key], atol=2e-7)


@pytest.mark.parametrize("seed", [0, 1, 2])
def test_single_factor_filter_is_forward_recursion(seed):
    w = tiny(seed, [5], [4], [[0]], [3], T=8, N=3)
    for K in (1, 4):
        q, lq, am = run("filter", w, K)
        for a in range(3):
            ref = hmm_forward(w["A"][0][0], w["B"][0][0], w["D"][0][0], w["obs"][a, :, 0], w["act"][a, :, 0])
            np.testing.assert_allclose(q[a], ref, atol=1e-12)
            np.testing.assert_allclose(lq[a], np.log(ref), atol=1e-10)
            assert (am[a, :, 0] == ref.argmax(axis=1)).all()


def test_single_factor_filter_matches_enumeration():
    w = tiny(5, [3], [3], [[0]], [2], T=4)
    q, _, _ = run("filter", w, 2)
    np.testing.assert_allclose(q[0], tm(w).exact_filter_marginals(), atol=1e-12)


# ---- P2: every modality on one factor -> factors decouple ------------------------

def test_decoupled_factors_are_exact_and_independent_of_K():
    w = tiny(7, [3, 2], [3, 2, 2], [[0], [1], [0]], [2, 1], T=3)
    exact = tm(w).exact_filter_marginals()
    for K in (1, 5):
        q, _, _ = run("filter", w, K)
        np.testing.assert_allclose(q[0], exact, atol=1e-12)


# ---- P3: the update is the coordinate optimum of Section III-A --------------------

@pytest.mark.parametrize("seed,sparsity", [(11, 0.0), (12, 0.5)])
def test_vmp_update_is_enumerated_coordinate_optimum(seed, sparsity):
    w = tiny(seed, [2, 3], [2, 3], [[0, 1], [1, 0]], [2, 1], T=3, sparsity=sparsity)
    model = tm(w)
    rng = np.random.default_rng(seed)
    S = 5
    q0 = np.concatenate([rng.dirichlet(np.ones(2), size=3), rng.dirichlet(np.ones(3), size=3)], axis=1)
    q1, _, _ = run("vmp", w, 1, q_init=q0[None])
    for t in range(3):
        for f in range(2):
            want = model.coordinate_optimum(q0, t, f)
            got = q1[0, t, model.off[f]:model.off[f + 1]]
            np.testing.assert_allclose(got, want, atol=1e-12)
    assert q1.shape == (1, 3, S)


def test_filter_step_is_enumerated_coordinate_optimum():
    # One filtering step is the T = 1 problem whose initial-state prior is the
    # predictive prior; with T = 1 the prior is D.
    w = tiny(21, [3, 2, 2], [3, 2], [[0, 1, 2], [2, 0]], [1, 1, 1], T=1)
    model = tm(w)
    rng = np.random.default_rng(3)
    q0 = np.concatenate([rng.dirichlet(np.ones(k), size=1) for k in (3, 2, 2)], axis=1)
    q1, _, _ = run("filter", w, 1, q_init=q0[None])
    for f in range(3):
        np.testing.assert_allclose(q1[0, 0, model.off[f]:model.off[f + 1]],
                                   model.coordinate_optimum(q0, 0, f), atol=1e-12)


def test_filter_recursion_uses_predictive_prior():
    # Step 2 of the filter equals a fresh one-step problem whose D is B_u q_1.
    w = tiny(22, [3, 2], [3, 2], [[0, 1], [1]], [2, 2], T=2)
    q, _, _ = run("filter", w, 6)
    D2 = []
    for f, (lo, hi) in enumerate([(0, 3), (3, 5)]):
        Bu = w["B"][f][0][:, :, w["act"][0, 0, f]].astype(np.float64)
        D2.append((Bu @ q[0, 0, lo:hi]).astype(np.float32)[None])
    w2 = dict(w, D=D2, obs=w["obs"][:, 1:], act=w["act"][:, :0])
    q2, _, _ = run("filter", w2, 6)
    np.testing.assert_allclose(q2[0, 0], q[0, 1], atol=5e-7)


def test_free_energy_never_increases_under_coordinate_updates():
    w = tiny(31, [2, 2], [2, 2], [[0, 1], [0]], [2, 2], T=3)
    model = tm(w)
    rng = np.random.default_rng(0)
    q = np.concatenate([rng.dirichlet(np.ones(2), size=3), rng.dirichlet(np.ones(2), size=3)], axis=1)
    f_prev = model.free_energy(q)
    assert f_prev >= -model.ln_evidence() - 1e-12
    for sweep in range(3):
        for t, f in itertools.product(range(3), range(2)):
            upd, _, _ = run("vmp", w, 1, q_init=q[None])
            cand = q.copy()
            cand[t, model.off[f]:model.off[f + 1]] = upd[0, t, model.off[f]:model.off[f + 1]]
            f_new = model.free_energy(cand)
            assert f_new <= f_prev + 1e-12
            # the coordinate minimiser beats random alternatives at that coordinate
            for _ in range(5):
                alt = q.copy()
                alt[t, model.off[f]:model.off[f + 1]] = rng.dirichlet(np.ones(2))
                assert model.free_energy(alt) >= f_new - 1e-12
            q, f_prev = cand, f_new
    assert f_prev >= -model.ln_evidence() - 1e-12


def test_jacobi_schedule_composes():
    # K iterations from a start equal K single iterations chained: every
    # coordinate of iteration k+1 reads iteration k only.
    w = tiny(41, [3, 2], [2, 3], [[0, 1], [1]], [2, 1], T=4, N=2)
    for algo in ("vmp", "mmp"):
        q3, _, _ = run(algo, w, 3)
        q = None
        for _ in range(3):
            q, _, _ = run(algo, w, 1, q_init=q)
        np.testing.assert_allclose(q, q3, atol=1e-14)


# ---- the marginal-message-passing reading: half weights and the reversed transition ----

def test_golden_mmp_future_message(golden_dir):
    # a transition matrix with unequal row sums and a mixed belief at the later step: the backward
    # message varies over states, so the reversed matrix's normalisation axis and the 1/2 weight show
    g = read_golden(os.path.join(golden_dir, "mmp_future_message.txt"))
    A = [g["A"].reshape(1, 2, 2).astype(np.float32)]
    B = [g["B"].reshape(1, 2, 2, 1).astype(np.float32)]
    D = [g["D"].reshape(1, 2).astype(np.float32)]
    obs = g["obs"].astype(np.int32).reshape(1, 2, 1)
    act = np.zeros((1, 1, 1), np.int32)
    start = np.stack([g["q1_start"], g["q2_start"]])[None]
    for algo in ("mmp", "vmp"):
        q, lq, _ = oracle.run(algo, [2], [2], [[0]], [1], 1, A, B, D, obs, act, 1, q_init=start)
        np.testing.assert_allclose(q[0, 0], g["q1_" + algo], atol=2e-7)     # inputs are float32
        np.testing.assert_allclose(q[0, 1], g["q2_" + algo], atol=2e-7)
        np.testing.assert_allclose(np.exp(lq), q, atol=1e-14)


def test_reversed_transition_of_a_permutation_is_its_transpose():
    # a deterministic, invertible transition: knowing s_{t+1} fixes s_t, so the backward message is
    # the later belief carried back through the permutation, whatever the prior on s_t
    perm = [2, 0, 3, 1]                      # s_{t+1} = perm[s_t]
    Bu = np.zeros((4, 4))
    for s, r in enumerate(perm):
        Bu[r, s] = 1.0
    np.testing.assert_array_equal(reversed_transition(Bu), Bu.T)
    A = [np.full((1, 2, 4), 0.5, np.float32)]
    B = [Bu.reshape(1, 4, 4, 1).astype(np.float32)]
    D = [np.full((1, 4), 0.25, np.float32)]
    q2 = np.array([0.1, 0.2, 0.3, 0.4])
    start = np.stack([np.full(4, 0.25), q2])[None]
    q, _, _ = oracle.run("mmp", [4], [2], [[0]], [1], 1, A, B, D, np.zeros((1, 2, 1), np.int32),
                         np.zeros((1, 1, 1), np.int32), 1, q_init=start)
    want = np.sqrt(q2[perm])                 # q_1[s] ∝ sqrt(q_2[perm[s]])
    np.testing.assert_allclose(q[0, 0], want / want.sum(), atol=1e-14)


@pytest.mark.parametrize("seed,n,m,dep,U,sparsity", [
    (91, [3], [3], [[0]], [2], 0.0),
    (92, [2, 3], [2, 3], [[0, 1], [1]], [2, 1], 0.0),
    (93, [3, 2], [3, 2], [[1, 0], [0]], [1, 3], 0.5),
])
def test_mmp_update_matches_the_reading_written_from_the_definition(seed, n, m, dep, U, sparsity):
    w = tiny(seed, n, m, dep, U, T=3, sparsity=sparsity)
    model = tm(w)
    rng = np.random.default_rng(seed)
    q0 = np.concatenate([rng.dirichlet(np.ones(k), size=3) for k in n], axis=1)
    q1, _, _ = run("mmp", w, 1, q_init=q0[None])
    np.testing.assert_allclose(q1[0], mmp_update_by_definition(model, q0), atol=1e-12)
    # and the iteration is that update composed with itself
    q2, _, _ = run("mmp", w, 2, q_init=q0[None])
    np.testing.assert_allclose(q2[0], mmp_update_by_definition(model, mmp_update_by_definition(model, q0)),
                               atol=1e-12)


def test_mmp_unreachable_next_state_gives_a_uniform_backward_column():
    # state 2 can never be entered (its row of B is zero): conditioning on s_{t+1} = 2 is undefined and
    # the reading takes the uniform prior there; a later belief with mass on state 2 exercises it
    Bu = np.array([[0.6, 0.2, 1.0], [0.4, 0.8, 0.0], [0.0, 0.0, 0.0]])
    R = reversed_transition(Bu)
    np.testing.assert_allclose(R[:, 2], 1.0 / 3.0)
    A = [np.array([[[0.5, 0.3, 0.2], [0.5, 0.7, 0.8]]], np.float32)]
    B = [Bu.reshape(1, 3, 3, 1).astype(np.float32)]
    D = [np.array([[0.2, 0.3, 0.5]], np.float32)]
    obs = np.array([[[1], [0]]], np.int32)
    q2 = np.array([0.25, 0.15, 0.6])
    start = np.stack([np.full(3, 1.0 / 3.0), q2])[None]
    q, _, _ = oracle.run("mmp", [3], [2], [[0]], [1], 1, A, B, D, obs, np.zeros((1, 1, 1), np.int32), 1,
                         q_init=start)
    Bf = B[0][0, :, :, 0].astype(np.float64)
    retro = np.array([0.25 * Bf[0, s] / Bf[0].sum() + 0.15 * Bf[1, s] / Bf[1].sum() + 0.6 / 3.0 for s in range(3)])
    want = D[0][0].astype(np.float64) * A[0][0, 1].astype(np.float64) * np.sqrt(retro)
    np.testing.assert_allclose(q[0, 0], want / want.sum(), atol=1e-14)


# ---- P6: Gauss-Seidel sweeps reach a fixed point, free energy never rising ---------

def test_gauss_seidel_sweeps_reach_a_fixed_point():
    w = tiny(32, [2, 3], [2, 3], [[0, 1], [1]], [2, 2], T=2)
    model = tm(w)
    rng = np.random.default_rng(1)
    q = np.concatenate([rng.dirichlet(np.ones(2), size=2), rng.dirichlet(np.ones(3), size=2)], axis=1)
    coords = list(itertools.product(range(2), range(2)))

    def sweep(q):
        for t, f in coords:           # one coordinate at a time: the Jacobi result, one block taken
            upd, _, _ = run("vmp", w, 1, q_init=q[None])
            q = q.copy()
            q[t, model.off[f]:model.off[f + 1]] = upd[0, t, model.off[f]:model.off[f + 1]]
        return q

    f_prev = model.free_energy(q)
    for i in range(500):
        q = sweep(q)
        if i < 40 or i % 20 == 0:     # the enumeration is the slow part; checked densely early on
            f_new = model.free_energy(q)
            assert f_new <= f_prev + 1e-12
            f_prev = f_new
    q_next = sweep(q)
    assert np.abs(q_next - q).max() < 1e-12
    assert model.free_energy(q_next) <= f_prev + 1e-12
    assert f_prev >= -model.ln_evidence() - 1e-12
    # at the fixed point every coordinate is its own enumerated optimum
    for t, f in coords:
        np.testing.assert_allclose(q[t, model.off[f]:model.off[f + 1]], model.coordinate_optimum(q, t, f),
                                   atol=1e-10)


# ---- non-trivial B-dependencies (transitions that read other factors' previous states) ----

def tiny_bdep(seed, n, m, dep, U, bdep, T, *, N=1, sparsity=0.0, b_sparsity=0.0):
    rng = np.random.default_rng(seed)
    A, B, D = make_model(rng, n, m, dep, U, 1, sparsity=sparsity, d_alpha=1.0, bdep=bdep, b_sparsity=b_sparsity)
    obs, act = sample_streams(rng, n, m, dep, U, 1, A, B, D, N, T, bdep=bdep)
    return dict(n=n, m=m, dep=dep, U=U, G=1, A=A, B=B, D=D, obs=obs, act=act, bdep=bdep)


def run_b(algo, w, K, **kw):
    return oracle.run(algo, w["n"], w["m"], w["dep"], w["U"], w["G"], w["A"], w["B"], w["D"], w["obs"], w["act"], K,
                      bdep=w["bdep"], **kw)


@pytest.mark.parametrize("seed,bdep,b_sparsity", [(101, [[0, 1], [1]], 0.0), (102, [[1], [0, 1]], 0.0),
                                                  (103, [[1, 0], [0]], 0.4)])
def test_vmp_with_b_dependencies_is_the_enumerated_coordinate_optimum(seed, bdep, b_sparsity):
    # the generic update of Section III-A on a model whose transitions read other factors' states:
    # every (t, f) block of one Jacobi iteration equals the optimum found by enumerating trajectories
    w = tiny_bdep(seed, [2, 3], [2, 3], [[0, 1], [1]], [2, 2], bdep, T=3, b_sparsity=b_sparsity)
    model = TinyModel(w["n"], w["m"], w["dep"], w["U"], w["A"], w["B"], w["D"], w["obs"][0], w["act"][0], bdep=bdep)
    rng = np.random.default_rng(seed)
    q0 = np.concatenate([rng.dirichlet(np.ones(2), size=3), rng.dirichlet(np.ones(3), size=3)], axis=1)
    q1, lq1, _ = run_b("vmp", w, 1, q_init=q0[None])
    for t in range(3):
        for f in range(2):
            np.testing.assert_allclose(q1[0, t, model.off[f]:model.off[f + 1]], model.coordinate_optimum(q0, t, f),
                                       atol=1e-12)
    np.testing.assert_allclose(np.exp(lq1), q1, atol=1e-12)


def test_filter_prior_with_b_dependencies_is_the_product_of_marginals_prediction():
    # step 2 of the filter equals a fresh one-step problem whose D is sum_parents B prod q_1, taken with
    # plain loops over the joint parent states
    bdep = [[0, 1], [1, 0]]
    w = tiny_bdep(111, [3, 2], [3, 2], [[0, 1], [1]], [2, 2], bdep, T=2)
    q, _, _ = run_b("filter", w, 5)
    D2 = []
    for f, (lo, hi) in enumerate([(0, 3), (3, 5)]):
        u = int(w["act"][0, 0, f])
        pred = np.zeros(hi - lo)
        for sn in range(hi - lo):
            for par in itertools.product(*[range(w["n"][g]) for g in bdep[f]]):
                wgt = 1.0
                for g, sg in zip(bdep[f], par):
                    wgt *= q[0, 0, [0, 3][g] + sg]
                pred[sn] += float(w["B"][f][(0, sn) + par + (u,)]) * wgt
        D2.append(pred.astype(np.float32)[None])
    w2 = dict(w, D=D2, obs=w["obs"][:, 1:], act=w["act"][:, :0])
    q2, _, _ = run_b("filter", w2, 5)
    np.testing.assert_allclose(q2[0, 0], q[0, 1], atol=5e-7)   # D2 was rounded to float32


def test_b_dependencies_on_the_factor_itself_are_the_plain_model():
    w = tiny(112, [3, 4, 2], [3, 2], [[0, 1], [1, 2]], [2, 3, 1], T=4, N=2, sparsity=0.5)
    for algo in ("filter", "vmp"):
        a = run(algo, w, 4)
        b = oracle.run(algo, w["n"], w["m"], w["dep"], w["U"], 1, w["A"], w["B"], w["D"], w["obs"], w["act"], 4,
                       bdep=[[0], [1], [2]])
        for x, y in zip(a, b):
            np.testing.assert_allclose(y, x, atol=1e-13)
    # ... and so does the damped update (the step on the log-beliefs does not see the parents)
    for algo in ("filter", "vmp"):
        a = oracle.run(algo, w["n"], w["m"], w["dep"], w["U"], 1, w["A"], w["B"], w["D"], w["obs"], w["act"], 5,
                       damping=0.6)
        b = oracle.run(algo, w["n"], w["m"], w["dep"], w["U"], 1, w["A"], w["B"], w["D"], w["obs"], w["act"], 5,
                       damping=0.6, bdep=[[0], [1], [2]])
        plain = run(algo, w, 5)
        assert np.abs(a[0] - plain[0]).max() > 1e-4          # the damping does something here
        for x, y in zip(a, b):
            np.testing.assert_allclose(y, x, atol=1e-13)
    # a transition declared on a superset of its true parents (B replicated along the new axis): same beliefs
    B = list(w["B"])
    B[1] = np.ascontiguousarray(np.repeat(w["B"][1][:, :, :, None, :], 2, axis=3))   # [1, 4, 4, n_2 = 2, 3]
    for algo in ("filter", "vmp"):
        a = run(algo, w, 4)[0]
        b = oracle.run(algo, w["n"], w["m"], w["dep"], w["U"], 1, w["A"], B, w["D"], w["obs"], w["act"], 4,
                       bdep=[[0], [1, 2], [2]])[0]
        np.testing.assert_allclose(b, a, atol=1e-12)


def test_deterministic_parents_give_the_exact_transition_column():
    # when the previous beliefs are point masses the prior is the transition's own column, whatever the
    # number of parents; and MMP is refused on such models
    bdep = [[0, 1], [1]]
    w = tiny_bdep(113, [3, 2], [3, 2], [[0], [1]], [2, 1], bdep, T=1, N=1)
    q_prev = np.array([[0.0, 1.0, 0.0, 1.0, 0.0]])
    act_prev = np.array([[1, 0]], np.int32)
    q, _, _ = run_b("filter", w, 1, q_prev=q_prev, act_prev=act_prev)
    A0 = w["A"][0][0].astype(np.float64)
    col = w["B"][0][0, :, 1, 0, 1].astype(np.float64)          # parents (s_0, s_1) = (1, 0), action 1
    want = A0[w["obs"][0, 0, 0]] * col
    np.testing.assert_allclose(q[0, 0, :3], want / want.sum(), atol=1e-12)
    with pytest.raises(ValueError):
        run_b("mmp", dict(w, obs=np.repeat(w["obs"], 2, axis=1), act=np.zeros((1, 1, 2), np.int32)), 2)


def test_free_energy_with_b_dependencies_never_increases():
    bdep = [[0, 1], [0]]
    w = tiny_bdep(114, [2, 2], [2, 2], [[0, 1], [0]], [2, 1], bdep, T=3)
    model = TinyModel(w["n"], w["m"], w["dep"], w["U"], w["A"], w["B"], w["D"], w["obs"][0], w["act"][0], bdep=bdep)
    rng = np.random.default_rng(0)
    q = np.concatenate([rng.dirichlet(np.ones(2), size=3), rng.dirichlet(np.ones(2), size=3)], axis=1)
    f_prev = model.free_energy(q)
    for sweep in range(2):
        for t, f in itertools.product(range(3), range(2)):
            upd, _, _ = run_b("vmp", w, 1, q_init=q[None])
            q = q.copy()
            q[t, model.off[f]:model.off[f + 1]] = upd[0, t, model.off[f]:model.off[f + 1]]
            f_new = model.free_energy(q)
            assert f_new <= f_prev + 1e-12
            f_prev = f_new
    assert f_prev >= -model.ln_evidence() - 1e-12


# ---- P4: window edge conventions ------------------------------------------------

def test_single_step_window_equals_filter_step():
    w = tiny(51, [4, 3], [3, 4], [[0, 1], [1, 0]], [2, 2], T=1, N=4)
    qf, lf, af = run("filter", w, 5)
    for algo in ("vmp", "mmp"):
        q, lq, am = run(algo, w, 5)
        np.testing.assert_allclose(q, qf, atol=1e-12)
        np.testing.assert_allclose(lq, lf, atol=1e-12)
        assert (am == af).all()


# ---- P8: normalisation ------------------------------------------------------------

@pytest.mark.parametrize("algo", ["filter", "vmp", "mmp"])
def test_beliefs_are_distributions(algo):
    w = make_config(1)
    q, lq, am = oracle.run_workload(w, algo)
    assert (q >= 0).all()
    off = np.concatenate([[0], np.cumsum(w.n)])
    for f in range(w.F):
        blk = q[..., off[f]:off[f + 1]]
        np.testing.assert_allclose(blk.sum(-1), 1.0, atol=1e-12)
        assert (blk.argmax(-1) == am[..., f]).all()
    np.testing.assert_allclose(np.exp(lq), q, atol=1e-12)


# ---- metamorphic properties ---------------------------------------------------------

def _base(seed=61, T=4, N=3):
    return tiny(seed, [3, 4, 2], [3, 2, 4], [[0, 1], [1, 2], [2, 0, 1]], [2, 3, 1], T=T, N=N, sparsity=0.5)


@pytest.mark.parametrize("algo", ["filter", "vmp", "mmp"])
def test_modality_permutation(algo):
    w = _base()
    q, _, _ = run(algo, w, 4)
    perm = [2, 0, 1]
    w2 = dict(w, m=[w["m"][i] for i in perm], dep=[w["dep"][i] for i in perm],
              A=[w["A"][i] for i in perm], obs=w["obs"][:, :, perm])
    q2, _, _ = run(algo, w2, 4)
    np.testing.assert_allclose(q2, q, atol=1e-12)


@pytest.mark.parametrize("algo", ["filter", "vmp", "mmp"])
def test_state_relabelling(algo):
    w = _base()
    q, _, _ = run(algo, w, 4)
    p = np.array([2, 0, 3, 1])  # new label j holds old state p[j] of factor 1
    A = [np.ascontiguousarray(np.take(w["A"][0], p, axis=3)),
         np.ascontiguousarray(np.take(w["A"][1], p, axis=2)),
         np.ascontiguousarray(np.take(w["A"][2], p, axis=4))]
    B = list(w["B"])
    B[1] = np.ascontiguousarray(w["B"][1][:, p][:, :, p])
    D = list(w["D"])
    D[1] = np.ascontiguousarray(w["D"][1][:, p])
    q2, _, _ = run(algo, dict(w, A=A, B=B, D=D), 4)
    want = q.copy()
    want[..., 3:7] = q[..., 3:7][..., p]
    np.testing.assert_allclose(q2, want, atol=1e-12)


@pytest.mark.parametrize("algo", ["filter", "vmp", "mmp"])
def test_uninformative_modality_and_dependency_superset(algo):
    w = _base()
    q, _, _ = run(algo, w, 4)
    N, T = w["obs"].shape[:2]
    # a modality whose A does not depend on the outcome
    const = np.full((1, 3, 4), 1.0 / 3.0, np.float32)
    w2 = dict(w, m=w["m"] + [3], dep=w["dep"] + [[1]], A=w["A"] + [const],
              obs=np.concatenate([w["obs"], np.ones((N, T, 1), np.int32)], axis=2))
    q2, _, _ = run(algo, w2, 4)
    np.testing.assert_allclose(q2, q, atol=1e-12)
    # modality 1 (deps [1,2]) declared on the superset [1,2,0], A replicated along the new axis
    rep = np.ascontiguousarray(np.repeat(w["A"][1][..., None], 3, axis=-1))
    dep = [w["dep"][0], [1, 2, 0], w["dep"][2]]
    q3, _, _ = run(algo, dict(w, dep=dep, A=[w["A"][0], rep, w["A"][2]]), 4)
    np.testing.assert_allclose(q3, q, atol=1e-12)


@pytest.mark.parametrize("algo", ["filter", "vmp", "mmp"])
def test_unobserved_and_singleton_factors(algo):
    w = _base()
    q, _, _ = run(algo, w, 4)
    N, T = w["obs"].shape[:2]
    rng = np.random.default_rng(9)
    # add a factor with one state and a factor no modality depends on
    Bx = rng.dirichlet(np.ones(3), size=(3, 2)).transpose(2, 0, 1)[None].astype(np.float32)  # [1,3,3,2]
    Dx = rng.dirichlet(np.ones(3))[None].astype(np.float32)
    act_x = rng.integers(0, 2, size=(N, T - 1, 1)).astype(np.int32)
    w2 = dict(w, n=w["n"] + [1, 3], U=w["U"] + [1, 2],
              B=w["B"] + [np.ones((1, 1, 1, 1), np.float32), Bx],
              D=w["D"] + [np.ones((1, 1), np.float32), Dx],
              act=np.concatenate([w["act"], np.zeros((N, T - 1, 1), np.int32), act_x], axis=2))
    q2, _, _ = run(algo, w2, 4)
    np.testing.assert_allclose(q2[..., :9], q, atol=1e-12)
    np.testing.assert_allclose(q2[..., 9], 1.0, atol=1e-15)
    if algo == "filter":
        # the unobserved factor just follows its transition recursion
        for a in range(N):
            p = Dx[0].astype(np.float64)
            for t in range(T):
                if t > 0:
                    p = Bx[0][:, :, act_x[a, t - 1, 0]].astype(np.float64) @ p
                np.testing.assert_allclose(q2[a, t, 10:], p / p.sum(), atol=1e-12)


@pytest.mark.parametrize("algo", ["filter", "vmp", "mmp"])
def test_shared_vs_replicated_model_and_batch_independence(algo):
    w = _base(N=4)
    q, _, am = run(algo, w, 3)
    rep = dict(w, G=4, A=[np.repeat(a, 4, axis=0) for a in w["A"]],
               B=[np.repeat(b, 4, axis=0) for b in w["B"]], D=[np.repeat(d, 4, axis=0) for d in w["D"]])
    q2, _, am2 = run(algo, rep, 3)
    assert np.array_equal(q2, q) and np.array_equal(am2, am)
    sub = dict(w, obs=w["obs"][[2]], act=w["act"][[2]])
    q3, _, _ = run(algo, sub, 3)
    assert np.array_equal(q3[0], q[2])


def test_threads_do_not_change_results():
    w = make_config(1)
    a = oracle.run_workload(w, threads=1)
    b = oracle.run_workload(w, threads=4)
    assert all(np.array_equal(x, y) for x, y in zip(a, b))


def test_zero_probabilities_use_the_clamped_log():
    # A with exact zeros: an observed outcome that is impossible under a state
    # drives that state's belief to (numerically) zero but stays finite.
    A = [np.array([[[1.0, 0.5], [0.0, 0.5]]], np.float32)]
    B = [np.eye(2, dtype=np.float32).reshape(1, 2, 2, 1)]
    D = [np.array([[0.5, 0.5]], np.float32)]
    q, lq, _ = oracle.run("filter", [2], [2], [[0]], [1], 1, A, B, D,
                          np.array([[[1]]], np.int32), None, 2)
    want = np.array([1e-16, 0.5]) / (1e-16 + 0.5)
    np.testing.assert_allclose(q[0, 0], want, rtol=1e-12)
    assert np.isfinite(lq).all()


# ---- filtering continued from a known belief (the recursion entered mid-stream) ----

def test_filter_continuation_equals_the_uninterrupted_run():
    w = tiny(61, [4, 3, 2], [3, 4], [[0, 1], [1, 2, 0]], [2, 3, 1], T=9, N=3, sparsity=0.5)
    q, lq, am = run("filter", w, 5)
    for cut in (1, 4, 8):
        head = dict(w, obs=w["obs"][:, :cut], act=w["act"][:, :cut - 1])
        tail = dict(w, obs=w["obs"][:, cut:], act=w["act"][:, cut:])
        qh, _, _ = run("filter", head, 5)
        np.testing.assert_array_equal(qh, q[:, :cut])
        qt, lqt, amt = run("filter", tail, 5, q_prev=qh[:, -1], act_prev=w["act"][:, cut - 1])
        np.testing.assert_array_equal(qt, q[:, cut:])
        np.testing.assert_array_equal(lqt, lq[:, cut:])
        np.testing.assert_array_equal(amt, am[:, cut:])


def test_single_factor_continuation_is_one_bayes_step():
    # softmax(ln A[o] + ln(B_u q_prev)), written out directly
    w = tiny(62, [5], [4], [[0]], [3], T=1, N=4)
    rng = np.random.default_rng(7)
    q_prev = rng.dirichlet(np.ones(5), size=4)
    act_prev = rng.integers(0, 3, size=(4, 1)).astype(np.int32)
    q, lq, _ = run("filter", w, 3, q_prev=q_prev, act_prev=act_prev)
    A, B = w["A"][0][0].astype(np.float64), w["B"][0][0].astype(np.float64)
    for a in range(4):
        post = A[w["obs"][a, 0, 0]] * (B[:, :, act_prev[a, 0]] @ q_prev[a])
        post /= post.sum()
        np.testing.assert_allclose(q[a, 0], post, atol=1e-14)
        np.testing.assert_allclose(lq[a, 0], np.log(post), atol=1e-12)


def test_continuation_arguments_are_checked():
    w = tiny(63, [3], [2], [[0]], [2], T=2)
    with pytest.raises((ValueError, AssertionError)):
        run("vmp", w, 2, q_prev=np.full((1, 3), 1 / 3))          # act_prev missing


@pytest.mark.parametrize("algo", ["vmp", "mmp"])
def test_window_continuation_replaces_the_prior_by_the_predictive_one(algo):
    # a window continued from q_prev equals the same window on a model whose D is B_u q_prev
    w = tiny(64, [4, 3], [3, 4], [[0, 1], [1]], [2, 3], T=4, sparsity=0.5)
    rng = np.random.default_rng(11)
    q_prev = np.concatenate([rng.dirichlet(np.ones(4)), rng.dirichlet(np.ones(3))])[None]
    act_prev = np.array([[1, 2]], np.int32)
    q, lq, am = run(algo, w, 5, q_prev=q_prev, act_prev=act_prev)
    D2 = []
    for f, (lo, hi) in enumerate([(0, 4), (4, 7)]):
        Bu = w["B"][f][0][:, :, act_prev[0, f]].astype(np.float64)
        D2.append((Bu @ q_prev[0, lo:hi]).astype(np.float32)[None])
    q2, _, _ = run(algo, dict(w, D=D2), 5)
    np.testing.assert_allclose(q, q2, atol=2e-6)      # D2 was rounded to float32


def test_single_step_windows_continue_like_the_filter():
    # T = 1: VMP = MMP = one filtering step, also when the step continues a stream
    w = tiny(65, [3, 4], [3, 2], [[0, 1], [1]], [2, 2], T=1, N=2)
    rng = np.random.default_rng(12)
    q_prev = np.concatenate([rng.dirichlet(np.ones(3), size=2), rng.dirichlet(np.ones(4), size=2)], axis=1)
    act_prev = rng.integers(0, 2, size=(2, 2)).astype(np.int32)
    qf, _, _ = run("filter", w, 4, q_prev=q_prev, act_prev=act_prev)
    for algo in ("vmp", "mmp"):
        qw, _, _ = run(algo, w, 4, q_prev=q_prev, act_prev=act_prev)
        np.testing.assert_allclose(qw, qf, atol=1e-12)


# ---- observations as categorical vectors: log-likelihood = log(A_i) . o^i (Section III-C) ----

def one_hot(w):
    N, T, M = w["obs"].shape
    out = np.zeros((N, T, int(np.sum(w["m"]))), np.float32)
    off = np.concatenate([[0], np.cumsum(w["m"])]).astype(int)
    for i in range(M):
        np.put_along_axis(out[:, :, off[i]:off[i + 1]], w["obs"][:, :, i:i + 1], 1.0, axis=2)
    return out


def run_soft(algo, w, K, soft):
    return oracle.run(algo, w["n"], w["m"], w["dep"], w["U"], w["G"], w["A"], w["B"], w["D"], None, w["act"], K,
                      obs_soft=soft)


@pytest.mark.parametrize("algo", ["filter", "vmp", "mmp"])
def test_one_hot_vectors_reproduce_index_observations(algo):
    w = tiny(71, [4, 3, 2], [3, 4, 2], [[0, 1], [1, 2, 0], [2]], [2, 3, 1], T=5, N=3, sparsity=0.5)
    q, lq, am = run(algo, w, 4)
    qs, lqs, ams = run_soft(algo, w, 4, one_hot(w))
    np.testing.assert_array_equal(qs, q)
    np.testing.assert_array_equal(lqs, lq)
    np.testing.assert_array_equal(ams, am)


def test_single_factor_soft_observation_is_a_geometric_mixture():
    # q proportional to D * prod_o A[o, :]^{w[o]}, written out directly
    w = tiny(72, [5], [4], [[0]], [2], T=1, N=3)
    rng = np.random.default_rng(3)
    soft = rng.dirichlet(np.ones(4), size=(3, 1)).astype(np.float32)
    q, lq, _ = run_soft("filter", w, 2, soft)
    A, D = w["A"][0][0].astype(np.float64), w["D"][0][0].astype(np.float64)
    for a in range(3):
        post = D * np.prod(A ** soft[a, 0].astype(np.float64)[:, None], axis=0)
        post /= post.sum()
        np.testing.assert_allclose(q[a, 0], post, rtol=1e-12)


def test_soft_log_likelihood_is_linear_in_the_observation_vector():
    # one sweep from the uniform start: the logits are prior + likelihood message, and the message is
    # linear in every modality's vector, so log-beliefs of a mixture are the mixture of log-beliefs up to
    # one constant per factor
    w = tiny(73, [3, 4], [3, 2], [[0, 1], [1]], [2, 2], T=1, N=1)
    o1 = one_hot(w)
    w2 = dict(w, obs=(w["obs"] + 1) % np.asarray(w["m"], np.int32))
    o2 = one_hot(w2)
    alpha = 0.3
    mix = (alpha * o1 + (1 - alpha) * o2).astype(np.float32)
    _, l1, _ = run_soft("filter", w, 1, o1)
    _, l2, _ = run_soft("filter", w, 1, o2)
    _, lm, _ = run_soft("filter", w, 1, mix)
    # float32 weights: use the values the oracle actually saw
    a32 = float(mix[0, 0, w["obs"][0, 0, 0]])
    for lo, hi in ((0, 3), (3, 7)):
        d = lm[0, 0, lo:hi] - (a32 * l1[0, 0, lo:hi] + (1 - a32) * l2[0, 0, lo:hi])
        np.testing.assert_allclose(d, d[0], atol=1e-6)


def test_soft_observations_weight_each_modality_separately():
    # a uniform vector on one modality carries no information about a factor only that modality sees ...
    w = tiny(74, [3, 2], [4, 3], [[0], [1]], [1, 1], T=1)
    soft = one_hot(w)
    soft[0, 0, :4] = 0.25
    q, _, _ = run_soft("filter", w, 3, soft)
    A0, D0 = w["A"][0][0].astype(np.float64), w["D"][0][0].astype(np.float64)
    post = D0 * np.exp(0.25 * np.log(np.maximum(A0, 1e-16)).sum(axis=0))
    np.testing.assert_allclose(q[0, 0, :3], post / post.sum(), rtol=1e-10)
    # ... and leaves the other factor's exact posterior untouched
    qh, _, _ = run("filter", w, 3)
    np.testing.assert_allclose(q[0, 0, 3:], qh[0, 0, 3:], rtol=1e-12)


# ---- damped update on log-beliefs ----

def test_damping_one_is_the_plain_update_and_small_steps_interpolate():
    w = tiny(81, [3, 4], [3, 2], [[0, 1], [1]], [2, 2], T=3)
    for algo in ("filter", "vmp", "mmp"):
        q, lq, _ = run(algo, w, 4)
        q1, lq1, _ = run(algo, w, 4, damping=1.0 - 1e-12)
        np.testing.assert_allclose(q1, q, atol=1e-9)


def test_single_factor_damped_filter_has_a_closed_form():
    # one factor: the plain update is the exact posterior p* whatever q is, so after k damped steps from
    # the uniform start  ln q_k = (1 - (1 - lambda)^k) ln p* + const
    w = tiny(82, [5], [4], [[0]], [2], T=1, N=2)
    lam = 0.35
    p_star, _, _ = run("filter", w, 1)
    for K in (1, 2, 5):
        q, _, _ = run("filter", w, K, damping=lam)
        for a in range(2):
            want = p_star[a, 0] ** (1.0 - (1.0 - lam) ** K)
            np.testing.assert_allclose(q[a, 0], want / want.sum(), rtol=1e-12)


def test_damping_keeps_the_fixed_points():
    # a fixed point of the plain map is a fixed point of the damped one: start both at a converged
    # belief (a decoupled model converges in one sweep) and nothing moves
    w = tiny(83, [3, 2], [3, 2, 2], [[0], [1], [0]], [2, 1], T=1)
    q, _, _ = run("filter", w, 3)
    q_init = q.copy()
    qd, _, _ = run("filter", w, 4, q_init=q_init, damping=0.4)
    np.testing.assert_allclose(qd, q, atol=1e-12)


def test_damped_windows_start_from_log_q_init():
    # the first damped step mixes the plain update with ln q_init
    w = tiny(84, [3, 4], [3, 2], [[0, 1], [1]], [2, 2], T=2)
    rng = np.random.default_rng(5)
    q_init = np.concatenate([rng.dirichlet(np.ones(3), size=(1, 2)), rng.dirichlet(np.ones(4), size=(1, 2))], axis=2)
    lam = 0.6
    for algo in ("vmp", "mmp"):
        _, lplain, _ = run(algo, w, 1, q_init=q_init)            # log of the plain update from q_init
        qd, _, _ = run(algo, w, 1, q_init=q_init, damping=lam)
        for lo, hi in ((0, 3), (3, 7)):
            mix = (1 - lam) * np.log(q_init[0, :, lo:hi]) + lam * lplain[0, :, lo:hi]
            want = np.exp(mix - mix.max(axis=1, keepdims=True))
            want /= want.sum(axis=1, keepdims=True)
            np.testing.assert_allclose(qd[0, :, lo:hi], want, rtol=1e-11)
