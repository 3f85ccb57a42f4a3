"""Brute-force checkers that pin the oracle on tiny models.

Everything here works from the *definition* of the generative model
(Section III-B: p(o,s|u) = p(s_1) prod p(s_t|s_{t-1},u_{t-1}) prod p(o_t|s_t))
by enumerating every joint hidden-state trajectory.  None of it shares code
with the oracle or the CUDA path, and none of it uses message formulas.
"""
from __future__ import annotations

import itertools

import numpy as np

EPS = 1e-16


def _ln(x):
    return np.log(np.maximum(np.asarray(x, dtype=np.float64), EPS))


class TinyModel:
    """One agent, shared model (G = 1 arrays indexed at g = 0)."""

    def __init__(self, n, m, dep, U, A, B, D, obs, act, bdep=None):
        self.n = [int(v) for v in n]
        self.m = [int(v) for v in m]
        self.dep = [list(d) for d in dep]
        self.U = [int(v) for v in U]
        self.A = [np.asarray(a[0], dtype=np.float64) for a in A]
        self.B = [np.asarray(b[0], dtype=np.float64) for b in B]
        self.D = [np.asarray(d[0], dtype=np.float64) for d in D]
        self.obs = np.asarray(obs)  # [T, M]
        self.act = np.asarray(act)  # [T-1, F]
        self.T = self.obs.shape[0]
        self.F = len(self.n)
        self.off = np.concatenate([[0], np.cumsum(self.n)]).astype(int)
        self.states = list(itertools.product(*[range(k) for k in self.n]))
        # B-dependencies: factor f's transition reads the previous states of bdep[f] (default: its own)
        self.bdep = [list(d) for d in bdep] if bdep is not None else [[f] for f in range(self.F)]

    # log p(o_t | s_t) for a joint state tuple
    def ln_emit(self, t, s):
        v = 0.0
        for i, d in enumerate(self.dep):
            v += _ln(self.A[i][(self.obs[t, i],) + tuple(s[f] for f in d)])
        return float(v)

    def ln_init(self, s):
        return float(sum(_ln(self.D[f][s[f]]) for f in range(self.F)))

    def ln_trans(self, t, s_next, s_prev):
        """ln p(s_t = s_next | s_{t-1} = s_prev, u_{t-1}); t >= 1."""
        return float(sum(_ln(self.B[f][(s_next[f],) + tuple(s_prev[g] for g in self.bdep[f]) + (self.act[t - 1, f],)])
                         for f in range(self.F)))

    def trajectories(self):
        return itertools.product(self.states, repeat=self.T)

    def ln_joint(self, traj):
        v = self.ln_init(traj[0])
        for t in range(self.T):
            v += self.ln_emit(t, traj[t])
            if t > 0:
                v += self.ln_trans(t, traj[t], traj[t - 1])
        return v

    def q_traj(self, q, traj):
        """Mean-field probability of a trajectory; q is [T, S]."""
        p = 1.0
        for t in range(self.T):
            for f in range(self.F):
                p *= q[t, self.off[f] + traj[t][f]]
        return p

    def free_energy(self, q):
        """F[q] = sum_s q(s) (ln q(s) - ln p(o, s | u)) over every trajectory."""
        total = 0.0
        for traj in self.trajectories():
            p = self.q_traj(q, traj)
            if p > 0.0:
                total += p * (np.log(p) - self.ln_joint(traj))
        return total

    def ln_evidence(self):
        return float(np.log(sum(np.exp(self.ln_joint(tr)) for tr in self.trajectories())))

    def coordinate_optimum(self, q, t, f):
        """softmax_s E_{q \\ (t,f)}[ ln p(o, s | u) ] by enumeration (Section III-A)."""
        x = np.zeros(self.n[f])
        for traj in self.trajectories():
            w = 1.0
            for tt in range(self.T):
                for ff in range(self.F):
                    if tt == t and ff == f:
                        continue
                    w *= q[tt, self.off[ff] + traj[tt][ff]]
            if w > 0.0:
                x[traj[t][f]] += w * self.ln_joint(traj)
        x -= x.max()
        e = np.exp(x)
        return e / e.sum()

    def exact_filter_marginals(self):
        """p(s_t^f | o_{1:t}, u) for every t and f by enumeration of the joint chain."""
        out = np.zeros((self.T, self.off[-1]))
        for t in range(self.T):
            sub = TinyModel.__new__(TinyModel)
            sub.__dict__.update(self.__dict__)
            sub.T = t + 1
            post = {}
            for traj in sub.trajectories():
                post[traj[t]] = post.get(traj[t], 0.0) + np.exp(sub.ln_joint(traj))
            z = sum(post.values())
            for s, p in post.items():
                for f in range(self.F):
                    out[t, self.off[f] + s[f]] += p / z
        return out


def hmm_forward(A, B, D, obs, act):
    """Textbook normalised forward recursion for a single-factor HMM.
    A: [m, n]; B: [n, n, U]; D: [n]; returns filtered marginals [T, n]."""
    A = np.asarray(A, np.float64)
    B = np.asarray(B, np.float64)
    alpha = np.asarray(D, np.float64) * A[obs[0]]
    alpha /= alpha.sum()
    out = [alpha]
    for t in range(1, len(obs)):
        pred = B[:, :, act[t - 1]] @ alpha
        alpha = pred * A[obs[t]]
        alpha /= alpha.sum()
        out.append(alpha)
    return np.stack(out)


def reversed_transition(Bu):
    """P(s_t = s | s_{t+1} = r) for a single factor whose s_t has a uniform
    prior, by enumerating the joint table of the pair (s_t, s_{t+1}) and
    conditioning on the second coordinate -- Bayes' rule on the definition
    p(s_{t+1} | s_t) = Bu[s_{t+1}, s_t] (Section III-B), no closed formula.
    Returns R[s, r].  A next state r that no s_t can reach has no posterior;
    there the marginal-message reading takes the prior itself (uniform)."""
    Bu = np.asarray(Bu, np.float64)
    n = Bu.shape[0]
    joint = np.zeros((n, n))            # joint[s, r] = p(s_t = s) p(s_{t+1} = r | s_t = s)
    for s in range(n):
        for r in range(n):
            joint[s, r] = (1.0 / n) * Bu[r, s]
    R = np.zeros((n, n))
    for r in range(n):
        evidence = sum(joint[s, r] for s in range(n))
        for s in range(n):
            R[s, r] = joint[s, r] / evidence if evidence > 0.0 else 1.0 / n
    return R


def mmp_update_by_definition(model, q):
    """One Jacobi marginal-message-passing update of every (t, f) of a TinyModel
    from the beliefs q [T, S], written from the reading's own words rather
    than from message formulas: the new belief is proportional to
        exp(E_{q_t \\ f}[ln p(o_t | s_t)])                       (likelihood, by enumeration)
      * p(s_1)                      at t = 1, else sqrt of the one-step prediction of s_t from q_{t-1}
      * sqrt of the one-step retrodiction of s_t from q_{t+1}     (none at the last step),
    the retrodiction being sum_r P(s_t | s_{t+1} = r) q_{t+1}[r] with the
    reversed kernel of reversed_transition.  Probabilities enter through the
    same floor 1e-16 as everywhere."""
    out = np.zeros_like(q)
    for t in range(model.T):
        for f in range(model.F):
            lo, hi = model.off[f], model.off[f + 1]
            x = np.zeros(model.n[f])
            for s in model.states:          # E over the other factors of ln p(o_t | s_t)
                w = 1.0
                for ff in range(model.F):
                    if ff != f:
                        w *= q[t, model.off[ff] + s[ff]]
                x[s[f]] += w * model.ln_emit(t, s)
            if t == 0:
                x += _ln(model.D[f])
            else:
                pred = np.zeros(model.n[f])
                Bu = model.B[f][:, :, model.act[t - 1, f]]
                for s_next in range(model.n[f]):
                    for s_prev in range(model.n[f]):
                        pred[s_next] += Bu[s_next, s_prev] * q[t - 1, lo + s_prev]
                x += 0.5 * _ln(pred)
            if t + 1 < model.T:
                R = reversed_transition(model.B[f][:, :, model.act[t, f]])
                retro = np.zeros(model.n[f])
                for s in range(model.n[f]):
                    for r in range(model.n[f]):
                        retro[s] += R[s, r] * q[t + 1, lo + r]
                x += 0.5 * _ln(retro)
            x -= x.max()
            e = np.exp(x)
            out[t, lo:hi] = e / e.sum()
    return out
