"""Pins of the fitter oracle (oracle/saf_fit_oracle.py) against things it does not compute itself:
brute-force Python loops, finite differences, torch autograd + torch.optim.Adam, closed forms, invariances of
Eq. "compact-prior", recovery of a planted pattern, and the FFT convolution.  CPU only."""
import math

import numpy as np
import pytest
import torch

import saf_inputs as si
from oracle import saf_fit_oracle as fo


def _brute_pattern(alpha, rho):
    """P^ of Eq. "compact-prior" by Python loops."""
    T = len(alpha)
    P = [[0.0] * T for _ in range(T)]
    logZ = [0.0] * T
    for i in range(T):
        z = 0.0
        for k in range(i + 1):
            z += math.exp(alpha[k] + rho[i - k])
        logZ[i] = math.log(z)
        for j in range(i + 1):
            P[i][j] = math.exp(alpha[j] + rho[i - j]) / z
    return np.array(P), np.array(logZ)


def _random_target(T, seed):
    return fo.target_from_mean_attention(si.mean_attention_maps(1, T, seed)[0])


# F1 ------------------------------------------------------------------------------------------------ target
def test_target_floor_and_rows_brute_force():
    T = 9
    rng = np.random.default_rng(0)
    A = rng.uniform(0, 1, (T, T))
    A[5, 2] = 0.0          # below the floor
    A[7, 0] = 1e-12
    A[2, 6] = 123.0        # above the diagonal: ignored
    P = fo.target_from_mean_attention(A)
    for i in range(T):
        row = [max(A[i, j], 1e-9) for j in range(i + 1)]
        s = sum(row)
        for j in range(T):
            want = row[j] / s if j <= i else 0.0
            assert abs(P[i, j] - want) < 1e-15
    assert abs(P[5, 2] - 1e-9 / sum(max(A[5, j], 1e-9) for j in range(6))) < 1e-20


# F2 ------------------------------------------------------------------------------------------------ marginals
def test_marginals_brute_force():
    T = 11
    P = _random_target(T, 3)
    ea, er, plogp = fo.marginals(P)
    for j in range(T):
        assert abs(ea[j] - sum(P[i, j] for i in range(j, T))) < 1e-14
    for d in range(T):
        assert abs(er[d] - sum(P[j + d, j] for j in range(T - d))) < 1e-14
    want = sum(P[i, j] * math.log(P[i, j]) for i in range(T) for j in range(i + 1))
    assert abs(plogp - want) < 1e-12
    # each marginal distributes the T units of row mass
    assert abs(ea.sum() - T) < 1e-12 and abs(er.sum() - T) < 1e-12


# F3 ------------------------------------------------------------------------------------------------ objective
def test_objective_brute_force_and_cross_entropy_identity():
    T = 10
    rng = np.random.default_rng(5)
    alpha, rho = rng.standard_normal(T), rng.standard_normal(T)
    P = _random_target(T, 7)
    ea, er, plogp = fo.marginals(P)
    Phat, logZ = _brute_pattern(alpha, rho)
    want = (sum(logZ) - sum(ea[j] * alpha[j] for j in range(T)) - sum(er[d] * rho[d] for d in range(T))) / T
    assert abs(fo.fit_objective(alpha, rho, ea, er) - want) < 1e-13
    # Eq. "fit-objective" is the row-averaged cross-entropy -(1/T) sum P log P^
    ce = -sum(P[i, j] * math.log(Phat[i][j]) for i in range(T) for j in range(i + 1)) / T
    assert abs(want - ce) < 1e-12


def test_objective_closed_form_T2():
    # T = 2: row 0 is the single entry 1; row 1 is a two-way softmax of (alpha0+rho1, alpha1+rho0)
    a0, a1, r0, r1 = 0.3, -0.7, 0.2, 1.1
    p10 = 0.25
    P = np.array([[1.0, 0.0], [p10, 1 - p10]])
    ea, er, _ = fo.marginals(P)
    assert np.allclose(ea, [1 + p10, 1 - p10]) and np.allclose(er, [2 - p10, p10])
    z0 = a0 + r0
    z1 = math.log(math.exp(a0 + r1) + math.exp(a1 + r0))
    want = (z0 + z1 - (1 + p10) * a0 - (1 - p10) * a1 - (2 - p10) * r0 - p10 * r1) / 2
    got = fo.fit_objective(np.array([a0, a1]), np.array([r0, r1]), ea, er)
    assert abs(got - want) < 1e-14
    # its minimum over the logit x = (a0+r1)-(a1+r0) is where sigmoid(x) = p10, with value H(p10)/2
    x = math.log(p10 / (1 - p10))
    opt = fo.fit_objective(np.array([x, 0.0]), np.array([0.0, 0.0]), ea, er)
    H = -(p10 * math.log(p10) + (1 - p10) * math.log(1 - p10))
    assert abs(opt - H / 2) < 1e-14


# F4 ------------------------------------------------------------------------------------------------ gradient
def test_gradient_finite_differences():
    T = 12
    rng = np.random.default_rng(11)
    alpha, rho = rng.standard_normal(T), 0.5 * rng.standard_normal(T)
    ea, er, _ = fo.marginals(_random_target(T, 2))
    ga, gr = fo.fit_gradient(alpha, rho, ea, er)
    h = 1e-6
    for k in range(T):
        e = np.zeros(T)
        e[k] = h
        fa = (fo.fit_objective(alpha + e, rho, ea, er) - fo.fit_objective(alpha - e, rho, ea, er)) / (2 * h)
        fr = (fo.fit_objective(alpha, rho + e, ea, er) - fo.fit_objective(alpha, rho - e, ea, er)) / (2 * h)
        assert abs(ga[k] - fa) < 1e-8 and abs(gr[k] - fr) < 1e-8


def test_gradient_is_fitted_minus_target_marginals_brute_force():
    T = 8
    rng = np.random.default_rng(4)
    alpha, rho = rng.standard_normal(T), rng.standard_normal(T)
    ea, er, _ = fo.marginals(_random_target(T, 9))
    Phat, _ = _brute_pattern(alpha, rho)
    ga, gr = fo.fit_gradient(alpha, rho, ea, er)
    for j in range(T):
        assert abs(ga[j] - (sum(Phat[i][j] for i in range(j, T)) - ea[j]) / T) < 1e-14
    for d in range(T):
        assert abs(gr[d] - (sum(Phat[j + d][j] for j in range(T - d)) - er[d]) / T) < 1e-14


def test_gradient_vanishes_at_planted_pattern():
    # a target that IS a compact pattern: its own parameters reproduce both marginals (optimality condition)
    T = 16
    rng = np.random.default_rng(8)
    alpha, rho = rng.standard_normal(T), -0.2 * np.arange(T) + 0.1 * rng.standard_normal(T)
    Phat, _ = _brute_pattern(alpha, rho)
    ea, er, plogp = fo.marginals(Phat)
    ga, gr = fo.fit_gradient(alpha, rho, ea, er)
    assert np.max(np.abs(ga)) < 1e-15 and np.max(np.abs(gr)) < 1e-15
    assert abs(fo.fit_kl_dense(Phat, alpha, rho)) < 1e-14
    assert abs(fo.fit_kl_from_stats(alpha, rho, ea, er, plogp)) < 1e-13


# F5 ------------------------------------------------------------------------------------------------ invariances
def test_gauge_invariance():
    # alpha + c + b j and rho - c + b d add b i to row i: absorbed by Z(i), the objective does not move
    T = 13
    rng = np.random.default_rng(6)
    alpha, rho = rng.standard_normal(T), rng.standard_normal(T)
    ea, er, _ = fo.marginals(_random_target(T, 1))
    base = fo.fit_objective(alpha, rho, ea, er)
    idx = np.arange(T)
    # sum_j eta_abs(j) j + sum_d eta_rel(d) d = sum_i i (every row has unit mass), so the shift cancels exactly
    moved = fo.fit_objective(alpha + 0.7 + 0.3 * idx, rho - 0.7 + 0.3 * idx, ea, er)
    assert abs(moved - base) < 1e-12


# F6 ------------------------------------------------------------------------------------------------ Fit
def _torch_objective(x, ea, er, T):
    """The objective written independently with torch ops (logsumexp over masked rows), for autograd."""
    alpha, rho = x[:T], x[T:]
    i = torch.arange(T)[:, None]
    j = torch.arange(T)[None, :]
    b = alpha[None, :] + rho[(i - j).clamp(min=0)]
    b = b.masked_fill(j > i, float("-inf"))
    return (torch.logsumexp(b, dim=1).sum() - (ea * alpha).sum() - (er * rho).sum()) / T


@pytest.mark.parametrize("T,steps", [(24, 1), (24, 7), (40, 60)])
def test_fit_matches_torch_adam(T, steps):
    P = _random_target(T, 13)
    ea, er, _ = fo.marginals(P)
    alpha, rho, logZ = fo.fit_compact(ea, er, steps=steps, lr=0.05)
    a0, r0 = fo.fit_init(er)
    x = torch.tensor(np.concatenate([a0, r0]), dtype=torch.float64, requires_grad=True)
    opt = torch.optim.Adam([x], lr=0.05)
    tea, ter = torch.tensor(ea), torch.tensor(er)
    for _ in range(steps):
        opt.zero_grad()
        _torch_objective(x, tea, ter, T).backward()
        opt.step()
    got = x.detach().numpy()
    assert np.max(np.abs(got[:T] - alpha)) < 1e-9
    assert np.max(np.abs(got[T:] - rho)) < 1e-9
    _, want_logZ = _brute_pattern(alpha, rho)
    assert np.max(np.abs(logZ - want_logZ)) < 1e-12


def test_fit_init_values():
    T = 6
    er = np.array([3.0, 1.5, 0.0, 2e-9, 0.8, 0.2])
    a, r = fo.fit_init(er)
    assert np.all(a == 0)
    for d in range(T):
        assert abs(r[d] - math.log(max(er[d] / (T - d), 1e-9))) < 1e-15


def test_fit_recovers_planted_pattern():
    # the objective is convex with its optimum where both marginals match; a planted compact target must be
    # fitted to a small KL within the prescribed 400 steps, and the loss must fall from its starting value
    T = 48
    rng = np.random.default_rng(21)
    alpha = 0.5 * rng.standard_normal(T)
    alpha[0] += 3.0
    rho = -0.15 * np.arange(T) + 0.1 * rng.standard_normal(T)
    P, _ = _brute_pattern(alpha, rho)
    ea, er, plogp = fo.marginals(P)
    a0, r0 = fo.fit_init(er)
    start = fo.fit_kl_from_stats(a0, r0, ea, er, plogp)
    fa, fr, _ = fo.fit_compact(ea, er, steps=400, lr=0.05)
    kappa = fo.fit_kl_dense(P, fa, fr)
    assert kappa < 0.02 and kappa < 0.1 * start
    ga, gr = fo.fit_gradient(fa, fr, ea, er)
    col = ga * T + ea
    assert np.max(np.abs(col - ea)) < 0.05 * np.max(ea)


# F7 ------------------------------------------------------------------------------------------------ KL
def test_kl_dense_brute_force_and_stats_identity():
    T = 14
    rng = np.random.default_rng(17)
    alpha, rho = rng.standard_normal(T), rng.standard_normal(T)
    P = _random_target(T, 19)
    ea, er, plogp = fo.marginals(P)
    Phat, _ = _brute_pattern(alpha, rho)
    want = sum(P[i, j] * math.log(P[i, j] / Phat[i][j]) for i in range(T) for j in range(i + 1)) / T
    assert abs(fo.fit_kl_dense(P, alpha, rho) - want) < 1e-13
    assert abs(fo.fit_kl_from_stats(alpha, rho, ea, er, plogp) - want) < 1e-12
    assert want > 0


# F8 ------------------------------------------------------------------------------------------------ convolution
def test_logZ_convolution_matches_dense_and_brute_force():
    T = 200
    rng = np.random.default_rng(23)
    alpha, rho = rng.standard_normal(T), -0.02 * np.arange(T) + 0.1 * rng.standard_normal(T)
    _, want = _brute_pattern(alpha, rho)
    got = fo.logZ_convolution(alpha, rho)
    assert np.max(np.abs(got - want)) < 1e-10
    dense, _ = fo._logZ_and_P(alpha, rho)
    assert np.max(np.abs(dense - want)) < 1e-12


def test_fit_head_end_to_end_accepts_compact_target_and_reports_kappa():
    T = 32
    A = si.mean_attention_maps(1, T, 29)[0]
    alpha, rho, logZ, kappa, ok = fo.fit_head(A, steps=400)
    P = fo.target_from_mean_attention(A)
    Phat, _ = _brute_pattern(alpha, rho)
    want = sum(P[i, j] * math.log(P[i, j] / Phat[i][j]) for i in range(T) for j in range(i + 1)) / T
    assert abs(kappa - want) < 1e-12
    assert ok == (kappa <= 0.2)
