"""CPU oracle for the compact-pattern fitter (the one-time step that produces alpha, rho, log Z of a frozen head).

TEST INFRASTRUCTURE ONLY.  Plain, slow, dense fp64 numpy; it shares no code with the CUDA path and is imported only
by the tests and by the benchmark's CPU-baseline leg; the product never calls it.

What it computes, in the paper's order and notation (0-based indices: alpha[j], j in [0,T); rho[d], d = i-j):

* target          - Algorithm 1 (selection and fitting loop): the causal entries of a mean attention map are floored
                    at 1e-9 and every row is normalised to sum to one; this is the target pattern P.
* marginals       - Sec. 3.2, below Eq. "fit-objective": eta_abs(j) = sum_{i>=j} P(i,j) (column sums) and
                    eta_rel(d) = sum_{i-j=d} P(i,j) (diagonal sums): the sufficient statistics of the fit.
* objective       - Eq. "fit-objective": L(alpha,rho) = (1/T) [ sum_i log Z(i) - sum_j eta_abs(j) alpha(j)
                    - sum_d eta_rel(d) rho(d) ],  Z(i) = sum_{k<=i} exp(alpha(k) + rho(i-k)) (Eq. "compact-prior").
* gradient        - Appendix "Compact fitting and storage": dL/dalpha(j) = (sum_i P^(i,j) - eta_abs(j)) / T and the
                    analogous dL/drho(d) = (sum_{i-j=d} P^(i,j) - eta_rel(d)) / T, with P^ formed densely.
* Fit             - Appendix "Selection, fitting, and installation": alpha = 0,
                    rho(d) = log max(eta_rel(d) / (T - d), 1e-9), then J = 400 Adam steps at learning rate 0.05 on the
                    objective, no early stopping.  The paper names the optimiser only; this file takes Adam as
                    published (beta1 0.9, beta2 0.999, eps 1e-8, bias-corrected moments,
                    x -= lr * mhat / (sqrt(vhat) + eps)).
* acceptance      - Algorithm 1: kappa = (1/T) sum_i KL(P[i,:i+1] || P^[i,:i+1]); a head passes if kappa <= 0.2 nats.
                    `fit_kl_dense` forms P^ and the KL row by row; `fit_kl_from_stats` is the same number from the
                    sufficient statistics (rows of P sum to one, so
                    kappa = L(alpha,rho) + (1/T) sum_{ij} P(i,j) log P(i,j)), which is how a fitter that never
                    forms the T x T matrix gets it.
* convolution form - Appendix "Compact fitting and storage" (the FFT fitter): Z(i) is the causal convolution of
                    exp(alpha) with exp(rho); `logZ_convolution` evaluates it with numpy's FFT.

Parity status: pinned in tests/test_fit_oracle_pins.py by brute-force Python loops on tiny inputs, finite differences
of the objective, torch autograd + torch.optim.Adam on an independently written objective, the closed form at T = 2,
gauge invariances of Eq. "compact-prior", the recovery of a planted (alpha, rho) and the agreement of the dense and
convolution normalisers.  The paper prints no worked numeric example.
"""
from __future__ import annotations

import numpy as np

FLOOR = 1e-9
ADAM_BETA1 = 0.9
ADAM_BETA2 = 0.999
ADAM_EPS = 1e-8


def _logZ_and_P(alpha: np.ndarray, rho: np.ndarray):
    """Dense log Z(i) and P^(i,j) of Eq. "compact-prior" (fp64, max-subtracted rows)."""
    T = alpha.shape[0]
    i = np.arange(T)[:, None]
    j = np.arange(T)[None, :]
    causal = j <= i
    b = np.where(causal, alpha[None, :].astype(np.float64) + rho.astype(np.float64)[np.clip(i - j, 0, T - 1)], -np.inf)
    m = b.max(axis=1, keepdims=True)
    e = np.exp(b - m)
    s = e.sum(axis=1, keepdims=True)
    return (m + np.log(s))[:, 0], e / s


def target_from_mean_attention(Abar: np.ndarray, floor: float = FLOOR) -> np.ndarray:
    """Algorithm 1: floor the causal entries of the mean attention map, then normalise every row."""
    T = Abar.shape[0]
    causal = np.tril(np.ones((T, T), dtype=bool))
    P = np.where(causal, np.maximum(Abar.astype(np.float64), floor), 0.0)
    return P / P.sum(axis=1, keepdims=True)


def marginals(P: np.ndarray):
    """eta_abs (column sums), eta_rel (diagonal sums) and sum_{ij} P log P of a causal row-stochastic P."""
    T = P.shape[0]
    P = P.astype(np.float64)
    eta_abs = np.tril(P).sum(axis=0)
    eta_rel = np.array([np.trace(P, offset=-d) for d in range(T)])
    causal = np.tril(np.ones((T, T), dtype=bool))
    plogp = float(np.sum(P[causal] * np.log(P[causal])))
    return eta_abs, eta_rel, plogp


def fit_objective(alpha, rho, eta_abs, eta_rel) -> float:
    """Eq. "fit-objective"."""
    T = alpha.shape[0]
    logZ, _ = _logZ_and_P(alpha, rho)
    return float((logZ.sum() - np.dot(eta_abs, alpha) - np.dot(eta_rel, rho)) / T)


def fit_gradient(alpha, rho, eta_abs, eta_rel):
    """Gradient of Eq. "fit-objective": fitted marginals minus target marginals, over T."""
    T = alpha.shape[0]
    _, Phat = _logZ_and_P(alpha, rho)
    col = Phat.sum(axis=0)
    diag = np.array([np.trace(Phat, offset=-d) for d in range(T)])
    return (col - eta_abs) / T, (diag - eta_rel) / T


def fit_init(eta_rel: np.ndarray, floor: float = FLOOR):
    """Fit's starting point: alpha = 0, rho(d) = log max(eta_rel(d) / (T - d), 1e-9)."""
    T = eta_rel.shape[0]
    d = np.arange(T)
    return np.zeros(T), np.log(np.maximum(eta_rel.astype(np.float64) / (T - d), floor))


def fit_compact(eta_abs, eta_rel, steps: int = 400, lr: float = 0.05):
    """Fit: `steps` Adam steps on Eq. "fit-objective" from the prescribed start.  Returns alpha, rho, log Z."""
    T = eta_abs.shape[0]
    eta_abs = eta_abs.astype(np.float64)
    eta_rel = eta_rel.astype(np.float64)
    alpha, rho = fit_init(eta_rel)
    x = np.concatenate([alpha, rho])
    m = np.zeros_like(x)
    v = np.zeros_like(x)
    for t in range(1, steps + 1):
        ga, gr = fit_gradient(x[:T], x[T:], eta_abs, eta_rel)
        g = np.concatenate([ga, gr])
        m = ADAM_BETA1 * m + (1.0 - ADAM_BETA1) * g
        v = ADAM_BETA2 * v + (1.0 - ADAM_BETA2) * g * g
        mhat = m / (1.0 - ADAM_BETA1 ** t)
        vhat = v / (1.0 - ADAM_BETA2 ** t)
        x = x - lr * mhat / (np.sqrt(vhat) + ADAM_EPS)
    alpha, rho = x[:T].copy(), x[T:].copy()
    logZ, _ = _logZ_and_P(alpha, rho)
    return alpha, rho, logZ


def fit_kl_dense(P: np.ndarray, alpha, rho) -> float:
    """kappa of Algorithm 1: mean over rows of KL(P[i,:i+1] || P^[i,:i+1]), with P^ formed densely."""
    T = P.shape[0]
    _, Phat = _logZ_and_P(alpha, rho)
    total = 0.0
    for i in range(T):
        p = P[i, : i + 1].astype(np.float64)
        q = Phat[i, : i + 1]
        nz = p > 0
        total += float(np.sum(p[nz] * (np.log(p[nz]) - np.log(q[nz]))))
    return total / T


def fit_kl_from_stats(alpha, rho, eta_abs, eta_rel, plogp: float) -> float:
    """The same kappa from the sufficient statistics: objective + (1/T) sum P log P."""
    T = alpha.shape[0]
    return fit_objective(alpha, rho, eta_abs, eta_rel) + plogp / T


def logZ_convolution(alpha, rho) -> np.ndarray:
    """log Z(i) as the causal convolution of exp(alpha) with exp(rho), evaluated with the FFT."""
    T = alpha.shape[0]
    ma, mr = float(np.max(alpha)), float(np.max(rho))
    A = np.exp(alpha.astype(np.float64) - ma)
    R = np.exp(rho.astype(np.float64) - mr)
    n = 1
    while n < 2 * T:
        n *= 2
    z = np.fft.irfft(np.fft.rfft(A, n) * np.fft.rfft(R, n), n)[:T]
    return np.log(np.maximum(z, np.finfo(np.float64).tiny)) + ma + mr


def fit_head(Abar: np.ndarray, steps: int = 400, lr: float = 0.05, eps_fit: float = 0.2):
    """One pass of Algorithm 1's loop body for a head: target, marginals, Fit, kappa, acceptance."""
    P = target_from_mean_attention(Abar)
    eta_abs, eta_rel, plogp = marginals(P)
    alpha, rho, logZ = fit_compact(eta_abs, eta_rel, steps, lr)
    kappa = fit_kl_dense(P, alpha, rho)
    return alpha, rho, logZ, kappa, bool(kappa <= eps_fit)
