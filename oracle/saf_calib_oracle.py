"""CPU oracle for the calibration statistics of a layer (Sec. 3.1 "Calibration and head selection").

TEST INFRASTRUCTURE ONLY.  Plain, slow, dense fp64 numpy; it shares no code with the CUDA path and is imported only
by the tests and by the benchmark's CPU-baseline leg; the product never calls it.

What it computes, for the N calibration sequences of one layer and each head h (0-based indices):

* attention maps   - Appendix A, Eq. "standard-head": A^(n) = softmax_causal(Q^(n) K^(n)T / sqrt(d_h)), lower
                     triangular including the diagonal, every row sums to one.
* empirical mean   - Sec. 3.1: A^ = (1/N) sum_n A^(n)   (the "post-softmax mean" that the fitter takes as its input).
* variance score   - Eq. "variance-score": s_var = 1 / ((N-1) T^2) * sum_n || A^(n) - A^ ||_F^2.
* forward-KL score - Eq. "forward-kl-score": s_KL = 1 / (N T) * sum_n sum_i KL( A^(n)[i,:i+1] || A^[i,:i+1] ),
                     with the convention 0 log 0 = 0.

Both scores are written exactly as the equations state them: the mean first, then a second pass over the N maps.
(The product accumulates sum_n ||A^(n)||^2 and sum_n sum A^(n) log A^(n) in one streaming pass and subtracts the
mean's terms at the end; that identity is checked in the tests, it is not used here.)

Parity status: pinned in tests/test_calib_oracle_pins.py by pure-Python loops on tiny inputs, torch's softmax on
masked logits, closed forms (identical sequences give zero scores; two sequences give
s_var = ||A1 - A2||_F^2 / (2 T^2) and s_KL = the Jensen-Shannon divergence averaged over rows) and the one-pass
identities.  The paper prints no worked numeric example.
"""
from __future__ import annotations

import numpy as np


def attention_maps(Q: np.ndarray, K: np.ndarray, scale: float | None = None) -> np.ndarray:
    """A^(n) for n < N of one head: Q, K are [N, T, D]; returns [N, T, T] fp64 (zeros above the diagonal)."""
    Q = Q.astype(np.float64)
    K = K.astype(np.float64)
    N, T, D = Q.shape
    if scale is None:
        scale = 1.0 / np.sqrt(D)
    causal = np.tril(np.ones((T, T), dtype=bool))
    out = np.empty((N, T, T))
    for n in range(N):
        S = (Q[n] @ K[n].T) * scale
        S = np.where(causal, S, -np.inf)
        m = S.max(axis=1, keepdims=True)
        e = np.exp(S - m)
        out[n] = e / e.sum(axis=1, keepdims=True)
    return out


def empirical_mean(A: np.ndarray) -> np.ndarray:
    """A^ = (1/N) sum_n A^(n)."""
    return A.astype(np.float64).sum(axis=0) / A.shape[0]


def variance_score(A: np.ndarray) -> float:
    """Eq. "variance-score"."""
    A = A.astype(np.float64)
    N, T, _ = A.shape
    mean = empirical_mean(A)
    total = 0.0
    for n in range(N):
        d = A[n] - mean
        total += float(np.sum(d * d))
    return total / ((N - 1) * T * T)


def forward_kl_score(A: np.ndarray) -> float:
    """Eq. "forward-kl-score" (0 log 0 = 0)."""
    A = A.astype(np.float64)
    N, T, _ = A.shape
    mean = empirical_mean(A)
    total = 0.0
    for n in range(N):
        for i in range(T):
            p = A[n, i, : i + 1]
            q = mean[i, : i + 1]
            nz = p > 0
            total += float(np.sum(p[nz] * (np.log(p[nz]) - np.log(q[nz]))))
    return total / (N * T)


def calibration_stats(Q: np.ndarray, K: np.ndarray, scale: float | None = None, kv_group: int = 1):
    """All heads of a layer.  Q is [N, H, T, D], K is [N, H // kv_group, T, D].
    Returns (mean [H, T, T], s_var [H], s_kl [H])."""
    N, H, T, D = Q.shape
    mean = np.empty((H, T, T))
    s_var = np.empty(H)
    s_kl = np.empty(H)
    for h in range(H):
        A = attention_maps(Q[:, h], K[:, h // kv_group], scale)
        mean[h] = empirical_mean(A)
        s_var[h] = variance_score(A) if N > 1 else np.nan
        s_kl[h] = forward_kl_score(A)
    return mean, s_var, s_kl
