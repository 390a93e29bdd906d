"""CPU oracle for the hybrid causal attention layer (ordinary softmax heads + frozen pattern heads).

TEST INFRASTRUCTURE ONLY.  This file is the plain, slow, dense fp64 statement of what the layer
computes.  It shares no code with the CUDA path and is imported only by the tests, by the smoke
check and by the benchmark's CPU-baseline leg; the product never calls it.

Every function is the paper's definition written out, dense and untiled (numpy matmul / exp / sum
serve as library steps; there is no online softmax, no key blocking, no factorised pattern):

* ordinary head   - Appendix A, Eq. "standard-head": S = Q K^T / sqrt(d_h), A = softmax_causal(S),
                    Z = A V; lower triangular including the diagonal, rows sum to one.
* frozen head     - Sec. 3.1: Z~ = P V with a fixed causal row-stochastic P, and Sec. 3.2,
                    Eq. "compact-prior": P^(i,j) = exp(alpha(j) + rho(i-j)) / Z(i) for j <= i, else 0,
                    Z(i) = sum_{k<=i} exp(alpha(k) + rho(i-k)).  Indices here are 0-based
                    (alpha[j], j in [0,T); rho[d], d = i-j in [0,T)).
* backward        - Sec. 3.3 / Appendix E.2: for a frozen head dV = P^T dZ and there are no
                    query/key gradients; alpha, rho and the normalisers get no gradient.  For an
                    ordinary head the gradients are the analytic derivatives of the definition:
                    dV = A^T dO, dP = dO V^T, delta_i = sum_j A_ij dP_ij, dS = A o (dP - delta),
                    dQ = scale dS K, dK = scale dS^T Q.

* pattern gradients - the control in which the compact patterns stay trainable (Appendix, trainable-pattern
                    ablation) differentiates the same definition: with the bias b_ij = alpha(j) + rho(i-j),
                    P^ = softmax_causal(b) and L = sum(O o dO), G = dO V^T,
                    dL/db_ij = P^_ij (G_ij - sum_k P^_ik G_ik), dL/dalpha(j) = sum_{i>=j} dL/db_ij,
                    dL/drho(d) = sum_{i-j=d} dL/db_ij.  The paper prints no formula for it; this is the
                    derivative of Eq. "compact-prior" written out.

Parity status: every function below is pinned by tests that do not go through this file's own
formulas (pure-Python brute force on tiny inputs, closed forms, shift invariance, the engineered
ordinary-head equivalence, torch's fp64 scaled_dot_product_attention + autograd, finite
differences); see tests/test_oracle_pins.py.  The paper prints no worked numeric example.
"""
from __future__ import annotations

import numpy as np


# ----------------------------------------------------------------------------- frozen pattern
def pattern_logZ(alpha: np.ndarray, rho: np.ndarray, T: int) -> np.ndarray:
    """log Z(i) = log sum_{k<=i} exp(alpha[k] + rho[i-k]), i in [0,T)  (Eq. "compact-prior").

    Uses only alpha[0..i] and rho[0..i]: the value for row i does not depend on T, so a vector
    computed at the stored length is valid for every shorter sequence."""
    a = np.asarray(alpha, dtype=np.float64)
    r = np.asarray(rho, dtype=np.float64)
    out = np.empty(T, dtype=np.float64)
    for i in range(T):
        t = a[: i + 1] + r[i::-1][: i + 1]      # alpha[k] + rho[i-k], k = 0..i
        m = t.max()
        out[i] = m + np.log(np.exp(t - m).sum())
    return out


def pattern_dense(alpha: np.ndarray, rho: np.ndarray, T: int, rows: slice | None = None) -> np.ndarray:
    """Dense P^ (Eq. "compact-prior") for the query rows in `rows` (default all) over all T keys.

    P^[i,j] = exp(alpha[j] + rho[i-j]) / Z(i) for j <= i, 0 for j > i.  Z(i) is summed explicitly
    over the causal row after subtracting the row maximum (which cancels in the ratio)."""
    a = np.asarray(alpha, dtype=np.float64)[:T]
    r = np.asarray(rho, dtype=np.float64)[:T]
    lo, hi, _ = (rows or slice(0, T)).indices(T)
    i = np.arange(lo, hi)[:, None]
    j = np.arange(T)[None, :]
    causal = j <= i
    bias = np.where(causal, a[j] + r[np.where(causal, i - j, 0)], -np.inf)
    e = np.exp(bias - bias.max(axis=1, keepdims=True))      # exp(-inf) = 0 above the diagonal
    return e / e.sum(axis=1, keepdims=True)


# ----------------------------------------------------------------------------- ordinary head
def softmax_causal(S: np.ndarray, row0: int = 0):
    """Causal softmax of score rows; row r of S is query index row0 + r, columns are all keys.
    Returns (A, LSE) with LSE_i = log sum_{k<=i} exp(S[i,k])."""
    n, T = S.shape
    i = (row0 + np.arange(n))[:, None]
    j = np.arange(T)[None, :]
    Sm = np.where(j <= i, S, -np.inf)
    m = Sm.max(axis=1, keepdims=True)
    e = np.exp(Sm - m)
    l = e.sum(axis=1, keepdims=True)
    return e / l, (m + np.log(l))[:, 0]


def ordinary_head_fwd(Q, K, V, scale, rows: slice | None = None):
    """O = softmax_causal(scale Q K^T) V for the query rows in `rows` (default all).
    Q,K,V: [T,D] float64.  Returns (O [n,D], LSE [n], A [n,T])."""
    T = Q.shape[0]
    lo, hi, _ = (rows or slice(0, T)).indices(T)
    S = scale * (Q[lo:hi] @ K.T)
    A, lse = softmax_causal(S, lo)
    return A @ V, lse, A


def ordinary_head_bwd(Q, K, V, dO, scale):
    """Analytic gradients of sum(O o dO) for one ordinary head.  Returns (dQ, dK, dV)."""
    O, _, A = ordinary_head_fwd(Q, K, V, scale)
    dV = A.T @ dO
    dP = dO @ V.T
    delta = (A * dP).sum(axis=1, keepdims=True)
    dS = A * (dP - delta)
    return scale * (dS @ K), scale * (dS.T @ Q), dV


# ----------------------------------------------------------------------------- frozen head
def frozen_head_fwd(V, alpha, rho, rows: slice | None = None):
    """O = P^ V for the query rows in `rows` (default all).  V: [T,D] float64."""
    P = pattern_dense(alpha, rho, V.shape[0], rows)
    return P @ V, P


def frozen_head_bwd(dO, alpha, rho):
    """dV = P^T dO; a frozen head has no query/key gradients."""
    P = pattern_dense(alpha, rho, dO.shape[0])
    return P.T @ dO


def pattern_grads_head(V, dO, alpha, rho):
    """Gradients of L = sum(O o dO), O = P^ V, with respect to alpha[0..T) and rho[0..T) of one head
    (V, dO: [T,D] float64).  Dense: the T x T matrices P^, G = dO V^T and dL/db are formed whole."""
    T = V.shape[0]
    P = pattern_dense(alpha, rho, T)
    G = dO @ V.T
    db = P * (G - (P * G).sum(axis=1, keepdims=True))       # softmax Jacobian applied row by row
    dalpha = db.sum(axis=0)                                  # alpha(j) enters every row i >= j at column j
    drho = np.array([np.trace(db, offset=-d) for d in range(T)])   # rho(d) enters the entries with i - j = d
    return dalpha, drho


def pattern_grads(V, dO, mask, alpha, rho):
    """dalpha, drho [H,Tp] summed over the batch; rows of ordinary heads and entries beyond T are zero.
    V: [B,Hkv,T,D] (head h reads V[:, h // (H/Hkv)]), dO: [B,H,T,D]."""
    B, H, T, _ = dO.shape
    g = H // V.shape[1]
    Tp = alpha.shape[1]
    dalpha, drho = np.zeros((H, Tp)), np.zeros((H, Tp))
    for h in range(H):
        if mask[h]:
            for b in range(B):
                da, dr = pattern_grads_head(V[b, h // g], dO[b, h], alpha[h], rho[h])
                dalpha[h, :T] += da
                drho[h, :T] += dr
    return dalpha, drho


# ----------------------------------------------------------------------------- the layer
def hybrid_attn_fwd(Q, K, V, mask, alpha, rho, scale=None):
    """Q: [B,H,T,D], K,V: [B,Hkv,T,D] float64 with Hkv dividing H (grouped-query path, Appendix E.2: query head h
    reads the shared key/value head h // (H/Hkv); Hkv = H is ordinary multi-head attention);
    mask: [H] (nonzero = frozen); alpha,rho: [H,Tp].
    Packed layout (Appendix E.2: replaced heads have no query/key slot on the multi-head path): when Q has fewer
    heads than the mask, Q and K hold the ordinary heads only, in head order.
    Returns O [B,H,T,D] and LSE [B,H,T] (0 for frozen heads, which have no softmax)."""
    B, _, T, D = V.shape
    H = len(mask)
    packed = Q is not None and Q.shape[1] != H
    slot = np.cumsum(np.asarray(mask) == 0) - 1            # ordinal of head h among the ordinary heads
    g = 1 if packed else H // V.shape[1]
    scale = 1.0 / np.sqrt(D) if scale is None else scale
    O = np.zeros((B, H, T, D))
    LSE = np.zeros((B, H, T))
    for h in range(H):
        if mask[h]:
            P = pattern_dense(alpha[h], rho[h], T)
            for b in range(B):
                O[b, h] = P @ V[b, h // g]
        else:
            hq, hk = (slot[h], slot[h]) if packed else (h, h // g)
            for b in range(B):
                O[b, h], LSE[b, h], _ = ordinary_head_fwd(Q[b, hq], K[b, hk], V[b, h // g], scale)
    return O, LSE


def hybrid_attn_bwd(Q, K, V, dO, mask, alpha, rho, scale=None):
    """Gradients of sum(O o dO) w.r.t. Q, K, V.  Frozen heads: dQ = dK = 0, dV = P^T dO.  With shared
    key/value heads (K, V: [B,Hkv,T,D]) the gradient of a shared head is the sum over the query heads that
    read it."""
    B, _, T, D = dO.shape
    H = len(mask)
    packed = Q is not None and Q.shape[1] != H       # Q, K, dQ, dK hold the ordinary heads only
    slot = np.cumsum(np.asarray(mask) == 0) - 1
    Hkv = V.shape[1]
    g = H // Hkv
    scale = 1.0 / np.sqrt(D) if scale is None else scale
    dQ = np.zeros(Q.shape if packed else (B, H, T, D))
    dK = np.zeros(K.shape if packed else (B, Hkv, T, D))
    dV = np.zeros((B, Hkv, T, D))
    for h in range(H):
        if mask[h]:
            P = pattern_dense(alpha[h], rho[h], T)
            for b in range(B):
                dV[b, h // g] += P.T @ dO[b, h]
        else:
            for b in range(B):
                hq, hk = (slot[h], slot[h]) if packed else (h, h // g)
                dq, dk, dv = ordinary_head_bwd(Q[b, hq], K[b, hk], V[b, h // g], dO[b, h], scale)
                dQ[b, hq] = dq
                dK[b, hk] += dk
                dV[b, h // g] += dv
    return dQ, dK, dV


# ----------------------------------------------------------------------------- large sizes
def head_fwd_panels(kind_frozen, Q, K, V, alpha, rho, scale, panel=512, rows: slice | None = None):
    """One (b,h) unit of the forward, evaluated in panels of query rows over ALL keys (still the
    dense definition; a panel only bounds memory).  Returns (O, LSE) for `rows`."""
    T = V.shape[0]
    lo, hi, _ = (rows or slice(0, T)).indices(T)
    O = np.empty((hi - lo, V.shape[1]))
    LSE = np.zeros(hi - lo)
    for r0 in range(lo, hi, panel):
        r1 = min(r0 + panel, hi)
        if kind_frozen:
            O[r0 - lo:r1 - lo], _ = frozen_head_fwd(V, alpha, rho, slice(r0, r1))
        else:
            O[r0 - lo:r1 - lo], LSE[r0 - lo:r1 - lo], _ = ordinary_head_fwd(Q, K, V, scale, slice(r0, r1))
    return O, LSE


def head_bwd_panels(kind_frozen, Q, K, V, dO, alpha, rho, scale, panel=512):
    """One (b,h) unit of the backward in panels of query rows over all keys.
    Returns (dQ, dK, dV); dQ and dK are zero for a frozen head."""
    T, D = V.shape
    dQ = np.zeros((T, D))
    dK = np.zeros((T, D))
    dV = np.zeros((T, D))
    for r0 in range(0, T, panel):
        r1 = min(r0 + panel, T)
        if kind_frozen:
            P = pattern_dense(alpha, rho, T, slice(r0, r1))
            dV += P.T @ dO[r0:r1]
        else:
            _, _, A = ordinary_head_fwd(Q, K, V, scale, slice(r0, r1))
            dV += A.T @ dO[r0:r1]
            dP = dO[r0:r1] @ V.T
            delta = (A * dP).sum(axis=1, keepdims=True)
            dS = A * (dP - delta)
            dQ[r0:r1] = scale * (dS @ K)
            dK += scale * (dS.T @ Q[r0:r1])
    return dQ, dK, dV
