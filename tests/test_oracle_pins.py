"""Pins for the fp64 CPU oracle: checks against things the paper and the mathematics fix,
none of which go through the oracle's own formulas.

Pins (each would fail under a plausible slip: dropped term, wrong sign, transposed operand,
off-by-one in the relative distance or the causal boundary):
  P1  rows of A and P^ sum to one, zeros above the diagonal           (Appendix A; Eq. compact-prior)
  P2  three routes to P^ agree: explicit Z(i) sums in pure Python, exp(alpha+rho-logZ) from the
      stored triple, causal softmax of the bias matrix                 (Eq. compact-prior; Alg. 1)
  P3  additive shifts of alpha / rho leave P^ unchanged                (Appendix E.1)
  P4  closed forms: alpha=rho=0 -> running mean; alpha=0, rho=-lambda d -> geometric normaliser;
      very negative rho for d>0 -> identity
  P5  all-ordinary layer == torch fp64 scaled_dot_product_attention(is_causal) and its autograd
  P6  frozen head == an ordinary head whose Q/K are engineered so that S[i,j] = alpha[j] - lambda (i-j) + c_i
  P7  gradients: frozen dQ = dK = 0; central finite differences of sum(O o dO) on tiny shapes;
      frozen dV against torch autograd through a dense P built with torch ops
  P8  pure-Python triple loops (math.exp) on tiny inputs for every output of the layer
  P9  grouped-query path (Appendix E.2): shared key/value heads == the multi-head layer on K, V repeated per
      query head, with the shared heads' gradients summed over their query heads (torch autograd through
      repeat_interleave; torch's own enable_gqa route for the all-ordinary case; finite differences)
  P11 packed Q/K layout (Appendix E.2: replaced heads have no query/key slot): equals the full layout with the
      ordinary heads scattered back, whatever sits in the frozen heads' slots; torch SDPA per ordinary head
  P10 pattern gradients (trainable-pattern control): central finite differences of sum(O o dO) through the
      layer's own forward, torch autograd through a causal softmax of the bias matrix, and the two zero-sum
      identities that shift invariance forces (sum_j dalpha(j) = 0, sum_d drho(d) = 0)
"""
import math

import numpy as np
import pytest
import torch

from oracle import saf_oracle as orc

RNG = np.random.default_rng(1234)


def _rand_head(T, D, rng=RNG):
    return (rng.standard_normal((T, D)), rng.standard_normal((T, D)), rng.standard_normal((T, D)),
            rng.standard_normal((T, D)))


def _rand_pattern(T, rng=RNG, slope=-0.05):
    return rng.standard_normal(T), slope * np.arange(T) + 0.1 * rng.standard_normal(T)


# ------------------------------------------------------------------ brute force (pure Python)
def brute_pattern(alpha, rho, T):
    P = [[0.0] * T for _ in range(T)]
    for i in range(T):
        Z = 0.0
        for k in range(i + 1):
            Z += math.exp(alpha[k] + rho[i - k])
        for j in range(i + 1):
            P[i][j] = math.exp(alpha[j] + rho[i - j]) / Z
    return np.array(P)


def brute_ordinary(Q, K, V, dO, scale):
    T, D = Q.shape
    A = np.zeros((T, T))
    for i in range(T):
        s = [scale * sum(Q[i][c] * K[j][c] for c in range(D)) for j in range(i + 1)]
        den = sum(math.exp(x) for x in s)
        for j in range(i + 1):
            A[i][j] = math.exp(s[j]) / den
    O = np.zeros((T, D))
    dV = np.zeros((T, D))
    dQ = np.zeros((T, D))
    dK = np.zeros((T, D))
    lse = np.zeros(T)
    for i in range(T):
        s = [scale * sum(Q[i][c] * K[j][c] for c in range(D)) for j in range(i + 1)]
        lse[i] = math.log(sum(math.exp(x) for x in s))
        for j in range(i + 1):
            for c in range(D):
                O[i][c] += A[i][j] * V[j][c]
                dV[j][c] += A[i][j] * dO[i][c]
    for i in range(T):
        dP = [sum(dO[i][c] * V[j][c] for c in range(D)) for j in range(i + 1)]
        delta = sum(A[i][j] * dP[j] for j in range(i + 1))
        for j in range(i + 1):
            dS = A[i][j] * (dP[j] - delta)
            for c in range(D):
                dQ[i][c] += scale * dS * K[j][c]
                dK[j][c] += scale * dS * Q[i][c]
    return O, lse, dQ, dK, dV


# ------------------------------------------------------------------ P1
@pytest.mark.parametrize("T", [1, 2, 7, 64, 129])
def test_p1_row_stochastic_and_causal(T):
    Q, K, V, _ = _rand_head(T, 8)
    _, _, A = orc.ordinary_head_fwd(Q, K, V, 0.3)
    a, r = _rand_pattern(T)
    P = orc.pattern_dense(a, r, T)
    for M in (A, P):
        assert np.abs(M.sum(axis=1) - 1.0).max() < 1e-12
        assert np.all(np.triu(M, 1) == 0.0)
        assert np.all(M[np.tril_indices(T)] > 0.0)


# ------------------------------------------------------------------ P2
@pytest.mark.parametrize("T", [1, 5, 33])
def test_p2_three_routes(T):
    a, r = _rand_pattern(T)
    P_def = brute_pattern(a, r, T)                                    # explicit Z(i)
    P_orc = orc.pattern_dense(a, r, T)
    logZ = orc.pattern_logZ(a, r, T)
    i = np.arange(T)[:, None]
    j = np.arange(T)[None, :]
    P_trip = np.where(j <= i, np.exp(a[j] + r[np.abs(i - j)] - logZ[:, None]), 0.0)
    bias = torch.tensor(np.where(j <= i, a[j] + r[np.abs(i - j)], -np.inf))
    P_soft = torch.softmax(bias, dim=1).numpy()
    for P in (P_orc, P_trip, P_soft):
        assert np.abs(P - P_def).max() < 1e-12


def test_p2_logZ_prefix_property():
    """Row i uses only alpha[0..i], rho[0..i]: logZ at a stored length serves every shorter T."""
    a, r = _rand_pattern(192)
    full = orc.pattern_logZ(a, r, 192)
    short = orc.pattern_logZ(a[:129], r[:129], 129)
    assert np.array_equal(full[:129], short)
    brute = [math.log(sum(math.exp(a[k] + r[i - k]) for k in range(i + 1))) for i in range(192)]
    assert np.abs(full - np.array(brute)).max() < 1e-12


def test_p2_rows_argument_is_a_row_slice():
    a, r = _rand_pattern(77)
    P = orc.pattern_dense(a, r, 77)
    assert np.array_equal(orc.pattern_dense(a, r, 77, slice(13, 40)), P[13:40])


# ------------------------------------------------------------------ P3
def test_p3_shift_invariance():
    a, r = _rand_pattern(50)
    P = orc.pattern_dense(a, r, 50)
    assert np.abs(orc.pattern_dense(a + 3.7, r - 11.0, 50) - P).max() < 1e-13
    # a tilt alpha(j)+c j, rho(d)+c d only adds c*i to row i, which the row normaliser absorbs
    c = 0.02
    P_t = orc.pattern_dense(a + c * np.arange(50), r + c * np.arange(50), 50)
    assert np.abs(P_t - P).max() < 1e-13


# ------------------------------------------------------------------ P4
def test_p4_uniform_pattern_closed_form():
    T, D = 40, 5
    V, dO = RNG.standard_normal((T, D)), RNG.standard_normal((T, D))
    z = np.zeros(T)
    P = orc.pattern_dense(z, z, T)
    i = np.arange(T)
    assert np.abs(P - np.tril(np.ones((T, T))) / (i[:, None] + 1)).max() < 1e-15
    assert np.abs(orc.pattern_logZ(z, z, T) - np.log(i + 1)).max() < 1e-14
    O, _ = orc.frozen_head_fwd(V, z, z)
    assert np.abs(O - np.cumsum(V, axis=0) / (i[:, None] + 1)).max() < 1e-13
    dV = orc.frozen_head_bwd(dO, z, z)
    expect = np.cumsum((dO / (i[:, None] + 1))[::-1], axis=0)[::-1]     # sum_{i>=j} dO_i/(i+1)
    assert np.abs(dV - expect).max() < 1e-13


def test_p4_geometric_normaliser():
    T, lam = 300, 0.05
    logZ = orc.pattern_logZ(np.zeros(T), -lam * np.arange(T), T)
    i = np.arange(T)
    closed = np.log((1 - np.exp(-lam * (i + 1))) / (1 - np.exp(-lam)))
    assert np.abs(logZ - closed).max() < 1e-12


def test_p4_identity_limit():
    T = 17
    V = RNG.standard_normal((T, 3))
    rho = np.full(T, -800.0)
    rho[0] = 0.0
    O, P = orc.frozen_head_fwd(V, RNG.standard_normal(T), rho)
    assert np.array_equal(P, np.eye(T))
    assert np.array_equal(O, V)


def test_p4_distance_direction():
    """rho is indexed by i-j (how far back the key lies): with rho = [0, big, -inf...] row i puts
    nearly all mass on key i-1, not i+1 and not on a fixed column."""
    T = 9
    rho = np.full(T, -50.0)
    rho[1] = 10.0
    P = orc.pattern_dense(np.zeros(T), rho, T)
    for i in range(1, T):
        assert P[i].argmax() == i - 1 and P[i, i - 1] > 0.999
    # alpha is indexed by the key: a spike on key 2 draws every row i >= 2 to column 2
    a = np.zeros(T)
    a[2] = 30.0
    P = orc.pattern_dense(a, np.zeros(T), T)
    assert all(P[i].argmax() == 2 for i in range(2, T))


# ------------------------------------------------------------------ P5
@pytest.mark.parametrize("B,H,T,D", [(2, 3, 33, 8), (1, 2, 129, 64)])
def test_p5_all_ordinary_equals_sdpa(B, H, T, D):
    rng = np.random.default_rng(5)
    Q, K, V, dO = (rng.standard_normal((B, H, T, D)) for _ in range(4))
    mask = np.zeros(H, dtype=np.uint8)
    O, LSE = orc.hybrid_attn_fwd(Q, K, V, mask, None, None)
    dQ, dK, dV = orc.hybrid_attn_bwd(Q, K, V, dO, mask, None, None)
    tq, tk, tv = (torch.tensor(x, requires_grad=True) for x in (Q, K, V))
    to = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, is_causal=True)
    to.backward(torch.tensor(dO))
    assert np.abs(O - to.detach().numpy()).max() < 1e-12
    for g, t in ((dQ, tq), (dK, tk), (dV, tv)):
        assert np.abs(g - t.grad.numpy()).max() < 1e-11
    s = torch.einsum("bhid,bhjd->bhij", tq.detach(), tk.detach()) / math.sqrt(D)
    s = s.masked_fill(torch.triu(torch.ones(T, T, dtype=torch.bool), 1), -math.inf)
    assert np.abs(LSE - torch.logsumexp(s, dim=-1).numpy()).max() < 1e-12


# ------------------------------------------------------------------ P6
def test_p6_frozen_equals_engineered_ordinary_head():
    T, D, lam, scale = 96, 8, 0.0625, 0.125
    rng = np.random.default_rng(6)
    alpha = rng.standard_normal(T)
    V = rng.standard_normal((T, D))
    dO = rng.standard_normal((T, D))
    Q = np.zeros((T, D))
    K = np.zeros((T, D))
    Q[:, 0] = Q[:, 1] = 1.0 / scale
    K[:, 0] = alpha
    K[:, 1] = lam * np.arange(T)            # S[i,j] = alpha[j] + lam*j = alpha[j] - lam*(i-j) + lam*i
    O_ord, _, A = orc.ordinary_head_fwd(Q, K, V, scale)
    O_frz, P = orc.frozen_head_fwd(V, alpha, -lam * np.arange(T))
    assert np.abs(A - P).max() < 1e-14
    assert np.abs(O_ord - O_frz).max() < 1e-13
    _, _, dV_ord = orc.ordinary_head_bwd(Q, K, V, dO, scale)
    assert np.abs(dV_ord - orc.frozen_head_bwd(dO, alpha, -lam * np.arange(T))).max() < 1e-13


# ------------------------------------------------------------------ P7
def test_p7_frozen_heads_have_zero_qk_grads_and_poisoned_qk_is_ignored():
    B, H, T, D = 2, 4, 20, 4
    rng = np.random.default_rng(7)
    Q, K, V, dO = (rng.standard_normal((B, H, T, D)) for _ in range(4))
    mask = np.array([0, 1, 0, 1], dtype=np.uint8)
    alpha, rho = rng.standard_normal((H, T)), rng.standard_normal((H, T))
    Q[:, 1] = np.nan
    K[:, 3] = np.nan
    O, LSE = orc.hybrid_attn_fwd(Q, K, V, mask, alpha, rho)
    dQ, dK, dV = orc.hybrid_attn_bwd(Q, K, V, dO, mask, alpha, rho)
    assert np.isfinite(O).all() and np.isfinite(dV).all()
    for h in (1, 3):
        assert not dQ[:, h].any() and not dK[:, h].any() and not LSE[:, h].any()
    for h in (0, 2):
        # query 0 sees a single key, so its softmax is constant and dQ[0] = 0; every other row is nonzero
        assert np.abs(dQ[:, h, 1:]).min() > 0 and np.abs(dK[:, h, :-1]).min() > 0


def test_p7_finite_differences():
    B, H, T, D = 1, 3, 11, 4
    rng = np.random.default_rng(8)
    Q, K, V, dO = (rng.standard_normal((B, H, T, D)) for _ in range(4))
    mask = np.array([0, 1, 0], dtype=np.uint8)
    alpha, rho = rng.standard_normal((H, T)), rng.standard_normal((H, T))
    dQ, dK, dV = orc.hybrid_attn_bwd(Q, K, V, dO, mask, alpha, rho)

    def loss(q, k, v):
        return (orc.hybrid_attn_fwd(q, k, v, mask, alpha, rho)[0] * dO).sum()

    h = 1e-6
    for name, X, G in (("Q", Q, dQ), ("K", K, dK), ("V", V, dV)):
        num = np.zeros_like(X)
        it = np.nditer(X, flags=["multi_index"])
        for _ in it:
            idx = it.multi_index
            old = X[idx]
            X[idx] = old + h
            lp = loss(Q, K, V)
            X[idx] = old - h
            lm = loss(Q, K, V)
            X[idx] = old
            num[idx] = (lp - lm) / (2 * h)
        assert np.abs(num - G).max() < 2e-8, name


def test_p7_frozen_dv_vs_autograd():
    T, D = 23, 5
    rng = np.random.default_rng(9)
    a, r = rng.standard_normal(T), rng.standard_normal(T)
    V, dO = rng.standard_normal((T, D)), rng.standard_normal((T, D))
    i = torch.arange(T)[:, None]
    j = torch.arange(T)[None, :]
    bias = torch.tensor(a)[j.expand(T, T)] + torch.tensor(r)[(i - j).clamp(min=0)]
    P = torch.softmax(bias.masked_fill(j > i, -math.inf), dim=1)
    tv = torch.tensor(V, requires_grad=True)
    (P @ tv).backward(torch.tensor(dO))
    assert np.abs(orc.frozen_head_bwd(dO, a, r) - tv.grad.numpy()).max() < 1e-13
    assert np.abs(orc.frozen_head_fwd(V, a, r)[0] - (P @ tv).detach().numpy()).max() < 1e-13


# ------------------------------------------------------------------ P8
def test_p8_brute_force_layer():
    B, H, T, D = 2, 3, 9, 3
    rng = np.random.default_rng(10)
    Q, K, V, dO = (rng.standard_normal((B, H, T, D)) for _ in range(4))
    mask = np.array([1, 0, 1], dtype=np.uint8)
    alpha, rho = rng.standard_normal((H, T + 4)), rng.standard_normal((H, T + 4))   # stored length > T
    scale = 1.0 / math.sqrt(D)
    O, LSE = orc.hybrid_attn_fwd(Q, K, V, mask, alpha, rho)
    dQ, dK, dV = orc.hybrid_attn_bwd(Q, K, V, dO, mask, alpha, rho)
    for b in range(B):
        for h in range(H):
            if mask[h]:
                P = brute_pattern(alpha[h], rho[h], T)
                eO = np.array([[sum(P[i][j] * V[b, h, j, c] for j in range(T)) for c in range(D)] for i in range(T)])
                edV = np.array([[sum(P[i][j] * dO[b, h, i, c] for i in range(T)) for c in range(D)] for j in range(T)])
                assert np.abs(O[b, h] - eO).max() < 1e-13
                assert np.abs(dV[b, h] - edV).max() < 1e-13
                assert not dQ[b, h].any() and not dK[b, h].any()
            else:
                eO, else_, edQ, edK, edV = brute_ordinary(Q[b, h], K[b, h], V[b, h], dO[b, h], scale)
                assert np.abs(O[b, h] - eO).max() < 1e-13
                assert np.abs(LSE[b, h] - else_).max() < 1e-13
                for g, e in ((dQ, edQ), (dK, edK), (dV, edV)):
                    assert np.abs(g[b, h] - e).max() < 1e-13


# ------------------------------------------------------------------ panel routes == dense
@pytest.mark.parametrize("frozen", [False, True])
def test_panel_routes_equal_dense(frozen):
    T, D = 150, 6
    rng = np.random.default_rng(11)
    Q, K, V, dO = _rand_head(T, D, rng)
    a, r = _rand_pattern(T, rng)
    scale = 0.2
    O, LSE = orc.head_fwd_panels(frozen, Q, K, V, a, r, scale, panel=64)
    gQ, gK, gV = orc.head_bwd_panels(frozen, Q, K, V, dO, a, r, scale, panel=64)
    if frozen:
        eO = orc.frozen_head_fwd(V, a, r)[0]
        eQ, eK, eV = np.zeros((T, D)), np.zeros((T, D)), orc.frozen_head_bwd(dO, a, r)
    else:
        eO, eL, _ = orc.ordinary_head_fwd(Q, K, V, scale)
        eQ, eK, eV = orc.ordinary_head_bwd(Q, K, V, dO, scale)
        assert np.abs(LSE - eL).max() < 1e-13
    for g, e in ((O, eO), (gQ, eQ), (gK, eK), (gV, eV)):
        assert np.abs(g - e).max() < 1e-12


# ------------------------------------------------------------------ P9 grouped-query path
@pytest.mark.parametrize("H,g,frozen", [(4, 2, ()), (6, 3, (1, 5)), (4, 4, (0, 2)), (4, 1, (3,))])
def test_p9_gqa_equals_repeated_kv(H, g, frozen):
    B, T, D = 2, 21, 8
    rng = np.random.default_rng(90 + H + g)
    Q, dO = rng.standard_normal((B, H, T, D)), rng.standard_normal((B, H, T, D))
    K, V = rng.standard_normal((B, H // g, T, D)), rng.standard_normal((B, H // g, T, D))
    mask = np.zeros(H, dtype=np.uint8)
    mask[list(frozen)] = 1
    alpha, rho = rng.standard_normal((H, T)), -0.1 * np.arange(T)[None, :] + 0.1 * rng.standard_normal((H, T))
    O, LSE = orc.hybrid_attn_fwd(Q, K, V, mask, alpha, rho)
    dQ, dK, dV = orc.hybrid_attn_bwd(Q, K, V, dO, mask, alpha, rho)
    assert dK.shape == K.shape and dV.shape == V.shape
    # torch: repeat the shared heads, dense attention weights per head, autograd sums the shared gradients
    tq, tk, tv = (torch.tensor(x, requires_grad=True) for x in (Q, K, V))
    kr, vr = tk.repeat_interleave(g, dim=1), tv.repeat_interleave(g, dim=1)
    causal = torch.tril(torch.ones(T, T, dtype=torch.bool))
    outs = []
    for h in range(H):
        if mask[h]:
            i, j = np.indices((T, T))
            bias = torch.tensor(alpha[h][j] + rho[h][np.clip(i - j, 0, None)])
            w = torch.softmax(bias.masked_fill(~causal, -math.inf), dim=-1)
            outs.append(torch.einsum("ij,bjd->bid", w, vr[:, h]))
        else:
            s = torch.einsum("bid,bjd->bij", tq[:, h], kr[:, h]) / math.sqrt(D)
            w = torch.softmax(s.masked_fill(~causal, -math.inf), dim=-1)
            outs.append(torch.einsum("bij,bjd->bid", w, vr[:, h]))
    to = torch.stack(outs, dim=1)
    to.backward(torch.tensor(dO))
    assert np.abs(O - to.detach().numpy()).max() < 1e-12
    assert np.abs(dQ - tq.grad.numpy()).max() < 1e-11
    assert np.abs(dK - tk.grad.numpy()).max() < 1e-11
    assert np.abs(dV - tv.grad.numpy()).max() < 1e-11
    for h in frozen:
        assert not dQ[:, h].any()


def test_p9_gqa_all_ordinary_equals_torch_enable_gqa():
    B, H, g, T, D = 2, 8, 4, 40, 16
    rng = np.random.default_rng(99)
    Q = rng.standard_normal((B, H, T, D))
    K, V = rng.standard_normal((B, H // g, T, D)), rng.standard_normal((B, H // g, T, D))
    O, _ = orc.hybrid_attn_fwd(Q, K, V, np.zeros(H, dtype=np.uint8), None, None)
    to = torch.nn.functional.scaled_dot_product_attention(torch.tensor(Q), torch.tensor(K), torch.tensor(V),
                                                          is_causal=True, enable_gqa=True)
    assert np.abs(O - to.numpy()).max() < 1e-12


def test_p9_gqa_finite_differences_of_shared_heads():
    B, H, g, T, D = 1, 4, 2, 7, 3
    rng = np.random.default_rng(91)
    Q, dO = rng.standard_normal((B, H, T, D)), rng.standard_normal((B, H, T, D))
    K, V = rng.standard_normal((B, H // g, T, D)), rng.standard_normal((B, H // g, T, D))
    mask = np.array([0, 1, 0, 0], dtype=np.uint8)
    alpha, rho = rng.standard_normal((H, T)), rng.standard_normal((H, T))
    _, dK, dV = orc.hybrid_attn_bwd(Q, K, V, dO, mask, alpha, rho)

    def loss(Kx, Vx):
        O, _ = orc.hybrid_attn_fwd(Q, Kx, Vx, mask, alpha, rho)
        return float((O * dO).sum())

    h = 1e-6
    for arr, grad, which in ((K, dK, 0), (V, dV, 1)):
        for idx in [(0, 0, 2, 1), (0, 1, 5, 0), (0, 1, 0, 2), (0, 0, 6, 2)]:
            ap, am = arr.copy(), arr.copy()
            ap[idx] += h
            am[idx] -= h
            fd = (loss(ap, V) - loss(am, V)) / (2 * h) if which == 0 else (loss(K, ap) - loss(K, am)) / (2 * h)
            assert abs(fd - grad[idx]) < 1e-7


# ------------------------------------------------------------------ P10 pattern gradients
def test_p10_pattern_grads_vs_torch_autograd():
    B, H, T, D, Tp = 2, 4, 19, 5, 24
    rng = np.random.default_rng(100)
    V = rng.standard_normal((B, H // 2, T, D))             # shared value heads (group of 2)
    dO = rng.standard_normal((B, H, T, D))
    mask = np.array([1, 0, 1, 1], dtype=np.uint8)
    alpha, rho = rng.standard_normal((H, Tp)), rng.standard_normal((H, Tp))
    da, dr = orc.pattern_grads(V, dO, mask, alpha, rho)
    ta, tr = torch.tensor(alpha, requires_grad=True), torch.tensor(rho, requires_grad=True)
    i, j = np.indices((T, T))
    causal = torch.tril(torch.ones(T, T, dtype=torch.bool))
    loss = 0.0
    for h in range(H):
        if not mask[h]:
            continue
        bias = ta[h][torch.tensor(j)] + tr[h][torch.tensor(np.clip(i - j, 0, None))]
        w = torch.softmax(bias.masked_fill(~causal, -math.inf), dim=-1)
        for b in range(B):
            loss = loss + ((w @ torch.tensor(V[b, h // 2])) * torch.tensor(dO[b, h])).sum()
    loss.backward()
    assert np.abs(da - ta.grad.numpy()).max() < 1e-11
    assert np.abs(dr - tr.grad.numpy()).max() < 1e-11
    assert not da[1].any() and not dr[1].any() and not da[:, T:].any() and not dr[:, T:].any()


def test_p10_pattern_grads_finite_differences_and_zero_sums():
    T, D = 11, 4
    rng = np.random.default_rng(101)
    V, dO = rng.standard_normal((T, D)), rng.standard_normal((T, D))
    alpha, rho = rng.standard_normal(T), rng.standard_normal(T)
    da, dr = orc.pattern_grads_head(V, dO, alpha, rho)

    def loss(a, r):
        O, _ = orc.frozen_head_fwd(V, a, r)
        return float((O * dO).sum())

    h = 1e-6
    for k in range(T):
        e = np.zeros(T)
        e[k] = h
        assert abs((loss(alpha + e, rho) - loss(alpha - e, rho)) / (2 * h) - da[k]) < 1e-7
        assert abs((loss(alpha, rho + e) - loss(alpha, rho - e)) / (2 * h) - dr[k]) < 1e-7
    # P^ does not change when a constant is added to all of alpha, or to all of rho (Appendix E.1)
    assert abs(da.sum()) < 1e-12 and abs(dr.sum()) < 1e-12
    # the last distance is reached by one entry only: (i, j) = (T-1, 0)
    P = orc.pattern_dense(alpha, rho, T)
    G = dO @ V.T
    assert abs(dr[T - 1] - P[T - 1, 0] * (G[T - 1, 0] - (P[T - 1] * G[T - 1]).sum())) < 1e-13


# ------------------------------------------------------------------ P11 packed Q/K layout
def test_p11_packed_qk_equals_full_layout_and_sdpa():
    B, H, T, D = 2, 5, 17, 6
    rng = np.random.default_rng(110)
    mask = np.array([0, 1, 0, 1, 0], dtype=np.uint8)
    ordinary = [h for h in range(H) if not mask[h]]
    Qp, Kp = rng.standard_normal((B, 3, T, D)), rng.standard_normal((B, 3, T, D))
    V, dO = rng.standard_normal((B, H, T, D)), rng.standard_normal((B, H, T, D))
    alpha, rho = rng.standard_normal((H, T)), rng.standard_normal((H, T))
    O, LSE = orc.hybrid_attn_fwd(Qp, Kp, V, mask, alpha, rho)
    dQ, dK, dV = orc.hybrid_attn_bwd(Qp, Kp, V, dO, mask, alpha, rho)
    assert dQ.shape == Qp.shape and dK.shape == Kp.shape and dV.shape == V.shape
    # full layout with poisoned frozen slots
    Qf, Kf = np.full((B, H, T, D), np.nan), np.full((B, H, T, D), np.nan)
    Qf[:, ordinary], Kf[:, ordinary] = Qp, Kp
    Of, LSEf = orc.hybrid_attn_fwd(Qf, Kf, V, mask, alpha, rho)
    dQf, dKf, dVf = orc.hybrid_attn_bwd(Qf, Kf, V, dO, mask, alpha, rho)
    assert np.array_equal(O, Of) and np.array_equal(LSE, LSEf) and np.array_equal(dV, dVf)
    assert np.array_equal(dQ, dQf[:, ordinary]) and np.array_equal(dK, dKf[:, ordinary])
    # torch, ordinary head by ordinary head: slot s of the packed tensors belongs to head ordinary[s]
    for s_, h in enumerate(ordinary):
        tq, tk, tv = (torch.tensor(x, requires_grad=True) for x in (Qp[:, s_], Kp[:, s_], V[:, h]))
        to = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, is_causal=True)
        to.backward(torch.tensor(dO[:, h]))
        assert np.abs(O[:, h] - to.detach().numpy()).max() < 1e-12
        assert np.abs(dQ[:, s_] - tq.grad.numpy()).max() < 1e-11
        assert np.abs(dK[:, s_] - tk.grad.numpy()).max() < 1e-11
        assert np.abs(dV[:, h] - tv.grad.numpy()).max() < 1e-11
