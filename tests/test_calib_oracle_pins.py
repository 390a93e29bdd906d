"""Pins of the calibration-statistics oracle (oracle/saf_calib_oracle.py) against things it does not compute itself:
pure-Python loops, torch's softmax, closed forms and the one-pass identities.  CPU only."""
import math

import numpy as np
import torch

from oracle import saf_calib_oracle as co


def _qk(N, T, D, seed):
    rng = np.random.default_rng(seed)
    return rng.standard_normal((N, T, D)), rng.standard_normal((N, T, D))


def _brute_maps(Q, K, scale):
    N, T, D = Q.shape
    A = [[[0.0] * T for _ in range(T)] for _ in range(N)]
    for n in range(N):
        for i in range(T):
            s = [scale * sum(Q[n, i, c] * K[n, j, c] for c in range(D)) for j in range(i + 1)]
            z = sum(math.exp(x) for x in s)
            for j in range(i + 1):
                A[n][i][j] = math.exp(s[j]) / z
    return np.array(A)


# C1 ------------------------------------------------------------------------------------------------ maps
def test_attention_maps_brute_force_and_torch():
    N, T, D = 3, 7, 4
    Q, K = _qk(N, T, D, 0)
    A = co.attention_maps(Q, K)
    want = _brute_maps(Q, K, 1 / math.sqrt(D))
    assert np.max(np.abs(A - want)) < 1e-14
    assert np.all(np.triu(A, k=1) == 0)
    assert np.max(np.abs(A.sum(axis=2) - 1)) < 1e-14
    tq, tk = torch.tensor(Q), torch.tensor(K)
    S = tq @ tk.transpose(1, 2) / math.sqrt(D)
    S = S.masked_fill(torch.triu(torch.ones(T, T, dtype=torch.bool), diagonal=1), float("-inf"))
    assert np.max(np.abs(A - torch.softmax(S, dim=-1).numpy())) < 1e-14
    # an explicit scale is honoured
    A2 = co.attention_maps(Q, K, scale=0.3)
    assert np.max(np.abs(A2 - _brute_maps(Q, K, 0.3))) < 1e-14


# C2 ------------------------------------------------------------------------------------------------ mean, variance
def test_mean_and_variance_score_brute_force():
    N, T, D = 4, 6, 3
    Q, K = _qk(N, T, D, 1)
    A = _brute_maps(Q, K, 1 / math.sqrt(D))
    mean = co.empirical_mean(A)
    for i in range(T):
        for j in range(T):
            assert abs(mean[i, j] - sum(A[n, i, j] for n in range(N)) / N) < 1e-15
    want = sum((A[n, i, j] - mean[i, j]) ** 2 for n in range(N) for i in range(T) for j in range(T)) / ((N - 1) * T * T)
    assert abs(co.variance_score(A) - want) < 1e-16
    # the same number as the mean over all T^2 entries of the unbiased sample variance across inputs
    assert abs(want - np.var(A, axis=0, ddof=1).sum() / (T * T)) < 1e-16


def test_forward_kl_score_brute_force():
    N, T, D = 3, 6, 3
    Q, K = _qk(N, T, D, 2)
    A = _brute_maps(Q, K, 1 / math.sqrt(D))
    mean = A.sum(axis=0) / N
    want = sum(A[n, i, j] * math.log(A[n, i, j] / mean[i, j]) for n in range(N) for i in range(T)
               for j in range(i + 1)) / (N * T)
    assert abs(co.forward_kl_score(A) - want) < 1e-15
    assert want > 0


# C3 ------------------------------------------------------------------------------------------------ closed forms
def test_identical_sequences_have_zero_scores():
    Q, K = _qk(1, 9, 4, 3)
    A = np.repeat(co.attention_maps(Q, K), 5, axis=0)
    assert co.variance_score(A) < 1e-30        # (sum of five equal numbers over five: last-bit rounding only)
    assert abs(co.forward_kl_score(A)) < 1e-16


def test_two_sequences_closed_forms():
    # N = 2: A^ is the midpoint, so s_var = ||A1 - A2||_F^2 / (2 T^2) and s_KL is the row-averaged
    # Jensen-Shannon divergence
    T = 8
    Q, K = _qk(2, T, 4, 4)
    A = co.attention_maps(Q, K)
    want_var = float(np.sum((A[0] - A[1]) ** 2)) / (2 * T * T)
    assert abs(co.variance_score(A) - want_var) < 1e-16
    js = 0.0
    for i in range(T):
        p, q = A[0, i, : i + 1], A[1, i, : i + 1]
        m = 0.5 * (p + q)
        js += 0.5 * float(np.sum(p * np.log(p / m))) + 0.5 * float(np.sum(q * np.log(q / m)))
    assert abs(co.forward_kl_score(A) - js / T) < 1e-15


def test_one_hot_versus_uniform_rows():
    # hand-built maps: sequence 0 attends to the newest key only, sequence 1 uniformly over the causal prefix
    T = 5
    A = np.zeros((2, T, T))
    for i in range(T):
        A[0, i, i] = 1.0
        A[1, i, : i + 1] = 1.0 / (i + 1)
    mean = 0.5 * (A[0] + A[1])
    want_var = sum((1 - 1 / (i + 1)) ** 2 + i * (1 / (i + 1)) ** 2 for i in range(T)) / (2 * T * T)
    assert abs(co.variance_score(A) - want_var) < 1e-16
    want_kl = 0.0
    for i in range(T):
        u = 1.0 / (i + 1)
        want_kl += math.log(1.0 / mean[i, i])                        # one-hot row: single term
        want_kl += sum(u * math.log(u / mean[i, j]) for j in range(i + 1))
    assert abs(co.forward_kl_score(A) - want_kl / (2 * T)) < 1e-15


# C4 ------------------------------------------------------------------------------------------------ identities
def test_one_pass_identities():
    # sum_n ||A_n - A^||^2 = sum_n ||A_n||^2 - N ||A^||^2 ; sum_n KL(A_n || A^) = sum_n sum A_n log A_n - N sum A^ log A^
    N, T, D = 5, 10, 4
    Q, K = _qk(N, T, D, 6)
    A = co.attention_maps(Q, K)
    mean = A.sum(axis=0) / N
    tri = np.tril_indices(T)
    var_one_pass = (float(np.sum(A * A)) - N * float(np.sum(mean * mean))) / ((N - 1) * T * T)
    assert abs(co.variance_score(A) - var_one_pass) < 1e-15
    plogp = sum(float(np.sum(A[n][tri] * np.log(A[n][tri]))) for n in range(N))
    kl_one_pass = (plogp - N * float(np.sum(mean[tri] * np.log(mean[tri])))) / (N * T)
    assert abs(co.forward_kl_score(A) - kl_one_pass) < 1e-14


def test_layer_driver_heads_and_shared_kv():
    N, H, T, D, g = 3, 4, 6, 4, 2
    rng = np.random.default_rng(7)
    Q = rng.standard_normal((N, H, T, D))
    K = rng.standard_normal((N, H // g, T, D))
    mean, s_var, s_kl = co.calibration_stats(Q, K, kv_group=g)
    for h in range(H):
        A = _brute_maps(Q[:, h], K[:, h // g], 1 / math.sqrt(D))
        assert np.max(np.abs(mean[h] - A.sum(axis=0) / N)) < 1e-14
        assert abs(s_var[h] - co.variance_score(A)) < 1e-16
        assert abs(s_kl[h] - co.forward_kl_score(A)) < 1e-15
    # a single sequence has no sample variance
    m1, v1, k1 = co.calibration_stats(Q[:1], K[:1], kv_group=g)
    assert np.all(np.isnan(v1)) and np.max(np.abs(k1)) < 1e-15
