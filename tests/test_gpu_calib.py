"""GPU parity of the calibration statistics (empirical mean attention, variance score, forward-KL score) against the
dense fp64 oracle.

Tolerances.  A probability is exp2(s c - lse') with s the fp32 tensor-core score of bf16 inputs (exact products, fp32
sums: about 1e-6 relative of |s| ~ 10, i.e. 1e-5 absolute in the exponent), lse' from the forward kernel (fp32) and
ex2.approx (2^-22): about 2e-5 relative per entry, asserted as |got - want| <= 1e-6 + 2e-4 want for the mean.  The
scores are differences of two nearly equal fp64 sums of such terms; with synthetic inputs the difference is a
sizeable fraction of the sums, and 1e-3 relative is asserted.  The forward-KL score also carries an absolute error
of about 1e-6 nats per row: p log p is summed as p s c minus the row normaliser, which assumes that the fp32
probabilities of a row sum to one (they do to about 1e-6), so 2e-6 absolute is allowed on top (it shows only when the
score itself is zero: a single sequence, or identical ones)."""
import numpy as np
import pytest
import torch

import paper_2609_34650_b200 as saf
import saf_inputs as si
from oracle import saf_calib_oracle as co

from gpu_util import Layer, f64

pytestmark = pytest.mark.gpu

SENTINEL = 7.0


def _workload(N, H, T, D, g=1, seed=0):
    return si.Workload(f"calib-{N}x{H}x{T}x{D}", N, H, T, D, (), -0.05, seed=seed, kv_group=g)


def _run(L, splits=1, sentinel=True):
    """Forward for the normalisers, then the statistics in `splits` calls over the sequences."""
    wl = L.inp.wl
    L.run(backward=False)
    ctx, dev = L.ctx, "cuda"
    mean = torch.full((wl.H, wl.T, wl.T), SENTINEL if sentinel else 0.0, device=dev)
    sumsq = torch.full((wl.H,), float("nan"), dtype=torch.float64, device=dev)
    plogp = torch.full((wl.H,), float("nan"), dtype=torch.float64, device=dev)
    bounds = np.linspace(0, wl.B, splits + 1).astype(int)
    for k in range(splits):
        lo, hi = int(bounds[k]), int(bounds[k + 1])
        Q, K, LSE = L.Q[lo:hi], L.K[lo:hi], L.LSE[lo:hi].contiguous()
        prob = saf.make_problem(Q, wl.T, k_like=K, v_like=L.V[lo:hi], o_like=L.O[lo:hi], kv_group=wl.kv_group, H=wl.H)
        ctx.saf_calib_accumulate(prob, Q, K, LSE, mean, sumsq, plogp, k > 0)
    s_var = torch.full((wl.H,), float("nan"), dtype=torch.float64, device=dev)
    s_kl = torch.full((wl.H,), float("nan"), dtype=torch.float64, device=dev)
    ctx.saf_calib_finalize(wl.H, wl.T, wl.B, mean, sumsq, plogp, s_var if wl.B > 1 else None, s_kl)
    torch.cuda.synchronize()
    code, detail = ctx.saf_last_device_status()
    assert code == saf.SAF_OK, f"device status {code} detail {detail:#x}"
    return mean.cpu().numpy().astype(np.float64), s_var.cpu().numpy(), s_kl.cpu().numpy()


def _check(L, mean, s_var, s_kl, heads=None):
    wl = L.inp.wl
    q, k, _, _ = f64(L.inp)
    T = wl.T
    tri = np.tril(np.ones((T, T), dtype=bool))
    for h in (heads if heads is not None else range(wl.H)):
        A = co.attention_maps(q[:, h], k[:, h // wl.kv_group])
        want = co.empirical_mean(A)
        got = mean[h]
        assert np.isfinite(got[tri]).all()
        err = np.abs(got - want)[tri]
        assert np.all(err <= 1e-6 + 2e-4 * want[tri]), f"mean head {h}: max err {err.max():.3e}"
        # inside the tiles that meet the triangle the part above the diagonal is zero; tiles above it are untouched
        blk = np.arange(T) // 128
        above = ~tri
        same_or_lower_tile = blk[None, :] <= blk[:, None]
        assert np.all(got[above & same_or_lower_tile] == 0.0)
        assert np.all(got[above & ~same_or_lower_tile] == SENTINEL)
        if wl.B > 1:
            wv = co.variance_score(A)
            assert abs(s_var[h] - wv) <= 1e-3 * wv + 1e-12, f"s_var head {h}: {s_var[h]} vs {wv}"
        wk = co.forward_kl_score(A)
        assert abs(s_kl[h] - wk) <= 1e-3 * wk + 2e-6, f"s_kl head {h}: {s_kl[h]} vs {wk}"


@pytest.mark.parametrize("N,H,T,D,g", [(3, 2, 300, 64, 1), (4, 2, 129, 128, 1), (2, 2, 200, 96, 1), (3, 4, 257, 64, 2),
                                       (2, 1, 1, 64, 1), (5, 1, 128, 64, 1), (2, 3, 516, 64, 1)])
def test_calibration_statistics_parity(N, H, T, D, g):
    L = Layer(si.generate(_workload(N, H, T, D, g, seed=N + T)), backward=False)
    _check(L, *_run(L))


@pytest.mark.parametrize("T,D,g", [(260, 64, 1), (257, 64, 1), (260, 128, 2), (131, 96, 1)])
def test_streaming_in_several_calls_equals_one_call(T, D, g):
    """Adding calls (old tile fetched and summed) against a single call; T = 257 and 131 take the path without TMA."""
    wl = _workload(6, 2, T, D, g, seed=3)
    L = Layer(si.generate(wl), backward=False)
    m1, v1, k1 = _run(L, splits=1)
    m3, v3, k3 = _run(L, splits=3)
    tri = np.tril(np.ones((wl.T, wl.T), dtype=bool))
    assert np.max(np.abs(m1 - m3)[:, tri]) < 1e-6
    assert np.max(np.abs(v1 - v3) / v1) < 1e-5 and np.max(np.abs(k1 - k3) / k1) < 1e-5
    _check(L, m3, v3, k3)


def test_single_sequence_has_zero_kl_and_mean_equals_its_map():
    L = Layer(si.generate(_workload(1, 2, 200, 64, seed=5)), backward=False)
    mean, s_var, s_kl = _run(L)
    assert np.all(np.abs(s_kl) < 1e-6)
    _check(L, mean, s_var, s_kl)


def test_identical_sequences_score_zero():
    wl = _workload(1, 2, 300, 64, seed=8)
    inp = si.generate(wl)
    wl4 = _workload(4, 2, 300, 64, seed=8)
    rep = si.Inputs(wl4, np.repeat(inp.q, 4, axis=0), np.repeat(inp.k, 4, axis=0), np.repeat(inp.v, 4, axis=0),
                    np.repeat(inp.do, 4, axis=0), inp.alpha, inp.rho, inp.mask)
    L = Layer(rep, backward=False)
    mean, s_var, s_kl = _run(L)
    # the one-pass differences cancel to rounding level: far below the scores of distinct sequences (~1e-4 .. 1e-1)
    assert np.all(s_var < 1e-9) and np.all(s_kl < 1e-5)


def test_config1_full_size_sampled_head():
    """The benchmark's shape (8 sequences, 12 heads, T = 4096, D = 64): one head against the oracle on sampled rows,
    its two scores in full, and row sums of the mean for every head."""
    wl = _workload(8, 12, 4096, 64, seed=11)
    L = Layer(si.generate(wl), backward=False)
    mean, s_var, s_kl = _run(L, sentinel=False)
    T = wl.T
    rows = mean.sum(axis=2)                       # zeros above the diagonal: each row of A^ sums to one
    assert np.max(np.abs(rows - 1.0)) < 2e-4
    q, k, _, _ = f64(L.inp)
    h = 5
    A = co.attention_maps(q[:, h], k[:, h])
    want = co.empirical_mean(A)
    for i in (0, 1, 127, 128, 129, 1000, 2047, 2048, 4095):
        err = np.abs(mean[h, i, : i + 1] - want[i, : i + 1])
        assert np.all(err <= 1e-6 + 2e-4 * want[i, : i + 1])
    wv, wk = co.variance_score(A), co.forward_kl_score(A)
    assert abs(s_var[h] - wv) <= 1e-3 * wv and abs(s_kl[h] - wk) <= 1e-3 * wk


def test_invalid_arguments():
    L = Layer(si.generate(_workload(2, 2, 64, 64)), backward=False)
    L.run(backward=False)
    ctx = L.ctx
    mean = torch.zeros(2, 64, 64, device="cuda")
    d = torch.zeros(2, dtype=torch.float64, device="cuda")
    for call in (lambda: ctx.saf_calib_accumulate(L.prob, None, L.K, L.LSE, mean, d, d, 0),
                 lambda: ctx.saf_calib_accumulate(L.prob, L.Q, L.K, None, mean, d, d, 0),
                 lambda: ctx.saf_calib_accumulate(L.prob, L.Q, L.K, L.LSE, None, d, d, 0),
                 lambda: ctx.saf_calib_finalize(2, 64, 0, mean, d, d, d, d),
                 lambda: ctx.saf_calib_finalize(2, 64, 1, mean, d, d, d, d)):
        with pytest.raises(saf.SafError) as e:
            call()
        assert e.value.code == saf.SAF_ERR_INVALID_ARG
