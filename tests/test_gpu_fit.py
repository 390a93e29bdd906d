"""GPU parity of the compact-pattern fitter (target marginals, Fit, acceptance statistic) against the fp64 oracle.

Tolerances.  The kernels take the exponentials in fp32 (ex2.approx: relative error about 2^-22 on top of an argument
rounded at magnitudes up to ~60, i.e. a few 1e-6 relative per term) and accumulate what feeds Adam, and Adam itself,
in fp64.  Marginals and normalisers are sums of positive terms, so they inherit that relative error: 2e-5 relative is
asserted.  Over the Adam steps the difference in the gradients (about 1e-6 relative) moves the parameters by far less
than one step (0.05) each time; the asserted bound on alpha, rho after J steps is 2e-3 absolute for J <= 50 and
2e-2 after 400 steps, with the quantities that do not depend on the path (loss, kappa: 1e-4 absolute) held tighter,
and the returned log Z, loss and kappa checked against the oracle evaluated AT the returned parameters (1e-4)."""
import numpy as np
import pytest
import torch

import paper_2609_34650_b200 as saf
import saf_inputs as si
from oracle import saf_fit_oracle as fo

pytestmark = pytest.mark.gpu


def _ctx():
    return saf.Context(0)


def _status(ctx):
    torch.cuda.synchronize()
    code, detail = ctx.saf_last_device_status()
    assert code == saf.SAF_OK, f"device status {code} detail {detail:#x}"


def _gpu_marginals(ctx, A):
    Hf, T, _ = A.shape
    dA = torch.from_numpy(A).cuda()
    ea = torch.full((Hf, T), float("nan"), dtype=torch.float64, device="cuda")
    er = torch.full((Hf, T), float("nan"), dtype=torch.float64, device="cuda")
    pl = torch.full((Hf,), float("nan"), dtype=torch.float64, device="cuda")
    ctx.saf_fit_marginals(Hf, T, dA, 1e-9, ea, er, pl)
    _status(ctx)
    return ea, er, pl


def _gpu_fit(ctx, ea, er, pl, steps, lr=0.05, stride=None):
    Hf, T = ea.shape
    stride = stride or T
    out = [torch.full((Hf, stride), float("nan"), dtype=torch.float32, device="cuda") for _ in range(3)]
    loss = torch.full((Hf,), float("nan"), dtype=torch.float64, device="cuda")
    kl = torch.full((Hf,), float("nan"), dtype=torch.float64, device="cuda")
    ctx.saf_fit_compact(Hf, T, ea, er, pl, steps, lr, out[0], out[1], out[2], stride, loss, kl)
    _status(ctx)
    a, r, z = (t.cpu().numpy().astype(np.float64) for t in out)
    return a, r, z, loss.cpu().numpy(), kl.cpu().numpy()


def _oracle_stats(A):
    P = [fo.target_from_mean_attention(A[h]) for h in range(A.shape[0])]
    st = [fo.marginals(p) for p in P]
    ea = np.stack([s[0] for s in st])
    er = np.stack([s[1] for s in st])
    pl = np.array([s[2] for s in st])
    return P, ea, er, pl


def _dev(x):
    return torch.from_numpy(np.ascontiguousarray(x, dtype=np.float64)).cuda()


# ------------------------------------------------------------------------------------------------ marginals
@pytest.mark.parametrize("Hf,T,seed", [(2, 300, 1), (3, 1100, 2), (1, 2500, 3), (1, 1, 4), (2, 33, 5),
                                       (1, 5000, 6), (1, 8200, 7)])       # (the last two: 32 columns per thread)
def test_marginals_parity(Hf, T, seed):
    # garbage above the diagonal must be ignored; a steep decay puts entries under the 1e-9 floor
    A = si.mean_attention_maps(Hf, T, seed, upper_fill=7.0, pmax=5.0)
    if T == 1100:
        tri = np.tril_indices(T)
        assert any((A[h][tri] < 1e-9).any() for h in range(Hf)), "the case should exercise the floor"
    P, ea, er, pl = _oracle_stats(A)
    g_ea, g_er, g_pl = (t.cpu().numpy() for t in _gpu_marginals(_ctx(), A))
    assert np.isfinite(g_ea).all() and np.isfinite(g_er).all() and np.isfinite(g_pl).all()
    assert np.max(np.abs(g_ea - ea) / ea) < 2e-5
    assert np.max(np.abs(g_er - er) / er) < 2e-5
    assert np.max(np.abs(g_pl - pl)) < 2e-5 * T + 1e-9
    # each marginal distributes the T units of row mass
    assert np.max(np.abs(g_ea.sum(axis=1) - T)) < 2e-5 * T


def test_marginals_many_heads_one_cta_each():
    # more heads than three CTAs per SM: one CTA per head walks every row
    Hf, T = 500, 64
    base = si.mean_attention_maps(4, T, 9)
    A = np.ascontiguousarray(base[np.arange(Hf) % 4])
    _, ea, er, pl = _oracle_stats(base)
    g_ea, g_er, g_pl = (t.cpu().numpy() for t in _gpu_marginals(_ctx(), A))
    for h in (0, 1, 250, 499):
        assert np.max(np.abs(g_ea[h] - ea[h % 4]) / ea[h % 4]) < 2e-5
        assert np.max(np.abs(g_er[h] - er[h % 4]) / er[h % 4]) < 2e-5
        assert abs(g_pl[h] - pl[h % 4]) < 2e-5 * T


# ------------------------------------------------------------------------------------------------ Fit
def _check_self_consistent(a, r, z, loss, kl, P, ea, er, pl, tol=1e-4):
    """Returned log Z, loss and kappa against the oracle evaluated at the RETURNED parameters."""
    for h in range(a.shape[0]):
        T = ea.shape[1]
        want_z, _ = fo._logZ_and_P(a[h, :T], r[h, :T])
        assert np.max(np.abs(z[h, :T] - want_z)) < tol
        assert abs(loss[h] - fo.fit_objective(a[h, :T], r[h, :T], ea[h], er[h])) < tol
        assert abs(kl[h] - fo.fit_kl_dense(P[h], a[h, :T], r[h, :T])) < tol


@pytest.mark.parametrize("T,steps,tol", [(300, 0, 1e-6), (300, 1, 1e-4), (300, 5, 5e-4), (517, 50, 2e-3), (96, 400, 2e-2),
                                         (1, 3, 1e-6), (2, 10, 1e-4), (33, 20, 1e-3)])
def test_fit_parity(T, steps, tol):
    Hf = 2
    A = si.mean_attention_maps(Hf, T, 11 + T)
    P, ea, er, pl = _oracle_stats(A)
    a, r, z, loss, kl = _gpu_fit(_ctx(), _dev(ea), _dev(er), _dev(pl), steps)
    assert all(np.isfinite(x).all() for x in (a, r, z, loss, kl))
    for h in range(Hf):
        wa, wr, wz = fo.fit_compact(ea[h], er[h], steps=steps, lr=0.05)
        assert np.max(np.abs(a[h] - wa)) < tol, f"alpha head {h}: {np.max(np.abs(a[h] - wa)):.3e}"
        assert np.max(np.abs(r[h] - wr)) < tol, f"rho head {h}: {np.max(np.abs(r[h] - wr)):.3e}"
        assert np.max(np.abs(z[h] - wz)) < max(2 * tol, 1e-5)
        assert abs(loss[h] - fo.fit_objective(wa, wr, ea[h], er[h])) < 1e-4
        assert abs(kl[h] - fo.fit_kl_dense(P[h], wa, wr)) < 1e-4
    _check_self_consistent(a, r, z, loss, kl, P, ea, er, pl)


def test_fit_long_sequence_two_steps():
    """T beyond 4096: the pass kernels stage more than 48 KB of operands per CTA."""
    T = 5000
    A = si.mean_attention_maps(1, T, 31)
    P, ea, er, pl = _oracle_stats(A)
    a, r, z, loss, kl = _gpu_fit(_ctx(), _dev(ea), _dev(er), _dev(pl), 2)
    wa, wr, wz = fo.fit_compact(ea[0], er[0], steps=2)
    assert np.max(np.abs(a[0] - wa)) < 2e-4 and np.max(np.abs(r[0] - wr)) < 2e-4 and np.max(np.abs(z[0] - wz)) < 1e-4
    assert abs(kl[0] - fo.fit_kl_dense(P[0], wa, wr)) < 1e-4


def test_fit_start_is_prescribed_point():
    T = 130
    A = si.mean_attention_maps(1, T, 3)
    P, ea, er, pl = _oracle_stats(A)
    a, r, z, loss, kl = _gpu_fit(_ctx(), _dev(ea), _dev(er), _dev(pl), 0)
    assert np.all(a == 0)
    want = np.log(np.maximum(er[0] / (T - np.arange(T)), 1e-9))
    assert np.max(np.abs(r[0] - want)) < 1e-6 * np.max(np.abs(want))


def test_fit_output_stride_and_untouched_padding():
    T, stride = 100, 160
    A = si.mean_attention_maps(2, T, 5)
    P, ea, er, pl = _oracle_stats(A)
    a, r, z, loss, kl = _gpu_fit(_ctx(), _dev(ea), _dev(er), _dev(pl), 3, stride=stride)
    assert np.isfinite(a[:, :T]).all() and np.isnan(a[:, T:]).all() and np.isnan(z[:, T:]).all()
    for h in range(2):
        wa, wr, wz = fo.fit_compact(ea[h], er[h], steps=3)
        assert np.max(np.abs(a[h, :T] - wa)) < 5e-4 and np.max(np.abs(r[h, :T] - wr)) < 5e-4


def test_fit_end_to_end_with_acceptance():
    """Mean attention map -> marginals -> Fit -> kappa, all on the GPU, against Algorithm 1's loop body."""
    Hf, T = 3, 200
    A = si.mean_attention_maps(Hf, T, 17)
    ctx = _ctx()
    ea, er, pl = _gpu_marginals(ctx, A)
    a, r, z, loss, kl = _gpu_fit(ctx, ea, er, pl, 400)
    for h in range(Hf):
        wa, wr, wz, kappa, ok = fo.fit_head(A[h], steps=400)
        assert abs(kl[h] - kappa) < 1e-4
        if abs(kappa - 0.2) > 1e-3:
            assert (kl[h] <= 0.2) == ok
        assert np.max(np.abs(a[h] - wa)) < 2e-2 and np.max(np.abs(r[h] - wr)) < 2e-2
        # the reconstructed pattern is what matters downstream: rows of P^ from the two parameter sets
        _, Pg = fo._logZ_and_P(a[h], r[h])
        _, Pw = fo._logZ_and_P(wa, wr)
        assert np.max(np.abs(Pg - Pw)) < 2e-3


def test_fit_planted_pattern_recovered():
    # a target that is itself a compact pattern: kappa must come out near zero and far below its starting value
    T = 256
    rng = np.random.default_rng(4)
    alpha = 0.5 * rng.standard_normal(T)
    alpha[0] += 3.0
    rho = -0.05 * np.arange(T) + 0.1 * rng.standard_normal(T)
    _, P = fo._logZ_and_P(alpha, rho)
    ea, er, pl = fo.marginals(P)
    ctx = _ctx()
    args = (_dev(ea[None]), _dev(er[None]), _dev(np.array([pl])))
    _, _, _, _, kl0 = _gpu_fit(ctx, *args, 0)
    a, r, z, loss, kl = _gpu_fit(ctx, *args, 400)
    assert 0 <= kl[0] + 1e-6 and kl[0] < 0.02 and kl[0] < 0.1 * kl0[0]
    assert abs(kl[0] - fo.fit_kl_dense(P, a[0], r[0])) < 1e-4


def test_fit_full_size_config1_heads():
    """The benchmark's shape (T = 4096, three heads): a few steps element-wise, then 400 steps checked through
    what holds at any size (the returned normalisers, loss and kappa belong to the returned parameters)."""
    Hf, T = 3, 4096
    A = si.mean_attention_maps(1, T, 23)
    A = np.ascontiguousarray(np.repeat(A, Hf, axis=0))
    A[1] = np.tril(A[1] ** 1.3)
    A[2] = np.tril(A[2] ** 0.7)
    ctx = _ctx()
    ea, er, pl = _gpu_marginals(ctx, A)
    P0 = fo.target_from_mean_attention(A[1])
    wea, wer, wpl = fo.marginals(P0)
    g_ea, g_er = ea.cpu().numpy(), er.cpu().numpy()
    assert np.max(np.abs(g_ea[1] - wea) / wea) < 2e-5 and np.max(np.abs(g_er[1] - wer) / wer) < 2e-5
    assert abs(pl.cpu().numpy()[1] - wpl) < 2e-5 * T
    a, r, z, loss, kl = _gpu_fit(ctx, ea, er, pl, 2)
    wa, wr, wz = fo.fit_compact(wea, wer, steps=2)
    assert np.max(np.abs(a[1] - wa)) < 2e-4 and np.max(np.abs(r[1] - wr)) < 2e-4 and np.max(np.abs(z[1] - wz)) < 1e-4
    a, r, z, loss, kl = _gpu_fit(ctx, ea, er, pl, 400)
    want_z, _ = fo._logZ_and_P(a[1], r[1])
    assert np.max(np.abs(z[1] - want_z)) < 1e-4
    assert abs(loss[1] - fo.fit_objective(a[1], r[1], wea, wer)) < 1e-4
    assert abs(kl[1] - fo.fit_kl_dense(P0, a[1], r[1])) < 1e-4
    start = fo.fit_kl_from_stats(*fo.fit_init(wer), wea, wer, wpl)
    assert kl[1] < start


# ------------------------------------------------------------------------------------------------ edges
def test_fit_no_heads_and_bad_arguments():
    ctx = _ctx()
    z = torch.zeros(4, dtype=torch.float64, device="cuda")
    f = torch.zeros(4, dtype=torch.float32, device="cuda")
    ctx.saf_fit_marginals(0, 4, None, 1e-9, z, z, z)          # no heads: nothing to do
    ctx.saf_fit_compact(0, 4, z, z, z, 5, 0.05, f, f, f, 4, None, None)
    for call in (lambda: ctx.saf_fit_marginals(1, 0, f, 1e-9, z, z, z),
                 lambda: ctx.saf_fit_marginals(1, 4, f, 0.0, z, z, z),
                 lambda: ctx.saf_fit_marginals(1, 4, None, 1e-9, z, z, z),
                 lambda: ctx.saf_fit_compact(1, 4, z, z, z, -1, 0.05, f, f, f, 4, None, None),
                 lambda: ctx.saf_fit_compact(1, 4, z, z, z, 1, 0.0, f, f, f, 4, None, None),
                 lambda: ctx.saf_fit_compact(1, 4, z, z, z, 1, 0.05, f, f, f, 3, None, None),
                 lambda: ctx.saf_fit_compact(1, 4, z, z, None, 1, 0.05, f, f, f, 4, None, z)):
        with pytest.raises(saf.SafError) as e:
            call()
        assert e.value.code == saf.SAF_ERR_INVALID_ARG
    with pytest.raises(saf.SafError) as e:
        ctx.saf_fit_compact(1, 16385, z, z, z, 1, 0.05, f, f, f, 16385, None, None)
    assert e.value.code == saf.SAF_ERR_UNSUPPORTED
    _status(ctx)
