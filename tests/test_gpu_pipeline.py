"""The one-time intervention end to end on the GPU (Algorithm 1, lines "measure", "fit", "install"): calibration
statistics of an all-ordinary layer -> mean attention map -> target marginals -> Fit -> kappa -> the fitted pattern
installed as a frozen head of the hybrid layer.  Every stage is checked against the oracle chain on the same inputs."""
import numpy as np
import pytest
import torch

import paper_2609_34650_b200 as saf
import saf_inputs as si
from oracle import saf_calib_oracle as co
from oracle import saf_fit_oracle as fo
from oracle import saf_oracle as orc

from gpu_util import Layer, assert_close, f64

pytestmark = pytest.mark.gpu


def test_calibrate_fit_install_and_run():
    N, H, T, D = 4, 2, 256, 64
    wl = si.Workload("pipeline", N, H, T, D, (), -0.05, seed=41)
    inp = si.generate(wl)
    L = Layer(inp, backward=False).run(backward=False)
    ctx, dev = L.ctx, "cuda"

    # 1. calibration statistics of the all-ordinary layer
    mean = torch.zeros(H, T, T, device=dev)
    sumsq = torch.zeros(H, dtype=torch.float64, device=dev)
    plogp = torch.zeros_like(sumsq)
    s_var, s_kl = torch.zeros_like(sumsq), torch.zeros_like(sumsq)
    ctx.saf_calib_accumulate(L.prob, L.Q, L.K, L.LSE, mean, sumsq, plogp, 0)
    ctx.saf_calib_finalize(H, T, N, mean, sumsq, plogp, s_var, s_kl)

    # 2. the head with the smaller variance score is the candidate (Algorithm 1 sorts by increasing score)
    q, k, v, _ = f64(inp)
    maps = [co.attention_maps(q[:, h], k[:, h]) for h in range(H)]
    want_var = np.array([co.variance_score(a) for a in maps])
    got_var = s_var.cpu().numpy()
    assert np.max(np.abs(got_var - want_var) / want_var) < 1e-3
    cand = int(np.argmin(got_var))
    assert cand == int(np.argmin(want_var))

    # 3. marginals of its mean map, Fit, kappa
    ea = torch.empty(1, T, dtype=torch.float64, device=dev)
    er = torch.empty_like(ea)
    pl = torch.empty(1, dtype=torch.float64, device=dev)
    ctx.saf_fit_marginals(1, T, mean[cand:cand + 1].contiguous(), 1e-9, ea, er, pl)
    alpha = torch.zeros(H, T, device=dev)
    rho = torch.zeros(H, T, device=dev)
    logZ_fit = torch.zeros(H, T, device=dev)
    kl = torch.empty(1, dtype=torch.float64, device=dev)
    ctx.saf_fit_compact(1, T, ea, er, pl, 400, 0.05, alpha[cand:], rho[cand:], logZ_fit[cand:], T, None, kl)
    torch.cuda.synchronize()
    code, detail = ctx.saf_last_device_status()
    assert code == saf.SAF_OK, f"device status {code} detail {detail:#x}"
    wa, wr, wz, kappa, ok = fo.fit_head(co.empirical_mean(maps[cand]), steps=400)
    a_g, r_g = alpha[cand].cpu().numpy().astype(np.float64), rho[cand].cpu().numpy().astype(np.float64)
    assert np.max(np.abs(a_g - wa)) < 2e-2 and np.max(np.abs(r_g - wr)) < 2e-2
    assert abs(kl.item() - kappa) < 2e-4
    if abs(kappa - 0.2) > 1e-3:
        assert (kl.item() <= 0.2) == ok

    # 4. install: the normalisers the attention kernels build from (alpha, rho) equal the fitter's
    mask = np.zeros(H, dtype=np.uint8)
    mask[cand] = 1
    logZ = torch.zeros(H, T, device=dev)
    ctx.saf_pattern_prepare(mask, alpha, rho, logZ)
    torch.cuda.synchronize()
    assert torch.max(torch.abs(logZ[cand] - logZ_fit[cand])).item() < 1e-4

    # 5. the layer with that head frozen, against the oracle with the GPU-fitted parameters
    O = torch.empty_like(L.O)
    LSE = torch.empty_like(L.LSE)
    ctx.saf_hybrid_attn_fwd(L.prob, L.Q, L.K, L.V, mask, alpha, rho, logZ, O, LSE)
    torch.cuda.synchronize()
    code, detail = ctx.saf_last_device_status()
    assert code == saf.SAF_OK, f"device status {code} detail {detail:#x}"
    got = O.float().cpu().numpy().astype(np.float64)
    for b in range(N):
        want, _ = orc.frozen_head_fwd(v[b, cand], a_g, r_g)
        assert_close(got[b, cand], want, f"frozen O[{b},{cand}]")
        other = 1 - cand
        want_o, _, _ = orc.ordinary_head_fwd(q[b, other], k[b, other], v[b, other], 1.0 / np.sqrt(D))
        assert_close(got[b, other], want_o, f"ordinary O[{b},{other}]")
