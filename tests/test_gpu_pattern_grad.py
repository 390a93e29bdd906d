"""GPU parity of the pattern gradients (dalpha, drho of the frozen heads) against the dense fp64 oracle."""
import numpy as np
import pytest
import torch

import paper_2609_34650_b200 as saf
import saf_inputs as si
from oracle import saf_oracle as orc

from gpu_util import Layer, f64, REL_L2

pytestmark = pytest.mark.gpu


def _pattern_grads(L):
    wl = L.inp.wl
    da = torch.full_like(L.alpha, float("nan"))
    dr = torch.full_like(L.alpha, float("nan"))
    L.ctx.saf_pattern_grad(L.prob, L.V, L.O, L.dO, L.mask, L.alpha, L.rho, L.logZ, da, dr)
    torch.cuda.synchronize()
    code, detail = L.ctx.saf_last_device_status()
    assert code == saf.SAF_OK, f"device status {code} detail {detail:#x}"
    return da.cpu().numpy().astype(np.float64), dr.cpu().numpy().astype(np.float64)


def _check(L):
    """dalpha / drho are sums of up to B*T products: the bound is relative (L2 1e-2 per head and vector, and a
    max-abs bound of 2e-2 of the vector's largest entry), exact zeros where the definition has none."""
    inp, wl = L.inp, L.inp.wl
    _, _, v, do = f64(inp)
    # the kernel's delta uses the bf16 O of the forward; the oracle's own O is exact: part of the tolerance
    eda, edr = orc.pattern_grads(v, do, inp.mask, inp.alpha.astype(np.float64), inp.rho.astype(np.float64))
    da, dr = _pattern_grads(L)
    assert np.isfinite(da).all() and np.isfinite(dr).all()
    for h in range(wl.H):
        if not inp.mask[h]:
            assert not da[h].any() and not dr[h].any(), "rows of ordinary heads must be zero"
            continue
        assert not da[h, wl.T:].any() and not dr[h, wl.T:].any(), "entries beyond T must be zero"
        for name, g, e in (("dalpha", da[h], eda[h]), ("drho", dr[h], edr[h])):
            rl = np.linalg.norm(g - e) / max(np.linalg.norm(e), 1e-8)
            ma = np.abs(g - e).max() / max(np.abs(e).max(), 1e-8)
            assert rl <= REL_L2 and ma <= 2e-2, f"{name}[{h}]: rel-L2 {rl:.3e}, max-abs/peak {ma:.3e}"


@pytest.mark.parametrize("T,Tp,frozen", [(256, 256, (1,)), (129, 192, (1, 3)), (300, 300, (0, 1, 2, 3)), (1, 8, (2,)),
                                         (127, 127, (0,))])
def test_pattern_grads_small(T, Tp, frozen):
    wl = si.Workload("pg", 2, 4, T, 64, frozen, -0.05, Tp=Tp, seed=70 + T)
    L = Layer(si.generate(wl), backward=False).run(backward=False)
    _check(L)


def test_pattern_grads_no_frozen_heads_gives_zeros():
    wl = si.Workload("pg0", 1, 2, 128, 64, (), -0.05, seed=71)
    L = Layer(si.generate(wl), backward=False).run(backward=False)
    da, dr = _pattern_grads(L)
    assert not da.any() and not dr.any()


def test_pattern_grads_head_dim_128_and_shared_value_heads():
    wl = si.Workload("pg128", 2, 8, 384, 128, (2, 3, 4), -0.02, seed=72, kv_group=4, backward=False)
    L = Layer(si.generate(wl), backward=False).run(backward=False)
    _check(L)


def test_pattern_grads_head_dim_96():
    wl = si.Workload("pg96", 2, 4, 300, 96, (0, 3), -0.03, seed=74, backward=False)
    L = Layer(si.generate(wl), backward=False).run(backward=False)
    _check(L)


@pytest.mark.parametrize("B,D", [(9, 64), (19, 64), (5, 128), (6, 96)])
def test_pattern_grads_batch_larger_than_the_resident_chunk(B, D):
    """The batch sum runs inside the contraction over at most 8 (D = 64) or 4 (wider heads) entries whose V tiles stay
    in shared memory; larger batches are cut into several such runs, the last one shorter."""
    wl = si.Workload("pgB", B, 2, 333, D, (1,), -0.02, seed=75 + B, backward=False)
    L = Layer(si.generate(wl), backward=False).run(backward=False)
    _check(L)


def test_pattern_grads_many_items_per_cta():
    """6 frozen heads x 9 key blocks with up to 9 query blocks each on 148 CTAs, ragged last block."""
    wl = si.Workload("pgmix", 8, 8, 1100, 64, (0, 2, 3, 5, 6, 7), -0.01, seed=73)
    L = Layer(si.generate(wl), backward=False).run(backward=False)
    _check(L)


def test_pattern_grads_config1_full_size_one_head():
    """The benchmark shape (8 x 12 x 4096 x 64, 3 frozen heads): one frozen head against the dense oracle."""
    wl = si.config(1)
    inp = si.generate(wl)
    L = Layer(inp, backward=False).run(backward=False)
    da, dr = _pattern_grads(L)
    _, _, v, do = f64(inp)
    h = wl.frozen_heads[1]
    eda, edr = np.zeros(wl.T), np.zeros(wl.T)
    for b in range(wl.B):
        a, r = orc.pattern_grads_head(v[b, h], do[b, h], inp.alpha[h].astype(np.float64), inp.rho[h].astype(np.float64))
        eda += a
        edr += r
    for name, g, e in (("dalpha", da[h, :wl.T], eda), ("drho", dr[h, :wl.T], edr)):
        rl = np.linalg.norm(g - e) / max(np.linalg.norm(e), 1e-8)
        ma = np.abs(g - e).max() / max(np.abs(e).max(), 1e-8)
        assert rl <= REL_L2 and ma <= 2e-2, f"{name}[{h}]: rel-L2 {rl:.3e}, max-abs/peak {ma:.3e}"
