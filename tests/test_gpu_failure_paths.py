"""GPU tests of the paths that only run when something is off: a bounded device wait that runs out, and pattern
tables that no longer describe the vectors a call passes."""
import numpy as np
import pytest
import torch

import paper_2609_34650_b200 as saf
import saf_inputs as si

from gpu_util import Layer
from test_gpu_parity import check_units, all_units

pytestmark = pytest.mark.gpu

DEV_TIMEOUT = 1                       # device status code in bits 24..31 of the status word
SITE_K_FULL, SITE_S_FULL = 45, 49     # wait sites of the D = 64 forward: issuer waiting for a key tile, compute
                                      # warps waiting for the scores of that tile


def test_a_wait_that_runs_out_is_reported_and_the_context_stays_usable(monkeypatch):
    """The producer of one tiny forward grid leaves out one key-tile load (a host-side switch, off by default), so the
    waits that depend on it reach their limit (20 ms here).  Every role must leave through the common teardown: the
    kernel ends, the status word names a wait site of that tile, and later calls work."""
    monkeypatch.setenv("SAF_WAIT_LIMIT_MS", "20")
    monkeypatch.setenv("SAF_SELFTEST_DROP_LOAD", "1")
    ctx = saf.Context(0)
    monkeypatch.delenv("SAF_SELFTEST_DROP_LOAD")
    monkeypatch.delenv("SAF_WAIT_LIMIT_MS")
    inp = si.generate(si.config(0))
    L = Layer(inp, ctx=ctx, backward=False)
    ctx.saf_pattern_prepare(L.mask, L.alpha, L.rho, L.logZ)
    ctx.saf_hybrid_attn_fwd(L.prob, L.Q, L.K, L.V, L.mask, L.alpha, L.rho, L.logZ, L.O, L.LSE)
    torch.cuda.synchronize()
    code, detail = ctx.saf_last_device_status()
    assert code == saf.SAF_ERR_DEVICE_TIMEOUT, (code, hex(detail))
    assert (detail >> 24) & 0xFF == DEV_TIMEOUT
    assert (detail >> 16) & 0xFF in (SITE_K_FULL, SITE_S_FULL), hex(detail)
    assert (detail & 0xFFFF) < 8                       # a CTA of the 8-item grid
    # the word was cleared by the query, and the device is fine: a context without the switch passes the same case
    code, detail = ctx.saf_last_device_status()
    assert code == saf.SAF_OK and detail == 0
    fresh = Layer(inp).run()
    check_units(fresh, all_units(inp.wl))


def test_vectors_rewritten_in_place_do_not_meet_stale_tables():
    """saf_pattern_prepare builds tensor-core tables and remembers the device pointers.  When alpha is then changed in
    place and only the normalisers are refreshed (by the entry point that has no context), the next layer call gets the
    same three pointers: it must compute the frozen heads from the new vectors, not from the old tables."""
    wl = si.Workload("stale", 2, 4, 300, 64, (1, 2), -0.05, seed=77)
    inp = si.generate(wl)
    L = Layer(inp).run()
    check_units(L, all_units(wl))
    new_alpha = (0.5 * inp.alpha + 0.3 * np.cos(0.11 * np.arange(inp.alpha.shape[1]))[None, :]).astype(np.float32)
    L.alpha.copy_(torch.from_numpy(new_alpha))          # same buffer, new contents
    saf.saf_pattern_logz_static(0, L.mask, L.alpha, L.rho, L.logZ)
    inp.alpha[...] = new_alpha
    for t in (L.O, L.LSE, *L.grads):
        t.fill_(float("nan"))
    L.run(prepare=False)
    check_units(L, all_units(wl))
    # after a new preparation the tables are used again and agree as well
    L.run(prepare=True)
    check_units(L, all_units(wl))
