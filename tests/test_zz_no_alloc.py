"""The entry point that allocates nothing (collected last on purpose: a run that stops at the first
failure has then already run every other test).

saf_pattern_logz_static serves host programs that cannot let a library allocate device memory - for
instance a server that gave all GPU memory to its own pool at start-up.  It must return the same row
normalisers as saf_pattern_prepare, whose mask copy lives in context-allocated memory, and a second
call must not see anything the first one left in the built-in scratch array."""
import numpy as np
import pytest
import torch

import paper_2609_34650_b200 as saf

pytestmark = pytest.mark.gpu


def _case(seed, H, Tp, frozen):
    g = torch.Generator(device="cuda")
    g.manual_seed(seed)
    alpha = torch.randn(H, Tp, device="cuda", generator=g)
    rho = -0.03 * torch.arange(Tp, device="cuda").float()[None, :] + 0.1 * torch.randn(H, Tp, device="cuda", generator=g)
    mask = np.zeros(H, np.uint8)
    mask[list(frozen)] = 1
    return mask, alpha, rho.contiguous()


def test_static_entry_point_matches_the_allocating_one_on_two_calls_in_a_row():
    ctx = saf.Context(0)
    # two different problems back to back: more heads and another mask first, so that the second call
    # would read stale bytes if it did not overwrite what it uses
    for seed, H, Tp, frozen in ((1, 6, 700, (0, 2, 3, 5)), (2, 4, 333, (1,))):
        mask, alpha, rho = _case(seed, H, Tp, frozen)
        want = torch.full((H, Tp), float("nan"), device="cuda")
        got = torch.full((H, Tp), float("nan"), device="cuda")
        ctx.saf_pattern_prepare(mask, alpha, rho, want)
        saf.saf_pattern_logz_static(0, mask, alpha, rho, got)
        torch.cuda.synchronize()
        for h in range(H):
            if mask[h]:
                assert torch.isfinite(got[h]).all()
                assert (got[h] - want[h]).abs().max().item() <= 5e-6     # same tolerance as the logZ parity test
            else:
                assert torch.isnan(got[h]).all()                         # rows of ordinary heads are not written


def test_static_entry_point_rejects_more_heads_than_its_scratch_holds():
    H, Tp = 1025, 8
    alpha = torch.zeros(H, Tp, device="cuda")
    out = torch.zeros(H, Tp, device="cuda")
    mask = np.ones(H, np.uint8)
    with pytest.raises(saf.SafError) as e:
        saf.saf_pattern_logz_static(0, mask, alpha, alpha, out)
    assert e.value.code == 1
