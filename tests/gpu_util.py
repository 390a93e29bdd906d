"""Helpers for the GPU parity tests: move seeded inputs to the device, call the layer through the
C-ABI binding, bring results back as float64 numpy arrays."""
import numpy as np
import torch

import paper_2609_34650_b200 as saf
import saf_inputs as si

MAX_ABS = 2e-2      # tolerance of the layer vs the fp64 oracle: bf16 inputs, fp32 accumulation
REL_L2 = 1e-2


def bf16_tensor(bits: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(bits.view(np.int16)).view(torch.bfloat16)


def errors(got: np.ndarray, want: np.ndarray):
    """(max-abs, relative L2) with the paper's definition ||u~-u|| / max(||u||, 1e-8) (Appendix E.2)."""
    d = got.astype(np.float64) - want
    return float(np.abs(d).max()) if d.size else 0.0, float(np.linalg.norm(d) / max(np.linalg.norm(want), 1e-8))


def assert_close(got, want, what, max_abs=MAX_ABS, rel_l2=REL_L2, degenerate=False):
    """max-abs <= max_abs and ||got - want||_2 / max(||want||_2, 1e-8) <= rel_l2 (the definition of Appendix E.2).

    `degenerate` is for sequences of one or two tokens only: there dQ is exactly zero or a near-cancelling
    difference of two terms, so there is almost no norm to be relative to, and the L2 error is taken against an
    RMS of 0.1 instead (inputs are N(0,1))."""
    assert np.isfinite(got).all(), f"{what}: non-finite values"
    ma, rl = errors(got, want)
    bound = rl
    if degenerate:
        bound = float(np.linalg.norm(got - want) / max(np.linalg.norm(want), 0.1 * np.sqrt(want.size)))
    assert ma <= max_abs and bound <= rel_l2, \
        f"{what}: max-abs {ma:.3e} (<= {max_abs}), rel-L2 {rl:.3e} (<= {rel_l2}; asserted {bound:.3e})"
    return ma, rl


def bf16_half_ulp(peak: float) -> float:
    """Half a bf16 unit in the last place at magnitude `peak` (8 significant bits)."""
    return 2.0 ** (np.floor(np.log2(max(peak, 1e-30))) - 8)


class Layer:
    """One seeded workload resident on the GPU plus its outputs."""

    def __init__(self, inp: si.Inputs, grad_dtype=saf.SAF_F32, backward=True, ctx=None, softmax_scale=0.0,
                 o_f32=False):
        self.inp = inp
        wl = inp.wl
        dev = "cuda"
        self.ctx = ctx or saf.Context(0)
        self.Q, self.K, self.V, self.dO = (bf16_tensor(x).to(dev) for x in (inp.q, inp.k, inp.v, inp.do))
        self.alpha = torch.from_numpy(inp.alpha).to(dev)
        self.rho = torch.from_numpy(inp.rho).to(dev)
        self.logZ = torch.zeros_like(self.alpha)
        self.O = torch.full_like(self.dO, float("nan"), dtype=torch.float32 if o_f32 else torch.bfloat16)
        self.LSE = torch.full((wl.B, wl.H, wl.T), float("nan"), device=dev)
        gd = torch.float32 if grad_dtype == saf.SAF_F32 else torch.bfloat16
        self.grads = [torch.full(t.shape, float("nan"), device=dev, dtype=gd)
                      for t in (self.Q, self.K, self.V)] if backward else None
        self.prob = saf.make_problem(self.Q, wl.stored_len, softmax_scale=softmax_scale, grad_dtype=grad_dtype,
                                     k_like=self.K, v_like=self.V, o_like=self.O, kv_group=wl.kv_group,
                                     packed_qk=wl.packed_qk, H=wl.H,
                                     o_dtype=saf.SAF_F32 if o_f32 else saf.SAF_BF16)
        self.mask = inp.mask

    def run(self, backward=True, prepare=True):
        c = self.ctx
        if prepare:
            c.saf_pattern_prepare(self.mask, self.alpha, self.rho, self.logZ)
        c.saf_hybrid_attn_fwd(self.prob, self.Q, self.K, self.V, self.mask, self.alpha, self.rho, self.logZ,
                              self.O, self.LSE)
        if backward:
            dQ, dK, dV = self.grads
            c.saf_hybrid_attn_bwd(self.prob, self.Q, self.K, self.V, self.O, self.dO, self.LSE, self.mask,
                                  self.alpha, self.rho, self.logZ, dQ, dK, dV)
        torch.cuda.synchronize()
        code, detail = c.saf_last_device_status()
        assert code == saf.SAF_OK, f"device status {code} detail {detail:#x}"
        self.check_whole_tensors(backward)
        return self

    def check_whole_tensors(self, backward=True):
        """Properties that hold for every (b,h) unit, checked over the whole tensors (the oracle comparison only
        visits sampled units at the full sizes): every output was written (they start as NaN) and is finite;
        frozen heads have LSE 0 and exactly zero dQ / dK."""
        wl = self.inp.wl
        assert torch.isfinite(self.O).all(), "O: unwritten or non-finite entries"
        assert torch.isfinite(self.LSE).all(), "LSE: unwritten or non-finite entries"
        fz = [h for h in range(wl.H) if self.mask[h]]
        if fz:
            assert not self.LSE[:, fz].any(), "LSE slots of frozen heads must be zero"
        if not backward:
            return
        for name, g in zip(("dQ", "dK", "dV"), self.grads):
            assert torch.isfinite(g).all(), f"{name}: unwritten or non-finite entries"
        if fz and not wl.packed_qk:
            assert not self.grads[0][:, fz].any(), "dQ of frozen heads must be exactly zero"
            if wl.kv_group == 1:
                assert not self.grads[1][:, fz].any(), "dK of frozen heads must be exactly zero"

    def host(self, t):
        return t.float().cpu().numpy().astype(np.float64)


def f64(inp: si.Inputs):
    return tuple(si.bf16_bits_to_f64(x) for x in (inp.q, inp.k, inp.v, inp.do))
