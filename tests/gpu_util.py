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


def assert_close(got, want, what, max_abs=MAX_ABS, rel_l2=REL_L2):
    assert np.isfinite(got).all(), f"{what}: non-finite values"
    ma, rl = errors(got, want)
    # Degenerate references (T = 1 or 2: dQ is exactly zero, or a near-cancelling difference of two
    # terms) have almost no norm to be relative to: the L2 error is then taken against an RMS of 0.1
    # (inputs are N(0,1); every non-degenerate output has a larger RMS).
    floor = 0.1 * np.sqrt(want.size)
    rl_floored = float(np.linalg.norm(got - want) / max(np.linalg.norm(want), floor))
    assert ma <= max_abs and rl_floored <= rel_l2, \
        f"{what}: max-abs {ma:.3e} (<= {max_abs}), rel-L2 {rl:.3e} / floored {rl_floored:.3e} (<= {rel_l2})"
    return ma, rl


class Layer:
    """One seeded workload resident on the GPU plus its outputs."""

    def __init__(self, inp: si.Inputs, grad_dtype=saf.SAF_F32, backward=True, ctx=None, softmax_scale=0.0):
        self.inp = inp
        wl = inp.wl
        dev = "cuda"
        self.ctx = ctx or saf.Context(0)
        self.Q, self.K, self.V, self.dO = (bf16_tensor(x).to(dev) for x in (inp.q, inp.k, inp.v, inp.do))
        self.alpha = torch.from_numpy(inp.alpha).to(dev)
        self.rho = torch.from_numpy(inp.rho).to(dev)
        self.logZ = torch.zeros_like(self.alpha)
        self.O = torch.full_like(self.dO, float("nan"))
        self.LSE = torch.full((wl.B, wl.H, wl.T), float("nan"), device=dev)
        gd = torch.float32 if grad_dtype == saf.SAF_F32 else torch.bfloat16
        self.grads = [torch.full(t.shape, float("nan"), device=dev, dtype=gd)
                      for t in (self.Q, self.K, self.V)] if backward else None
        self.prob = saf.make_problem(self.Q, wl.stored_len, softmax_scale=softmax_scale, grad_dtype=grad_dtype,
                                     k_like=self.K, v_like=self.V, o_like=self.O, kv_group=wl.kv_group,
                                     packed_qk=wl.packed_qk, H=wl.H)
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
        return self

    def host(self, t):
        return t.float().cpu().numpy().astype(np.float64)


def f64(inp: si.Inputs):
    return tuple(si.bf16_bits_to_f64(x) for x in (inp.q, inp.k, inp.v, inp.do))
