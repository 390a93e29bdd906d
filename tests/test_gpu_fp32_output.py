"""GPU parity with fp32 output (saf_problem.o_dtype = SAF_F32): the forward writes O unrounded, and the backward,
the pattern gradients and the row term delta_i = dO_i . O_i read that O."""
import numpy as np
import pytest
import torch

import paper_2609_34650_b200 as saf
import saf_inputs as si

from gpu_util import Layer, REL_L2
from test_gpu_parity import _check_gqa_layer, _check_packed_layer
from test_gpu_pattern_grad import _check as _check_pattern_grads

pytestmark = pytest.mark.gpu


def _is_bf16_representable(x: torch.Tensor) -> torch.Tensor:
    return x.bfloat16().float() == x


@pytest.mark.parametrize("B,H,T,D,frozen,g,packed", [
    (2, 4, 300, 64, (1, 3), 1, False),     # D = 64 kernel: both kinds of item, ragged last block
    (1, 4, 257, 64, (), 2, False),         # all ordinary, shared key/value heads
    (2, 3, 129, 64, (0, 1, 2), 1, False),  # all frozen
    (2, 4, 200, 128, (2,), 1, False),      # 128-wide kernels
    (1, 4, 160, 96, (0, 3), 1, False),     # 96-wide heads on the 128-wide kernels
    (2, 4, 140, 64, (1,), 1, True),        # packed Q/K layout
])
def test_fp32_output_forward_backward(B, H, T, D, frozen, g, packed):
    wl = si.Workload("o-f32", B, H, T, D, frozen, -0.05, seed=900 + T + D, kv_group=g, packed_qk=packed)
    L = Layer(si.generate(wl), o_f32=True).run()
    assert L.O.dtype == torch.float32
    # the output is not a widened bf16 tensor: most entries carry bits below bf16's last place
    assert _is_bf16_representable(L.O).float().mean().item() < 0.2
    (_check_packed_layer if packed else _check_gqa_layer)(L, True)


@pytest.mark.parametrize("T", [1, 2, 3, 5, 7])
def test_fp32_output_short_sequences_meet_the_stated_gradient_bound(T):
    """With the bf16 output, sequences shorter than 8 need twice the relative bound on the gradients because the
    rounding of O enters dP - delta unaveraged; with the fp32 output the stated bound holds as it is."""
    wl = si.Workload("o-f32-short", 3, 4, T, 64, (2,), -0.3, seed=950 + T)
    L = Layer(si.generate(wl), o_f32=True).run()
    _check_gqa_layer(L, True, grad_rel_l2=REL_L2)


def test_fp32_output_pattern_gradients():
    wl = si.Workload("o-f32-pg", 2, 4, 300, 64, (0, 2), -0.05, seed=960, backward=False)
    L = Layer(si.generate(wl), backward=False, o_f32=True).run(backward=False)
    _check_pattern_grads(L)


def test_fp32_output_bench_shape_agrees_with_the_bf16_run():
    """The benchmark shape with fp32 output: every entry written and finite (Layer.run checks that), the output within
    half a bf16 unit in the last place of the bf16 run's, the gradients within 5e-3 (relative L2) of it."""
    wl = si.config(1)
    inp = si.generate(wl)
    L32 = Layer(inp, o_f32=True).run()
    L16 = Layer(inp, ctx=L32.ctx).run()
    d = (L32.O - L16.O.float()).abs().max().item()
    peak = L32.O.abs().max().item()
    assert d <= 2.0 ** -8 * peak, f"fp32 and bf16 outputs differ by {d:.3e} at peak {peak:.3e}"
    for g32, g16 in zip(L32.grads, L16.grads):
        rel = (torch.linalg.vector_norm(g32 - g16) / torch.linalg.vector_norm(g16)).item()
        assert rel < 5e-3, f"gradients from the two outputs differ by {rel:.3e} (relative L2)"


def test_fp32_output_is_refused_by_the_host_buffer_entry():
    import ctypes as C
    wl = si.Workload("o-f32-host", 1, 2, 128, 64, (1,), -0.05, seed=970)
    L = Layer(si.generate(wl), o_f32=True)
    mask = np.ascontiguousarray(L.mask, dtype=np.uint8)
    rc = L.ctx._lib.saf_hybrid_attn_step_host(L.ctx._h, C.byref(L.prob), None, None, None, None,
                                              mask.ctypes.data_as(C.POINTER(C.c_uint8)), None, None, 0, None, None,
                                              None, None, None)
    assert rc == saf.SAF_ERR_UNSUPPORTED
