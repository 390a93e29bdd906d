"""GPU parity: the CUDA path, called through the C-ABI binding, against the fp64 oracle on the same
seeded inputs.  Tolerance (bf16 inputs, fp32 accumulation): max-abs 2e-2, relative L2 1e-2."""
import numpy as np
import pytest
import torch

import paper_2609_34650_b200 as saf
import saf_inputs as si
from oracle import saf_oracle as orc

from gpu_util import Layer, assert_close, errors, f64, bf16_tensor, bf16_half_ulp, MAX_ABS, REL_L2

pytestmark = pytest.mark.gpu


def check_units(L: Layer, units, backward=True, rows=None, panel=512):
    """Compare the (b,h) units in `units` (all rows, or the row slice `rows` of the forward)."""
    inp, wl = L.inp, L.inp.wl
    q, k, v, do = f64(inp)
    scale = 1.0 / np.sqrt(wl.D)
    O, LSE = L.host(L.O), L.host(L.LSE)
    G = [L.host(g) for g in L.grads] if backward else None
    worst = {}
    deg = wl.T <= 2                                      # one or two tokens: see assert_close
    for b, h in units:
        fr = bool(inp.mask[h])
        eO, eL = orc.head_fwd_panels(fr, q[b, h], k[b, h], v[b, h], inp.alpha[h], inp.rho[h], scale, panel, rows)
        sl = rows or slice(0, wl.T)
        worst[("O", fr)] = assert_close(O[b, h][sl], eO, f"O[{b},{h}] frozen={fr}", degenerate=deg)
        if fr:
            assert not LSE[b, h].any(), "LSE slot of a frozen head must be zero"
        else:
            assert np.abs(LSE[b, h][sl] - eL).max() < 1e-4, f"LSE[{b},{h}]"
        if backward:
            e = orc.head_bwd_panels(fr, q[b, h], k[b, h], v[b, h], do[b, h], inp.alpha[h], inp.rho[h], scale, panel)
            for name, g, ee in zip(("dQ", "dK", "dV"), G, e):
                if fr and name != "dV":
                    assert not g[b, h].any(), f"{name}[{b},{h}] of a frozen head must be exactly zero"
                else:
                    assert_close(g[b, h], ee, f"{name}[{b},{h}] frozen={fr}", degenerate=deg)
    return worst


def sampled_units(wl, n, seed, backward=True):
    """Units for the full-size comparisons: `n` (b,h) pairs from a seeded draw that holds at least one frozen and
    one ordinary head where the workload has them, plus the unit of the last work item of the last CTA of the
    scheduler's list (the tail of the persistent grid)."""
    rng = np.random.default_rng(seed)
    fz = [h for h in range(wl.H) if wl.mask[h]]
    od = [h for h in range(wl.H) if not wl.mask[h]]
    units = []
    if fz:
        units.append((int(rng.integers(wl.B)), int(rng.choice(fz))))
    if od:
        units.append((int(rng.integers(wl.B)), int(rng.choice(od))))
    while len(units) < n:
        u = (int(rng.integers(wl.B)), int(rng.integers(wl.H)))
        if u not in units:
            units.append(u)
    n_ctas = torch.cuda.get_device_properties(0).multi_processor_count
    items, offsets = saf.saf_build_worklist(wl.B, wl.H, wl.T, wl.mask, backward, n_ctas)
    last = items[offsets[-1] - 1]
    tail = (int(last[0]), int(last[1]))
    if tail not in units:
        units.append(tail)
    return units


def grads_with_rounded_output(inp):
    """The backward's formulas (Sec. 3.3 / Appendix E.2) with delta_i = dO_i . O_i taken from the bf16-rounded O,
    as the layer is handed it, instead of the exact sum_j A_ij dP_ij: a test-side restatement built from the
    oracle's forward (no value comes from the GPU).  Same layouts as oracle.hybrid_attn_bwd."""
    wl = inp.wl
    q, k, v, do = f64(inp)
    mask = inp.mask
    H, T, D = wl.H, wl.T, wl.D
    packed = wl.packed_qk
    slot = np.cumsum(np.asarray(mask) == 0) - 1
    g = wl.kv_group
    scale = 1.0 / np.sqrt(D)
    dQ, dK, dV = np.zeros(q.shape), np.zeros(k.shape), np.zeros(v.shape)
    for h in range(H):
        for b in range(wl.B):
            if mask[h]:
                dV[b, h // g] += orc.frozen_head_bwd(do[b, h], inp.alpha[h], inp.rho[h])
                continue
            hq, hk = (slot[h], slot[h]) if packed else (h, h // g)
            O, _, A = orc.ordinary_head_fwd(q[b, hq], k[b, hk], v[b, h // g], scale)
            O_r = si.bf16_bits_to_f64(si.f32_to_bf16_bits(O.astype(np.float32)))
            dP = do[b, h] @ v[b, h // g].T
            dS = A * (dP - (do[b, h] * O_r).sum(axis=1, keepdims=True))
            dQ[b, hq] = scale * (dS @ k[b, hk])
            dK[b, hk] += scale * (dS.T @ q[b, hq])
            dV[b, h // g] += A.T @ do[b, h]
    return dQ, dK, dV


def check_bf16_grads_against_oracle(L16):
    """bf16 gradients against the fp64 oracle: the result is rounded once more, so the absolute bound grows by half
    a bf16 unit in the last place at the tensor's largest magnitude; the relative L2 bound is unchanged."""
    inp, wl = L16.inp, L16.inp.wl
    q, k, v, do = f64(inp)
    want = orc.hybrid_attn_bwd(q, k, v, do, inp.mask, inp.alpha.astype(np.float64), inp.rho.astype(np.float64))
    for name, got, ee in zip(("dQ", "dK", "dV"), (L16.host(g) for g in L16.grads), want):
        assert got.shape == ee.shape, name
        shared = wl.kv_group if name == "dV" else 1
        for b in range(ee.shape[0]):
            for h in range(ee.shape[1]):
                if not ee[b, h].any():
                    assert not got[b, h].any(), f"{name}[{b},{h}] must be exactly zero"
                    continue
                bound = MAX_ABS * np.sqrt(shared) + bf16_half_ulp(np.abs(ee[b, h]).max())
                assert_close(got[b, h], ee[b, h], f"bf16 {name}[{b},{h}]", max_abs=bound, degenerate=wl.T <= 2)


def all_units(wl):
    return [(b, h) for b in range(wl.B) for h in range(wl.H)]


# --------------------------------------------------------------------------- small, exhaustive
def test_config0_tiny_all_units():
    L = Layer(si.generate(si.config(0))).run()
    check_units(L, all_units(L.inp.wl))


def test_paper_test_shape_T129_stored_192():
    """Batch 2, T=129, 4 heads x 64, stored pattern length 192, heads 1 and 3 frozen (Appendix E.2)."""
    wl = si.Workload("paper-shape", 2, 4, 129, 64, (1, 3), -0.05, Tp=192, seed=3)
    L = Layer(si.generate(wl)).run()
    check_units(L, all_units(wl))


def test_error_scale_against_the_papers_own_test():
    """Error-scale sanity on the shape of the paper's kernel test: the relative L2 errors of O and dV against the fp64
    oracle stay within three times the figures the paper prints for its BF16 run (tests/golden; the inputs differ -
    seeded N(0,1) tensors here, a RoPE layer there - so only the scale is comparable)."""
    import os
    gold = {}
    with open(os.path.join(os.path.dirname(__file__), "golden", "paper_gradient_errors_bf16.txt")) as f:
        for line in f:
            if line.strip() and not line.startswith("#"):
                name, ma, rl = line.split()
                gold[name] = (float(ma), float(rl))
    wl = si.Workload("paper-test", 2, 4, 129, 64, (1, 3), -0.05, Tp=192, seed=5)
    L = Layer(si.generate(wl)).run()
    inp = L.inp
    q, k, v, do = f64(inp)
    eO, _ = orc.hybrid_attn_fwd(q, k, v, inp.mask, inp.alpha.astype(np.float64), inp.rho.astype(np.float64))
    _, _, eV = orc.hybrid_attn_bwd(q, k, v, do, inp.mask, inp.alpha.astype(np.float64), inp.rho.astype(np.float64))
    _, rl_o = errors(L.host(L.O), eO)
    _, rl_v = errors(L.host(L.grads[2]), eV)
    assert rl_o <= 3 * gold["output"][1], (rl_o, gold["output"])
    assert rl_v <= 3 * gold["dV"][1], (rl_v, gold["dV"])


@pytest.mark.parametrize("T", [1, 2, 127, 128, 255, 257, 384])
def test_ragged_lengths(T):
    wl = si.Workload(f"ragged{T}", 1, 3, T, 64, (1,), -0.05, seed=T)
    L = Layer(si.generate(wl)).run()
    check_units(L, all_units(wl))


@pytest.mark.parametrize("frozen", [(), (0, 1, 2, 3)])
def test_empty_and_full_frozen_sets(frozen):
    wl = si.Workload("sets", 2, 4, 320, 64, frozen, -0.05, seed=11)
    L = Layer(si.generate(wl)).run()
    check_units(L, all_units(wl))


def test_head_dim_128_forward():
    wl = si.Workload("d128", 2, 4, 640, 128, (2,), -0.01, alpha0_spike=4.0, backward=False, seed=5)
    L = Layer(si.generate(wl), backward=False).run(backward=False)
    check_units(L, all_units(wl), backward=False)


@pytest.mark.parametrize("T,frozen,g", [(300, (1, 2), 1), (129, (), 1), (384, (0, 1, 2, 3), 2)])
def test_head_dim_96_forward(T, frozen, g):
    """The paper's 1B model uses 16 heads of dimension 96: forward on the 128-wide kernel with TMA zero padding."""
    wl = si.Workload("d96", 2, 4, T, 96, frozen, -0.03, seed=96 + T, kv_group=g, backward=False)
    L = Layer(si.generate(wl), backward=False).run(backward=False)
    _check_gqa_layer(L, False)


@pytest.mark.parametrize("T,frozen,g", [(300, (1, 2), 1), (130, (), 1), (260, (0, 3), 2)])
def test_head_dim_96_forward_backward(T, frozen, g):
    """Head dimension 96 (the paper's 1B model) through the 128-wide kernels, gradients with row length 96."""
    wl = si.Workload("d96fb", 2, 4, T, 96, frozen, -0.03, seed=196 + T, kv_group=g)
    _check_gqa_layer(Layer(si.generate(wl)).run(), True)


@pytest.mark.parametrize("T,frozen", [(128, ()), (300, (1, 3)), (1, (0,)), (129, (0, 1, 2, 3)), (513, (2,))])
def test_head_dim_128_forward_backward(T, frozen):
    """The 128-wide backward kernel: ordinary heads and the tensor-core frozen form, ragged lengths."""
    wl = si.Workload("d128fb", 2, 4, T, 128, frozen, -0.03, seed=128 + T)
    L = Layer(si.generate(wl)).run()
    check_units(L, all_units(wl))


def test_head_dim_128_backward_general_frozen_form_and_bf16():
    """Wide-range pattern (tensor-core form refused): P^^T half tiles with one exponential per element."""
    wl = si.Workload("d128wide", 1, 3, 300, 128, (0, 2), -0.4, seed=131)
    inp = si.generate(wl)
    inp.alpha[0] *= 8.0
    inp.do[:] = si.f32_to_bf16_bits(si.bf16_bits_to_f32(inp.do) / 16.0)
    L = Layer(inp).run()
    check_units(L, all_units(wl))
    L16 = Layer(inp, grad_dtype=saf.SAF_BF16).run()
    for g32, g16 in zip(L.grads, L16.grads):
        a, b = L.host(g32), L.host(g16)
        assert np.abs(a - b).max() <= 2.0 ** -8 * max(np.abs(a).max(), 1.0) + 1e-6
    check_bf16_grads_against_oracle(L16)


def test_head_dim_128_backward_shared_and_packed_heads():
    wl = si.Workload("d128gqa", 2, 8, 260, 128, (1, 6), -0.03, seed=132, kv_group=4)
    _check_gqa_layer(Layer(si.generate(wl)).run(), True)
    wl = si.Workload("d128packed", 2, 5, 200, 128, (0, 3), -0.03, seed=133, packed_qk=True)
    _check_packed_layer(Layer(si.generate(wl)).run(), True)


def test_head_dim_128_backward_many_items_per_cta():
    wl = si.Workload("d128mix", 4, 6, 1100, 128, (0, 3, 4), -0.02, seed=134)
    L = Layer(si.generate(wl)).run()
    check_units(L, [(0, 0), (3, 5), (1, 3), (2, 1), (3, 4), (0, 2)])


def test_multi_tile_scheduler_mix():
    """Several items per CTA of both kinds: 8 x 6 heads x 9 blocks = 432 forward items on 296 CTAs."""
    wl = si.Workload("mix", 8, 6, 1100, 64, (0, 3, 4), -0.05, seed=21)
    L = Layer(si.generate(wl)).run()
    check_units(L, [(0, 0), (7, 5), (3, 3), (5, 1), (2, 4), (6, 2)])


def test_item_kinds_alternate_within_a_cta():
    """Ordinary items, frozen items in the tensor-core form and frozen items in the general form (a head whose pattern
    leaves the factorised form's range) follow one another in the CTAs' work lists: 8 x 8 heads x 10 blocks = 640
    forward items on 296 CTAs.  The tensor-core frozen tiles run a shared-memory ring of their own that is laid over
    the other kinds' stages, so every change of kind is a hand-over between the rings."""
    T = 1200
    wl = si.Workload("kinds", 8, 8, T, 64, (0, 2, 3, 5, 6), -0.05, seed=23)
    inp = si.generate(wl)
    for h in (2, 5):                                     # far outside the range of the tensor-core form
        inp.alpha[h] = (inp.alpha[h] + 25.0 * np.sin(0.37 * np.arange(T))).astype(np.float32)
    # such patterns put a row's mass on a few keys, whose dV then sums hundreds of output gradients; dO / 16 (exact
    # in bf16) keeps the gradients in the value range the absolute tolerance is meant for
    inp.do[...] = si.f32_to_bf16_bits(si.bf16_bits_to_f32(inp.do) / 16.0)
    L = Layer(inp).run()
    check_units(L, [(0, 0), (0, 2), (1, 1), (2, 5), (3, 3), (4, 4), (5, 6), (6, 7), (7, 2), (7, 0)])


# --------------------------------------------------------------------------- invariants on the GPU
def test_frozen_heads_never_read_q_k_and_get_zero_grads():
    wl = si.Workload("poison", 2, 4, 300, 64, (0, 2), -0.05, seed=8)
    inp = si.generate(wl)
    clean = Layer(inp).run()
    L = Layer(inp)
    for h in wl.frozen_heads:
        L.Q[:, h] = float("nan")
        L.K[:, h] = float("nan")
    L.run()
    assert torch.equal(L.O, clean.O)
    assert torch.equal(L.grads[2], clean.grads[2])
    for h in wl.frozen_heads:
        assert not L.grads[0][:, h].any() and not L.grads[1][:, h].any()
    for h in (1, 3):
        assert L.grads[0][:, h].abs().max() > 0 and L.grads[1][:, h].abs().max() > 0


def test_frozen_head_equals_engineered_ordinary_head_on_gpu():
    """S[i,j] = alpha[j] + lambda j (+ row constant) makes an ordinary head equal the frozen head
    (alpha, rho = -lambda d); all values exactly representable in bf16."""
    T, D, lam, scale = 256, 64, 2.0 ** -4, 0.125
    rng = np.random.default_rng(0)
    alpha = si.bf16_bits_to_f32(si.f32_to_bf16_bits(rng.standard_normal(T).astype(np.float32)))
    wl = si.Workload("p6", 1, 2, T, D, (1,), -lam, seed=1)
    inp = si.generate(wl)
    q = np.zeros((T, D), np.float32)
    k = np.zeros((T, D), np.float32)
    q[:, 0] = q[:, 1] = 1.0 / scale
    k[:, 0] = alpha
    k[:, 1] = lam * np.arange(T)
    inp.q[0, 0], inp.k[0, 0] = si.f32_to_bf16_bits(q), si.f32_to_bf16_bits(k)
    inp.v[0, 1], inp.do[0, 1] = inp.v[0, 0], inp.do[0, 0]
    inp.alpha[1] = alpha
    inp.rho[1] = -lam * np.arange(T)
    L = Layer(inp).run()
    O, dV = L.host(L.O), L.host(L.grads[2])
    assert np.abs(O[0, 0] - O[0, 1]).max() < MAX_ABS         # two bf16-rounded outputs of values up to ~3
    ma, rl = errors(dV[0, 0], dV[0, 1])
    assert ma < MAX_ABS and rl < REL_L2


def test_exact_exponent_fallback_for_wide_range_patterns():
    """alpha / rho ranges far beyond fp32's factorised range (rho rising 0.9 per step) still match."""
    T = 300
    wl = si.Workload("wide", 1, 2, T, 64, (0, 1), 0.9, seed=4)
    inp = si.generate(wl)
    inp.alpha[1] = (40.0 * np.sin(np.arange(T))).astype(np.float32)
    # such a pattern puts every row's mass on the earliest keys, so dV[0] sums ~T output gradients;
    # dO / 16 (exact in bf16) keeps the gradient in the value range the absolute tolerance is meant for
    inp.do[...] = si.f32_to_bf16_bits(si.bf16_bits_to_f32(inp.do) / 16.0)
    L = Layer(inp).run()
    check_units(L, all_units(wl))


def test_values_beyond_fp16_range_take_the_general_frozen_path():
    """The tensor-core form of a frozen head stages a V and w dO in fp16; tensors that would overflow there
    must be detected per call and handled by the general (bf16 pattern tile) path.  V and dO scaled by 2^17
    (exact in bf16) must give O and dV scaled by 2^17."""
    wl = si.Workload("range", 1, 2, 300, 64, (0,), -0.05, seed=31)
    inp = si.generate(wl)
    ref = Layer(inp).run()
    big = si.generate(wl)
    k = 2.0 ** 17
    big.v[...] = si.f32_to_bf16_bits(si.bf16_bits_to_f32(big.v) * k)
    big.do[...] = si.f32_to_bf16_bits(si.bf16_bits_to_f32(big.do) * k)
    L = Layer(big).run()
    q, kk, v, do = f64(inp)
    scale = 1.0 / np.sqrt(wl.D)
    eO, _ = orc.head_fwd_panels(True, q[0, 0], kk[0, 0], v[0, 0], inp.alpha[0], inp.rho[0], scale)
    _, _, edV = orc.head_bwd_panels(True, q[0, 0], kk[0, 0], v[0, 0], do[0, 0], inp.alpha[0], inp.rho[0], scale)
    assert_close(L.host(L.O)[0, 0] / k, eO, "O of the scaled problem")
    assert_close(L.host(L.grads[2])[0, 0] / k, edV, "dV of the scaled problem")
    # and the unscaled problem went through the tensor-core form with much smaller error on dV
    ma, rl = errors(ref.host(ref.grads[2])[0, 0], edV)
    assert rl < 1e-3


def test_stale_state_fuzz_on_one_context():
    """Mask / pattern / shape changes on one context (cached work lists, workspaces) stay correct."""
    ctx = saf.Context(0)
    rng = np.random.default_rng(99)
    for step in range(12):
        H = int(rng.integers(1, 5))
        T = int(rng.choice([64, 129, 200, 256, 300]))
        nf = int(rng.integers(0, H + 1))
        frozen = tuple(sorted(rng.choice(H, nf, replace=False).tolist()))
        wl = si.Workload(f"fuzz{step}", int(rng.integers(1, 3)), H, T, 64, frozen, -0.05, Tp=T + int(rng.integers(0, 40)),
                         seed=100 + step)
        L = Layer(si.generate(wl), ctx=ctx).run()
        check_units(L, all_units(wl))


def test_strided_views_bthd_layout():
    """Q/K/V/O/dO given as [B,T,H,D] storage viewed as [B,H,T,D] (non-contiguous heads)."""
    wl = si.Workload("strided", 2, 3, 260, 64, (1,), -0.05, seed=13)
    inp = si.generate(wl)
    L = Layer(inp)
    for name in ("Q", "K", "V", "dO", "O"):
        t = getattr(L, name)
        setattr(L, name, t.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3))
    L.prob = saf.make_problem(L.Q, wl.stored_len, k_like=L.K, v_like=L.V, o_like=L.O)
    L.run()
    check_units(L, all_units(wl))


def test_bf16_gradients():
    """grad_dtype = bf16: one extra rounding of the result; |dV| reaches ~8 for concentrated
    patterns, where half a bf16 ulp is 1.6e-2, so the max-abs bound is 2e-2 + 1.6e-2."""
    inp = si.generate(si.config(0))
    L = Layer(inp, grad_dtype=saf.SAF_BF16).run()
    ref = Layer(inp).run()
    for g16, g32 in zip(L.grads, ref.grads):
        ma, rl = errors(L.host(g16), L.host(g32))
        assert ma <= 3.2e-2 and rl <= 5e-3
    check_bf16_grads_against_oracle(L)


def test_forward_is_deterministic_and_internal_prepare_matches():
    inp = si.generate(si.Workload("det", 2, 4, 400, 64, (2,), -0.05, seed=17))
    A = Layer(inp).run()
    B = Layer(inp)
    B.logZ = None                      # library computes the normalisers itself
    B.run(prepare=False)
    assert torch.equal(A.O, B.O) and torch.equal(A.LSE, B.LSE)
    assert torch.equal(A.grads[1], B.grads[1]) and torch.equal(A.grads[2], B.grads[2])
    ez = orc.pattern_logZ(inp.alpha[2], inp.rho[2], 400)
    assert np.abs(A.logZ[2].cpu().numpy() - ez).max() < 5e-6


def test_host_buffer_step_matches_device_path():
    inp = si.generate(si.Workload("host", 2, 3, 200, 64, (1,), -0.05, seed=23))
    D = Layer(inp).run()
    wl = inp.wl
    ctx = saf.Context(0)
    pin = lambda t: t.pin_memory()
    Q, K, V, dO = (pin(bf16_tensor(x)) for x in (inp.q, inp.k, inp.v, inp.do))
    alpha, rho = pin(torch.from_numpy(inp.alpha)), pin(torch.from_numpy(inp.rho))
    O = pin(torch.empty_like(Q))
    LSE = pin(torch.empty(wl.B, wl.H, wl.T))
    dQ, dK, dV = (pin(torch.empty(Q.shape, dtype=torch.float32)) for _ in range(3))
    prob = saf.make_problem(Q, wl.stored_len)
    for prepare in (1, 0):
        ctx.saf_hybrid_attn_step_host(prob, Q, K, V, dO, inp.mask, alpha, rho, prepare, O, LSE, dQ, dK, dV)
        assert torch.equal(O, D.O.cpu()) and torch.equal(LSE, D.LSE.cpu())
        assert torch.equal(dK, D.grads[1].cpu()) and torch.equal(dV, D.grads[2].cpu())
        ma, rl = errors(dQ.numpy().astype(np.float64), D.host(D.grads[0]))
        assert ma < 1e-4                       # atomics order only


@pytest.mark.parametrize("g,gd", [(1, saf.SAF_F32), (2, saf.SAF_F32), (1, saf.SAF_BF16)])
def test_host_buffer_step_in_chunks_matches_device_path(g, gd):
    """Large enough to be cut into chunks of whole batch entries (11 entries -> chunks of 2 and a last one of 1)."""
    inp = si.generate(si.Workload("host-chunks", 11, 4, 2048, 64, (2,), -0.05, seed=29, kv_group=g))
    D = Layer(inp, grad_dtype=gd).run()
    wl = inp.wl
    ctx = saf.Context(0)
    pin = lambda t: t.pin_memory()
    Q, K, V, dO = (pin(bf16_tensor(x)) for x in (inp.q, inp.k, inp.v, inp.do))
    alpha, rho = pin(torch.from_numpy(inp.alpha)), pin(torch.from_numpy(inp.rho))
    O = pin(torch.empty_like(Q))
    LSE = pin(torch.empty(wl.B, wl.H, wl.T))
    gdt = torch.float32 if gd == saf.SAF_F32 else torch.bfloat16
    dQ, dK, dV = (pin(torch.full(t.shape, float("nan"), dtype=gdt)) for t in (Q, K, V))
    prob = saf.make_problem(Q, wl.stored_len, grad_dtype=gd, k_like=K, v_like=V, o_like=O, kv_group=g, H=wl.H)
    ctx.saf_hybrid_attn_step_host(prob, Q, K, V, dO, inp.mask, alpha, rho, 1, O, LSE, dQ, dK, dV)
    assert torch.equal(O, D.O.cpu()) and torch.equal(LSE, D.LSE.cpu())
    for got, want, exact in ((dQ, D.grads[0], False), (dK, D.grads[1], g == 1), (dV, D.grads[2], g == 1)):
        if exact:
            assert torch.equal(got, want.cpu())
        else:                                  # accumulated with atomics: order only
            ma, rl = errors(got.float().numpy().astype(np.float64), D.host(want))
            assert ma < (1e-4 if gd == saf.SAF_F32 else 2e-2) and np.isfinite(got.float().numpy()).all()


@pytest.mark.parametrize("D,g", [(128, 1), (96, 2)])
def test_host_buffer_step_wide_heads_in_chunks(D, g):
    """The host-buffer step on the 128-wide kernels (head dimension 128, and 96 with shared key/value heads), cut
    into chunks of whole batch entries, against the device path on the same inputs."""
    inp = si.generate(si.Workload("host-wide", 9, 4, 1024, D, (1, 3), -0.05, seed=33, kv_group=g))
    Dv = Layer(inp).run()
    wl = inp.wl
    ctx = saf.Context(0)
    pin = lambda t: t.pin_memory()
    Q, K, V, dO = (pin(bf16_tensor(x)) for x in (inp.q, inp.k, inp.v, inp.do))
    alpha, rho = pin(torch.from_numpy(inp.alpha)), pin(torch.from_numpy(inp.rho))
    O = pin(torch.empty_like(Q))
    LSE = pin(torch.empty(wl.B, wl.H, wl.T))
    dQ, dK, dV = (pin(torch.full(t.shape, float("nan"), dtype=torch.float32)) for t in (Q, K, V))
    prob = saf.make_problem(Q, wl.stored_len, k_like=K, v_like=V, o_like=O, kv_group=g, H=wl.H)
    ctx.saf_hybrid_attn_step_host(prob, Q, K, V, dO, inp.mask, alpha, rho, 1, O, LSE, dQ, dK, dV)
    assert torch.equal(O, Dv.O.cpu()) and torch.equal(LSE, Dv.LSE.cpu())
    for got, want, exact in ((dQ, Dv.grads[0], False), (dK, Dv.grads[1], g == 1), (dV, Dv.grads[2], g == 1)):
        if exact:
            assert torch.equal(got, want.cpu())
        else:                                  # accumulated with reduce-adds: order only
            ma, rl = errors(got.numpy().astype(np.float64), Dv.host(want))
            assert ma < 1e-4 and np.isfinite(got.numpy()).all()


def test_forward_backward_capture_into_a_cuda_graph():
    """After a warm-up call (which allocates the context's workspaces and uploads the work lists) a forward +
    backward step records into a CUDA graph, and replays reproduce the eager results bit for bit (dQ to rounding:
    its reduce-adds arrive in varying order)."""
    inp = si.generate(si.Workload("graph", 2, 4, 600, 64, (1,), -0.05, seed=71))
    L = Layer(inp)
    s = torch.cuda.Stream()
    with torch.cuda.stream(s):
        L.run()
        want = [t.clone() for t in (L.O, L.LSE, *L.grads)]
        for t in (L.O, L.LSE, *L.grads):
            t.fill_(float("nan"))
        g = torch.cuda.CUDAGraph()
        c = L.ctx
        with torch.cuda.graph(g, stream=s):
            c.saf_hybrid_attn_fwd(L.prob, L.Q, L.K, L.V, L.mask, L.alpha, L.rho, L.logZ, L.O, L.LSE)
            c.saf_hybrid_attn_bwd(L.prob, L.Q, L.K, L.V, L.O, L.dO, L.LSE, L.mask, L.alpha, L.rho, L.logZ, *L.grads)
        for _ in range(2):
            g.replay()
        torch.cuda.synchronize()
    code, detail = L.ctx.saf_last_device_status()
    assert code == saf.SAF_OK, f"device status {code} detail {detail:#x}"
    got = (L.O, L.LSE, *L.grads)
    assert torch.equal(got[0], want[0]) and torch.equal(got[1], want[1])
    assert torch.equal(got[3], want[3]) and torch.equal(got[4], want[4])
    assert (got[2] - want[2]).abs().max().item() < 1e-4


def test_invalid_arguments_are_rejected():
    inp = si.generate(si.Workload("bad", 1, 2, 64, 64, (1,), -0.05))
    L = Layer(inp)
    L.prob.Tp = 32                             # T > Tp
    with pytest.raises(saf.SafError) as e:
        L.run()
    assert e.value.code == 1
    L = Layer(inp)
    L.prob.D = 80                              # supported: 64, 96, 128
    with pytest.raises(saf.SafError) as e:
        L.run()
    assert e.value.code == 2
    L = Layer(inp)
    L.prob.q_strides[2] = 60                   # not a multiple of 8 elements
    with pytest.raises(saf.SafError) as e:
        L.run()
    assert e.value.code == 1


# --------------------------------------------------------------------------- grouped-query path
def _check_gqa_layer(L, backward, grad_rel_l2=REL_L2, expected_grads=None):
    """Whole layer against the dense oracle: K, V (and dK, dV) have H / kv_group heads."""
    inp, wl = L.inp, L.inp.wl
    deg = wl.T <= 2
    q, k, v, do = f64(inp)
    O, LSE = L.host(L.O), L.host(L.LSE)
    eO, eL = orc.hybrid_attn_fwd(q, k, v, inp.mask, inp.alpha.astype(np.float64), inp.rho.astype(np.float64))
    for b in range(wl.B):
        for h in range(wl.H):
            assert_close(O[b, h], eO[b, h], f"O[{b},{h}]", degenerate=deg)
            if inp.mask[h]:
                assert not LSE[b, h].any()
            else:
                assert np.abs(LSE[b, h] - eL[b, h]).max() < 1e-4
    if not backward:
        return
    dQ, dK, dV = (L.host(g) for g in L.grads)
    eQ, eK, eV = expected_grads or orc.hybrid_attn_bwd(q, k, v, do, inp.mask, inp.alpha.astype(np.float64),
                                                       inp.rho.astype(np.float64))
    assert dK.shape == eK.shape and dV.shape == eV.shape
    for b in range(wl.B):
        for h in range(wl.H):
            if inp.mask[h]:
                assert not dQ[b, h].any(), "dQ of a frozen head must be exactly zero"
            else:
                assert_close(dQ[b, h], eQ[b, h], f"dQ[{b},{h}]", rel_l2=grad_rel_l2, degenerate=deg)
        for hk in range(wl.H // wl.kv_group):
            assert_close(dK[b, hk], eK[b, hk], f"dK[{b},kv {hk}]", rel_l2=grad_rel_l2, degenerate=deg)
            # a shared head's dV sums kv_group heads: the absolute bound scales with the number of terms
            assert_close(dV[b, hk], eV[b, hk], f"dV[{b},kv {hk}]", max_abs=MAX_ABS * np.sqrt(wl.kv_group),
                         rel_l2=grad_rel_l2, degenerate=deg)


@pytest.mark.parametrize("H,g,frozen,T", [(8, 4, (1, 6), 300), (4, 2, (), 257), (6, 3, (0, 1, 2), 200),
                                          (4, 4, (0, 1, 2, 3), 129), (4, 1, (2,), 130)])
def test_gqa_shared_kv_heads_forward_backward(H, g, frozen, T):
    """Query head h reads key/value head h // g; the shared heads' gradients sum over their query heads; a group
    may be all ordinary, mixed or all frozen (then its dK is exactly zero)."""
    wl = si.Workload("gqa", 2, H, T, 64, frozen, -0.05, seed=40 + H + g, kv_group=g)
    L = Layer(si.generate(wl)).run()
    _check_gqa_layer(L, True)
    if g > 1 and len(frozen) == H:
        assert not L.host(L.grads[1]).any()


def test_gqa_head_dim_128_forward():
    wl = si.Workload("gqa128", 1, 8, 384, 128, (2, 3), -0.02, seed=44, kv_group=4, backward=False)
    L = Layer(si.generate(wl), backward=False).run(backward=False)
    _check_gqa_layer(L, False)


def test_gqa_qwen_like_geometry_sampled():
    """32 query heads on 8 shared key/value heads, D = 128, forward only (the long-context geometry)."""
    wl = si.Workload("gqa-qwen", 1, 32, 2048, 128, tuple(range(0, 32, 4)), -0.002, alpha0_spike=4.0, seed=45,
                     kv_group=4, backward=False)
    inp = si.generate(wl)
    L = Layer(inp, backward=False).run(backward=False)
    q, k, v, _ = f64(inp)
    O = L.host(L.O)
    for h in (0, 5, 31):
        fr = bool(inp.mask[h])
        eO, _ = orc.head_fwd_panels(fr, q[0, h], k[0, h // 4], v[0, h // 4], inp.alpha[h], inp.rho[h],
                                    1.0 / np.sqrt(wl.D), 1024, None)
        assert_close(O[0, h], eO, f"O[0,{h}] frozen={fr}")


def test_gqa_bf16_gradients_and_bad_group():
    """bf16 gradients of shared heads: accumulated in fp32, rounded once at the end."""
    wl = si.Workload("gqa-bf16", 2, 4, 200, 64, (1,), -0.05, seed=46, kv_group=2)
    inp = si.generate(wl)
    L32 = Layer(inp).run()
    L16 = Layer(inp, grad_dtype=saf.SAF_BF16).run()
    for g32, g16, name in zip(L32.grads, L16.grads, ("dQ", "dK", "dV")):
        a, b = L32.host(g32), L16.host(g16)
        assert a.shape == b.shape
        assert np.abs(a - b).max() <= 2.0 ** -8 * max(np.abs(a).max(), 1.0) + 1e-6, name   # one bf16 rounding
    check_bf16_grads_against_oracle(L16)
    L = Layer(inp)
    L.prob.kv_group = 3                        # does not divide H
    with pytest.raises(saf.SafError) as e:
        L.run()
    assert e.value.code == 1


# --------------------------------------------------------------------------- packed Q/K layout
def _check_packed_layer(L, backward, grad_rel_l2=REL_L2, expected_grads=None):
    inp, wl = L.inp, L.inp.wl
    deg = wl.T <= 2
    q, k, v, do = f64(inp)
    al, rh = inp.alpha.astype(np.float64), inp.rho.astype(np.float64)
    O, LSE = L.host(L.O), L.host(L.LSE)
    eO, eL = orc.hybrid_attn_fwd(q, k, v, inp.mask, al, rh)
    for b in range(wl.B):
        for h in range(wl.H):
            assert_close(O[b, h], eO[b, h], f"O[{b},{h}]", degenerate=deg)
            if inp.mask[h]:
                assert not LSE[b, h].any()
            else:
                assert np.abs(LSE[b, h] - eL[b, h]).max() < 1e-4
    if not backward:
        return
    dQ, dK, dV = (L.host(g) for g in L.grads)
    eQ, eK, eV = expected_grads or orc.hybrid_attn_bwd(q, k, v, do, inp.mask, al, rh)
    assert dQ.shape == eQ.shape and dK.shape == eK.shape and dV.shape == eV.shape
    for b in range(wl.B):
        for s_ in range(dQ.shape[1]):
            assert_close(dQ[b, s_], eQ[b, s_], f"dQ[{b},slot {s_}]", rel_l2=grad_rel_l2, degenerate=deg)
            assert_close(dK[b, s_], eK[b, s_], f"dK[{b},slot {s_}]", rel_l2=grad_rel_l2, degenerate=deg)
        for h in range(wl.H):
            assert_close(dV[b, h], eV[b, h], f"dV[{b},{h}]", rel_l2=grad_rel_l2, degenerate=deg)


@pytest.mark.parametrize("H,frozen,T,gd", [(6, (1, 4), 300, "f32"), (4, (0, 3), 129, "bf16"), (3, (), 200, "f32"),
                                           (5, (0, 1, 2, 3), 257, "f32")])
def test_packed_qk_layout_forward_backward(H, frozen, T, gd):
    """Q, K, dQ, dK hold only the ordinary heads (Appendix E.2: replaced heads have no query/key slot)."""
    wl = si.Workload("packed", 2, H, T, 64, frozen, -0.05, seed=50 + H + T, packed_qk=True)
    L = Layer(si.generate(wl), grad_dtype=saf.SAF_F32 if gd == "f32" else saf.SAF_BF16).run()
    if gd == "f32":
        _check_packed_layer(L, True)
    else:
        L32 = Layer(L.inp).run()
        for g32, g16 in zip(L32.grads, L.grads):
            a, b = L32.host(g32), L.host(g16)
            assert a.shape == b.shape and np.abs(a - b).max() <= 2.0 ** -8 * max(np.abs(a).max(), 1.0) + 1e-6
        check_bf16_grads_against_oracle(L)


def test_packed_qk_layout_head_dim_128_forward_and_errors():
    wl = si.Workload("packed128", 1, 6, 384, 128, (1, 2, 5), -0.02, seed=57, packed_qk=True, backward=False)
    L = Layer(si.generate(wl), backward=False).run(backward=False)
    _check_packed_layer(L, False)
    L = Layer(si.generate(si.Workload("packed-bad", 1, 4, 128, 64, (1,), -0.05, seed=58, packed_qk=True)))
    L.prob.kv_group = 2                        # the packed layout is a multi-head layout
    with pytest.raises(saf.SafError) as e:
        L.run()
    assert e.value.code == 1


# --------------------------------------------------------------------------- seeded random geometries
def _random_workload(seed):
    """A geometry drawn from the options of the layer (head size, grouping, packed layout, frozen set, lengths
    around tile edges, stored pattern longer than the sequence, sink-like alpha, decay rate)."""
    rng = np.random.default_rng(1000 + seed)
    D = int(rng.choice([64, 96, 128]))
    layout = rng.choice(["mha", "gqa", "packed"])
    g = int(rng.choice([2, 3, 4])) if layout == "gqa" else 1
    H = g * int(rng.integers(1, 4)) if layout == "gqa" else int(rng.integers(1, 7))
    B = int(rng.integers(1, 4))
    T = int(rng.choice([rng.integers(1, 130), rng.integers(130, 400), 128 * rng.integers(1, 4) + rng.choice([-1, 0, 1])]))
    nf = int(rng.integers(0, H + 1))
    frozen = tuple(sorted(rng.choice(H, size=nf, replace=False).tolist()))
    Tp = T + int(rng.integers(0, 70)) if rng.random() < 0.4 else 0
    spike = float(rng.choice([0.0, 3.0]))
    slope = float(rng.choice([-0.3, -0.05, -0.005]))
    return si.Workload(f"random-{seed}", B, H, max(T, 1), D, frozen, slope, Tp=Tp, alpha0_spike=spike,
                       seed=2000 + seed, kv_group=g, packed_qk=(layout == "packed"))


@pytest.mark.parametrize("seed", range(24))
def test_random_geometries_forward_backward(seed):
    """Combinations that no fixed case pairs up (for example 96-wide heads with shared key/value heads and a
    stored pattern longer than the sequence), each against the dense oracle over the whole layer."""
    wl = _random_workload(seed)
    L = Layer(si.generate(wl)).run()
    # The backward forms delta_i = dO_i . O_i from the bf16 O it is given.  With rows of only a few keys, dP - delta
    # nearly cancels and that rounding of O (2^-9 relative) is not averaged out: measured at T = 3 the gradients lie
    # within 2.5e-3 (relative L2) of the oracle's formulas evaluated with the same rounded O, but up to 1.1e-2 from
    # the oracle's exact delta.  Sequences shorter than 8 therefore get twice the relative bound on the gradients.
    # That the doubled bound is needed only for this reason is asserted, not assumed: against the same formulas with
    # delta from the rounded O the stated bound holds at every length.
    tol = 2 * REL_L2 if wl.T < 8 else REL_L2
    check = _check_packed_layer if wl.packed_qk else _check_gqa_layer
    check(L, True, grad_rel_l2=tol)
    if wl.T < 8:
        check(L, True, grad_rel_l2=REL_L2, expected_grads=grads_with_rounded_output(L.inp))


# --------------------------------------------------------------------------- full sizes, sampled
def test_config1_full_size_sampled_units():
    wl = si.config(1)
    L = Layer(si.generate(wl)).run()
    check_units(L, sampled_units(wl, 4, seed=101), panel=1024)


@pytest.mark.parametrize("nf", [0, 6, 9, 12])
def test_config3_sweep_full_size_sampled_units(nf):
    wl = si.config(3, nf)
    L = Layer(si.generate(wl)).run()
    check_units(L, sampled_units(wl, 2, seed=300 + nf), panel=1024)


def test_config2_full_size_sampled_units():
    wl = si.config(2)
    L = Layer(si.generate(wl)).run()
    check_units(L, sampled_units(wl, 2, seed=102), panel=1024)


def test_long_sequence_16k_forward_backward_sampled_units():
    """T = 16384 (the longest training context of the paper's cross-context comparison): 128 key blocks per head."""
    wl = si.Workload("long-16k", 1, 3, 16384, 64, (1,), -0.005, seed=61)
    L = Layer(si.generate(wl)).run()
    check_units(L, [(0, 0), (0, 1)], panel=1024)


def test_config4_long_prefill_sampled_row_panels():
    wl = si.config(4)
    L = Layer(si.generate(wl), backward=False).run(backward=False)
    oh = [h for h in range(wl.H) if h not in wl.frozen_heads][5]
    for rows in (slice(0, 256), slice(16300, 16500), slice(wl.T - 256, wl.T)):
        check_units(L, [(0, wl.frozen_heads[0]), (0, oh)], backward=False, rows=rows, panel=256)
