"""Seeded synthetic inputs for the hybrid (ordinary + frozen head) causal attention layer.

This module is the only code shared by the CPU oracle's tests and the CUDA path's tests and
benchmark.  It draws random tensors and packs them; it contains none of the method's arithmetic
(no softmax, no pattern reconstruction, no normalisers).

Workload shapes follow the paper's settings: a GPT-2-124M-shaped layer (12 heads x 64, T=4096,
micro-batch 8), a "1B/8K"-shaped layer, a frozen-rate sweep (nested subsets of one seeded head
ranking, as the paper's rate comparisons use), and a long causal prefill at a 32-query-head x 128
geometry.  Preference vectors: the absolute-key-position vector is iid N(0,1) (the paper's
"structured random" control, Sec. 3.2); the relative-distance vector decays linearly with distance
plus N(0, 0.1^2) noise, optionally with a +4 spike on key 0 imitating an attention sink.

Draw order (fixed, so that every consumer sees identical bits for a given seed):
Q, K, V, dO as [B,H,T,D] float32 standard normals rounded to bf16 (round-to-nearest-even), then for
each frozen head in increasing head index: alpha [Tp] ~ N(0,1), then the rho noise [Tp] ~ N(0,1);
rho = slope * d + 0.1 * noise.  alpha and rho are stored as float32.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np


# --------------------------------------------------------------------------- bf16 bit helpers
def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 to bfloat16 (round-to-nearest-even); returns the uint16 bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    rounded = u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))
    return (rounded >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """Exact widening of bfloat16 bit patterns (uint16) to float32."""
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def bf16_bits_to_f64(b: np.ndarray) -> np.ndarray:
    return bf16_bits_to_f32(b).astype(np.float64)


# --------------------------------------------------------------------------- workload description
@dataclass(frozen=True)
class Workload:
    name: str
    B: int
    H: int
    T: int
    D: int
    frozen_heads: tuple           # sorted head indices that are frozen
    rho_slope: float              # rho(d) = rho_slope * d + 0.1 * noise
    Tp: int = 0                   # stored pattern length (0 -> T)
    alpha0_spike: float = 0.0     # added to alpha[0] (attention-sink-like)
    backward: bool = True
    seed: int = 0
    kv_group: int = 1             # grouped-query attention: query heads per shared key/value head
    packed_qk: bool = False       # Q and K carry only the ordinary heads, in head order (multi-head only)

    @property
    def stored_len(self) -> int:
        return self.Tp if self.Tp > 0 else self.T

    @property
    def mask(self) -> np.ndarray:
        m = np.zeros(self.H, dtype=np.uint8)
        m[list(self.frozen_heads)] = 1
        return m

    def flops(self, backward: bool | None = None) -> float:
        """Algorithmic FLOPs of the layer: one causal matmul = 2*D*T(T+1)/2 per (b,h);
        ordinary head 2 (fwd) + 5 (bwd) matmuls, frozen head 1 + 1."""
        bw = self.backward if backward is None else backward
        hf = len(self.frozen_heads)
        ho = self.H - hf
        unit = self.B * self.D * self.T * (self.T + 1)
        return float(unit * ((7 * ho + 2 * hf) if bw else (2 * ho + hf)))


def sweep_frozen_heads(H: int, n_frozen: int, seed: int = 0) -> tuple:
    """Nested frozen sets: one seeded permutation of the head indices, first n_frozen are frozen."""
    perm = np.random.default_rng(1000 + seed).permutation(H)
    return tuple(sorted(int(h) for h in perm[:n_frozen]))


def config(k: int, n_frozen: int | None = None, seed: int = 0) -> Workload:
    """The five benchmark/test configurations (k = 0..4).  `n_frozen` overrides the frozen count
    (config 3 is config 1's shape with n_frozen in {0,3,6,9,12}).  k = 5, 6 are two extra shapes for the wider
    head dimensions: config 1's layer at head dimension 128, and the layer of the paper's 1B model (16 heads of
    dimension 96, batch 2 per rank, 8K context); k = 7 is a grouped-query forward (32 query heads, 8 key/value heads of
    dimension 128)."""
    if k == 0:
        nf = 1 if n_frozen is None else n_frozen
        return Workload("tiny", 1, 4, 256, 64, sweep_frozen_heads(4, nf, seed), -0.05, seed=seed)
    if k in (1, 3):
        nf = 3 if n_frozen is None else n_frozen
        nm = "gpt2-124m-4k" if k == 1 else f"sweep-124m-4k-f{nf}"
        return Workload(nm, 8, 12, 4096, 64, sweep_frozen_heads(12, nf, seed), -0.05, seed=seed)
    if k == 2:
        nf = 8 if n_frozen is None else n_frozen
        return Workload("1b-8k", 4, 32, 8192, 64, sweep_frozen_heads(32, nf, seed), -0.01, seed=seed)
    if k == 4:
        nf = 8 if n_frozen is None else n_frozen
        return Workload("prefill-32k-d128", 1, 32, 32768, 128, sweep_frozen_heads(32, nf, seed),
                        -0.002, alpha0_spike=4.0, backward=False, seed=seed)
    if k == 5:
        nf = 3 if n_frozen is None else n_frozen
        return Workload("124m-4k-d128", 8, 12, 4096, 128, sweep_frozen_heads(12, nf, seed), -0.05, seed=seed)
    if k == 6:
        nf = 4 if n_frozen is None else n_frozen
        return Workload("1b-paper-8k-d96", 2, 16, 8192, 96, sweep_frozen_heads(16, nf, seed), -0.01, seed=seed)
    if k == 7:
        # grouped-query attention at the shape of the paper's GQA attention-operator timings (Appendix E.2): 32 query
        # heads on 8 shared key/value heads of dimension 128, batch 4, 4K context, forward only; 30 % of the query
        # heads replaced unless n_frozen says otherwise
        nf = 10 if n_frozen is None else n_frozen
        return Workload("gqa-32q-8kv-4k-d128", 4, 32, 4096, 128, sweep_frozen_heads(32, nf, seed), -0.01, seed=seed,
                        kv_group=4, backward=False)
    raise ValueError(f"unknown config {k}")


@dataclass
class Inputs:
    wl: Workload
    q: np.ndarray       # [B,H,T,D] uint16 (bf16 bits)
    k: np.ndarray       # [B,H/kv_group,T,D]
    v: np.ndarray
    do: np.ndarray      # [B,H,T,D] uint16 (bf16 bits); drawn even for forward-only workloads
    alpha: np.ndarray   # [H,Tp] float32 (rows of ordinary heads are zero)
    rho: np.ndarray     # [H,Tp] float32
    mask: np.ndarray = field(default=None)  # [H] uint8


def _normal_bf16(rng: np.random.Generator, shape) -> np.ndarray:
    out = np.empty(shape, dtype=np.uint16)
    flat = out.reshape(shape[0] * shape[1], -1)
    for r in range(flat.shape[0]):          # one (b,h) slab at a time keeps peak memory low
        flat[r] = f32_to_bf16_bits(rng.standard_normal(flat.shape[1], dtype=np.float32))
    return out


def generate(wl: Workload) -> Inputs:
    rng = np.random.default_rng(wl.seed)
    shape = (wl.B, wl.H, wl.T, wl.D)
    kv_shape = (wl.B, wl.H // wl.kv_group, wl.T, wl.D)
    qk_shape = (wl.B, wl.H - len(wl.frozen_heads), wl.T, wl.D)
    q = _normal_bf16(rng, qk_shape if wl.packed_qk else shape)
    k = _normal_bf16(rng, qk_shape if wl.packed_qk else kv_shape)
    v = _normal_bf16(rng, kv_shape)
    do = _normal_bf16(rng, shape)
    tp = wl.stored_len
    alpha = np.zeros((wl.H, tp), dtype=np.float32)
    rho = np.zeros((wl.H, tp), dtype=np.float32)
    d = np.arange(tp, dtype=np.float64)
    for h in wl.frozen_heads:
        a = rng.standard_normal(tp)
        noise = rng.standard_normal(tp)
        a[0] += wl.alpha0_spike
        alpha[h] = a.astype(np.float32)
        rho[h] = (wl.rho_slope * d + 0.1 * noise).astype(np.float32)
    return Inputs(wl, q, k, v, do, alpha, rho, wl.mask)


# --------------------------------------------------------------------------- inputs of the compact-pattern fitter
def mean_attention_maps(Hf: int, T: int, seed: int = 0, upper_fill: float = 0.0, pmax: float = 3.0) -> np.ndarray:
    """Synthetic stand-ins for calibration-time mean attention maps, float32 [Hf, T, T].

    Row i holds positive weights over keys j <= i that sum to one: a power-law decay in the distance i-j (exponent
    drawn per head from U(1,pmax), so far entries fall below the fitter's 1e-9 floor), a per-head weight on key 0
    (U(0,0.5), attention-sink-like), a per-key factor and element-wise log-normal noise (sigma 0.3), then scaled so
    that the row sums to one.  Entries above the diagonal are `upper_fill` (a consumer must ignore them).
    Draw order per head: exponent, sink weight, key factors [T], noise [T,T].
    """
    rng = np.random.default_rng(seed)
    out = np.empty((Hf, T, T), dtype=np.float32)
    i = np.arange(T)[:, None]
    j = np.arange(T)[None, :]
    causal = j <= i
    dist = np.where(causal, i - j, 0).astype(np.float64)
    for h in range(Hf):
        p = rng.uniform(1.0, pmax)
        sink = rng.uniform(0.0, 0.5)
        keyf = np.exp(0.5 * rng.standard_normal(T))
        noise = np.exp(0.3 * rng.standard_normal((T, T), dtype=np.float32).astype(np.float64))
        w = (1.0 + dist) ** (-p) * keyf[None, :] * noise
        w = np.where(causal, w, 0.0)
        w = w / w.sum(axis=1, keepdims=True) * (1.0 - sink)
        w[:, 0] += sink
        out[h] = np.where(causal, w, upper_fill).astype(np.float32)
    return out
