"""ctypes binding of libsaf_b200.so: the same names as the C ABI, argument marshalling only.

Tensors are passed as torch CUDA tensors (device memory and streams are torch's); every step of
the computation runs in the library's kernels.  There is no fallback: if the shared library is
missing or the device is not sm_100-class the calls raise.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libsaf_b200.so")

SAF_OK = 0
SAF_ERR_INVALID_ARG, SAF_ERR_UNSUPPORTED, SAF_ERR_CUDA, SAF_ERR_DEVICE_TIMEOUT, SAF_ERR_ARCH, SAF_ERR_NOMEM = range(1, 7)
SAF_BF16, SAF_F32 = 0, 1
SAF_KERNEL_FWD, SAF_KERNEL_BWD, SAF_KERNEL_BWD_PREP, SAF_KERNEL_BWD_FINALIZE, SAF_KERNEL_LOGZ, SAF_KERNEL_SCALE = range(6)
SAF_KERNEL_PGRAD, SAF_KERNEL_FIT, SAF_KERNEL_FIT_MARGINALS, SAF_KERNEL_CALIB, SAF_KERNEL_CALIB_FINALIZE = 6, 7, 8, 9, 10


class SafProblem(C.Structure):
    _fields_ = [("B", C.c_int32), ("H", C.c_int32), ("T", C.c_int32), ("D", C.c_int32), ("Tp", C.c_int32),
                ("softmax_scale", C.c_float), ("grad_dtype", C.c_int32), ("kv_group", C.c_int32),
                ("packed_qk", C.c_int32), ("o_dtype", C.c_int32),
                ("q_strides", C.c_int64 * 3), ("k_strides", C.c_int64 * 3), ("v_strides", C.c_int64 * 3),
                ("o_strides", C.c_int64 * 3)]


class SafError(RuntimeError):
    def __init__(self, code: int, what: str):
        self.code = code
        super().__init__(f"{what}: status {code} ({status_string(code)})")


_lib = None


def load_library() -> C.CDLL:
    """dlopen the shared library and declare the prototypes.  Raises if it has not been built."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise FileNotFoundError(f"{LIB_PATH} not built; run `python -m paper_2609_34650_b200.build`")
    lib = C.CDLL(LIB_PATH)
    vp, i32, u8p, f32p = C.c_void_p, C.c_int32, C.POINTER(C.c_uint8), C.c_void_p
    pp = C.POINTER(SafProblem)
    lib.saf_version.restype = C.c_int
    lib.saf_status_string.restype = C.c_char_p
    lib.saf_status_string.argtypes = [C.c_int]
    lib.saf_create.argtypes = [C.POINTER(vp), C.c_int]
    lib.saf_destroy.argtypes = [vp]
    lib.saf_pattern_prepare.argtypes = [vp, i32, i32, u8p, f32p, f32p, f32p, vp]
    lib.saf_hybrid_attn_fwd.argtypes = [vp, pp, vp, vp, vp, u8p, f32p, f32p, f32p, vp, f32p, vp]
    lib.saf_hybrid_attn_bwd.argtypes = [vp, pp, vp, vp, vp, vp, vp, f32p, u8p, f32p, f32p, f32p, vp, vp, vp, vp]
    lib.saf_hybrid_attn_step_host.argtypes = [vp, pp, vp, vp, vp, vp, u8p, f32p, f32p, i32, vp, f32p, vp, vp, vp]
    lib.saf_pattern_grad.argtypes = [vp, pp, vp, vp, vp, u8p, f32p, f32p, f32p, f32p, f32p, vp]
    lib.saf_fit_marginals.argtypes = [vp, i32, i32, vp, C.c_float, vp, vp, vp, vp]
    lib.saf_fit_compact.argtypes = [vp, i32, i32, vp, vp, vp, i32, C.c_double, vp, vp, vp, C.c_int64, vp, vp, vp]
    lib.saf_calib_accumulate.argtypes = [vp, pp, vp, vp, vp, vp, vp, vp, i32, vp]
    lib.saf_calib_finalize.argtypes = [vp, i32, i32, C.c_int64, vp, vp, vp, vp, vp, vp]
    lib.saf_last_device_status.argtypes = [vp, C.POINTER(C.c_int32)]
    lib.saf_set_profiling.argtypes = [vp, i32]
    lib.saf_get_kernel_time.argtypes = [vp, i32, C.POINTER(C.c_float), C.POINTER(C.c_int32)]
    lib.saf_pattern_logz_static.argtypes = [i32, i32, i32, u8p, f32p, f32p, f32p, vp]
    lib.saf_pattern_logz_static.restype = C.c_int
    lib.saf_build_worklist.argtypes = [i32, i32, i32, u8p, i32, i32, i32, C.POINTER(C.c_int32), C.POINTER(C.c_int32)]
    for name in ("saf_create", "saf_destroy", "saf_pattern_prepare", "saf_hybrid_attn_fwd", "saf_hybrid_attn_bwd",
                 "saf_hybrid_attn_step_host", "saf_last_device_status", "saf_build_worklist", "saf_set_profiling",
                 "saf_get_kernel_time", "saf_pattern_grad", "saf_fit_marginals", "saf_fit_compact", "saf_calib_accumulate", "saf_calib_finalize"):
        getattr(lib, name).restype = C.c_int
    _lib = lib
    return lib


def status_string(code: int) -> str:
    return load_library().saf_status_string(code).decode()


def saf_version() -> int:
    return load_library().saf_version()


def _check(code: int, what: str):
    if code != SAF_OK:
        raise SafError(code, what)


def _mask_ptr(mask):
    m = np.ascontiguousarray(np.asarray(mask, dtype=np.uint8))
    return m, m.ctypes.data_as(C.POINTER(C.c_uint8))


def _ptr(t):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream():
    import torch
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def saf_build_worklist(B, H, T, mask, backward, n_ctas, frozen_weight_pct=60):
    """Host-only: returns (items [n,4] int32 = (b,h,block,kind), offsets [n_ctas+1] int32)."""
    lib = load_library()
    nblk = (T + 127) // 128
    items = np.zeros((B * H * nblk, 4), dtype=np.int32)
    offsets = np.zeros(n_ctas + 1, dtype=np.int32)
    m, mp = _mask_ptr(mask)
    _check(lib.saf_build_worklist(B, H, T, mp, int(backward), n_ctas, frozen_weight_pct,
                                  items.ctypes.data_as(C.POINTER(C.c_int32)),
                                  offsets.ctypes.data_as(C.POINTER(C.c_int32))), "saf_build_worklist")
    return items, offsets


def saf_pattern_logz_static(device, mask, alpha, rho, logZ_out):
    """Row normalisers through the entry point that allocates nothing (no context; at most 1024 heads)."""
    H, Tp = alpha.shape
    m, mp = _mask_ptr(mask)
    _check(load_library().saf_pattern_logz_static(device, H, Tp, mp, _ptr(alpha), _ptr(rho), _ptr(logZ_out), _stream()),
           "saf_pattern_logz_static")


def make_problem(q_like, Tp, softmax_scale=0.0, grad_dtype=SAF_F32, k_like=None, v_like=None, o_like=None,
                 kv_group=1, packed_qk=False, H=None, o_dtype=SAF_BF16):
    """saf_problem from [B,H,T,D] torch tensors (any strides with a unit feature stride); with kv_group > 1
    k_like / v_like are the [B,H/kv_group,T,D] shared key/value tensors."""
    B, Hq, T, D = q_like.shape
    H = Hq if H is None else H              # packed_qk: q_like has only the ordinary heads, pass H
    p = SafProblem()
    p.B, p.H, p.T, p.D, p.Tp = B, H, T, D, Tp
    p.softmax_scale = softmax_scale
    p.grad_dtype = grad_dtype
    p.kv_group = kv_group
    p.packed_qk = int(packed_qk)
    p.o_dtype = o_dtype
    for name, t in (("q_strides", q_like), ("k_strides", k_like if k_like is not None else q_like),
                    ("v_strides", v_like if v_like is not None else q_like),
                    ("o_strides", o_like if o_like is not None else q_like)):
        assert t.stride(3) == 1, "feature stride must be 1"
        arr = getattr(p, name)
        arr[0], arr[1], arr[2] = t.stride(0), t.stride(1), t.stride(2)
    return p


class Context:
    """Owns a saf_ctx on one CUDA device."""

    def __init__(self, device: int = 0):
        self._lib = load_library()
        self._h = C.c_void_p()
        _check(self._lib.saf_create(C.byref(self._h), device), "saf_create")

    def close(self):
        if self._h:
            self._lib.saf_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def saf_pattern_prepare(self, mask, alpha, rho, logZ_out):
        H, Tp = alpha.shape
        m, mp = _mask_ptr(mask)
        _check(self._lib.saf_pattern_prepare(self._h, H, Tp, mp, _ptr(alpha), _ptr(rho), _ptr(logZ_out), _stream()),
               "saf_pattern_prepare")

    def saf_hybrid_attn_fwd(self, prob, Q, K, V, mask, alpha, rho, logZ, O, LSE):
        m, mp = _mask_ptr(mask)
        _check(self._lib.saf_hybrid_attn_fwd(self._h, C.byref(prob), _ptr(Q), _ptr(K), _ptr(V), mp, _ptr(alpha),
                                             _ptr(rho), _ptr(logZ), _ptr(O), _ptr(LSE), _stream()),
               "saf_hybrid_attn_fwd")

    def saf_hybrid_attn_bwd(self, prob, Q, K, V, O, dO, LSE, mask, alpha, rho, logZ, dQ, dK, dV):
        m, mp = _mask_ptr(mask)
        _check(self._lib.saf_hybrid_attn_bwd(self._h, C.byref(prob), _ptr(Q), _ptr(K), _ptr(V), _ptr(O), _ptr(dO),
                                             _ptr(LSE), mp, _ptr(alpha), _ptr(rho), _ptr(logZ), _ptr(dQ), _ptr(dK),
                                             _ptr(dV), _stream()), "saf_hybrid_attn_bwd")

    def saf_pattern_grad(self, prob, V, O, dO, mask, alpha, rho, logZ, dalpha, drho):
        m, mp = _mask_ptr(mask)
        _check(self._lib.saf_pattern_grad(self._h, C.byref(prob), _ptr(V), _ptr(O), _ptr(dO), mp, _ptr(alpha),
                                          _ptr(rho), _ptr(logZ), _ptr(dalpha), _ptr(drho), _stream()),
               "saf_pattern_grad")

    def saf_fit_marginals(self, Hf, T, mean_attn, floor_value, eta_abs, eta_rel, plogp):
        _check(self._lib.saf_fit_marginals(self._h, int(Hf), int(T), _ptr(mean_attn), float(floor_value), _ptr(eta_abs),
                                           _ptr(eta_rel), _ptr(plogp), _stream()), "saf_fit_marginals")

    def saf_fit_compact(self, Hf, T, eta_abs, eta_rel, plogp, steps, lr, alpha, rho, logZ, out_stride, loss, kl):
        _check(self._lib.saf_fit_compact(self._h, int(Hf), int(T), _ptr(eta_abs), _ptr(eta_rel), _ptr(plogp),
                                         int(steps), float(lr), _ptr(alpha), _ptr(rho), _ptr(logZ), int(out_stride),
                                         _ptr(loss), _ptr(kl), _stream()), "saf_fit_compact")

    def saf_calib_accumulate(self, prob, Q, K, LSE, mean_sum, sumsq, sum_plogp, accumulate):
        _check(self._lib.saf_calib_accumulate(self._h, C.byref(prob), _ptr(Q), _ptr(K), _ptr(LSE), _ptr(mean_sum),
                                              _ptr(sumsq), _ptr(sum_plogp), int(bool(accumulate)), _stream()),
               "saf_calib_accumulate")

    def saf_calib_finalize(self, H, T, n_total, mean, sumsq, sum_plogp, s_var, s_kl):
        _check(self._lib.saf_calib_finalize(self._h, int(H), int(T), int(n_total), _ptr(mean), _ptr(sumsq),
                                            _ptr(sum_plogp), _ptr(s_var), _ptr(s_kl), _stream()), "saf_calib_finalize")

    def saf_hybrid_attn_step_host(self, prob, Q, K, V, dO, mask, alpha, rho, prepare, O, LSE, dQ, dK, dV):
        """All tensor arguments are HOST tensors (torch CPU tensors, ideally pinned) or None."""
        m, mp = _mask_ptr(mask)
        _check(self._lib.saf_hybrid_attn_step_host(self._h, C.byref(prob), _ptr(Q), _ptr(K), _ptr(V), _ptr(dO), mp,
                                                   _ptr(alpha), _ptr(rho), int(prepare), _ptr(O), _ptr(LSE), _ptr(dQ),
                                                   _ptr(dK), _ptr(dV)), "saf_hybrid_attn_step_host")

    def saf_set_profiling(self, enable: bool):
        _check(self._lib.saf_set_profiling(self._h, int(enable)), "saf_set_profiling")

    def saf_get_kernel_time(self, which: int):
        """(total milliseconds, launches) of kernel `which` since the previous query."""
        ms, n = C.c_float(0.0), C.c_int32(0)
        _check(self._lib.saf_get_kernel_time(self._h, which, C.byref(ms), C.byref(n)), "saf_get_kernel_time")
        return ms.value, n.value

    def saf_last_device_status(self):
        detail = C.c_int32(0)
        code = self._lib.saf_last_device_status(self._h, C.byref(detail))
        return code, detail.value
