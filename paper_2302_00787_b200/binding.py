"""Thin ctypes binding of libfsharp.so: the same names as include/fsharp.h, argument
marshalling only.  torch is used for device memory and streams; every step of the path
runs in the library's CUDA kernels.  There is no CPU fallback: if the library is missing
or a call fails, an exception is raised."""
from __future__ import annotations

import ctypes as C
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
# FSHARP_LIB selects another build of the library (the debug build with index checks: lib/libfsharp_debug.so)
LIB_PATH = os.environ.get("FSHARP_LIB") or os.path.join(_HERE, "lib", "libfsharp.so")

FSHARP_F32, FSHARP_BF16 = 0, 1
VARIANTS = {"posrf": 0, "gerf": 1, "saderf": 2, "aderf": 3, "sderf": 4}
POOL_PER_BH, POOL_PER_HEAD = 0, 1
STAB_NONE, STAB_ROW, STAB_GROUP = 0, 1, 2
IMPL_AUTO, IMPL_SIMT, IMPL_TENSOR = 0, 1, 2

EXPORTS = [
    "fsharp_create", "fsharp_destroy", "fsharp_set_stream", "fsharp_set_impl", "fsharp_status",
    "fsharp_launch_count", "fsharp_workspace_bytes", "fsharp_strerror", "fsharp_stats_doubles",
    "fsharp_params_doubles", "fsharp_stats", "fsharp_fit_params", "fsharp_featurize", "fsharp_attend",
    "fsharp_forward_host", "fsharp_pair_estimate", "fsharp_set_timing", "fsharp_read_timing",
    "fsharp_kernel_name", "fsharp_static_scratch_bytes", "fsharp_featurize_static", "fsharp_kernel_apply",
    "fsharp_key_state_splits", "fsharp_attend_key_state", "fsharp_attend_with_state", "fsharp_attend_backward",
    "fsharp_selftest_bounded_wait",
]


class FsharpError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {strerror(code)} ({code})")


class fsharp_dims(C.Structure):
    _fields_ = [("B", C.c_int32), ("H", C.c_int32), ("Lq", C.c_int32), ("Lk", C.c_int32),
                ("d", C.c_int32), ("dv", C.c_int32), ("M", C.c_int32), ("pool", C.c_int32),
                ("q_stride", C.c_int64 * 3), ("k_stride", C.c_int64 * 3),
                ("v_stride", C.c_int64 * 3), ("y_stride", C.c_int64 * 3),
                ("omega_head_stride", C.c_int64)]


_lib = None


def load_library() -> C.CDLL:
    """Loads lib/libfsharp.so (built by build.py); raises if it is not there."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise FileNotFoundError(
            f"{LIB_PATH} not found: build it with `python -m paper_2302_00787_b200.build` "
            "(there is no fallback implementation)")
    lib = C.CDLL(LIB_PATH)
    vp, i32, i64, f32, f64 = C.c_void_p, C.c_int, C.c_int64, C.c_float, C.c_double
    dims_p = C.POINTER(fsharp_dims)
    sig = {
        "fsharp_create": (i32, [C.POINTER(vp), i32, vp]),
        "fsharp_destroy": (i32, [vp]),
        "fsharp_set_stream": (i32, [vp, vp]),
        "fsharp_set_impl": (i32, [vp, i32]),
        "fsharp_status": (i32, [vp, C.POINTER(i32)]),
        "fsharp_launch_count": (i64, [vp]),
        "fsharp_workspace_bytes": (C.c_size_t, [vp]),
        "fsharp_strerror": (C.c_char_p, [i32]),
        "fsharp_stats_doubles": (C.c_size_t, [i32]),
        "fsharp_params_doubles": (C.c_size_t, [i32]),
        "fsharp_stats": (i32, [vp, vp, vp, dims_p, i32, f32, vp]),
        "fsharp_fit_params": (i32, [vp, vp, i32, i32, i32, f64, vp]),
        "fsharp_featurize": (i32, [vp, vp, vp, vp, i32, dims_p, i32, f32, i32, vp, vp]),
        "fsharp_attend": (i32, [vp, vp, vp, vp, vp, vp, dims_p, i32, i32, i32, f32, vp]),
        "fsharp_kernel_apply": (i32, [vp, vp, vp, vp, vp, vp, f64, dims_p, i32, f32, vp]),
        "fsharp_attend_backward": (i32, [vp, vp, vp, vp, vp, vp, vp, dims_p, i32, i32, i32, f32, vp, vp, vp]),
        "fsharp_key_state_splits": (i32, [vp, dims_p]),
        "fsharp_attend_key_state": (i32, [vp, vp, vp, vp, vp, dims_p, i32, f32, vp, vp]),
        "fsharp_attend_with_state": (i32, [vp, vp, vp, vp, vp, vp, dims_p, i32, i32, f32, vp, vp, i32, vp]),
        "fsharp_forward_host": (i32, [vp, vp, vp, vp, vp, dims_p, i32, i32, i32, i32, f32, vp]),
        "fsharp_pair_estimate": (i32, [vp, vp, vp, vp, vp, i64, i32, i32, i32, vp, vp, vp]),
        "fsharp_set_timing": (i32, [vp, i32]),
        "fsharp_selftest_bounded_wait": (i32, [vp, i32]),
        "fsharp_read_timing": (i32, [vp, i32, C.POINTER(C.c_float), C.POINTER(i32)]),
        "fsharp_kernel_name": (C.c_char_p, [i32]),
        "fsharp_static_scratch_bytes": (C.c_size_t, []),
        "fsharp_featurize_static": (i32, [vp, vp, vp, vp, i32, dims_p, i32, f32, i32, vp, vp, vp]),
    }
    for name, (res, args) in sig.items():
        fn = getattr(lib, name)
        fn.restype = res
        fn.argtypes = args
    _lib = lib
    return lib


def strerror(code: int) -> str:
    return load_library().fsharp_strerror(code).decode()


def stats_doubles(d: int) -> int:
    return load_library().fsharp_stats_doubles(d)


def params_doubles(d: int) -> int:
    return load_library().fsharp_params_doubles(d)


def _check(rc: int, where: str) -> None:
    if rc != 0:
        raise FsharpError(rc, where)


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return FSHARP_F32
    if t.dtype == torch.bfloat16:
        return FSHARP_BF16
    raise TypeError(f"unsupported dtype {t.dtype}")


def _strides(t: torch.Tensor):
    """Element strides (batch, head, token) of a [B,H,L,inner] tensor, innermost contiguous."""
    if t.dim() != 4 or (t.shape[3] > 1 and t.stride(3) != 1):
        raise ValueError("expected a [B, H, L, inner] tensor whose last dimension is contiguous")
    return (C.c_int64 * 3)(t.stride(0), t.stride(1), t.stride(2))


def make_dims(B, H, Lq, Lk, d, dv, M, pool=POOL_PER_BH, q=None, k=None, v=None, y=None,
              omega_head_stride=0) -> fsharp_dims:
    dm = fsharp_dims()
    dm.B, dm.H, dm.Lq, dm.Lk, dm.d, dm.dv, dm.M, dm.pool = B, H, Lq, Lk, d, dv, M, pool
    for name, t in (("q_stride", q), ("k_stride", k), ("v_stride", v), ("y_stride", y)):
        if t is not None:
            setattr(dm, name, _strides(t))
    dm.omega_head_stride = omega_head_stride
    return dm


class Context:
    """Owns one fsharp_ctx bound to a CUDA device and stream."""

    def __init__(self, device: int = 0, stream: torch.cuda.Stream | None = None):
        self.lib = load_library()
        if not torch.cuda.is_available():
            raise RuntimeError("a CUDA device is required (no CPU implementation exists)")
        self.device = device
        self._h = C.c_void_p()
        sp = stream.cuda_stream if stream is not None else torch.cuda.current_stream(device).cuda_stream
        _check(self.lib.fsharp_create(C.byref(self._h), device, C.c_void_p(sp)), "fsharp_create")

    def close(self):
        if getattr(self, "_h", None) is not None and self._h.value:
            self.lib.fsharp_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- plumbing
    def set_stream(self, stream: torch.cuda.Stream):
        _check(self.lib.fsharp_set_stream(self._h, C.c_void_p(stream.cuda_stream)), "fsharp_set_stream")

    def set_impl(self, impl: int):
        _check(self.lib.fsharp_set_impl(self._h, impl), "fsharp_set_impl")

    def status(self) -> int:
        code = C.c_int(0)
        _check(self.lib.fsharp_status(self._h, C.byref(code)), "fsharp_status")
        return code.value

    def launch_count(self) -> int:
        return self.lib.fsharp_launch_count(self._h)

    def workspace_bytes(self) -> int:
        return self.lib.fsharp_workspace_bytes(self._h)

    def selftest_bounded_wait(self, limit_us: int = 1000):
        _check(self.lib.fsharp_selftest_bounded_wait(self._h, limit_us), "fsharp_selftest_bounded_wait")

    def set_timing(self, on: bool):
        _check(self.lib.fsharp_set_timing(self._h, int(on)), "fsharp_set_timing")

    def read_timing(self) -> dict:
        """{kernel name: (total milliseconds, launches)} since the last read."""
        cap = 32
        ms = (C.c_float * cap)()
        n = (C.c_int * cap)()
        _check(self.lib.fsharp_read_timing(self._h, cap, ms, n), "fsharp_read_timing")
        out = {}
        for i in range(cap):
            if n[i]:
                out[self.lib.fsharp_kernel_name(i).decode()] = (float(ms[i]), int(n[i]))
        return out

    # -- the path
    def fsharp_stats(self, Q, K, pool=POOL_PER_BH, qk_scale=1.0, out=None):
        B, H, Lq, d = Q.shape
        Lk = K.shape[2]
        dm = make_dims(B, H, Lq, Lk, d, d, 16, pool, q=Q, k=K)
        G = B * H if pool == POOL_PER_BH else H
        if out is None:
            out = torch.empty(G, stats_doubles(d), dtype=torch.float64, device=Q.device)
        _check(self.lib.fsharp_stats(self._h, Q.data_ptr(), K.data_ptr(), C.byref(dm), _dtype_code(Q),
                                     qk_scale, out.data_ptr()), "fsharp_stats")
        return out

    def fsharp_fit_params(self, stats, d, variant, ridge=0.0, out=None):
        G = stats.shape[0]
        v = VARIANTS[variant] if isinstance(variant, str) else variant
        if out is None:
            out = torch.empty(G, params_doubles(d), dtype=torch.float64, device=stats.device)
        _check(self.lib.fsharp_fit_params(self._h, stats.data_ptr(), G, d, v, ridge, out.data_ptr()),
               "fsharp_fit_params")
        return out

    def fsharp_featurize(self, X, Omega, params, side, pool=POOL_PER_BH, qk_scale=1.0, stab=STAB_ROW):
        B, H, L, d = X.shape
        M = Omega.shape[-2]
        ohs = Omega.stride(0) if Omega.dim() == 3 else 0
        dm = make_dims(B, H, L, L, d, d, M, pool, q=X, k=X, omega_head_stride=ohs)
        phi = torch.empty(B, H, L, M, dtype=torch.float32, device=X.device)
        ls = None
        if stab == STAB_ROW:
            ls = torch.empty(B, H, L, dtype=torch.float32, device=X.device)
        elif stab == STAB_GROUP:
            ls = torch.empty(B, H, dtype=torch.float32, device=X.device)
        _check(self.lib.fsharp_featurize(self._h, X.data_ptr(), Omega.data_ptr(), params.data_ptr(), side,
                                         C.byref(dm), _dtype_code(X), qk_scale, stab, phi.data_ptr(),
                                         ls.data_ptr() if ls is not None else None), "fsharp_featurize")
        return phi, ls

    def fsharp_attend(self, Q, K, V, Omega, params, causal=False, chunk=0, pool=POOL_PER_BH, qk_scale=1.0,
                      out=None):
        B, H, Lq, d = Q.shape
        Lk, dv = K.shape[2], V.shape[3]
        M = Omega.shape[-2]
        ohs = Omega.stride(0) if Omega.dim() == 3 else 0
        if out is None:
            out = torch.empty(B, H, Lq, dv, dtype=Q.dtype, device=Q.device)
        dm = make_dims(B, H, Lq, Lk, d, dv, M, pool, q=Q, k=K, v=V, y=out, omega_head_stride=ohs)
        _check(self.lib.fsharp_attend(self._h, Q.data_ptr(), K.data_ptr(), V.data_ptr(), Omega.data_ptr(),
                                      params.data_ptr(), C.byref(dm), _dtype_code(Q), int(bool(causal)), chunk,
                                      qk_scale, out.data_ptr()), "fsharp_attend")
        return out

    def fsharp_attend_backward(self, Q, K, V, dY, Omega, params, causal=False, chunk=0, pool=POOL_PER_BH,
                               qk_scale=1.0):
        """(dQ, dK, dV) for the cotangent dY of fsharp_attend's Y; each gradient has its tensor's shape and strides."""
        B, H, Lq, d = Q.shape
        Lk, dv = K.shape[2], V.shape[3]
        M = Omega.shape[-2]
        ohs = Omega.stride(0) if Omega.dim() == 3 else 0
        dQ, dK, dV = (torch.empty_strided(t.shape, t.stride(), dtype=t.dtype, device=t.device) for t in (Q, K, V))
        dm = make_dims(B, H, Lq, Lk, d, dv, M, pool, q=Q, k=K, v=V, y=dY, omega_head_stride=ohs)
        _check(self.lib.fsharp_attend_backward(self._h, Q.data_ptr(), K.data_ptr(), V.data_ptr(), dY.data_ptr(),
                                               Omega.data_ptr(), params.data_ptr(), C.byref(dm), _dtype_code(Q),
                                               int(bool(causal)), chunk, qk_scale, dQ.data_ptr(), dK.data_ptr(),
                                               dV.data_ptr()), "fsharp_attend_backward")
        return dQ, dK, dV

    def fsharp_attend_key_state(self, K, V, Omega, params, pool=POOL_PER_BH, qk_scale=1.0):
        """Key-side sums of this call's keys: (state [B*H, ns, 80, 256] fp32, shifts [B*H, ns, 2] fp32)."""
        B, H, Lk, d = K.shape
        dv, M = V.shape[3], Omega.shape[-2]
        ohs = Omega.stride(0) if Omega.dim() == 3 else 0
        dm = make_dims(B, H, Lk, Lk, d, dv, M, pool, q=K, k=K, v=V, omega_head_stride=ohs)
        ns = self.lib.fsharp_key_state_splits(self._h, C.byref(dm))
        _check(min(ns, 0), "fsharp_key_state_splits")
        state = torch.empty(B * H, ns, 80, 256, dtype=torch.float32, device=K.device)
        shifts = torch.empty(B * H, ns, 2, dtype=torch.float32, device=K.device)
        _check(self.lib.fsharp_attend_key_state(self._h, K.data_ptr(), V.data_ptr(), Omega.data_ptr(), params.data_ptr(),
                                                C.byref(dm), _dtype_code(K), qk_scale, state.data_ptr(),
                                                shifts.data_ptr()), "fsharp_attend_key_state")
        return state, shifts

    def fsharp_attend_with_state(self, Q, K, V, Omega, params, states, shifts, causal=False, pool=POOL_PER_BH,
                                 qk_scale=1.0, out=None):
        """Attention of Q over the keys behind `states` (and, causal, over K, V under the mask).  states
        [B*H, n, 80, 256] and shifts [B*H, n, 2] fp32 contiguous, or None (causal only: nothing precedes)."""
        B, H, Lq, d = Q.shape
        M = Omega.shape[-2]
        ohs = Omega.stride(0) if Omega.dim() == 3 else 0
        n = 0 if states is None else states.shape[1]
        if n:
            if not (states.is_contiguous() and shifts.is_contiguous() and states.dtype == torch.float32
                    and shifts.dtype == torch.float32 and tuple(states.shape) == (B * H, n, 80, 256)
                    and tuple(shifts.shape) == (B * H, n, 2)):
                raise ValueError("states / shifts: contiguous fp32 [B*H, n, 80, 256] / [B*H, n, 2]")
        dv = V.shape[3] if V is not None else 64
        if out is None:
            out = torch.empty(B, H, Lq, dv, dtype=Q.dtype, device=Q.device)
        if causal:
            dm = make_dims(B, H, Lq, K.shape[2], d, dv, M, pool, q=Q, k=K, v=V, y=out, omega_head_stride=ohs)
        else:
            dm = make_dims(B, H, Lq, Lq, d, dv, M, pool, q=Q, k=Q, v=out, y=out, omega_head_stride=ohs)
        _check(self.lib.fsharp_attend_with_state(
            self._h, Q.data_ptr(), K.data_ptr() if causal else None, V.data_ptr() if causal else None, Omega.data_ptr(),
            params.data_ptr(), C.byref(dm), _dtype_code(Q), int(bool(causal)), qk_scale,
            states.data_ptr() if n else None, shifts.data_ptr() if n else None, n, out.data_ptr()),
            "fsharp_attend_with_state")
        return out

    def fsharp_kernel_apply(self, X, Y, Cmat, Omega, params, alpha=0.0, pool=POOL_PER_BH, qk_scale=1.0, out=None):
        B, H, Lq, d = X.shape
        Lk, dv = Y.shape[2], Cmat.shape[3]
        M = Omega.shape[-2]
        ohs = Omega.stride(0) if Omega.dim() == 3 else 0
        if out is None:
            out = torch.empty(B, H, Lq, dv, dtype=X.dtype, device=X.device)
        dm = make_dims(B, H, Lq, Lk, d, dv, M, pool, q=X, k=Y, v=Cmat, y=out, omega_head_stride=ohs)
        _check(self.lib.fsharp_kernel_apply(self._h, X.data_ptr(), Y.data_ptr(), Cmat.data_ptr(), Omega.data_ptr(),
                                            params.data_ptr(), float(alpha), C.byref(dm), _dtype_code(X), qk_scale,
                                            out.data_ptr()), "fsharp_kernel_apply")
        return out

    def fsharp_forward_host(self, Q, K, V, Omega, variant, causal=False, chunk=0, pool=POOL_PER_BH,
                            qk_scale=1.0, out=None):
        """Q, K, V, Omega, out: HOST tensors (dense; pinned memory recommended)."""
        for t in (Q, K, V, Omega):
            if t.is_cuda or not t.is_contiguous():
                raise ValueError("fsharp_forward_host takes dense host tensors")
        B, H, Lq, d = Q.shape
        Lk, dv = K.shape[2], V.shape[3]
        M = Omega.shape[0]
        if out is None:
            out = torch.empty(B, H, Lq, dv, dtype=Q.dtype).pin_memory()
        dm = make_dims(B, H, Lq, Lk, d, dv, M, pool)
        v = VARIANTS[variant] if isinstance(variant, str) else variant
        _check(self.lib.fsharp_forward_host(self._h, Q.data_ptr(), K.data_ptr(), V.data_ptr(), Omega.data_ptr(),
                                            C.byref(dm), _dtype_code(Q), v, int(bool(causal)), chunk, qk_scale,
                                            out.data_ptr()), "fsharp_forward_host")
        return out

    def fsharp_pair_estimate(self, X, Y, Omega, params, want_variance=True, want_pooled=False, est=None):
        """Returns (est [R, npairs], var_cf [npairs] or None) and, with want_pooled, a third item: a float64
        tensor [2] = (pooled empirical, pooled closed-form) relative variance."""
        npairs, d = X.shape
        R, M = Omega.shape[0], Omega.shape[1]
        if est is None:
            est = torch.empty(R, npairs, dtype=torch.float32, device=X.device)
        var = torch.empty(npairs, dtype=torch.float64, device=X.device) if (want_variance or want_pooled) else None
        pooled = torch.empty(2, dtype=torch.float64, device=X.device) if want_pooled else None
        _check(self.lib.fsharp_pair_estimate(self._h, X.data_ptr(), Y.data_ptr(), Omega.data_ptr(),
                                             params.data_ptr(), npairs, d, M, R, est.data_ptr(),
                                             var.data_ptr() if var is not None else None,
                                             pooled.data_ptr() if pooled is not None else None), "fsharp_pair_estimate")
        return (est, var, pooled) if want_pooled else (est, var)


def static_scratch_bytes() -> int:
    return load_library().fsharp_static_scratch_bytes()


def fsharp_featurize_static(X, Omega, params, side, phi, logscale=None, pool=POOL_PER_BH, qk_scale=1.0,
                            stab=STAB_ROW, stream=None, device_status=None) -> int:
    """The feature map without any device allocation by the library: the caller supplies the
    outputs (phi [B,H,L,M] float32, logscale as for fsharp_featurize) and the library's fixed
    in-module scratch is used.  Returns the C return code instead of raising, so a caller can
    test for the size limit (-10)."""
    lib = load_library()
    B, H, L, d = X.shape
    M = Omega.shape[-2]
    ohs = Omega.stride(0) if Omega.dim() == 3 else 0
    dm = make_dims(B, H, L, L, d, d, M, pool, q=X, k=X, omega_head_stride=ohs)

    # the kernels write through these pointers unchecked: refuse anything they would overrun
    def need(t, name, dtype, shape):
        if t.device != X.device or t.dtype != dtype or tuple(t.shape) != shape or not t.is_contiguous():
            raise ValueError(f"{name}: expected a contiguous {dtype} tensor of shape {shape} on {X.device}")
    need(phi, "phi", torch.float32, (B, H, L, M))
    if stab == STAB_ROW:
        if logscale is not None:
            need(logscale, "logscale", torch.float32, (B, H, L))
    elif stab == STAB_GROUP:
        if logscale is not None:
            need(logscale, "logscale", torch.float32, (B, H))
    if device_status is not None:
        need(device_status, "device_status", torch.int32, (1,))
    sp = stream.cuda_stream if stream is not None else torch.cuda.current_stream(X.device).cuda_stream
    with torch.cuda.device(X.device):          # the entry point launches on the current device
        return lib.fsharp_featurize_static(
            C.c_void_p(sp), X.data_ptr(), Omega.data_ptr(), params.data_ptr(), side, C.byref(dm), _dtype_code(X),
            qk_scale, stab, phi.data_ptr(), logscale.data_ptr() if logscale is not None else None,
            device_status.data_ptr() if device_status is not None else None)


def unpack_params(blob: torch.Tensor, d: int):
    """Splits one group's parameter blob (a 1-D float64 tensor or array) into named pieces."""
    b = blob.detach().cpu().numpy() if isinstance(blob, torch.Tensor) else blob
    dd = d * d
    t = b[5 * dd:]
    return {"A": b[0:dd].reshape(d, d), "B1": b[dd:2 * dd].reshape(d, d), "B2": b[2 * dd:3 * dd].reshape(d, d),
            "C1": b[3 * dd:4 * dd].reshape(d, d), "C2": b[4 * dd:5 * dd].reshape(d, d),
            "logD": float(t[0]), "objective": float(t[1]), "phi": float(t[2])}


def pack_params(p: dict, d: int):
    """Builds a parameter blob (numpy float64) from matrices A, B1, B2, C1, C2 and logD."""
    import numpy as np
    out = np.zeros(5 * d * d + 8, dtype=np.float64)
    for i, k in enumerate(("A", "B1", "B2", "C1", "C2")):
        out[i * d * d:(i + 1) * d * d] = np.asarray(p[k], dtype=np.float64).reshape(-1)
    t = out[5 * d * d:]
    t[0] = p["logD"]
    t[1] = p.get("objective", 0.0)
    return out
