"""ctypes binding of libada.so -- same names as include/ada.h, marshalling only.

Every step of the selection runs inside the CUDA library; this module converts
torch tensors to pointers, allocates output tensors, and raises on any
non-zero status.  There is no fallback: if the shared library has not been
built (python -m paper_2605_03110_b200.build) loading fails loudly.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libada.so")

ADA_OK = 0
ADA_F32, ADA_BF16 = 0, 1
ADA_CROSS_CAUSAL = 1
ADA_ATTN_CAUSAL = 1
ADA_ENGINE_AUTO, ADA_ENGINE_FFMA, ADA_ENGINE_TCGEN05, ADA_ENGINE_TCGEN05_PAIR = 0, 1, 2, 3

SYMBOLS = [
    "ada_create", "ada_destroy", "ada_set_engine", "ada_normalize", "ada_select_full",
    "ada_cascade_step", "ada_select_full_host", "ada_cascade_step_host", "ada_gram_op_count",
    "ada_device_status", "ada_profile_enable", "ada_profile_read", "ada_status_string",
    "ada_select_full_noalloc", "ada_set_cooperative", "ada_selftest_wait_timeout", "ada_nearest_rep",
    "ada_select_full_heads", "ada_cascade_step_heads", "ada_set_dependent_launch",
    "ada_cascade_step_adaptive", "ada_attention_reps", "ada_set_row_compaction",
]
ADA_NOALLOC_MAX_T = 16384

_lib = None


class TauPolicy(C.Structure):
    """ada_tau_policy: tau' = clip(tau + gain * (target_turnover - rho), tau_min, tau_max)."""
    _fields_ = [("target_turnover", C.c_double), ("gain", C.c_double), ("tau_min", C.c_double),
                ("tau_max", C.c_double)]


class AdaError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {status_string(status)} ({status})")


def lib() -> C.CDLL:
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(
                f"{LIB_PATH} is missing: build it with `python -m paper_2605_03110_b200.build`; "
                "there is no CPU fallback")
        L = C.CDLL(LIB_PATH)
        vp, i64, i32p, fp = C.c_void_p, C.c_int64, C.c_void_p, C.c_void_p
        L.ada_create.argtypes = [C.POINTER(vp), C.c_int, i64, i64, i64, C.c_int]
        L.ada_destroy.argtypes = [vp]
        L.ada_set_engine.argtypes = [vp, C.c_int]
        L.ada_set_cooperative.argtypes = [vp, C.c_int]
        L.ada_set_dependent_launch.argtypes = [vp, C.c_int]
        L.ada_set_row_compaction.argtypes = [vp, i64]
        L.ada_selftest_wait_timeout.argtypes = [vp, C.c_int, vp]
        L.ada_normalize.argtypes = [vp, vp, i64, i64, i64, i64, C.c_int, vp, fp, i32p, i32p, vp, vp]
        L.ada_select_full.argtypes = [vp, vp, i64, i64, i64, i64, C.c_int, C.c_double, i32p, i32p,
                                      fp, vp]
        L.ada_cascade_step.argtypes = [vp, vp, i64, i64, i64, i64, C.c_int, C.c_double,
                                       i32p, i32p, i32p, i32p, i32p, i32p, i32p, i32p, fp, fp,
                                       C.c_uint32, vp]
        L.ada_cascade_step_adaptive.argtypes = [vp, vp, i64, i64, i64, i64, C.c_int, vp,
                                                C.POINTER(TauPolicy), i32p, i32p, i32p, i32p, i32p,
                                                i32p, i32p, i32p, fp, fp, fp, C.c_uint32, vp]
        L.ada_select_full_heads.argtypes = L.ada_select_full.argtypes
        L.ada_cascade_step_heads.argtypes = L.ada_cascade_step.argtypes
        L.ada_nearest_rep.argtypes = [vp, vp, i64, i64, i64, i64, C.c_int, i32p, i32p, i32p, fp, vp]
        L.ada_attention_reps.argtypes = [vp, vp, vp, vp, i64, i64, i64, i64, C.c_int, i32p, i32p, i32p, fp,
                                         i64, C.c_uint32, vp]
        L.ada_select_full_host.argtypes = [vp, vp, i64, i64, i64, C.c_int, C.c_double, i32p, i32p, fp, vp]
        L.ada_cascade_step_host.argtypes = [vp, vp, i64, i64, i64, C.c_int, C.c_double,
                                            i32p, i32p, i32p, i32p, i32p, i32p, i32p, i32p, fp, fp,
                                            C.c_uint32, vp]
        L.ada_select_full_noalloc.argtypes = [vp, i64, i64, i64, C.c_int, C.c_double, i32p, i32p,
                                              fp, vp]
        L.ada_gram_op_count.argtypes = [C.c_int, i64, i64, i64]
        L.ada_gram_op_count.restype = C.c_uint64
        L.ada_device_status.argtypes = [vp, vp, C.POINTER(i64)]
        L.ada_profile_enable.argtypes = [vp, C.c_int]
        L.ada_profile_read.argtypes = [vp, C.POINTER(C.c_char_p), C.POINTER(i64),
                                       C.POINTER(C.c_double), C.c_int]
        L.ada_status_string.argtypes = [C.c_int]
        L.ada_status_string.restype = C.c_char_p
        for name in SYMBOLS:
            if name not in ("ada_gram_op_count", "ada_status_string"):
                getattr(L, name).restype = C.c_int
        _lib = L
    return _lib


def status_string(s: int) -> str:
    return lib().ada_status_string(int(s)).decode()


def _check(st: int, where: str) -> None:
    if st != ADA_OK:
        raise AdaError(st, where)


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    return None if t is None else t.data_ptr()


def _stream(stream) -> Optional[int]:
    if stream is None:
        stream = torch.cuda.current_stream()
    return stream.cuda_stream or None


def dtype_of(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return ADA_F32
    if t.dtype == torch.bfloat16:
        return ADA_BF16
    raise TypeError(f"unsupported activation dtype {t.dtype}")


def _shape(X: torch.Tensor):
    if X.dim() == 2:
        X = X.unsqueeze(0)
    if X.dim() != 3 or X.stride(2) != 1 or (X.shape[0] > 1 and X.stride(0) != X.shape[1] * X.stride(1)):
        raise ValueError("X must be (B,)T x d, unit inner stride, sequences densely stacked")
    B, T, d = X.shape
    return X, B, T, d, X.stride(1)


class Context:
    """Owner of an ada_ctx handle."""

    def __init__(self, maxB: int, maxT: int, maxd: int, dtype: int, device: int = 0):
        h = C.c_void_p()
        _check(lib().ada_create(C.byref(h), device, maxB, maxT, maxd, dtype), "ada_create")
        self.h, self.device, self.dtype = h, device, dtype
        self.maxB, self.maxT, self.maxd = maxB, maxT, maxd

    def close(self):
        if self.h:
            lib().ada_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def ada_create(maxB: int, maxT: int, maxd: int, dtype: int, device: int = 0) -> Context:
    return Context(maxB, maxT, maxd, dtype, device)


def ada_destroy(ctx: Context) -> None:
    ctx.close()


def ada_set_engine(ctx: Context, engine: int) -> None:
    _check(lib().ada_set_engine(ctx.h, engine), "ada_set_engine")


def ada_set_cooperative(ctx: Context, on: bool) -> None:
    _check(lib().ada_set_cooperative(ctx.h, int(bool(on))), "ada_set_cooperative")


def ada_set_row_compaction(ctx: Context, min_rows: int) -> None:
    """Sequence length from which a large inherited set's complement is copied out for the cross step."""
    _check(lib().ada_set_row_compaction(ctx.h, int(min_rows)), "ada_set_row_compaction")


def ada_set_dependent_launch(ctx: Context, on: bool) -> None:
    _check(lib().ada_set_dependent_launch(ctx.h, int(bool(on))), "ada_set_dependent_launch")


def ada_selftest_wait_timeout(ctx: Context, limit_ms: int = 50, stream=None) -> None:
    """Enqueue the bounded-wait self-test; ada_device_status then reports ADA_ERR_TIMEOUT."""
    _check(lib().ada_selftest_wait_timeout(ctx.h, int(limit_ms), _stream(stream)),
           "ada_selftest_wait_timeout")


def ada_gram_op_count(cascade: bool, T: int, d: int, r: int = 0) -> int:
    return int(lib().ada_gram_op_count(int(bool(cascade)), T, d, r))


def ada_device_status(ctx: Context, stream=None):
    """Returns (status, n_zero_norm_rows); synchronises the stream."""
    n = C.c_int64(0)
    st = lib().ada_device_status(ctx.h, _stream(stream), C.byref(n))
    return st, n.value


def ada_normalize(ctx: Context, X: torch.Tensor, want_xhat=False, rep_idx=None, rep_cnt=None,
                  stream=None):
    """Returns (inv_norm, Xhat or None, Xrep or None)."""
    X, B, T, d, ldx = _shape(X)
    inv = torch.empty((B, T), dtype=torch.float32, device=X.device)
    xhat = torch.empty((B, T, d), dtype=X.dtype, device=X.device) if want_xhat else None
    xrep = torch.zeros((B, T, d), dtype=X.dtype, device=X.device) if rep_idx is not None else None
    _check(lib().ada_normalize(ctx.h, X.data_ptr(), B, T, d, ldx, dtype_of(X), _ptr(xhat),
                               inv.data_ptr(), _ptr(rep_idx), _ptr(rep_cnt), _ptr(xrep),
                               _stream(stream)), "ada_normalize")
    return inv, xhat, xrep


def ada_select_full(ctx: Context, X: torch.Tensor, tau: float, rep_idx=None, rep_cnt=None,
                    gamma=None, want_gamma=True, stream=None):
    """Definition 1.  Returns (rep_idx[B,T] int32, rep_cnt[B] int32, gamma[B,T] or None)."""
    X, B, T, d, ldx = _shape(X)
    dev = X.device
    if rep_idx is None:
        rep_idx = torch.empty((B, T), dtype=torch.int32, device=dev)
    if rep_cnt is None:
        rep_cnt = torch.empty((B,), dtype=torch.int32, device=dev)
    if gamma is None and want_gamma:
        gamma = torch.empty((B, T), dtype=torch.float32, device=dev)
    _check(lib().ada_select_full(ctx.h, X.data_ptr(), B, T, d, ldx, dtype_of(X), float(tau),
                                 rep_idx.data_ptr(), rep_cnt.data_ptr(), _ptr(gamma),
                                 _stream(stream)), "ada_select_full")
    return rep_idx, rep_cnt, gamma


class CascadeOut:
    __slots__ = ("rep_out", "rep_out_cnt", "add_idx", "add_cnt", "rem_idx", "rem_cnt",
                 "gamma_rep", "gamma_cross")

    def __init__(self, B, T, dev, want_gamma):
        i32 = dict(dtype=torch.int32, device=dev)
        self.rep_out = torch.empty((B, T), **i32)
        self.add_idx = torch.empty((B, T), **i32)
        self.rem_idx = torch.empty((B, T), **i32)
        self.rep_out_cnt = torch.empty((B,), **i32)
        self.add_cnt = torch.empty((B,), **i32)
        self.rem_cnt = torch.empty((B,), **i32)
        self.gamma_rep = torch.empty((B, T), dtype=torch.float32, device=dev) if want_gamma else None
        self.gamma_cross = torch.empty((B, T), dtype=torch.float32, device=dev) if want_gamma else None


def ada_cascade_step(ctx: Context, X: torch.Tensor, tau: float, rep_in: torch.Tensor,
                     rep_in_cnt: torch.Tensor, out: Optional[CascadeOut] = None, flags: int = 0,
                     want_gamma=True, stream=None) -> CascadeOut:
    """Algorithm 1.  `out` buffers are reused when given."""
    X, B, T, d, ldx = _shape(X)
    if out is None:
        out = CascadeOut(B, T, X.device, want_gamma)
    _check(lib().ada_cascade_step(ctx.h, X.data_ptr(), B, T, d, ldx, dtype_of(X), float(tau),
                                  rep_in.data_ptr(), rep_in_cnt.data_ptr(), out.rep_out.data_ptr(),
                                  out.rep_out_cnt.data_ptr(), out.add_idx.data_ptr(),
                                  out.add_cnt.data_ptr(), out.rem_idx.data_ptr(),
                                  out.rem_cnt.data_ptr(), _ptr(out.gamma_rep),
                                  _ptr(out.gamma_cross), flags, _stream(stream)),
           "ada_cascade_step")
    return out


def ada_cascade_step_adaptive(ctx: Context, X: torch.Tensor, tau_state: torch.Tensor,
                              policy: Optional[TauPolicy], rep_in: torch.Tensor,
                              rep_in_cnt: torch.Tensor, out: Optional[CascadeOut] = None,
                              flags: int = 0, want_gamma=True, turnover: Optional[torch.Tensor] = None,
                              stream=None) -> CascadeOut:
    """Section 8.1: Algorithm 1 with the per-sequence threshold tau_state (float64[B] on the
    device, updated in place when a policy is given); `turnover` (float32[B]) receives Eq. 6."""
    X, B, T, d, ldx = _shape(X)
    assert tau_state.dtype == torch.float64 and tau_state.is_cuda and tau_state.numel() == B
    if out is None:
        out = CascadeOut(B, T, X.device, want_gamma)
    _check(lib().ada_cascade_step_adaptive(
        ctx.h, X.data_ptr(), B, T, d, ldx, dtype_of(X), tau_state.data_ptr(),
        None if policy is None else C.byref(policy), rep_in.data_ptr(), rep_in_cnt.data_ptr(),
        out.rep_out.data_ptr(), out.rep_out_cnt.data_ptr(), out.add_idx.data_ptr(),
        out.add_cnt.data_ptr(), out.rem_idx.data_ptr(), out.rem_cnt.data_ptr(),
        _ptr(out.gamma_rep), _ptr(out.gamma_cross), _ptr(turnover), flags, _stream(stream)),
        "ada_cascade_step_adaptive")
    return out


def _shape_heads(X: torch.Tensor):
    if X.dim() != 3 or X.stride(2) != 1 or X.stride(1) != X.shape[2]:
        raise ValueError("X must be T x h x d_h with the heads of a token side by side")
    T, h, d_h = X.shape
    return T, h, d_h, X.stride(0)


def ada_select_full_heads(ctx: Context, X: torch.Tensor, tau: float, rep_idx=None, rep_cnt=None,
                          gamma=None, want_gamma=True, stream=None):
    """Section 8.5: Definition 1 per head of X (T, h, d_h).  Returns (rep_idx[h,T], rep_cnt[h],
    gamma[h,T] or None)."""
    T, h, d_h, ldx = _shape_heads(X)
    dev = X.device
    if rep_idx is None:
        rep_idx = torch.empty((h, T), dtype=torch.int32, device=dev)
    if rep_cnt is None:
        rep_cnt = torch.empty((h,), dtype=torch.int32, device=dev)
    if gamma is None and want_gamma:
        gamma = torch.empty((h, T), dtype=torch.float32, device=dev)
    _check(lib().ada_select_full_heads(ctx.h, X.data_ptr(), T, h, d_h, ldx, dtype_of(X), float(tau),
                                       rep_idx.data_ptr(), rep_cnt.data_ptr(), _ptr(gamma),
                                       _stream(stream)), "ada_select_full_heads")
    return rep_idx, rep_cnt, gamma


def ada_cascade_step_heads(ctx: Context, X: torch.Tensor, tau: float, rep_in: torch.Tensor,
                           rep_in_cnt: torch.Tensor, out: Optional[CascadeOut] = None,
                           flags: int = 0, want_gamma=True, stream=None) -> CascadeOut:
    """Section 8.5: Algorithm 1 per head of X (T, h, d_h); lists are [h, T], counts [h]."""
    T, h, d_h, ldx = _shape_heads(X)
    if out is None:
        out = CascadeOut(h, T, X.device, want_gamma)
    _check(lib().ada_cascade_step_heads(ctx.h, X.data_ptr(), T, h, d_h, ldx, dtype_of(X),
                                        float(tau), rep_in.data_ptr(), rep_in_cnt.data_ptr(),
                                        out.rep_out.data_ptr(), out.rep_out_cnt.data_ptr(),
                                        out.add_idx.data_ptr(), out.add_cnt.data_ptr(),
                                        out.rem_idx.data_ptr(), out.rem_cnt.data_ptr(),
                                        _ptr(out.gamma_rep), _ptr(out.gamma_cross), flags,
                                        _stream(stream)), "ada_cascade_step_heads")
    return out


def ada_nearest_rep(ctx: Context, X: torch.Tensor, rep_idx: torch.Tensor, rep_cnt: torch.Tensor,
                    want_gamma=True, stream=None):
    """Section 2.3.  Returns (nearest_idx[B,T] int32, nearest_gamma[B,T] or None)."""
    X, B, T, d, ldx = _shape(X)
    near = torch.empty((B, T), dtype=torch.int32, device=X.device)
    g = torch.empty((B, T), dtype=torch.float32, device=X.device) if want_gamma else None
    _check(lib().ada_nearest_rep(ctx.h, X.data_ptr(), B, T, d, ldx, dtype_of(X), rep_idx.data_ptr(),
                                 rep_cnt.data_ptr(), near.data_ptr(), _ptr(g), _stream(stream)),
           "ada_nearest_rep")
    return near, g


def ada_attention_reps(ctx: Context, Q: torch.Tensor, K: torch.Tensor, V: torch.Tensor,
                       rep_idx: torch.Tensor, rep_cnt: torch.Tensor, nearest_idx=None, out=None,
                       flags: int = 0, stream=None) -> torch.Tensor:
    """Section 2.3, Eq. 2: attention on the representative rows of Q, K, V (each T x h x d_h,
    bf16), expanded to every token through nearest_idx when given.  Returns out fp32 [T, h, d_h]
    (rows that receive nothing are left as they are: zeros in a fresh tensor)."""
    T, h, d_h, ld = _shape_heads(Q)
    for X in (K, V):
        if X.shape != Q.shape or X.stride() != Q.stride():
            raise ValueError("Q, K, V must share shape and strides")
    if out is None:
        out = torch.zeros((T, h, d_h), dtype=torch.float32, device=Q.device)
    _check(lib().ada_attention_reps(ctx.h, Q.data_ptr(), K.data_ptr(), V.data_ptr(), T, h, d_h, ld,
                                    dtype_of(Q), rep_idx.data_ptr(), rep_cnt.data_ptr(),
                                    _ptr(nearest_idx), out.data_ptr(), out.stride(0), flags,
                                    _stream(stream)), "ada_attention_reps")
    return out


def ada_select_full_host(ctx: Context, X: torch.Tensor, tau: float, rep_idx: torch.Tensor,
                         rep_cnt: torch.Tensor, gamma: Optional[torch.Tensor] = None,
                         stream=None) -> None:
    """HOST tensors in and out (pinned memory recommended); returns after `stream` is idle."""
    X, B, T, d, ldx = _shape(X)
    assert not X.is_cuda and ldx == d
    _check(lib().ada_select_full_host(ctx.h, X.data_ptr(), B, T, d, dtype_of(X), float(tau),
                                      rep_idx.data_ptr(), rep_cnt.data_ptr(), _ptr(gamma),
                                      _stream(stream)), "ada_select_full_host")


def ada_cascade_step_host(ctx: Context, X: torch.Tensor, tau: float, rep_in, rep_in_cnt, rep_out,
                          rep_out_cnt, add_idx, add_cnt, rem_idx, rem_cnt, gamma_rep=None,
                          gamma_cross=None, flags: int = 0, stream=None) -> None:
    X, B, T, d, ldx = _shape(X)
    assert not X.is_cuda and ldx == d
    _check(lib().ada_cascade_step_host(ctx.h, X.data_ptr(), B, T, d, dtype_of(X), float(tau),
                                       rep_in.data_ptr(), rep_in_cnt.data_ptr(), rep_out.data_ptr(),
                                       rep_out_cnt.data_ptr(), add_idx.data_ptr(), add_cnt.data_ptr(),
                                       rem_idx.data_ptr(), rem_cnt.data_ptr(), _ptr(gamma_rep),
                                       _ptr(gamma_cross), flags, _stream(stream)),
           "ada_cascade_step_host")


def ada_select_full_noalloc(X: torch.Tensor, tau: float, rep_idx: torch.Tensor,
                            rep_cnt: torch.Tensor, gamma: Optional[torch.Tensor] = None,
                            stream=None) -> None:
    """Full selection of ONE sequence (T x d) with no context and no allocation inside the
    library: the caller passes every buffer (rep_idx: T int32, rep_cnt: 1 int32, gamma:
    optional T float32) and the library's scratch is a fixed device array, so this is the
    call for code that may not allocate device memory.  T <= ADA_NOALLOC_MAX_T; calls on
    one device must not overlap on the GPU (they share the scratch)."""
    if X.dim() == 3 and X.shape[0] == 1:
        X = X[0]
    if X.dim() != 2 or X.stride(1) != 1:
        raise ValueError("X must be T x d with unit inner stride")
    T, d = X.shape
    st = lib().ada_select_full_noalloc(X.data_ptr(), T, d, X.stride(0), dtype_of(X), float(tau),
                                       rep_idx.data_ptr(), rep_cnt.data_ptr(), _ptr(gamma),
                                       _stream(stream))
    if st == 3:
        raise AdaError(st, f"ada_select_full_noalloc: T={T} exceeds ADA_NOALLOC_MAX_T="
                           f"{ADA_NOALLOC_MAX_T}")
    _check(st, "ada_select_full_noalloc")


def ada_profile_enable(ctx: Context, on: bool) -> None:
    _check(lib().ada_profile_enable(ctx.h, int(on)), "ada_profile_enable")


def ada_profile_read(ctx: Context):
    """Returns {kernel name: (launches, total_ms)} since the last read."""
    cap = 32
    names = (C.c_char_p * cap)()
    cnt = (C.c_int64 * cap)()
    ms = (C.c_double * cap)()
    n = lib().ada_profile_read(ctx.h, names, cnt, ms, cap)
    return {names[i].decode(): (int(cnt[i]), float(ms[i])) for i in range(min(n, cap))}
