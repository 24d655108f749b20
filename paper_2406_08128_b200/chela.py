"""Thin Python binding of libchela's C ABI (argument marshalling only).

Each function mirrors the C entry point of the same name: it reads shapes and device pointers
from torch tensors, allocates the output and the workspace with torch, and passes torch's
current CUDA stream.  Every step of the computation runs in the library's kernels.  There is no
CPU fallback: if ``libchela.so`` has not been built (``python -m paper_2406_08128_b200.build``)
loading fails with an error.
"""
from __future__ import annotations

import ctypes
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libchela.so")

OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_WORKSPACE, ERR_CUDA, ERR_TIMEOUT = range(6)
F32, BF16, BF16_PAIR = 0, 1, 2
NORM_NONE, NORM_RMS = 0, 1

_DTYPES = {torch.float32: F32, torch.bfloat16: BF16}
_lib = None

_c_int, _c_float, _c_size_t, _vp = ctypes.c_int, ctypes.c_float, ctypes.c_size_t, ctypes.c_void_p

_SIGNATURES = {
    "chela_status_string": (ctypes.c_char_p, [_c_int]),
    "chela_version": (_c_int, []),
    "chela_linattn_kernel_kind": (_c_int, [_c_int] * 6 + [_c_int, _c_int]),
    "chela_shortconv_fwd": (_c_int, [_vp, _vp, _vp, _vp, _c_int, _c_int, _c_int, _c_int, _c_int, _c_int, _vp]),
    "chela_second_short_width": (_c_int, [_c_int]),
    "chela_shortconv_reparam": (_c_int, [_vp, _c_int, _vp, _c_int, _vp, _c_int, _vp]),
    "chela_longconv_workspace_bytes": (_c_size_t, [_c_int, _c_int, _c_int, _c_int, _c_int]),
    "chela_longconv_fwd": (_c_int, [_vp, _vp, _vp, _c_int, _vp, _c_int, _c_int, _c_int, _c_int, _c_int,
                                    _vp, _c_size_t, _vp]),
    "chela_linattn_workspace_bytes": (_c_size_t, [_c_int] * 6),
    "chela_linattn_fwd": (_c_int, [_vp, _vp, _vp, _vp] + [_c_int] * 6 + [_c_int, _c_int, _c_int, _c_float,
                                   _c_float, _vp, _c_size_t, _vp]),
    "chela_linattn_carry_fwd": (_c_int, [_vp, _vp, _vp, _vp, _vp, _vp] + [_c_int] * 6 + [_c_int, _c_int, _c_int, _c_float,
                                         _c_float, _vp, _c_size_t, _vp]),
    "chela_linattn_split_plan": (_c_int, [_c_int] * 6 + [_vp, _vp, _vp]),
    "chela_linattn_step": (_c_int, [_vp] * 5 + [_c_int] * 4 + [_c_int, _c_int, _c_int, _c_float, _c_float, _vp]),
    "chela_linattn_bwd_workspace_bytes": (_c_size_t, [_c_int] * 5),
    "chela_linattn_bwd": (_c_int, [_vp] * 7 + [_c_int] * 5 + [_c_int, _c_int, _c_float, _c_float, _vp, _c_size_t, _vp]),
    "chela_dense_workspace_bytes": (_c_size_t, []),
    "chela_dense_fwd": (_c_int, [_vp, _vp, _vp, _vp, _c_int, _c_int, _c_int, _c_int, _c_int, _c_int, _c_int, _vp,
                                 _c_size_t, _vp]),
    "chela_async_status": (_c_int, [_vp, _vp]),
    "chela_debug_wait_control": (None, [ctypes.c_longlong, _c_int]),
    "chela_debug_sm_clock": (_c_int, [_vp, ctypes.c_longlong, _vp]),
    "chela_linattn_static_ws_status": (_c_int, [_vp]),
    "chela_linattn_fwd_static_ws": (_c_int, [_vp, _vp, _vp, _vp] + [_c_int] * 6 + [_c_int, _c_int, _c_int, _c_float,
                                             _c_float, _vp]),
    "chela_mixer_workspace_bytes": (_c_size_t, [_c_int] * 5 + [_c_int]),
    "chela_mixer_gated_workspace_bytes": (_c_size_t, [_c_int] * 5 + [_c_int]),
    "chela_mixer_gated_fwd": (_c_int, [_vp, _vp, _c_int, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _c_int, _c_int,
                                       _vp, _c_int, _c_int, _c_int, _c_int, _c_int, _c_int, _c_int, _c_int, _c_float,
                                       _vp, _c_size_t, _vp]),
    "chela_longconv_spectrum_bytes": (_c_size_t, [_c_int, _c_int]),
    "chela_longconv_prepare": (_c_int, [_vp, _c_int, _c_int, _vp, _c_size_t, _vp]),
    "chela_longconv_prepared_fwd": (_c_int, [_vp, _vp, _vp, _c_int, _vp, _c_int, _c_int, _c_int, _c_int, _c_int, _vp, _c_size_t, _vp]),
    "chela_mixer_prepared_fwd": (_c_int, [_vp, _vp, _c_int, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _c_int, _c_int,
                                          _vp, _c_int, _c_int, _c_int, _c_int, _c_int, _c_int, _c_int, _c_int, _c_float,
                                          _vp, _c_size_t, _vp]),
    "chela_mixer_fwd": (_c_int, [_vp, _vp, _c_int, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _c_int, _c_int, _vp,
                                 _c_int, _c_int, _c_int, _c_int, _c_int, _c_int, _c_int, _c_int, _c_float,
                                 _vp, _c_size_t, _vp]),
}


class ChelaError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__("%s: %s (status %d)" % (where, status_string(status), status))


def exported_symbols():
    """Names the C header declares (the loader resolves every one of them)."""
    return sorted(_SIGNATURES)


def lib():
    """Load libchela.so (once).  Raises if the library has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError("libchela.so is missing: build it with `python -m paper_2406_08128_b200.build` "
                               "(there is no CPU fallback)")
        handle = ctypes.CDLL(LIB_PATH)
        for name, (res, args) in _SIGNATURES.items():
            fn = getattr(handle, name)
            fn.restype, fn.argtypes = res, args
        _lib = handle
    return _lib


def status_string(status: int) -> str:
    return lib().chela_status_string(int(status)).decode()


def version() -> int:
    return int(lib().chela_version())


def _check(status: int, where: str):
    if status != OK:
        raise ChelaError(int(status), where)


def _ptr(t):
    return None if t is None else _vp(t.data_ptr())


def _stream():
    return _vp(torch.cuda.current_stream().cuda_stream)


def _dt(t) -> int:
    return _DTYPES[t.dtype]


def _tdtype(code: int):
    return torch.float32 if code == F32 else torch.bfloat16


def _workspace(nbytes: int, device):
    return torch.empty(max(int(nbytes), 16), dtype=torch.uint8, device=device)


def linattn_kernel_kind(B, H, L, d_k, d_v, chunk, in_dtype=BF16, out_dtype=F32) -> int:
    return int(lib().chela_linattn_kernel_kind(B, H, L, d_k, d_v, chunk, in_dtype, out_dtype))


def shortconv_fwd(x, w, bias=None, act=True, out=None):
    """x [B,L,D] (bf16/f32), w [D,width] f32 -> y like x."""
    B, L, D = x.shape
    y = torch.empty_like(x) if out is None else out
    _check(lib().chela_shortconv_fwd(_ptr(x), _ptr(w), _ptr(bias), _ptr(y), B, L, D, w.shape[1], int(bool(act)),
                                     _dt(x), _stream()), "chela_shortconv_fwd")
    return y


def second_short_width(L: int) -> int:
    """Width of the length-dependent short kernel, 2 log10(L) + 1 rounded to the nearest odd integer."""
    return int(lib().chela_second_short_width(int(L)))


def shortconv_reparam(w1, w2):
    """Merge two parallel short kernels [D,width1], [D,width2] (fp32) into one [D,max(width)] kernel."""
    D = w1.shape[0]
    merged = torch.empty((D, max(w1.shape[1], w2.shape[1])), dtype=torch.float32, device=w1.device)
    _check(lib().chela_shortconv_reparam(_ptr(w1), w1.shape[1], _ptr(w2), w2.shape[1], _ptr(merged), D, _stream()),
           "chela_shortconv_reparam")
    return merged


def longconv_workspace_bytes(B, L, D, in_dtype=BF16, out_dtype=F32) -> int:
    return int(lib().chela_longconv_workspace_bytes(B, L, D, in_dtype, out_dtype))


def longconv_fwd(x, k_long, w_short=None, out_dtype=F32, out=None, workspace=None):
    """x [B,L,D], k_long [D,L] f32, optional short taps [D,width] f32 -> z [B,L,D] of out_dtype."""
    B, L, D = x.shape
    z = torch.empty((B, L, D), dtype=_tdtype(out_dtype), device=x.device) if out is None else out
    if workspace is None:
        workspace = _workspace(longconv_workspace_bytes(B, L, D, _dt(x), out_dtype), x.device)
    width = 0 if w_short is None else w_short.shape[1]
    _check(lib().chela_longconv_fwd(_ptr(x), _ptr(k_long), _ptr(w_short), width, _ptr(z), B, L, D, _dt(x),
                                    _dt(z), _ptr(workspace), workspace.numel(), _stream()), "chela_longconv_fwd")
    return z


def linattn_workspace_bytes(B, H, L, d_k, d_v, chunk) -> int:
    return int(lib().chela_linattn_workspace_bytes(B, H, L, d_k, d_v, chunk))


def linattn_fwd(q, k, v, chunk=64, out_dtype=F32, norm=NORM_RMS, eps=1e-6, scale=1.0, out=None, workspace=None,
                in_dtype=None):
    """q,k [B,L,H,d_k], v [B,L,H,d_v] -> o [B,L,H,d_v] of out_dtype.

    With in_dtype=BF16_PAIR q, k, v are [2,B,L,H,d] bf16 tensors (high plane, low plane)."""
    in_dtype = _dt(q) if in_dtype is None else in_dtype
    B, L, H, d_k = q.shape[-4:]
    d_v = v.shape[-1]
    o = torch.empty((B, L, H, d_v), dtype=_tdtype(out_dtype), device=q.device) if out is None else out
    if workspace is None:
        workspace = _workspace(linattn_workspace_bytes(B, H, L, d_k, d_v, chunk), q.device)
    _check(lib().chela_linattn_fwd(_ptr(q), _ptr(k), _ptr(v), _ptr(o), B, H, L, d_k, d_v, chunk, in_dtype, _dt(o),
                                   int(norm), float(eps), float(scale), _ptr(workspace), workspace.numel(),
                                   _stream()), "chela_linattn_fwd")
    return o


def linattn_carry_fwd(q, k, v, state_in=None, chunk=64, out_dtype=F32, norm=NORM_RMS, eps=1e-6, scale=1.0, out=None,
                      state_out=None, workspace=None, in_dtype=None):
    """chela_linattn_carry_fwd: returns (o, state_out); state tensors are [B,H,d_k,d_v] fp32."""
    in_dtype = _dt(q) if in_dtype is None else in_dtype
    B, L, H, d_k = q.shape[-4:]
    d_v = v.shape[-1]
    o = torch.empty((B, L, H, d_v), dtype=_tdtype(out_dtype), device=q.device) if out is None else out
    if state_out is None:
        state_out = torch.empty((B, H, d_k, d_v), dtype=torch.float32, device=q.device)
    if workspace is None:
        workspace = _workspace(linattn_workspace_bytes(B, H, L, d_k, d_v, chunk), q.device)
    _check(lib().chela_linattn_carry_fwd(_ptr(q), _ptr(k), _ptr(v), _ptr(o), _ptr(state_in), _ptr(state_out), B, H, L,
                                         d_k, d_v, chunk, in_dtype, _dt(o), int(norm), float(eps), float(scale),
                                         _ptr(workspace), workspace.numel(), _stream()), "chela_linattn_carry_fwd")
    return o, state_out


def linattn_split_plan(B, H, L, d=64, in_dtype=BF16, sms=0):
    """chela_linattn_split_plan: (groups, first_chunks, other_chunks), or None if no tensor-core kernel takes d."""
    g, c0, c = ctypes.c_int(0), ctypes.c_int(0), ctypes.c_int(0)
    ok = lib().chela_linattn_split_plan(B, H, L, d, int(in_dtype), int(sms), ctypes.byref(g), ctypes.byref(c0), ctypes.byref(c))
    return (g.value, c0.value, c.value) if ok else None


def linattn_step(q, k, v, state, out_dtype=F32, norm=NORM_RMS, eps=1e-6, scale=1.0, out=None):
    """chela_linattn_step: one token per sequence; q, k, v [B,H,d]; state [B,H,d,d] fp32 is updated in place."""
    B, H, d_k = q.shape
    d_v = v.shape[2]
    o = torch.empty((B, H, d_v), dtype=_tdtype(out_dtype), device=q.device) if out is None else out
    _check(lib().chela_linattn_step(_ptr(q), _ptr(k), _ptr(v), _ptr(o), _ptr(state), B, H, d_k, d_v, _dt(q), _dt(o),
                                    int(norm), float(eps), float(scale), _stream()), "chela_linattn_step")
    return o


def linattn_bwd(q, k, v, d_o, norm=NORM_RMS, eps=1e-6, scale=1.0, workspace=None):
    """Gradients (dq, dk, dv), fp32, of linattn_fwd for the output gradient d_o (same dtype as q)."""
    B, L, H, d_k = q.shape
    d_v = v.shape[3]
    dq, dk, dv = (torch.empty(t.shape, dtype=torch.float32, device=q.device) for t in (q, k, v))
    if workspace is None:
        workspace = _workspace(int(lib().chela_linattn_bwd_workspace_bytes(B, H, L, d_k, d_v)), q.device)
    _check(lib().chela_linattn_bwd(_ptr(q), _ptr(k), _ptr(v), _ptr(d_o), _ptr(dq), _ptr(dk), _ptr(dv), B, H, L, d_k, d_v,
                                   _dt(q), int(norm), float(eps), float(scale), _ptr(workspace), workspace.numel(),
                                   _stream()), "chela_linattn_bwd")
    return dq, dk, dv


def linattn_fwd_static_ws(q, k, v, chunk=64, out_dtype=F32, norm=NORM_RMS, eps=1e-6, scale=1.0, out=None):
    """chela_linattn_fwd_static_ws: same result as linattn_fwd, scratch from the library's built-in array.

    For hosts that cannot allocate device memory; here torch still allocates the output unless ``out`` is
    given, the library call itself allocates nothing.
    """
    B, L, H, d_k = q.shape
    d_v = v.shape[3]
    o = torch.empty((B, L, H, d_v), dtype=_tdtype(out_dtype), device=q.device) if out is None else out
    _check(lib().chela_linattn_fwd_static_ws(_ptr(q), _ptr(k), _ptr(v), _ptr(o), B, H, L, d_k, d_v, chunk, _dt(q),
                                             _dt(o), int(norm), float(eps), float(scale), _stream()),
           "chela_linattn_fwd_static_ws")
    return o


def dense_fwd(a, w, bias=None, act=False, a_dtype=None, y_dtype=BF16, out=None, workspace=None):
    """y = act(a w + bias).  a [M,K] (a bf16 pair is passed as a [2,M,K] bf16 tensor with a_dtype=BF16_PAIR),
    w [K,N]; returns y [M,N] (or [2,M,N] bf16 for y_dtype=BF16_PAIR)."""
    a_dtype = _dt(a) if a_dtype is None else a_dtype
    M, K = a.shape[-2], a.shape[-1]
    N = w.shape[1]
    if out is None:
        shape = (2, M, N) if y_dtype == BF16_PAIR else (M, N)
        out = torch.empty(shape, dtype=torch.float32 if y_dtype == F32 else torch.bfloat16, device=a.device)
    if workspace is None:
        workspace = _workspace(int(lib().chela_dense_workspace_bytes()), a.device)
    _check(lib().chela_dense_fwd(_ptr(a), _ptr(w), _ptr(bias), _ptr(out), M, K, N, int(act), a_dtype, _dt(w),
                                 y_dtype, _ptr(workspace), workspace.numel(), _stream()), "chela_dense_fwd")
    return out


def async_status(workspace) -> int:
    """Synchronise the current stream and return the asynchronous status recorded in ``workspace``."""
    return int(lib().chela_async_status(_ptr(workspace), _stream()))


def longconv_prepare(k_long, out=None):
    """chela_longconv_prepare: the spectra of the long kernels k_long [D, L] (and the twiddle table) in a device buffer."""
    D, L = k_long.shape
    n = int(lib().chela_longconv_spectrum_bytes(L, D))
    if n == 0:
        raise ChelaError(ERR_UNSUPPORTED, "chela_longconv_spectrum_bytes")
    spec = torch.empty(n, dtype=torch.uint8, device=k_long.device) if out is None else out
    _check(lib().chela_longconv_prepare(_ptr(k_long), L, D, _ptr(spec), spec.numel(), _stream()), "chela_longconv_prepare")
    return spec


def longconv_prepared_fwd(x, spectrum, w_short=None, out_dtype=F32, out=None, workspace=None):
    """chela_longconv_prepared_fwd: chela_longconv_fwd with prepared spectra in place of the kernels."""
    B, L, D = x.shape
    z = torch.empty((B, L, D), dtype=_tdtype(out_dtype), device=x.device) if out is None else out
    if workspace is None:
        workspace = _workspace(longconv_workspace_bytes(B, L, D, _dt(x), out_dtype), x.device)
    _check(lib().chela_longconv_prepared_fwd(_ptr(x), _ptr(spectrum), _ptr(w_short), 0 if w_short is None else w_short.shape[1],
                                             _ptr(z), B, L, D, _dt(x), _dt(z), _ptr(workspace), workspace.numel(), _stream()),
           "chela_longconv_prepared_fwd")
    return z


def mixer_prepared_fwd(x, w_short, spectrum, w_q, w_k, w_v, H, w_a=None, w_o=None, chunk=64, b_q=None, b_k=None, b_v=None,
                       b_a=None, b_o=None, qk_diag=False, v_silu=True, out_dtype=F32, norm=NORM_RMS, eps=1e-6, out=None,
                       workspace=None):
    """chela_mixer_prepared_fwd: the mixer (gated when w_a and w_o are given) with prepared long-kernel spectra."""
    B, L, D = x.shape
    o = torch.empty((B, L, D), dtype=_tdtype(out_dtype), device=x.device) if out is None else out
    if workspace is None:
        need = mixer_gated_workspace_bytes(B, L, D, H, chunk, _dt(x)) if w_a is not None else mixer_workspace_bytes(B, L, D, H, chunk, _dt(x))
        workspace = _workspace(need, x.device)
    _check(lib().chela_mixer_prepared_fwd(_ptr(x), _ptr(w_short), w_short.shape[1], _ptr(spectrum), _ptr(w_q), _ptr(w_k), _ptr(w_v),
                                          _ptr(b_q), _ptr(b_k), _ptr(b_v), _ptr(w_a), _ptr(b_a), _ptr(w_o), _ptr(b_o), int(qk_diag),
                                          int(v_silu), _ptr(o), B, L, D, H, chunk, _dt(x), _dt(o), int(norm), float(eps),
                                          _ptr(workspace), workspace.numel(), _stream()), "chela_mixer_prepared_fwd")
    return o


def debug_wait_control(limit_cycles=0, skip_arrival=0) -> None:
    """chela_debug_wait_control: the wait limit (SM cycles, 0 = default) and the skipped-arrival test hook."""
    lib().chela_debug_wait_control(int(limit_cycles), int(skip_arrival))


def debug_sm_clock_mhz(spin_cycles=400000, device=None) -> float:
    """chela_debug_sm_clock on the current stream: the SM clock in MHz as SM cycles over global-timer nanoseconds."""
    out = torch.zeros(2, dtype=torch.int64, device=device if device is not None else torch.device("cuda", torch.cuda.current_device()))
    _check(lib().chela_debug_sm_clock(_ptr(out), int(spin_cycles), _stream()), "chela_debug_sm_clock")
    cycles, ns = (int(x) for x in out.cpu())
    return cycles * 1000.0 / max(ns, 1)


def linattn_static_ws_status() -> int:
    """Synchronise the current stream and return the status word of the built-in scratch (current device)."""
    return int(lib().chela_linattn_static_ws_status(_stream()))


def mixer_workspace_bytes(B, L, D, H, chunk, in_dtype=BF16) -> int:
    return int(lib().chela_mixer_workspace_bytes(B, L, D, H, chunk, in_dtype))


def mixer_fwd(x, w_short, k_long, w_q, w_k, w_v, H, chunk=64, b_q=None, b_k=None, b_v=None, qk_diag=False,
              v_silu=True, out_dtype=F32, norm=NORM_RMS, eps=1e-6, out=None, workspace=None):
    """x [B,L,D] -> o [B,L,D]; weights as in the C header."""
    B, L, D = x.shape
    o = torch.empty((B, L, D), dtype=_tdtype(out_dtype), device=x.device) if out is None else out
    if workspace is None:
        workspace = _workspace(mixer_workspace_bytes(B, L, D, H, chunk, _dt(x)), x.device)
    _check(lib().chela_mixer_fwd(_ptr(x), _ptr(w_short), w_short.shape[1], _ptr(k_long), _ptr(w_q), _ptr(w_k),
                                 _ptr(w_v), _ptr(b_q), _ptr(b_k), _ptr(b_v), int(bool(qk_diag)),
                                 int(bool(v_silu)), _ptr(o), B, L, D, H, chunk, _dt(x), _dt(o), int(norm),
                                 float(eps), _ptr(workspace), workspace.numel(), _stream()), "chela_mixer_fwd")
    return o


def mixer_gated_workspace_bytes(B, L, D, H, chunk, in_dtype=BF16) -> int:
    return int(lib().chela_mixer_gated_workspace_bytes(B, L, D, H, chunk, in_dtype))


def mixer_gated_fwd(x, w_short, k_long, w_q, w_k, w_v, w_a, w_o, H, chunk=64, b_q=None, b_k=None, b_v=None, b_a=None,
                    b_o=None, qk_diag=False, v_silu=True, out_dtype=F32, norm=NORM_RMS, eps=1e-6, out=None, workspace=None):
    """x [B,L,D] -> u [B,L,D]: the mixer with its gates G_a, G_o and the residual mix."""
    B, L, D = x.shape
    u = torch.empty((B, L, D), dtype=_tdtype(out_dtype), device=x.device) if out is None else out
    if workspace is None:
        workspace = _workspace(mixer_gated_workspace_bytes(B, L, D, H, chunk, _dt(x)), x.device)
    _check(lib().chela_mixer_gated_fwd(_ptr(x), _ptr(w_short), w_short.shape[1], _ptr(k_long), _ptr(w_q), _ptr(w_k), _ptr(w_v),
                                       _ptr(b_q), _ptr(b_k), _ptr(b_v), _ptr(w_a), _ptr(b_a), _ptr(w_o), _ptr(b_o),
                                       int(bool(qk_diag)), int(bool(v_silu)), _ptr(u), B, L, D, H, chunk, _dt(x), _dt(u),
                                       int(norm), float(eps), _ptr(workspace), workspace.numel(), _stream()),
           "chela_mixer_gated_fwd")
    return u
