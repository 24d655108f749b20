"""float64 CPU oracle for the CHELA token-mixer hot path (ctypes wrapper).

TEST INFRASTRUCTURE ONLY: used by the tests, the smoke check and the benchmark's
CPU-baseline leg.  It shares nothing with the CUDA library and must not be
imported by the product package.

Every function takes and returns C-contiguous float64 numpy arrays.  The
arithmetic lives in ``chela_oracle.c`` (plain loops, own radix-2 FFT); this
module only marshals arguments.  The normaliser choice (gain-free row RMS) is a
reading of the paper's "Norm": parity unpinned for that choice, the
un-normalised output (``norm=False``) is pinned on its own.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "chela_oracle.c")
_LIB_PATH = os.path.join(_HERE, "libchela_oracle.so")
_lib = None

_dp = ctypes.POINTER(ctypes.c_double)


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (-O2, OpenMP) if the shared object is stale."""
    if (not force and os.path.exists(_LIB_PATH)
            and os.path.getmtime(_LIB_PATH) >= os.path.getmtime(_SRC)):
        return _LIB_PATH
    tmp = _LIB_PATH + ".tmp.%d" % os.getpid()
    subprocess.check_call(["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-std=c11",
                           "-o", tmp, _SRC, "-lm"])
    os.replace(tmp, _LIB_PATH)
    return _LIB_PATH


def _load():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.oracle_num_threads.restype = ctypes.c_int
    return _lib


def num_threads() -> int:
    return int(_load().oracle_num_threads())


def _f64(a):
    return np.ascontiguousarray(a, dtype=np.float64)


def _p(a):
    return None if a is None else a.ctypes.data_as(_dp)


def _shape_qkv(q, k, v):
    q, k, v = _f64(q), _f64(k), _f64(v)
    B, L, H, dk = q.shape
    assert k.shape == q.shape and v.shape[:3] == q.shape[:3]
    return q, k, v, B, L, H, dk, v.shape[3]


def linattn_quadratic(q, k, v, scale=1.0, norm=True, eps=1e-6):
    """Quadratic masked form of causal linear attention (Eq. 2 + causal mask)."""
    q, k, v, B, L, H, dk, dv = _shape_qkv(q, k, v)
    o = np.empty_like(v)
    _load().oracle_linattn_quadratic(_p(q), _p(k), _p(v), _p(o), B, H, L, dk, dv,
                                     ctypes.c_double(scale), int(bool(norm)), ctypes.c_double(eps))
    return o


def linattn_recurrent(q, k, v, scale=1.0, norm=True, eps=1e-6, state_in=None, return_state=False):
    """Token-by-token recurrent form: S_t = S_{t-1} + k_t v_t^T, r_t = scale * S_t^T q_t."""
    q, k, v, B, L, H, dk, dv = _shape_qkv(q, k, v)
    o = np.empty_like(v)
    s_in = None if state_in is None else _f64(state_in)
    s_out = np.empty((B, H, dk, dv)) if return_state else None
    _load().oracle_linattn_recurrent(_p(q), _p(k), _p(v), _p(o), B, H, L, dk, dv,
                                     ctypes.c_double(scale), int(bool(norm)), ctypes.c_double(eps),
                                     _p(s_in), _p(s_out))
    return (o, s_out) if return_state else o


def linattn_chunked(q, k, v, chunk, scale=1.0, norm=True, eps=1e-6):
    """Chunked (tiled) form of Sec. 4.1 with chunk size ``chunk``."""
    q, k, v, B, L, H, dk, dv = _shape_qkv(q, k, v)
    o = np.empty_like(v)
    _load().oracle_linattn_chunked(_p(q), _p(k), _p(v), _p(o), B, H, L, dk, dv, int(chunk),
                                   ctypes.c_double(scale), int(bool(norm)), ctypes.c_double(eps))
    return o


def shortconv(x, w, bias=None, act=True):
    """y[b,t,c] = act(bias[c] + sum_j w[c,j] x[b,t-j,c]); act = SiLU (Eq. 7, inner part)."""
    x, w = _f64(x), _f64(w)
    B, L, D = x.shape
    assert w.shape[0] == D
    b = None if bias is None else _f64(bias)
    y = np.empty_like(x)
    _load().oracle_shortconv(_p(x), _p(w), _p(b), _p(y), B, L, D, w.shape[1], int(bool(act)))
    return y


def longconv_direct(a, k):
    """Causal long convolution by its defining sum, O(L^2)."""
    a, k = _f64(a), _f64(k)
    B, L, D = a.shape
    assert k.shape == (D, L)
    z = np.empty_like(a)
    _load().oracle_longconv_direct(_p(a), _p(k), _p(z), B, L, D)
    return z


def longconv_fft(a, k):
    """Causal long convolution through the FFT theorem (Eq. 6), zero-padded to >= 2L."""
    a, k = _f64(a), _f64(k)
    B, L, D = a.shape
    assert k.shape == (D, L)
    z = np.empty_like(a)
    _load().oracle_longconv_fft(_p(a), _p(k), _p(z), B, L, D)
    return z


def mixer(x, w_short, k_long, w_q, w_k, w_v, H, b_q=None, b_k=None, b_v=None,
          qk_diag=False, v_silu=True, norm=True, eps=1e-6, use_fft=True, return_z=False):
    """Mixer composition: short conv + SiLU, long conv, Q/K/V formation, per-head attention."""
    x, w_short, k_long = _f64(x), _f64(w_short), _f64(k_long)
    w_q, w_k, w_v = _f64(w_q), _f64(w_k), _f64(w_v)
    B, L, D = x.shape
    assert D % H == 0
    bq = None if b_q is None else _f64(b_q)
    bk = None if b_k is None else _f64(b_k)
    bv = None if b_v is None else _f64(b_v)
    o = np.empty_like(x)
    z = np.empty_like(x) if return_z else None
    _load().oracle_mixer(_p(x), _p(w_short), w_short.shape[1], _p(k_long), _p(w_q), _p(w_k), _p(w_v),
                         _p(bq), _p(bk), _p(bv), int(bool(qk_diag)), int(bool(v_silu)), _p(o), _p(z),
                         B, L, D, H, int(bool(norm)), ctypes.c_double(eps), int(bool(use_fft)))
    return (o, z) if return_z else o


def dense(x, w, bias=None, act=False):
    """y = act(x w + bias) by the plain triple loop; act = SiLU (Eq. 12)."""
    x, w = _f64(x), _f64(w)
    M, K = x.shape
    assert w.shape[0] == K
    N = w.shape[1]
    b = None if bias is None else _f64(bias)
    y = np.empty((M, N))
    _load().oracle_dense(_p(x), _p(w), _p(b), _p(y), ctypes.c_size_t(M), K, N, int(bool(act)))
    return y


def mixer_gated(x, w_short, k_long, w_q, w_k, w_v, w_a, w_o, H, b_q=None, b_k=None, b_v=None, b_a=None, b_o=None,
                qk_diag=False, v_silu=True, norm=True, eps=1e-6, use_fft=True):
    """Mixer with gates: U = O . silu(Z W_a + b_a) . sigmoid(Z W_o + b_o) + X . (1 - sigmoid(...)) (Eqs. 8-9, 13-14)."""
    x, w_short, k_long = _f64(x), _f64(w_short), _f64(k_long)
    w_q, w_k, w_v, w_a, w_o = _f64(w_q), _f64(w_k), _f64(w_v), _f64(w_a), _f64(w_o)
    B, L, D = x.shape
    opt = lambda b: None if b is None else _f64(b)
    bq, bk, bv, ba, bo = opt(b_q), opt(b_k), opt(b_v), opt(b_a), opt(b_o)
    u = np.empty_like(x)
    _load().oracle_mixer_gated(_p(x), _p(w_short), w_short.shape[1], _p(k_long), _p(w_q), _p(w_k), _p(w_v),
                               _p(bq), _p(bk), _p(bv), _p(w_a), _p(ba), _p(w_o), _p(bo), int(bool(qk_diag)),
                               int(bool(v_silu)), _p(u), B, L, D, H, int(bool(norm)), ctypes.c_double(eps),
                               int(bool(use_fft)))
    return u


def linattn_backward(q, k, v, d_o, scale=1.0, norm=True, eps=1e-6):
    """Gradients (dq, dk, dv) of causal linear attention for the output gradient d_o, by the O(L^2) definition."""
    q, k, v, B, L, H, dk, dv = _shape_qkv(q, k, v)
    d_o = _f64(d_o)
    dq, dk_, dv_ = np.empty_like(q), np.empty_like(k), np.empty_like(v)
    _load().oracle_linattn_backward(_p(q), _p(k), _p(v), _p(d_o), _p(dq), _p(dk_), _p(dv_), B, H, L, dk, dv,
                                    ctypes.c_double(scale), int(bool(norm)), ctypes.c_double(eps))
    return dq, dk_, dv_
