"""Pins for the float64 CPU oracle: closed forms, hand-worked values, textbook/library special
cases, invariants and brute force -- none of them re-uses the oracle's own code."""
import os

import numpy as np
import pytest

import oracle

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def rnd(seed, *shape):
    return np.random.default_rng(seed).standard_normal(shape)


def numpy_quadratic(q, k, v, scale=1.0):
    """tril(Q K^T) V per (b,h) with library matmuls."""
    B, L, H, _ = q.shape
    out = np.zeros_like(v)
    for b in range(B):
        for h in range(H):
            a = np.tril(q[b, :, h] @ k[b, :, h].T) * scale
            out[b, :, h] = a @ v[b, :, h]
    return out


def rms_norm(r, eps=1e-6):
    return r / np.sqrt((r * r).mean(axis=-1, keepdims=True) + eps)


# ---------------------------------------------------------------- linear attention

def test_hand_worked_example():
    rows = {}
    for line in open(os.path.join(GOLD, "linattn_tiny.txt")):
        if line.startswith("#") or not line.strip():
            continue
        key, *vals = line.split()
        rows[key] = np.array([float(x) for x in vals])
    q = rows["q"].reshape(1, 3, 1, 2)
    k = rows["k"].reshape(1, 3, 1, 2)
    v = rows["v"].reshape(1, 3, 1, 2)
    r = rows["r"].reshape(1, 3, 1, 2)
    assert np.array_equal(oracle.linattn_quadratic(q, k, v, norm=False), r)
    o, s = oracle.linattn_recurrent(q, k, v, norm=False, return_state=True)
    assert np.array_equal(o, r)
    assert np.array_equal(s.reshape(-1), rows["S"])
    for c in (1, 2, 3, 5):
        assert np.array_equal(oracle.linattn_chunked(q, k, v, c, norm=False), r)


def test_brute_force_python_loops():
    B, L, H, dk, dv = 2, 9, 2, 3, 4
    q, k, v = rnd(1, B, L, H, dk), rnd(2, B, L, H, dk), rnd(3, B, L, H, dv)
    ref = np.zeros((B, L, H, dv))
    for b in range(B):
        for h in range(H):
            for t in range(L):
                for s in range(t + 1):
                    a = sum(q[b, t, h, i] * k[b, s, h, i] for i in range(dk))
                    for j in range(dv):
                        ref[b, t, h, j] += 0.5 * a * v[b, s, h, j]
    for out in (oracle.linattn_quadratic(q, k, v, scale=0.5, norm=False),
                oracle.linattn_recurrent(q, k, v, scale=0.5, norm=False),
                oracle.linattn_chunked(q, k, v, 4, scale=0.5, norm=False)):
        assert np.allclose(out, ref, rtol=0, atol=1e-12)


@pytest.mark.parametrize("chunk", [1, 2, 3, 7, 16, 37, 42])
@pytest.mark.parametrize("norm", [False, True])
def test_three_forms_agree(chunk, norm):
    B, L, H, dk, dv = 2, 37, 3, 8, 5
    q, k, v = rnd(4, B, L, H, dk), rnd(5, B, L, H, dk), rnd(6, B, L, H, dv)
    a = oracle.linattn_quadratic(q, k, v, norm=norm)
    b = oracle.linattn_recurrent(q, k, v, norm=norm)
    c = oracle.linattn_chunked(q, k, v, chunk, norm=norm)
    lib = numpy_quadratic(q, k, v)
    lib = rms_norm(lib) if norm else lib
    scale = np.abs(lib).max()
    for out in (a, b, c):
        assert np.abs(out - lib).max() <= 1e-12 * scale


def test_chunk_invariance_config_size():
    q, k, v = (x / 8 for x in (rnd(7, 1, 1024, 2, 64), rnd(8, 1, 1024, 2, 64), rnd(9, 1, 1024, 2, 64)))
    ref = oracle.linattn_recurrent(q, k, v)
    quad = oracle.linattn_quadratic(q, k, v)
    assert np.abs(quad - ref).max() < 1e-10
    for c in (16, 64, 128, 256):
        assert np.abs(oracle.linattn_chunked(q, k, v, c) - ref).max() < 1e-10


def test_closed_forms():
    L, dk, dv = 20, 6, 4
    ones = lambda d: np.ones((1, L, 1, d))
    r = oracle.linattn_recurrent(ones(dk), ones(dk), ones(dv), norm=False)
    assert np.array_equal(r[0, :, 0, :], np.outer(np.arange(1, L + 1) * dk, np.ones(dv)))
    o = oracle.linattn_chunked(ones(dk), ones(dk), ones(dv), 7, norm=True, eps=0.0)
    assert np.allclose(o, 1.0, atol=1e-14)
    # q_t = k_s = e_0 -> prefix sum of V (library cumsum)
    e0 = np.zeros((1, L, 1, dk)); e0[..., 0] = 1.0
    v = rnd(10, 1, L, 1, dv)
    for out in (oracle.linattn_quadratic(e0, e0, v, norm=False), oracle.linattn_chunked(e0, e0, v, 6, norm=False)):
        assert np.allclose(out[0, :, 0], np.cumsum(v[0, :, 0], axis=0), atol=1e-13)
    # d_k = 1: r_t = q_t * sum_{s<=t} k_s v_s
    q1, k1 = rnd(11, 1, L, 1, 1), rnd(12, 1, L, 1, 1)
    ref = q1[0, :, 0] * np.cumsum(k1[0, :, 0] * v[0, :, 0], axis=0)
    assert np.allclose(oracle.linattn_recurrent(q1, k1, v, norm=False)[0, :, 0], ref, atol=1e-13)
    # L = 1: r_0 = <q_0,k_0> v_0
    q, k, vv = rnd(13, 1, 1, 1, dk), rnd(14, 1, 1, 1, dk), rnd(15, 1, 1, 1, dv)
    assert np.allclose(oracle.linattn_quadratic(q, k, vv, norm=False).ravel(), (q.ravel() @ k.ravel()) * vv.ravel())


def test_q_k_roles_not_swapped():
    # with k = e_0 everywhere and generic q: r_t = q_t[0] * cumsum(v)_t ; swapping q,k breaks this
    L, dk, dv = 12, 4, 3
    q, v = rnd(16, 1, L, 1, dk), rnd(17, 1, L, 1, dv)
    k = np.zeros((1, L, 1, dk)); k[..., 0] = 1.0
    ref = q[0, :, 0, :1] * np.cumsum(v[0, :, 0], axis=0)
    for out in (oracle.linattn_quadratic(q, k, v, norm=False), oracle.linattn_recurrent(q, k, v, norm=False),
                oracle.linattn_chunked(q, k, v, 5, norm=False)):
        assert np.allclose(out[0, :, 0], ref, atol=1e-13)


@pytest.mark.parametrize("form", ["quadratic", "recurrent", "chunked"])
def test_causality(form):
    B, L, H, dk, dv, t0 = 1, 50, 2, 4, 4, 23
    q, k, v = rnd(18, B, L, H, dk), rnd(19, B, L, H, dk), rnd(20, B, L, H, dv)
    fn = {"quadratic": oracle.linattn_quadratic, "recurrent": oracle.linattn_recurrent,
          "chunked": lambda *a, **kw: oracle.linattn_chunked(*a, 8, **kw)}[form]
    base = fn(q, k, v)
    q2, k2, v2 = q.copy(), k.copy(), v.copy()
    for a in (q2, k2, v2):
        a[:, t0:] = rnd(21, *a[:, t0:].shape)
    pert = fn(q2, k2, v2)
    assert np.array_equal(base[:, :t0], pert[:, :t0])
    assert not np.allclose(base[:, t0:], pert[:, t0:])


def test_linearity_and_heads_independent():
    B, L, H, dk, dv = 1, 16, 2, 4, 4
    q, k, v, v2 = rnd(22, B, L, H, dk), rnd(23, B, L, H, dk), rnd(24, B, L, H, dv), rnd(25, B, L, H, dv)
    f = lambda q, k, v: oracle.linattn_chunked(q, k, v, 4, norm=False)
    assert np.allclose(f(q, k, 2 * v + v2), 2 * f(q, k, v) + f(q, k, v2), atol=1e-12)
    assert np.allclose(f(3 * q, k, v), 3 * f(q, k, v), atol=1e-12)
    assert np.allclose(f(q, -2 * k, v), -2 * f(q, k, v), atol=1e-12)
    # each (b,h) is an independent problem
    single = f(q[:, :, 1:2], k[:, :, 1:2], v[:, :, 1:2])
    assert np.array_equal(f(q, k, v)[:, :, 1:2], single)


def test_state_carry_two_halves_equal_full():
    B, L, H, dk, dv = 2, 30, 2, 4, 3
    q, k, v = rnd(26, B, L, H, dk), rnd(27, B, L, H, dk), rnd(28, B, L, H, dv)
    full = oracle.linattn_recurrent(q, k, v)
    o1, s1 = oracle.linattn_recurrent(q[:, :13], k[:, :13], v[:, :13], return_state=True)
    o2 = oracle.linattn_recurrent(q[:, 13:], k[:, 13:], v[:, 13:], state_in=s1)
    assert np.allclose(np.concatenate([o1, o2], axis=1), full, atol=1e-13)
    # final state = K^T V with a library matmul
    assert np.allclose(s1[1, 0], k[1, :13, 0].T @ v[1, :13, 0], atol=1e-13)


def test_normaliser_properties():
    B, L, H, dk, dv = 1, 24, 2, 8, 16
    q, k, v = rnd(29, B, L, H, dk), rnd(30, B, L, H, dk), rnd(31, B, L, H, dv)
    o = oracle.linattn_recurrent(q, k, v, norm=True, eps=1e-6)
    assert np.allclose(np.sqrt((o * o).mean(-1)), 1.0, atol=1e-5)
    raw = oracle.linattn_recurrent(q, k, v, norm=False)
    assert np.allclose(o, rms_norm(raw, 1e-6), atol=1e-13)
    # scale invariance (eps = 0) and zero row -> zero, no NaN
    a = oracle.linattn_quadratic(q, k, v, scale=1.0, norm=True, eps=0.0)
    b = oracle.linattn_quadratic(q, k, v, scale=7.5, norm=True, eps=0.0)
    assert np.allclose(a, b, atol=1e-12)
    z = oracle.linattn_chunked(q, k, np.zeros_like(v), 5, norm=True)
    assert np.array_equal(z, np.zeros_like(v))


# ---------------------------------------------------------------- convolutions

def test_shortconv_special_cases():
    B, L, D = 2, 11, 3
    x = rnd(32, B, L, D)
    w = np.zeros((D, 3)); w[:, 0] = 1.0
    assert np.array_equal(oracle.shortconv(x, w, act=False), x)
    w = np.zeros((D, 3)); w[:, 1] = 1.0
    y = oracle.shortconv(x, w, act=False)
    assert np.array_equal(y[:, 1:], x[:, :-1]) and np.array_equal(y[:, 0], np.zeros((B, D)))
    s = rnd(33, D, 1)
    assert np.allclose(oracle.shortconv(x, s, act=False), x * s[:, 0], atol=1e-15)
    bias = rnd(34, D)
    assert np.allclose(oracle.shortconv(x, s, bias=bias, act=False), x * s[:, 0] + bias, atol=1e-15)


def test_shortconv_vs_numpy_convolve_and_silu():
    B, L, D, W = 2, 40, 5, 3
    x, w = rnd(35, B, L, D), rnd(36, D, W)
    y = oracle.shortconv(x, w, act=False)
    for b in range(B):
        for c in range(D):
            assert np.allclose(y[b, :, c], np.convolve(x[b, :, c], w[c])[:L], atol=1e-13)
    ya = oracle.shortconv(x, w, act=True)
    assert np.allclose(ya, y * 0.5 * (1.0 + np.tanh(0.5 * y)), atol=1e-13)  # silu via tanh identity
    # known values: silu(0) = 0, silu(x) -> x for large x, silu(-x) -> 0
    pts = np.array([0.0, 40.0, -40.0, 1.0]).reshape(1, 4, 1)
    got = oracle.shortconv(pts, np.ones((1, 1)), act=True).ravel()
    assert got[0] == 0.0 and abs(got[1] - 40.0) < 1e-12 and abs(got[2]) < 1e-12
    assert abs(got[3] - 0.7310585786300049) < 1e-15  # 1 / (1 + e^-1)


def test_shortconv_is_longconv_with_padded_taps():
    B, L, D, W = 1, 33, 4, 3
    x, w = rnd(37, B, L, D), rnd(38, D, W)
    kpad = np.zeros((D, L)); kpad[:, :W] = w
    assert np.allclose(oracle.shortconv(x, w, act=False), oracle.longconv_direct(x, kpad), atol=1e-13)


@pytest.mark.parametrize("L", [1, 2, 3, 5, 64, 1000])
def test_longconv_fft_equals_direct_and_numpy(L):
    B, D = 2, 3
    a, k = rnd(39 + L, B, L, D), rnd(40 + L, D, L)
    zd, zf = oracle.longconv_direct(a, k), oracle.longconv_fft(a, k)
    scale = np.abs(zd).max()
    assert np.abs(zd - zf).max() <= 1e-10 * scale
    for b in range(B):
        for c in range(D):
            assert np.allclose(zd[b, :, c], np.convolve(a[b, :, c], k[c])[:L], atol=1e-11 * max(scale, 1))


def test_longconv_special_kernels_and_causality():
    B, L, D = 1, 100, 2
    a = rnd(41, B, L, D)
    for fn in (oracle.longconv_direct, oracle.longconv_fft):
        k = np.zeros((D, L)); k[:, 0] = 1.0
        assert np.allclose(fn(a, k), a, atol=1e-12)
        k = np.zeros((D, L)); k[:, 7] = 1.0
        z = fn(a, k)
        assert np.allclose(z[:, 7:], a[:, :-7], atol=1e-12) and np.allclose(z[:, :7], 0, atol=1e-12)
        assert np.allclose(fn(a, np.ones((D, L))), np.cumsum(a, axis=1), atol=1e-11)
        kk = rnd(42, D, L)
        z = fn(a, kk)
        # first sample has exactly one term: rules out the circular reading of Eq. 6
        assert np.allclose(z[0, 0], kk[:, 0] * a[0, 0], atol=1e-12)
        a2 = a.copy(); a2[:, 60:] += 1.0
        assert np.allclose(fn(a2, kk)[:, :60], z[:, :60], atol=1e-11)


# ---------------------------------------------------------------- mixer composition

def numpy_mixer(x, w_short, k_long, w_q, w_k, w_v, H):
    B, L, D = x.shape
    a = np.zeros_like(x)
    for b in range(B):
        for c in range(D):
            a[b, :, c] = np.convolve(x[b, :, c], w_short[c])[:L]
    a = a / (1 + np.exp(-a))
    z = np.zeros_like(x)
    for b in range(B):
        for c in range(D):
            z[b, :, c] = np.convolve(a[b, :, c], k_long[c])[:L]
    q, k = z @ w_q, z @ w_k
    v = x @ w_v
    v = v / (1 + np.exp(-v))
    d = D // H
    sh = (B, L, H, d)
    return rms_norm(numpy_quadratic(q.reshape(sh), k.reshape(sh), v.reshape(sh))).reshape(B, L, D), z


@pytest.mark.parametrize("use_fft", [True, False])
def test_mixer_composition(use_fft):
    B, L, D, H = 2, 48, 8, 2
    x, ws, kl = rnd(43, B, L, D), rnd(44, D, 3), rnd(45, D, L) * np.exp(-0.05 * np.arange(L))
    wq, wk, wv = (rnd(s, D, D) / np.sqrt(D) for s in (46, 47, 48))
    o, z = oracle.mixer(x, ws, kl, wq, wk, wv, H, use_fft=use_fft, return_z=True)
    ro, rz = numpy_mixer(x, ws, kl, wq, wk, wv, H)
    assert np.allclose(z, rz, atol=1e-11)
    assert np.allclose(o, ro, atol=1e-9)


def test_mixer_qk_diag_equals_dense_diagonal_and_bias():
    B, L, D, H = 1, 20, 6, 3
    x, ws, kl = rnd(49, B, L, D), rnd(50, D, 3), rnd(51, D, L)
    aq, ak, bq, bk, bv = rnd(52, D), rnd(53, D), rnd(54, D), rnd(55, D), rnd(56, D)
    wv = rnd(57, D, D)
    a = oracle.mixer(x, ws, kl, aq, ak, wv, H, b_q=bq, b_k=bk, b_v=bv, qk_diag=True)
    b = oracle.mixer(x, ws, kl, np.diag(aq), np.diag(ak), wv, H, b_q=bq, b_k=bk, b_v=bv, qk_diag=False)
    assert np.allclose(a, b, atol=1e-11)
    c = oracle.mixer(x, ws, kl, np.diag(aq), np.diag(ak), wv, H)
    assert not np.allclose(a, c, atol=1e-6)  # the biases are really applied


def test_mixer_head_split_is_contiguous_column_blocks():
    # W_v routes input channel 0 only to column j: the output can be non-zero only in j's head.
    B, L, D, H = 1, 10, 8, 4
    x, ws, kl = rnd(58, B, L, D), rnd(59, D, 3), rnd(60, D, L)
    wq, wk = rnd(61, D, D), rnd(62, D, D)
    for j in (0, 3, 5):
        wv = np.zeros((D, D)); wv[0, j] = 1.0
        o = oracle.mixer(x, ws, kl, wq, wk, wv, H, v_silu=False, norm=False)
        nz = np.nonzero(np.abs(o).sum(axis=(0, 1)))[0]
        assert list(nz) == [j]
    # Q restricted to the columns of head 1 (columns 2,3 at d = 2): only that head's outputs survive.
    wq1 = np.zeros((D, D)); wq1[:, 2:4] = wq[:, 2:4]
    o = oracle.mixer(x, ws, kl, wq1, wk, rnd(63, D, D), H, v_silu=False, norm=False)
    assert list(np.nonzero(np.abs(o).sum(axis=(0, 1)))[0]) == [2, 3]


# ---------------------------------------------------------------- gates (Eqs. 8, 9, 13, 14)

def test_gated_mixer_limits_and_numpy_composition():
    B, L, D, H = 2, 24, 8, 2
    x, ws, kl = rnd(70, B, L, D), rnd(71, D, 3), rnd(72, D, L) * np.exp(-0.05 * np.arange(L))
    wq, wk, wv, wa, wo = (rnd(s, D, D) / np.sqrt(D) for s in (73, 74, 75, 76, 77))
    ba, bo = rnd(78, D), rnd(79, D)
    o, z = oracle.mixer(x, ws, kl, wq, wk, wv, H, return_z=True)
    u = oracle.mixer_gated(x, ws, kl, wq, wk, wv, wa, wo, H, b_a=ba, b_o=bo)
    ga = z @ wa + ba
    ga = ga / (1 + np.exp(-ga))
    go = 1 / (1 + np.exp(-(z @ wo + bo)))
    assert np.allclose(u, o * ga * go + x * (1 - go), atol=1e-10)
    zero = np.zeros((D, D))
    # output gate closed (b_o -> -inf): U = X exactly
    closed = oracle.mixer_gated(x, ws, kl, wq, wk, wv, wa, zero, H, b_a=ba, b_o=np.full(D, -800.0))
    assert np.array_equal(closed, x)
    # output gate open, attention gate constant silu(b) = 1 (b = 1.2784645...): U = O
    b1 = 1.2784645427610738
    assert abs(b1 / (1 + np.exp(-b1)) - 1.0) < 1e-15
    opened = oracle.mixer_gated(x, ws, kl, wq, wk, wv, zero, zero, H, b_a=np.full(D, b1), b_o=np.full(D, 800.0))
    assert np.allclose(opened, o, atol=1e-13)
    # zero gate weights and biases: G_a = silu(0) = 0 and G_o = 1/2, so U = X / 2
    half = oracle.mixer_gated(x, ws, kl, wq, wk, wv, zero, zero, H)
    assert np.allclose(half, 0.5 * x, atol=1e-15)


def test_parallel_short_kernels_equal_one_merged_kernel():
    """Structural re-parameterisation (Sec. 4.2) is linear in the taps: pinned on the oracle's short conv."""
    B, L, D = 2, 50, 4
    x, w3, w9 = rnd(80, B, L, D), rnd(81, D, 3), rnd(82, D, 9)
    merged = w9.copy()
    merged[:, :3] += w3
    both = oracle.shortconv(x, w3, act=False) + oracle.shortconv(x, w9, act=False)
    assert np.allclose(oracle.shortconv(x, merged, act=False), both, atol=1e-13)


# ---------------------------------------------------------------- backward (finite differences)

@pytest.mark.parametrize("norm", [False, True])
def test_backward_matches_central_finite_differences(norm):
    B, L, H, dk, dv = 1, 7, 2, 3, 4
    q, k, v, w = rnd(90, B, L, H, dk), rnd(91, B, L, H, dk), rnd(92, B, L, H, dv), rnd(93, B, L, H, dv)
    loss = lambda q_, k_, v_: float((oracle.linattn_quadratic(q_, k_, v_, scale=0.7, norm=norm, eps=1e-3) * w).sum())
    dq, dk_, dv_ = oracle.linattn_backward(q, k, v, w, scale=0.7, norm=norm, eps=1e-3)
    h = 1e-6
    for arr, grad, which in ((q, dq, 0), (k, dk_, 1), (v, dv_, 2)):
        fd = np.zeros_like(arr)
        for idx in np.ndindex(arr.shape):
            args_p, args_m = [q.copy(), k.copy(), v.copy()], [q.copy(), k.copy(), v.copy()]
            args_p[which][idx] += h
            args_m[which][idx] -= h
            fd[idx] = (loss(*args_p) - loss(*args_m)) / (2 * h)
        assert np.abs(fd - grad).max() <= 1e-6 * max(1.0, np.abs(grad).max())


def test_backward_is_causal_and_linear_in_the_output_gradient():
    B, L, H, d = 1, 20, 1, 4
    q, k, v, g1, g2 = (rnd(s, B, L, H, d) for s in (94, 95, 96, 97, 98))
    a = oracle.linattn_backward(q, k, v, g1, norm=False)
    b = oracle.linattn_backward(q, k, v, g2, norm=False)
    c = oracle.linattn_backward(q, k, v, 2 * g1 - g2, norm=False)
    for x, y, z in zip(a, b, c):
        assert np.allclose(z, 2 * x - y, atol=1e-12)
    # an output gradient that is non-zero only at token t0 reaches keys/values at s <= t0 and the query at t0 only
    t0 = 8
    g = np.zeros((B, L, H, d)); g[:, t0] = 1.0
    dq, dk_, dv_ = oracle.linattn_backward(q, k, v, g, norm=True)
    assert np.all(dq[:, :t0] == 0) and np.all(dq[:, t0 + 1:] == 0) and np.any(dq[:, t0] != 0)
    assert np.all(dk_[:, t0 + 1:] == 0) and np.all(dv_[:, t0 + 1:] == 0) and np.any(dk_[:, :t0 + 1] != 0)
