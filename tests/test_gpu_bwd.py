"""GPU parity: chela_linattn_bwd against the float64 oracle (gradients from the definition)."""
import numpy as np
import pytest

import oracle
from paper_2406_08128_b200 import chela, inputs
from util import rel_err, to_device, to_numpy

pytestmark = pytest.mark.gpu

TOLB = 1e-4


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("B,L,H,d", [(1, 1, 1, 64), (2, 63, 2, 64), (1, 300, 3, 64), (2, 1000, 2, 64), (1, 200, 2, 128),
                                     (1, 777, 1, 128),
                                     (1, 2100, 1, 64), (1, 2100, 1, 128)])   # the last two: split along L (state kernel)
@pytest.mark.parametrize("norm", [True, False])
def test_gradients_match_the_oracle(dtype, B, L, H, d, norm):
    q, k, v = inputs.qkv(70 + L + d, B, L, H, d, d, dtype)
    d_o = inputs.qkv(71 + L + d, B, L, H, d, d, dtype, std=1.0)[0]
    dq, dk, dv = chela.linattn_bwd(*(to_device(a, dtype) for a in (q, k, v, d_o)),
                                   norm=chela.NORM_RMS if norm else chela.NORM_NONE, scale=0.5)
    rq, rk, rv = oracle.linattn_backward(q, k, v, d_o, scale=0.5, norm=norm)
    # fp32 arithmetic on inputs that are exact in the storage dtype: the fp32 bound of the forward pass.
    # With a single token the normaliser makes g orthogonal to r up to eps / n^2, so dq and dk are a small
    # residual of a cancellation: that one case gets an order of magnitude more.
    tol = 1e-3 if (L == 1 and norm) else TOLB
    if dtype == "bf16":
        # tensor-core path.  Without the normaliser the scores and G are single bf16 values like the forward
        # pass; with it every rounded intermediate (scores, state, G) is carried as a bf16 pair.
        tol = 1e-3 if norm else 2e-2
    for got, ref in ((dq, rq), (dk, rk), (dv, rv)):
        assert rel_err(to_numpy(got), ref) <= tol, rel_err(to_numpy(got), ref)


def test_backward_argument_checks():
    import torch
    q = torch.zeros(1, 64, 1, 64, device="cuda")
    with pytest.raises(chela.ChelaError) as e:
        chela.linattn_bwd(q, q, q, q, workspace=torch.zeros(16, dtype=torch.uint8, device="cuda"))
    assert e.value.status == chela.ERR_WORKSPACE
    q32 = torch.zeros(1, 64, 1, 32, device="cuda")
    with pytest.raises(chela.ChelaError) as e:
        chela.linattn_bwd(q32, q32, q32, q32, workspace=torch.zeros(1 << 20, dtype=torch.uint8, device="cuda"))
    assert e.value.status == chela.ERR_UNSUPPORTED


def test_backward_at_the_benchmark_size_by_directional_derivatives():
    """B16 L16384 H16 d64 bf16, the launch configuration the benchmark times.  The O(L^2) gradient oracle takes most
    of a minute per head there, so the check uses a property that holds at any size: for sampled (batch, head)
    pairs, the gradients' inner product with a direction equals the central difference of the float64 oracle's
    forward pass along that direction.  Directions: the computed gradient itself (overall scale), and random
    directions confined to one token row of q, k or v (64 numbers, so that the inner product is a sizeable
    fraction of |g_row| |direction| and a wrong row shows)."""
    import torch
    B, L, H, d = 16, 16384, 16, 64
    q, k, v = inputs.qkv(90, B, L, H, d, d, "bf16")
    d_o = inputs.qkv(91, B, L, H, d, d, "bf16", std=1.0)[0]
    dq, dk, dv = chela.linattn_bwd(*(to_device(a, "bf16") for a in (q, k, v, d_o)), norm=chela.NORM_RMS, scale=1.0)
    torch.cuda.synchronize()
    rng = np.random.default_rng(92)

    def central_difference(x, go, dirs, eps):
        f = [float((go * oracle.linattn_recurrent(*[a + s * eps * dd for a, dd in zip(x, dirs)])).sum()) for s in (1.0, -1.0)]
        return (f[0] - f[1]) / (2 * eps)

    for b, h in ((0, 0), (B - 1, H - 1), (int(rng.integers(B)), int(rng.integers(H)))):
        sl = (slice(b, b + 1), slice(None), slice(h, h + 1))
        x = [np.asarray(a[sl], dtype=np.float64) for a in (q, k, v)]
        go = np.asarray(d_o[sl], dtype=np.float64)
        grads = [to_numpy(g[b:b + 1, :, h:h + 1]).astype(np.float64) for g in (dq, dk, dv)]
        # along the gradient: num = <g_true, g>, ana = |g|^2
        gnorm2 = sum(float((g * g).sum()) for g in grads)
        num = central_difference(x, go, grads, 1e-4 / np.sqrt(gnorm2 / (3 * L * d)))
        assert abs(num - gnorm2) <= 2e-3 * gnorm2, (b, h, num, gnorm2)
        # one token row of one operand at a time (early, late and random tokens)
        for which in range(3):
            for t in (0, L - 1, int(rng.integers(L)), int(rng.integers(L))):
                dirs = [np.zeros_like(a) for a in x]
                dirs[which][0, t, 0, :] = rng.standard_normal(d)
                grow, drow = grads[which][0, t, 0, :], dirs[which][0, t, 0, :]
                ana = float((grow * drow).sum())
                num = central_difference(x, go, dirs, 1e-3)
                assert abs(num - ana) <= 1e-2 * np.linalg.norm(grow) * np.linalg.norm(drow), (b, h, which, t, num, ana)


@pytest.mark.parametrize("B,L,H,d", [(1, 16384, 8, 64), (4, 32768, 16, 64), (1, 16384, 4, 128), (16, 4096, 16, 64)])
def test_back_to_back_backward_calls_on_split_sequences(B, L, H, d):
    """Calls queued without a host synchronisation in between (split sequences: every launch is a state kernel
    plus a main kernel that starts beside it).  No wait may give up (a give-up costs about a second and sets the
    status word, which the later launches of a call must not erase), and every call returns the first call's bits."""
    import time
    import torch
    gen = torch.Generator(device="cuda").manual_seed(5)
    q, k, v = ((torch.randn((B, L, H, d), device="cuda", generator=gen) * 0.125).to(torch.bfloat16) for _ in range(3))
    d_o = torch.randn((B, L, H, d), device="cuda", generator=gen).to(torch.bfloat16)
    ws = torch.zeros(int(chela.lib().chela_linattn_bwd_workspace_bytes(B, H, L, d, d)), dtype=torch.uint8, device="cuda")
    first = [g.clone() for g in chela.linattn_bwd(q, k, v, d_o, workspace=ws)]
    torch.cuda.synchronize()
    for _ in range(8):
        grads = chela.linattn_bwd(q, k, v, d_o, workspace=ws)
    torch.cuda.synchronize()
    assert chela.async_status(ws) == chela.OK   # no bounded wait gave up
    for a, b in zip(first, grads):
        assert torch.equal(a, b)
