"""GPU parity: chela_linattn_fwd (through the C ABI) against the float64 oracle."""
import numpy as np
import pytest

import oracle
from paper_2406_08128_b200 import chela, inputs
from util import rel_err, to_device, to_numpy

pytestmark = pytest.mark.gpu

TOL = {"f32": 1e-4, "bf16": 2e-2}   # max|err| / RMS(oracle output)


def run(q, k, v, dtype, chunk, norm=True, scale=1.0, out_dtype=chela.F32):
    import torch
    o = chela.linattn_fwd(to_device(q, dtype), to_device(k, dtype), to_device(v, dtype), chunk=chunk,
                          out_dtype=out_dtype, norm=chela.NORM_RMS if norm else chela.NORM_NONE, scale=scale)
    torch.cuda.synchronize()
    return to_numpy(o)


def test_config1_fp32_quadratic_and_recurrent():
    # B=1, H=1, L=1024, d=64, C=64, seed 0, N(0,1)/sqrt(64)
    q, k, v = inputs.qkv(0, 1, 1024, 1, 64, 64, "f32")
    for norm in (True, False):
        got = run(q, k, v, "f32", 64, norm=norm)
        assert rel_err(got, oracle.linattn_quadratic(q, k, v, norm=norm)) <= TOL["f32"]
        assert rel_err(got, oracle.linattn_recurrent(q, k, v, norm=norm)) <= TOL["f32"]


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("d,chunk", [(64, 64), (64, 128), (128, 64), (128, 128)])
@pytest.mark.parametrize("L", [1, 63, 64, 65, 200, 333])
def test_small_shapes_ragged_tails(dtype, d, chunk, L):
    B, H = 2, 3
    q, k, v = inputs.qkv(10 + L, B, L, H, d, d, dtype)
    for norm in (True, False):
        got = run(q, k, v, dtype, chunk, norm=norm)
        ref = oracle.linattn_recurrent(q, k, v, norm=norm)
        assert rel_err(got, ref) <= TOL[dtype], (dtype, d, chunk, L, norm)


def test_config2_bf16_full_size():
    # B=8, H=8, L=4096, d=64, C=64
    q, k, v = inputs.qkv(1, 8, 4096, 8, 64, 64, "bf16")
    got = run(q, k, v, "bf16", 64)
    ref = oracle.linattn_recurrent(q, k, v)
    assert rel_err(got, ref) <= TOL["bf16"]
    # a few (b,h) pairs also against the quadratic definition
    for b, h in ((0, 0), (7, 7), (3, 5)):
        sl = (slice(b, b + 1), slice(None), slice(h, h + 1))
        quad = oracle.linattn_quadratic(q[sl], k[sl], v[sl])
        assert rel_err(got[sl], quad) <= TOL["bf16"]


def test_chunk_invariance_and_causality_on_gpu():
    q, k, v = inputs.qkv(5, 2, 700, 4, 64, 64, "bf16")
    a = run(q, k, v, "bf16", 64)
    b = run(q, k, v, "bf16", 128)
    assert rel_err(a, b) <= TOL["bf16"]
    q2, k2, v2 = inputs.qkv(6, 2, 700, 4, 64, 64, "bf16")
    t0 = 389
    for x, y in ((q2, q), (k2, k), (v2, v)):
        x[:, :t0] = y[:, :t0]
    c = run(q2, k2, v2, "bf16", 64)
    assert np.array_equal(a[:, :t0], c[:, :t0])
    assert not np.allclose(a[:, t0:], c[:, t0:])


def test_scale_and_bf16_output():
    q, k, v = inputs.qkv(7, 1, 300, 2, 64, 64, "bf16")
    got = run(q, k, v, "bf16", 64, norm=False, scale=0.125)
    assert rel_err(got, oracle.linattn_recurrent(q, k, v, scale=0.125, norm=False)) <= TOL["bf16"]
    got = run(q, k, v, "bf16", 64, out_dtype=chela.BF16)
    # bf16 storage costs up to half an ulp (2^-8 relative) of the largest element on top of the bound
    ref = oracle.linattn_recurrent(q, k, v)
    assert np.abs(got - ref).max() <= 2e-2 * np.sqrt(np.mean(ref ** 2)) + 2.0 ** -8 * np.abs(ref).max()


@pytest.mark.parametrize("B,L", inputs.sweep_shapes())
def test_sweep_shapes_sampled(B, L):
    """Full sweep sizes (B*L = 262144, H=16, d=64, C=64): the oracle checks sampled (b,h) pairs."""
    import torch
    H, d = 16, 64
    q, k, v = inputs.qkv(100 + int(np.log2(L)), B, L, H, d, d, "bf16")
    o = chela.linattn_fwd(to_device(q, "bf16"), to_device(k, "bf16"), to_device(v, "bf16"), chunk=64)
    torch.cuda.synchronize()
    rng = np.random.default_rng(L)
    pairs = {(0, 0), (B - 1, H - 1)} | {(int(rng.integers(B)), int(rng.integers(H))) for _ in range(4)}
    for b, h in pairs:
        sl = (slice(b, b + 1), slice(None), slice(h, h + 1))
        ref = oracle.linattn_recurrent(q[sl], k[sl], v[sl])
        got = to_numpy(o[b:b + 1, :, h:h + 1])
        assert rel_err(got, ref) <= TOL["bf16"], (B, L, b, h)
    assert bool(torch.isfinite(o).all())


@pytest.mark.parametrize("B,L,H", [(1, 8192, 2), (1, 5000, 3), (1, 2100, 1)])
def test_sequences_split_along_length_head_dim_128(B, L, H):
    q, k, v = inputs.qkv(45 + L, B, L, H, 128, 128, "bf16")
    assert chela.linattn_workspace_bytes(B, H, L, 128, 128, 64) >= 512 + 128 * 128 * 4
    got = run(q, k, v, "bf16", 128)
    assert rel_err(got, oracle.linattn_recurrent(q, k, v)) <= TOL["bf16"]


@pytest.mark.parametrize("B,L,H", [(1, 8192, 2), (1, 5000, 3), (1, 2100, 1), (2, 4096, 1)])
def test_sequences_split_along_length(B, L, H):
    """Few (batch, head) pairs: the tensor-core path splits each sequence into groups of chunks whose
    initial states come from a separate K^T V pass; the result must still match the oracle."""
    import torch
    q, k, v = inputs.qkv(40 + L, B, L, H, 64, 64, "bf16")
    assert chela.linattn_workspace_bytes(B, H, L, 64, 64, 64) > 512 + 64 * 64 * 4 - 1
    for norm in (True, False):
        got = run(q, k, v, "bf16", 64, norm=norm)
        assert rel_err(got, oracle.linattn_recurrent(q, k, v, norm=norm)) <= TOL["bf16"]


def test_async_status_is_ok_and_tensor_core_path_is_used():
    import torch
    assert chela.linattn_kernel_kind(2, 2, 256, 64, 64, 64, chela.BF16, chela.F32) == 2
    assert chela.linattn_kernel_kind(2, 2, 256, 128, 128, 128, chela.BF16, chela.F32) == 2
    assert chela.linattn_kernel_kind(2, 2, 256, 128, 128, 128, chela.F32, chela.F32) == 1
    assert chela.linattn_kernel_kind(2, 2, 256, 64, 64, 64, chela.F32, chela.F32) == 1
    q, k, v = inputs.qkv(3, 2, 256, 2, 64, 64, "bf16")
    ws = torch.zeros(chela.linattn_workspace_bytes(2, 2, 256, 64, 64, 64), dtype=torch.uint8, device="cuda")
    chela.linattn_fwd(to_device(q, "bf16"), to_device(k, "bf16"), to_device(v, "bf16"), workspace=ws)
    assert chela.async_status(ws) == chela.OK


def test_workspace_too_small_is_rejected():
    import torch
    q, k, v = (to_device(a, "bf16") for a in inputs.qkv(3, 1, 4096, 1, 64, 64, "bf16"))
    need = chela.linattn_workspace_bytes(1, 1, 4096, 64, 64, 64)
    ws = torch.zeros(need - 16, dtype=torch.uint8, device="cuda")
    with pytest.raises(chela.ChelaError) as e:
        chela.linattn_fwd(q, k, v, workspace=ws)
    assert e.value.status == chela.ERR_WORKSPACE


def _pair(a):
    import torch
    hi = inputs.round_bf16(a.astype(np.float32))
    lo = inputs.round_bf16((a.astype(np.float64) - hi).astype(np.float32))
    return torch.stack([to_device(hi, "bf16"), to_device(lo, "bf16")]).contiguous(), hi.astype(np.float64) + lo


@pytest.mark.parametrize("B,L,H", [(1, 64, 1), (1, 200, 2), (2, 1000, 3), (1, 8192, 2), (3, 4096, 8)])
@pytest.mark.parametrize("norm", [True, False])
@pytest.mark.parametrize("d", [64, 128])
def test_bf16_pair_inputs_reach_fp32_like_accuracy(B, L, H, norm, d):
    """Q, K, V as bf16 pairs (hi + lo planes): three-term tensor-core products, error far below the
    single-bf16 bound (this is the mixer's attention path)."""
    rng = np.random.default_rng(B + L + H)
    q, k, v = (rng.standard_normal((B, L, H, d), dtype=np.float32) * 2 for _ in range(3))
    (qd, qv), (kd, kv), (vd, vv) = _pair(q), _pair(k), _pair(v)
    assert chela.linattn_kernel_kind(B, H, L, d, d, 64, chela.BF16_PAIR, chela.F32) == 2
    o = chela.linattn_fwd(qd, kd, vd, chunk=64, norm=chela.NORM_RMS if norm else chela.NORM_NONE, in_dtype=chela.BF16_PAIR)
    ref = oracle.linattn_recurrent(qv, kv, vv, norm=norm)
    assert rel_err(to_numpy(o), ref) <= 5e-4


@pytest.mark.parametrize("B,L,H,d", [(2, 8192, 2, 64), (16, 2048, 16, 64), (1, 8192, 2, 128)])
def test_calls_can_be_captured_in_a_cuda_graph(B, L, H, d):
    """The library only enqueues work on the caller's stream (memset, kernels, a programmatic dependent launch for
    split sequences), so a call with caller-owned output and workspace can be captured and replayed; the replay
    gives the eager call's bits."""
    import torch
    q, k, v = (to_device(a, "bf16") for a in inputs.qkv(7, B, L, H, d, d, "bf16"))
    o_eager = torch.empty(B, L, H, d, device="cuda")
    o_graph = torch.empty_like(o_eager)
    ws = torch.zeros(chela.linattn_workspace_bytes(B, H, L, d, d, 64) + 16, dtype=torch.uint8, device="cuda")
    chela.linattn_fwd(q, k, v, out=o_eager, workspace=ws)
    torch.cuda.synchronize()
    graph, side = torch.cuda.CUDAGraph(), torch.cuda.Stream()
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            chela.linattn_fwd(q, k, v, out=o_graph, workspace=ws)
    graph.replay()
    graph.replay()
    torch.cuda.synchronize()
    assert chela.async_status(ws) == chela.OK
    assert torch.equal(o_eager, o_graph)


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
@pytest.mark.parametrize("d", [64, 128])
def test_degenerate_inputs_zero_rows_and_all_ones(dtype, d):
    """Zero queries give exactly zero rows through the normaliser (no NaN from 0 * rsqrt(eps)); all-ones inputs give
    the closed form r_t = (t + 1) d, whose normalised rows are all ones (a row of equal entries has RMS = |entry|)."""
    import torch
    B, L, H = 2, 300, 2
    dt = torch.bfloat16 if dtype == "bf16" else torch.float32
    ones = torch.ones(B, L, H, d, device="cuda", dtype=dt)
    zeros = torch.zeros_like(ones)
    o = chela.linattn_fwd(zeros, ones, ones)
    assert bool((o == 0).all())
    o = chela.linattn_fwd(ones, ones, zeros)
    assert bool((o == 0).all())
    r = chela.linattn_fwd(ones, ones, ones, norm=chela.NORM_NONE)
    t = torch.arange(1, L + 1, device="cuda", dtype=torch.float32)[None, :, None, None] * d
    assert bool((r == t.expand_as(r)).all())      # exact: small integers in fp32 accumulation
    o = chela.linattn_fwd(ones, ones, ones)
    assert float((o - 1).abs().max()) <= 1e-6


@pytest.mark.parametrize("B,L,H,d", [(1, 2100, 1, 64), (3, 4100, 1, 64), (2, 16384, 8, 64), (8, 4096, 8, 64), (1, 65536, 2, 64),
                                     (37, 2048, 4, 64), (1, 8192, 2, 128), (2, 16384, 4, 128)])
@pytest.mark.parametrize("pair", [False, True])
def test_queued_calls_are_deterministic(B, L, H, d, pair):
    """Twelve calls queued without a host synchronisation (unsplit and split shapes, where the state kernel and the
    main kernel of a call overlap): the same bits every time, no wait gives up, and no call takes the second that a
    give-up would cost."""
    import time
    import torch
    gen = torch.Generator(device="cuda").manual_seed(11)
    shape = (2, B, L, H, d) if pair else (B, L, H, d)
    q, k, v = ((torch.randn(shape, device="cuda", generator=gen) * 0.125).to(torch.bfloat16) for _ in range(3))
    if pair:   # low planes three orders of magnitude below the high planes, as a real hi/lo split has them
        for t in (q, k, v):
            t[1] *= 2.0 ** -9
    kw = {"in_dtype": chela.BF16_PAIR} if pair else {}
    ws = torch.zeros(chela.linattn_workspace_bytes(B, H, L, d, d, 64) + 16, dtype=torch.uint8, device="cuda")
    o = torch.empty(B, L, H, d, device="cuda")
    first = chela.linattn_fwd(q, k, v, out=o, workspace=ws, **kw).clone()
    torch.cuda.synchronize()
    outs = []
    for _ in range(12):
        outs.append(chela.linattn_fwd(q, k, v, out=torch.empty_like(o), workspace=ws, **kw))
    torch.cuda.synchronize()
    assert chela.async_status(ws) == chela.OK   # no bounded wait gave up
    assert bool(torch.isfinite(first).all())
    for x in outs:
        assert torch.equal(first, x)
