"""GPU parity: chela_mixer_fwd against the float64 oracle composition."""
import numpy as np
import pytest

import oracle
from paper_2406_08128_b200 import chela, inputs
from util import rel_err, to_device, to_numpy

pytestmark = pytest.mark.gpu

TOL = 2e-2


def dev_f32(a):
    import torch
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).cuda()


def run_mixer(m, H, chunk, dtype="bf16", **kw):
    o = chela.mixer_fwd(to_device(m["x"], dtype), dev_f32(m["w_short"]), dev_f32(m["k_long"]),
                        to_device(m["w_q"], dtype), to_device(m["w_k"], dtype), to_device(m["w_v"], dtype),
                        H, chunk=chunk, **kw)
    return to_numpy(o)


@pytest.mark.parametrize("B,L,D,H,chunk", [(2, 300, 128, 2, 64), (1, 1000, 256, 2, 128), (2, 2048, 512, 8, 64),
                                           (1, 100, 64, 1, 64)])
def test_mixer_small(B, L, D, H, chunk):
    m = inputs.mixer(2, B, L, D)
    got = run_mixer(m, H, chunk)
    ref = oracle.mixer(m["x"], m["w_short"], m["k_long"], m["w_q"], m["w_k"], m["w_v"], H)
    assert rel_err(got, ref) <= TOL
    raw = run_mixer(m, H, chunk, norm=chela.NORM_NONE)
    ref_raw = oracle.mixer(m["x"], m["w_short"], m["k_long"], m["w_q"], m["w_k"], m["w_v"], H, norm=False)
    assert rel_err(raw, ref_raw) <= TOL


def test_mixer_qk_diag_biases_and_no_silu():
    B, L, D, H = 2, 500, 128, 2
    m = inputs.mixer(3, B, L, D)
    rng = np.random.default_rng(4)
    aq = inputs.round_bf16(rng.standard_normal(D, dtype=np.float32) / 12)
    ak = inputs.round_bf16(rng.standard_normal(D, dtype=np.float32) / 12)
    bq, bk, bv = (rng.standard_normal(D, dtype=np.float32) * 0.1 for _ in range(3))
    o = chela.mixer_fwd(to_device(m["x"], "bf16"), dev_f32(m["w_short"]), dev_f32(m["k_long"]),
                        to_device(aq, "bf16"), to_device(ak, "bf16"), to_device(m["w_v"], "bf16"), H,
                        b_q=dev_f32(bq), b_k=dev_f32(bk), b_v=dev_f32(bv), qk_diag=True, v_silu=False)
    ref = oracle.mixer(m["x"], m["w_short"], m["k_long"], aq, ak, m["w_v"], H, b_q=bq, b_k=bk, b_v=bv,
                       qk_diag=True, v_silu=False)
    assert rel_err(to_numpy(o), ref) <= TOL


def test_mixer_config4_shape_reduced_length():
    """Config 4 layer (D=1024, H=8, head dim 128, C=128) at L=2048 so that the oracle finishes in seconds."""
    B, L, D, H = 1, 2048, 1024, 8
    m = inputs.mixer(3, B, L, D)
    got = run_mixer(m, H, 128)
    ref = oracle.mixer(m["x"], m["w_short"], m["k_long"], m["w_q"], m["w_k"], m["w_v"], H)
    assert rel_err(got, ref) <= TOL


def test_mixer_config3_shape_one_batch():
    """Config 3 layer (D=512, H=8, L=16384, C=64) on one batch row: the oracle's FFT form finishes in seconds."""
    B, L, D, H = 1, 16384, 512, 8
    m = inputs.mixer(2, B, L, D)
    got = run_mixer(m, H, 64)
    ref = oracle.mixer(m["x"], m["w_short"], m["k_long"], m["w_q"], m["w_k"], m["w_v"], H)
    assert rel_err(got, ref) <= TOL


@pytest.mark.parametrize("seed,B,L,D,H,chunk", [(2, 4, 16384, 512, 8, 64), (3, 8, 8192, 1024, 8, 128)])
def test_mixer_configs_3_and_4_full_size_sampled_rows(seed, B, L, D, H, chunk):
    """Configs 3 and 4 at their full sizes, i.e. the launch configuration the benchmark times; the oracle checks
    the first and the last batch row (rows are independent: a row's oracle takes its slice of x alone)."""
    m = inputs.mixer(seed, B, L, D)
    got = run_mixer(m, H, chunk)
    assert np.isfinite(got).all()
    for b in (0, B - 1):
        ref = oracle.mixer(m["x"][b:b + 1], m["w_short"], m["k_long"], m["w_q"], m["w_k"], m["w_v"], H)
        assert rel_err(got[b:b + 1], ref) <= TOL, b


@pytest.mark.parametrize("B,L,D,H,chunk,dtype", [(2, 300, 128, 2, 64, "bf16"), (1, 1000, 256, 2, 128, "bf16"),
                                                 (1, 2048, 512, 8, 64, "bf16"), (1, 200, 64, 1, 64, "f32")])
def test_gated_mixer(B, L, D, H, chunk, dtype):
    m = inputs.mixer(5, B, L, D, dtype=dtype)
    rng = np.random.default_rng(6)
    w_a, w_o = (inputs.round_storage(rng.standard_normal((D, D), dtype=np.float32) / np.sqrt(D) / 12, dtype) for _ in range(2))
    b_a, b_o = (rng.standard_normal(D, dtype=np.float32) * 0.5 for _ in range(2))
    dev = lambda a: to_device(a, dtype)
    u = chela.mixer_gated_fwd(dev(m["x"]), dev_f32(m["w_short"]), dev_f32(m["k_long"]), dev(m["w_q"]), dev(m["w_k"]),
                              dev(m["w_v"]), dev(w_a), dev(w_o), H, chunk=chunk, b_a=dev_f32(b_a), b_o=dev_f32(b_o))
    ref = oracle.mixer_gated(m["x"], m["w_short"], m["k_long"], m["w_q"], m["w_k"], m["w_v"], w_a, w_o, H, b_a=b_a, b_o=b_o)
    assert rel_err(to_numpy(u), ref) <= TOL


@pytest.mark.parametrize("seed,B,L,D,H,chunk", [(12, 4, 16384, 512, 8, 64), (13, 8, 8192, 1024, 8, 128)])
def test_gated_mixer_configs_3_and_4_full_size_sampled_rows(seed, B, L, D, H, chunk):
    """The gated call (Eqs. 8, 9, 13, 14) at the full sizes of configs 3 and 4; the oracle checks the first and last batch row."""
    m = inputs.mixer(seed, B, L, D)
    rng = np.random.default_rng(seed + 100)
    w_a, w_o = (inputs.round_storage(rng.standard_normal((D, D), dtype=np.float32) / np.sqrt(D) / 12, "bf16") for _ in range(2))
    b_a, b_o = (rng.standard_normal(D, dtype=np.float32) * 0.5 for _ in range(2))
    dev = lambda a: to_device(a, "bf16")
    u = to_numpy(chela.mixer_gated_fwd(dev(m["x"]), dev_f32(m["w_short"]), dev_f32(m["k_long"]), dev(m["w_q"]), dev(m["w_k"]),
                                       dev(m["w_v"]), dev(w_a), dev(w_o), H, chunk=chunk, b_a=dev_f32(b_a), b_o=dev_f32(b_o)))
    assert np.isfinite(u).all()
    for b in (0, B - 1):
        ref = oracle.mixer_gated(m["x"][b:b + 1], m["w_short"], m["k_long"], m["w_q"], m["w_k"], m["w_v"], w_a, w_o, H,
                                 b_a=b_a, b_o=b_o)
        assert rel_err(u[b:b + 1], ref) <= TOL, b


@pytest.mark.parametrize("B,L,D,H", [(1, 32768, 128, 2), (2, 40000, 128, 1)])
def test_mixer_on_sequences_longer_than_one_fft_row(B, L, D, H):
    """L > 16384: the long convolution goes block by block; the rest of the layer is the same path."""
    m = inputs.mixer(21, B, L, D, decay=0.0003)
    got = run_mixer(m, H, 64)
    ref = oracle.mixer(m["x"], m["w_short"], m["k_long"], m["w_q"], m["w_k"], m["w_v"], H)
    assert rel_err(got, ref) <= TOL


def test_mixer_call_can_be_captured_in_a_cuda_graph():
    import torch
    B, L, D, H = 1, 2048, 512, 8
    m = inputs.mixer(9, B, L, D)
    args = (to_device(m["x"], "bf16"), dev_f32(m["w_short"]), dev_f32(m["k_long"]), to_device(m["w_q"], "bf16"),
            to_device(m["w_k"], "bf16"), to_device(m["w_v"], "bf16"), H)
    ws = torch.zeros(chela.mixer_workspace_bytes(B, L, D, H, 64), dtype=torch.uint8, device="cuda")
    o_eager = torch.empty(B, L, D, device="cuda")
    o_graph = torch.empty_like(o_eager)
    chela.mixer_fwd(*args, chunk=64, out=o_eager, workspace=ws)
    torch.cuda.synchronize()
    graph, side = torch.cuda.CUDAGraph(), torch.cuda.Stream()
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            chela.mixer_fwd(*args, chunk=64, out=o_graph, workspace=ws)
    graph.replay()
    torch.cuda.synchronize()
    assert torch.equal(o_eager, o_graph)


@pytest.mark.parametrize("B,L,D,H,chunk", [(1, 2048, 512, 8, 64), (2, 1000, 256, 2, 128), (1, 4096, 1024, 8, 128)])
def test_queued_mixer_calls_are_deterministic(B, L, D, H, chunk):
    import torch
    m = inputs.mixer(10, B, L, D)
    args = (to_device(m["x"], "bf16"), dev_f32(m["w_short"]), dev_f32(m["k_long"]), to_device(m["w_q"], "bf16"),
            to_device(m["w_k"], "bf16"), to_device(m["w_v"], "bf16"), H)
    ws = torch.zeros(chela.mixer_workspace_bytes(B, L, D, H, chunk), dtype=torch.uint8, device="cuda")
    first = chela.mixer_fwd(*args, chunk=chunk, workspace=ws).clone()
    torch.cuda.synchronize()
    outs = [chela.mixer_fwd(*args, chunk=chunk, workspace=ws) for _ in range(8)]
    torch.cuda.synchronize()
    assert chela.async_status(ws) == chela.OK
    for o in outs:
        assert torch.equal(first, o)


@pytest.mark.parametrize("B,L,D,H", [(2, 1500, 128, 2), (1, 300, 64, 1), (1, 2048, 256, 4)])
def test_prepared_spectra_give_the_same_mixer_and_long_convolution(B, L, D, H):
    """chela_longconv_prepare + the *_prepared_fwd calls: the kernel spectra computed once for constant weights.  Same
    kernels on the same spectra, so the outputs equal those of the unprepared calls bit for bit, and the oracle's
    within the bound."""
    import torch
    m = inputs.mixer(11, B, L, D)
    x, ws_, kl = to_device(m["x"], "bf16"), dev_f32(m["w_short"]), dev_f32(m["k_long"])
    wq, wk, wv = (to_device(m[n], "bf16") for n in ("w_q", "w_k", "w_v"))
    spec = chela.longconv_prepare(kl)
    z0 = chela.longconv_fwd(x, kl, ws_)
    z1 = chela.longconv_prepared_fwd(x, spec, ws_)
    assert torch.equal(z0, z1)
    assert rel_err(to_numpy(z1), oracle.longconv_fft(oracle.shortconv(m["x"], m["w_short"]), m["k_long"])) <= 2e-5
    o0 = chela.mixer_fwd(x, ws_, kl, wq, wk, wv, H)
    o1 = chela.mixer_prepared_fwd(x, ws_, spec, wq, wk, wv, H)
    o2 = chela.mixer_prepared_fwd(x, ws_, spec, wq, wk, wv, H)   # the buffer is read, never written
    assert torch.equal(o0, o1) and torch.equal(o1, o2)
    assert rel_err(to_numpy(o1), oracle.mixer(m["x"], m["w_short"], m["k_long"], m["w_q"], m["w_k"], m["w_v"], H)) <= TOL
    # a buffer that is too small, and the missing spectrum, are refused before anything is launched
    small = torch.empty(64, dtype=torch.uint8, device="cuda")
    assert chela.lib().chela_longconv_prepare(kl.data_ptr(), L, D, small.data_ptr(), small.numel(), None) == chela.ERR_WORKSPACE
    with pytest.raises(chela.ChelaError):
        chela.mixer_prepared_fwd(x, ws_, None, wq, wk, wv, H)
