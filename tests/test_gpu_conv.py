"""GPU parity: short conv and long conv entry points against the float64 oracle."""
import numpy as np
import pytest

import oracle
from paper_2406_08128_b200 import chela, inputs
from util import rel_err, to_device, to_numpy

pytestmark = pytest.mark.gpu


def dev_f32(a):
    import torch
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).cuda()


@pytest.mark.parametrize("dtype,tol", [("f32", 1e-5), ("bf16", 1e-2)])
@pytest.mark.parametrize("B,L,D,width", [(2, 1, 8, 3), (1, 2, 16, 3), (3, 100, 40, 3), (2, 257, 512, 3),
                                         (1, 64, 24, 1), (1, 50, 8, 9), (1, 33, 8, 16)])
@pytest.mark.parametrize("act", [True, False])
def test_shortconv(dtype, tol, B, L, D, width, act):
    rng = np.random.default_rng(B * 1000 + L + D + width)
    x = inputs.round_storage(rng.standard_normal((B, L, D), dtype=np.float32), dtype)
    w = (rng.standard_normal((D, width), dtype=np.float32) / np.sqrt(width)).astype(np.float32)
    bias = rng.standard_normal(D, dtype=np.float32) if L % 2 else None
    got = to_numpy(chela.shortconv_fwd(to_device(x, dtype), dev_f32(w), None if bias is None else dev_f32(bias), act=act))
    ref = oracle.shortconv(x, w, bias=bias, act=act)
    if dtype == "bf16":  # output storage rounding only: half an ulp of the largest element
        assert np.abs(got - ref).max() <= 2.0 ** -8 * np.abs(ref).max()
    else:
        assert rel_err(got, ref) <= tol


@pytest.mark.parametrize("B,L,D", [(1, 1, 8), (2, 3, 8), (2, 5, 16), (1, 16, 8), (2, 17, 24), (1, 64, 8),
                                   (2, 1000, 40), (1, 1025, 8), (3, 2047, 8), (1, 4096, 16), (2, 5000, 8), (1, 8192, 8),
                                   (1, 16384, 8), (1, 16383, 8)])
@pytest.mark.parametrize("fused_short", [False, True])
def test_longconv_against_direct_and_fft_oracle(B, L, D, fused_short):
    m = inputs.mixer(300 + L, B, L, D, dtype="bf16", decay=0.001)
    x, k_long, w_short = m["x"], m["k_long"], m["w_short"]
    z = to_numpy(chela.longconv_fwd(to_device(x, "bf16"), dev_f32(k_long), dev_f32(w_short) if fused_short else None))
    a = oracle.shortconv(x, w_short, act=True) if fused_short else x.astype(np.float64)
    ref = oracle.longconv_fft(a, k_long)
    assert rel_err(z, ref) <= 2e-5
    if L <= 5000:
        assert rel_err(z, oracle.longconv_direct(a, k_long)) <= 2e-5
    # first sample has a single term: the product is the causal, not the circular, convolution
    assert np.allclose(z[:, 0], k_long[:, 0] * a[:, 0], rtol=1e-4, atol=1e-4)


@pytest.mark.parametrize("B,L,D", [(1, 16385, 8), (1, 32768, 8), (2, 40000, 16), (1, 65536, 8), (1, 100000, 8)])
@pytest.mark.parametrize("fused_short", [False, True])
def test_longconv_longer_than_one_shared_memory_row(B, L, D, fused_short):
    """Rows beyond 16384 tokens go block by block with the block spectra in the workspace (Eq. 6 has no length limit);
    also through the prepared-spectra entry point."""
    m = inputs.mixer(900 + L, B, L, D, dtype="bf16", decay=0.0002)
    x, k_long, w_short = m["x"], m["k_long"], m["w_short"]
    ws = dev_f32(w_short) if fused_short else None
    z = to_numpy(chela.longconv_fwd(to_device(x, "bf16"), dev_f32(k_long), ws))
    a = oracle.shortconv(x, w_short, act=True) if fused_short else x.astype(np.float64)
    ref = oracle.longconv_fft(a, k_long)
    assert rel_err(z, ref) <= 2e-5
    # every block boundary carries the tails of the blocks before it: check the samples around each on their own
    for t0 in range(16384, L, 16384):
        sl = slice(t0 - 4, min(L, t0 + 4))
        assert np.abs(z[:, sl] - ref[:, sl]).max() <= 2e-5 * np.abs(ref).max()
    assert np.allclose(z[:, 0], k_long[:, 0] * a[:, 0], rtol=1e-4, atol=1e-4)
    spec = chela.longconv_prepare(dev_f32(k_long))
    z2 = to_numpy(chela.longconv_prepared_fwd(to_device(x, "bf16"), spec, ws))
    assert np.array_equal(z2, z)


def test_longconv_f32_input_and_bf16_output():
    B, L, D = 2, 300, 16
    m = inputs.mixer(7, B, L, D, dtype="f32")
    z = to_numpy(chela.longconv_fwd(to_device(m["x"], "f32"), dev_f32(m["k_long"]), out_dtype=chela.BF16))
    ref = oracle.longconv_fft(m["x"], m["k_long"])
    assert np.abs(z - ref).max() <= 2.0 ** -8 * np.abs(ref).max()  # bf16 storage of the output


def test_reparameterised_short_kernels_match_the_parallel_pair():
    """Two parallel short kernels (width 3 and the length-dependent width) summed before SiLU, against one
    call with the merged kernel from chela_shortconv_reparam; both against the oracle."""
    import torch
    B, L, D = 2, 4096, 64
    w2 = chela.second_short_width(L)
    assert w2 == 9 and chela.second_short_width(1024) == 7 and chela.second_short_width(65536) == 11
    rng = np.random.default_rng(90)
    x = inputs.round_bf16(rng.standard_normal((B, L, D), dtype=np.float32))
    wa = rng.standard_normal((D, 3), dtype=np.float32) / 3
    wb = rng.standard_normal((D, w2), dtype=np.float32) / 3
    merged = chela.shortconv_reparam(dev_f32(wa), dev_f32(wb))
    ref_taps = wb.copy()
    ref_taps[:, :3] += wa
    assert np.array_equal(to_numpy(merged), ref_taps.astype(np.float64))
    y = to_numpy(chela.shortconv_fwd(to_device(x, "bf16"), merged, act=True))
    pre = oracle.shortconv(x, wa, act=False) + oracle.shortconv(x, wb, act=False)
    ref = pre / (1 + np.exp(-pre))
    assert np.abs(y - ref).max() <= 2.0 ** -8 * np.abs(ref).max()
    # and through the fused long-conv entry point (width 9 takes the generic short-conv path)
    k_long = (rng.standard_normal((D, L), dtype=np.float32) * np.exp(-0.001 * np.arange(L))).astype(np.float32)
    z = to_numpy(chela.longconv_fwd(to_device(x, "bf16"), dev_f32(k_long), merged))
    assert rel_err(z, oracle.longconv_fft(ref, k_long)) <= 2e-5
