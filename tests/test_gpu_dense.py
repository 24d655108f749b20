"""GPU parity: chela_dense_fwd (Q/K/V formation building block) against the float64 oracle."""
import numpy as np
import pytest

import oracle
from paper_2406_08128_b200 import chela, inputs
from util import to_device, to_numpy

pytestmark = pytest.mark.gpu


def split_pair(a):
    hi = inputs.round_bf16(a.astype(np.float32))
    lo = inputs.round_bf16((a.astype(np.float64) - hi).astype(np.float32))
    return hi, lo


def pair_to_device(a):
    import torch
    hi, lo = split_pair(a)
    return torch.stack([to_device(hi, "bf16"), to_device(lo, "bf16")]).contiguous(), hi.astype(np.float64) + lo


@pytest.mark.parametrize("M,K,N", [(128, 64, 128), (256, 512, 256), (1000, 128, 384), (4096, 512, 1024), (100, 1024, 128), (300, 192, 512),
                                   (1, 64, 128)])
@pytest.mark.parametrize("a_pair,y_pair", [(False, False), (True, True), (False, True), (True, False)])
def test_tensor_core_path(M, K, N, a_pair, y_pair):
    import torch
    rng = np.random.default_rng(M + K + N)
    a = rng.standard_normal((M, K), dtype=np.float32) * 3
    w = inputs.round_bf16(rng.standard_normal((K, N), dtype=np.float32) / np.sqrt(K))
    bias = rng.standard_normal(N, dtype=np.float32) if M % 2 == 0 else None
    act = K == 512
    if a_pair:
        a_dev, a_val = pair_to_device(a)
    else:
        hi = inputs.round_bf16(a)
        a_dev, a_val = to_device(hi, "bf16"), hi.astype(np.float64)
    ws = torch.zeros(chela.lib().chela_dense_workspace_bytes(), dtype=torch.uint8, device="cuda")
    y = chela.dense_fwd(a_dev, to_device(w, "bf16"), None if bias is None else torch.from_numpy(bias).cuda(), act=act,
                        a_dtype=chela.BF16_PAIR if a_pair else chela.BF16,
                        y_dtype=chela.BF16_PAIR if y_pair else chela.BF16, workspace=ws)
    assert chela.async_status(ws) == chela.OK
    got = to_numpy(y)
    got = got[0] + got[1] if y_pair else got
    ref = oracle.dense(a_val, w, bias=bias, act=act)
    # fp32 accumulation + output storage: a bf16 pair keeps ~16 bits, a single bf16 8 bits, of the largest element
    tol = (2.0 ** -15 if y_pair else 2.0 ** -8) * np.abs(ref).max()
    assert np.abs(got - ref).max() <= tol


def test_simt_path_fp32_and_odd_shapes():
    import torch
    rng = np.random.default_rng(5)
    M, K, N = 77, 40, 24
    a = rng.standard_normal((M, K), dtype=np.float32)
    w = rng.standard_normal((K, N), dtype=np.float32)
    y = chela.dense_fwd(torch.from_numpy(a).cuda(), torch.from_numpy(w).cuda(), act=True, y_dtype=chela.F32)
    ref = oracle.dense(a, w, act=True)
    assert np.abs(to_numpy(y) - ref).max() <= 1e-5 * np.abs(ref).max()
    # a pair outside the tensor-core shapes is refused, not silently degraded
    a_dev, _ = pair_to_device(a)
    with pytest.raises(chela.ChelaError) as e:
        chela.dense_fwd(a_dev, to_device(inputs.round_bf16(w), "bf16"), a_dtype=chela.BF16_PAIR, y_dtype=chela.BF16)
    assert e.value.status == chela.ERR_UNSUPPORTED
