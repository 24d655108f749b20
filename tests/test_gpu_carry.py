"""GPU parity: state carry across calls (segment-wise sequential evaluation) against the float64 oracle."""
import numpy as np
import pytest

import oracle
from paper_2406_08128_b200 import chela, inputs
from util import rel_err, to_device, to_numpy

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("dtype,tol,d", [("bf16", 2e-2, 64), ("bf16", 2e-2, 128), ("f32", 1e-4, 64), ("f32", 1e-4, 128)])
@pytest.mark.parametrize("B,H,cuts", [(2, 3, (0, 100, 101, 400, 1000)), (1, 2, (0, 4096, 9000)), (1, 1, (0, 1, 2, 3, 70))])
def test_segments_with_carried_state_equal_one_call(dtype, tol, d, B, H, cuts):
    import torch
    L = cuts[-1]
    q, k, v = inputs.qkv(50 + L + d, B, L, H, d, d, dtype)
    ref, ref_state = oracle.linattn_recurrent(q, k, v, return_state=True)
    state = None
    outs = []
    for a, b in zip(cuts[:-1], cuts[1:]):
        qs, ks, vs = (to_device(np.ascontiguousarray(x[:, a:b]), dtype) for x in (q, k, v))
        o, state = chela.linattn_carry_fwd(qs, ks, vs, state_in=state)
        outs.append(to_numpy(o))
    got = np.concatenate(outs, axis=1)
    assert rel_err(got, ref) <= tol
    # the final state is K^T V of the whole sequence (fp32 accumulation)
    assert np.abs(to_numpy(state) - ref_state).max() <= (2e-3 if dtype == "bf16" else 1e-5) * np.abs(ref_state).max()


def test_state_out_without_state_in_and_oracle_state_in():
    import torch
    B, L, H, d = 1, 300, 2, 64
    q, k, v = inputs.qkv(60, B, L, H, d, d, "bf16")
    rng = np.random.default_rng(61)
    s0 = rng.standard_normal((B, H, d, d)).astype(np.float32)
    ref, ref_state = oracle.linattn_recurrent(q, k, v, state_in=s0, return_state=True)
    o, s1 = chela.linattn_carry_fwd(to_device(q, "bf16"), to_device(k, "bf16"), to_device(v, "bf16"),
                                    state_in=torch.from_numpy(s0).cuda())
    assert rel_err(to_numpy(o), ref) <= 2e-2
    assert np.abs(to_numpy(s1) - ref_state).max() <= 2e-3 * np.abs(ref_state).max()
