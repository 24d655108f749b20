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


@pytest.mark.parametrize("d", [64, 128])
def test_aliased_state_on_sequences_that_several_ctas_share(d):
    """state_in and state_out the same buffer, on a shape where a sequence is shared between CTAs (d = 64: by stride)
    or split along L (d = 128): every CTA starts from the initial state although one of them overwrites the buffer."""
    import torch
    B, H, L = 1, 2, 8192
    q, k, v = inputs.qkv(66 + d, B, 2 * L, H, d, d, "bf16")
    ref, ref_state = oracle.linattn_recurrent(q, k, v, return_state=True)
    state = torch.zeros(B, H, d, d, device="cuda")
    outs = []
    for a in (0, L):
        qs, ks, vs = (to_device(np.ascontiguousarray(x[:, a:a + L]), "bf16") for x in (q, k, v))
        o, _ = chela.linattn_carry_fwd(qs, ks, vs, state_in=state, state_out=state)
        outs.append(to_numpy(o))
    assert rel_err(np.concatenate(outs, axis=1), ref) <= 2e-2
    assert np.abs(to_numpy(state) - ref_state).max() <= 2e-3 * np.abs(ref_state).max()


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


@pytest.mark.parametrize("dtype,tol", [("bf16", 1e-4), ("f32", 1e-4)])
@pytest.mark.parametrize("B,H,d,T,norm", [(2, 3, 64, 40, True), (1, 2, 128, 25, True), (3, 1, 64, 10, False), (1, 1, 128, 5, False)])
def test_decode_steps_equal_the_sequence(dtype, tol, B, H, d, T, norm):
    """Token-by-token chela_linattn_step from a prefix state reproduces the oracle's outputs over the whole
    sequence (fp32 state and arithmetic on inputs exact in the storage dtype: the fp32 bound)."""
    import torch
    P = 70   # prefix evaluated by the chunked kernel, then T decode steps
    q, k, v = inputs.qkv(80 + d + T, B, P + T, H, d, d, dtype)
    ref, ref_state = oracle.linattn_recurrent(q, k, v, norm=norm, scale=0.5, return_state=True)
    nrm = chela.NORM_RMS if norm else chela.NORM_NONE
    qd, kd, vd = (to_device(x, dtype) for x in (q, k, v))
    _, state = chela.linattn_carry_fwd(qd[:, :P].contiguous(), kd[:, :P].contiguous(), vd[:, :P].contiguous(), norm=nrm, scale=0.5)
    if dtype == "bf16":   # the prefix state of the tensor kernel carries bf16-score rounding; take the oracle's
        state = torch.from_numpy(oracle.linattn_recurrent(q[:, :P], k[:, :P], v[:, :P], return_state=True)[1].astype(np.float32)).cuda()
    outs = []
    for t in range(P, P + T):
        outs.append(to_numpy(chela.linattn_step(qd[:, t].contiguous(), kd[:, t].contiguous(), vd[:, t].contiguous(), state,
                                                norm=nrm, scale=0.5)))
    got = np.stack(outs, axis=1)
    assert rel_err(got, ref[:, P:]) <= tol
    assert np.abs(to_numpy(state) - ref_state).max() <= 1e-5 * np.abs(ref_state).max()


def test_decode_step_argument_checks():
    import torch
    q = torch.zeros(1, 1, 32, device="cuda")
    s = torch.zeros(1, 1, 32, 32, device="cuda")
    with pytest.raises(chela.ChelaError) as e:
        chela.linattn_step(q, q, q, s)
    assert e.value.status == chela.ERR_UNSUPPORTED
