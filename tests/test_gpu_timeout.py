"""A bounded device-side wait that runs out: the kernel must return by itself, report CHELA_ERR_TIMEOUT with the
site of the wait, free its TMEM, and leave the context usable (the next ordinary call on the same workspace gives
the oracle's values).  The wait is made to run out on the host's request: chela_debug_wait_control sets a limit of
a few milliseconds and asks the first CTA to leave out one mbarrier arrival.  Nothing faults, traps or spins without
a bound."""
import numpy as np
import pytest

import oracle
from paper_2406_08128_b200 import chela, inputs
from util import rel_err, to_device, to_numpy

pytestmark = pytest.mark.gpu

LIMIT = 6_000_000   # SM cycles: about 3 ms


def header(ws):
    import torch
    torch.cuda.synchronize()
    return ws[:48].view(torch.int32).cpu().tolist()


@pytest.mark.parametrize("B,L,H,kind", [(1, 1024, 2, "one CTA per SM, sequences shared by stride"),
                                        (1, 640, 160, "two CTAs per SM, one sequence each")])
def test_linear_attention_wait_runs_out_and_the_next_call_is_clean(B, L, H, kind):
    import torch
    q, k, v = inputs.qkv(91, B, L, H, 64, 64, "bf16")
    dq, dk, dv = (to_device(a, "bf16") for a in (q, k, v))
    ws = torch.zeros(chela.linattn_workspace_bytes(B, H, L, 64, 64, 64) + 64, dtype=torch.uint8, device="cuda")
    out = torch.empty(B, L, H, 64, device="cuda")
    try:
        chela.debug_wait_control(LIMIT, 1)
        chela.linattn_fwd(dq, dk, dv, chunk=64, out=out, workspace=ws)
        assert chela.async_status(ws) == chela.ERR_TIMEOUT
    finally:
        chela.debug_wait_control(0, 0)
    words = header(ws)
    assert words[0] == chela.ERR_TIMEOUT
    assert words[8] > 0 and words[9] == 0, words        # a site code, recorded by CTA 0 (the one asked to skip)
    assert words[11] >= B * H, words                    # its grid size
    # the same workspace, hook off: TMEM was freed, nothing is left in flight, the result is the oracle's
    ws[32:48] = 0
    got = chela.linattn_fwd(dq, dk, dv, chunk=64, out=out, workspace=ws)
    assert chela.async_status(ws) == chela.OK
    assert rel_err(to_numpy(got), oracle.linattn_recurrent(q, k, v)) <= 2e-2


def test_projection_wait_runs_out_and_the_next_call_is_clean():
    import torch
    # 300 tiles of 128 x 128 on at most 148 CTAs: CTA 0 comes back to the accumulator buffer whose hand-back was skipped
    M, K, N = 128 * 300, 64, 128
    rng = np.random.default_rng(5)
    a = inputs.round_bf16(rng.standard_normal((M, K)).astype(np.float32))
    w = inputs.round_bf16((rng.standard_normal((K, N)) / 8).astype(np.float32))
    da, dw = to_device(a, "bf16"), to_device(w, "bf16")
    ws = torch.zeros(max(int(chela.lib().chela_dense_workspace_bytes()), 64), dtype=torch.uint8, device="cuda")
    y = torch.empty(M, N, dtype=torch.bfloat16, device="cuda")
    try:
        chela.debug_wait_control(LIMIT, 1)
        chela.dense_fwd(da, dw, y_dtype=chela.BF16, out=y, workspace=ws)
        assert chela.async_status(ws) == chela.ERR_TIMEOUT
    finally:
        chela.debug_wait_control(0, 0)
    got = chela.dense_fwd(da, dw, y_dtype=chela.BF16, out=y, workspace=ws)
    assert chela.async_status(ws) == chela.OK
    ref = oracle.dense(a, w)
    assert rel_err(to_numpy(got), ref) <= 2e-2


def test_sm_clock_probe_reports_a_plausible_clock():
    """chela_debug_sm_clock: SM cycles over global-timer nanoseconds, a few hundred microseconds of spinning."""
    mhz = chela.debug_sm_clock_mhz()
    assert 300.0 < mhz < 3000.0, mhz
