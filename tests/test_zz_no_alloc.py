"""chela_linattn_fwd_static_ws: the entry point for hosts that cannot allocate device memory (no
workspace argument; scratch comes from an array built into the library).  Collected last on purpose.

It must give what chela_linattn_fwd gives (and what the oracle gives), on consecutive calls that reuse the
built-in scratch with different shapes: calls whose sequences are shared between several CTAs or split along L
(d = 128: the scratch then carries per-group state sums) followed by calls that are not, and back."""
import numpy as np
import pytest

import oracle
from paper_2406_08128_b200 import chela, inputs
from util import rel_err, to_device, to_numpy

pytestmark = pytest.mark.gpu

TOL = 2e-2   # the bf16 bound the other linear-attention tests use


def both(seed, B, L, H, norm, d=64):
    """(built-in scratch result, workspace entry point's result, oracle's result)"""
    import torch
    host = inputs.qkv(seed, B, L, H, d, d, "bf16")
    q, k, v = (to_device(a, "bf16") for a in host)
    ref = chela.linattn_fwd(q, k, v, chunk=64, norm=norm)
    out = torch.empty_like(ref)
    # the set-up call: the first one on a device looks the built-in array up (the runtime places it then)
    chela.linattn_fwd_static_ws(q, k, v, chunk=64, norm=norm, out=out)
    torch.cuda.synchronize()
    out.zero_()
    free0 = torch.cuda.mem_get_info()[0]
    got = chela.linattn_fwd_static_ws(q, k, v, chunk=64, norm=norm, out=out)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free0          # the call took no device memory
    assert chela.linattn_static_ws_status() == chela.OK    # and no bounded wait gave up
    return to_numpy(got), to_numpy(ref), oracle.linattn_recurrent(*host, norm=norm == chela.NORM_RMS)


def test_two_calls_in_a_row_match_the_workspace_entry_point():
    # call 1: B*H = 2, d = 128 -> split into groups (the built-in scratch holds their state sums)
    assert chela.linattn_workspace_bytes(1, 2, 8192, 128, 128, 64) > 512
    got, ref, orc = both(71, 1, 8192, 2, chela.NORM_RMS, d=128)
    assert np.isfinite(got).all() and rel_err(got, ref) <= TOL and rel_err(got, orc) <= TOL
    # call 2, straight after, different shape, one CTA per sequence: stale scratch contents must not matter
    got, ref, orc = both(72, 4, 700, 96, chela.NORM_NONE)
    assert np.isfinite(got).all() and rel_err(got, ref) <= TOL and rel_err(got, orc) <= TOL
    # call 3: few sequences again, shared between CTAs by stride
    got, ref, orc = both(73, 1, 5000, 3, chela.NORM_RMS)
    assert np.isfinite(got).all() and rel_err(got, ref) <= TOL and rel_err(got, orc) <= TOL
    # call 4: d = 128 split again with another group count
    got, ref, orc = both(75, 1, 4000, 3, chela.NORM_RMS, d=128)
    assert np.isfinite(got).all() and rel_err(got, ref) <= TOL and rel_err(got, orc) <= TOL


def test_calls_beyond_the_built_in_scratch_are_refused_before_anything_is_launched():
    """d = 128, one sequence of 160 000 tokens: one 64 KiB state sum per group and a group per SM exceed 8 MiB."""
    import torch
    B, H, L, d = 1, 1, 160_000, 128
    assert chela.linattn_workspace_bytes(B, H, L, d, d, 64) > 8 << 20
    tiny = torch.zeros(16, dtype=torch.bfloat16, device="cuda")   # never read: the refusal comes first
    st = chela.lib().chela_linattn_fwd_static_ws(tiny.data_ptr(), tiny.data_ptr(), tiny.data_ptr(), tiny.data_ptr(), B, H, L, d, d, 64,
                                                 int(chela.BF16), int(chela.F32), int(chela.NORM_RMS), 1e-6, 1.0, None)
    assert st == chela.ERR_WORKSPACE


def test_fp32_inputs_and_argument_errors():
    import torch
    q, k, v = (to_device(a, "f32") for a in inputs.qkv(74, 1, 300, 2, 64, 64, "f32"))
    ref = chela.linattn_fwd(q, k, v)
    got = chela.linattn_fwd_static_ws(q, k, v)
    torch.cuda.synchronize()
    assert rel_err(to_numpy(got), to_numpy(ref)) <= 1e-4
    L = chela.lib()
    assert L.chela_linattn_fwd_static_ws(None, None, None, None, 1, 1, 64, 64, 64, 64, 1, 0, 1, 1e-6, 1.0, None) \
        == chela.ERR_INVALID_ARG
    bad = torch.zeros(1, 64, 1, 32, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(chela.ChelaError) as e:
        chela.linattn_fwd_static_ws(bad, bad, bad)
    assert e.value.status == chela.ERR_UNSUPPORTED
