"""chela_linattn_fwd_static_ws: the entry point for hosts that cannot allocate device memory (no
workspace argument; scratch comes from an array built into the library).  Collected last on purpose.

It must give what chela_linattn_fwd gives, on consecutive calls that reuse the built-in scratch with
different shapes: one call whose sequences are split along L (the scratch then carries per-group state
sums) followed by one that is not split, and back."""
import numpy as np
import pytest

from paper_2406_08128_b200 import chela, inputs
from util import rel_err, to_device, to_numpy

pytestmark = pytest.mark.gpu

TOL = 2e-2   # the bf16 bound the other linear-attention tests use


def both(seed, B, L, H, norm):
    import torch
    q, k, v = (to_device(a, "bf16") for a in inputs.qkv(seed, B, L, H, 64, 64, "bf16"))
    ref = chela.linattn_fwd(q, k, v, chunk=64, norm=norm)
    out = torch.empty_like(ref)
    got = chela.linattn_fwd_static_ws(q, k, v, chunk=64, norm=norm, out=out)
    torch.cuda.synchronize()
    return to_numpy(got), to_numpy(ref)


def test_two_calls_in_a_row_match_the_workspace_entry_point():
    # call 1: B*H = 2 -> split into groups (the built-in scratch holds their state sums)
    assert chela.linattn_workspace_bytes(1, 2, 8192, 64, 64, 64) > 512
    got, ref = both(71, 1, 8192, 2, chela.NORM_RMS)
    assert np.isfinite(got).all() and rel_err(got, ref) <= TOL
    # call 2, straight after, different shape, not split: stale scratch contents must not matter
    got, ref = both(72, 4, 700, 96, chela.NORM_NONE)
    assert np.isfinite(got).all() and rel_err(got, ref) <= TOL
    # call 3: split again with another group count
    got, ref = both(73, 1, 5000, 3, chela.NORM_RMS)
    assert np.isfinite(got).all() and rel_err(got, ref) <= TOL


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
