"""CPU-side checks of the C ABI: the library loads, exports every declared symbol, and rejects
bad arguments before touching a GPU."""
import ctypes
import os
import re

import pytest

from paper_2406_08128_b200 import build, chela

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return chela.lib()


def header_symbols():
    text = open(os.path.join(ROOT, "include", "chela.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(chela_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = header_symbols()
    assert names == chela.exported_symbols()
    raw = ctypes.CDLL(chela.LIB_PATH)
    for n in names:
        assert getattr(raw, n) is not None


def test_status_strings_and_version(lib):
    assert chela.version() >= 100
    assert chela.status_string(chela.OK) == "ok"
    seen = {chela.status_string(s) for s in range(6)}
    assert len(seen) == 6


def test_kernel_kind_and_workspace_queries(lib):
    assert chela.linattn_kernel_kind(1, 1, 1024, 64, 64, 64, chela.F32, chela.F32) == 1
    assert chela.linattn_kernel_kind(1, 1, 1024, 32, 32, 64) == 0
    assert chela.linattn_kernel_kind(1, 1, 1024, 64, 128, 64) == 0
    assert chela.linattn_kernel_kind(1, 1, 1024, 64, 64, 48) == 0
    assert chela.linattn_workspace_bytes(1, 1, 1024, 32, 32, 64) == 0
    assert chela.longconv_workspace_bytes(2, 100, 16) > 2 * 100 * 16 * 4
    assert chela.mixer_workspace_bytes(1, 128, 128, 2, 64) > chela.longconv_workspace_bytes(1, 128, 128)


def test_invalid_arguments_rejected_without_gpu(lib):
    L = chela.lib()
    null = None
    one = ctypes.c_void_p(256)  # never dereferenced: validation fails first
    # null pointers
    assert L.chela_linattn_fwd(null, one, one, one, 1, 1, 64, 64, 64, 64, 1, 0, 1, 1e-6, 1.0, null, 0, null) \
        == chela.ERR_INVALID_ARG
    # misaligned pointer
    assert L.chela_linattn_fwd(ctypes.c_void_p(260), one, one, one, 1, 1, 64, 64, 64, 64, 1, 0, 1, 1e-6, 1.0,
                               null, 0, null) == chela.ERR_INVALID_ARG
    # unsupported head dim / chunk
    assert L.chela_linattn_fwd(one, one, one, one, 1, 1, 64, 32, 32, 64, 1, 0, 1, 1e-6, 1.0, null, 0, null) \
        == chela.ERR_UNSUPPORTED
    assert L.chela_linattn_fwd(one, one, one, one, 1, 1, 64, 64, 64, 32, 1, 0, 1, 1e-6, 1.0, null, 0, null) \
        == chela.ERR_UNSUPPORTED
    # bad sizes / dtype / norm
    assert L.chela_linattn_fwd(one, one, one, one, 0, 1, 64, 64, 64, 64, 1, 0, 1, 1e-6, 1.0, null, 0, null) \
        == chela.ERR_INVALID_ARG
    assert L.chela_linattn_fwd(one, one, one, one, 1, 1, 64, 64, 64, 64, 7, 0, 1, 1e-6, 1.0, null, 0, null) \
        == chela.ERR_INVALID_ARG
    assert L.chela_linattn_fwd(one, one, one, one, 1, 1, 64, 64, 64, 64, 1, 0, 3, 1e-6, 1.0, null, 0, null) \
        == chela.ERR_INVALID_ARG
    # short conv
    assert L.chela_shortconv_fwd(one, one, null, one, 1, 8, 8, 3, 1, 1, null) == chela.ERR_INVALID_ARG  # x == y
    two = ctypes.c_void_p(512)
    assert L.chela_shortconv_fwd(one, one, null, two, 1, 8, 8, 17, 1, 1, null) == chela.ERR_UNSUPPORTED
    assert L.chela_shortconv_fwd(one, one, null, two, 1, 8, 12, 3, 1, 1, null) == chela.ERR_UNSUPPORTED
    # long conv: length limit and workspace
    assert L.chela_longconv_fwd(one, one, null, 0, two, 1, 262145, 8, 1, 0, two, 1 << 40, null) == chela.ERR_UNSUPPORTED
    assert L.chela_longconv_fwd(one, one, null, 0, two, 1, 64, 8, 1, 0, null, 0, null) == chela.ERR_WORKSPACE
    assert L.chela_longconv_fwd(one, one, null, 0, two, 1, 64, 8, 1, 0, two, 16, null) == chela.ERR_WORKSPACE
    # mixer: D not divisible by H, head dim unsupported, workspace too small
    args = [one, one, 3, one, one, one, one, null, null, null, 0, 1, two]
    tail = [1, 0, 1, 1e-6]
    assert L.chela_mixer_fwd(*args, 1, 64, 128, 3, 64, *tail, two, 1 << 40, null) == chela.ERR_INVALID_ARG
    assert L.chela_mixer_fwd(*args, 1, 64, 128, 4, 64, *tail, two, 1 << 40, null) == chela.ERR_UNSUPPORTED
    assert L.chela_mixer_fwd(*args, 1, 64, 128, 2, 64, *tail, two, 64, null) == chela.ERR_WORKSPACE


def test_missing_library_fails_loudly(monkeypatch):
    monkeypatch.setattr(chela, "_lib", None)
    monkeypatch.setattr(chela, "LIB_PATH", os.path.join(ROOT, "does_not_exist.so"))
    with pytest.raises(RuntimeError, match="no CPU fallback"):
        chela.lib()


def test_split_plan_covers_every_sequence_exactly(lib):
    """Host logic of how a sequence is shared between CTAs (no GPU: the SM count is passed in).  Grouped plans: the
    groups tile the sequence's chunks exactly, none is empty, all but the last are full.  Strided plans (plain bf16,
    d = 64; reported with zero chunk counts): every CTA owns at least four chunks and there is one CTA per SM at most.
    Both: no more CTAs than are resident at once, and one CTA per sequence once there are as many (batch, head)
    pairs as SMs."""
    sms = 148
    for d, pair in ((64, False), (64, True), (128, False)):
        dt = chela.BF16_PAIR if pair else chela.BF16
        for bh in (1, 2, 3, 7, 32, 64, 73, 74, 96, 128, 147, 148, 149, 256):
            for L in (1, 63, 64, 65, 1000, 1024, 2047, 2048, 2100, 4096, 5000, 8192, 16384, 32768, 65536, 65600, 131072):
                plan = chela.linattn_split_plan(1, bh, L, d=d, in_dtype=dt, sms=sms)
                assert plan is not None
                G, c0, c = plan
                nch = (L + 63) // 64
                if G > 1 and c0 == 0:   # strided: CTA g owns chunks g, g + G, ...
                    assert d == 64 and not pair and c == 0
                    assert 2 <= G <= 4 and nch // G >= 4 and bh * G <= sms, (d, pair, bh, L, plan)
                    continue
                assert G >= 1 and c0 >= 1 and c >= 1, (d, pair, bh, L, plan)
                if G == 1:
                    assert c0 >= nch
                else:
                    # groups 0 .. G-2 are full and leave at least one chunk for the last one, which fits in c
                    assert c0 + (G - 2) * c < nch <= c0 + (G - 1) * c, (d, pair, bh, L, plan)
                    assert min(c0, c) >= 7, (d, pair, bh, L, plan)          # groups stay long enough to amortise the state pass
                    per_sm = 1 if (pair or d == 128) else 2
                    assert bh * G <= per_sm * sms, (d, pair, bh, L, plan)   # every CTA of the call is resident
                if bh >= sms:
                    assert G == 1
    assert chela.linattn_split_plan(1, 1, 100, d=32) is None
