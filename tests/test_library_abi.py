"""Host-side checks that need no GPU: the shared library loads, exports every function that
include/ulorl.h declares, and its pure host functions behave."""
import ctypes
import os
import re

import pytest

from paper_2507_19766_b200 import binding as B

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2507_19766_b200 import build
    build.build()
    return B.load_library()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "ulorl.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(ulorl_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = declared_functions()
    assert "ulorl_token_loss_fwd" in names and "ulorl_token_loss_bwd" in names
    for n in names:
        assert hasattr(lib, n), n
    assert set(B.EXPORTS) <= set(names)


def test_struct_sizes_match_header(lib):
    # 9 int32 + 5 float + (pad) int64 + 8 int32 + 1 float (+ pad)
    assert ctypes.sizeof(B.CParams) == 104
    assert ctypes.sizeof(B.CStats) == 4 * (2 + 6 + 3 * 16 + 4)


def test_workspace_bytes_is_a_pure_host_function(lib):
    p = B.Params(T=131072, H=2048, V=151936, num_seqs=1, dtype="bf16")
    n = B.workspace_bytes(p)
    # one 18944-token panel (74 CTA pairs x 256 tokens) of bf16 dz dominates
    assert 18944 * 151936 * 2 <= n <= 18944 * 151936 * 2 + (64 << 20)
    small = B.Params(T=512, H=256, V=4096, num_seqs=4, dtype="f32")
    assert 512 * 4096 * 4 <= B.workspace_bytes(small) <= 512 * 4096 * 4 + (4 << 20)
    with pytest.raises(B.UlorlError):
        B.workspace_bytes(B.Params(T=8, H=60, V=128, num_seqs=1))
    with pytest.raises(B.UlorlError):
        B.workspace_bytes(B.Params(T=8, H=64, V=128, num_seqs=1, inv_temperature=0.0))
    with pytest.raises(B.UlorlError):
        B.workspace_bytes(B.Params(T=8, H=64, V=128, num_seqs=1, dtype="f32", kernel_path="tensor"))


def test_status_strings(lib):
    assert B.status_string(0) == "ok"
    assert "workspace" in B.status_string(-3)
    assert "target" in B.status_string(-6)
    assert B.launch_count() >= 0


def test_null_arguments_are_rejected_without_a_device(lib):
    p = B.Params(T=8, H=64, V=128, num_seqs=1).to_c()
    args = [None] * 17
    code = lib.ulorl_token_loss_fwd(ctypes.byref(p), *args, None, 0, None)
    assert code == -1
    code = lib.ulorl_token_loss_bwd(ctypes.byref(p), *([None] * 8), None, 0, None)
    assert code == -1
    assert lib.ulorl_token_loss_fwd(None, *args, None, 0, None) == -1


def golden_thresholds():
    rows = []
    for line in open(os.path.join(ROOT, "tests", "golden", "decision_thresholds.txt")):
        if line.startswith("#") or not line.strip():
            continue
        kind, pbits, _, vbits, _ = line.split()
        rows.append((kind, int(pbits, 16), int(vbits, 16)))
    return rows


def test_decision_thresholds_of_the_library_match_the_correctly_rounded_logarithms(lib):
    """The bit-exact decision contract rests on these float32 constants; the golden values come from a
    60-digit decimal logarithm (tests/golden/make_decision_thresholds.py), not from libm."""
    import struct
    f = lambda b: struct.unpack("<f", struct.pack("<I", b))[0]
    bits = lambda x: struct.unpack("<I", struct.pack("<f", x))[0]
    seen = set()
    for kind, pbits, vbits in golden_thresholds():
        kw = dict(T=8, H=64, V=128, num_seqs=1)
        if kind == "ln_tau":
            got = B.decision_thresholds(B.Params(mpt_tau=f(pbits), **kw))[0]
        elif kind == "ln_1p_eps":
            got = B.decision_thresholds(B.Params(clip_eps_high=f(pbits), **kw))[1]
        else:
            got = B.decision_thresholds(B.Params(clip_eps_low=f(pbits), **kw))[2]
        assert bits(got) == vbits, (kind, hex(pbits), hex(bits(got)), hex(vbits))
        seen.add(kind)
    assert seen == {"ln_tau", "ln_1p_eps", "ln_1m_eps"}
    assert B.decision_thresholds(B.Params(clip_eps_low=1.0, T=8, H=64, V=128, num_seqs=1))[2] == float("-inf")
