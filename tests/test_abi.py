"""The C-ABI library loads, exports every symbol the header declares, and rejects
bad arguments before touching the GPU (no compute calls here)."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2604_05250_b200 import build, binding
    build.build()
    return binding.lib()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "dualdiff.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(dd_[a-z_0-9]+)\s*\(", text)))


def test_exports_match_header(lib):
    from paper_2604_05250_b200 import binding
    names = declared_symbols()
    assert names == sorted(binding.EXPORTS)
    for n in names:
        assert getattr(lib, n) is not None


def test_version_and_strings(lib):
    assert lib.dd_version() >= 100
    assert lib.dd_status_string(0) == b"ok"
    assert b"invalid" in lib.dd_status_string(-1)
    assert lib.dd_launch_count() >= 0


def test_workspace_bytes(lib):
    assert lib.dd_verify_workspace_bytes(0, 1, 1) == 0
    small = lib.dd_verify_workspace_bytes(1, 256, 126464)
    big = lib.dd_verify_workspace_bytes(16, 256, 126464)
    assert 0 < small < big < (64 << 20)


def test_bad_arguments_rejected_without_a_gpu(lib):
    p = ctypes.c_void_p(16)        # never dereferenced: validation comes first
    null = ctypes.c_void_p(0)
    # attention
    assert lib.dd_bidir_attention(null, p, p, p, 1, 1, 128, 128, 0.1, null) == -1
    assert lib.dd_bidir_attention(p, p, p, p, 0, 1, 128, 128, 0.1, null) == -1
    assert lib.dd_bidir_attention(p, p, p, p, 1, 1, 128, 128, float("nan"), null) == -1
    assert lib.dd_bidir_attention(p, p, p, p, 1, 1, 128, 96, 0.1, null) == -2
    assert lib.dd_bidir_attention(p, p, p, ctypes.c_void_p(24), 1, 1, 128, 128, 0.1, null) == -2
    assert lib.dd_bidir_attention(p, p, p, p, 1, 1, 128, 128, -1.0, null) == -2
    # verify
    ok = dict(mode=1, tau=0.5, k=1, seed=0, B=1, P=4, V=64)

    def call(dra=p, ver=p, tok=p, fl=p, otok=p, omask=p, **kw):
        a = dict(ok, **kw)
        return lib.dd_verify(dra, ver, tok, fl, a["mode"], a["tau"], a["k"], a["seed"],
                             otok, omask, null, a["B"], a["P"], a["V"], null)
    assert call(ver=null) == -1
    assert call(dra=null) == -1                  # KL mode needs the drafter
    assert call(tok=null) == -1 and call(fl=null) == -1 and call(otok=null) == -1 and call(omask=null) == -1
    assert call(k=-1) == -1 and call(B=0) == -1 and call(P=0) == -1 and call(V=0) == -1
    assert call(mode=3) == -1 and call(mode=1 | 0x400) == -1
    assert call(tau=float("nan")) == -1
    assert call(P=8193) == -2


def test_binding_fails_loudly_without_library(monkeypatch, tmp_path):
    from paper_2604_05250_b200 import binding
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", str(tmp_path / "missing.so"))
    with pytest.raises(RuntimeError, match="no fallback"):
        binding.lib()
