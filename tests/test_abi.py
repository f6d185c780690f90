"""CPU-side checks of the C ABI: the library loads, exports every function the header
declares, and rejects bad arguments on the host (no kernel is launched here)."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2605_16579_b200 import arl2

    return arl2.load(build_if_missing=True)


def declared_functions():
    text = open(os.path.join(ROOT, "include", "arl2.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(arl2_[a-z0-9_]+)\s*\(", text)))


def test_header_functions_are_exported(lib):
    from paper_2605_16579_b200 import arl2

    names = declared_functions()
    assert "arl2_create" in names and "arl2_denoise_step" in names and "arl2_commit" in names
    assert "arl2_reset" in names
    for n in names:
        assert hasattr(lib, n), f"{n} is declared in include/arl2.h but not exported"
    assert sorted(arl2.EXPORTS) == names


def test_config_struct_matches_header():
    from paper_2605_16579_b200 import arl2

    assert ctypes.sizeof(arl2.arl2_config) == 40


def test_workspace_bytes_and_argument_errors(lib):
    from paper_2605_16579_b200 import arl2

    cfg = arl2.make_config(1, 12, 4680, 128, "bf16")
    n = arl2.arl2_workspace_bytes(cfg)
    tensor = 4680 * 12 * 128 * 2
    assert n >= tensor and n % 256 == 0
    for bad in (dict(D=96), dict(L=0), dict(B=0), dict(H=0)):
        kw = dict(B=1, H=2, L=16, D=64)
        kw.update(bad)
        c = arl2.make_config(kw["B"], kw["H"], kw["L"], kw["D"], "fp32")
        assert lib.arl2_workspace_bytes(ctypes.byref(c)) == 0
        assert lib.arl2_last_error() != b""
    c = arl2.make_config(1, 2, 16, 64, "fp32")
    c.struct_size = 12
    assert lib.arl2_workspace_bytes(ctypes.byref(c)) == 0
    c = arl2.make_config(1, 2, 16, 64, "fp32", commit_rule=1)
    assert lib.arl2_workspace_bytes(ctypes.byref(c)) == 0
    # create: NULL buffers are rejected on the host before any CUDA call
    c = arl2.make_config(1, 2, 16, 64, "fp32")
    ctx = ctypes.c_void_p()
    assert lib.arl2_create(ctypes.byref(c), None, None, 0, None, ctypes.byref(ctx)) == -1
    assert ctx.value is None
    # NULL context
    assert lib.arl2_reset(None, -1, None) == -1
    assert lib.arl2_commit(None, None, None, None, None) == -1
    assert lib.arl2_commit_delta(None, None, None, None, None, None) == -1
    assert lib.arl2_commit_tokens(None, None, None, None, None, None) == -1
    # the token-gate scratch is reserved only on request: three [B, H, ceil(L/128)*128, D] fp32 tensors
    c0 = arl2.make_config(1, 12, 4680, 128, "bf16")
    c1 = arl2.make_config(1, 12, 4680, 128, "bf16", flags=arl2.ARL2_FLAG_TOKEN_GATES)
    extra = arl2.arl2_workspace_bytes(c1) - arl2.arl2_workspace_bytes(c0)
    assert 3 * 12 * 4680 * 128 * 4 <= extra <= 3 * 12 * (4680 + 128) * 128 * 4 + (1 << 20)
    assert lib.arl2_launch_count(None) == 0
    assert lib.arl2_version().startswith(b"arl2")


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    from paper_2605_16579_b200 import arl2

    monkeypatch.setattr(arl2, "_lib", None)
    monkeypatch.setattr(arl2, "LIB_PATH", str(tmp_path / "nope.so"))
    with pytest.raises(arl2.Arl2Error):
        arl2.load()


def test_product_path_does_not_import_the_oracle():
    pkg = os.path.join(ROOT, "paper_2605_16579_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".h", ".cuh")):
                text = open(os.path.join(dirpath, f)).read()
                assert not re.search(r"(import|from)\s+\S*oracle|arl2_oracle|oracle/", text), \
                    f"{f} reaches for the oracle"
