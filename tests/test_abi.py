"""The C-ABI library loads without a GPU and exports every function include/cvlc.h declares."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "cvlc.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(cvlc_[a-z0-9_]+)\s*\(", text)))


def test_header_functions_are_exported():
    from paper_2402_03770_b200 import binding as B
    lib = B.lib()
    names = declared_functions()
    assert "cvlc_plan" in names and "cvlc_encode" in names and "cvlc_decode_aggregate" in names
    for name in names:
        assert hasattr(lib, name), name
    assert sorted(B.EXPORTS) == names


def test_host_only_helpers_without_gpu():
    from paper_2402_03770_b200 import binding as B
    import oracle as O
    p = B.make_params(11_200_000, 22_400_000)
    po = O.make_params(11_200_000, 22_400_000)
    assert B.cvlc_stream_bytes(p) == 64 + 1866 * 1500 == O.stream_bytes(po)
    assert p.scale_B == po.scale_B
    assert B.cvlc_plan_workspace_bytes(p) >= 256 + 4096 * 8 + 256
    assert B.cvlc_encode_workspace_bytes(p) >= 16 * p.d
    assert B.cvlc_encode_batch_workspace_bytes(p, 100, 1 << 20) < 100 * B.cvlc_encode_workspace_bytes(p)
    assert B.cvlc_decode_workspace_bytes(100) > 0 and B.cvlc_decode_workspace_bytes(5000) == 0
    assert B.status_string(B.CVLC_ERR_BAD_STREAM) == "malformed stream"
    assert C_sizeof_plan() == 512


def C_sizeof_plan():
    from paper_2402_03770_b200 import binding as B
    return ctypes.sizeof(B.CvlcPlan)


def test_binding_raises_when_library_is_missing(monkeypatch, tmp_path):
    from paper_2402_03770_b200 import binding as B
    monkeypatch.setattr(B, "_lib", None)
    monkeypatch.setattr(B, "LIB_PATH", str(tmp_path / "nope.so"))
    with pytest.raises(RuntimeError):
        B.lib()


def test_header_is_plain_c(tmp_path):
    """include/cvlc.h is a C header: it compiles as C11 with no CUDA or C++ in sight, and the two structs that cross
    the boundary have the sizes the binding assumes"""
    import subprocess
    src = tmp_path / "t.c"
    src.write_text('#include "cvlc.h"\n'
                   '_Static_assert(sizeof(cvlc_plan_t) == 512, "plan");\n'
                   '_Static_assert(sizeof(cvlc_literal_plan_t) == 64, "literal plan");\n'
                   '_Static_assert(sizeof(cvlc_params) == 56, "params");\n'
                   'int main(void) { return CVLC_OK; }\n')
    r = subprocess.run(["gcc", "-std=c11", "-Wall", "-Wextra", "-Werror", "-fsyntax-only", "-I", os.path.join(ROOT, "include"), str(src)],
                       capture_output=True, text=True)
    assert r.returncode == 0, r.stderr
    from paper_2402_03770_b200 import binding as B
    assert ctypes.sizeof(B.CvlcParams) == 56 and ctypes.sizeof(B.CvlcLiteralPlan) == 64
