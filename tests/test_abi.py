"""The shared library builds, loads, and exports every symbol the header declares (no GPU needed)."""
import ctypes
import os
import re

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "remoe.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(remoe_[a-z_0-9]+)\s*\(", text)))


def test_library_exports_header_symbols():
    from paper_2605_27081_b200 import build, binding
    path = build.build_library()
    lib = ctypes.CDLL(path)
    names = _declared()
    assert "remoe_decode_step" in names and "remoe_stack_create" in names and len(names) >= 15
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(binding.EXPORTS) == names
    assert binding.strerror(0) == "ok" and "page-locked" in binding.strerror(binding.REMOE_E_NOT_PINNED)


def test_struct_layouts_match_header():
    from paper_2605_27081_b200 import binding
    assert ctypes.sizeof(binding.remoe_shape) == 11 * 4
    assert ctypes.sizeof(binding.remoe_cache_counters) == 6 * 8
    text = open(os.path.join(ROOT, "include", "remoe.h")).read()
    body = re.search(r"typedef struct \{(.*?)\} remoe_shape;", text, flags=re.S).group(1)
    fields = re.findall(r"int32_t\s+([a-z_]+);", body)
    assert fields == [n for n, _ in binding.remoe_shape._fields_]


def test_header_is_plain_c(tmp_path):
    """The boundary is a C ABI: the header must compile as C99 on its own, without warnings."""
    import shutil
    import subprocess
    cc = shutil.which("gcc") or shutil.which("cc")
    if cc is None:
        import pytest
        pytest.skip("no C compiler")
    src = tmp_path / "use_header.c"
    src.write_text('#include "remoe.h"\nint main(void) { remoe_shape s; remoe_cache_counters c; (void)s; (void)c; return REMOE_OK; }\n')
    res = subprocess.run([cc, "-std=c99", "-Wall", "-Wextra", "-pedantic", "-Werror", "-fsyntax-only",
                          "-I", os.path.join(ROOT, "include"), str(src)], capture_output=True, text=True)
    assert res.returncode == 0, res.stderr
