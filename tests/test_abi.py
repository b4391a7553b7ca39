"""Host-side checks of the C-ABI library that need no GPU: it loads, exports every symbol the
header declares, sizes workspaces sensibly and names its status codes."""
import ctypes
import os
import re

import pytest

from paper_1905_03381_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return binding.lib()


def test_every_declared_symbol_is_exported(lib):
    header = open(os.path.join(ROOT, "include", "autoassist.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(aa_[a-z_]+)\s*\(", header))
    assert declared, "no prototypes found in the header"
    for name in sorted(declared):
        assert hasattr(lib, name), f"{name} is declared in include/autoassist.h but not exported"
    for name in binding.EXPORTS:
        assert name in declared, f"binding lists {name}, which the header does not declare"


def test_status_strings(lib):
    seen = set()
    for code in range(8):
        s = binding.status_string(code)
        assert s and s != "unknown status"
        seen.add(s)
    assert len(seen) == 8
    assert binding.status_string(99) == "unknown status"


def test_workspace_bytes_grows_with_limits_and_rejects_bad_arguments(lib):
    def ws(rows, d, hidden=0):
        n = ctypes.c_size_t(0)
        st = lib.aa_workspace_bytes(rows, d, hidden, ctypes.byref(n))
        return st, n.value

    st, small = ws(4096, 64)
    assert st == binding.AA_OK and small >= 256 + 8 * 129 + 4 * 4096
    st, big = ws(1 << 24, 512)
    assert st == binding.AA_OK and big > small
    assert big < (1 << 30)               # modest even for the largest sweep pool
    st, wide = ws(16384, 1 << 18)
    assert st == binding.AA_OK and wide < (1 << 27) + (1 << 22)   # partials are capped at 64 MiB
    assert ws(-1, 64)[0] == binding.AA_ERR_INVALID_ARG
    assert ws(10, 0)[0] == binding.AA_ERR_INVALID_ARG
    assert lib.aa_workspace_bytes(10, 10, 0, None) == binding.AA_ERR_INVALID_ARG


def test_null_context_is_rejected_without_touching_the_device(lib):
    assert lib.aa_destroy(None) == binding.AA_ERR_INVALID_ARG
    assert lib.aa_launch_count(None) == -1
    assert lib.aa_device_status(None, None) == binding.AA_ERR_INVALID_ARG
    assert lib.aa_create(None, 1, 1, 0, None, 0, None) == binding.AA_ERR_INVALID_ARG


def test_struct_layouts_match_the_header():
    # field offsets as a C compiler lays out include/autoassist.h (LP64)
    assert ctypes.sizeof(binding.aa_feat) == 96
    assert binding.aa_feat.nnz.offset == 64 and binding.aa_feat.id_base.offset == 88
    assert ctypes.sizeof(binding.aa_assistant) == 80
    assert ctypes.sizeof(binding.aa_logits) == 40


def test_header_compiles_as_plain_c(tmp_path):
    import subprocess

    src = tmp_path / "t.c"
    src.write_text('#include "autoassist.h"\n'
                   "_Static_assert(sizeof(aa_feat) == 96, \"aa_feat\");\n"
                   "_Static_assert(sizeof(aa_assistant) == 80, \"aa_assistant\");\n"
                   "_Static_assert(sizeof(aa_logits) == 40, \"aa_logits\");\n"
                   "int main(void) { return 0; }\n")
    subprocess.check_call(["gcc", "-std=c11", "-Wall", "-Werror", "-I", os.path.join(ROOT, "include"),
                           "-c", str(src), "-o", str(tmp_path / "t.o")])
