"""The C-ABI library loads without a GPU and exports every function include/*.h declares;
the Python binding lists the same names.  No compute call is made here."""
import ctypes
import os
import re

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    names = set()
    inc = os.path.join(ROOT, "include")
    for f in sorted(os.listdir(inc)):
        if f.endswith(".h"):
            text = re.sub(r"/\*.*?\*/", "", open(os.path.join(inc, f)).read(), flags=re.S)
            names |= set(re.findall(r"\b(syn_[a-z0-9_]+)\s*\(", text))
    return sorted(names)


def test_header_declares_the_three_calls_of_the_problem_statement():
    names = _declared()
    for must in ("syn_model_load", "syn_kv_alloc", "syn_verify_batch"):
        assert must in names


def test_library_exports_every_declared_symbol():
    from paper_2511_07423_b200 import build
    lib = ctypes.CDLL(build.build())
    for name in _declared():
        assert hasattr(lib, name), name


def test_headers_are_plain_c(tmp_path):
    """The boundary is a C ABI: both headers compile as C99 (no C++ in the signatures), and a C program that
    uses their types and constants links against the library."""
    import shutil
    import subprocess
    from paper_2511_07423_b200 import build
    gcc = shutil.which("gcc")
    if gcc is None:
        import pytest
        pytest.skip("no C compiler")
    src = tmp_path / "use_abi.c"
    src.write_text(
        '#include "synera.h"\n#include "synera_sched.h"\n#include <string.h>\n'
        "int main(void) {\n"
        "    syn_sampling s = {1, 1.0f, 1.0f, 1};\n"
        "    syn_sched *sc = 0;\n"
        "    int32_t prompt[3] = {1, 2, 3};\n"
        "    syn_sched_batch b;\n"
        "    (void)s;\n"
        "    if (strcmp(syn_strerror(SYN_E_CHUNK_LEN), \"unknown error\") == 0) return 1;\n"
        "    if (syn_sched_create(0, 0, 8, 16, SYN_MAX_CHUNK, &sc) != SYN_OK) return 2;\n"
        "    if (syn_sched_add_request(sc, 7, prompt, 3) != SYN_OK) return 3;\n"
        "    if (syn_sched_peek(sc, &b) != SYN_OK || b.kind != SYN_SCHED_PREFILL || b.n_tokens != 3) return 4;\n"
        "    syn_sched_free(sc);\n"
        "    return 0;\n}\n")
    lib = build.build()
    exe = tmp_path / "use_abi"
    inc = os.path.join(ROOT, "include")
    subprocess.check_call([gcc, "-std=c99", "-Wall", "-Wextra", "-pedantic", "-Werror", "-I", inc, str(src), "-o", str(exe),
                           lib, "-Wl,-rpath," + os.path.dirname(lib)])
    assert subprocess.call([str(exe)]) == 0


def test_binding_lists_the_header_names():
    from paper_2511_07423_b200 import binding
    assert sorted(binding.EXPORTS + binding.SCHED_EXPORTS) == _declared()


def test_strerror_names_every_code_without_a_device():
    from paper_2511_07423_b200 import binding
    lib = binding.load_library()
    seen = set()
    for code in range(0, -12, -1):
        s = lib.syn_strerror(code).decode()
        assert s and s != "unknown error"
        seen.add(s)
    assert len(seen) == 12
    for code in range(-20, -24, -1):   # the scheduler's codes
        assert lib.syn_strerror(code).decode().startswith("scheduler:")
    assert lib.syn_strerror(-99).decode() == "unknown error"


def test_product_package_never_imports_the_oracle():
    pkg = os.path.join(ROOT, "paper_2511_07423_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                src = open(os.path.join(dirpath, f)).read()
                assert not re.search(r"^\s*(from|import)\s+oracle|liboracle|synera_oracle", src, flags=re.M), f
