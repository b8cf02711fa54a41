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
