"""The C-ABI library loads without a GPU and exports every function include/hispec.h declares
(no compute calls here)."""
import ctypes
import os
import re

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    src = open(os.path.join(ROOT, "include", "hispec.h")).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    return sorted(set(re.findall(r"\b(hispec_[a-z_]+)\s*\(", src)))


def test_library_exports_every_declared_symbol():
    from paper_2510_01336_b200 import build, binding
    lib = ctypes.CDLL(build.build())
    names = _declared()
    assert {"hispec_draft", "hispec_verify_intermediate", "hispec_verify_target"} <= set(names)
    for n in names:
        assert hasattr(lib, n), n
    assert set(binding.EXPORTS) == set(names)


def test_host_side_argument_checks_need_no_gpu():
    from paper_2510_01336_b200 import binding
    lib = binding.load()
    assert lib.hispec_create(None, None, None) == -1            # HISPEC_EINVAL
    assert lib.hispec_destroy(None) == -1
    assert lib.hispec_strerror(-2).decode().startswith("request exceeds")
    assert lib.hispec_launch_count(None) == 0


def test_oracle_is_not_reachable_from_the_product():
    """The product package never imports the oracle (and the oracle never imports the product)."""
    pkg = os.path.join(ROOT, "paper_2510_01336_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                txt = open(os.path.join(dirpath, f)).read()
                assert "oracle" not in txt.lower() or f == "workload.py", f
    for f in os.listdir(os.path.join(ROOT, "oracle")):
        if f.endswith((".py", ".c")):
            assert "paper_2510_01336_b200" not in open(os.path.join(ROOT, "oracle", f)).read(), f
