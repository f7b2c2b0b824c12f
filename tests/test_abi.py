"""The C-ABI library loads without a GPU and exports every symbol gett.h declares."""
import ctypes
import os
import re

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    names = set()
    inc = os.path.join(ROOT, "include")
    for f in os.listdir(inc):
        if f.endswith(".h"):
            txt = open(os.path.join(inc, f)).read()
            names |= set(re.findall(r"GETT_API\s+[\w\s\*]+?\b(gett_\w+)\s*\(", txt))
    return names


def test_library_exports_every_declared_symbol():
    from paper_1607_00145_b200 import library_path
    lib = ctypes.CDLL(library_path())
    names = _declared()
    assert {"gett_plan_create", "gett_contract", "gett_plan_destroy", "gett_plan_get_info",
            "gett_plan_get_table", "gett_status_string"} <= names
    for n in names:
        assert hasattr(lib, n), n


def test_status_strings():
    import paper_1607_00145_b200 as g
    assert g.gett_status_string(0) == "ok"
    assert len({g.gett_status_string(i) for i in range(9)}) == 9
    assert g.gett_status_string(99) == "unknown status"


def test_optional_pair_library_is_self_contained():
    """The CTA-pair variant lives in a library of its own next to the main one: when its sources
    are in the tree it is built, loads without a GPU and exports its one entry point; without
    them the main library is complete by itself (checked by every other test)."""
    from paper_1607_00145_b200 import library_path
    src = os.path.join(ROOT, "paper_1607_00145_b200", "csrc", "kernel_umma_mc.cu")
    pair = library_path().replace(".so", "_mc.so")
    if not os.path.exists(src):
        assert not os.path.exists(pair)
        return
    assert os.path.exists(pair), "run python -m paper_1607_00145_b200.build"
    assert hasattr(ctypes.CDLL(pair), "gett_launch_umma_pair")
    # the files that name copies delivered to a whole cluster are listed for multi-GPU runs
    listed = open(os.path.join(ROOT, ".gpurunignore.multi")).read()
    for f in ("csrc/kernel_umma_mc.cu", "csrc/ptx_sm100_mc.cuh", "libgett_b200_mc.so"):
        assert f in listed


def test_package_and_build_module_import_without_the_library(tmp_path):
    """A fresh checkout has no shared library yet: importing the package and its build module
    must still work (the library is loaded at the first call), and a call without the library
    must fail loudly instead of falling back to anything."""
    import subprocess
    import sys
    code = ("import os, sys\n"
            f"sys.path.insert(0, {ROOT!r})\n"
            f"os.environ['GETT_LIBRARY'] = {str(tmp_path / 'absent.so')!r}\n"
            "import paper_1607_00145_b200 as g\n"
            "from paper_1607_00145_b200 import build\n"
            "assert callable(build.build)\n"
            "try:\n"
            "    g.gett_status_string(0)\n"
            "except ImportError as e:\n"
            "    print('loud:', 'no fallback' in str(e))\n")
    r = subprocess.run([sys.executable, "-c", code], capture_output=True, text=True)
    assert r.returncode == 0, r.stderr
    assert "loud: True" in r.stdout
