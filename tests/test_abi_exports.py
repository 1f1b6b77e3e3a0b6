"""The library loads and exports every function include/dl.h declares (no GPU needed)."""
import ctypes
import os
import re

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "dl.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(dl_[a-z0-9_]+)\s*\(", text)))


def test_header_and_binding_agree_and_symbols_exist():
    from paper_2412_00876_b200 import build, binding
    path = build.build()
    lib = ctypes.CDLL(path)
    names = declared_functions()
    assert len(names) >= 18
    for n in names:
        assert hasattr(lib, n), f"{n} declared in dl.h but not exported"
    assert sorted(binding.EXPORTS) == names
    # a host-only call works without a device
    assert b"cache" in binding.lib().dl_status_str(binding.DL_ERR_CAPACITY)


def test_checked_twin_exports_the_same_and_says_so():
    """libdl_sparse_checked.so (-DDL_BOUNDS=1) has the same interface; the two tell themselves apart."""
    from paper_2412_00876_b200 import build
    normal, checked = ctypes.CDLL(build.build()), ctypes.CDLL(build.build(checked=True))
    for n in declared_functions():
        assert hasattr(checked, n), f"{n} missing from the checked build"
    assert normal.dl_build_is_checked() == 0 and checked.dl_build_is_checked() == 1


def test_product_code_never_imports_the_oracle():
    pkg = os.path.join(ROOT, "paper_2412_00876_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith(".py"):
                src = open(os.path.join(dirpath, f)).read()
                assert not re.search(r"^\s*(import|from)\s+oracle", src, flags=re.M), f
