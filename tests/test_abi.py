"""The C-ABI library loads without a GPU and exports every symbol the header declares."""
import os
import re

from paper_2111_09389_b200 import _lib

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "lpdt.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(lpdt_[a-z0-9_]+)\s*\(", text)))


def test_header_symbols_are_exported_and_bound():
    lib = _lib.lib()
    names = declared_symbols()
    assert len(names) >= 20
    for n in names:
        assert hasattr(lib, n), n
        assert n in _lib.SIGNATURES, f"{n} has no ctypes signature"
    assert set(_lib.SIGNATURES) == set(names)


def test_version_and_status_strings():
    lib = _lib.lib()
    assert b"sm_100a" in lib.lpdt_version()
    assert lib.lpdt_status_string(0) == b"ok"
    assert lib.lpdt_status_string(3) == b"workspace missing or too small"


def test_binding_names_match_the_abi():
    from paper_2111_09389_b200 import api
    for n in declared_symbols():
        if n == "lpdt_status_string":
            continue
        assert hasattr(api, n), n
