"""The C-ABI library loads without a GPU and exports every symbol the public header declares."""
import ctypes
import os
import re

import pytest

from paper_2605_10380_b200 import agx

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    names = []
    for fn in sorted(os.listdir(os.path.join(ROOT, "include"))):
        if not fn.endswith(".h"):
            continue
        text = open(os.path.join(ROOT, "include", fn)).read()
        text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
        names += re.findall(r"AGX_API\s+[\w\s\*]+?\b(agx_\w+)\s*\(", text)
    return names


def test_header_declares_the_three_named_calls():
    names = declared_symbols()
    for must in ("agx_kv_append", "agx_attn_prefixed", "agx_accept_greedy"):
        assert must in names
    assert len(names) == len(set(names))


def test_library_exports_every_declared_symbol():
    lib = agx.load()
    names = declared_symbols()
    assert names
    for n in names:
        assert hasattr(lib, n), f"libagx.so does not export {n}"
    assert sorted(names) == sorted(agx.EXPORTS)


def test_status_strings_without_gpu():
    assert agx.status_string(0) == "ok"
    assert "invalid" in agx.status_string(-1)
    assert agx.status_string(-99) == "unknown status"


def test_binding_fails_loudly_when_library_missing(monkeypatch, tmp_path):
    monkeypatch.setattr(agx, "_lib", None)
    monkeypatch.setattr(agx, "_LIB_PATH", tmp_path / "libagx.so")
    with pytest.raises(RuntimeError, match="no CPU fallback"):
        agx.load()


def test_no_oracle_in_product_package():
    """The product package never imports the oracle (and the oracle never imports the package)."""
    pkg = os.path.join(ROOT, "paper_2605_10380_b200")
    for dirpath, _, files in os.walk(pkg):
        for fn in files:
            if fn.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, fn)).read()
                assert not re.search(r"^\s*(import|from)\s+oracle\b", text, flags=re.M), fn
                assert "agx_oracle" not in text, fn
    for fn in os.listdir(os.path.join(ROOT, "oracle")):
        if fn.endswith((".py", ".c")):
            text = open(os.path.join(ROOT, "oracle", fn)).read()
            assert "paper_2605_10380_b200" not in text and "libagx.so" not in text, fn
