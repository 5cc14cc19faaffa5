"""The product path has no CPU fallback: without the shared library the binding cannot be
imported, and it never imports the oracle."""
import importlib
import os
import sys

import pytest


def test_binding_import_fails_loudly_without_the_library(monkeypatch, tmp_path):
    from paper_2101_06983_b200 import _build
    monkeypatch.setattr(_build, "LIB", str(tmp_path / "libgradcache.so"))
    sys.modules.pop("paper_2101_06983_b200.binding", None)
    with pytest.raises(ImportError, match="no fallback"):
        importlib.import_module("paper_2101_06983_b200.binding")
    sys.modules.pop("paper_2101_06983_b200.binding", None)


def test_package_never_touches_the_oracle():
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    pkg = os.path.join(root, "paper_2101_06983_b200")
    for dirpath, _, files in os.walk(pkg):
        for fn in files:
            if fn.endswith((".py", ".cu", ".h", ".cuh")):
                text = open(os.path.join(dirpath, fn)).read()
                assert "oracle" not in text, fn
