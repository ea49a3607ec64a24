"""The C-ABI library loads and exports every symbol the public header declares.
No compute call is made, so this runs without a GPU."""
import os
import re

import pytest

import __graft_entry__ as entry
from paper_2211_17192_b200 import binding

HEADER_DIR = os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))), "include")


def declared_functions():
    names = []
    for fname in sorted(os.listdir(HEADER_DIR)):
        if not fname.endswith(".h"):
            continue
        text = open(os.path.join(HEADER_DIR, fname)).read()
        text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
        names += re.findall(r"\b(spec_[a-z0-9_]+)\s*\(", text)
    return sorted(set(names))


@pytest.fixture(scope="module")
def library():
    entry.build()
    return binding.lib()


def test_every_declared_symbol_is_exported(library):
    names = declared_functions()
    assert "spec_verify_sample" in names and "spec_last_error" in names
    for name in names:
        assert hasattr(library, name), f"{name} is declared in include/ but not exported"


def test_argument_errors_are_reported_without_touching_the_gpu(library):
    assert library.spec_verify_sample(None, None, None, None, 4, 3, 100, 1.0, None, None, None, 0, None) == -1
    assert b"null pointer" in library.spec_last_error()
    assert library.spec_verify_sample(None, None, None, None, 4, 65, 100, 1.0, None, None, None, 0, None) == -1
    assert b"gamma" in library.spec_last_error()
    assert library.spec_verify_sample(None, None, None, None, 4, 3, 100, -1.0, None, None, None, 0, None) == -1
    assert library.spec_verify_sample(None, None, None, None, 0, 3, 100, 1.0, None, None, None, 0, None) == 0
    assert library.spec_sample(None, None, 3, 0, 1.0, None, None) == -1
    assert library.spec_uniforms(1, None, None, 3, 5, None, None) == -1
    assert library.spec_verify_sample_workspace_bytes(64, 7, 32000) >= 64 * 15 * 4 * 8
