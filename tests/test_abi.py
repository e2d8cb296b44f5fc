"""The C-ABI library loads without a GPU and exports every symbol that include/prox.h declares."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "prox.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(prox_[a-z_]+)\s*\(", text)))


def test_header_declares_the_contract_functions():
    syms = declared_symbols()
    for name in ["prox_create", "prox_query_batch", "prox_reset_cache", "prox_destroy"]:
        assert name in syms


def test_library_exports_every_declared_symbol():
    import __graft_entry__ as g
    g.build()
    from paper_2503_05530_b200 import prox
    lib = ctypes.CDLL(prox.LIB_PATH)
    for name in declared_symbols():
        assert hasattr(lib, name), f"{name} is declared in prox.h but not exported"


def test_calls_without_handle_are_rejected_on_the_host():
    from paper_2503_05530_b200 import prox
    lib = prox.load_library()
    assert lib.prox_query_batch(None, None, 1, None, None, None, None) == prox.ERR_INVALID_ARG
    assert lib.prox_reset_cache(None, None) == prox.ERR_INVALID_ARG
    assert b"NULL" in lib.prox_last_error()
    lib.prox_destroy(None)
    assert not lib.prox_create(None, 10, 16, 1, 1, 0.5, 0)
    # the wider constructors check their own arguments before they touch the device
    assert not lib.prox_create_rho(None, 10, 16, 1, 1, 0.5, 0, 0) and b"rho" in lib.prox_last_error()
    assert not lib.prox_create_metric(None, 10, 16, 1, 1, 0.5, 0, 1, 7) and b"metric" in lib.prox_last_error()
    assert not lib.prox_create_lsh(None, 10, 16, 1, 25, 4, None, 0.5, 0, 1) and b"L must" in lib.prox_last_error()
    assert not lib.prox_create_lsh(None, 10, 16, 1, 3, 0, None, 0.5, 0, 1) and b"bucket" in lib.prox_last_error()


def test_binding_fails_loudly_without_the_library(monkeypatch):
    from paper_2503_05530_b200 import prox
    monkeypatch.setattr(prox, "_lib", None)
    monkeypatch.setattr(prox, "LIB_PATH", "/nonexistent/libprox.so")
    with pytest.raises(prox.ProxError):
        prox.load_library()
