"""The C-ABI library loads and exports every entry point the header declares (no GPU needed)."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "kvq.h")


@pytest.fixture(scope="module")
def kvq_lib():
    from paper_2604_04722_b200 import build, binding
    build.build()
    return binding.lib()


def _declared():
    text = open(HEADER).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(kvq_[a-z_0-9]+)\s*\(", text)))


def test_header_declares_the_five_calls_of_the_boundary():
    names = _declared()
    for must in ("kvq_create", "kvq_select_bits", "kvq_append", "kvq_decode_attn", "kvq_destroy"):
        assert must in names


def test_every_declared_symbol_is_exported_and_bound(kvq_lib):
    from paper_2604_04722_b200 import binding
    names = _declared()
    assert len(names) >= 15
    for name in names:
        assert hasattr(kvq_lib, name), name
        assert name in binding.SIGNATURES, "binding lacks %s" % name
        assert callable(getattr(binding, name)), name
    for name in binding.SIGNATURES:
        assert name in names, "binding has %s which the header does not declare" % name


def test_host_side_argument_checks_need_no_device(kvq_lib):
    h = ctypes.c_void_p()
    assert kvq_lib.kvq_create(None, 1, 1, 1, 64, 16, 1) == -1
    assert kvq_lib.kvq_create(ctypes.byref(h), 1, 9, 3, 32, 16, 1) == -1      # head_dim must be 64
    assert kvq_lib.kvq_create(ctypes.byref(h), 1, 9, 4, 64, 16, 1) == -1      # q_heads % kv_heads
    assert kvq_lib.kvq_create(ctypes.byref(h), 0, 9, 3, 64, 16, 1) == -1
    assert h.value is None
    assert kvq_lib.kvq_destroy(None) == 0
    assert kvq_lib.kvq_strerror(-2) == b"append would exceed max_ctx"
    assert kvq_lib.kvq_strerror(0) == b"ok"
    assert kvq_lib.kvq_decode_attn(None, 0, None, None, None) == -1


def test_binding_fails_loudly_without_the_library(monkeypatch):
    from paper_2604_04722_b200 import binding
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", os.path.join(ROOT, "does_not_exist.so"))
    with pytest.raises(RuntimeError, match="no CPU fallback"):
        binding.lib()
