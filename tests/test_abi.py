"""The C-ABI library loads without a GPU and exports every symbol the header declares."""
import ctypes as C
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def binding():
    from paper_2504_03702_b200 import build
    build.build()
    from paper_2504_03702_b200 import binding as B
    return B


def declared_functions():
    names = set()
    for fn in os.listdir(os.path.join(ROOT, "include")):
        if fn.endswith(".h"):
            text = open(os.path.join(ROOT, "include", fn)).read()
            text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
            names |= set(re.findall(r"\b(pre_[a-z_0-9]+)\s*\(", text))
    return names


def test_every_declared_symbol_is_exported(binding):
    names = declared_functions()
    assert {"pre_create", "pre_destroy", "pre_anticipate", "pre_route_batch", "pre_step", "pre_status"} <= names
    raw = C.CDLL(binding.LIB_PATH)
    for n in names:
        assert hasattr(raw, n), f"{n} declared in include/ but not exported"
    assert names == set(binding.EXPORTS), "binding and header disagree on the entry points"


def test_error_strings_and_null_handling(binding):
    B = binding
    assert B.pre_strerror(B.PRE_OK) == "ok"
    for code in (B.PRE_EINVAL, B.PRE_ECAPACITY, B.PRE_EBADREQ, B.PRE_ETIMEOUT, B.PRE_ECUDA, B.PRE_ENOMEM):
        assert B.pre_strerror(code) and "unknown" not in B.pre_strerror(code)
    assert "unknown" in B.pre_strerror(-99)
    assert B.pre_destroy(None) == B.PRE_EINVAL
    assert B.pre_status(None, 0) == B.PRE_EINVAL
    assert B.pre_anticipate(None, 0, 0, 0, 0, 0, 0, 0, 0) == B.PRE_EINVAL
    assert B.pre_route_batch(None, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0) == B.PRE_EINVAL
    assert B.pre_step(None, 0, 0, 0, 0, 0, 0, 0, 0, 0) == B.PRE_EINVAL


@pytest.mark.parametrize("args", [
    (0, 64, 100, 0.8, 1.0, 10),        # no instances
    (8, 0, 100, 0.8, 1.0, 10),         # no horizon
    (8, 8193, 100, 0.8, 1.0, 10),      # horizon above the documented maximum
    (8, 64, 0, 0.8, 1.0, 10),          # no capacity
    (8, 64, 100, float("nan"), 1.0, 10),
    (8, 64, 100, 0.8, -1.0, 10),
    (8, 64, 100, 0.8, 1.0, 0),         # empty table
    (8, 64, 100, 0.8, 1.0, 2 ** 31),   # table too large
])
def test_bad_config_is_refused_on_the_host(binding, args):
    code, ctx = binding.pre_create(*args)
    assert code == binding.PRE_EINVAL and ctx is None


def test_missing_library_is_loud(binding, tmp_path, monkeypatch):
    import importlib.util
    src = os.path.join(ROOT, "paper_2504_03702_b200", "binding.py")
    dst = tmp_path / "binding_copy.py"
    dst.write_text(open(src).read())
    spec = importlib.util.spec_from_file_location("binding_copy", dst)
    mod = importlib.util.module_from_spec(spec)
    with pytest.raises(ImportError, match="no CPU fallback"):
        spec.loader.exec_module(mod)
