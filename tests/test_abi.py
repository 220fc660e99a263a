"""The C-ABI library loads without a GPU and exports every symbol include/aj_verify.h declares."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def built():
    from paper_2504_20039_b200 import build as b

    return b.build()


def _declared():
    text = open(os.path.join(ROOT, "include", "aj_verify.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(aj_[a-z_0-9]+)\s*\(", text)))


def test_header_symbols_are_exported(built):
    lib = ctypes.CDLL(built)
    names = _declared()
    assert {"aj_create", "aj_verify", "aj_verify_host", "aj_destroy", "aj_last_status"} <= set(names)
    for n in names:
        assert hasattr(lib, n), n


def test_binding_covers_the_header(built):
    import paper_2504_20039_b200 as aj
    from paper_2504_20039_b200 import binding

    aj.lib()
    assert sorted(binding.EXPORTS) == _declared()
    assert "sm_100a" in aj.version()
    assert aj.status_string(aj.AJ_ERR_TIMEOUT)


def test_argument_checks_need_no_device(built):
    import torch

    import paper_2504_20039_b200 as aj

    for args in [(0, 0, 4, 256, 128, 1000), (0, 1, 0, 256, 128, 1000), (0, 1, 2000, 256, 128, 1000),
                 (0, 1, 4, 0, 128, 1000), (0, 1, 4, 256, -1, 1000), (0, 1, 4, 256, 128, 0), (-1, 1, 4, 256, 128, 1000)]:
        with pytest.raises(aj.AjError) as e:
            aj.Handle(*args)
        assert e.value.status == aj.AJ_ERR_INVALID_ARG, args
    with pytest.raises(aj.AjError) as e:
        aj.Handle(0, 1, 4, 250, 128, 1000, aj.AJ_BF16)
    assert e.value.status == aj.AJ_ERR_UNSUPPORTED
    with pytest.raises(aj.AjError) as e:
        aj.Handle(0, 1, 4, 256, 128, 1000, 7)
    assert e.value.status == aj.AJ_ERR_INVALID_ARG
    if not torch.cuda.is_available():  # no device: creation fails cleanly, there is no CPU fallback
        with pytest.raises(aj.AjError) as e:
            aj.Handle(0, 1, 4, 256, 128, 1000)
        assert e.value.status == aj.AJ_ERR_CUDA


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    from paper_2504_20039_b200 import binding

    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", str(tmp_path / "nope.so"))
    with pytest.raises(ImportError):
        binding.lib()
