"""The C-ABI library loads and exports every symbol include/draco.h declares
(no compute calls: this runs without a GPU)."""
import ctypes
import os
import re

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "draco.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(draco_[a-z_A-Z0-9]+)\s*\(", text)))


def test_library_builds_loads_and_exports_every_declared_symbol():
    from paper_1803_09877_b200 import build
    path = build.build()
    lib = ctypes.CDLL(path)
    names = _declared()
    assert len(names) >= 18
    for name in names:
        assert hasattr(lib, name), name


def test_binding_covers_every_declared_symbol():
    from paper_1803_09877_b200 import build
    build.build()
    from paper_1803_09877_b200 import binding
    assert sorted(binding.EXPORTS) == _declared()
    assert binding.lib.draco_strerror(-1) == b"invalid argument"


def test_argument_checks_need_no_device():
    from paper_1803_09877_b200 import build
    build.build()
    from paper_1803_09877_b200 import binding
    h = ctypes.c_void_p()
    # 2 s + 1 > n violates the corollary of Theorem 1; rejected before any CUDA call
    assert binding.lib.draco_plan_create(4, 2, 100, binding.REP, ctypes.byref(h)) == binding.EINVAL
    assert binding.lib.draco_plan_create(0, 0, 100, binding.REP, ctypes.byref(h)) == binding.EINVAL
    assert binding.lib.draco_plan_create(15, 2, 0, binding.CYC, ctypes.byref(h)) == binding.EINVAL
    assert binding.lib.draco_plan_create(15, 2, 10, 7, ctypes.byref(h)) == binding.EINVAL
    assert binding.lib.draco_plan_create(200, 2, 10, binding.CYC, ctypes.byref(h)) == binding.EINVAL
    assert binding.lib.draco_encode(None, None, None, None) == binding.EINVAL


def test_missing_library_fails_loudly(monkeypatch):
    """There is no CPU fallback: without libdraco.so the binding refuses to load."""
    import pytest
    from paper_1803_09877_b200 import build
    build.build()
    from paper_1803_09877_b200 import binding
    monkeypatch.setattr(binding, "_PKG", "/nonexistent-directory")
    with pytest.raises(binding.DracoError, match="no CPU fallback"):
        binding._load()
