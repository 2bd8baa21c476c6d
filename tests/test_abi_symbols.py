"""The shared library loads without a GPU and exports every function the header declares;
argument errors are reported before any CUDA work."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2603_08343_b200 import build
    build.build()
    from paper_2603_08343_b200 import binding
    return binding.lib()


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "wht_affine.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(wht_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    from paper_2603_08343_b200 import binding
    names = _declared_functions()
    assert len(names) >= 12
    for name in names:
        assert hasattr(lib, name), f"{name} declared in wht_affine.h but not exported"
    assert sorted(binding.EXPORTS) == names


def test_argument_errors_need_no_gpu(lib):
    buf = (ctypes.c_char * 4096)()
    base = ctypes.addressof(buf)
    p = ctypes.c_void_p((base + 15) & ~15)
    off = ctypes.c_void_p(p.value + 4)
    s = None
    assert lib.wht_affine_fwd(p, p, p, p, 4, 12, 0, s) == -2          # not a power of two
    assert lib.wht_affine_fwd(p, p, p, p, 4, 4, 0, s) == -2           # below 8
    assert lib.wht_affine_fwd(p, p, p, p, 4, 65536, 0, s) == -2       # above 32768
    assert lib.wht_affine_fwd(p, p, p, p, -1, 256, 0, s) == -3
    assert lib.wht_affine_fwd(p, p, p, p, 4, 256, 7, s) == -4
    assert lib.wht_affine_fwd(None, p, p, p, 4, 256, 0, s) == -1
    assert lib.wht_affine_fwd(p, p, p, off, 4, 256, 0, s) == -5
    assert lib.wht_affine_fwd_decode(p, None, p, p, 4, 256, 1, s) == -1
    assert lib.wht_affine_fwd_residual(p, p, p, None, p, 4, 256, 1, s) == -1
    assert lib.wht_affine_fwd_residual(p, p, p, off, p, 4, 256, 1, s) == -5
    assert lib.wht_affine_bwd(p, p, p, p, None, p, 4, 256, 2, s) == -1
    assert lib.wht_affine_bwd(p, off, p, p, p, p, 4, 256, 2, s) == -5
    assert lib.wht_affine_bwd_ws(p, p, p, p, p, p, 4, 100, 2, p, 64, s) == -2
    assert lib.wht_copy_rows(None, p, 4, 256, 1, s) == -1
    assert lib.wht_affine_reduce_grads(p, 3, 100, p, p, s) == -2
    assert lib.wht_affine_reduce_grads(None, 3, 256, p, p, s) == -1
    assert lib.wht_affine_fwd_grouped(p, p, p, p, 4, 768, 512, 0, s) == -2
    assert lib.wht_affine_fwd_grouped(p, p, p, p, 4, 768, 256, 7, s) == -4
    assert lib.wht_affine_bwd_grouped(p, p, p, p, None, p, 4, 768, 256, 0, p, 64, s) == -1
    assert lib.wht_affine_set_variant(9) == -8 and lib.wht_affine_set_variant(6) == -8
    assert lib.wht_affine_set_variant(0) == 0 and lib.wht_affine_get_variant() == 0
    assert lib.wht_affine_fwd(p, p, p, p, 0, 256, 0, s) == 0           # T == 0: nothing to do
    assert b"power of two" in lib.wht_affine_status_string(-2)
    assert lib.wht_affine_shutdown() == 0


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    import importlib
    from paper_2603_08343_b200 import binding
    monkeypatch.setattr(binding, "LIB_PATH", str(tmp_path / "absent.so"))
    with pytest.raises(ImportError):
        binding._load()
    importlib.reload(binding)
