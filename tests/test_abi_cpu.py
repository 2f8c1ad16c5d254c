"""Host-side checks that need no GPU: the library builds, loads and exports every symbol
the header declares; argument errors are reported, not crashed on."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2511_21317_b200 import build, binding
    build.build()
    return binding.load_library()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "httm.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(httm_[a-z_]+)\s*\(", text)))


def test_header_symbols_are_exported(lib):
    from paper_2511_21317_b200 import binding
    names = declared_symbols()
    assert len(names) >= 10 and "httm_create" in names and "httm_global_attention" in names
    assert "httm_dense_attention" in names and "httm_destroy" in names
    for n in names:
        assert hasattr(lib, n), f"{n} is declared in include/httm.h but not exported by libhttm.so"
    assert sorted(binding.EXPORTED_SYMBOLS) == names


def test_null_arguments_are_errors(lib):
    assert lib.httm_create(None, None) == -1
    assert b"null" in lib.httm_last_error(None)
    assert lib.httm_destroy(None) == 0
    assert lib.httm_launch_count(None) == 0
    v = ctypes.c_int64()
    assert lib.httm_query(None, 0, ctypes.byref(v)) == -1


def test_create_rejects_bad_configs(lib):
    from paper_2511_21317_b200 import binding
    import torch

    def make(**kw):
        base = dict(frames=2, grid_h=4, grid_w=4, blk_frames=2, blk_h=2, blk_w=2, ratio_q=0.5, ratio_kv=0.5)
        base.update(kw)
        return binding.HttmConfig(**base)

    for bad, code in ((make(frames=0), -1), (make(ratio_q=1.0), -1), (make(ratio_kv=-0.1), -1), (make(head_dim=128), -2),
                      (make(grid_h=128, grid_w=128, blk_h=64, blk_w=64), -2), (make(blk_w=0), -1), (make(device=99), -1)):
        with pytest.raises(binding.HttmError) as e:
            binding.Httm(bad)
        assert e.value.code == code, (bad, e.value)
    if not torch.cuda.is_available():   # without a device a valid config must fail cleanly, not crash
        with pytest.raises(binding.HttmError):
            binding.Httm(make())


def test_missing_library_fails_loudly(monkeypatch):
    from paper_2511_21317_b200 import binding
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", "/nonexistent/libhttm.so")
    with pytest.raises(ImportError):
        binding.load_library()
