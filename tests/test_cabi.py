"""The C-ABI library builds, loads and exports every function the header declares (no GPU needed)."""
import ctypes
import os
import re

from paper_2603_01399_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "quasar.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(quasar_[a-z_0-9]+)\s*\(", text)))


def test_library_builds_and_exports_every_declared_symbol():
    path = build.build()
    assert os.path.exists(path)
    lib = ctypes.CDLL(path)
    names = _declared()
    assert "quasar_quantize" in names and "quasar_verify" in names and "quasar_kv_commit" in names
    for n in names:
        assert hasattr(lib, n), f"{n} declared in quasar.h but not exported"


def test_binding_covers_every_declared_symbol():
    assert sorted(binding.SIGNATURES) == _declared()


def test_host_side_argument_errors_need_no_gpu():
    lib = binding.lib()
    assert lib.quasar_quantize(None, -1, 8, None, None, None) == -1
    assert lib.quasar_quantize(None, 4, 12, None, None, None) == -2          # K not a multiple of 8
    assert b"multiple of 8" in lib.quasar_last_error()
    assert lib.quasar_quantize(None, 4, 16, None, None, None) == -1          # NULL pointer
    assert lib.quasar_quantize(8, 4, 16, 16, 16, None) == -4                 # misaligned pointer, nothing launched
    out = ctypes.c_size_t(0)
    assert lib.quasar_linear_workspace_bytes(6, 4096, 4096, ctypes.byref(out)) == 0 and out.value > 0
    assert lib.quasar_linear(16, 16, 16, 0, 4, 64, 24, 16, 0, None, 16, 1 << 30, None) == -2   # K % 16 != 0
    assert lib.quasar_verify(None, None, None, None, None, 1, 1, None, None, None, None, None, 0, None, None) == -1
    cfg = binding.Config(1, 256, 4, 2, 48, 688, 1024, 0, 1e6, 1e-6, 0, 128, 0, 0)  # head_dim 48 unsupported
    w = binding.Weights()
    h = ctypes.c_void_p()
    assert lib.quasar_model_create(ctypes.byref(cfg), ctypes.byref(w), ctypes.byref(h)) == -2
