"""The C-ABI library builds, loads without a GPU and exports every symbol include/efq.h declares."""
import ctypes
import os
import re

from paper_2609_09721_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "efq.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(efq_\w+|exp_then_quantize_\w+)\s*\(", text)))


def test_header_symbols_are_exported():
    lib = ctypes.CDLL(build.build())
    names = _declared_symbols()
    assert "efq_probgen" in names and "efq_attention_fwd" in names and "exp_then_quantize_attention_fwd" in names
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(binding.EXPORTS) == names


def test_status_strings_and_version():
    assert binding.version().startswith("efq-b200")
    assert binding.status_string(0) == "ok"
    assert "timed out" in binding.status_string(7)
    assert len({binding.status_string(i) for i in range(8)}) == 8


def test_host_side_validation_needs_no_gpu():
    L = binding.lib()
    # negative sizes and null pointers are rejected before any CUDA call
    assert L.efq_probgen(None, 0, None, -1, 4, 1.0, None, None, None, None) == 1
    assert L.efq_probgen(None, 0, None, 0, 0, 1.0, None, None, None, None) == 0      # empty problem is a no-op
    assert L.efq_probgen(None, 64, None, 4, 64, 1.0, None, None, None, None) == 1
    p = binding.EfqParams(-3.06, -1.0, 0, 0)
    assert L.efq_probgen(16, 64, 16, 4, 64, 1.0, ctypes.byref(p), 16, 16, None) == 1   # h <= 0
    p = binding.EfqParams(-3.06, 2.3, 0, 0)
    assert L.efq_probgen(16, 32, 16, 4, 64, 1.0, ctypes.byref(p), 16, 16, None) == 1   # ld < cols
    assert L.efq_probgen(20, 64, 16, 4, 64, 1.0, ctypes.byref(p), 16, 16, None) == 3   # misaligned scores
    assert L.efq_probgen(16, 66, 16, 4, 64, 1.0, ctypes.byref(p), 16, 16, None) == 3   # ld % 4 != 0
    assert L.exp_then_quantize_probgen(16, 64, 16, 4, 64, 1.0, 5, 16, 16, None) == 1   # bad scale_mode
    assert L.exp_then_quantize_probgen(16, 64, 16, 4, 64, 1.0, -1, 16, 16, None) == 1
