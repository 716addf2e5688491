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


def _varlen_bytes(cu_q, cu_k, Hq, Hkv, d=128):
    n = len(cu_q) - 1
    cq = (ctypes.c_int64 * len(cu_q))(*cu_q)
    ck = (ctypes.c_int64 * len(cu_k))(*cu_k)
    return int(binding.lib().efq_attention_varlen_workspace_bytes(cq, ck, n, Hq, Hkv, d))


def test_workspace_planning_is_host_logic():
    """Sizes of the workspaces follow from the shapes alone (no GPU): the MXFP4 copies take about 0.53 B per
    element, a packed batch needs room for all of its sequences side by side, a decode step packs the query heads
    of a KV group into one tile, and bad prefix sums are refused."""
    one = binding.efq_attention_workspace_bytes(1, 8, 2, 1000, 3000, 128)
    # Q codes + scales of 8 heads x 1024 padded rows, K and V of 2 heads x 3072 padded keys: (64 + 4) B per row
    assert one >= 8 * 1024 * 68 + 2 * 2 * 3072 * 68 and one < 1.2 * (8 * 1024 * 68 + 2 * 2 * 3072 * 68) + 8192
    assert binding.efq_attention_workspace_bytes(1, 8, 3, 128, 128, 128) == 0          # Hq % Hkv != 0
    assert binding.efq_attention_workspace_bytes(1, 8, 2, 128, 128, 64) == 0           # d != 128
    two = _varlen_bytes([0, 1000, 2000], [0, 3000, 6000], 8, 2)
    assert two >= 2 * (one - 8192) and two < 2.2 * one                                # both sequences resident
    with_empty = _varlen_bytes([0, 1000, 1000, 2000], [0, 3000, 3500, 6500], 8, 2)    # a sequence without queries adds nothing
    assert abs(with_empty - two) < 4096
    decode = _varlen_bytes(list(range(65)), [512 * i for i in range(65)], 8, 2)        # 64 sequences, one query token each
    unpacked_q = 64 * 8 * 128 * 68                                                     # one padded tile per query head
    packed_q = 64 * 2 * 128 * 68                                                       # one per KV head
    kv = 64 * 2 * 2 * 512 * 68
    assert decode < kv + packed_q + (unpacked_q - packed_q) // 2 and decode > kv + packed_q
    assert _varlen_bytes([1, 5], [0, 5], 8, 2) == 0                                    # prefix sums must start at 0
    assert _varlen_bytes([0, 5, 3], [0, 5, 9], 8, 2) == 0                              # and never decrease
    assert _varlen_bytes([0, 5], [0, 5], 8, 3) == 0
    assert _varlen_bytes([0], [0], 8, 2) > 0                                           # an empty batch is valid
