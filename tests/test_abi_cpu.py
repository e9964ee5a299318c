"""CPU-side checks of the C ABI: the library builds, loads without a GPU and
exports every symbol that include/ecq.h declares.  No compute call is made."""
import ctypes
import os
import re

import pytest

from paper_1806_08054_b200 import binding
from paper_1806_08054_b200.build import build_library

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "ecq.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(ecq_[a-z_0-9]+)\s*\(", text)))


def test_header_declares_the_three_core_calls():
    syms = declared_symbols()
    for name in ("ecq_create", "ecq_encode", "ecq_decode_mean", "ecq_destroy", "ecq_status"):
        assert name in syms


def test_library_builds_loads_and_exports_every_declared_symbol():
    path = build_library()
    lib = ctypes.CDLL(path)
    for name in declared_symbols():
        assert hasattr(lib, name), "missing export: " + name


def test_host_only_entry_points_answer_without_a_gpu():
    L = binding.lib()
    assert binding.strerror(binding.ECQ_OK) == "ok"
    assert "argument" in binding.strerror(binding.ECQ_ERR_ARG)
    assert L.ecq_create(None, 1, 32, 1, 1.0, 0.9, 0) == binding.ECQ_ERR_ARG
    assert L.ecq_code_bits(None) == 0 and L.ecq_num_buckets(None) == 0
    assert L.ecq_encode(None, 0, 0, None, None, None, None, None) == binding.ECQ_ERR_ARG
    assert L.ecq_status(None, None) == binding.ECQ_ERR_ARG
    assert isinstance(binding.ecq_launch_count(), int)


def test_binding_refuses_host_tensors():
    import torch
    with pytest.raises(ValueError):
        binding.ecq_encode(1, 0, 0, torch.zeros(4), torch.zeros(4),
                           torch.zeros(1, dtype=torch.int32), torch.zeros(1))


def test_pointer_table_refuses_host_tensors_and_wrong_types():
    import torch
    with pytest.raises(ValueError):
        binding.pointer_table([torch.zeros(4)], torch.float32, "grads")
    with pytest.raises(ValueError):
        binding.ecq_decode_mean(1, [torch.zeros(1, dtype=torch.int32)], [], torch.zeros(4))
