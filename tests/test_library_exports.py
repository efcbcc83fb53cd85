"""CPU-only: the C-ABI library builds, loads and exports every symbol the public header declares."""
import ctypes
import os
import re

import pytest
import torch

from paper_2604_04215_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    names = set()
    for fn in os.listdir(os.path.join(ROOT, "include")):
        if fn.endswith(".h"):
            text = open(os.path.join(ROOT, "include", fn)).read()
            text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
            names |= set(re.findall(r"\b(dare_[a-z_0-9]+)\s*\(", text))
    return names


def test_library_exports_every_declared_symbol():
    build.build()
    lib = ctypes.CDLL(binding.LIB_PATH)
    declared = _declared()
    assert {"dare_attn_block", "dare_lmhead_confidence", "dare_unmask_select", "dare_denoise_block"} <= declared
    for name in declared:
        assert hasattr(lib, name), name
    assert set(binding.EXPORTS) <= declared


def test_status_strings_need_no_gpu():
    lib = binding.load()
    assert lib.dare_status_string(0) == b"ok"
    for code in range(-8, 0):
        assert lib.dare_status_string(code) not in (b"ok", b"unknown status")
    assert lib.dare_status_string(-99) == b"unknown status"


def test_product_path_never_touches_the_oracle():
    """The package may not import or read anything under oracle/ (the oracle is test infrastructure)."""
    pkg = os.path.join(ROOT, "paper_2604_04215_b200")
    for base, _, files in os.walk(pkg):
        for fn in files:
            if fn.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(base, fn)).read()
                assert not re.search(r"(from|import)\s+oracle|oracle[/.]\w|dare_oracle", text), fn


def test_binding_refuses_a_tensor_that_is_not_on_the_current_device(monkeypatch):
    """The library launches on the current device and checks that the context belongs to it (DARE_ERR_DEVICE); the
    binding closes the other half: a buffer on another GPU is refused before its address reaches the library.
    Checked with a stand-in for a tensor, so that no GPU is needed."""
    import pytest
    import torch

    class FakeDevice:
        index = 1

    class FakeTensor:
        is_cuda = True
        dtype = torch.int32
        device = FakeDevice()

        def is_contiguous(self):
            return True

        def data_ptr(self):
            return 0x1000

    monkeypatch.setattr(torch.cuda, "current_device", lambda: 0)
    with pytest.raises(ValueError, match="current device"):
        binding._ptr(FakeTensor(), torch.int32)
    monkeypatch.setattr(torch.cuda, "current_device", lambda: 1)
    assert binding._ptr(FakeTensor(), torch.int32).value == 0x1000


def test_count_outputs_on_the_host_must_be_page_locked():
    """n_committed / n_remaining may live in pinned host memory (the kernel writes them there); pageable host memory,
    which the device cannot address, is refused in the binding."""
    assert binding._count_ptr(None) is None
    with pytest.raises(ValueError, match="page-locked"):
        binding._count_ptr(torch.zeros(4, dtype=torch.int32))


def test_null_context_is_refused_before_anything_else():
    lib = binding.load()
    out = ctypes.c_uint32(0)
    assert lib.dare_device_status(None, None, ctypes.byref(out)) == -1
    h, m = ctypes.c_uint64(0), ctypes.c_uint64(0)
    assert lib.dare_tmap_cache_stats(None, ctypes.byref(h), ctypes.byref(m)) == -1
    assert lib.dare_status_string(-8).startswith(b"the current CUDA device")
