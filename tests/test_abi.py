"""The C-ABI library loads and exports every function that include/ssd.h declares (no GPU needed)."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    src = open(os.path.join(ROOT, "include", "ssd.h")).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    return sorted(set(re.findall(r"\b(ssd_[a-z0-9_]+)\s*\(", src)))


def test_header_declares_the_three_main_calls():
    names = _declared()
    for n in ("ssd_load_weights", "ssd_prefill", "ssd_decode_block"):
        assert n in names


def test_library_exports_every_declared_symbol():
    import __graft_entry__
    __graft_entry__.build()
    from paper_2510_04147_b200 import binding
    lib = ctypes.CDLL(binding.LIB_PATH)
    for name in _declared():
        assert hasattr(lib, name), name
    assert sorted(binding.EXPORTS) == _declared()


def test_binding_declares_prototypes_and_fails_loudly_without_gpu():
    import torch
    from paper_2510_04147_b200 import binding, workloads as wl
    lib = binding.load_library()
    assert lib.ssd_create.argtypes is not None
    if torch.cuda.is_available():
        pytest.skip("GPU present")
    cfg = binding.config_from_workload(wl.TINY, max_drafts=4)
    ctx = ctypes.c_void_p()
    rc = lib.ssd_create(ctypes.byref(cfg), None, ctypes.byref(ctx))
    assert rc == -4 and not ctx.value                      # SSD_ERR_CUDA: no CPU path
    assert b"no CUDA device" in lib.ssd_last_error(None)
    bad = binding.config_from_workload(wl.TINY.replace(head_dim=48), max_drafts=4)
    assert lib.ssd_create(ctypes.byref(bad), None, ctypes.byref(ctx)) == -2
