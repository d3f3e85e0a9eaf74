"""The C-ABI library loads on a host without a GPU and exports every symbol include/ekv.h declares."""
import ctypes
import os
import re

import paper_2608_23658_b200 as ekv

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    names = []
    for fn in sorted(os.listdir(os.path.join(ROOT, "include"))):
        if fn.endswith(".h"):
            text = open(os.path.join(ROOT, "include", fn)).read()
            names += re.findall(r"EKV_API\s+[\w\s\*]+?\b(ekv_\w+)\s*\(", text)
    return names


def test_every_declared_symbol_is_exported():
    names = _declared()
    assert len(names) >= 14 and len(set(names)) == len(names)
    lib = ctypes.CDLL(ekv.library_path())
    for n in names:
        assert hasattr(lib, n), n


def test_binding_covers_the_abi():
    for n in _declared():
        assert hasattr(ekv, n), n


def test_status_strings_and_no_device_error():
    assert ekv.ekv_status_string(0) == "EKV_OK"
    assert ekv.ekv_status_string(5) == "EKV_ERR_BLOCK_OOB"
    assert ekv.ekv_status_string(99) == "EKV_ERR_UNKNOWN"
    import torch
    if not torch.cuda.is_available():
        # no fallback: without a device the real backend refuses loudly
        try:
            ekv.ekv_pool_create(num_q_heads=4, num_kv_heads=2, head_dim=64, base_blocks=256)
        except ekv.EkvError as e:
            assert e.status == ekv.Status.ERR_CUDA
        else:
            raise AssertionError("pool creation succeeded without a CUDA device")
