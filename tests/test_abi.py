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


def test_header_is_plain_c_and_usable_from_a_c_program(tmp_path):
    """include/ekv.h compiles as strict C99 and a C program drives the host-side calls (block pool, controller,
    status strings, NULL handling) through the shared library."""
    import shutil
    import subprocess
    cc = shutil.which("gcc") or shutil.which("cc")
    assert cc, "a C compiler is part of this build's toolchain"
    exe = str(tmp_path / "c_consumer")
    libdir = os.path.dirname(ekv.library_path())
    subprocess.run([cc, "-std=c99", "-Wall", "-Wextra", "-Werror", "-pedantic", "-I" + os.path.join(ROOT, "include"),
                    os.path.join(ROOT, "tests", "c_consumer.c"), "-o", exe, "-L" + libdir, "-lekv",
                    "-Wl,-rpath," + libdir], check=True)
    out = subprocess.run([exe], check=True, capture_output=True, text=True).stdout
    assert out.strip() == "ok", out
