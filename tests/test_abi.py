"""The C-ABI library loads without a GPU and exports what include/nsml.h
declares; host-only entry points (sizes, strings) behave as documented."""
import ctypes
import os
import re

import pytest

from paper_2506_16235_b200 import build as nsml_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def nsml():
    nsml_build.build()
    import paper_2506_16235_b200 as mod

    return mod


def declared_functions():
    text = open(os.path.join(ROOT, "include", "nsml.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(nsml_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(nsml):
    names = declared_functions()
    assert len(names) >= 20 and "nsml_compress" in names and "nsml_select_ratio" in names
    raw = ctypes.CDLL(nsml_build.LIB_PATH)
    for name in names:
        assert hasattr(raw, name), f"{name} declared in nsml.h but not exported"


def test_binding_covers_every_symbol(nsml):
    for name in declared_functions():
        assert getattr(nsml.lib, name).argtypes is not None, name


def test_k_rule_and_sizes(nsml):
    assert nsml.nsml_k_of(100, 0.07) == 8
    assert nsml.nsml_k_of(100, 0.29) == 29
    assert nsml.nsml_k_of(1 << 20, 0.01) == 10486
    assert nsml.nsml_k_of(10, 1.0) == 10 and nsml.nsml_k_of(1000, 1e-9) == 1
    for bad in ((0, 0.5), (10, 0.0), (10, 1.5), (10, float("nan")), (1 << 31, 0.5)):
        assert nsml.nsml_k_of(*bad) == 0
    k = 10486
    idx = (4 * k + 15) // 16 * 16
    assert nsml.nsml_payload_bytes(1 << 20, 0.01, 8) == 64 + idx + (k + 15) // 16 * 16 + (11 * 4 + 15) // 16 * 16
    assert nsml.nsml_payload_bytes(1 << 20, 0.01, 16) == 64 + idx + (2 * k + 15) // 16 * 16
    assert nsml.nsml_payload_bytes(1 << 20, 0.01, 4) == 0
    assert nsml.nsml_workspace_bytes(1 << 20, 0) >= 12 * (1 << 20)
    assert nsml.nsml_workspace_bytes(1 << 20, 7) == 0
    assert nsml.nsml_accumulate_workspace_bytes(1 << 20, 4) > 0
    assert nsml.nsml_accumulate_workspace_bytes(1 << 20, 65) == 0


def test_header_struct_is_64_bytes(nsml):
    import numpy as np

    raw = nsml.pack_payload(1000, 8, np.array([1, 5, 9], np.uint32), codes=np.array([1, -2, 3], np.int8),
                            scales=np.array([0.5], np.float32))
    assert raw.size == nsml.nsml_payload_bytes(1000, 0.003, 8)
    back = nsml.unpack_payload(raw)
    assert (back["n"], back["k"], back["bits"], back["idx_off"], back["val_off"], back["scale_off"]) == (1000, 3, 8, 64, 80, 96)
    assert back["idx"].tolist() == [1, 5, 9] and back["codes"].tolist() == [1, -2, 3]


def test_strerror_and_names(nsml):
    assert nsml.nsml_strerror(0) == "ok"
    for code in range(-7, 0):
        assert nsml.nsml_strerror(code) not in ("ok", "unknown status")
    assert nsml.nsml_strerror(-99) == "unknown status"
    assert len(nsml.kernel_names()) == nsml.lib.nsml_kernel_count() >= 5
    assert nsml.nsml_launch_count() == 0 or nsml.nsml_launch_count() > 0


def test_device_calls_reject_bad_arguments_before_touching_cuda(nsml):
    # argument validation happens before any CUDA call, so this runs without a GPU
    buf = (ctypes.c_char * 4096)()
    addr = (ctypes.addressof(buf) + 255) // 256 * 256
    assert nsml.lib.nsml_compress(None, 100, 0, 0.5, 8, None, addr, 4096, addr, 4096, None) == nsml.NSML_ERR_ARG
    assert nsml.lib.nsml_compress(addr, 0, 0, 0.5, 8, None, addr, 4096, addr, 4096, None) == nsml.NSML_ERR_ARG
    assert nsml.lib.nsml_compress(addr, 100, 3, 0.5, 8, None, addr, 4096, addr, 4096, None) == nsml.NSML_ERR_ARG
    assert nsml.lib.nsml_compress(addr, 100, 0, 1.5, 8, None, addr, 4096, addr, 4096, None) == nsml.NSML_ERR_ARG
    assert nsml.lib.nsml_compress(addr, 100, 0, 0.5, 9, None, addr, 4096, addr, 4096, None) == nsml.NSML_ERR_ARG
    assert nsml.lib.nsml_compress(addr + 4, 100, 0, 0.5, 8, None, addr, 4096, addr, 4096, None) == nsml.NSML_ERR_ARG
    assert nsml.lib.nsml_compress(addr, 100, 0, 0.5, 8, None, addr, 16, addr, 4096, None) == nsml.NSML_ERR_CAPACITY
    assert nsml.lib.nsml_compress(addr, 100000, 0, 0.5, 8, None, addr, 1 << 30, addr, 4096, None) == nsml.NSML_ERR_CAPACITY
    ptrs = (ctypes.c_void_p * 1)(addr)
    assert nsml.lib.nsml_decompress_accumulate(ptrs, 0, addr, 100, 1, addr, 4096, None) == nsml.NSML_ERR_ARG
    assert nsml.lib.nsml_decompress_accumulate(ptrs, 65, addr, 100, 1, addr, 4096, None) == nsml.NSML_ERR_ARG
    assert nsml.lib.nsml_decompress_accumulate(ptrs, 1, addr, 100, 1, addr, 16, None) == nsml.NSML_ERR_CAPACITY
    assert nsml.lib.nsml_decompress_accumulate(None, 1, addr, 100, 1, addr, 4096, None) == nsml.NSML_ERR_ARG


def test_sized_entry_points_check_their_size_arguments_on_the_host(nsml):
    # sizes are plain host arguments: they are checked before anything is copied or launched (runs without a GPU)
    import numpy as np

    n, k = 5000, 40
    raw = nsml.pack_payload(n, 8, np.arange(k, dtype=np.uint32) * 7, codes=np.ones(k, np.int8),
                            scales=np.array([0.5], np.float32))
    buf = (ctypes.c_char * 4096)()
    scratch = (ctypes.addressof(buf) + 255) // 256 * 256  # stands in for a device pointer; never dereferenced here
    dense = np.zeros(n, np.float32)
    ptrs = (ctypes.c_void_p * 1)(raw.ctypes.data)
    too_short = (ctypes.c_size_t * 1)(63)  # not even a header
    assert nsml.lib.nsml_decompress_accumulate_host(ptrs, too_short, 1, dense.ctypes.data, n, 1, scratch, 1 << 40,
                                                    None) == nsml.NSML_ERR_ARG
    assert nsml.lib.nsml_decompress_accumulate_sized(ptrs, None, 1, scratch, n, 1, scratch, 4096, None) == nsml.NSML_ERR_ARG
    assert nsml.lib.nsml_decompress_accumulate_sized(ptrs, too_short, 1, scratch, n, 1, scratch, 4096, None) == nsml.NSML_ERR_ARG


def test_list_block_candidates_knob_checks_its_range(nsml):
    # a plain host-side setting: no GPU needed
    for bad in (0, 1023, 8193, -5):
        assert nsml.lib.nsml_set_list_block_candidates(bad) == nsml.NSML_ERR_ARG
    for good in (1024, 8192, 4096):  # leaves the default in place
        assert nsml.lib.nsml_set_list_block_candidates(good) == nsml.NSML_OK
