"""CPU-side checks of the boundary: the library builds, loads without a GPU driver and
exports every symbol the header declares; host-side argument checks; the mask generator's
counter-based RNG against its published known-answer vectors."""
import ctypes
import os
import re

import numpy as np
import pytest

import paper_2309_06626_b200 as asx
from paper_2309_06626_b200 import build as asx_build
from philox_ref import philox4x32_10, random_block_mask

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def L():
    asx_build.build()
    return asx.lib()


def test_library_exports_every_declared_symbol(L):
    header = open(os.path.join(ROOT, "include", "asx.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(asx_[a-z_0-9]+)\s*\(", header))
    assert declared, "no declarations found"
    assert declared == set(asx.EXPORTS)
    for name in declared:
        assert hasattr(L, name), name


def test_no_torch_or_python_dependency_in_the_library():
    out = os.popen(f"ldd {asx.lib_path()}").read()
    assert "torch" not in out and "python" not in out and "libcuda.so" not in out


def test_status_strings(L):
    names = {L.asx_status_string(i).decode() for i in range(9)}
    assert len(names) == 9 and "ok" in names
    assert L.asx_status_string(1234).decode() == "unknown status"


def test_create_layer_argument_checks(L):
    h = ctypes.c_void_p()
    assert L.asx_create_layer(64, 64, 3, 3, 1, 1, None) == 1
    for bad in [(0, 64, 3, 3, 1, 1), (64, 0, 3, 3, 1, 1), (64, 64, 0, 3, 1, 1), (64, 64, 3, 3, 0, 1),
                (64, 64, 3, 3, 1, -1)]:
        assert L.asx_create_layer(*bad, ctypes.byref(h)) == 1 and not h.value
    assert L.asx_create_layer(64, 64, 300, 3, 1, 1, ctypes.byref(h)) == 2
    assert L.asx_create_layer(64, 64, 3, 3, 1, 1, ctypes.byref(h)) == 0 and h.value
    # host-side checks that come before any CUDA call
    m = np.ones(8, np.uint8)
    assert L.asx_set_mask(None, m.ctypes.data, 8, None) == 1
    assert L.asx_set_mask(h, None, 8, None) == 1
    assert L.asx_set_mask(h, m.ctypes.data, 0, None) == 1
    assert L.asx_set_mask_random(h, 8, 1.5, 1, 0, None) == 1
    assert L.asx_set_mask_random(h, 8, 0.5, 0, 0, None) == 1
    assert L.asx_run(h, None, 1, 8, 8, None, None, None, 0, None) == 1
    buf = (ctypes.c_char * 64)()
    p = ctypes.addressof(buf)
    assert L.asx_run(h, p, 1, 8, 8, p, None, p, 1 << 20, None) == 1  # unknown flag
    assert L.asx_run(h, p, 1, 8, 8, p, None, p, 64 | 8, None) == 2   # fp32 storage with a compact output: unsupported
    assert L.asx_run(h, p, 1, 8, 8, p, None, p, 0, None) == 3        # no mask yet
    assert L.asx_get_kept(h, None, None) == 3
    assert L.asx_destroy(h) == 0
    assert L.asx_destroy(None) == 0
    assert L.asx_compact_scratch_bytes(-1) == 0
    assert L.asx_compact_scratch_bytes(0) == 16
    assert L.asx_compact_scratch_bytes(4097) == 8 + 16
    assert L.asx_compact(None, -1, None, None, None, 0, None) == 1


def test_philox_known_answers():
    """Known-answer vectors of Philox4x32-10 from the Random123 distribution's test file."""
    assert philox4x32_10((0, 0, 0, 0), (0, 0)) == (0x6627e8d5, 0xe169c58d, 0xbc57ac4c, 0x9b00dbd8)
    assert philox4x32_10((0xffffffff,) * 4, (0xffffffff,) * 2) == (0x408f276d, 0x41c83b0e, 0xa20bc7c6, 0x6d5451fd)
    assert philox4x32_10((0x243f6a88, 0x85a308d3, 0x13198a2e, 0x03707344), (0xa4093822, 0x299f31d0)) == \
        (0xd16cfe09, 0x94fdcceb, 0x5001e420, 0x24126ea1)


def test_reference_mask_generator_structure():
    m = random_block_mask(1000, 0.3, 4, 42)
    assert m.size == 1000 and int((m.reshape(-1, 4).max(1) == 0).sum()) == 75
    assert np.all(m.reshape(-1, 4).min(1) == m.reshape(-1, 4).max(1))
    assert np.all(random_block_mask(17, 0.0, 3, 1) == 1) and np.all(random_block_mask(17, 1.0, 3, 1) == 0)
