"""CPU checks of the C-ABI boundary: the library builds, loads and exports what the header declares,
and host-side argument validation answers before anything touches a GPU."""
import ctypes
import os
import re

import paper_2509_21302_b200 as q

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "qvggt.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(qvggt_[a-z0-9_]+)\s*\(", text)))


def test_library_builds_and_exports_every_declared_symbol():
    q.build()
    L = q.lib()
    names = declared_functions()
    assert len(names) >= 8
    for n in names:
        assert hasattr(L, n), n
    assert set(names) == set(q.EXPORTS)


def test_status_strings():
    L = q.lib()
    seen = {L.qvggt_status_string(s) for s in range(0, -8, -1)}
    assert len(seen) == 8 and all(seen)
    assert L.qvggt_status_string(-99) == b"unknown status"


def test_argument_validation_needs_no_gpu():
    L = q.lib()
    h = ctypes.c_void_p(123)
    fake = 0x1000  # a 16-byte-aligned non-NULL address that is never dereferenced on these paths
    assert L.qvggt_prepare_weights(None, None, fake, None, 128, 1024, 0, None, ctypes.byref(h)) == -1
    assert h.value is None                                     # *out is cleared on failure
    assert L.qvggt_prepare_weights(fake, None, fake, None, 128, 1024, 0, None, None) == -1
    assert L.qvggt_prepare_weights(fake, None, fake, None, 128, 1000, 0, None, ctypes.byref(h)) == -2   # K not 2^10 / 2^12
    assert L.qvggt_prepare_weights(fake, None, fake, None, 100, 1024, 0, None, ctypes.byref(h)) == -2   # N % 128
    assert L.qvggt_prepare_weights(fake + 2, None, fake, None, 128, 1024, 0, None, ctypes.byref(h)) == -3
    assert L.qvggt_rotate_smooth_quantize(None, fake, 1024, 4, 0, fake, fake, None) == -1
    assert L.qvggt_w4a4_linear(None, fake, fake, 4, 0, fake, 1024, None, None) == -1
    assert L.qvggt_weights_view(None, None, None, None, None, None, None) == -1
    assert L.qvggt_device_status(None, None, None) == -1
    assert L.qvggt_calibrate_smooth(fake, 4, fake, 4, 512, 0.5, 0.01, 100.0, fake, fake, None) == -2
    assert L.qvggt_calibrate_smooth(None, 4, fake, 4, 1024, 0.5, 0.01, 100.0, fake, fake, None) == -1
    L.qvggt_free_weights(None)                                 # allowed


def test_no_oracle_or_cpu_fallback_in_the_product_path():
    pkg = os.path.join(ROOT, "paper_2509_21302_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, f)).read()
                assert "oracle" not in text.lower().replace("no cpu fallback", ""), f
