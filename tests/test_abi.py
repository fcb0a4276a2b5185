"""Host-side checks that need no GPU: the library loads, exports what the header
declares, and refuses bad arguments before touching a device."""
import ctypes as C
import os
import re

import pytest

from paper_2410_01518_b200 import ipot

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "ipot.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(ipot_[a-z_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    L = ipot.lib()
    names = declared_symbols()
    assert len(names) >= 15
    for s in names:
        assert hasattr(L, s), f"{s} is declared in ipot.h but not exported"
    assert sorted(ipot.SYMBOLS) == names, "the Python binding and the header disagree"


def test_strerror_and_null_handling():
    assert ipot.ipot_strerror(0) == "ok"
    for code in range(-6, 0):
        assert "unknown" not in ipot.ipot_strerror(code)
    assert "unknown" in ipot.ipot_strerror(-99)
    L = ipot.lib()
    assert L.ipot_destroy(None) == 0
    assert L.ipot_append_chunk(None, None, None, 1) == ipot.IPOT_E_INVALID
    assert L.ipot_score_and_compress(None, None, 1, None) == ipot.IPOT_E_INVALID
    assert L.ipot_view(None, None, None, None) == ipot.IPOT_E_INVALID
    assert L.ipot_sync_status(None) == ipot.IPOT_E_INVALID


@pytest.mark.parametrize("args", [
    (0, 1, 1, 8, 2, 64), (512, 512, 1, 8, 2, 64), (512, 0, 1, 8, 2, 64), (512, 256, 1, 8, 3, 64),
    (512, 256, 1, 8, 2, 60), (512, 256, 1, 8, 2, 16), (512, 256, 0, 8, 2, 64), (40000, 256, 1, 8, 2, 64),
])
def test_create_rejects_bad_shapes_before_any_device_work(args):
    h = C.c_void_p()
    assert ipot.lib().ipot_create(*args, C.byref(h)) == ipot.IPOT_E_INVALID
    assert h.value is None


def test_no_fallback_without_a_device():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a device is present")
    with pytest.raises(ipot.IpotError) as e:
        ipot.ipot_create(512, 256, 1, 8, 2, 64)
    assert e.value.code == ipot.IPOT_E_CUDA
