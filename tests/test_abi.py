"""CPU-only checks of the boundary: the shared library loads and exports every symbol the
header declares; status strings exist; the binding refuses to run without the library."""
import ctypes
import os
import re

from paper_2506_13472_b200 import binding as rb

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "rosaq.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(rosaq_[a-z_0-9]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    names = declared_symbols()
    assert "rosaq_calib_cov" in names and "rosaq_quantize" in names and "rosaq_linear" in names
    lib = ctypes.CDLL(rb.LIB_PATH)
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(rb.EXPORTS) == names


def test_strerror_covers_all_codes():
    seen = {rb.strerror(s) for s in range(0, -8, -1)}
    assert len(seen) == 8 and "unknown status" not in seen
    assert rb.strerror(-99) == "unknown status"


def test_no_cpu_fallback_in_the_product_package():
    pkg = os.path.join(ROOT, "paper_2506_13472_b200")
    for fn in os.listdir(pkg):
        if fn.endswith(".py"):
            src = open(os.path.join(pkg, fn)).read()
            assert "oracle" not in src.replace("oracle's", "").replace("CPU oracle", ""), fn


def test_create_without_gpu_returns_a_code():
    import torch
    if torch.cuda.is_available():
        return
    h = ctypes.c_void_p()
    st = rb.lib().rosaq_create(ctypes.byref(h), 0)
    assert st < 0 and not h.value
