"""The C-ABI boundary without a GPU: libmrem.so builds, loads, and exports every function that include/mrem.h
declares; the Python binding knows the same set.  No compute call is made here."""
import ctypes
import os
import re

from paper_2109_15082_b200 import binding as B
from paper_2109_15082_b200 import build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    names = set()
    inc = os.path.join(ROOT, "include")
    for fn in sorted(os.listdir(inc)):
        if not fn.endswith(".h"):
            continue
        text = open(os.path.join(inc, fn)).read()
        text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)             # declarations only, not their comments
        names.update(re.findall(r"\b(mrem_[a-z0-9_]+)\s*\(", text))
    return names


def test_library_exports_every_declared_function():
    path = build.build()
    lib = ctypes.CDLL(path)
    declared = _declared()
    assert len(declared) >= 40 and "mrem_module_forward" in declared and "mrem_recon_loss_noalloc" in declared
    missing = [n for n in sorted(declared) if not hasattr(lib, n)]
    assert not missing, missing


def test_binding_covers_the_header():
    assert set(B.EXPORTS) == _declared()
    lib = B.lib()
    assert all(hasattr(lib, n) for n in B.EXPORTS)
    # host-only calls answer without a device: the error text of a failed create is a string, a null context an argument error
    assert isinstance(lib.mrem_last_error(None), (bytes, type(None), int))
    assert lib.mrem_poll_status(None, None) == -1
