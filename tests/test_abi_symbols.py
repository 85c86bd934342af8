"""The C-ABI library builds, loads without a GPU and exports every symbol the header declares."""
import ctypes
import os
import re

from paper_2608_24067_b200 import build as som_build
from paper_2608_24067_b200 import som

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "som.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(som_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    path = som_build.build()
    lib = ctypes.CDLL(path)
    names = _declared()
    assert "som_create" in names and "som_bmu" in names and "som_norms" in names and "som_destroy" in names
    for n in names:
        assert hasattr(lib, n), "missing export: " + n
    assert sorted(som.EXPORTS) == names


def test_host_only_calls_without_gpu():
    """Calls that touch no device: status strings and null-handle behaviour."""
    lib = som.load_library()
    assert lib.som_status_string(0) == b"SOM_OK"
    assert lib.som_status_string(2) == b"SOM_ERR_NORMS_STALE"
    assert lib.som_status_string(99) == b"SOM_ERR_UNKNOWN"
    assert lib.som_destroy(None) == 0
    assert lib.som_last_cuda_error(None) == 0
    assert lib.som_launch_count(None) == 0
    out = ctypes.c_void_p()
    assert lib.som_create(ctypes.byref(out), 0, 0, None) == 1  # invalid arguments, checked first
    assert lib.som_norms(None, None) == 1
    assert lib.som_bmu(None, None, None, 0, None, None, None) == 1
    assert lib.som_bmu2(None, None, None, 0, None, None, None, None, None) == 1
    assert lib.som_bmu_values(None, None, None, None, 0, None, None, None) == 1
    assert lib.som_update(None, 1, 1, None, None, 0, None, 1, None) == 1
    assert lib.som_bmu_host_async(None, None, None, 0, None, None, None) == 1
    assert lib.som_host_sync(None) == 1
    assert lib.som_last_uncertain(None) == 0
    assert lib.som_create_f16(ctypes.byref(out), 0, 0, None) == 1
    assert lib.som_norms_noalloc(0, 0, None, None, None) == 1


def test_no_signature_mentions_torch():
    text = open(os.path.join(ROOT, "include", "som.h")).read()
    assert "torch" not in text and "at::" not in text
