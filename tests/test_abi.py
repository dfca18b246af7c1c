"""The C-ABI library loads and exports every symbol that include/flashgmm.h declares (no compute without a GPU)."""
import ctypes
import re
from pathlib import Path

import pytest

ROOT = Path(__file__).resolve().parent.parent


@pytest.fixture(scope="module")
def libpath():
    from paper_2606_10896_b200 import build

    return build.build()


def _declared():
    text = (ROOT / "include" / "flashgmm.h").read_text()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(gmm_[a-z0-9_]+)\s*\(", text)))


def test_header_declares_the_boundary():
    names = _declared()
    for must in ("gmm_create", "gmm_destroy", "gmm_em_step", "gmm_finalize", "gmm_fit", "gmm_assign_topm",
                 "gmm_scratch_bytes", "gmm_strerror", "gmm_last_error"):
        assert must in names


def test_library_exports_every_declared_symbol(libpath):
    lib = ctypes.CDLL(str(libpath))
    for name in _declared():
        assert hasattr(lib, name), f"libflashgmm.so does not export {name}"


def test_binding_covers_every_declared_symbol(libpath):
    from paper_2606_10896_b200 import flashgmm

    assert sorted(flashgmm.EXPORTS) == _declared()


def test_host_only_entry_points(libpath):
    lib = ctypes.CDLL(str(libpath))
    lib.gmm_strerror.restype = ctypes.c_char_p
    lib.gmm_version.restype = ctypes.c_char_p
    lib.gmm_scratch_bytes.restype = ctypes.c_size_t
    assert lib.gmm_strerror(0) == b"ok"
    assert b"timed out" in lib.gmm_strerror(-6)
    assert b"sm_100a" in lib.gmm_version()
    # scratch depends on (D, K) only: parameters, partials, exchange slots, and on the tensor path the two fp16 planes of
    # Y for one launch of the tile kernel (2^19 points x 1 KB = 512 MiB) -- well under 1 GiB, whatever N is
    a = lib.gmm_scratch_bytes(128, 1024)
    assert (1 << 29) < a < (1 << 30)
    assert lib.gmm_scratch_bytes(16, 8) < (1 << 27)       # shapes off the tensor path carry no planes
    assert lib.gmm_scratch_bytes(0, 5) == 0
    # a null context is rejected, not dereferenced
    assert lib.gmm_destroy(None) == -1
    assert lib.gmm_set_path(None, 0) == -1


def test_product_package_does_not_reference_the_oracle():
    pkg = ROOT / "paper_2606_10896_b200"
    pat = re.compile(r"^\s*(from|import|#\s*include)\b.*oracle", re.M | re.I)
    for p in list(pkg.rglob("*.py")) + list(pkg.rglob("*.cu")) + list(pkg.rglob("*.cuh")):
        text = p.read_text()
        assert not pat.search(text), p
        assert "gmm_oracle" not in text, p
