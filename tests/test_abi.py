"""The C-ABI library loads and exports every symbol include/roomie.h declares (no GPU needed)."""
import ctypes
import os
import re

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "roomie.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(roomie_[a-z_0-9]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    from paper_2607_16784_b200 import build
    path = build.build()
    dll = ctypes.CDLL(path)
    names = _declared()
    assert len(names) >= 12
    for n in names:
        assert hasattr(dll, n), n
    import paper_2607_16784_b200 as pkg
    assert sorted(pkg.EXPORTS) == names


def test_host_side_argument_checks():
    """Calls that must be rejected before any CUDA work (safe without a GPU)."""
    import paper_2607_16784_b200 as pkg
    dll = ctypes.CDLL(pkg.lib_path())
    dll.roomie_strerror.restype = ctypes.c_char_p
    assert dll.roomie_strerror(0) == b"ok"
    assert b"invalid" in dll.roomie_strerror(-1)
    assert dll.roomie_occupancy(None, None, None, None) == -1
    assert dll.roomie_library_build(None, None, None, None, None) == -1
    assert dll.roomie_place(None, 0, None, None, None, 0, None, None, None, None, None) == -1

    class Spec(ctypes.Structure):
        _fields_ = [(n, ctypes.c_uint32) for n in "abcde"]
    dll.roomie_share_table_floats.restype = ctypes.c_size_t
    assert dll.roomie_share_table_floats(ctypes.byref(Spec(108, 65536, 164 * 1024, 2048, 32))) == 2 * 64 + 1
    assert dll.roomie_share_table_floats(ctypes.byref(Spec(108, 1 << 18, 164 * 1024, 2048, 32))) == 0   # RANGE
