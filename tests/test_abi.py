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
    import importlib.util
    spec = importlib.util.spec_from_file_location("_roomie_build", os.path.join(ROOT, "paper_2607_16784_b200", "build.py"))
    build = importlib.util.module_from_spec(spec)                  # by path: the package itself needs the library
    spec.loader.exec_module(build)
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


def test_workspace_size_queries_are_host_only():
    """The two size queries read only the host copy of the profile offsets: they answer without a GPU, agree with
    each other on a single pair, grow with the alignment count and refuse a record table that is not 16-byte aligned."""
    import numpy as np
    import paper_2607_16784_b200 as pkg
    from paper_2607_16784_b200 import roomie as rm
    dll = ctypes.CDLL(pkg.lib_path())
    dll.roomie_pair_workspace_bytes.restype = ctypes.c_size_t
    dll.roomie_pair_workspace_bytes.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_uint64, ctypes.c_uint64]
    dll.roomie_pair_interference_workspace_bytes.restype = ctypes.c_size_t
    dll.roomie_pair_interference_workspace_bytes.argtypes = [ctypes.c_void_p, ctypes.c_uint32, ctypes.c_uint32,
                                                             ctypes.c_void_p]
    offsets = np.array([0, 5000, 5003, 9000], np.uint32)
    fake = 0x10000                                           # never dereferenced by the size queries

    def library(records_ptr):
        return rm._Library(3, 9000, offsets.ctypes.data, fake, records_ptr, fake, fake,
                           rm._Spec(108, 65536, 164 * 1024, 2048, 32))

    def opts(mode, n_align):
        return rm._Opts(mode, n_align, 0, 0.5, 8, 0, 0)

    lib = library(fake)
    one = dll.roomie_pair_interference_workspace_bytes(ctypes.byref(lib), 0, 2, ctypes.byref(opts(0, 1)))
    many = dll.roomie_pair_interference_workspace_bytes(ctypes.byref(lib), 0, 2, ctypes.byref(opts(0, 8)))
    assert 0 < one < many
    # pair (0, 2) is pair index 2 of the upper triangle (0,0), (0,1), (0,2), (1,1), ...
    assert dll.roomie_pair_workspace_bytes(ctypes.byref(lib), ctypes.byref(opts(0, 1)), 2, 3) == one
    whole = dll.roomie_pair_workspace_bytes(ctypes.byref(lib), ctypes.byref(opts(0, 1)), 0, 6)
    assert whole > one
    assert dll.roomie_pair_workspace_bytes(ctypes.byref(lib), ctypes.byref(opts(0, 1)), 4, 4) == 0       # empty range
    assert dll.roomie_pair_interference_workspace_bytes(ctypes.byref(lib), 0, 3, ctypes.byref(opts(0, 1))) == 0
    assert dll.roomie_pair_interference_workspace_bytes(ctypes.byref(lib), 0, 2, ctypes.byref(opts(9, 1))) == 0
    # the full Cartesian product of a 5000 x 3997 pair is beyond the 4096 alignments a pair may have
    assert dll.roomie_pair_interference_workspace_bytes(ctypes.byref(lib), 0, 2, ctypes.byref(opts(0, 0))) == 0
    bad = library(fake + 8)
    assert dll.roomie_pair_interference_workspace_bytes(ctypes.byref(bad), 0, 2, ctypes.byref(opts(0, 1))) == 0
    dll.roomie_pair_matrix.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_uint64, ctypes.c_uint64,
                                       ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_size_t,
                                       ctypes.c_void_p]
    assert dll.roomie_pair_matrix(ctypes.byref(bad), ctypes.byref(opts(0, 1)), 0, 6, fake, None, fake * 16, 1 << 20,
                                  None) == -1                # INVALID_ARG before any CUDA call


def test_occupancy_kernel_choice_never_vectorises_a_misaligned_array():
    """The 128-bit occupancy kernel may only be chosen when every array it touches with 128-bit accesses is
    16-byte aligned; a table or output that is only 4-byte aligned (one profile's slice of a concatenated table)
    must get the scalar kernel even when n is a multiple of four.  Pointer values only: nothing is dereferenced."""
    import paper_2607_16784_b200 as pkg
    from paper_2607_16784_b200 import roomie as rm
    dll = ctypes.CDLL(pkg.lib_path())
    base = 0x7F0000000000

    def variant(n, cols=(0, 0, 0, 0), packed=0, occ=0, theo=0, phi=0, no_phi=False, no_packed=False):
        step = 1 << 24
        t = rm._Table(n, *(base + i * step + off for i, off in enumerate(cols)))
        o = rm._OccOut(None if no_packed else base + 4 * step + packed, base + 5 * step + occ, base + 6 * step + theo,
                       None if no_phi else base + 7 * step + phi, None)
        return dll.roomie_occupancy_variant(ctypes.byref(t), ctypes.byref(o))

    assert variant(1024) == 1 | (0xF << 4)                      # everything aligned, n % 4 == 0: all rows wide
    assert variant(1025) == 1 | (0x1 << 4)                      # row c starts 4*c*n bytes in: only row 0 stays aligned
    assert variant(1026) == 1 | (0x5 << 4)                      # n % 4 == 2: rows 0 and 2
    assert variant(1493273) & 1                                 # the benchmark's kernel count takes the wide loads
    assert variant(1024, no_phi=True) == 1 and variant(1024, no_packed=True) == 1 | (0xF << 4)
    assert variant(3) == 0                                      # fewer than four kernels
    for i in range(4):                                          # any input column off by one element
        cols = [0, 0, 0, 0]
        cols[i] = 4
        assert variant(1024, cols=tuple(cols)) == 0
    for kw in (dict(packed=4), dict(occ=8), dict(theo=12)):     # any 128-bit output off the boundary
        assert variant(1024, **kw) == 0
    assert variant(1024, phi=4) == 1                            # phi alone misaligned: wide loads, scalar phi rows
    assert variant(1023, phi=4) == 1 | (0x2 << 4)               # 4 + 4*1023 = 4096: row 1 happens to be aligned
    assert dll.roomie_occupancy_variant(None, None) == -1
