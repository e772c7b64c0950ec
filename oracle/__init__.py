"""ctypes front end of the CPU oracle (``roomie_oracle.c``).

TEST INFRASTRUCTURE ONLY: the oracle is the slow, plain statement of what the
hot path computes, written from the paper.  Only the tests, the smoke check and
the benchmark's CPU-baseline leg may import this package; the product path
never does, and this package never imports the CUDA package.

The functions below marshal numpy arrays into the C entry points and hold no
arithmetic of their own.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "roomie_oracle.c")
_LIB = os.path.join(_HERE, "libroomie_oracle.so")

TIMELINE, LOCKSTEP = 0, 1
DETAILED_EQUAL, DETAILED_PRIORITY, DETAILED_FCFS = 2, 3, 4


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (float ops stay float: no FMA contraction)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp%d" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-fopenmp", "-ffp-contract=off",
                               "-fno-fast-math", "-shared", "-fPIC", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


class _Spec(C.Structure):
    _fields_ = [(n, C.c_uint32) for n in
                ("num_sms", "regs_per_sm", "smem_per_sm", "threads_per_sm", "blocks_per_sm")]


class _Lib(C.Structure):
    _fields_ = [("P", C.c_uint32), ("K", C.c_uint32),
                ("offsets", C.c_void_p), ("start", C.c_void_p), ("dt", C.c_void_p),
                ("phi", C.c_void_p), ("T", C.c_void_p), ("spec", _Spec)]


_dll = None


def _lib():
    global _dll
    if _dll is None:
        _dll = C.CDLL(build())
        _dll.oracle_pair.restype = C.c_uint32
        _dll.oracle_pair_matrix.restype = C.c_uint64
        _dll.oracle_timeline.restype = C.c_int
        _dll.oracle_max_threads.restype = C.c_int
    return _dll


def _p(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _spec(spec) -> _Spec:
    return _Spec(spec.num_sms, spec.regs_per_sm, spec.smem_per_sm,
                 spec.threads_per_sm, spec.blocks_per_sm)


def _u32(a):
    return np.ascontiguousarray(a, dtype=np.uint32)


@dataclass
class Occupancy:
    b_lim: np.ndarray
    b_res: np.ndarray
    limiter: np.ndarray
    warps: np.ndarray
    occ: np.ndarray
    occ_theo: np.ndarray
    phi: np.ndarray            # uint32 [4, n]: warps, registers, smem bytes, block slots
    n_unlaunchable: int


def occupancy(grid, threads, regs, smem, spec) -> Occupancy:
    grid, threads, regs, smem = map(_u32, (grid, threads, regs, smem))
    n = len(grid)
    out = [np.zeros(n, dtype=np.uint32) for _ in range(4)]
    occ = np.zeros(n, dtype=np.float32)
    occ_theo = np.zeros(n, dtype=np.float32)
    phi = np.zeros((4, n), dtype=np.uint32)
    bad = C.c_uint32(0)
    s = _spec(spec)
    _lib().oracle_occupancy(C.c_uint32(n), _p(grid), _p(threads), _p(regs), _p(smem), C.byref(s),
                            _p(out[0]), _p(out[1]), _p(out[2]), _p(out[3]),
                            _p(occ), _p(occ_theo), _p(phi), C.byref(bad))
    return Occupancy(out[0], out[1], out[2], out[3], occ, occ_theo, phi, int(bad.value))


@dataclass
class OracleLibrary:
    """Occupancy + tick timelines of a kernel library (arrays kept alive here)."""
    spec: object
    offsets: np.ndarray
    start: np.ndarray
    dt: np.ndarray
    T: np.ndarray
    occ: Occupancy
    status: int

    def _c(self) -> _Lib:
        return _Lib(len(self.offsets) - 1, len(self.start), _p(self.offsets), _p(self.start),
                    _p(self.dt), _p(self.occ.phi), _p(self.T), _spec(self.spec))

    @property
    def num_profiles(self):
        return len(self.offsets) - 1


def timeline(offsets, dur_us, gap_us):
    offsets = _u32(offsets)
    dur = np.ascontiguousarray(dur_us, dtype=np.float32)
    gap = np.ascontiguousarray(gap_us, dtype=np.float32)
    K = len(dur)
    start = np.zeros(K, dtype=np.uint32)
    dt = np.zeros(K, dtype=np.uint32)
    T = np.zeros(len(offsets) - 1, dtype=np.uint64)
    st = _lib().oracle_timeline(C.c_uint32(len(offsets) - 1), _p(offsets), _p(dur), _p(gap),
                                _p(start), _p(dt), _p(T))
    return start, dt, T, int(st)


def library_build(lib) -> OracleLibrary:
    """`lib` is a roomie_synth.Library (or anything with the same array fields)."""
    occ = occupancy(lib.grid_blocks, lib.block_threads, lib.regs_per_thread,
                    lib.smem_per_block, lib.spec)
    start, dt, T, st = timeline(lib.offsets, lib.dur_us, lib.gap_us)
    return OracleLibrary(lib.spec, _u32(lib.offsets), start, dt, T, occ, st)


@dataclass
class PairDetail:
    P_ab: float
    P_ba: float
    evals: int
    kept: int
    s_i: np.ndarray
    s_j: np.ndarray
    delta_i: np.ndarray
    delta_j: np.ndarray
    V: np.ndarray
    evals_c: np.ndarray


def pair(olib: OracleLibrary, a: int, b: int, *, mode=TIMELINE, n_align=1, start_filter=0,
         cap_align: int = 0) -> PairDetail:
    if cap_align == 0:
        qa = int(olib.offsets[a + 1] - olib.offsets[a])
        qb = int(olib.offsets[b + 1] - olib.offsets[b])
        cap_align = qa * qb if n_align == 0 else n_align * n_align
    si = np.zeros(cap_align, dtype=np.uint32)
    sj = np.zeros(cap_align, dtype=np.uint32)
    di = np.zeros(cap_align, dtype=np.float64)
    dj = np.zeros(cap_align, dtype=np.float64)
    V = np.zeros(cap_align, dtype=np.uint64)
    ev = np.zeros(cap_align, dtype=np.uint64)
    pab, pba, evt = C.c_double(0), C.c_double(0), C.c_uint64(0)
    cl = olib._c()
    kept = _lib().oracle_pair(C.byref(cl), C.c_uint32(a), C.c_uint32(b), C.c_int(mode),
                              C.c_uint32(n_align), C.c_int(start_filter),
                              C.byref(pab), C.byref(pba), C.byref(evt), C.c_uint32(cap_align),
                              _p(si), _p(sj), _p(di), _p(dj), _p(V), _p(ev))
    k = min(kept, cap_align)
    return PairDetail(pab.value, pba.value, int(evt.value), int(kept),
                      si[:k], sj[:k], di[:k], dj[:k], V[:k], ev[:k])


def pair_matrix(olib: OracleLibrary, *, mode=TIMELINE, n_align=1, start_filter=0,
                pair_begin: int = 0, pair_end: int | None = None, num_threads: int = 0):
    """Returns (P matrix float64 [P, P], scored pairings)."""
    P = olib.num_profiles
    total = P * (P + 1) // 2
    pair_end = total if pair_end is None else pair_end
    Pm = np.zeros((P, P), dtype=np.float64)
    cl = olib._c()
    ev = _lib().oracle_pair_matrix(C.byref(cl), C.c_int(mode), C.c_uint32(n_align),
                                   C.c_int(start_filter), C.c_uint64(pair_begin),
                                   C.c_uint64(pair_end), _p(Pm), C.c_int(num_threads))
    return Pm, int(ev)


def max_threads() -> int:
    return int(_lib().oracle_max_threads())


def multi_estimate(Pm32, ids, incoming):
    """performance_drop(M) for M = ids + [incoming]; returns (mu f32, mean f32, mu f64, mean f64)."""
    Pm32 = np.ascontiguousarray(Pm32, dtype=np.float32)
    P = Pm32.shape[0]
    ids = np.ascontiguousarray(ids, dtype=np.int32)
    r = len(ids)
    mu = np.zeros(r + 1, dtype=np.float32)
    mu64 = np.zeros(r + 1, dtype=np.float64)
    mean, mean64 = C.c_float(0), C.c_double(0)
    _lib().oracle_multi_estimate(_p(Pm32), C.c_uint32(P), _p(ids), C.c_uint32(r),
                                 C.c_int32(int(incoming)), _p(mu), C.byref(mean),
                                 _p(mu64), C.byref(mean64))
    return mu, np.float32(mean.value), mu64, mean64.value


@dataclass
class Placement:
    gpu: np.ndarray
    mean: np.ndarray
    mu_arr: np.ndarray
    near_tie: np.ndarray
    ids: np.ndarray
    expiry: np.ndarray
    count: np.ndarray
    tick: int


def place(Pm32, num_gpus, max_residents, ids, expiry, count, tick, arr_id, arr_life, lam,
          admit_rule: int = 0, objective: int = 0) -> Placement:
    """Runs the placement stream on copies of the state arrays."""
    Pm32 = np.ascontiguousarray(Pm32, dtype=np.float32)
    P = Pm32.shape[0]
    ids = np.array(ids, dtype=np.int32).reshape(-1).copy()
    expiry = np.array(expiry, dtype=np.uint32).reshape(-1).copy()
    count = np.array(count, dtype=np.uint32).copy()
    arr_id = np.ascontiguousarray(arr_id, dtype=np.int32)
    arr_life = np.ascontiguousarray(arr_life, dtype=np.uint32)
    n = len(arr_id)
    gpu = np.zeros(n, dtype=np.int32)
    mean = np.zeros(n, dtype=np.float32)
    mu_arr = np.zeros(n, dtype=np.float32)
    near = np.zeros(n, dtype=np.uint8)
    t = C.c_uint32(int(tick))
    _lib().oracle_place(_p(Pm32), C.c_uint32(P), C.c_uint32(num_gpus), C.c_uint32(max_residents),
                        _p(ids), _p(expiry), _p(count), C.byref(t), _p(arr_id), _p(arr_life),
                        C.c_uint32(n), C.c_float(lam), C.c_int(admit_rule), C.c_int(objective),
                        _p(gpu), _p(mean), _p(mu_arr), _p(near))
    return Placement(gpu, mean, mu_arr, near, ids, expiry, count, int(t.value))


def assignment_cost(Pm32, models, gpu_of):
    """Average predicted drop of a deployment (float32 as defined, float64 shadow)."""
    Pm32 = np.ascontiguousarray(Pm32, dtype=np.float32)
    models = np.ascontiguousarray(models, dtype=np.int32)
    gpu_of = np.ascontiguousarray(gpu_of, dtype=np.int32)
    c64 = C.c_double(0)
    _lib().oracle_assignment_cost.restype = C.c_float
    c = _lib().oracle_assignment_cost(_p(Pm32), C.c_uint32(Pm32.shape[0]), _p(models), C.c_uint32(len(models)),
                                      _p(gpu_of), C.byref(c64))
    return np.float32(c), c64.value


def optimal_assignment(Pm32, models, num_gpus, max_residents):
    """Exhaustive search; returns (lowest cost float32, one optimal assignment, assignments tried)."""
    Pm32 = np.ascontiguousarray(Pm32, dtype=np.float32)
    models = np.ascontiguousarray(models, dtype=np.int32)
    best = np.full(len(models), -1, dtype=np.int32)
    tried = C.c_uint64(0)
    _lib().oracle_optimal_assignment.restype = C.c_float
    c = _lib().oracle_optimal_assignment(_p(Pm32), C.c_uint32(Pm32.shape[0]), _p(models), C.c_uint32(len(models)),
                                         C.c_uint32(num_gpus), C.c_uint32(max_residents), _p(best), C.byref(tried))
    return np.float32(c), best, int(tried.value)
