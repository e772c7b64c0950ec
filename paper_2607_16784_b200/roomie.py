"""ctypes binding of libroomie.so: same names as the C entry points, torch tensors in and out."""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass

import numpy as np
import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_PKG, "libroomie.so")

TIMELINE, LOCKSTEP = 0, 1
DETAILED_EQUAL, DETAILED_PRIORITY, DETAILED_FCFS = 2, 3, 4

EXPORTS = [
    "roomie_occupancy", "roomie_occupancy_variant", "roomie_library_build",
    "roomie_pair_workspace_bytes", "roomie_pair_matrix", "roomie_pair_interference",
    "roomie_pair_interference_workspace_bytes", "roomie_selftest_bounded_wait",
    "roomie_pair_interference_static",
    "roomie_multi_estimate", "roomie_place", "roomie_place_batch", "roomie_optimal_workspace_bytes",
    "roomie_optimal_assignment", "roomie_assignment_cost", "roomie_strerror", "roomie_last_cuda_error",
    "roomie_launch_count", "roomie_reset_launch_count", "roomie_profile_enable", "roomie_profile_walk_ms",
]


class RoomieError(RuntimeError):
    pass


def lib_path() -> str:
    return _LIB_PATH


def _load():
    if not os.path.exists(_LIB_PATH):
        raise ImportError(
            f"{_LIB_PATH} is missing: build it with `python paper_2607_16784_b200/build.py` "
            "(nvcc, sm_100a).  This package has no CPU or PyTorch fallback.")
    dll = C.CDLL(_LIB_PATH)
    dll.roomie_strerror.restype = C.c_char_p
    dll.roomie_last_cuda_error.restype = C.c_char_p
    dll.roomie_launch_count.restype = C.c_uint64
    dll.roomie_pair_workspace_bytes.restype = C.c_size_t
    dll.roomie_pair_workspace_bytes.argtypes = [C.c_void_p, C.c_void_p, C.c_uint64, C.c_uint64]
    dll.roomie_selftest_bounded_wait.argtypes = [C.c_void_p, C.c_uint64, C.c_void_p]
    dll.roomie_pair_interference_workspace_bytes.restype = C.c_size_t
    dll.roomie_pair_interference_workspace_bytes.argtypes = [C.c_void_p, C.c_uint32, C.c_uint32, C.c_void_p]
    dll.roomie_pair_matrix.argtypes = [C.c_void_p, C.c_void_p, C.c_uint64, C.c_uint64, C.c_void_p,
                                       C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p]
    dll.roomie_pair_interference.argtypes = [C.c_void_p, C.c_uint32, C.c_uint32, C.c_void_p, C.c_void_p,
                                             C.c_void_p, C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p]
    dll.roomie_pair_interference_static.argtypes = [C.c_void_p, C.c_uint32, C.c_uint32, C.c_void_p, C.c_void_p,
                                                    C.c_void_p, C.c_void_p, C.c_void_p]
    dll.roomie_optimal_workspace_bytes.restype = C.c_size_t
    dll.roomie_optimal_workspace_bytes.argtypes = [C.c_uint32]
    dll.roomie_optimal_assignment.argtypes = [C.c_void_p, C.c_uint32, C.c_void_p, C.c_uint32, C.c_uint32, C.c_uint32,
                                              C.c_uint32, C.c_void_p, C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p]
    dll.roomie_assignment_cost.argtypes = [C.c_void_p, C.c_uint32, C.c_void_p, C.c_void_p, C.c_uint32, C.c_uint32,
                                           C.c_void_p, C.c_void_p]
    dll.roomie_occupancy.argtypes = [C.c_void_p] * 4
    dll.roomie_library_build.argtypes = [C.c_void_p] * 5
    dll.roomie_multi_estimate.argtypes = [C.c_void_p, C.c_uint32, C.c_void_p, C.c_void_p, C.c_void_p,
                                          C.c_uint32, C.c_uint32, C.c_void_p, C.c_void_p, C.c_void_p]
    dll.roomie_place.argtypes = [C.c_void_p, C.c_uint32, C.c_void_p, C.c_void_p, C.c_void_p, C.c_uint32,
                                 C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
    dll.roomie_place_batch.argtypes = [C.c_void_p, C.c_uint32, C.c_void_p, C.c_void_p, C.c_void_p, C.c_uint32,
                                       C.c_uint32, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
    return dll


_dll = _load()


def _check(rc: int, what: str):
    if rc != 0:
        msg = _dll.roomie_strerror(rc).decode()
        if rc == -3:
            msg += ": " + _dll.roomie_last_cuda_error().decode()
        raise RoomieError(f"{what} failed ({rc}): {msg}")


class _Spec(C.Structure):
    _fields_ = [(n, C.c_uint32) for n in
                ("num_sms", "regs_per_sm", "smem_per_sm", "threads_per_sm", "blocks_per_sm")]


class _Table(C.Structure):
    _fields_ = [("n", C.c_uint32), ("grid_blocks", C.c_void_p), ("block_threads", C.c_void_p),
                ("regs_per_thread", C.c_void_p), ("smem_per_block", C.c_void_p)]


class _OccOut(C.Structure):
    _fields_ = [("packed4", C.c_void_p), ("occ", C.c_void_p), ("occ_theo", C.c_void_p),
                ("phi", C.c_void_p), ("n_unlaunchable", C.c_void_p)]


class _Library(C.Structure):
    _fields_ = [("num_profiles", C.c_uint32), ("num_kernels", C.c_uint32),
                ("offsets_host", C.c_void_p), ("offsets", C.c_void_p), ("records", C.c_void_p),
                ("T", C.c_void_p), ("status", C.c_void_p), ("spec", _Spec)]


class _Opts(C.Structure):
    _fields_ = [("walk_mode", C.c_int32), ("n_align", C.c_uint32), ("start_filter", C.c_int32),
                ("lam", C.c_float), ("max_residents", C.c_uint32), ("admit_rule", C.c_int32),
                ("objective", C.c_int32)]


class _Detail(C.Structure):
    _fields_ = [("capacity", C.c_uint32), ("n_kept", C.c_void_p), ("s_i", C.c_void_p), ("s_j", C.c_void_p),
                ("delta_i", C.c_void_p), ("delta_j", C.c_void_p), ("V", C.c_void_p), ("evals", C.c_void_p)]


class _State(C.Structure):
    _fields_ = [("num_gpus", C.c_uint32), ("max_residents", C.c_uint32), ("ids", C.c_void_p),
                ("expiry", C.c_void_p), ("count", C.c_void_p), ("tick", C.c_void_p)]


@dataclass(frozen=True)
class GpuSpec:
    num_sms: int
    regs_per_sm: int
    smem_per_sm: int
    threads_per_sm: int
    blocks_per_sm: int


def _cspec(spec) -> _Spec:
    return _Spec(spec.num_sms, spec.regs_per_sm, spec.smem_per_sm, spec.threads_per_sm, spec.blocks_per_sm)


def _stream(stream=None):
    s = torch.cuda.current_stream() if stream is None else stream
    return C.c_void_p(s.cuda_stream)


def _ptr(t):
    return None if t is None else C.c_void_p(t.data_ptr())


def _dev(t, dtype):
    """Device tensor of `dtype` from a tensor or array; unsigned 32/64-bit arrays are
    reinterpreted as the signed torch dtype of the same width (bit pattern kept)."""
    if not isinstance(t, torch.Tensor):
        a = np.ascontiguousarray(t)
        if a.dtype == np.uint32:
            a = a.view(np.int32)
        elif a.dtype == np.uint64:
            a = a.view(np.int64)
        t = torch.from_numpy(a)
    if t.dtype != dtype:
        t = t.to(dtype)
    if not t.is_cuda:
        t = t.cuda()
    return t.contiguous()


def _table(grid, threads, regs, smem):
    g, t, r, s = (_dev(x, torch.int32) for x in (grid, threads, regs, smem))
    n = g.numel()
    if not (t.numel() == r.numel() == s.numel() == n):
        raise ValueError("kernel table columns differ in length")
    return _Table(n, g.data_ptr(), t.data_ptr(), r.data_ptr(), s.data_ptr()), (g, t, r, s)


def occupancy(grid, threads, regs, smem, spec, stream=None):
    """roomie_occupancy: Eq. 1 for every kernel.  Returns a dict of device tensors:
    b_lim, b_res, limiter, warps (uint8 views of the packed word), occ, occ_theo (float32),
    phi (int32 [4, n]), n_unlaunchable (int32 [1])."""
    tab, keep = _table(grid, threads, regs, smem)
    n = tab.n
    dev = keep[0].device
    packed = torch.empty(n, dtype=torch.int32, device=dev)
    occ = torch.empty(n, dtype=torch.float32, device=dev)
    occ_theo = torch.empty(n, dtype=torch.float32, device=dev)
    phi = torch.empty((4, n), dtype=torch.int32, device=dev)
    bad = torch.zeros(1, dtype=torch.int32, device=dev)
    out = _OccOut(packed.data_ptr(), occ.data_ptr(), occ_theo.data_ptr(), phi.data_ptr(), bad.data_ptr())
    cs = _cspec(spec)
    _check(_dll.roomie_occupancy(C.byref(tab), C.byref(cs), C.byref(out), _stream(stream)), "roomie_occupancy")
    b = packed.view(torch.uint8).view(n, 4)
    return dict(b_lim=b[:, 0], b_res=b[:, 1], limiter=b[:, 2], warps=b[:, 3], occ=occ,
                occ_theo=occ_theo, phi=phi, n_unlaunchable=bad, packed4=packed)


class Library:
    """Device-resident kernel library (walk records, T, share table) plus its C view."""

    def __init__(self, offsets, spec, device):
        self.offsets_host = np.ascontiguousarray(offsets, dtype=np.uint32)
        self.spec = spec
        P, K = len(self.offsets_host) - 1, int(self.offsets_host[-1])
        self.num_profiles, self.num_kernels = P, K
        self.offsets = torch.empty(P + 1, dtype=torch.int32, device=device)
        self.records = torch.empty((K, 4), dtype=torch.int32, device=device)
        self.T = torch.empty(P, dtype=torch.int64, device=device)
        cs = _cspec(spec)
        self.status = torch.zeros(1, dtype=torch.int32, device=device)
        self.c = _Library(P, K, self.offsets_host.ctypes.data, self.offsets.data_ptr(),
                          self.records.data_ptr(), self.T.data_ptr(), self.status.data_ptr(), cs)

    def status_flags(self) -> int:
        """Synchronises and returns the sticky ROOMIE_FLAG_* bits."""
        return int(self.status.item()) & 0xFFFFFFFF

    def check(self):
        f = self.status_flags()
        if f:
            names = [n for b, n in ((1, "TICK_OVERFLOW"), (2, "BAD_TIME"), (4, "WORKSPACE"), (8, "WAIT_TIMEOUT")) if f & b]
            raise RoomieError("library status flags set: " + "|".join(names))


def library_build(grid, threads, regs, smem, dur_us, gap_us, offsets, spec, stream=None, out: Library | None = None) -> Library:
    """roomie_library_build: occupancy + tick timelines -> 16-byte walk records."""
    tab, keep = _table(grid, threads, regs, smem)
    d, g = _dev(dur_us, torch.float32), _dev(gap_us, torch.float32)
    lib = out if out is not None else Library(offsets, spec, keep[0].device)
    _check(_dll.roomie_library_build(C.byref(lib.c), C.byref(tab), _ptr(d), _ptr(g), _stream(stream)),
           "roomie_library_build")
    return lib


def _opts(mode=TIMELINE, n_align=1, start_filter=0, lam=0.5, max_residents=0, admit_rule=0, objective=0) -> _Opts:
    return _Opts(int(mode), int(n_align), int(start_filter), float(lam), int(max_residents),
                 int(admit_rule), int(objective))


def pair_workspace_bytes(lib: Library, *, mode=TIMELINE, n_align=1, start_filter=0,
                         pair_begin=0, pair_end=None) -> int:
    total = lib.num_profiles * (lib.num_profiles + 1) // 2
    o = _opts(mode, n_align, start_filter)
    return int(_dll.roomie_pair_workspace_bytes(C.byref(lib.c), C.byref(o), pair_begin,
                                                total if pair_end is None else pair_end))


def _workspace(nbytes, device):
    return torch.empty(max(int(nbytes), 256), dtype=torch.uint8, device=device)


def pair_matrix(lib: Library, *, mode=TIMELINE, n_align=1, start_filter=0, pair_begin=0, pair_end=None,
                out=None, evals=None, workspace=None, max_workspace_bytes=1 << 30, stream=None):
    """roomie_pair_matrix: P[i][j] for the unordered pairs [pair_begin, pair_end).
    Returns (P float32 [P, P] device tensor, evals int64 [1] device tensor)."""
    P = lib.num_profiles
    total = P * (P + 1) // 2
    pair_end = total if pair_end is None else pair_end
    dev = lib.records.device
    if out is None:
        out = torch.zeros((P, P), dtype=torch.float32, device=dev)
    if evals is None:
        evals = torch.zeros(1, dtype=torch.int64, device=dev)
    o = _opts(mode, n_align, start_filter)
    if workspace is None:
        need = int(_dll.roomie_pair_workspace_bytes(C.byref(lib.c), C.byref(o), pair_begin, pair_end))
        workspace = _workspace(min(need, max_workspace_bytes), dev)
    _check(_dll.roomie_pair_matrix(C.byref(lib.c), C.byref(o), pair_begin, pair_end, _ptr(out), _ptr(evals),
                                   _ptr(workspace), workspace.numel(), _stream(stream)), "roomie_pair_matrix")
    return out, evals


def _pair_outputs(dev, detail_capacity, out2=None):
    if out2 is None:
        out2 = torch.zeros(2, dtype=torch.float32, device=dev)
    evals = None if detail_capacity < 0 else torch.zeros(1, dtype=torch.int64, device=dev)
    res = dict(P2=out2, evals=evals)
    det = None
    if detail_capacity > 0:
        cap = int(detail_capacity)
        res.update(n_kept=torch.zeros(1, dtype=torch.int32, device=dev),
                   s_i=torch.zeros(cap, dtype=torch.int32, device=dev),
                   s_j=torch.zeros(cap, dtype=torch.int32, device=dev),
                   delta_i=torch.zeros(cap, dtype=torch.float32, device=dev),
                   delta_j=torch.zeros(cap, dtype=torch.float32, device=dev),
                   V=torch.zeros(cap, dtype=torch.int64, device=dev),
                   evals_c=torch.zeros(cap, dtype=torch.int32, device=dev))
        det = _Detail(cap, res["n_kept"].data_ptr(), res["s_i"].data_ptr(), res["s_j"].data_ptr(),
                      res["delta_i"].data_ptr(), res["delta_j"].data_ptr(), res["V"].data_ptr(),
                      res["evals_c"].data_ptr())
    return res, det


def pair_interference(lib: Library, a: int, b: int, *, mode=TIMELINE, n_align=1, start_filter=0,
                      detail_capacity=0, workspace=None, stream=None):
    """roomie_pair_interference: one ordered pair.  Returns a dict with P_ab, P_ba (float32 [2] tensor
    `P2`), evals and, when detail_capacity > 0, the per-alignment arrays."""
    dev = lib.records.device
    o = _opts(mode, n_align, start_filter)
    res, det = _pair_outputs(dev, detail_capacity)
    if workspace is None:
        workspace = _workspace(_dll.roomie_pair_interference_workspace_bytes(C.byref(lib.c), a, b, C.byref(o)), dev)
    _check(_dll.roomie_pair_interference(C.byref(lib.c), a, b, C.byref(o), _ptr(res["P2"]), _ptr(res["evals"]),
                                         C.byref(det) if det is not None else None, _ptr(workspace),
                                         workspace.numel(), _stream(stream)), "roomie_pair_interference")
    return res


def pair_interference_static(lib: Library, a: int, b: int, *, mode=TIMELINE, n_align=1, start_filter=0,
                             detail_capacity=0, out2=None, stream=None):
    """roomie_pair_interference_static: the same result computed in the library's built-in scratch
    array - for callers that cannot allocate device memory.  Calls that overlap on the GPU race.
    With `out2` (float32 [2] device tensor) given and no detail requested, the binding itself creates no
    tensor either: the evaluation count is then not returned."""
    o = _opts(mode, n_align, start_filter)
    res, det = _pair_outputs(lib.records.device, -1 if (out2 is not None and detail_capacity == 0) else detail_capacity, out2)
    _check(_dll.roomie_pair_interference_static(C.byref(lib.c), a, b, C.byref(o), _ptr(res["P2"]),
                                                _ptr(res["evals"]), C.byref(det) if det is not None else None,
                                                _stream(stream)), "roomie_pair_interference_static")
    return res


def multi_estimate(Pmat, resident_ids, count, incoming, max_residents=None, stream=None):
    """roomie_multi_estimate, batched: resident_ids [n_sets, R], count [n_sets], incoming [n_sets].
    Returns (mu float32 [n_sets, R+1], mean float32 [n_sets])."""
    Pm = _dev(Pmat, torch.float32)
    ids = _dev(resident_ids, torch.int32)
    cnt = _dev(count, torch.int32)
    inc = _dev(incoming, torch.int32)
    n = inc.numel()
    R = int(max_residents if max_residents is not None else (ids.numel() // max(n, 1)))
    mu = torch.zeros((n, R + 1), dtype=torch.float32, device=Pm.device)
    mean = torch.zeros(n, dtype=torch.float32, device=Pm.device)
    _check(_dll.roomie_multi_estimate(_ptr(Pm), Pm.shape[0], _ptr(ids) if ids.numel() else None, _ptr(cnt),
                                      _ptr(inc), n, R, _ptr(mu), _ptr(mean), _stream(stream)),
           "roomie_multi_estimate")
    return mu, mean


class ClusterState:
    """Device-resident cluster state (ids, expiry, count, tick), updated in place by place()."""

    def __init__(self, num_gpus, max_residents, ids, expiry, count, tick=0, device="cuda"):
        self.num_gpus, self.max_residents = int(num_gpus), int(max_residents)
        self.ids = _dev(np.asarray(ids, dtype=np.int32).reshape(-1), torch.int32).clone()
        self.expiry = _dev(np.asarray(expiry, dtype=np.uint32).reshape(-1).view(np.int32), torch.int32).clone()
        self.count = _dev(np.asarray(count, dtype=np.uint32).view(np.int32), torch.int32).clone()
        self.tick = torch.tensor([int(tick)], dtype=torch.int32, device=self.ids.device)
        self.c = _State(self.num_gpus, self.max_residents, self.ids.data_ptr(), self.expiry.data_ptr(),
                        self.count.data_ptr(), self.tick.data_ptr())

    @classmethod
    def from_tensors(cls, num_gpus, max_residents, ids, expiry, count, tick):
        """Wraps int32 device tensors (ids [G*R], expiry [G*R], count [G], tick [1]) without copying."""
        self = cls.__new__(cls)
        self.num_gpus, self.max_residents = int(num_gpus), int(max_residents)
        self.ids, self.expiry, self.count, self.tick = ids, expiry, count, tick
        self.c = _State(self.num_gpus, self.max_residents, ids.data_ptr(), expiry.data_ptr(),
                        count.data_ptr(), tick.data_ptr())
        return self


def place(Pmat, state: ClusterState, arr_id, arr_life, lam=0.5, want_mean=True, stream=None,
          admit_rule=0, objective=0):
    """roomie_place: Algorithm 2 over a stream of arrivals.  Returns (gpu int32 [n], mean, mu_arr)."""
    Pm = _dev(Pmat, torch.float32)
    aid = _dev(arr_id, torch.int32)
    life = _dev(np.asarray(arr_life, dtype=np.uint32).view(np.int32) if not isinstance(arr_life, torch.Tensor)
                else arr_life, torch.int32)
    n = aid.numel()
    gpu = torch.empty(n, dtype=torch.int32, device=Pm.device)
    mean = torch.empty(n, dtype=torch.float32, device=Pm.device) if want_mean else None
    mu_arr = torch.empty(n, dtype=torch.float32, device=Pm.device) if want_mean else None
    o = _opts(lam=lam, max_residents=state.max_residents, admit_rule=admit_rule, objective=objective)
    _check(_dll.roomie_place(_ptr(Pm), Pm.shape[0], C.byref(state.c), _ptr(aid), _ptr(life), n, C.byref(o),
                             _ptr(gpu), _ptr(mean), _ptr(mu_arr), _stream(stream)), "roomie_place")
    return gpu, mean, mu_arr


def place_batch(Pmat, num_gpus, max_residents, ids, expiry, count, tick, arr_id, arr_life, lam=0.5,
                want_mean=False, stream=None, admit_rule=0, objective=0):
    """roomie_place_batch: S independent arrival streams, one CTA each.  ids/expiry [S, G*R], count [S, G],
    tick [S], arr_id/arr_life [S, n] (int32 device tensors or arrays; the state tensors are updated in place
    when they already are contiguous int32 device tensors).  Returns (gpu int32 [S, n], mean, mu_arr, state)."""
    Pm = _dev(Pmat, torch.float32)
    u32 = lambda x: x if isinstance(x, torch.Tensor) else np.asarray(x, dtype=np.uint32).view(np.int32)
    ids_t, exp_t, cnt_t, tick_t = (_dev(ids, torch.int32), _dev(u32(expiry), torch.int32),
                                   _dev(u32(count), torch.int32), _dev(u32(tick), torch.int32))
    aid, life = _dev(arr_id, torch.int32), _dev(u32(arr_life), torch.int32)
    S, n = aid.shape[0], aid.shape[1]
    if ids_t.numel() != S * num_gpus * max_residents or cnt_t.numel() != S * num_gpus or tick_t.numel() != S \
            or life.shape != aid.shape:
        raise ValueError("per-stream arrays do not match the number of streams")
    state = _State(int(num_gpus), int(max_residents), ids_t.data_ptr(), exp_t.data_ptr(), cnt_t.data_ptr(),
                   tick_t.data_ptr())
    gpu = torch.empty((S, n), dtype=torch.int32, device=Pm.device)
    mean = torch.empty((S, n), dtype=torch.float32, device=Pm.device) if want_mean else None
    mu_arr = torch.empty((S, n), dtype=torch.float32, device=Pm.device) if want_mean else None
    o = _opts(lam=lam, max_residents=max_residents, admit_rule=admit_rule, objective=objective)
    _check(_dll.roomie_place_batch(_ptr(Pm), Pm.shape[0], C.byref(state), _ptr(aid), _ptr(life), n, S, C.byref(o),
                                   _ptr(gpu), _ptr(mean), _ptr(mu_arr), _stream(stream)), "roomie_place_batch")
    return gpu, mean, mu_arr, dict(ids=ids_t, expiry=exp_t, count=cnt_t, tick=tick_t)


def optimal_assignment(Pmat, models, num_gpus, max_residents, want_assign=True, stream=None):
    """roomie_optimal_assignment: models [S, n] -> (best_cost float32 [S], best_assign int32 [S, n] or None)."""
    Pm = _dev(Pmat, torch.float32)
    m = _dev(models, torch.int32)
    S, n = m.shape
    cost = torch.empty(S, dtype=torch.float32, device=Pm.device)
    assign = torch.empty((S, n), dtype=torch.int32, device=Pm.device) if want_assign else None
    ws = _workspace(_dll.roomie_optimal_workspace_bytes(S), Pm.device)
    _check(_dll.roomie_optimal_assignment(_ptr(Pm), Pm.shape[0], _ptr(m), n, S, int(num_gpus), int(max_residents),
                                          _ptr(cost), _ptr(assign), _ptr(ws), ws.numel(), _stream(stream)),
           "roomie_optimal_assignment")
    return cost, assign


def assignment_cost(Pmat, models, gpu_of, stream=None):
    """roomie_assignment_cost: average predicted drop of given deployments, float32 [S]."""
    Pm = _dev(Pmat, torch.float32)
    m, a = _dev(models, torch.int32), _dev(gpu_of, torch.int32)
    S, n = m.shape
    cost = torch.empty(S, dtype=torch.float32, device=Pm.device)
    _check(_dll.roomie_assignment_cost(_ptr(Pm), Pm.shape[0], _ptr(m), _ptr(a), n, S, _ptr(cost), _stream(stream)),
           "roomie_assignment_cost")
    return cost


def launch_count() -> int:
    return int(_dll.roomie_launch_count())


def reset_launch_count():
    _dll.roomie_reset_launch_count()


def selftest_bounded_wait(limit_ns: int = 1_000_000, stream=None) -> int:
    """roomie_selftest_bounded_wait: one CTA waits `limit_ns` for a copy nobody issues.  Returns the status
    word afterwards (ROOMIE_FLAG_WAIT_TIMEOUT = 8 must be set)."""
    word = torch.zeros(1, dtype=torch.int32, device="cuda")
    _check(_dll.roomie_selftest_bounded_wait(_ptr(word), C.c_uint64(int(limit_ns)), _stream(stream)),
           "roomie_selftest_bounded_wait")
    return int(word.item())


def profile_enable(on: bool = True):
    """roomie_profile_enable: bracket every pairwise-walk kernel launch with CUDA events."""
    _check(_dll.roomie_profile_enable(int(bool(on))), "roomie_profile_enable")


def profile_walk_ms():
    """roomie_profile_walk_ms: (summed kernel milliseconds, launches) since the last read."""
    ms, n = C.c_float(0), C.c_uint32(0)
    _check(_dll.roomie_profile_walk_ms(C.byref(ms), C.byref(n)), "roomie_profile_walk_ms")
    return float(ms.value), int(n.value)
