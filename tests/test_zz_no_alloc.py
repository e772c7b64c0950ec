"""The entry point for callers that cannot allocate device memory.

`roomie_pair_interference_static` keeps its scratch in an array that is part of the library
image, so a controller that was handed device pointers but owns no allocator (or must not
stall the device with a cudaMalloc) can still score a pair.  This file is collected last on
purpose: if it fails, a run that stops at the first failure has already run everything else.

Checked through the C ABI against the ordinary entry point, on two calls in a row - the
second call finds the first one's leftovers in the shared array and must not be disturbed
by them - and the size limit must be reported as an error, not exceeded.
"""
import numpy as np
import pytest

import roomie_synth as rs

pytestmark = pytest.mark.gpu

RTOL = 1e-5


def same(got, want):
    for k in ("n_kept", "s_i", "s_j", "evals_c", "V", "evals"):
        assert np.array_equal(got[k].cpu().numpy(), want[k].cpu().numpy()), k
    for k in ("delta_i", "delta_j", "P2"):
        g, w = got[k].cpu().numpy().astype(np.float64), want[k].cpu().numpy().astype(np.float64)
        assert np.all(np.abs(g - w) <= RTOL * np.abs(w)), k


def test_static_scratch_entry_point_matches_workspace_entry_point():
    import torch
    if not torch.cuda.is_available():
        pytest.fail("gpu-marked test run without a CUDA device")
    import paper_2607_16784_b200 as rm

    lib = rs.make_library(2)                       # 32 profiles of 200-2000 kernels
    gl = rm.library_build(lib.grid_blocks, lib.block_threads, lib.regs_per_thread, lib.smem_per_block,
                          lib.dur_us, lib.gap_us, lib.offsets, lib.spec)
    calls = [(3, 17, dict(mode=0, n_align=8, start_filter=1)),     # many walks, several tiles each
             (5, 5, dict(mode=0, n_align=1, start_filter=0)),      # one walk: far less scratch than the call before
             (30, 2, dict(mode=1, n_align=4, start_filter=0)),
             (7, 21, dict(mode=3, n_align=4, start_filter=1)),     # Section 3.2 simulator: the scratch also holds its walk sort
             (9, 4, dict(mode=2, n_align=2, start_filter=0))]
    # warm both entry points once, so that what is measured below is the call and not the first-use set-up of
    # the runtime (module loading) or of torch's caching allocator
    rm.pair_interference_static(gl, 0, 1, detail_capacity=64, **calls[0][2])
    rm.pair_interference(gl, 0, 1, detail_capacity=64, **calls[0][2])
    for _, _, kw in calls:                          # every kernel of every mode loaded once (the driver loads lazily)
        rm.pair_interference_static(gl, 1, 0, **kw)
    torch.cuda.synchronize()
    # several calls in a row on the shared array, each compared with the workspace variant
    for a, b, kw in calls:
        out2 = torch.zeros(2, dtype=torch.float32, device="cuda")
        torch.cuda.synchronize()
        held, free = torch.cuda.memory_allocated(), torch.cuda.mem_get_info()[0]
        rm.pair_interference_static(gl, a, b, out2=out2, **kw)     # outputs given: the call itself gets no memory
        torch.cuda.synchronize()
        assert torch.cuda.memory_allocated() == held               # nothing from torch's allocator ...
        assert torch.cuda.mem_get_info()[0] >= free                # ... and nothing from the driver
        got = rm.pair_interference_static(gl, a, b, detail_capacity=64, **kw)
        want = rm.pair_interference(gl, a, b, detail_capacity=64, **kw)
        same(got, want)
        assert torch.equal(out2, got["P2"])
        assert int(want["n_kept"].item()) > 0 and float(want["P2"].max()) > 0    # (with priority the first model loses nothing)
    # Algorithm 1 as printed over the full alignment set, with per-alignment detail (the variant that does need
    # scratch): two short profiles so that the q_a x q_b alignments fit the array
    small = rs.make_library(0)
    gs = rm.library_build(small.grid_blocks, small.block_threads, small.regs_per_thread, small.smem_per_block,
                          small.dur_us, small.gap_us, small.offsets, small.spec)
    got = rm.pair_interference_static(gs, 0, 1, mode=1, n_align=0, detail_capacity=2500)
    want = rm.pair_interference(gs, 0, 1, mode=1, n_align=0, detail_capacity=2500)
    same(got, want)
    assert int(want["n_kept"].item()) == 2500
    # the same call twice in a row gives the same bits
    a, b, kw = calls[0]
    first = rm.pair_interference_static(gl, a, b, detail_capacity=64, **kw)
    second = rm.pair_interference_static(gl, a, b, detail_capacity=64, **kw)
    for k in first:
        assert torch.equal(first[k], second[k]), k
    assert gl.status_flags() == 0


def test_static_scratch_limit_is_an_error():
    import torch
    if not torch.cuda.is_available():
        pytest.fail("gpu-marked test run without a CUDA device")
    import paper_2607_16784_b200 as rm

    lib = rs.make_library(3, num_profiles=16)      # profiles of up to ~4600 kernels
    gl = rm.library_build(lib.grid_blocks, lib.block_threads, lib.regs_per_thread, lib.smem_per_block,
                          lib.dur_us, lib.gap_us, lib.offsets, lib.spec)
    q = lib.q()
    a, b = (int(x) for x in np.argsort(q)[-2:])
    assert q[a] + q[b] > 8192
    # 64 x 64 alignments of two very long profiles need more scratch than the built-in array holds
    with pytest.raises(rm.RoomieError, match="workspace too small"):
        rm.pair_interference_static(gl, a, b, mode=0, n_align=64, start_filter=0)
    # ... while the workspace variant takes the same request, and a smaller one still fits the array
    big = rm.pair_interference(gl, a, b, mode=0, n_align=64, start_filter=0)
    ok = rm.pair_interference_static(gl, a, b, mode=0, n_align=8, start_filter=0)
    assert float(big["P2"][0]) > 0 and float(ok["P2"][0]) > 0
