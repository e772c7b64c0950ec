"""Pins for the oracle's occupancy (Eq. 1) and tick timeline.

None of the expected values below come from the oracle: they are hand-derived
fixtures, an independent block-by-block SM filler, and invariants.
"""
import itertools
import os

import numpy as np
import pytest

import roomie_synth as rs

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _rows(name):
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if line:
                yield line.split()


def test_hand_derived_eq1_values(oracle):
    for row in _rows("occupancy_eq1.txt"):
        v = [float(x) for x in row]
        spec = rs.GpuSpec(*[int(x) for x in v[0:5]])
        thr, regs, smem, grid = [int(x) for x in v[5:9]]
        o = oracle.occupancy([grid], [thr], [regs], [smem], spec)
        got = (int(o.b_lim[0]), int(o.b_res[0]), int(o.limiter[0]), int(o.warps[0]))
        assert got == tuple(int(x) for x in v[9:13]), row
        assert o.occ[0] == np.float32(v[13]), row
        W = spec.threads_per_sm // 32
        assert o.occ_theo[0] == np.float32(((thr + 31) // 32) * got[0]) / np.float32(W)


def _fill_sms(grid, thr, regs, smem, spec):
    """Hand the grid's blocks to the SMs one at a time, round-robin, each SM
    keeping running totals; stop at the first block that does not fit.  Returns
    the largest number of blocks resident on one SM."""
    wb = -(-thr // 32)
    used = [[0, 0, 0, 0] for _ in range(spec.num_sms)]   # warps, regs, smem, blocks
    resident = [0] * spec.num_sms
    cap = (spec.threads_per_sm // 32, spec.regs_per_sm, spec.smem_per_sm, spec.blocks_per_sm)
    need = (wb, regs * 32 * wb, smem, 1)
    for blk in range(grid):
        sm = blk % spec.num_sms
        if any(used[sm][c] + need[c] > cap[c] for c in range(4)):
            break
        for c in range(4):
            used[sm][c] += need[c]
        resident[sm] += 1
    return max(resident), used[0]


def test_brute_force_block_filler(oracle):
    spec = rs.GpuSpec(3, 4096, 8192, 256, 6)
    cases = list(itertools.product([1, 2, 5, 7, 18, 40], [32, 33, 64, 96, 128, 256, 288],
                                   [0, 8, 16, 24, 40], [0, 1024, 3000, 8192, 9000]))
    grid, thr, regs, smem = (np.array(x, dtype=np.uint32) for x in zip(*cases))
    o = oracle.occupancy(grid, thr, regs, smem, spec)
    for k, (g, t, r, s) in enumerate(cases):
        b, used0 = _fill_sms(g, t, r, s, spec)
        assert int(o.b_res[k]) == b, (g, t, r, s)
        # SM 0 is the fullest SM; its running totals are the demand vector phi
        assert [int(o.phi[c, k]) for c in range(4)] == used0, (g, t, r, s)
        assert int(o.warps[k]) == used0[0]


def test_brute_force_real_specs(oracle):
    rng = np.random.default_rng(7)
    for spec in (rs.SPEC_CLOUD, rs.SPEC_EDGE):
        n = 60
        thr = rng.choice([32, 64, 96, 128, 256, 512, 1024], n)
        regs = rng.integers(0, 33, n) * 8
        smem = rng.integers(0, 200, n) * 1024
        grid = rng.integers(1, 6000, n)
        o = oracle.occupancy(grid, thr, regs, smem, spec)
        for k in range(n):
            b, _ = _fill_sms(int(grid[k]), int(thr[k]), int(regs[k]), int(smem[k]), spec)
            assert int(o.b_res[k]) == b


def test_invariants_and_monotonicity(oracle):
    lib = rs.make_library(2, feasible=False)
    spec = lib.spec
    o = oracle.occupancy(lib.grid_blocks, lib.block_threads, lib.regs_per_thread,
                         lib.smem_per_block, spec)
    W = spec.threads_per_sm // 32
    cap = np.array([W, spec.regs_per_sm, spec.smem_per_sm, spec.blocks_per_sm])[:, None]
    assert (o.phi <= cap).all()
    assert ((o.occ >= 0) & (o.occ <= 1)).all() and (o.b_res <= o.b_lim).all()
    assert o.n_unlaunchable == int((o.b_lim == 0).sum()) and o.n_unlaunchable > 0
    assert (o.occ[o.b_lim == 0] == 0).all()
    # more registers / shared memory / threads never raises the block count
    more_regs = oracle.occupancy(lib.grid_blocks, lib.block_threads, lib.regs_per_thread + 8,
                                 lib.smem_per_block, spec)
    more_smem = oracle.occupancy(lib.grid_blocks, lib.block_threads, lib.regs_per_thread,
                                 lib.smem_per_block + 1024, spec)
    assert (more_regs.b_lim <= o.b_lim).all() and (more_smem.b_lim <= o.b_lim).all()
    # grid large enough -> resident blocks equal Eq. 1's b
    big = oracle.occupancy(np.full_like(lib.grid_blocks, 10**6), lib.block_threads,
                           lib.regs_per_thread, lib.smem_per_block, spec)
    assert (big.b_res == big.b_lim).all() and (big.limiter < 4).all()
    assert np.array_equal(big.occ, big.occ_theo)


def test_timeline_ticks(oracle):
    # rint of a float32 product, half to even; at least one tick per kernel
    dur = np.array([0.0, 0.0004, 0.0005, 0.0015, 0.0025, 1.0, 20.1234, 1e5], dtype=np.float32)
    gap = np.array([0.0, 3.0, 0.0005, 0.0, 1.5, 0.25, 0.0, 7.0], dtype=np.float32)
    start, dt, T, st = oracle.timeline([0, 3, 8], dur, gap)
    want_dt = np.maximum(1, np.rint(dur * np.float32(1000.0)).astype(np.int64))
    want_g = np.rint(gap * np.float32(1000.0)).astype(np.int64)
    assert st == 0
    assert list(dt) == list(want_dt)
    assert list(dt[:5]) == [1, 1, 1, 2, 2]            # 0.5 -> 0 -> clamp 1; 1.5 -> 2; 2.5 -> 2
    for lo, hi in ((0, 3), (3, 8)):
        t = 0
        for k in range(lo, hi):
            assert start[k] == t
            t += int(want_dt[k]) + int(want_g[k])
    assert list(T) == [int(want_dt[:3].sum()), int(want_dt[3:].sum())]


def test_timeline_range_error(oracle):
    dur = np.full(30, 1e5, dtype=np.float32)           # 30 * 1e8 ticks > 2^31
    _, _, _, st = oracle.timeline([0, 30], dur, np.zeros(30, dtype=np.float32))
    assert st != 0
    _, _, _, st = oracle.timeline([0, 1], np.array([-1.0], dtype=np.float32),
                                  np.zeros(1, dtype=np.float32))
    assert st != 0
    for c in range(5):
        lib = rs.make_library(c)
        assert oracle.timeline(lib.offsets, lib.dur_us, lib.gap_us)[3] == 0
