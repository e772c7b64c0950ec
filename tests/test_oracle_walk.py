"""Pins for the oracle's alignment walk, alignment set, median and gamma
(Algorithm 1, Section 3.2).  Expected values come from a hand-worked example,
an independent tick-by-tick stepper, closed forms and invariants - never from
the oracle itself."""
import os
from fractions import Fraction
from types import SimpleNamespace

import numpy as np
import pytest

import roomie_synth as rs

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
TIMELINE, LOCKSTEP = 0, 1


def make_lib(profiles, spec=rs.SPEC_CLOUD):
    """profiles: list of lists of (threads, regs, smem, grid, dur_us, gap_us)."""
    rows = [k for p in profiles for k in p]
    off = np.cumsum([0] + [len(p) for p in profiles]).astype(np.uint32)
    col = lambda i, dt: np.array([r[i] for r in rows], dtype=dt)
    return SimpleNamespace(spec=spec, offsets=off, block_threads=col(0, np.uint32),
                           regs_per_thread=col(1, np.uint32), smem_per_block=col(2, np.uint32),
                           grid_blocks=col(3, np.uint32), dur_us=col(4, np.float32),
                           gap_us=col(5, np.float32))


def read_example():
    prof = {"X": [], "Y": []}
    res = {}
    with open(os.path.join(GOLDEN, "worked_example.txt")) as f:
        for line in f:
            t = line.split("#")[0].split()
            if not t:
                continue
            if t[0] in prof:
                prof[t[0]].append(tuple(float(x) for x in t[1:]))
            else:
                res[t[0]] = [float(x) for x in t[1:]]
    return prof, res


def test_worked_example(oracle):
    prof, res = read_example()
    X = [(int(a), int(b), int(c), int(d), e, g) for a, b, c, d, e, g in prof["X"]]
    Y = [(int(a), int(b), int(c), int(d), e, g) for a, b, c, d, e, g in prof["Y"]]
    ol = oracle.library_build(make_lib([X, Y]))
    for name, mode in (("TIMELINE", TIMELINE), ("LOCKSTEP", LOCKSTEP)):
        ev, dx, dy, V, pxy, pyx = res[name]
        d = oracle.pair(ol, 0, 1, mode=mode, n_align=1, start_filter=0)
        assert d.kept == 1 and d.evals == int(ev)
        assert d.delta_i[0] == pytest.approx(dx * 1000, rel=1e-12)      # ticks are ns
        assert d.delta_j[0] == pytest.approx(dy * 1000, rel=1e-12)
        assert int(d.V[0]) == int(V * 1000)
        assert d.P_ab == pytest.approx(pxy, rel=1e-12)
        assert d.P_ba == pytest.approx(pyx, rel=1e-12)
        # the mirrored call returns the mirrored result
        m = oracle.pair(ol, 1, 0, mode=mode, n_align=1, start_filter=0)
        assert (m.P_ab, m.P_ba) == (d.P_ba, d.P_ab)


# ---------------------------------------------------------------------------
# independent tick-by-tick stepper: no two-pointer logic at all
# ---------------------------------------------------------------------------
def _active(start, dt, base, s, t):
    """index of the kernel (>= s) running at re-based time t, or None (gap / finished)."""
    for k in range(s, len(start)):
        a0 = start[k] - base
        if a0 <= t < a0 + dt[k]:
            return k
    return None


def stepper(ol, a, b, si, sj):
    oa, ob = int(ol.offsets[a]), int(ol.offsets[b])
    qa, qb = int(ol.offsets[a + 1]) - oa, int(ol.offsets[b + 1]) - ob
    sa, da = ol.start[oa:oa + qa].astype(int), ol.dt[oa:oa + qa].astype(int)
    sb, db = ol.start[ob:ob + qb].astype(int), ol.dt[ob:ob + qb].astype(int)
    pa, pb = ol.occ.phi[:, oa:oa + qa].astype(int), ol.occ.phi[:, ob:ob + qb].astype(int)
    cap = [ol.spec.threads_per_sm // 32, ol.spec.regs_per_sm, ol.spec.smem_per_sm, ol.spec.blocks_per_sm]
    end = min(sa[-1] + da[-1] - sa[si], sb[-1] + db[-1] - sb[sj])   # one model runs out
    di = dj = Fraction(0)
    V = 0
    for t in range(end):
        ka, kb = _active(sa, da, sa[si], si, t), _active(sb, db, sb[sj], sj, t)
        if ka is None or kb is None:
            continue
        if pa[0, ka] == 0 or pb[0, kb] == 0:
            continue
        if any(pa[c, ka] + pb[c, kb] > cap[c] for c in range(4)):
            di += Fraction(int(pa[0, ka]), int(pa[0, ka] + pb[0, kb]))
            dj += Fraction(int(pb[0, kb]), int(pa[0, ka] + pb[0, kb]))
            V += 1
    return di, dj, V


def tiny_lib(seed, n_prof=3, qmax=7, spec=rs.SPEC_CLOUD):
    rng = np.random.default_rng(seed)
    profs = []
    for _ in range(n_prof):
        q = int(rng.integers(1, qmax + 1))
        p = []
        for _ in range(q):
            p.append((int(rng.choice([64, 128, 256, 1024])), int(rng.choice([32, 64, 128, 200])),
                      int(rng.choice([0, 16384, 65536, 98304])), int(rng.choice([50, 400, 10000])),
                      float(rng.integers(1, 20)) / 1000.0, float(rng.integers(0, 6)) / 1000.0))
        profs.append(p)
    return make_lib(profs, spec)


@pytest.mark.parametrize("seed", range(6))
def test_walk_against_tick_stepper(oracle, seed):
    lib = tiny_lib(seed, spec=rs.SPEC_CLOUD if seed % 2 == 0 else rs.SPEC_EDGE)
    ol = oracle.library_build(lib)
    P = ol.num_profiles
    hits = 0
    for a in range(P):
        for b in range(P):
            d = oracle.pair(ol, a, b, mode=TIMELINE, n_align=0, start_filter=0)
            qa = int(ol.offsets[a + 1] - ol.offsets[a])
            qb = int(ol.offsets[b + 1] - ol.offsets[b])
            assert d.kept == qa * qb
            for c in range(d.kept):
                di, dj, V = stepper(ol, a, b, int(d.s_i[c]), int(d.s_j[c]))
                assert d.delta_i[c] == pytest.approx(float(di), rel=1e-12, abs=1e-12)
                assert d.delta_j[c] == pytest.approx(float(dj), rel=1e-12, abs=1e-12)
                assert int(d.V[c]) == V
                assert d.delta_i[c] + d.delta_j[c] == pytest.approx(V, rel=1e-12)
                hits += V > 0
    assert hits > 0


def test_eval_count_is_walk_length(oracle):
    # hand-checkable: A = 3 kernels of 4 ticks, B = 2 kernels of 6 ticks, no gaps.
    # pairings: (0,0) (1,0) (1,1) (2,1)  then both end at 12 -> 4 scored pairings
    k = (256, 64, 0, 10000)
    lib = make_lib([[k + (0.004, 0.0)] * 3, [k + (0.006, 0.0)] * 2])
    ol = oracle.library_build(lib)
    d = oracle.pair(ol, 0, 1, mode=TIMELINE)
    assert d.evals == 4
    assert int(d.V[0]) == 12 and d.delta_i[0] == pytest.approx(6.0)
    # a tie advances both models at once: 3 x 4 ticks vs 3 x 4 ticks -> 3 pairings
    lib = make_lib([[k + (0.004, 0.0)] * 3, [k + (0.004, 0.0)] * 3])
    assert oracle.pair(oracle.library_build(lib), 0, 1, mode=TIMELINE).evals == 3


def test_no_interference_gives_exact_zero(oracle):
    small = (64, 16, 0, 100)             # one block per SM: (2 warps, 1024 regs, 0, 1 block)
    lib = make_lib([[small + (0.01, 0.001)] * 5, [small + (0.007, 0.002)] * 4])
    ol = oracle.library_build(lib)
    for mode in (TIMELINE, LOCKSTEP):
        d = oracle.pair(ol, 0, 1, mode=mode, n_align=0)
        assert d.P_ab == 0.0 and d.P_ba == 0.0 and not d.delta_i.any() and not d.V.any()
        assert oracle.pair(ol, 0, 1, mode=mode, n_align=4, start_filter=1).kept == 0


def test_unlaunchable_kernel_never_charged(oracle):
    heavy = (256, 64, 0, 10000)
    dead = (1024, 72, 0, 10000)          # registers of one block exceed the SM: b = 0
    lib = make_lib([[heavy + (0.01, 0.0), dead + (0.01, 0.0), heavy + (0.01, 0.0)],
                    [heavy + (0.03, 0.0)]])
    ol = oracle.library_build(lib)
    assert ol.occ.n_unlaunchable == 1
    d = oracle.pair(ol, 0, 1, mode=TIMELINE)
    assert int(d.V[0]) == 20 and d.delta_i[0] == pytest.approx(10.0)


def test_time_scaling_leaves_slowdown_unchanged(oracle):
    lib = rs.make_library(1, num_profiles=4)
    ol = oracle.library_build(lib)
    base, _ = oracle.pair_matrix(ol, n_align=4, start_filter=1)
    # scale the integer timelines by 3 (exact in ticks)
    ol3 = oracle.OracleLibrary(ol.spec, ol.offsets, ol.start * 3, ol.dt * 3, ol.T * np.uint64(3), ol.occ, 0)
    scaled, _ = oracle.pair_matrix(ol3, n_align=4, start_filter=1)
    np.testing.assert_allclose(scaled, base, rtol=1e-12)
    assert base.max() > 0


def test_slowdown_bounded_by_gamma(oracle):
    lib = rs.make_library(1, num_profiles=6)
    ol = oracle.library_build(lib)
    q = lib.q().astype(float)
    gamma = np.maximum(q[:, None] / q[None, :], 1.0)
    for kw in (dict(n_align=1), dict(n_align=8, start_filter=1)):
        Pm, _ = oracle.pair_matrix(ol, **kw)
        assert (Pm <= gamma + 1e-12).all() and (Pm >= 0).all()


def test_lockstep_equals_timeline_on_equal_durations(oracle):
    rng = np.random.default_rng(3)
    profs = []
    for q in (9, 14, 5):
        profs.append([(int(rng.choice([128, 256, 1024])), int(rng.choice([32, 64, 128])),
                       int(rng.choice([0, 49152, 98304])), 10000, 0.025, 0.0) for _ in range(q)])
    ol = oracle.library_build(make_lib(profs))
    for a in range(3):
        for b in range(3):
            t = oracle.pair(ol, a, b, mode=TIMELINE, n_align=0)
            l = oracle.pair(ol, a, b, mode=LOCKSTEP, n_align=0)
            assert np.array_equal(t.delta_i, l.delta_i) and np.array_equal(t.delta_j, l.delta_j)
            assert t.P_ab == l.P_ab and t.P_ba == l.P_ba and t.evals == l.evals
            assert t.delta_i.max() > 0


def test_lockstep_is_algorithm_1_as_printed(oracle):
    """Plain transcription check on random data: delta = sum of d_ki * o_ki/(o_ki+o_kj)
    over k_i = s_i+t, k_j = s_j+t whenever the combined demand exceeds the SM."""
    lib = rs.make_library(0, feasible=False)
    ol = oracle.library_build(lib)
    cap = np.array([64, 65536, 167936, 32])
    d = oracle.pair(ol, 0, 1, mode=LOCKSTEP, n_align=0)
    assert d.kept == 2500
    o = ol.occ.occ.astype(np.float64)
    for c in range(0, d.kept, 97):
        si, sj = int(d.s_i[c]), int(d.s_j[c])
        tot = 0.0
        for t in range(min(50 - si, 50 - sj)):
            ka, kb = si + t, 50 + sj + t
            if o[ka] > 0 and o[kb] > 0 and (ol.occ.phi[:, ka].astype(int) + ol.occ.phi[:, kb] > cap).any():
                tot += float(ol.dt[ka]) * o[ka] / (o[ka] + o[kb])
        assert d.delta_i[c] == pytest.approx(tot, rel=1e-12)


def test_alignment_grid_median_gamma_closed_form(oracle):
    # two identical profiles of q identical self-interfering kernels, w = 1/2:
    # delta(s_i, s_j) = D/2 * min(q - s_i, q - s_j)
    k = (256, 64, 0, 10000, 0.05, 0.0)
    ol = oracle.library_build(make_lib([[k] * 8, [k] * 8]))
    D = 50.0
    d = oracle.pair(ol, 0, 1, n_align=2)
    assert sorted(zip(d.s_i, d.s_j)) == [(0, 0), (0, 4), (4, 0), (4, 4)]
    assert sorted(d.delta_i) == [2 * D, 2 * D, 2 * D, 4 * D]
    assert d.P_ab == pytest.approx(0.25) and d.P_ba == pytest.approx(0.25)   # median 2D over T = 8D
    assert oracle.pair(ol, 0, 1, n_align=1).P_ab == pytest.approx(0.5)
    # even count -> mean of the two middle values: A = 0 on q = 2 gives deltas {2,1,1,1} * D/2
    ol2 = oracle.library_build(make_lib([[k] * 2, [k] * 2]))
    assert oracle.pair(ol2, 0, 1, n_align=0).P_ab == pytest.approx((D / 2) / (2 * D))
    # odd count: q = (3, 1): deltas for s_i = 0,1,2 are all D/2 -> median D/2; gamma = 3 and 1
    ol3 = oracle.library_build(make_lib([[k] * 3, [k]]))
    d3 = oracle.pair(ol3, 0, 1, n_align=0)
    assert d3.kept == 3
    assert d3.P_ab == pytest.approx(3.0 * (D / 2) / (3 * D))
    assert d3.P_ba == pytest.approx(1.0 * (D / 2) / D)
    # q_i = 2 q_j -> gamma_ij = 2, gamma_ji = 1
    ol4 = oracle.library_build(make_lib([[k] * 8, [k] * 4]))
    d4 = oracle.pair(ol4, 0, 1, n_align=1)
    assert d4.P_ab == pytest.approx(2.0 * (4 * D / 2) / (8 * D))
    assert d4.P_ba == pytest.approx(1.0 * (4 * D / 2) / (4 * D))


def test_alignment_count_matches_printed_scenario_count(oracle):
    # Introduction: ten models of fifty kernels give 112 500 pairwise alignment scenarios
    k = (256, 64, 0, 10000, 0.001, 0.0)
    ol = oracle.library_build(make_lib([[k] * 50] * 10))
    total = 0
    for a in range(10):
        for b in range(a + 1, 10):
            total += oracle.pair(ol, a, b, n_align=0, cap_align=1).kept
    assert total == 112500


def test_start_grid_and_filter(oracle):
    lib = rs.make_library(0)
    ol = oracle.library_build(lib)
    q = lib.q()
    d = oracle.pair(ol, 0, 1, n_align=8, start_filter=0)
    want = [(t * int(q[0]) // 8, u * int(q[1]) // 8) for t in range(8) for u in range(8)]
    assert list(zip(d.s_i, d.s_j)) == want
    f = oracle.pair(ol, 0, 1, n_align=8, start_filter=1)
    cap = np.array([64, 65536, 167936, 32])
    keep = [(s, t) for s, t in want
            if (ol.occ.phi[:, ol.offsets[0] + s].astype(int) + ol.occ.phi[:, ol.offsets[1] + t] > cap).any()]
    assert list(zip(f.s_i, f.s_j)) == keep and 0 < len(keep) < 64
    # grid on a short profile: duplicates removed
    k = (256, 64, 0, 10000, 0.001, 0.0)
    ol2 = oracle.library_build(make_lib([[k] * 3, [k] * 20]))
    g = oracle.pair(ol2, 0, 1, n_align=8)
    assert sorted(set(g.s_i)) == [0, 1, 2] and g.kept == 3 * 8


def test_matrix_equals_pairs_and_is_thread_independent(oracle):
    lib = rs.make_library(1, num_profiles=5)
    ol = oracle.library_build(lib)
    Pm, ev = oracle.pair_matrix(ol, n_align=8, start_filter=1, num_threads=1)
    Pm4, ev4 = oracle.pair_matrix(ol, n_align=8, start_filter=1, num_threads=4)
    assert np.array_equal(Pm, Pm4) and ev == ev4
    tot = 0
    for a in range(5):
        for b in range(a, 5):
            d = oracle.pair(ol, a, b, n_align=8, start_filter=1)
            assert Pm[a, b] == d.P_ab
            if a != b:
                assert Pm[b, a] == d.P_ba
            tot += d.evals
    assert tot == ev
    # a range of pair indices fills only those entries
    part, _ = oracle.pair_matrix(ol, n_align=8, start_filter=1, pair_begin=5, pair_end=9)
    mask = np.zeros((5, 5), bool)
    mask[1, 1:5] = True
    mask[1:5, 1] = True
    assert np.array_equal(part[mask], Pm[mask]) and not part[~mask].any()
