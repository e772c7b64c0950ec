"""Pins for the oracle's Section 3.2 simulator (adjusted occupancy, two-phase execution, partition policies):
the paper's two-phase formula on hand cases, closed forms per policy and per rate, and an independent tick-by-tick
integrator (exact rationals, no event logic) at every rate b~/b the policies produce."""
from fractions import Fraction

import numpy as np
import pytest

import roomie_synth as rs
from test_oracle_walk import make_lib

EQUAL, PRIORITY, FCFS = 2, 3, 4
# (threads, regs, smem, grid): register-limited, 4 blocks of 8 warps fill the cloud SM's 65536 registers
HEAVY = (256, 64, 0, 10000)
# 2 blocks, half the registers: two of them fit side by side
HALF = (256, 64, 0, 200)


def sim(oracle, profs, mode, a=0, b=1, **kw):
    ol = oracle.library_build(make_lib(profs))
    return oracle.pair(ol, a, b, mode=mode, **kw), ol


def test_two_phase_formula_of_the_paper(oracle):
    # a: d = 10, b: d = 30 (us), both heavy, EQUAL: each runs with 2 of its 4 blocks -> rate 1/2.
    # a ends at 20 (delay 10); b has done 10 of its 30, the rest runs alone: ends at 40 (delay 10).
    # Paper: d~e_b = 30 * 2 = 60, Delta = 20, d~_b = 20 + (60 - 20) * 1/2 = 40.
    d, _ = sim(oracle, [[HEAVY + (10.0, 0.0)], [HEAVY + (30.0, 0.0)]], EQUAL)
    assert d.delta_i[0] == pytest.approx(10000.0) and d.delta_j[0] == pytest.approx(10000.0)
    assert d.P_ab == pytest.approx(10.0 / 10.0) and d.P_ba == pytest.approx(10.0 / 30.0)


def test_policies_on_identical_kernels(oracle):
    profs = [[HEAVY + (10.0, 0.0)], [HEAVY + (10.0, 0.0)]]
    # EQUAL: both at half rate for 20 us -> each loses 10
    d, _ = sim(oracle, profs, EQUAL)
    assert (d.delta_i[0], d.delta_j[0]) == (pytest.approx(10000.0), pytest.approx(10000.0))
    # PRIORITY / FCFS (tie -> model i): i keeps all its blocks, nothing is left for j, which waits 10 us;
    # the run ends when i is done, so j's wait is its delay
    for mode in (PRIORITY, FCFS):
        d, _ = sim(oracle, profs, mode)
        assert d.delta_i[0] == 0.0 and d.delta_j[0] == pytest.approx(10000.0)
    # mirrored call: priority moves with the first model of the ordered pair
    d, _ = sim(oracle, profs, PRIORITY, a=1, b=0)
    assert d.delta_i[0] == 0.0 and d.delta_j[0] == pytest.approx(10000.0)


def test_partial_remainder_under_priority(oracle):
    # i: HALF (2 blocks, 32768 regs), j: HEAVY (4 blocks): combined 6 blocks' registers exceed the SM;
    # j gets floor((65536 - 32768) / 16384) = 2 of its 4 blocks -> rate 1/2 while i runs (10 us), then 25 us alone
    d, _ = sim(oracle, [[HALF + (10.0, 0.0)], [HEAVY + (30.0, 0.0)]], PRIORITY)
    assert d.delta_i[0] == 0.0 and d.delta_j[0] == pytest.approx(5000.0)
    # EQUAL: i fits in half an SM untouched (2 blocks), j is cut to 2 of 4 -> same numbers
    d, _ = sim(oracle, [[HALF + (10.0, 0.0)], [HEAVY + (30.0, 0.0)]], EQUAL)
    assert d.delta_i[0] == 0.0 and d.delta_j[0] == pytest.approx(5000.0)


def test_fcfs_follows_start_times(oracle):
    # i: a light kernel (no interference) for 4 us, then HEAVY; j: HEAVY for 20 us from t = 0.
    # j's kernel started first, so under FCFS it keeps the SM and i's second kernel waits until t = 20;
    # the run ends there (j is done): i lost 16 us, j nothing.  Under PRIORITY i pre-empts: j loses 10.
    light = (64, 0, 0, 100)                  # no register demand: fits beside anything
    profs = [[light + (4.0, 0.0), HEAVY + (10.0, 0.0)], [HEAVY + (20.0, 0.0)]]
    d, _ = sim(oracle, profs, FCFS)
    assert d.delta_i[0] == pytest.approx(16000.0) and d.delta_j[0] == 0.0
    d, _ = sim(oracle, profs, PRIORITY)
    assert d.delta_i[0] == 0.0 and d.delta_j[0] == pytest.approx(10000.0)


def test_no_interference_and_gaps(oracle):
    light = (64, 0, 0, 100)
    for mode in (EQUAL, PRIORITY, FCFS):
        d, _ = sim(oracle, [[light + (5.0, 1.0)] * 4, [light + (3.0, 2.0)] * 5], mode, n_align=0)
        assert not d.delta_i.any() and not d.delta_j.any() and d.P_ab == 0.0
    # a gap of model j shields model i: j = HEAVY 10 us, gap 10 us, HEAVY 10 us; i = HEAVY 20 us starting with j.
    # EQUAL: 0..20 both at 1/2 -> j's first kernel ends at 20 (i has 10 left), gap 20..30: i finishes alone at 30
    d, _ = sim(oracle, [[HEAVY + (20.0, 0.0)], [HEAVY + (10.0, 10.0), HEAVY + (10.0, 0.0)]], EQUAL)
    assert d.delta_i[0] == pytest.approx(10000.0) and d.delta_j[0] == pytest.approx(10000.0)


# ---------------------------------------------------------------------------------------
# independent tick-by-tick integrator.  It knows nothing of events: every tick it looks at the two active
# kernels, decides how many blocks each runs with, and moves each forward by one tick's worth of work (exact
# rationals).  A kernel is complete at the first tick boundary at which its work is used up; its successor (or
# the gap before it) starts there.  That is the simulator's definition, whatever b~/b is, so no restriction on
# durations or rates is needed.
# ---------------------------------------------------------------------------------------
def stepper(ol, a, b, si, sj, policy):
    cap = [ol.spec.threads_per_sm // 32, ol.spec.regs_per_sm, ol.spec.smem_per_sm, ol.spec.blocks_per_sm]

    def load(m, s):
        o = int(ol.offsets[m]); q = int(ol.offsets[m + 1]) - o
        return dict(st=ol.start[o:o + q].astype(int), dt=ol.dt[o:o + q].astype(int),
                    phi=ol.occ.phi[:, o:o + q].astype(int), k=s, q=q, work=Fraction(int(ol.dt[o + s])),
                    gap=0, began=0, lost=Fraction(0))
    M = [load(a, si), load(b, sj)]
    t = 0
    rates = set()
    while M[0]["k"] < M[0]["q"] and M[1]["k"] < M[1]["q"]:
        rate = [Fraction(1), Fraction(1)]
        if M[0]["gap"] == 0 and M[1]["gap"] == 0:
            ph = [m["phi"][:, m["k"]] for m in M]
            if ph[0][0] > 0 and ph[1][0] > 0 and any(ph[0][c] + ph[1][c] > cap[c] for c in range(4)):
                nb = [int(p[3]) for p in ph]
                per = [[int(p[c]) // int(p[3]) for c in range(3)] + [1] for p in ph]

                def fit(m, avail):
                    return min([nb[m]] + [avail[c] // per[m][c] for c in range(4) if per[m][c] > 0])
                if policy == EQUAL:
                    bt = [fit(m, [x // 2 for x in cap]) for m in range(2)]
                    if bt == [0, 0]:
                        bt = [nb[0], 0] if M[0]["began"] <= M[1]["began"] else [0, nb[1]]
                    elif bt[0] == 0:
                        bt[1] = nb[1]
                    elif bt[1] == 0:
                        bt[0] = nb[0]
                else:
                    first = 0 if (policy == PRIORITY or M[0]["began"] <= M[1]["began"]) else 1
                    other = 1 - first
                    left = [cap[c] - int(ph[first][c]) for c in range(4)]
                    bt = [0, 0]
                    bt[first] = nb[first]
                    bt[other] = fit(other, left)
                rate = [Fraction(bt[m], nb[m]) for m in range(2)]
                rates.update(rate)
        t += 1
        for i, m in enumerate(M):
            if m["gap"] > 0:
                m["gap"] -= 1
                if m["gap"] == 0:
                    m["began"] = t
                continue
            m["lost"] += 1 - rate[i]
            m["work"] -= rate[i]
            if m["work"] <= 0:
                done = m["k"]
                m["k"] += 1
                if m["k"] < m["q"]:
                    m["gap"] = int(m["st"][m["k"]] - (m["st"][done] + m["dt"][done]))
                    m["work"] = Fraction(int(m["dt"][m["k"]]))
                    if m["gap"] == 0:
                        m["began"] = t
    return M[0]["lost"], M[1]["lost"], rates


@pytest.mark.parametrize("seed", range(4))
def test_against_unit_step_integrator(oracle, seed):
    rng = np.random.default_rng(seed)
    kinds = [HEAVY, HALF, (64, 0, 0, 100), (128, 0, 81920, 10000)]      # rates stay in {0, 1/2, 1}
    profs = []
    for _ in range(2):
        q = int(rng.integers(2, 7))
        profs.append([kinds[int(rng.integers(0, 4))] + (1.024 * int(rng.integers(1, 5)),
                                                        1.024 * int(rng.integers(0, 3))) for _ in range(q)])
    ol = oracle.library_build(make_lib(profs))
    hits = 0
    for policy in (EQUAL, PRIORITY, FCFS):
        d = oracle.pair(ol, 0, 1, mode=policy, n_align=0)
        for c in range(d.kept):
            li, lj, _ = stepper(ol, 0, 1, int(d.s_i[c]), int(d.s_j[c]), policy)
            assert d.delta_i[c] == pytest.approx(float(li), abs=1e-9), (policy, c)
            assert d.delta_j[c] == pytest.approx(float(lj), abs=1e-9), (policy, c)
            hits += li > 0 or lj > 0
    assert hits > 0


# kernel kinds on the cloud SM (65536 registers, 64 warps) whose partitions give every rate of the common case:
#   HEAVY  4 blocks x 16384 registers      THREE  the same kernel, 3 blocks resident (grid of 324 on 108 SMs)
#   HALF   2 such blocks                   ONE    1 such block
#   TRIO   3 blocks x 20480 registers (256 threads x 80 registers)
# PRIORITY / FCFS: beside HALF, HEAVY keeps 2 of 4 (1/2) and TRIO 1 of 3 (1/3); beside ONE, HEAVY keeps 3 of 4
# (3/4) and TRIO 2 of 3 (2/3); beside THREE, HEAVY keeps 1 of 4 (1/4), TRIO none (it waits).
# EQUAL (32768 registers each): HEAVY 2 of 4, TRIO 1 of 3, THREE 2 of 3, HALF and ONE untouched.
THREE = (256, 64, 0, 324)
ONE = (256, 64, 0, 100)
TRIO = (256, 80, 0, 10000)
LIGHT = (64, 0, 0, 100)
SMEM5 = (128, 0, 81920, 10000)            # 2 blocks by shared memory; two of them never fit together


def test_general_rates_hand_cases(oracle):
    """One kernel against one kernel, durations in whole ticks: d_i = 12 ticks, d_j = 36 ticks, model i first."""
    t = 0.001                                                       # one tick in microseconds

    def run(ki, kj, policy, di=12, dj=36):
        d, _ = sim(oracle, [[ki + (di * t, 0.0)], [kj + (dj * t, 0.0)]], policy)
        return d.delta_i[0], d.delta_j[0]
    # PRIORITY: i untouched for its 12 ticks; j runs at rate r meanwhile and loses 12 (1 - r)
    assert run(ONE, HEAVY, PRIORITY) == (0.0, pytest.approx(3.0))       # r = 3/4
    assert run(ONE, TRIO, PRIORITY) == (0.0, pytest.approx(4.0))        # r = 2/3
    assert run(HALF, TRIO, PRIORITY) == (0.0, pytest.approx(8.0))       # r = 1/3
    assert run(THREE, HEAVY, PRIORITY) == (0.0, pytest.approx(9.0))     # r = 1/4
    assert run(THREE, TRIO, PRIORITY) == (0.0, pytest.approx(12.0))     # r = 0: j waits for all 12 ticks
    # EQUAL: THREE keeps 2 of 3 blocks (12 ticks of work take 18), HEAVY 2 of 4 meanwhile (loses 18 / 2)
    assert run(THREE, HEAVY, EQUAL) == (pytest.approx(6.0), pytest.approx(9.0))
    # a duration that the rate does not divide: 10 ticks of work at 3/4 take ceil(40 / 3) = 14 whole ticks;
    # j (priority to i = ONE with 20 ticks) runs 14 ticks at 3/4 and loses 14 / 4
    assert run(ONE, HEAVY, PRIORITY, di=20, dj=10) == (0.0, pytest.approx(3.5))


def _random_general_profiles(seed):
    rng = np.random.default_rng(100 + seed)
    kinds = [HEAVY, HALF, THREE, ONE, TRIO, LIGHT, SMEM5]
    t = 0.001
    profs = []
    for _ in range(2):
        q = int(rng.integers(2, 8))
        profs.append([kinds[int(rng.integers(0, len(kinds)))] +
                      (t * int(rng.integers(1, 90)), t * int(rng.integers(0, 3)) * int(rng.integers(0, 25)))
                      for _ in range(q)])
    return profs


@pytest.mark.parametrize("seed", range(8))
def test_general_rates_against_tick_integrator(oracle, seed):
    """Random short profiles of the kinds above with arbitrary whole-tick durations and gaps, every alignment,
    every policy, against the tick-by-tick integrator."""
    ol = oracle.library_build(make_lib(_random_general_profiles(seed)))
    for policy in (EQUAL, PRIORITY, FCFS):
        for a, b in ((0, 1), (1, 0), (0, 0)):
            d = oracle.pair(ol, a, b, mode=policy, n_align=0)
            for c in range(d.kept):
                li, lj, _ = stepper(ol, a, b, int(d.s_i[c]), int(d.s_j[c]), policy)
                assert d.delta_i[c] == pytest.approx(float(li), rel=1e-12, abs=1e-12), (policy, a, b, c)
                assert d.delta_j[c] == pytest.approx(float(lj), rel=1e-12, abs=1e-12), (policy, a, b, c)


def test_general_rate_cases_cover_every_rate(oracle):
    """The random cases above are only a pin at general rates if those rates occur in them."""
    seen = set()
    for seed in range(8):
        ol = oracle.library_build(make_lib(_random_general_profiles(seed)))
        for policy in (EQUAL, PRIORITY, FCFS):
            for a, b in ((0, 1), (1, 0)):
                for si, sj in ((0, 0), (1, 0), (0, 1), (1, 1)):
                    seen |= stepper(ol, a, b, si, sj, policy)[2]
    want = {Fraction(0), Fraction(1, 4), Fraction(1, 3), Fraction(1, 2), Fraction(2, 3), Fraction(3, 4), Fraction(1)}
    assert want <= seen, sorted(want - seen)


def test_detailed_is_at_least_as_pessimistic_as_waiting_never(oracle):
    """Sanity on a real mix: delays are non-negative and bounded by the time the other model runs."""
    lib = rs.make_library(1, num_profiles=4)
    ol = oracle.library_build(lib)
    for mode in (EQUAL, PRIORITY, FCFS):
        Pm, _ = oracle.pair_matrix(ol, mode=mode, n_align=4, start_filter=1)
        assert (Pm >= 0).all() and Pm.max() > 0
