#!/usr/bin/env python
"""Benchmark of the Roomie interference-model hot path on B200.

One step = one pass of the whole path over one batch of synthetic input:
  occupancy of every kernel (Eq. 1) -> library build (tick timelines, walk records) -> full
  pairwise slowdown matrix (Algorithm 1 lines 6-20) -> batched multi-model estimate of the
  cluster's what-if sets -> placement of an arrival stream (Algorithm 2).

Default workload: the large all-pairs configuration (512 profiles of 1 000-5 000 kernels, all
131 328 unordered pairs incl. the diagonal, both directions, base alignment setting) plus the
online-placement cluster shape (64 GPUs, 10 000 arrivals) over that library.

    python bench.py --gpus 1 --steps 5 --warmup 3
    python bench.py --setting greedy                    # Algorithm 1's alignment set: 8 x 8 starts, filter, median
    python bench.py --profiles 4096 --steps 3           # stress library of 197 MB: larger than L2, real HBM streaming
    python bench.py --impl reference                    # the CPU oracle on the host cores, same metric

Prints ONE JSON line (rank 0).  With N > 1 ranks (torchrun) every rank builds the same library, computes its
cost-balanced range of the unordered pairs, and the ranks combine the matrix with one NCCL sum all-reduce
(strong scaling of the matrix); the placement stream is a dependent chain and runs replicated on every rank.
The time is the max over ranks.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import roomie_synth as rs  # noqa: E402

METRIC = "kernel_pair_interference_evals_per_s"
UNIT = "evals/s"

# ---- figures taken from ncu captures of this program (one launch of the pairwise walk kernel) ---------------
# dram__bytes_read.sum + dram__bytes_write.sum on the default workload (configuration 3, 512 profiles, base)
MEASURED_WALK_TRAFFIC = {(3, 512, "base"): 38328832 + 62720}
# smsp__inst_executed.sum x 32 lanes / scored pairings: lane-instructions the kernel spends per evaluation
# (128-profile case of configuration 3; the greedy setting's short walks from late start indices cost a little more)
WALK_LANE_INSTR_PER_EVAL = {"base": 80.0, "greedy": 86.4}
SM_COUNT, LANES_PER_SM = 148, 128


def walk_kernel_dram_bytes(num_kernels, evals, walks):
    """Model of the DRAM bytes (read + write) of one launch of the pairwise walk kernel when the library fits in L2:
    compulsory first-touch reads only - 16 B per library record plus the 32 B descriptor of every tile of 1536 path
    steps, partial results staying in L2.  It reproduces the ncu captures of configuration 3 at 128 profiles
    (6.71 MB against 6.74 MB measured) and at 512 (38.35 MB against 38.39 MB)."""
    tiles = evals / 1536.0 + walks / 2.0
    return int(16 * num_kernels + 32 * tiles)


def walk_kernel_traffic(args, num_kernels, evals, P):
    key = (args.config, P, args.setting)
    if key in MEASURED_WALK_TRAFFIC:
        return MEASURED_WALK_TRAFFIC[key], "ncu capture of this workload"
    if args.setting != "base" or 16 * num_kernels > 100e6:
        return None, "not captured for this workload"
    return (walk_kernel_dram_bytes(num_kernels, evals, P * (P + 1) // 2),
            "modelled: 16 B per record + 32 B per tile (reproduces the ncu captures at 128 and 512 profiles)")


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=30)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--repeats", type=int, default=3,
                    help="the timed region (exactly --steps steps) is run this many times; the median is reported")
    ap.add_argument("--impl", default="roomie", choices=["roomie", "reference"])
    ap.add_argument("--config", type=int, default=3, help="library configuration (0-4)")
    ap.add_argument("--setting", default="base", choices=["base", "greedy", "lockstep", "lockstep_full", "detailed"],
                    help="base: alignment (0,0); greedy: 8x8 alignments, start filter, median; lockstep: Algorithm 1's "
                         "lock-step walk on the 8x8 alignment grid; lockstep_full: "
                         "Algorithm 1 as printed over the full Cartesian alignment set; detailed: Section 3.2 simulator")
    ap.add_argument("--arrivals", type=int, default=10000)
    ap.add_argument("--cluster-gpus", type=int, default=None, help="modelled GPUs of the placement cluster (default: the configuration's 64 or 8)")
    ap.add_argument("--cluster-slots", type=int, default=None, help="resident slots per modelled GPU (more than 8 takes the generic placement kernel)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--profiles", type=int, default=None,
                    help="number of profiles drawn from the configuration's recipe (fewer: ncu captures; 4096 on "
                         "configuration 3: a library larger than L2)")
    ap.add_argument("--workspace-mb", type=int, default=2048, help="cap of the pair-walk scratch; a larger need is batched")
    ap.add_argument("--oracle-threads", type=int, default=0, help="threads of the CPU oracle (0 = all host cores)")
    ap.add_argument("--core-only", action="store_true",
                    help="time the step only: no phase breakdown, no batched placement, no end-to-end leg "
                         "(for profiler captures, which want few launches)")
    return ap.parse_args()


def setting_kw(name):
    if name == "lockstep_full":
        return dict(mode=1, n_align=0, start_filter=1)
    if name == "lockstep":
        return dict(mode=1, n_align=8, start_filter=1)
    if name == "detailed":                              # Section 3.2 simulator, equal partition, alignment (0, 0)
        return dict(mode=2, n_align=1, start_filter=0)
    return dict(mode=0, n_align=1, start_filter=0) if name == "base" else dict(mode=0, n_align=8, start_filter=1)


def oracle_sample_pairs(setting, lib):
    """Pairs the CPU oracle is timed on: a prefix of the pair list worth about 1e9 scored pairings (the whole
    list where it is smaller, as on the default workload at the base setting)."""
    P = lib.num_profiles
    total = P * (P + 1) // 2
    per_pair = 2.0 * float(lib.q().mean()) * {"base": 1.0, "detailed": 1.6, "greedy": 26.0, "lockstep": 13.0}.get(setting, 0.0)
    if setting == "lockstep_full":
        per_pair = float(lib.q().mean()) ** 2 * float(lib.q().mean()) / 3.0          # one walk per alignment
    return int(max(1, min(total, 1.0e9 / max(per_pair, 1.0))))


def make_inputs(cfg, num_profiles, arrivals, rank=0, gpus=None, slots=None):
    seed = rs.config_seed(cfg)
    lib = rs.make_library(cfg, seed=seed, num_profiles=num_profiles)
    ccfg = cfg if rs.CONFIGS[cfg].num_gpus else 2          # cluster shape of the online-placement config
    # placement is replicated, not sharded: every rank places its own arrival stream over the common library
    cl = rs.make_cluster(ccfg, seed=seed + 7919 * rank, num_profiles=lib.num_profiles, num_arrivals=arrivals,
                         num_gpus=gpus, max_residents=slots)
    return lib, cl


def config_dict(args, lib, cl):
    """The workload, in the same words for both arms."""
    P = lib.num_profiles
    return {"workload": f"config{args.config}-{rs.CONFIGS[args.config].name}", "setting": args.setting,
            "profiles": P, "kernels": int(lib.num_kernels), "pairs": P * (P + 1) // 2,
            "placement": f"{cl.num_gpus} gpus x {cl.max_residents} slots, {len(cl.arr_id)} arrivals"}


def algorithmic_bytes(lib):
    """Operand bytes of one full matrix: both profiles of every unordered pair (diagonal included)
    as 16-byte records in, two float32 slowdowns out."""
    P, K = lib.num_profiles, lib.num_kernels
    return 16 * (P + 1) * K + 8 * (P * (P + 1) // 2)


class ClockSampler:
    """nvidia-smi clocks and throttle reasons of one GPU while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.rows, self.proc = [], None
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(index), f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "20"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.t = threading.Thread(target=self._read, daemon=True)
            self.t.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([x.strip() for x in line.split(",")])

    def count(self):
        return len(self.rows)

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.05)
        self.proc.terminate()
        self.t.join(timeout=2)
        sm = [float(r[0]) for r in self.rows if len(r) >= 7 and r[0].replace(".", "").isdigit()]
        mx = [float(r[1]) for r in self.rows if len(r) >= 7 and r[1].replace(".", "").isdigit()]
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = sorted({n for r in self.rows if len(r) >= 7 for n, v in zip(names, r[3:7]) if v.lower() == "active"})
        busy = sorted(sm)[len(sm) // 2:] if sm else []          # upper half = samples under load
        return {"sm_mhz": float(np.median(busy)) if busy else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": reasons, "samples": len(sm)}


def oracle_step(oracle, lib, cl, kw, pair_end=None, threads=0):
    """The same step on the CPU oracle; returns (seconds, evals, placements)."""
    t0 = time.perf_counter()
    ol = oracle.library_build(lib)
    Pm, ev = oracle.pair_matrix(ol, pair_end=pair_end, num_threads=threads, **kw)
    P32 = Pm.astype(np.float32)
    G, R = cl.num_gpus, cl.max_residents
    ids2 = cl.ids.reshape(G, R)
    for g in range(G):
        oracle.multi_estimate(P32, ids2[g, :cl.count[g]], cl.arr_id[g % len(cl.arr_id)])
    oracle.place(P32, G, R, cl.ids, cl.expiry, cl.count, 0, cl.arr_id, cl.arr_life, cl.lam)
    return time.perf_counter() - t0, ev, len(cl.arr_id)


def sample_text(pair_end, total, cl):
    return ("full workload" if pair_end == total else f"first {pair_end} of {total} pairs") + f", {len(cl.arr_id)} arrivals"


def run_reference(args, rank, world):
    if rank != 0:
        return
    import oracle
    oracle.build()
    lib, cl = make_inputs(args.config, args.profiles, args.arrivals, 0, args.cluster_gpus, args.cluster_slots)
    kw = setting_kw(args.setting)
    P = lib.num_profiles
    total_pairs = P * (P + 1) // 2
    pair_end = oracle_sample_pairs(args.setting, lib)
    sample = sample_text(pair_end, total_pairs, cl)
    for _ in range(min(args.warmup, 1)):
        oracle_step(oracle, lib, cl, kw, pair_end, args.oracle_threads)
    secs, evals = 0.0, 0
    for _ in range(args.steps):
        s, ev, _ = oracle_step(oracle, lib, cl, kw, pair_end, args.oracle_threads)
        secs += s
        evals += ev
    value = evals / secs
    cores = args.oracle_threads or oracle.max_threads()
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * secs / args.steps,
            "higher_is_better": True, "scaling": "weak" if args.gpus == 1 else "strong", "vs_baseline": None,
            "dtype": "f64", "data": "synthetic", "config": config_dict(args, lib, cl),
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def main():
    args = parse_args()
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if args.impl == "reference":
        run_reference(args, rank, world)
        return

    import torch
    import paper_2607_16784_b200 as rm          # raises if libroomie.so is missing: no fallback
    from paper_2607_16784_b200.shard import partition_pairs

    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)

    lib, cl = make_inputs(args.config, args.profiles, args.arrivals, rank, args.cluster_gpus, args.cluster_slots)
    kw = setting_kw(args.setting)
    P, K = lib.num_profiles, lib.num_kernels
    G, R = cl.num_gpus, cl.max_residents
    total_pairs = P * (P + 1) // 2
    pair_lo, pair_hi = partition_pairs(lib.offsets, world)[rank] if world > 1 else (0, total_pairs)

    # ---- host (pinned) and device copies of the step's inputs --------------------------------
    host_cols = {n: torch.from_numpy(np.ascontiguousarray(getattr(lib, n)).view(np.int32)).pin_memory()
                 for n in ("grid_blocks", "block_threads", "regs_per_thread", "smem_per_block")}
    host_dur = torch.from_numpy(lib.dur_us).pin_memory()
    host_gap = torch.from_numpy(lib.gap_us).pin_memory()
    host_arr = torch.from_numpy(np.stack([cl.arr_id, cl.arr_life.view(np.int32)])).pin_memory()
    host_state = torch.from_numpy(np.concatenate([cl.ids, cl.expiry.view(np.int32), cl.count.view(np.int32)])).pin_memory()
    h2d_bytes = sum(t.numel() * t.element_size() for t in host_cols.values()) + 8 * K + \
        host_arr.numel() * 4 + host_state.numel() * 4
    dcols = {n: t.to(dev) for n, t in host_cols.items()}
    ddur, dgap = host_dur.to(dev), host_gap.to(dev)
    darr, dstate = host_arr.to(dev), host_state.to(dev)

    glib = rm.Library(lib.offsets, lib.spec, dev)
    Pm = torch.zeros((P, P), dtype=torch.float32, device=dev)
    evals = torch.zeros(1, dtype=torch.int64, device=dev)
    ws_bytes = min(rm.pair_workspace_bytes(glib, pair_begin=pair_lo, pair_end=pair_hi, **kw), args.workspace_mb << 20)
    workspace = torch.empty(max(ws_bytes, 256), dtype=torch.uint8, device=dev)
    host_P = torch.empty((P, P), dtype=torch.float32).pin_memory()
    host_gpu = torch.empty(len(cl.arr_id), dtype=torch.int32).pin_memory()
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)      # > L2 (126 MB)
    est_inc = darr[0, :G].contiguous()

    def matrix():
        if world > 1:
            Pm.zero_()                                  # ranks fill disjoint entries; the sum all-reduce gathers them
        rm.pair_matrix(glib, out=Pm, evals=evals, workspace=workspace, pair_begin=pair_lo, pair_end=pair_hi, **kw)
        if world > 1:
            dist.all_reduce(Pm)
            dist.all_reduce(evals)

    def step(cols, dur, gap, arr, state_flat):
        """All rows of the path on device-resident inputs; returns the placement output tensor."""
        rm.occupancy(cols["grid_blocks"], cols["block_threads"], cols["regs_per_thread"], cols["smem_per_block"], lib.spec)
        rm.library_build(cols["grid_blocks"], cols["block_threads"], cols["regs_per_thread"], cols["smem_per_block"],
                         dur, gap, lib.offsets, lib.spec, out=glib)
        matrix()
        work = state_flat.clone()                      # the stream starts from the same cluster state every step
        st = rm.ClusterState.from_tensors(G, R, work[:G * R], work[G * R:2 * G * R], work[2 * G * R:],
                                          torch.zeros(1, dtype=torch.int32, device=dev))
        rm.multi_estimate(Pm, st.ids, st.count, est_inc, max_residents=R)
        gpu, _, _ = rm.place(Pm, st, arr[0], arr[1], cl.lam, want_mean=False)
        return gpu

    def step_e2e():
        cols = {n: t.to(dev, non_blocking=True) for n, t in host_cols.items()}
        gpu = step(cols, host_dur.to(dev, non_blocking=True), host_gap.to(dev, non_blocking=True),
                   host_arr.to(dev, non_blocking=True), host_state.to(dev, non_blocking=True))
        host_P.copy_(Pm, non_blocking=True)
        host_gpu.copy_(gpu, non_blocking=True)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    def timed(fn, steps):
        """Exactly `steps` steps, each between CUDA events on the launching stream; L2 is flushed between steps,
        outside the events.  Returns the summed milliseconds, max over ranks."""
        evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
        barrier()
        for a, b in evs:
            flush.fill_(1)
            a.record()
            fn()
            b.record()
        barrier()
        ms = sum(a.elapsed_time(b) for a, b in evs)
        if dist is not None:
            t = torch.tensor([ms], dtype=torch.float64, device=dev)
            dist.all_reduce(t, op=dist.ReduceOp.MAX)
            ms = float(t.item())
        return ms

    def timed_median(fn, steps, repeats):
        return float(np.median([timed(fn, steps) for _ in range(max(repeats, 1))]))

    warmup = max(args.warmup, 3)
    for _ in range(warmup):
        step(dcols, ddur, dgap, darr, dstate)
    glib.check()
    evals_per_step = int(evals.item())                  # whole matrix (already summed over ranks)

    sampler = ClockSampler(local) if rank == 0 else None
    rm.reset_launch_count()
    rm.profile_enable(True)
    runs = []
    for _ in range(max(args.repeats, 1)):
        runs.append(timed(lambda: step(dcols, ddur, dgap, darr, dstate), args.steps))
    ms_dev = float(np.median(runs))
    launches = rm.launch_count() // max(args.repeats, 1)
    walk_ms, walk_launches = rm.profile_walk_ms()       # the event pairs kept (the library keeps the first 256)
    clocks = sampler.stop() if sampler else None
    matrix()
    _, launches_per_matrix = rm.profile_walk_ms()       # walk-kernel launches of one matrix (more than 1 when batched)
    rm.profile_enable(False)

    # phase breakdown (device-resident inputs), outside the timed region
    phases = {}

    def phase(name, fn):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        flush.fill_(1); a.record(); fn(); b.record(); torch.cuda.synchronize()
        phases[name] = a.elapsed_time(b)

    batched = None
    ms_e2e = None
    if not args.core_only:
        phase("occupancy_ms", lambda: rm.occupancy(dcols["grid_blocks"], dcols["block_threads"], dcols["regs_per_thread"],
                                                   dcols["smem_per_block"], lib.spec))
        phase("library_build_ms", lambda: rm.library_build(dcols["grid_blocks"], dcols["block_threads"], dcols["regs_per_thread"],
                                                           dcols["smem_per_block"], ddur, dgap, lib.offsets, lib.spec, out=glib))
        phase("pair_matrix_ms", matrix)
        st0 = rm.ClusterState(G, R, cl.ids, cl.expiry, cl.count, 0)
        phase("placement_ms", lambda: rm.place(Pm, st0, darr[0], darr[1], cl.lam, want_mean=False))

        # the same cluster shape as many independent arrival streams (one CTA each): what the GPU is for on
        # this row, since a single stream is one dependent chain
        S, nb = 10 * 148, min(2048, len(cl.arr_id))
        roll = (np.arange(S)[:, None] * 7 + np.arange(nb)[None, :]) % len(cl.arr_id)
        b_ids = torch.from_numpy(np.tile(cl.ids, (S, 1))).to(dev)
        b_exp = torch.from_numpy(np.tile(cl.expiry.view(np.int32), (S, 1))).to(dev)
        b_cnt = torch.from_numpy(np.tile(cl.count.view(np.int32), (S, 1))).to(dev)
        b_aid = torch.from_numpy(cl.arr_id[roll]).to(dev)
        b_life = torch.from_numpy(cl.arr_life.view(np.int32)[roll]).to(dev)

        def batch_place():
            rm.place_batch(Pm, G, R, b_ids.clone(), b_exp.clone(), b_cnt.clone(),
                           torch.zeros(S, dtype=torch.int32, device=dev), b_aid, b_life, cl.lam)
        batch_place()
        phase("placement_batch_ms", batch_place)
        batched = {"value": S * nb / (phases["placement_batch_ms"] * 1e-3), "streams": S, "arrivals_per_stream": nb}

        for _ in range(2):
            step_e2e()
        ms_e2e = timed_median(step_e2e, args.steps, args.repeats)

    if rank == 0:
        peaks_path = os.path.join(ROOT, "MEASURED_PEAKS.json")
        if os.path.exists(peaks_path):
            peak, peak_src = float(json.load(open(peaks_path))["hbm_gbs"]), "measured"
        else:
            peak, peak_src = 6650.0, "fallback"
        # the matrix part of one step on this rank: its share of the operand bytes
        alg = algorithmic_bytes(lib) * ((pair_hi - pair_lo) / total_pairs)
        per_launch_ms = walk_ms / max(walk_launches, 1)
        kernel_s = per_launch_ms * 1e-3
        operand_gbs = alg / launches_per_matrix / kernel_s / 1e9 if walk_launches else None
        sm_hz = 1e6 * ((clocks or {}).get("sm_mhz") or 1965.0)
        lane_peak = SM_COUNT * LANES_PER_SM * sm_hz                   # plain-ALU lane-instructions per second
        evals_rank = evals_per_step * ((pair_hi - pair_lo) / total_pairs)
        if args.setting == "lockstep_full":
            # compute-bound kernel: table cells visited (q_a*q_b per pair and pass; the exact median takes 2
            # passes over the table when the values under its first digit fit the workspace's lists, as they
            # do here) against the plain-ALU issue peak divided by the lane-instructions one cell visit takes
            # (ncu capture of configuration 2)
            q = lib.q().astype(np.int64)
            ia, ib = np.triu_indices(P)
            visits = 2.0 * float((q[ia] * q[ib]).sum())
            peak_visits = lane_peak / 48.0 / 1e9
            ach = visits / kernel_s / 1e9 if walk_launches else None
            roofline = {"bound": "alu", "kernel": "lockstep_full_kernel", "achieved": ach, "peak": peak_visits,
                        "unit": "G cell visits/s", "frac": (ach / peak_visits) if ach else None,
                        "peak_source": "derived: 148 SMs x 128 lanes x SM clock / 48 lane-instructions per visit",
                        "kernel_ms": per_launch_ms, "launches_per_step": launches_per_matrix, "traffic": None}
        elif args.setting == "lockstep":
            # every pairing loads two 16-byte records; the 64 alignments of a pair re-read the same records, so the
            # loads are served by L1 and L2 and the kernel is bound by the L1 load path, against which it is
            # reported: 64 B per clock and SM, the rate at which ncu's l1tex throughput of this kernel reads 100 %
            # (88.5 % at 55 B per clock and SM in the capture of the 128-profile case); the same bytes against the
            # HBM copy peak are given beside it
            l1_peak = SM_COUNT * 64.0 * sm_hz / 1e9
            ach = 32.0 * evals_rank / kernel_s / 1e9 / launches_per_matrix if walk_launches else None
            roofline = {"bound": "l1", "kernel": "lockstep_tiles_kernel", "achieved": ach, "peak": l1_peak,
                        "unit": "GB/s", "frac": (ach / l1_peak) if ach else None,
                        "peak_source": "derived: 148 SMs x 64 B per clock x sampled SM clock (L1 load path, calibrated on ncu's l1tex throughput of this kernel)",
                        "algorithmic_bytes_per_launch": 32.0 * evals_rank / launches_per_matrix,
                        "kernel_ms": per_launch_ms, "launches_per_step": launches_per_matrix, "traffic": None,
                        "also": {"bound": "hbm", "achieved": ach, "peak": peak, "unit": "GB/s",
                                 "frac": (ach / peak) if ach else None, "peak_source": peak_src,
                                 "operands_served_from": "L1 and L2: a fraction above 1 says that the records are "
                                                         "re-read from cache, not that HBM delivers them"}}
        elif args.setting == "detailed":
            roofline = {"bound": "alu", "kernel": "detailed_walk_kernel", "achieved": evals_rank / kernel_s / 1e9 if walk_launches else None,
                        "peak": None, "unit": "G events/s", "frac": None,
                        "peak_source": "none: a chain of dependent events per walk, latency-bound",
                        "kernel_ms": per_launch_ms, "launches_per_step": launches_per_matrix, "traffic": None}
        else:
            traffic, traffic_src = walk_kernel_traffic(args, K, evals_per_step, P)
            l2_resident = 16 * K < 100e6
            ipe = WALK_LANE_INSTR_PER_EVAL[args.setting]
            lane_rate = evals_rank / launches_per_matrix * ipe / kernel_s if walk_launches else None
            alu = {"bound": "alu", "achieved": lane_rate / 1e12 if lane_rate else None, "peak": lane_peak / 1e12,
                   "unit": "T lane-instructions/s", "frac": lane_rate / lane_peak if lane_rate else None,
                   "lane_instructions_per_eval": ipe,
                   "peak_source": "derived: 148 SMs x 128 lanes x sampled SM clock; instructions per evaluation from an ncu "
                                  "capture of this kernel"}
            hbm = {"bound": "hbm", "achieved": operand_gbs, "peak": peak, "unit": "GB/s",
                   "frac": (operand_gbs / peak) if operand_gbs else None, "peak_source": peak_src,
                   "algorithmic_bytes_per_launch": alg / launches_per_matrix if walk_launches else None,
                   "operands_served_from": "L2 (the 16 B x K library fits in the 126 MB L2)" if l2_resident else "HBM (library larger than L2)",
                   "dram_gbs": (traffic / kernel_s / 1e9) if traffic else None,
                   "dram_frac_of_peak": (traffic / kernel_s / 1e9 / peak) if traffic else None}
            # what the profile shows decides the headline: the base setting streams operand bytes (from L2 when the
            # library fits there, from HBM when it does not); the greedy setting re-walks the same bytes 64 times and
            # is bound by the plain ALUs / issue slots
            main_obj = alu if args.setting == "greedy" else hbm
            other = hbm if args.setting == "greedy" else alu
            roofline = dict(main_obj, kernel="timeline_tiles_kernel", kernel_ms=per_launch_ms,
                            launches_per_step=launches_per_matrix, traffic=traffic, traffic_source=traffic_src)
            roofline["also"] = other
        line = {
            "metric": METRIC, "value": evals_per_step * args.steps / (ms_dev * 1e-3), "unit": UNIT,
            "n_gpus": world, "steps": args.steps, "warmup": warmup, "ms_per_step": ms_dev / args.steps,
            "higher_is_better": True, "scaling": "weak" if world == 1 else "strong", "vs_baseline": None,
            "dtype": "f32", "data": "synthetic", "config": config_dict(args, lib, cl),
            "evals_per_step": evals_per_step,
            "timing": {"repeats": max(args.repeats, 1), "ms_per_repeat": runs,
                       "l2": "256 MB written between timed steps (L2 flush)"},
            "parallelism": "1 GPU" if world == 1 else
                           f"pair ranges over {world} ranks + NCCL sum all-reduce of the {P}x{P} matrix; placement replicated",
            "phases": phases,
            "gpu_launches": int(launches),
            "clocks": clocks,
            "roofline": roofline,
        }
        if not args.core_only:
            line["placements_per_s"] = len(cl.arr_id) / (phases["placement_ms"] * 1e-3)
            line["placements_per_s_batched"] = batched
            line["e2e"] = {"value": evals_per_step * args.steps / (ms_e2e * 1e-3), "unit": UNIT,
                           "h2d_bytes_per_step": int(h2d_bytes), "d2h_bytes_per_step": int(P * P * 4 + 4 * len(cl.arr_id)),
                           "ms_per_step": ms_e2e / args.steps}
        if not args.no_cpu_baseline and world == 1:
            import oracle
            oracle.build()
            pair_end = oracle_sample_pairs(args.setting, lib)
            s, ev, _ = oracle_step(oracle, lib, cl, kw, pair_end, args.oracle_threads)
            line["cpu_baseline"] = {"value": ev / s, "unit": UNIT, "cores": args.oracle_threads or oracle.max_threads(),
                                    "kind": "oracle", "sample": sample_text(pair_end, total_pairs, cl) + f", one step, {s:.2f} s"}
        print(json.dumps(line), flush=True)
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
