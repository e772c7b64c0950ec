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
    python bench.py --impl reference          # the CPU oracle on the host cores, same metric

Prints ONE JSON line (rank 0).  With N > 1 ranks (torchrun) every rank processes its own
seeded library (weak scaling, no data-path collective) and the time is the max over ranks.
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


def walk_kernel_dram_bytes(num_kernels, evals, walks):
    """Model of the DRAM bytes (read + write) of one launch of the pairwise walk kernel: compulsory first-touch
    reads only - 16 B per library record plus the 32 B descriptor of every tile of 1536 path steps, partial
    results staying in L2; every further read of a record is served by L2.  It reproduces the ncu captures of
    configuration 3 (profiles/timeline_tiles_kernel_config3.md): 6.71 MB against 6.74 MB measured at 128
    profiles, 38.35 MB against 38.39 MB at 512."""
    tiles = evals / 1536.0 + walks / 2.0
    return int(16 * num_kernels + 32 * tiles)


# dram__bytes_read.sum + dram__bytes_write.sum of one launch on the default workload (configuration 3, all 512
# profiles, base setting), from an ncu capture of this program (profiles/timeline_tiles_kernel_config3.md)
MEASURED_WALK_TRAFFIC = {(3, 512, "base"): 38328832 + 62720}


def walk_kernel_traffic(args, num_kernels, evals, P):
    if args.setting != "base":
        return None, "not captured for this setting"
    key = (args.config, P, args.setting)
    if key in MEASURED_WALK_TRAFFIC:
        return MEASURED_WALK_TRAFFIC[key], "ncu capture of this workload (profiles/timeline_tiles_kernel_config3.md)"
    return (walk_kernel_dram_bytes(num_kernels, evals, P * (P + 1) // 2),
            "modelled: 16 B per record + 32 B per tile, which reproduces the ncu captures of configuration 3 at 128 "
            "and 512 profiles (profiles/timeline_tiles_kernel_config3.md)")


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=30)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="roomie", choices=["roomie", "reference"])
    ap.add_argument("--config", type=int, default=3, help="library configuration (0-4)")
    ap.add_argument("--setting", default="base", choices=["base", "greedy", "lockstep_full", "detailed"],
                    help="base: alignment (0,0); greedy: 8x8 alignments, start filter, median; lockstep_full: "
                         "Algorithm 1 as printed over the full Cartesian alignment set (use configs 1, 2 or 4)")
    ap.add_argument("--arrivals", type=int, default=10000)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--profiles", type=int, default=None, help="truncate the library (ncu captures)")
    ap.add_argument("--oracle-threads", type=int, default=0, help="threads of the CPU oracle (0 = all host cores)")
    return ap.parse_args()


def setting_kw(name):
    if name == "lockstep_full":
        return dict(mode=1, n_align=0, start_filter=1)
    if name == "detailed":                              # Section 3.2 simulator, equal partition, alignment (0, 0)
        return dict(mode=2, n_align=1, start_filter=0)
    return dict(mode=0, n_align=1, start_filter=0) if name == "base" else dict(mode=0, n_align=8, start_filter=1)


def oracle_sample_pairs(setting, total_pairs):
    """Pairs the CPU oracle is timed on: all of them at the base setting, a bounded prefix otherwise."""
    if setting in ("base", "detailed"):
        return total_pairs
    return max(1, total_pairs // (32 if setting == "greedy" else 512))


def make_inputs(cfg, rank, num_profiles, arrivals):
    seed = rs.config_seed(cfg) + 7919 * rank
    lib = rs.make_library(cfg, seed=seed, num_profiles=num_profiles)
    ccfg = cfg if rs.CONFIGS[cfg].num_gpus else 2          # cluster shape of the online-placement config
    cl = rs.make_cluster(ccfg, seed=seed, num_profiles=lib.num_profiles, num_arrivals=arrivals)
    return lib, cl


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
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.t = threading.Thread(target=self._read, daemon=True)
            self.t.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([x.strip() for x in line.split(",")])

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
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


def run_reference(args, rank, world):
    if rank != 0:
        return
    import oracle
    oracle.build()
    lib, cl = make_inputs(args.config, 0, args.profiles, args.arrivals)
    kw = setting_kw(args.setting)
    P = lib.num_profiles
    total_pairs = P * (P + 1) // 2
    # bounded sample: the base setting runs whole; the greedy one on the first 1/32 of the pairs
    pair_end = oracle_sample_pairs(args.setting, total_pairs)
    sample = ("full workload" if pair_end == total_pairs else f"first {pair_end} of {total_pairs} pairs") + \
             f", {len(cl.arr_id)} arrivals"
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
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": f"config{args.config}-{rs.CONFIGS[args.config].name}", "setting": args.setting,
                       "profiles": P, "kernels": lib.num_kernels, "sample": sample},
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

    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)

    lib, cl = make_inputs(args.config, rank, args.profiles, args.arrivals)
    kw = setting_kw(args.setting)
    P, K = lib.num_profiles, lib.num_kernels
    G, R = cl.num_gpus, cl.max_residents

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
    ws_bytes = min(rm.pair_workspace_bytes(glib, **kw), 2 << 30)
    workspace = torch.empty(ws_bytes, dtype=torch.uint8, device=dev)
    host_P = torch.empty((P, P), dtype=torch.float32).pin_memory()
    host_gpu = torch.empty(len(cl.arr_id), dtype=torch.int32).pin_memory()
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)      # > L2 (126 MB)
    est_inc = darr[0, :G].contiguous()

    def step(cols, dur, gap, arr, state_flat):
        """All rows of the path on device-resident inputs; returns the placement output tensor."""
        rm.occupancy(cols["grid_blocks"], cols["block_threads"], cols["regs_per_thread"], cols["smem_per_block"], lib.spec)
        rm.library_build(cols["grid_blocks"], cols["block_threads"], cols["regs_per_thread"], cols["smem_per_block"],
                         dur, gap, lib.offsets, lib.spec, out=glib)
        rm.pair_matrix(glib, out=Pm, evals=evals, workspace=workspace, **kw)
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
        """Per-step CUDA events on the launching stream; L2 is flushed between steps, outside them."""
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

    for _ in range(max(args.warmup, 3)):
        step(dcols, ddur, dgap, darr, dstate)
    glib.check()
    evals_per_step = int(evals.item())

    sampler = ClockSampler(local) if rank == 0 else None
    rm.reset_launch_count()
    rm.profile_enable(True)
    ms_dev = timed(lambda: step(dcols, ddur, dgap, darr, dstate), args.steps)
    launches = rm.launch_count()
    walk_ms, walk_launches = rm.profile_walk_ms()
    rm.profile_enable(False)
    clocks = sampler.stop() if sampler else None

    # phase breakdown (device-resident inputs), one extra untimed-for-the-metric pass
    phases = {}
    def phase(name, fn):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        flush.fill_(1); a.record(); fn(); b.record(); torch.cuda.synchronize()
        phases[name] = a.elapsed_time(b)
    phase("occupancy_ms", lambda: rm.occupancy(dcols["grid_blocks"], dcols["block_threads"], dcols["regs_per_thread"],
                                               dcols["smem_per_block"], lib.spec))
    phase("library_build_ms", lambda: rm.library_build(dcols["grid_blocks"], dcols["block_threads"], dcols["regs_per_thread"],
                                                       dcols["smem_per_block"], ddur, dgap, lib.offsets, lib.spec, out=glib))
    phase("pair_matrix_ms", lambda: rm.pair_matrix(glib, out=Pm, evals=evals, workspace=workspace, **kw))
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

    for _ in range(2):
        step_e2e()
    ms_e2e = timed(step_e2e, args.steps)

    if world > 1:
        t = torch.tensor([evals_per_step], dtype=torch.int64, device=dev)
        dist.all_reduce(t)
        evals_all = int(t.item())
    else:
        evals_all = evals_per_step

    if rank == 0:
        peaks_path = os.path.join(ROOT, "MEASURED_PEAKS.json")
        if os.path.exists(peaks_path):
            peak, peak_src = float(json.load(open(peaks_path))["hbm_gbs"]), "measured"
        else:
            peak, peak_src = 6650.0, "fallback"
        alg = algorithmic_bytes(lib)
        per_launch_ms = walk_ms / max(walk_launches, 1)
        launches_per_matrix = walk_launches / args.steps
        achieved = alg / launches_per_matrix / (per_launch_ms * 1e-3) / 1e9 if walk_launches else None
        if args.setting == "lockstep_full":
            # compute-bound kernel: table cells visited (q_a*q_b per pair and pass; the exact median takes 3
            # passes, 4 when the number of kept alignments is even: 3 are counted) against the plain-ALU issue
            # peak, 148 SMs x 128 lanes x SM clock, divided by the 53 lane-instructions one cell visit takes
            # (profiles/lockstep_full_kernel_config2.md)
            q = lib.q().astype(np.int64)
            ia, ib = np.triu_indices(P)
            visits = 3.0 * float((q[ia] * q[ib]).sum())
            peak_visits = 148 * 128 * 1.965e9 / 53.0 / 1e9
            ach = visits / (per_launch_ms * 1e-3) / 1e9 if walk_launches else None
            roofline = {"bound": "alu", "kernel": "lockstep_full_kernel", "achieved": ach, "peak": peak_visits,
                        "unit": "G cell visits/s", "frac": (ach / peak_visits) if ach else None,
                        "peak_source": "derived: 148 SMs x 128 lanes x 1.965 GHz / 53 lane-instructions per visit",
                        "kernel_ms": per_launch_ms, "launches_per_step": launches_per_matrix, "traffic": None}
        else:
            roofline = None
        line = {
            "metric": METRIC, "value": evals_all * args.steps / (ms_dev * 1e-3), "unit": UNIT,
            "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms_dev / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": f"config{args.config}-{rs.CONFIGS[args.config].name}", "setting": args.setting,
                       "profiles": P, "kernels": K, "pairs": P * (P + 1) // 2, "evals_per_step": evals_per_step,
                       "placement": f"{G} gpus x {R} slots, {len(cl.arr_id)} arrivals",
                       "l2": "256 MB written between timed steps (L2 flush); the 24 MB library is re-read from L2 within a step"},
            "placements_per_s": len(cl.arr_id) / (phases["placement_ms"] * 1e-3),
            "placements_per_s_batched": {"value": S * nb / (phases["placement_batch_ms"] * 1e-3), "streams": S,
                                         "arrivals_per_stream": nb},
            "phases": phases,
            "e2e": {"value": evals_all * args.steps / (ms_e2e * 1e-3), "unit": UNIT,
                    "h2d_bytes_per_step": int(h2d_bytes), "d2h_bytes_per_step": int(P * P * 4 + 4 * len(cl.arr_id)),
                    "ms_per_step": ms_e2e / args.steps},
            "gpu_launches": int(launches),
            "clocks": clocks,
            "roofline": roofline or {"bound": "hbm", "kernel": {"lockstep_full": "lockstep_full_kernel", "detailed": "detailed_walk_kernel"}.get(args.setting, "timeline_tiles_kernel"), "achieved": achieved, "peak": peak,
                         "unit": "GB/s", "frac": (achieved / peak) if achieved else None, "peak_source": peak_src,
                         "algorithmic_bytes_per_launch": alg / launches_per_matrix if walk_launches else None,
                         "kernel_ms": per_launch_ms, "launches_per_step": launches_per_matrix,
                         "traffic": walk_kernel_traffic(args, K, evals_per_step, P)[0],
                         "traffic_source": walk_kernel_traffic(args, K, evals_per_step, P)[1],
                         "note": "the library (16 B x K) is L2-resident: operand bytes are re-read from L2, not from HBM"},
        }
        if not args.no_cpu_baseline:
            import oracle
            oracle.build()
            total_pairs = P * (P + 1) // 2
            pair_end = oracle_sample_pairs(args.setting, total_pairs)
            s, ev, _ = oracle_step(oracle, lib, cl, kw, pair_end, args.oracle_threads)
            line["cpu_baseline"] = {"value": ev / s, "unit": UNIT, "cores": args.oracle_threads or oracle.max_threads(), "kind": "oracle",
                                    "sample": ("full workload" if pair_end == total_pairs else
                                               f"first {pair_end} of {total_pairs} pairs") + f", one step, {s:.2f} s"}
        print(json.dumps(line), flush=True)
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
