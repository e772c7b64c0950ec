"""Seeded synthetic inputs for the Roomie interference-model hot path.

This module only *draws inputs*: kernel launch configurations, isolated
durations, inter-kernel gaps, profile lengths, initial cluster residents and
arrival streams.  It holds none of the method's arithmetic (no occupancy, no
ticks, no interference scoring) so that the CPU oracle and the CUDA path can
both consume its arrays without sharing any compute code.

Random numbers come from a counter-based generator: a splitmix64 finaliser
applied to a key mixed from (seed, profile, kernel, field).  Every value is
therefore a pure function of its coordinates and the config seed; arrays are
reproducible across machines and numpy versions.

The distributions stand in for the paper's workloads (kernel profiles of 19
TorchVision models measured on A100 / Jetson Xavier, Table 3), which are not
redistributable; shapes, sizes and value ranges follow the five benchmark
configurations of this build.
"""
from __future__ import annotations

from dataclasses import dataclass, field
import numpy as np

__all__ = [
    "GpuSpec", "SPEC_CLOUD", "SPEC_EDGE", "CONFIGS", "config_seed",
    "make_library", "make_cluster", "uniform01", "Library", "Cluster",
]

_M64 = np.uint64(0xFFFFFFFFFFFFFFFF)
_C_SEED = np.uint64(0x9E3779B97F4A7C15)
_C_PROF = np.uint64(0xBF58476D1CE4E5B9)
_C_KERN = np.uint64(0x94D049BB133111EB)
_C_FIELD = np.uint64(0xD6E8FEB86659FD93)

# field ids (one independent stream per field)
F_KIND, F_THREADS, F_GRID_A, F_GRID_B, F_REGS, F_SMEM_ZERO, F_SMEM_VAL, \
    F_DUR_A, F_DUR_B, F_GAP, F_GAP_MIX, F_QLEN, F_RES_COUNT, F_RES_ID, \
    F_ARR_ID, F_ARR_LIFE = range(16)


def _mix(z: np.ndarray) -> np.ndarray:
    z = (z ^ (z >> np.uint64(30))) * np.uint64(0xBF58476D1CE4E5B9)
    z = (z ^ (z >> np.uint64(27))) * np.uint64(0x94D049BB133111EB)
    return z ^ (z >> np.uint64(31))


def rand_u64(seed: int, profile, kernel, fld: int) -> np.ndarray:
    """splitmix64-style hash of (seed, profile, kernel, field) -> uint64."""
    with np.errstate(over="ignore"):
        p = np.asarray(profile, dtype=np.uint64)
        k = np.asarray(kernel, dtype=np.uint64)
        x = (np.uint64(seed) * _C_SEED + p * _C_PROF + k * _C_KERN
             + np.uint64(fld) * _C_FIELD)
        return _mix(_mix(x + _C_SEED))


def uniform01(seed: int, profile, kernel, fld: int) -> np.ndarray:
    """float64 uniform in [0, 1) from the top 53 bits."""
    return (rand_u64(seed, profile, kernel, fld) >> np.uint64(11)).astype(np.float64) * 2.0 ** -53


def _normal(seed, profile, kernel, fa, fb):
    u1 = uniform01(seed, profile, kernel, fa)
    u2 = uniform01(seed, profile, kernel, fb)
    return np.sqrt(-2.0 * np.log1p(-u1)) * np.cos(2.0 * np.pi * u2)


@dataclass(frozen=True)
class GpuSpec:
    """Per-SM limits of the modelled GPU (not of the GPU the code runs on)."""
    num_sms: int
    regs_per_sm: int
    smem_per_sm: int
    threads_per_sm: int
    blocks_per_sm: int

    def as_array(self) -> np.ndarray:
        return np.array([self.num_sms, self.regs_per_sm, self.smem_per_sm,
                         self.threads_per_sm, self.blocks_per_sm], dtype=np.uint32)


SPEC_CLOUD = GpuSpec(108, 65536, 164 * 1024, 2048, 32)
SPEC_EDGE = GpuSpec(16, 65536, 164 * 1024, 1536, 16)


@dataclass(frozen=True)
class Config:
    name: str
    index: int
    spec: GpuSpec
    num_profiles: int
    q_min: int
    q_max: int
    mix: str                 # "generic" | "cnn" | "transformer"
    dur: tuple               # ("lognormal", median_us, sigma) | ("pareto", alpha, min_us)
    gap: tuple               # ("exp", mean_us) | ("mix", w1, mean1, mean2)
    # placement part (0 GPUs = none)
    num_gpus: int = 0
    max_residents: int = 0
    num_arrivals: int = 0
    init_residents_max: int = 0
    lifetime_mean: float = 0.0
    lam: float = 0.5         # degradation budget used in all the paper's experiments


CONFIGS = {
    0: Config("tiny-pairwise", 0, SPEC_CLOUD, 2, 50, 50, "generic",
              ("lognormal", 20.0, 1.2), ("exp", 3.0)),
    1: Config("all-pairs-library", 1, SPEC_CLOUD, 16, 150, 400, "cnn",
              ("lognormal", 20.0, 1.2), ("exp", 3.0)),
    2: Config("online-placement", 2, SPEC_CLOUD, 32, 200, 2000, "transformer",
              ("lognormal", 20.0, 1.2), ("exp", 3.0),
              num_gpus=64, max_residents=8, num_arrivals=10000,
              init_residents_max=3, lifetime_mean=128.0),
    3: Config("large-all-pairs", 3, SPEC_CLOUD, 512, 1000, 5000, "transformer",
              ("lognormal", 40.0, 1.5), ("exp", 3.0)),
    4: Config("edge-device", 4, SPEC_EDGE, 128, 300, 3000, "transformer",
              ("pareto", 1.5, 5.0), ("mix", 0.8, 1.0, 200.0),
              num_gpus=8, max_residents=4, num_arrivals=4096,
              init_residents_max=3, lifetime_mean=16.0),
}


def config_seed(index: int) -> int:
    return 260716784 + 1000 * index


@dataclass
class Library:
    """Struct-of-arrays kernel table for P profiles concatenated (K kernels)."""
    spec: GpuSpec
    offsets: np.ndarray          # uint32 [P+1]
    grid_blocks: np.ndarray      # uint32 [K]
    block_threads: np.ndarray    # uint32 [K]
    regs_per_thread: np.ndarray  # uint32 [K]
    smem_per_block: np.ndarray   # uint32 [K]
    dur_us: np.ndarray           # float32 [K] isolated kernel duration
    gap_us: np.ndarray           # float32 [K] idle time after the kernel
    seed: int = 0

    @property
    def num_profiles(self) -> int:
        return len(self.offsets) - 1

    @property
    def num_kernels(self) -> int:
        return int(self.offsets[-1])

    def q(self) -> np.ndarray:
        return np.diff(self.offsets.astype(np.int64))

    def profile(self, m: int) -> slice:
        return slice(int(self.offsets[m]), int(self.offsets[m + 1]))


@dataclass
class Cluster:
    """Initial cluster state and arrival stream for the placement step."""
    num_gpus: int
    max_residents: int
    ids: np.ndarray        # int32 [G*R]  profile id per slot, -1 = free
    expiry: np.ndarray     # uint32 [G*R] arrival tick at which the slot frees, 0 = never
    count: np.ndarray      # uint32 [G]
    arr_id: np.ndarray     # int32 [n]
    arr_life: np.ndarray   # uint32 [n]  lifetime in arrival ticks, 0 = forever
    lam: float = 0.5


def _pick(u, values, weights):
    cdf = np.cumsum(np.asarray(weights, dtype=np.float64))
    cdf[-1] = 1.0
    return np.asarray(values)[np.searchsorted(cdf, u, side="right").clip(0, len(values) - 1)]


def _kernel_fields(seed, spec, mix, prof, kidx, feasible):
    """Launch configuration of kernels `kidx` of profile `prof` under a mix."""
    n = len(kidx)
    u_kind = uniform01(seed, prof, kidx, F_KIND)
    u_thr = uniform01(seed, prof, kidx, F_THREADS)
    u_regs = uniform01(seed, prof, kidx, F_REGS)
    u_sz = uniform01(seed, prof, kidx, F_SMEM_ZERO)
    u_sv = uniform01(seed, prof, kidx, F_SMEM_VAL)

    # generic draw (benchmark configuration 0)
    thr_gen = _pick(u_thr, [64, 128, 256, 512, 1024], [.1, .3, .35, .2, .05])
    regs_gen = 16 + np.floor(u_regs * 240).astype(np.int64)          # [16, 255]
    smem_gen = np.where(u_sz < 0.4, 0, 256 * (1 + np.floor(u_sv * 384).astype(np.int64)))

    # CNN-like: 70 % conv-shaped (256 threads, 0-48 KB smem), 30 % elementwise
    conv = u_thr < 0.7
    thr_cnn = np.where(conv, 256, 1024)
    smem_cnn = np.where(conv, 256 * np.floor(u_sv * 193).astype(np.int64), 0)

    # GEMM-shaped: 128/256 threads, 100-200 registers, 32-96 KB smem
    thr_gemm = np.where(u_thr < 0.5, 128, 256)
    regs_gemm = 100 + np.floor(u_regs * 101).astype(np.int64)
    smem_gemm = 32768 + 256 * np.floor(u_sv * 257).astype(np.int64)

    if mix == "generic":
        thr, regs, smem = thr_gen, regs_gen, smem_gen
    elif mix == "cnn":
        thr, regs, smem = thr_cnn, regs_gen, smem_cnn
    elif mix == "transformer":
        gemm = u_kind < 0.6
        thr = np.where(gemm, thr_gemm, thr_cnn)
        regs = np.where(gemm, regs_gemm, regs_gen)
        smem = np.where(gemm, smem_gemm, smem_cnn)
    else:
        raise ValueError(mix)

    regs = (regs + 7) // 8 * 8
    if feasible:
        # keep the kernel launchable on the modelled SM: registers of one block fit
        cap = (spec.regs_per_sm // (32 * ((thr + 31) // 32))) // 8 * 8
        regs = np.minimum(regs, cap)
    z = _normal(seed, prof, kidx, F_GRID_A, F_GRID_B)
    grid = np.clip(np.rint(256.0 * np.exp(1.5 * z)), 1, 65535)
    return (grid.astype(np.uint32), thr.astype(np.uint32),
            regs.astype(np.uint32), smem.astype(np.uint32))


def _durations(seed, prof, kidx, dur):
    if dur[0] == "lognormal":
        z = _normal(seed, prof, kidx, F_DUR_A, F_DUR_B)
        d = dur[1] * np.exp(dur[2] * z)
    elif dur[0] == "pareto":
        u = uniform01(seed, prof, kidx, F_DUR_A)
        d = dur[2] * np.power(1.0 - u, -1.0 / dur[1])
    else:
        raise ValueError(dur)
    return np.minimum(d, 1.0e5).astype(np.float32)


def _gaps(seed, prof, kidx, gap):
    u = uniform01(seed, prof, kidx, F_GAP)
    e = -np.log1p(-u)
    if gap[0] == "exp":
        g = gap[1] * e
    elif gap[0] == "mix":
        um = uniform01(seed, prof, kidx, F_GAP_MIX)
        g = np.where(um < gap[1], gap[2], gap[3]) * e
    else:
        raise ValueError(gap)
    return np.minimum(g, 1.0e5).astype(np.float32)


def make_library(cfg, *, seed: int | None = None, feasible: bool = True,
                 num_profiles: int | None = None) -> Library:
    """Draw the kernel library of a benchmark configuration.

    `cfg` is a Config or its index.  `num_profiles` truncates/extends the
    library (profiles are independent streams, so a prefix of a larger library
    equals the smaller one).  `feasible=False` skips the register clamp so
    that unlaunchable kernels appear (used by tests).
    """
    if not isinstance(cfg, Config):
        cfg = CONFIGS[int(cfg)]
    seed = config_seed(cfg.index) if seed is None else seed
    P = cfg.num_profiles if num_profiles is None else num_profiles
    pid = np.arange(P, dtype=np.uint64)
    uq = uniform01(seed, pid, np.uint64(0xFFFFFFFF), F_QLEN)
    q = cfg.q_min + np.floor(uq * (cfg.q_max - cfg.q_min + 1)).astype(np.int64)
    offsets = np.zeros(P + 1, dtype=np.int64)
    np.cumsum(q, out=offsets[1:])
    K = int(offsets[-1])
    prof = np.repeat(pid, q)
    kidx = (np.arange(K, dtype=np.int64) - np.repeat(offsets[:-1], q)).astype(np.uint64)
    grid, thr, regs, smem = _kernel_fields(seed, cfg.spec, cfg.mix, prof, kidx, feasible)
    return Library(cfg.spec, offsets.astype(np.uint32), grid, thr, regs, smem,
                   _durations(seed, prof, kidx, cfg.dur), _gaps(seed, prof, kidx, cfg.gap), seed)


def make_cluster(cfg, *, seed: int | None = None, num_profiles: int | None = None,
                 num_gpus: int | None = None, num_arrivals: int | None = None,
                 max_residents: int | None = None) -> Cluster:
    """Initial residents (0..init_residents_max per GPU, uniform over the
    library) and a uniform arrival stream with geometric lifetimes."""
    if not isinstance(cfg, Config):
        cfg = CONFIGS[int(cfg)]
    seed = config_seed(cfg.index) if seed is None else seed
    P = cfg.num_profiles if num_profiles is None else num_profiles
    G = cfg.num_gpus if num_gpus is None else num_gpus
    R = cfg.max_residents if max_residents is None else max_residents
    n = cfg.num_arrivals if num_arrivals is None else num_arrivals
    gid = np.arange(G, dtype=np.uint64)
    cnt = np.floor(uniform01(seed, gid, np.uint64(0), F_RES_COUNT)
                   * (cfg.init_residents_max + 1)).astype(np.int64)
    cnt = np.minimum(cnt, R)
    ids = np.full((G, R), -1, dtype=np.int32)
    for s in range(min(R, cfg.init_residents_max)):
        col = np.floor(uniform01(seed, gid, np.uint64(s), F_RES_ID) * P).astype(np.int32)
        ids[:, s] = np.where(s < cnt, col, -1)
    aid = np.arange(n, dtype=np.uint64)
    arr_id = np.floor(uniform01(seed, np.uint64(0), aid, F_ARR_ID) * P).astype(np.int32)
    p = 1.0 / cfg.lifetime_mean if cfg.lifetime_mean > 0 else 1.0
    if p >= 1.0:
        life = np.ones(n, dtype=np.uint32)
    else:
        u = uniform01(seed, np.uint64(0), aid, F_ARR_LIFE)
        life = np.maximum(1, np.ceil(np.log1p(-u) / np.log1p(-p))).astype(np.uint32)
    return Cluster(G, R, ids.reshape(-1), np.zeros(G * R, dtype=np.uint32),
                   cnt.astype(np.uint32), arr_id, life, cfg.lam)
