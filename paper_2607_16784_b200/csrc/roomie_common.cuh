// Internal definitions shared by the CUDA translation units of libroomie.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>
#include "roomie.h"

namespace roomie {

// ---- packed per-SM demand phi (Eq. 2) -------------------------------------------------
// low word : registers bits 0-19 (guard bit 19), warps bits 20-29 (guard bit 29)
// high word: shared-memory bytes bits 0-21 (guard bit 21), block slots bits 22-31 (guard 31)
// Every field holds a value < 2^(width-2), so the sum of two demands never reaches the guard
// bit, and (Phi | guard) - phi_a - phi_b keeps the guard bit exactly when the sum fits.
constexpr uint32_t kGuardLo = (1u << 19) | (1u << 29);
constexpr uint32_t kGuardHi = (1u << 21) | (1u << 31);
constexpr int kWarpShift = 20;

struct PhiCap {          // (Phi | guard) packed, per word
    uint32_t lo, hi;
};

__host__ __device__ inline PhiCap make_cap(const roomie_gpu_spec& s) {
    PhiCap c;
    c.lo = kGuardLo | s.regs_per_sm | ((s.threads_per_sm / 32u) << kWarpShift);
    c.hi = kGuardHi | s.smem_per_sm | (s.blocks_per_sm << 22);
    return c;
}

// Eq. 2 for two kernels: true when some resource's combined demand exceeds the SM.
__device__ __forceinline__ bool phi_exceeds(uint32_t slack_lo, uint32_t slack_hi,   // cap - phi_a
                                            uint32_t b_lo, uint32_t b_hi) {
    const uint32_t t_lo = slack_lo - b_lo, t_hi = slack_hi - b_hi;
    return ((~t_lo & kGuardLo) | (~t_hi & kGuardHi)) != 0u;
}

struct OccResult {
    uint32_t b_lim, b_res, limiter, warps;
    uint32_t phi_regs, phi_smem;
    float occ, occ_theo;
};

// Section 3.1, Eq. 1 (see roomie_occupancy in roomie.h for the exact rules).  32-bit arithmetic: a
// limit that would need more than 32 bits is a limit of zero blocks (the block does not fit).
__device__ __forceinline__ OccResult occupancy_of(uint32_t grid, uint32_t threads, uint32_t regs,
                                                  uint32_t smem, const roomie_gpu_spec& s) {
    const uint32_t W = s.threads_per_sm / 32u;
    const uint32_t Wb = threads / 32u + ((threads & 31u) ? 1u : 0u);
    const uint32_t kInf = 0xffffffffu;
    uint32_t b = Wb ? W / Wb : 0u;                                   // warp limit
    uint32_t which = 0;
    const uint32_t l1 = s.blocks_per_sm;                             // block-slot limit
    // registers of one block = regs * 32 * Wb (threads padded to whole warps)
    const unsigned long long regs_block64 = (unsigned long long)regs * 32u * Wb;
    const uint32_t regs_block = regs_block64 > s.regs_per_sm ? 0u : (uint32_t)regs_block64;
    const uint32_t l2 = regs_block64 == 0 ? kInf : (regs_block ? s.regs_per_sm / regs_block : 0u);
    const uint32_t l3 = smem ? s.smem_per_sm / smem : kInf;
    if (l1 < b) { b = l1; which = 1; }
    if (l2 < b) { b = l2; which = 2; }
    if (l3 < b) { b = l3; which = 3; }
    const uint32_t b_grid = grid ? (grid - 1u) / s.num_sms + 1u : 0u;
    uint32_t br = b;
    if (b_grid < b) { br = b_grid; which = 4; }
    OccResult r;
    r.b_lim = b;
    r.b_res = br;
    r.limiter = which;
    r.warps = Wb * br;                                               // br <= W / Wb
    r.phi_regs = br * regs_block;                                    // br <= R / regs_block (0 when br = 0)
    r.phi_smem = br * smem;                                          // br <= S / smem
    r.occ = W ? __fdiv_rn((float)r.warps, (float)W) : 0.0f;
    r.occ_theo = W ? __fdiv_rn((float)(Wb * b), (float)W) : 0.0f;
    return r;
}

// ---- pair-walk work descriptors (device scratch) --------------------------------------
struct __align__(16) WalkInfo {      // one per (pair, alignment slot)
    uint32_t tile_base;              // first tile of the walk in the tile list
    uint32_t n_tiles;
    uint32_t length;                 // merge-path states (TIMELINE) / pairings (LOCKSTEP)
    uint32_t valid;                  // alignment kept
};

struct __align__(16) TileDesc {      // one per tile of a walk
    uint32_t recA, recB;             // first record of each side (global record index)
    uint32_t cntA, cntB;             // records consumed from each side inside the tile
    uint32_t baseA, baseB;           // start ticks of the alignment's first kernels
    uint32_t flags;                  // bit0: one more A record exists after the tile, bit1: same for B
    uint32_t walk;                   // walk slot (diagnostics)
};

struct __align__(8) TilePartial {    // one per tile
    float di, dj;
    unsigned long long V;
    uint32_t ties;
    uint32_t pad;
};

constexpr uint32_t kMaxAlignSlots = 4096;   // alignments per pair the finalize kernel can rank

// ---- mbarrier helpers (shared-memory barriers that asynchronous copies complete on) ----------------------
constexpr unsigned long long kWaitNs = 1000000000ull;                    // bound of every wait on a copy: 1 s
constexpr uint32_t kWaitSpins = 1u << 24;
#ifdef __CUDACC__
__device__ __forceinline__ uint32_t smem_addr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_addr(bar)), "r"(count) : "memory");
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
// one arrival that also announces `bytes` of copies that will complete on the barrier
__device__ __forceinline__ void mbar_arrive_expect(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_addr(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(smem_addr(bar)), "r"(parity) : "memory");
    return ok != 0;
}
__device__ __forceinline__ unsigned long long global_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    return t;
}
// waits for the phase with the given parity; gives up after kWaitNs (and, should the timer not
// advance, after kWaitSpins polls)
__device__ __forceinline__ bool mbar_wait_bounded(uint64_t* bar, uint32_t parity, unsigned long long limit_ns = kWaitNs) {
    if (mbar_try_wait(bar, parity)) return true;
    const unsigned long long t0 = global_ns();
    for (uint32_t spin = 0; spin < kWaitSpins; ++spin) {
        if (mbar_try_wait(bar, parity)) return true;
        if (global_ns() - t0 > limit_ns) return false;
    }
    return false;
}
#endif  // __CUDACC__

// thread-local launch counter and CUDA error capture (roomie_api.cu)
void note_launch();
int check_cuda(cudaError_t e);
void profile_mark(cudaStream_t st, bool begin);   // no-op unless profiling is enabled
int sm_count();                                  // SMs of the current device (cached)
int validate_spec(const roomie_gpu_spec* s);     // roomie_library.cu

}  // namespace roomie

#define ROOMIE_CUDA_OK(expr)                                  \
    do {                                                      \
        int _st = ::roomie::check_cuda((expr));               \
        if (_st != ROOMIE_OK) return _st;                     \
    } while (0)
