// Pairwise interference (Algorithm 1, lines 6-20): plan -> tile walk -> finalize.
//
// The event-driven walk over two kernel timelines is a merge of the two sorted lists of kernel
// end times: every walk iteration consumes the kernel that ends first.  That makes the walk a
// merge path, which can be cut at any diagonal by a binary search, so one walk is split into
// tiles of kTileItems path steps and each tile into per-thread slices.  The delay sums are
// order-free (every overlapping pairing is met exactly once), so tiles are summed afterwards
// in a fixed order and the result does not depend on how the path was cut.
//
//   plan      one thread per (pair, alignment): alignment kept?  path length, tiles, and the
//             path split point of every tile (binary searches on the global records)
//   tiles     one CTA per tile: stage the tile's records in shared memory, per-thread merge
//             path search + kItems sequential steps, warp-shuffle reduction -> one partial
//   finalize  one CTA per pair: sum partials per alignment, median over alignments, gamma, /T
#include "roomie_common.cuh"
#include <vector>

namespace roomie {

constexpr int kTileThreads = 128;
constexpr int kItems = 12;                              // path steps per thread
constexpr int kTileItems = kTileThreads * kItems;       // path steps per tile

struct PairSet {                  // which pairs a launch covers
    uint64_t pair_begin;          // first triangular pair index (explicit == 0)
    uint32_t n_pairs;
    uint32_t explicit_pair;       // 1: the single ordered pair (a, b)
    uint32_t a, b;
};

struct LibView {
    const uint4* records;
    const uint32_t* offsets;
    const unsigned long long* T;
    uint32_t P;
    PhiCap cap;
};

__device__ __forceinline__ void pair_of(const PairSet& ps, uint32_t P, uint32_t local, uint32_t& a, uint32_t& b) {
    if (ps.explicit_pair) { a = ps.a; b = ps.b; return; }
    const unsigned long long p = ps.pair_begin + local;
    // row a of the upper triangle starts at a*P - a(a-1)/2
    const double n = 2.0 * P + 1.0;
    long long r = (long long)((n - sqrt(n * n - 8.0 * (double)p)) * 0.5);
    if (r < 0) r = 0;
    if (r > (long long)P - 1) r = P - 1;
    auto row_start = [P](long long x) { return (unsigned long long)(x * P - x * (x - 1) / 2); };
    while (r > 0 && row_start(r) > p) --r;
    while (r + 1 < (long long)P && row_start(r + 1) <= p) ++r;
    a = (uint32_t)r;
    b = a + (uint32_t)(p - row_start(r));
}

// alignment grid of one model: |G(q, A)| and its c-th element (A = 0: every index)
__device__ __forceinline__ uint32_t grid_count(uint32_t q, uint32_t A) { return (A == 0 || A > q) ? q : A; }
__device__ __forceinline__ uint32_t grid_start(uint32_t q, uint32_t A, uint32_t c) {
    return (A == 0 || A > q) ? c : (uint32_t)(((unsigned long long)c * q) / A);
}

struct PlanArgs {
    LibView lib;
    PairSet ps;
    uint32_t slots;          // alignment slots per pair
    uint32_t n_align;
    int start_filter;
    int lockstep;
    WalkInfo* walks;
    TileDesc* tiles;
    uint32_t* tile_counter;  // [0] tiles allocated so far
    uint32_t tile_capacity;
    uint32_t* status;
};

// merge-path split: number of A records among the first d merged items; A goes first on equal
// end times.  Keys are end ticks re-based to the alignment's start.
__device__ __forceinline__ uint32_t path_split_global(const uint4* __restrict__ A, const uint4* __restrict__ B,
                                                      uint32_t na, uint32_t nb, uint32_t baseA, uint32_t baseB,
                                                      uint32_t d) {
    uint32_t lo = d > nb ? d - nb : 0u, hi = d < na ? d : na;
    while (lo < hi) {
        const uint32_t mid = (lo + hi) >> 1;
        const uint32_t ea = __ldg(&A[mid].y) - baseA;
        const uint32_t eb = __ldg(&B[d - 1 - mid].y) - baseB;
        if (ea <= eb) lo = mid + 1; else hi = mid;
    }
    return lo;
}

__global__ void __launch_bounds__(256) plan_kernel(PlanArgs g) {
    const unsigned long long w = (unsigned long long)blockIdx.x * blockDim.x + threadIdx.x;
    const unsigned long long n_walks = (unsigned long long)g.ps.n_pairs * g.slots;
    const int lane = threadIdx.x & 31;
    bool valid = w < n_walks;
    uint32_t a = 0, b = 0, offa = 0, offb = 0, si = 0, sj = 0, na = 0, nb = 0, baseA = 0, baseB = 0;
    uint32_t L = 0, n_tiles = 0, final_tie = 0;
    const uint4 *RA = nullptr, *RB = nullptr;
    if (valid) {
        const uint32_t local = (uint32_t)(w / g.slots), c = (uint32_t)(w % g.slots);
        pair_of(g.ps, g.lib.P, local, a, b);
        offa = g.lib.offsets[a]; offb = g.lib.offsets[b];
        const uint32_t qa = g.lib.offsets[a + 1] - offa, qb = g.lib.offsets[b + 1] - offb;
        const uint32_t ga = grid_count(qa, g.n_align), gb = grid_count(qb, g.n_align);
        const uint32_t ca = c / gb, cb = c % gb;
        valid = ca < ga;
        if (valid) {
            si = grid_start(qa, g.n_align, ca);
            sj = grid_start(qb, g.n_align, cb);
            RA = g.lib.records + offa + si;
            RB = g.lib.records + offb + sj;
            const uint4 ra = __ldg(RA), rb = __ldg(RB);
            if (g.start_filter)
                valid = phi_exceeds(g.lib.cap.lo - ra.z, g.lib.cap.hi - ra.w, rb.z, rb.w);
            na = qa - si; nb = qb - sj;
            baseA = ra.x; baseB = rb.x;
        }
        if (valid) {
            if (g.lockstep) {
                L = na < nb ? na : nb;
            } else {
                // the walk ends when one model runs out: count the path states up to there
                const uint32_t endA = __ldg(&RA[na - 1].y) - baseA, endB = __ldg(&RB[nb - 1].y) - baseB;
                if (endA <= endB) {          // A runs out first: B kernels ending strictly before
                    uint32_t lo = 0, hi = nb;
                    while (lo < hi) {
                        const uint32_t mid = (lo + hi) >> 1;
                        if (__ldg(&RB[mid].y) - baseB < endA) lo = mid + 1; else hi = mid;
                    }
                    L = na + lo;
                    // the tile kernel counts every state with equal end times as a tie; the walk's
                    // last state is one when A's last kernel ends together with a B kernel, but no
                    // intermediate state follows it, so it is given back here
                    if (lo < nb && __ldg(&RB[lo].y) - baseB == endA) final_tie = 1;
                } else {                     // B runs out first: A kernels ending at or before
                    uint32_t lo = 0, hi = na;
                    while (lo < hi) {
                        const uint32_t mid = (lo + hi) >> 1;
                        if (__ldg(&RA[mid].y) - baseA <= endB) lo = mid + 1; else hi = mid;
                    }
                    L = nb + lo;
                }
            }
            n_tiles = (L + kTileItems - 1) / kTileItems;
        }
    }
    // warp-aggregated allocation of tile slots
    uint32_t incl = n_tiles;
#pragma unroll
    for (int s = 1; s < 32; s <<= 1) {
        const uint32_t up = __shfl_up_sync(0xffffffffu, incl, s);
        if (lane >= s) incl += up;
    }
    const uint32_t warp_total = __shfl_sync(0xffffffffu, incl, 31);
    uint32_t base = 0;
    if (lane == 31 && warp_total) base = atomicAdd(g.tile_counter, warp_total);
    base = __shfl_sync(0xffffffffu, base, 31) + incl - n_tiles;
    if (w < n_walks) {
        WalkInfo wi;
        wi.tile_base = base; wi.n_tiles = n_tiles; wi.length = L + final_tie; wi.valid = valid ? 1u : 0u;
        g.walks[w] = wi;
    }
    if (!valid || n_tiles == 0) return;
    if (base + n_tiles > g.tile_capacity) {          // never expected: the host sizes the list
        atomicOr(g.status, ROOMIE_FLAG_WORKSPACE);
        g.walks[w].n_tiles = 0;
        TileDesc z;
        z.recA = z.recB = z.cntA = z.cntB = z.baseA = z.baseB = z.flags = 0; z.walk = (uint32_t)w;
        for (uint32_t k = 0; k < n_tiles && base + k < g.tile_capacity; ++k) g.tiles[base + k] = z;
        return;
    }
    uint32_t x0 = 0;
    for (uint32_t k = 0; k < n_tiles; ++k) {
        const uint32_t d0 = k * kTileItems;
        const uint32_t d1 = (d0 + kTileItems < L) ? d0 + kTileItems : L;
        uint32_t x1;
        if (g.lockstep) x1 = d1;
        else if (d1 == L) {
            // end of the walk: whichever side ran out
            const uint32_t endA = __ldg(&RA[na - 1].y) - baseA, endB = __ldg(&RB[nb - 1].y) - baseB;
            x1 = (endA <= endB) ? na : L - nb;
        } else x1 = path_split_global(RA, RB, na, nb, baseA, baseB, d1);
        TileDesc t;
        if (g.lockstep) {
            t.recA = offa + si + d0; t.recB = offb + sj + d0;
            t.cntA = d1 - d0; t.cntB = d1 - d0;
            t.flags = 0;
        } else {
            const uint32_t y0 = d0 - x0, y1 = d1 - x1;
            t.recA = offa + si + x0; t.recB = offb + sj + y0;
            t.cntA = x1 - x0; t.cntB = y1 - y0;
            t.flags = (x1 < na ? 1u : 0u) | (y1 < nb ? 2u : 0u);
        }
        t.baseA = baseA; t.baseB = baseB;
        t.walk = (uint32_t)w;
        g.tiles[base + k] = t;
        x0 = x1;
    }
}

// ---------------------------------------------------------------------------------------
// TIMELINE tiles
// ---------------------------------------------------------------------------------------
struct TileArgs {
    const uint4* records;
    const TileDesc* tiles;
    const uint32_t* tile_counter;
    uint32_t tile_capacity;
    TilePartial* partials;
    PhiCap cap;
    uint32_t* status;            // library status word (sticky flags)
};

// Shared-memory layout of one tile.  The tile's A records sit at unified indices 0, 1, 2, ... and
// its B records at b_off, b_off + 1, ... with b_off the A count rounded up to a multiple of kChunk.
// Nothing else lives in shared memory: the diagonal search probes the end ticks inside the records
// and the reciprocal of o_i + o_j comes from the special-function unit, which leaves room for 8
// resident CTAs (32 warps) per SM.
//
// Staging is done by the copy engine, not by the threads: the records are copied as they are, in
// chunks of kChunk records (2 KB, `cp.async.bulk` global -> shared, completion on an mbarrier), so
// that neither the global loads nor the shared-memory stores of the staging pass through the SM's
// load/store pipe, which bounded this kernel while threads staged the records.  Measured on the
// 512-profile workload: 256-byte chunks 2.37 ms, 2 KB chunks 1.99 ms, one copy per side 3.5 ms (a
// single copy is latency-bound; a few dozen in flight per SM are not).  One slot of padding follows
// every chunk.  What staging by threads did on the way is done by the walk instead: B's ticks are
// moved into A's time frame when a B record is taken (A's ticks stay as stored), and Eq. 2 is
// Phi|guards - phi_a - phi_b.  Timelines end below 2^31 ticks, so a B tick in A's frame stays below 2^32:
// times are compared as unsigned numbers, and since all times of one walk lie within 2^31 ticks of each
// other an overlap is the signed difference of two of them.
//
// kItems = 12 steps per thread: the lanes of a warp then start 12 path steps apart, which spreads
// their 16-byte record reads over the bank groups better than a power of two does (16 steps and
// 6 CTAs: 1.99 ms, 17 steps: 1.91 ms, 12 steps and 8 CTAs: 1.89 ms).
constexpr int kPadShift = 7;
constexpr int kChunk = 1 << kPadShift;                                  // records per bulk copy
__device__ __forceinline__ uint32_t rec_slot(uint32_t i) { return i + (i >> kPadShift); }
constexpr int kTileLoad = kTileItems + 2;                               // one look-ahead record per side
constexpr int kTopIndex = kTileLoad + kChunk;                           // unified indices stay below this
constexpr int kRecSlots = kTopIndex + (kTopIndex >> kPadShift) + 1;
constexpr int kTileCtasPerSm = 8;

template <bool kWithV>
__device__ __forceinline__ void block_reduce_store(float di, float dj, unsigned long long V, uint32_t ties,
                                                   TilePartial* out, float* s_f, unsigned long long* s_v,
                                                   uint32_t* s_t, int nwarps) {
#pragma unroll
    for (int s = 16; s > 0; s >>= 1) {
        di += __shfl_xor_sync(0xffffffffu, di, s);
        dj += __shfl_xor_sync(0xffffffffu, dj, s);
        if (kWithV) V += __shfl_xor_sync(0xffffffffu, V, s);
        ties += __shfl_xor_sync(0xffffffffu, ties, s);
    }
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    if (lane == 0) { s_f[2 * wid] = di; s_f[2 * wid + 1] = dj; s_v[wid] = V; s_t[wid] = ties; }
    __syncthreads();
    if (threadIdx.x == 0) {
        TilePartial p;
        p.di = 0.0f; p.dj = 0.0f; p.V = 0; p.ties = 0; p.pad = 0;
        for (int w = 0; w < nwarps; ++w) { p.di += s_f[2 * w]; p.dj += s_f[2 * w + 1]; p.V += s_v[w]; p.ties += s_t[w]; }
        *out = p;
    }
}

// float of a small non-negative integer without the conversion unit
__device__ __forceinline__ float small_int_to_float(uint32_t v) {
    return __uint_as_float(0x4B000000u | v) - 8388608.0f;
}

// ---- asynchronous staging: bulk copies that complete on an mbarrier (helpers in roomie_common.cuh) ----
// bytes: a multiple of 16; both addresses 16-byte aligned
__device__ __forceinline__ void bulk_copy_g2s(void* dst, const void* src, uint32_t bytes, uint64_t* bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_addr(dst)), "l"(src), "r"(bytes), "r"(smem_addr(bar)) : "memory");
}

// copies of one tile: chunk c of A goes to the slots from (kChunk + 1) c on, chunk c of B to those from
// (kChunk + 1) (b_off / kChunk + c) on
__device__ __forceinline__ void stage_tile_async(const uint4* __restrict__ records, const TileDesc& d, uint32_t loadA,
                                                 uint32_t loadB, uint32_t b_off, uint4* s_rec, uint64_t* bar) {
    const uint32_t nA = (loadA + kChunk - 1) / kChunk, nB = (loadB + kChunk - 1) / kChunk;
    for (uint32_t c = threadIdx.x; c < nA + nB; c += kTileThreads) {
        const bool isA = c < nA;
        const uint32_t k = isA ? c : c - nA;
        const uint32_t left = (isA ? loadA : loadB) - k * kChunk;
        const uint32_t cnt = left < (uint32_t)kChunk ? left : (uint32_t)kChunk;
        const uint4* src = records + (isA ? d.recA : d.recB) + k * kChunk;
        uint4* dst = s_rec + (size_t)(kChunk + 1) * ((isA ? 0u : b_off / kChunk) + k);
        bulk_copy_g2s(dst, src, cnt * (uint32_t)sizeof(uint4), bar);
    }
}

// 1/x to one unit in the last place (special-function unit); the delay sums are float32 within
// 1e-5 relative either way
__device__ __forceinline__ float fast_rcp(float x) {
    float r;
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(x));
    return r;
}

// one step of the walk for the pairing (ra, rb).  A step that is not live (ragged tail of a walk)
// touches nothing: the registers may then hold a record from beyond the staged range.
// ra holds A's record as stored, rb holds B's with its ticks moved into A's frame (+ delta).
// fa, fb: the two kernels' resident warps as floats (o = warps / W; W cancels in o_i / (o_i + o_j)).
// Two kernels without a resident block never interfere, so the guard of the reciprocal only keeps
// 0 * inf out of the sums.
#define ROOMIE_WALK_STEP(live)                                                                         \
    if (live) {                                                                                        \
        const uint32_t Ea = ra.y, Eb = rb.y;                                                           \
        const int32_t ov = (int32_t)(min(Ea, Eb) - max(ra.x, rb.x));                                   \
        const bool hit = (ov > 0) && phi_exceeds(cap.lo - ra.z, cap.hi - ra.w, rb.z, rb.w);            \
        const float tw = (hit ? (float)ov : 0.0f) * fast_rcp(fmaxf(fa + fb, 1.0f));  /* overlap/(o_i+o_j) */ \
        di = fmaf(tw, fa, di);                                                                         \
        dj = fmaf(tw, fb, dj);                                                                         \
        if (kWithV) V += hit ? (unsigned long long)(uint32_t)ov : 0ull;                                \
        ties += (Ea == Eb) ? 1u : 0u;                                                                  \
        /* the kernel that ends first is replaced by its model's next one: a single load for the   */  \
        /* whole warp, whichever side each lane advances                                           */  \
        const bool adv_a = Ea <= Eb;                                                                   \
        x += adv_a ? 1u : 0u;                                                                          \
        ib += adv_a ? 0u : 1u;                                                                         \
        const uint4 r = s_rec[rec_slot(adv_a ? x : ib)];                                               \
        const float f = small_int_to_float(r.z >> kWarpShift);                                         \
        if (adv_a) {                                                                                   \
            ra = r; fa = f;                                                                            \
        } else {                                                                                       \
            rb = r; rb.x += delta; rb.y += delta; fb = f;                                              \
        }                                                                                              \
    }

template <bool kWithV>
__global__ void __launch_bounds__(kTileThreads, kTileCtasPerSm) timeline_tiles_kernel(TileArgs g) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    uint4* s_rec = reinterpret_cast<uint4*>(smem_raw);
    __shared__ __align__(8) uint64_t s_bar;
    __shared__ float s_f[2 * kTileThreads / 32];
    __shared__ unsigned long long s_v[kTileThreads / 32];
    __shared__ uint32_t s_t[kTileThreads / 32];

    __shared__ TileDesc s_desc[2];                         // this tile's descriptor and the next one's, fetched ahead
    if (threadIdx.x == 0) mbar_init(&s_bar, 1);
    const uint32_t n_tiles = min(*g.tile_counter, g.tile_capacity);
    if (blockIdx.x >= n_tiles) return;
    if (threadIdx.x == 0) s_desc[0] = g.tiles[blockIdx.x];
    __syncthreads();
    const PhiCap cap = g.cap;
    uint32_t parity = 0, buf = 0;
    // The records of a tile are on their way before the CTA turns to it: those of the first tile from here, those
    // of every later one from the end of the walk before it (the tile's sums are still being added up then).
    auto expect_tile = [&](const TileDesc& dn) {           // one thread: the bytes the barrier will see
        const uint32_t la = dn.cntA + (dn.flags & 1u), lb = dn.cntB + ((dn.flags >> 1) & 1u);
        mbar_arrive_expect(&s_bar, (la + lb) * (uint32_t)sizeof(uint4));
    };
    auto stage_tile = [&](const TileDesc& dn) {            // every thread: its share of the bulk copies
        const uint32_t la = dn.cntA + (dn.flags & 1u), lb = dn.cntB + ((dn.flags >> 1) & 1u);
        stage_tile_async(g.records, dn, la, lb, (la + kChunk - 1) & ~(uint32_t)(kChunk - 1), s_rec, &s_bar);
    };
    if (threadIdx.x == 32) expect_tile(s_desc[0]);
    __syncthreads();
    stage_tile(s_desc[0]);

    for (uint32_t t = blockIdx.x; t < n_tiles; t += gridDim.x, buf ^= 1u) {
        const TileDesc d = s_desc[buf];
        const bool more = t + gridDim.x < n_tiles;
        if (threadIdx.x == 32) {                           // the next descriptor arrives while this tile is walked
            if (more) {
                const uint32_t dst = smem_addr(&s_desc[buf ^ 1u]);
                const TileDesc* src = &g.tiles[t + gridDim.x];
                asm volatile("cp.async.ca.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
                asm volatile("cp.async.ca.shared.global [%0], [%1], 16;" ::"r"(dst + 16u), "l"(reinterpret_cast<const char*>(src) + 16) : "memory");
            }
            asm volatile("cp.async.commit_group;" ::: "memory");
        }
        const uint32_t loadA = d.cntA + (d.flags & 1u);
        const uint32_t b_off = (loadA + kChunk - 1) & ~(uint32_t)(kChunk - 1);
        // a thread whose wait has succeeded sees the tile's records; whether every thread's has is settled at the
        // barrier after the walk
        const bool arrived = mbar_wait_bounded(&s_bar, parity);
        parity ^= 1u;
        const uint32_t len = d.cntA + d.cntB;
        const uint32_t diag = threadIdx.x * kItems;
        const uint32_t delta = d.baseA - d.baseB;          // B tick + delta = the same instant in A's ticks
        float di = 0.0f, dj = 0.0f;
        unsigned long long V = 0;
        uint32_t ties = 0;
        if (arrived && diag < len) {
            // this thread's start point on the tile's merge path (A first on equal end times):
            // B record y sits at unified index b_off + y
            uint32_t lo = diag > d.cntB ? diag - d.cntB : 0u, hi = diag < d.cntA ? diag : d.cntA;
            const uint32_t bdiag = b_off + diag - 1u;                      // index of B[diag - 1 - mid] is bdiag - mid
            while (lo < hi) {
                const uint32_t mid = (lo + hi) >> 1;
                if (s_rec[rec_slot(mid)].y <= s_rec[rec_slot(bdiag - mid)].y + delta) lo = mid + 1;
                else hi = mid;
            }
            uint32_t x = lo, ib = b_off + (diag - lo);
            uint4 ra = s_rec[rec_slot(x)], rb = s_rec[rec_slot(ib)];
            rb.x += delta; rb.y += delta;
            float fa = small_int_to_float(ra.z >> kWarpShift), fb = small_int_to_float(rb.z >> kWarpShift);
            if (len - diag >= (uint32_t)kItems) {
#pragma unroll
                for (int s = 0; s < kItems; ++s) ROOMIE_WALK_STEP(true)
            } else {
                const uint32_t steps = len - diag;
#pragma unroll
                for (int s = 0; s < kItems; ++s) ROOMIE_WALK_STEP((uint32_t)s < steps)
            }
        }
        if (threadIdx.x == 32) {                           // (its own copy of the next descriptor has landed)
            asm volatile("cp.async.wait_group 0;" ::: "memory");
            if (more && arrived) expect_tile(s_desc[buf ^ 1u]);
        }
        // this tile's records are consumed, the next descriptor is in place
        if (!__syncthreads_and(arrived)) {
            // a copy did not arrive within the bound: report it, give the copies in flight one more
            // bounded wait so that none lands after the CTA has gone, and stop (nothing of the next tile is in flight)
            if (threadIdx.x == 0) atomicOr(g.status, ROOMIE_FLAG_WAIT_TIMEOUT);
            if (!arrived) mbar_wait_bounded(&s_bar, parity ^ 1u);
            return;
        }
        if (more) stage_tile(s_desc[buf ^ 1u]);
        block_reduce_store<kWithV>(di, dj, V, ties, &g.partials[t], s_f, s_v, s_t, kTileThreads / 32);
    }
}
#undef ROOMIE_WALK_STEP

// Self-test of the bounded wait: one CTA announces 16 bytes on a barrier, issues no copy, and waits
// with the given limit.  The wait must run out; the kernel then raises the same status bit a real
// time-out raises and returns, leaving the context usable.
__global__ void __launch_bounds__(32) wait_selftest_kernel(uint32_t* status, unsigned long long limit_ns) {
    __shared__ __align__(8) uint64_t s_bar;
    if (threadIdx.x == 0) {
        mbar_init(&s_bar, 1);
        mbar_arrive_expect(&s_bar, 16);
    }
    __syncwarp();
    const bool arrived = mbar_wait_bounded(&s_bar, 0, limit_ns);
    if (!__all_sync(0xffffffffu, arrived) && threadIdx.x == 0) atomicOr(status, ROOMIE_FLAG_WAIT_TIMEOUT);
}

// ---------------------------------------------------------------------------------------
// LOCKSTEP tiles (Algorithm 1 as printed): pairing t of the walk is (s_i + t, s_j + t)
// ---------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kTileThreads, 16) lockstep_tiles_kernel(TileArgs g) {
    __shared__ float s_f[2 * kTileThreads / 32];
    __shared__ unsigned long long s_v[kTileThreads / 32];
    __shared__ uint32_t s_t[kTileThreads / 32];
    const uint32_t n_tiles = min(*g.tile_counter, g.tile_capacity);
    for (uint32_t t = blockIdx.x; t < n_tiles; t += gridDim.x) {
        const TileDesc d = g.tiles[t];
        float di = 0.0f, dj = 0.0f;
        unsigned long long V = 0;
        // one pairing per thread and trip; batching four pairings' loads per trip was measured slower (more
        // instructions, fewer resident warps: 1.37 ms against 1.29 ms on a 128-profile library)
#pragma unroll 2
        for (uint32_t i = threadIdx.x; i < d.cntA; i += kTileThreads) {
            const uint4 ra = __ldg(&g.records[d.recA + i]), rb = __ldg(&g.records[d.recB + i]);
            if (phi_exceeds(g.cap.lo - ra.z, g.cap.hi - ra.w, rb.z, rb.w)) {
                const float wa = small_int_to_float(ra.z >> kWarpShift), wb = small_int_to_float(rb.z >> kWarpShift);
                const float inv = fast_rcp(wa + wb);              // an interfering pair has resident warps on both sides
                const uint32_t da = ra.y - ra.x, db = rb.y - rb.x;
                di = fmaf((float)da * inv, wa, di);
                dj = fmaf((float)db * inv, wb, dj);
                V += (unsigned long long)da + db;
            }
        }
        __syncthreads();
        block_reduce_store<true>(di, dj, V, 0u, &g.partials[t], s_f, s_v, s_t, kTileThreads / 32);
    }
}

// ---------------------------------------------------------------------------------------
// finalize: one CTA per pair
// ---------------------------------------------------------------------------------------
struct FinalArgs {
    LibView lib;
    PairSet ps;
    uint32_t slots;
    uint32_t n_align;
    const WalkInfo* walks;
    const TilePartial* partials;
    float* P_out;                 // matrix [P*P] (or out2 for an explicit pair)
    unsigned long long* evals_out;
    roomie_pair_detail detail;    // capacity 0 = none
};

// k-th smallest of v[0..n) by rank counting (ties ordered by index); one warp, every lane returns it
__device__ float select_rank(const float* v, uint32_t n, uint32_t k, int lane) {
    float pick = 0.0f;
    bool mine = false;
    for (uint32_t e = lane; e < n; e += 32) {
        const float x = v[e];
        uint32_t rank = 0;
        for (uint32_t j = 0; j < n; ++j) {
            const float y = v[j];
            rank += (y < x) || (y == x && j < e);
        }
        if (rank == k) { pick = x; mine = true; }
    }
    const uint32_t who = __ballot_sync(0xffffffffu, mine);        // exactly one lane holds rank k
    return __shfl_sync(0xffffffffu, pick, __ffs(who) - 1);
}

// P[a][b], P[b][a] from the two medians (gamma = max(q_i/q_j, 1), Eq. 4 with M = {i, j})
__device__ __forceinline__ void store_pair_values(const LibView& lib, const PairSet& ps, float* P_out, uint32_t a,
                                                  uint32_t b, uint32_t qa, uint32_t qb, float med_i, float med_j) {
    const unsigned long long Ta = lib.T[a], Tb = lib.T[b];
    const float fa = (float)qa, fb = (float)qb;
    const float g_ab = fmaxf(__fdiv_rn(fa, fb), 1.0f), g_ba = fmaxf(__fdiv_rn(fb, fa), 1.0f);
    const float p_ab = Ta ? __fdiv_rn(g_ab * med_i, (float)Ta) : 0.0f;
    const float p_ba = Tb ? __fdiv_rn(g_ba * med_j, (float)Tb) : 0.0f;
    if (ps.explicit_pair) {
        P_out[0] = p_ab; P_out[1] = p_ba;
    } else {
        P_out[(size_t)a * lib.P + b] = p_ab;
        if (a != b) P_out[(size_t)b * lib.P + a] = p_ba;
    }
}
__device__ __forceinline__ void store_pair(const FinalArgs& g, uint32_t a, uint32_t b, uint32_t qa, uint32_t qb,
                                           float med_i, float med_j) {
    store_pair_values(g.lib, g.ps, g.P_out, a, b, qa, qb, med_i, med_j);
}

// one warp per pair: ordered sum of the tile partials of every alignment, ordered compaction of
// the kept alignments, medians by rank counting
constexpr int kFinalWarps = 8;
__global__ void __launch_bounds__(kFinalWarps * 32) finalize_kernel(FinalArgs g) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    const uint32_t local = blockIdx.x * (blockDim.x >> 5) + wid;
    if (local >= g.ps.n_pairs) return;                       // whole warp leaves together
    float* v_i = reinterpret_cast<float*>(smem_raw) + (size_t)wid * 2 * g.slots;
    float* v_j = v_i + g.slots;
    uint32_t a, b;
    pair_of(g.ps, g.lib.P, local, a, b);
    const uint32_t qa = g.lib.offsets[a + 1] - g.lib.offsets[a], qb = g.lib.offsets[b + 1] - g.lib.offsets[b];
    const uint32_t gb = grid_count(qb, g.n_align);
    const WalkInfo* walks = g.walks + (size_t)local * g.slots;

    uint32_t n = 0;
    unsigned long long evals = 0;
    for (uint32_t c0 = 0; c0 < g.slots; c0 += 32) {
        const uint32_t c = c0 + lane;
        bool valid = false;
        float di = 0.0f, dj = 0.0f;
        unsigned long long V = 0;
        uint32_t ev = 0;
        if (c < g.slots) {
            const WalkInfo wi = walks[c];
            valid = wi.valid != 0;
            if (valid) {
                uint32_t ties = 0;
                for (uint32_t k = 0; k < wi.n_tiles; ++k) {          // fixed order: tile 0, 1, ...
                    const TilePartial p = g.partials[wi.tile_base + k];
                    di += p.di; dj += p.dj; V += p.V; ties += p.ties;
                }
                ev = wi.length - ties;
                evals += ev;
            }
        }
        const uint32_t ballot = __ballot_sync(0xffffffffu, valid);
        const uint32_t pos = n + __popc(ballot & ((1u << lane) - 1u));
        if (valid) {
            v_i[pos] = di; v_j[pos] = dj;
            if (pos < g.detail.capacity) {
                const uint32_t ca = c / gb, cb = c % gb;
                if (g.detail.s_i) g.detail.s_i[pos] = grid_start(qa, g.n_align, ca);
                if (g.detail.s_j) g.detail.s_j[pos] = grid_start(qb, g.n_align, cb);
                if (g.detail.delta_i) g.detail.delta_i[pos] = di;
                if (g.detail.delta_j) g.detail.delta_j[pos] = dj;
                if (g.detail.V) g.detail.V[pos] = V;
                if (g.detail.evals) g.detail.evals[pos] = ev;
            }
        }
        n += __popc(ballot);
    }
    __syncwarp();
    float med_i = 0.0f, med_j = 0.0f;
    if (n > 0) {
        const uint32_t k1 = (n - 1) / 2, k2 = n / 2;
        const float i1 = select_rank(v_i, n, k1, lane);
        const float i2 = (k2 == k1) ? i1 : select_rank(v_i, n, k2, lane);
        const float j1 = select_rank(v_j, n, k1, lane);
        const float j2 = (k2 == k1) ? j1 : select_rank(v_j, n, k2, lane);
        med_i = 0.5f * (i1 + i2);
        med_j = 0.5f * (j1 + j2);
    }
#pragma unroll
    for (int s = 16; s > 0; s >>= 1) evals += __shfl_xor_sync(0xffffffffu, evals, s);
    if (lane == 0) {
        store_pair(g, a, b, qa, qb, med_i, med_j);
        if (g.detail.n_kept) *g.detail.n_kept = n;
        if (g.evals_out && evals) atomicAdd(g.evals_out, evals);
    }
}

// one alignment per pair and no per-alignment outputs (the base setting): one thread per pair
__global__ void __launch_bounds__(256) finalize_single_kernel(FinalArgs g) {
    const uint32_t local = blockIdx.x * blockDim.x + threadIdx.x;
    unsigned long long evals = 0;
    if (local < g.ps.n_pairs) {
        uint32_t a, b;
        pair_of(g.ps, g.lib.P, local, a, b);
        const uint32_t qa = g.lib.offsets[a + 1] - g.lib.offsets[a], qb = g.lib.offsets[b + 1] - g.lib.offsets[b];
        const WalkInfo wi = g.walks[local];
        float di = 0.0f, dj = 0.0f;
        if (wi.valid) {
            uint32_t ties = 0;
            for (uint32_t k = 0; k < wi.n_tiles; ++k) {
                const TilePartial p = g.partials[wi.tile_base + k];
                di += p.di; dj += p.dj; ties += p.ties;
            }
            evals = wi.length - ties;
        }
        store_pair(g, a, b, qa, qb, 0.5f * (di + di), 0.5f * (dj + dj));   // median of one value, same arithmetic
    }
#pragma unroll
    for (int s = 16; s > 0; s >>= 1) evals += __shfl_xor_sync(0xffffffffu, evals, s);
    if ((threadIdx.x & 31) == 0 && g.evals_out && evals) atomicAdd(g.evals_out, evals);
}

#include "roomie_lockstep_full.cuh"
#include "roomie_detailed.cuh"

// ---------------------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------------------
struct PairRange { uint32_t a, b; };

static void pair_of_host(uint64_t p, uint32_t P, uint32_t& a, uint32_t& b) {
    uint64_t r = 0, start = 0;
    // rows shrink by one each; walk rows (P is at most a few thousand, and this runs once per batch edge)
    while (r + 1 < P && start + (P - r) <= p) { start += P - r; ++r; }
    a = (uint32_t)r; b = (uint32_t)(r + (p - start));
}

static uint32_t host_grid_count(uint32_t q, uint32_t A) { return (A == 0 || A > q) ? q : A; }

struct Need { uint64_t walks, tiles, side; };     // side: 8-byte per-kernel records of the Section 3.2 simulator
constexpr uint64_t kDetailedExtraTiles = 160;     // 5 KB: the 1026-word bucket table of the walk sort

// upper bound of walk slots and tiles for pairs [p0, p1): a walk of a pair has at most
// q_a + q_b - 1 steps whatever its alignment.  Short ranges are counted pair by pair; long ones row by
// row from prefix sums over the profiles (a matrix of 131 328 pairs would otherwise keep the GPU waiting
// for 0.1 ms of host arithmetic in every call), rounding each row up, i.e. by less than one tile per walk.
static bool batch_need(const roomie_library* lib, const roomie_opts* o, bool explicit_pair, uint32_t ea, uint32_t eb,
                       uint64_t p0, uint64_t p1, uint32_t slots, Need& need) {
    const uint32_t* off = lib->offsets_host;
    const uint32_t P = lib->num_profiles;
    const bool detailed = o->walk_mode >= ROOMIE_WALK_DETAILED_EQUAL, lockstep = o->walk_mode == ROOMIE_WALK_LOCKSTEP;
    uint64_t tiles = 0;
    auto add = [&](uint32_t a, uint32_t b) {
        const uint32_t qa = off[a + 1] - off[a], qb = off[b + 1] - off[b];
        const uint64_t n = (uint64_t)host_grid_count(qa, o->n_align) * host_grid_count(qb, o->n_align);
        const uint64_t per = detailed ? 1                                  // one result record per walk
                             : lockstep ? ((uint64_t)(qa < qb ? qa : qb) + kTileItems - 1) / kTileItems
                                        : ((uint64_t)qa + qb - 1 + kTileItems - 1) / kTileItems;
        tiles += n * per;
    };
    if (explicit_pair) add(ea, eb);
    else if (p1 - p0 <= 64) {
        uint32_t a, b;
        pair_of_host(p0, P, a, b);
        for (uint64_t p = p0; p < p1; ++p) {
            add(a, b);
            if (++b == P) { ++a; b = a; }
        }
    } else {
        // G1[b] = sum of alignment starts g of the profiles before b, G2[b] = sum of g * q
        static thread_local std::vector<uint64_t> G1, G2;
        G1.assign((size_t)P + 1, 0); G2.assign((size_t)P + 1, 0);
        for (uint32_t b = 0; b < P; ++b) {
            const uint64_t q = off[b + 1] - off[b], g = host_grid_count((uint32_t)q, o->n_align);
            G1[b + 1] = G1[b] + g;
            G2[b + 1] = G2[b] + g * q;
        }
        uint32_t a, b;
        pair_of_host(p0, P, a, b);
        for (uint64_t left = p1 - p0; left > 0;) {
            const uint64_t cnt = left < (uint64_t)(P - b) ? left : (uint64_t)(P - b);      // pairs (a, b .. b + cnt)
            const uint64_t qa = off[a + 1] - off[a], ga = host_grid_count((uint32_t)qa, o->n_align);
            const uint64_t sg = G1[b + cnt] - G1[b], sgq = G2[b + cnt] - G2[b];
            uint64_t row;                                                  // sum over the row of g_b * tiles per walk
            if (detailed) row = sg;
            else if (lockstep) row = ((sgq < qa * sg ? sgq : qa * sg) + sg * (kTileItems - 1)) / kTileItems + 1;   // min(q_a, q_b) <= q_a, q_b
            else row = (sgq + sg * (qa + kTileItems - 2)) / kTileItems + 1;
            tiles += ga * row;
            left -= cnt; ++a; b = a;
        }
    }
    need.walks = (explicit_pair ? 1 : (p1 - p0)) * (uint64_t)slots;
    if (detailed) tiles = need.walks + kDetailedExtraTiles;       // one result per walk slot + the sort's bucket table
    need.tiles = tiles;
    need.side = !detailed ? 0 : explicit_pair ? (uint64_t)(off[ea + 1] - off[ea]) + (off[eb + 1] - off[eb]) : lib->num_kernels;
    return true;
}

static size_t align_up(size_t x) { return (x + 255) & ~(size_t)255; }

static size_t bytes_for(const Need& n) {
    return 256 + align_up(n.walks * sizeof(WalkInfo)) + align_up(n.tiles * sizeof(TileDesc)) +
           align_up(n.tiles * sizeof(TilePartial)) + align_up(n.side * sizeof(uint64_t));
}

static int slots_for(const roomie_library* lib, const roomie_opts* o, bool explicit_pair, uint32_t ea, uint32_t eb,
                     uint32_t& slots) {
    if (o->n_align > 0) {
        if ((uint64_t)o->n_align * o->n_align > kMaxAlignSlots) return ROOMIE_ERR_CAPACITY;
        slots = o->n_align * o->n_align;
        return ROOMIE_OK;
    }
    // full Cartesian product: the largest q_a * q_b among the pairs involved
    const uint32_t* off = lib->offsets_host;
    uint64_t m;
    if (explicit_pair) m = (uint64_t)(off[ea + 1] - off[ea]) * (off[eb + 1] - off[eb]);
    else {
        uint64_t q1 = 0;
        for (uint32_t p = 0; p < lib->num_profiles; ++p) { const uint64_t q = off[p + 1] - off[p]; if (q > q1) q1 = q; }
        m = q1 * q1;
    }
    if (m > kMaxAlignSlots) return ROOMIE_ERR_CAPACITY;
    slots = (uint32_t)m;
    return ROOMIE_OK;
}

// Algorithm 1 as printed with the full Cartesian alignment set, one CTA per pair.  With a workspace the grid is
// persistent: the workspace holds the counter the CTAs take their pairs from and, per CTA and direction, a list for
// the values under the median's first digit.  Without one (or with one too small for useful lists) every pass goes
// over the table and the grid has one CTA per item of work.
static uint32_t full_ctas() { return 2u * (uint32_t)sm_count(); }
static size_t full_smem_bytes(const roomie_library* lib) {
    return sizeof(FullShared) + (2u * (lib->spec.threads_per_sm / 32u) + 1u) * sizeof(double);
}
static uint64_t largest_table(const roomie_library* lib) {
    uint64_t q1 = 0;
    for (uint32_t p = 0; p < lib->num_profiles; ++p) {
        const uint64_t q = lib->offsets_host[p + 1] - lib->offsets_host[p];
        if (q > q1) q1 = q;
    }
    return q1 * q1;
}
// what lets every pair of the library use the lists, within a fixed bound
static size_t full_workspace_bytes(const roomie_library* lib) {
    uint64_t cap = largest_table(lib) / 8 + kFullMinList;           // the first digit's bin holds a few per cent
    if (cap > (1u << 19)) cap = 1u << 19;
    return 256 + (size_t)full_ctas() * 2 * cap * sizeof(uint32_t);
}

static int run_lockstep_full(const roomie_library* lib, const roomie_opts* o, const PairSet& ps, float* P_out,
                             uint64_t* evals_out, void* workspace, size_t workspace_bytes, cudaStream_t st) {
    FullArgs fa;
    fa.lib.records = static_cast<const uint4*>(lib->records);
    fa.lib.offsets = lib->offsets;
    fa.lib.T = reinterpret_cast<const unsigned long long*>(lib->T);
    fa.lib.P = lib->num_profiles;
    fa.lib.cap = make_cap(lib->spec);
    fa.ps = ps; fa.start_filter = o->start_filter;
    fa.n_inv = 2u * (lib->spec.threads_per_sm / 32u) + 1u;
    fa.P_out = P_out; fa.evals_out = reinterpret_cast<unsigned long long*>(evals_out);
    fa.max_cells = largest_table(lib);
    const uint64_t items = (uint64_t)ps.n_pairs * kFullClasses;
    if (items > 0x7fffffffull) return ROOMIE_ERR_CAPACITY;
    uint32_t grid = (uint32_t)items;
    fa.work_counter = nullptr; fa.lists = nullptr; fa.list_cap = 0;
    const uint32_t ctas = full_ctas() < grid ? full_ctas() : grid;
    if (workspace && workspace_bytes >= 256 + (size_t)ctas * 2 * kFullMinList * sizeof(uint32_t)) {
        uint64_t cap = (workspace_bytes - 256) / ((size_t)ctas * 2 * sizeof(uint32_t));
        if (cap > 0x7fffffffull) cap = 0x7fffffffull;
        fa.work_counter = static_cast<uint32_t*>(workspace);
        fa.lists = reinterpret_cast<uint32_t*>(static_cast<unsigned char*>(workspace) + 256);
        fa.list_cap = (uint32_t)cap;
        grid = ctas;
        ROOMIE_CUDA_OK(cudaMemsetAsync(fa.work_counter, 0, sizeof(uint32_t), st));
    }
    const size_t smem = full_smem_bytes(lib);
    static thread_local int smem_set_for = -1;
    int dev = 0;
    ROOMIE_CUDA_OK(cudaGetDevice(&dev));
    if (smem_set_for != dev) {
        ROOMIE_CUDA_OK(cudaFuncSetAttribute(lockstep_full_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                            (int)(sizeof(FullShared) + 4096)));
        smem_set_for = dev;
    }
    if (smem > sizeof(FullShared) + 4096) return ROOMIE_ERR_CAPACITY;
    profile_mark(st, true);
    lockstep_full_kernel<<<grid, kFullThreads, smem, st>>>(fa);
    profile_mark(st, false);
    note_launch();
    ROOMIE_CUDA_OK(cudaGetLastError());
    return ROOMIE_OK;
}

static bool wants_lockstep_full(const roomie_opts* o) { return o->walk_mode == ROOMIE_WALK_LOCKSTEP && o->n_align == 0; }

static int check_lib(const roomie_library* lib, const roomie_opts* o) {
    if (!lib || !o || !lib->offsets_host || !lib->offsets || !lib->records || !lib->T ||
        !lib->status || lib->num_profiles == 0)
        return ROOMIE_ERR_INVALID_ARG;
    // 16-byte loads and bulk copies of the records: a misaligned table would fault on the device
    if (reinterpret_cast<uintptr_t>(lib->records) & 15u) return ROOMIE_ERR_INVALID_ARG;
    if (o->walk_mode < ROOMIE_WALK_TIMELINE || o->walk_mode > ROOMIE_WALK_DETAILED_FCFS) return ROOMIE_ERR_INVALID_ARG;
    return validate_spec(&lib->spec);
}

static int run_batch(const roomie_library* lib, const roomie_opts* o, const PairSet& ps, uint32_t slots,
                     const Need& need, float* P_out, uint64_t* evals_out, const roomie_pair_detail* detail,
                     unsigned char* ws, cudaStream_t st) {
    uint32_t* counter = reinterpret_cast<uint32_t*>(ws);
    WalkInfo* walks = reinterpret_cast<WalkInfo*>(ws + 256);
    TileDesc* tiles = reinterpret_cast<TileDesc*>(ws + 256 + align_up(need.walks * sizeof(WalkInfo)));
    TilePartial* partials = reinterpret_cast<TilePartial*>(reinterpret_cast<unsigned char*>(tiles) +
                                                           align_up(need.tiles * sizeof(TileDesc)));
    ROOMIE_CUDA_OK(cudaMemsetAsync(counter, 0, 256, st));
    LibView lv;
    lv.records = static_cast<const uint4*>(lib->records);
    lv.offsets = lib->offsets;
    lv.T = reinterpret_cast<const unsigned long long*>(lib->T);
    lv.P = lib->num_profiles;
    lv.cap = make_cap(lib->spec);

    if (o->walk_mode >= ROOMIE_WALK_DETAILED_EQUAL) {
        // Section 3.2 simulator: the walks are sorted by expected length (plan, scan, scatter), then persistent
        // lanes pull them; every walk writes its result where the tile partials go.  The sort's scratch lives in
        // the tile-descriptor area: 32 bytes per walk plus kDetailedExtraTiles descriptors are reserved, 30 bytes
        // per walk and the bucket table are used.  The per-kernel side records follow the partial results.
        unsigned char* area = reinterpret_cast<unsigned char*>(tiles);
        DetailedArgs da;
        da.lib = lv; da.ps = ps; da.slots = slots; da.n_align = o->n_align; da.start_filter = o->start_filter;
        da.spec = lib->spec; da.walks = walks; da.partials = partials; da.status = lib->status;
        da.seeds = reinterpret_cast<WalkSeed*>(area);
        da.order = reinterpret_cast<uint32_t*>(area + need.walks * sizeof(WalkSeed));
        da.bucket = reinterpret_cast<uint16_t*>(area + need.walks * (sizeof(WalkSeed) + sizeof(uint32_t)));
        da.hist = reinterpret_cast<uint32_t*>(area + ((need.walks * 30 + 15) & ~(uint64_t)15));
        da.side = reinterpret_cast<unsigned long long*>(reinterpret_cast<unsigned char*>(partials) +
                                                        align_up(need.tiles * sizeof(TilePartial)));
        if (ps.explicit_pair) {
            const uint32_t* off = lib->offsets_host;
            da.n_ranges = 2;
            da.range[0].first_record = off[ps.a]; da.range[0].count = off[ps.a + 1] - off[ps.a]; da.range[0].first_side = 0;
            da.range[1].first_record = off[ps.b]; da.range[1].count = off[ps.b + 1] - off[ps.b];
            da.range[1].first_side = da.range[0].count;
        } else {
            da.n_ranges = 1;
            da.range[0].first_record = 0; da.range[0].count = lib->num_kernels; da.range[0].first_side = 0;
            da.range[1] = da.range[0];
        }
        uint32_t qmax = 1;
        if (ps.explicit_pair) {
            const uint32_t* off = lib->offsets_host;
            qmax = off[ps.a + 1] - off[ps.a];
            if (off[ps.b + 1] - off[ps.b] > qmax) qmax = off[ps.b + 1] - off[ps.b];
        } else {
            for (uint32_t p = 0; p < lib->num_profiles; ++p)
                if (lib->offsets_host[p + 1] - lib->offsets_host[p] > qmax) qmax = lib->offsets_host[p + 1] - lib->offsets_host[p];
        }
        da.shift = 0;
        while (((2ull * qmax) >> da.shift) >= (uint64_t)kSortBuckets) ++da.shift;
        ROOMIE_CUDA_OK(cudaMemsetAsync(da.hist, 0, (kSortBuckets + 2) * sizeof(uint32_t), st));
        uint64_t sblocks = (need.side + 255) / 256;
        if (sblocks > (uint64_t)sm_count() * 8) sblocks = (uint64_t)sm_count() * 8;
        detailed_side_kernel<<<(unsigned)(sblocks ? sblocks : 1), 256, 0, st>>>(da);
        note_launch();
        uint64_t pblocks = (need.walks + 255) / 256;
        if (pblocks > (uint64_t)sm_count() * 8) pblocks = (uint64_t)sm_count() * 8;
        detailed_plan_kernel<<<(unsigned)pblocks, 256, 0, st>>>(da);
        note_launch();
        detailed_scan_kernel<<<1, kSortBuckets, 0, st>>>(da.hist);
        note_launch();
        detailed_scatter_kernel<<<(unsigned)pblocks, 256, 0, st>>>(da);
        note_launch();
        ROOMIE_CUDA_OK(cudaGetLastError());
        uint64_t wblocks = (need.walks + kDetailedThreads - 1) / kDetailedThreads;
        if (wblocks > (uint64_t)sm_count() * 12) wblocks = (uint64_t)sm_count() * 12;
        profile_mark(st, true);
        if (o->walk_mode == ROOMIE_WALK_DETAILED_EQUAL)
            detailed_walk_kernel<ROOMIE_WALK_DETAILED_EQUAL><<<(unsigned)wblocks, kDetailedThreads, 0, st>>>(da);
        else if (o->walk_mode == ROOMIE_WALK_DETAILED_PRIORITY)
            detailed_walk_kernel<ROOMIE_WALK_DETAILED_PRIORITY><<<(unsigned)wblocks, kDetailedThreads, 0, st>>>(da);
        else
            detailed_walk_kernel<ROOMIE_WALK_DETAILED_FCFS><<<(unsigned)wblocks, kDetailedThreads, 0, st>>>(da);
        profile_mark(st, false);
        note_launch();
        ROOMIE_CUDA_OK(cudaGetLastError());
    } else {
    PlanArgs pa;
    pa.lib = lv; pa.ps = ps; pa.slots = slots; pa.n_align = o->n_align; pa.start_filter = o->start_filter;
    pa.lockstep = o->walk_mode == ROOMIE_WALK_LOCKSTEP;
    pa.walks = walks; pa.tiles = tiles; pa.tile_counter = counter;
    pa.tile_capacity = (uint32_t)need.tiles; pa.status = lib->status;
    const uint64_t plan_blocks = (need.walks + 255) / 256;
    plan_kernel<<<(unsigned)plan_blocks, 256, 0, st>>>(pa);
    note_launch();
    ROOMIE_CUDA_OK(cudaGetLastError());

    TileArgs ta;
    ta.records = lv.records; ta.tiles = tiles; ta.tile_counter = counter; ta.tile_capacity = (uint32_t)need.tiles; ta.partials = partials;
    ta.cap = lv.cap; ta.status = lib->status;
    profile_mark(st, true);
    if (pa.lockstep) {
        uint64_t grid = (uint64_t)sm_count() * 16;            // 64 resident warps per SM: the loads' latency is what is hidden
        if (grid > need.tiles) grid = need.tiles ? need.tiles : 1;
        lockstep_tiles_kernel<<<(unsigned)grid, kTileThreads, 0, st>>>(ta);
    } else {
        const size_t smem = (size_t)kRecSlots * sizeof(uint4);
        auto kern = detail ? timeline_tiles_kernel<true> : timeline_tiles_kernel<false>;
        if (smem > 48 * 1024)
            ROOMIE_CUDA_OK(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        // persistent grid: as many CTAs as fit at once, each striding over the tile list
        int per_sm = (int)((228 * 1024) / (smem + 1024 + 128));
        per_sm = per_sm < 1 ? 1 : (per_sm > kTileCtasPerSm ? kTileCtasPerSm : per_sm);
        uint64_t grid = (uint64_t)sm_count() * per_sm;
        if (grid > need.tiles) grid = need.tiles ? need.tiles : 1;
        kern<<<(unsigned)grid, kTileThreads, smem, st>>>(ta);
    }
    profile_mark(st, false);
    note_launch();
    ROOMIE_CUDA_OK(cudaGetLastError());
    }

    FinalArgs fa;
    fa.lib = lv; fa.ps = ps; fa.slots = slots; fa.n_align = o->n_align; fa.walks = walks; fa.partials = partials;
    fa.P_out = P_out; fa.evals_out = reinterpret_cast<unsigned long long*>(evals_out);
    if (detail) fa.detail = *detail; else { roomie_pair_detail z = {}; fa.detail = z; }
    if (slots == 1 && !detail) {
        finalize_single_kernel<<<(ps.n_pairs + 255) / 256, 256, 0, st>>>(fa);
    } else {
        uint32_t wpb = (uint32_t)((96 * 1024) / ((size_t)slots * 2 * sizeof(float)));   // warps (= pairs) per CTA
        wpb = wpb < 1 ? 1 : (wpb > kFinalWarps ? kFinalWarps : wpb);
        const size_t fsmem = (size_t)wpb * slots * 2 * sizeof(float);
        if (fsmem > 48 * 1024)
            ROOMIE_CUDA_OK(cudaFuncSetAttribute(finalize_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)fsmem));
        finalize_kernel<<<(ps.n_pairs + wpb - 1) / wpb, wpb * 32, fsmem, st>>>(fa);
    }
    note_launch();
    ROOMIE_CUDA_OK(cudaGetLastError());
    return ROOMIE_OK;
}

}  // namespace roomie

using namespace roomie;

// ---------------------------------------------------------------------------------------
// Scratch for roomie_pair_interference_static: part of the library image, so every GPU that
// loads the library keeps it until the process exits.  Host code must not pass the symbol
// itself to a kernel (on the host its name is only a handle): the device address is looked up
// once per device with cudaGetSymbolAddress while that device is current.
// ---------------------------------------------------------------------------------------
namespace roomie {
constexpr size_t kStaticScratchBytes = ROOMIE_STATIC_SCRATCH_BYTES;
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];
constexpr int kMaxDevices = 64;
static void* g_static_scratch_addr[kMaxDevices];       // device address per device ordinal, 0 = not looked up yet

static int static_scratch_for_current_device(void** out) {
    int dev = 0;
    ROOMIE_CUDA_OK(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return ROOMIE_ERR_INVALID_ARG;
    void* p = __atomic_load_n(&g_static_scratch_addr[dev], __ATOMIC_ACQUIRE);
    if (!p) {
        ROOMIE_CUDA_OK(cudaGetSymbolAddress(&p, g_static_scratch));
        if (!p) return ROOMIE_ERR_CUDA;
        __atomic_store_n(&g_static_scratch_addr[dev], p, __ATOMIC_RELEASE);   // same value from every thread
    }
    *out = p;
    return ROOMIE_OK;
}
}  // namespace roomie

extern "C" int roomie_selftest_bounded_wait(uint32_t* status, uint64_t limit_ns, void* stream) {
    if (!status || limit_ns == 0 || limit_ns > 1000000000ull) return ROOMIE_ERR_INVALID_ARG;
    wait_selftest_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(status, limit_ns);
    note_launch();
    ROOMIE_CUDA_OK(cudaGetLastError());
    return ROOMIE_OK;
}

extern "C" size_t roomie_pair_workspace_bytes(const roomie_library* lib, const roomie_opts* opts,
                                              uint64_t pair_begin, uint64_t pair_end) {
    if (check_lib(lib, opts) != ROOMIE_OK) return 0;
    const uint64_t total = (uint64_t)lib->num_profiles * (lib->num_profiles + 1) / 2;
    if (pair_end > total) pair_end = total;
    if (pair_begin >= pair_end) return 0;
    if (wants_lockstep_full(opts)) return full_workspace_bytes(lib);
    uint32_t slots;
    if (slots_for(lib, opts, false, 0, 0, slots) != ROOMIE_OK) return 0;
    Need need;
    batch_need(lib, opts, false, 0, 0, pair_begin, pair_end, slots, need);
    return bytes_for(need);
}

extern "C" size_t roomie_pair_interference_workspace_bytes(const roomie_library* lib, uint32_t a, uint32_t b,
                                                           const roomie_opts* opts) {
    if (check_lib(lib, opts) != ROOMIE_OK || a >= lib->num_profiles || b >= lib->num_profiles) return 0;
    uint32_t slots;
    if (slots_for(lib, opts, true, a, b, slots) != ROOMIE_OK) return 0;
    Need need;
    batch_need(lib, opts, true, a, b, 0, 1, slots, need);
    return bytes_for(need);
}

extern "C" int roomie_pair_matrix(const roomie_library* lib, const roomie_opts* opts, uint64_t pair_begin,
                                  uint64_t pair_end, float* P_out, uint64_t* evals_out, void* workspace,
                                  size_t workspace_bytes, void* stream) {
    int rc = check_lib(lib, opts);
    if (rc != ROOMIE_OK) return rc;
    if (!P_out || !workspace || (reinterpret_cast<uintptr_t>(workspace) & 255u)) return ROOMIE_ERR_INVALID_ARG;
    const uint64_t total = (uint64_t)lib->num_profiles * (lib->num_profiles + 1) / 2;
    if (pair_end > total) pair_end = total;
    if (pair_begin > pair_end) return ROOMIE_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (evals_out) ROOMIE_CUDA_OK(cudaMemsetAsync(evals_out, 0, sizeof(uint64_t), st));
    if (pair_begin == pair_end) return ROOMIE_OK;
    if (wants_lockstep_full(opts)) {
        if (pair_end - pair_begin >= (1ull << 31)) return ROOMIE_ERR_CAPACITY;
        PairSet ps;
        ps.pair_begin = pair_begin; ps.n_pairs = (uint32_t)(pair_end - pair_begin); ps.explicit_pair = 0; ps.a = ps.b = 0;
        return run_lockstep_full(lib, opts, ps, P_out, evals_out, workspace, workspace_bytes, st);
    }
    uint32_t slots;
    rc = slots_for(lib, opts, false, 0, 0, slots);
    if (rc != ROOMIE_OK) return rc;

    uint64_t p0 = pair_begin;
    while (p0 < pair_end) {
        // largest batch [p0, p1) whose scratch fits: try everything, then halve
        uint64_t p1 = pair_end;
        Need need;
        for (;;) {
            batch_need(lib, opts, false, 0, 0, p0, p1, slots, need);
            if (bytes_for(need) <= workspace_bytes && need.walks < (1ull << 31) && need.tiles < (1ull << 31)) break;
            if (p1 - p0 == 1) return ROOMIE_ERR_CAPACITY;
            p1 = p0 + (p1 - p0) / 2;
        }
        PairSet ps;
        ps.pair_begin = p0; ps.n_pairs = (uint32_t)(p1 - p0); ps.explicit_pair = 0; ps.a = ps.b = 0;
        rc = run_batch(lib, opts, ps, slots, need, P_out, evals_out, nullptr, static_cast<unsigned char*>(workspace), st);
        if (rc != ROOMIE_OK) return rc;
        p0 = p1;
    }
    return ROOMIE_OK;
}

extern "C" int roomie_pair_interference(const roomie_library* lib, uint32_t a, uint32_t b, const roomie_opts* opts,
                                        float* out2, uint64_t* evals_out, const roomie_pair_detail* detail,
                                        void* workspace, size_t workspace_bytes, void* stream) {
    int rc = check_lib(lib, opts);
    if (rc != ROOMIE_OK) return rc;
    if (!out2 || !workspace || (reinterpret_cast<uintptr_t>(workspace) & 255u) || a >= lib->num_profiles ||
        b >= lib->num_profiles)
        return ROOMIE_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (evals_out) ROOMIE_CUDA_OK(cudaMemsetAsync(evals_out, 0, sizeof(uint64_t), st));
    if (wants_lockstep_full(opts) && !detail) {
        PairSet fps;
        fps.pair_begin = 0; fps.n_pairs = 1; fps.explicit_pair = 1; fps.a = a; fps.b = b;
        return run_lockstep_full(lib, opts, fps, out2, evals_out, workspace, workspace_bytes, st);
    }
    uint32_t slots;
    rc = slots_for(lib, opts, true, a, b, slots);
    if (rc != ROOMIE_OK) return rc;
    Need need;
    batch_need(lib, opts, true, a, b, 0, 1, slots, need);
    if (bytes_for(need) > workspace_bytes) return ROOMIE_ERR_CAPACITY;
    PairSet ps;
    ps.pair_begin = 0; ps.n_pairs = 1; ps.explicit_pair = 1; ps.a = a; ps.b = b;
    return run_batch(lib, opts, ps, slots, need, out2, evals_out, detail, static_cast<unsigned char*>(workspace), st);
}

extern "C" int roomie_pair_interference_static(const roomie_library* lib, uint32_t a, uint32_t b,
                                               const roomie_opts* opts, float* out2, uint64_t* evals_out,
                                               const roomie_pair_detail* detail, void* stream) {
    int rc = check_lib(lib, opts);
    if (rc != ROOMIE_OK) return rc;
    if (!out2 || a >= lib->num_profiles || b >= lib->num_profiles) return ROOMIE_ERR_INVALID_ARG;
    if (wants_lockstep_full(opts) && !detail) {                      // that path needs no scratch at all
        cudaStream_t fst = static_cast<cudaStream_t>(stream);
        if (evals_out) ROOMIE_CUDA_OK(cudaMemsetAsync(evals_out, 0, sizeof(uint64_t), fst));
        PairSet fps;
        fps.pair_begin = 0; fps.n_pairs = 1; fps.explicit_pair = 1; fps.a = a; fps.b = b;
        return run_lockstep_full(lib, opts, fps, out2, evals_out, nullptr, 0, fst);
    }
    uint32_t slots;
    rc = slots_for(lib, opts, true, a, b, slots);
    if (rc != ROOMIE_OK) return rc;
    Need need;
    batch_need(lib, opts, true, a, b, 0, 1, slots, need);
    if (bytes_for(need) > kStaticScratchBytes) return ROOMIE_ERR_CAPACITY;   // beyond the built-in scratch
    void* scratch = nullptr;
    rc = static_scratch_for_current_device(&scratch);
    if (rc != ROOMIE_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (evals_out) ROOMIE_CUDA_OK(cudaMemsetAsync(evals_out, 0, sizeof(uint64_t), st));
    PairSet ps;
    ps.pair_begin = 0; ps.n_pairs = 1; ps.explicit_pair = 1; ps.a = a; ps.b = b;
    // run_batch zeroes the tile counter at the head of the scratch; everything else in it is
    // written by the plan kernel before it is read, so the previous call's contents do not matter
    return run_batch(lib, opts, ps, slots, need, out2, evals_out, detail, static_cast<unsigned char*>(scratch), st);
}
