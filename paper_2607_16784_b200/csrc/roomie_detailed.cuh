// Section 3.2 in full (adjusted occupancy, two-phase execution, partition policies) as a walk mode of its
// own.  Included by roomie_pairs.cu inside namespace roomie.
//
// The model, in whole ticks.  Two kernel sequences run side by side from an alignment.  The work of a kernel
// is counted in block-ticks: d * b for a kernel of d ticks that runs alone with b resident blocks.  While the
// combined demand of the two active kernels exceeds the SM (Eq. 2) the partition policy leaves each b~ <= b
// blocks, and a kernel does b~ block-ticks per tick (rate o~/o = b~/b): it completes ceil(left / b~) ticks
// later unless the other one completes first, which ends the interference (two-phase execution) - the survivor
// goes on with what is left, against the other model's next kernel or its idle gap.  Every tick spent with b~
// of b blocks delays the kernel by (b - b~)/b.  Gaps are not stretched; the run ends when either sequence is
// exhausted.  Since all times are integers, which kernel completes first and which started earlier (FCFS) never
// depend on rounding.
//   EQUAL     each kernel may use half of every SM resource; if only one of the two fits into a half, the
//             other waits and that one keeps all its blocks; if neither does, the one that started earlier
//             (the first model on a tie) runs alone.
//   PRIORITY  the first model's kernel keeps its blocks; the second gets the blocks that fit into what is left
//             of every resource (none: it waits).
//   FCFS      the same with the kernel that started earlier in the first role (first model on a tie).
//
// A walk is a chain of dependent events, so the parallelism is across walks, and the cost of a warp is its
// longest walk times the instructions of one pass over the event code.  What keeps that product down:
// (1) the walks of a batch are put in descending order of their expected length by a counting sort (plan ->
// scan -> scatter), so the 32 walks of a warp are alike and the longest start first; (2) warps are persistent
// and every lane pulls its next walk from a shared counter when it is done; (3) what depends on a kernel alone
// (its blocks, the demand of one block, the blocks that fit into half an SM) is worked out once per kernel
// of the library into an 8-byte side record, not once per event; (4) the record and side record of each model's
// next kernel are already in registers when the active one completes; (5) the event code is written without
// data-dependent branches except "a kernel completed" (the partition, the time to the next event and the
// bookkeeping of both models are selects), so the lanes of a warp execute it together instead of one after the
// other; the one division an event needs goes through a reciprocal with an integer correction.

constexpr int kSortBuckets = 1024;
constexpr int kDetailedThreads = 128;
constexpr int kEventsPerLook = 4;          // events a lane simulates between two looks at the walk queue

struct WalkSeed {              // what a lane needs to start a walk, written by the plan kernel
    uint32_t recA, recB;       // global index of each model's first record of the alignment
    uint32_t nA, nB;           // records from there to the end of each sequence
    uint32_t sideA, sideB;     // index of the first side record of each model
};

// Per-kernel side record (64 bits): bits 0-7 blocks the kernel runs with alone (1 stands in for a kernel without
// a resident block: it never interferes and takes its isolated time), 8-15 blocks that fit into half an SM,
// 16-23 warps of one block, 24-43 shared-memory bytes of one block, 44-61 registers of one block.
struct SideRange { uint32_t first_record, count, first_side; };

struct DetailedArgs {
    LibView lib;
    PairSet ps;
    uint32_t slots, n_align;
    int start_filter;
    roomie_gpu_spec spec;
    WalkInfo* walks;
    TilePartial* partials;
    WalkSeed* seeds;           // [n_walks]
    uint32_t* order;           // [n_walks] walk slots, longest first
    uint16_t* bucket;          // [n_walks] sort bucket of every kept walk
    uint32_t* hist;            // [kSortBuckets] counts, then cursors; [kSortBuckets] = kept walks; [+1] = next to hand out
    uint32_t shift;            // bucket = (nA + nB) >> shift, reversed
    uint32_t* status;          // library status word
    unsigned long long* side;  // side records
    SideRange range[2];        // which records have side records, and where (an explicit pair: its two profiles)
    uint32_t n_ranges;
};

// ---- arithmetic helpers ---------------------------------------------------------------------------------
// x / d for an exact multiple x < 2^22 of d >= 1: the approximate quotient is within 1/2 of the true one
__device__ __forceinline__ uint32_t div_exact(uint32_t x, uint32_t d) {
    return (uint32_t)__float2int_rn(__fdividef((float)x, (float)d));
}
// floor(x / d) for x < 2^23, d >= 1: approximate quotient, one correction step in integers
__device__ __forceinline__ uint32_t div_floor(uint32_t x, uint32_t d) {
    uint32_t q = (uint32_t)__fdividef((float)x, (float)d);
    const int32_t r = (int32_t)x - (int32_t)(q * d);
    q -= r < 0 ? 1u : 0u;
    q += (r >= 0 && (uint32_t)r >= d) ? 1u : 0u;
    return q;
}
// ceil(x / d) for x < 2^47, 1 <= d <= 255, with magic = ceil(2^64 / d) (2^64 - 1 for d = 1): the high half of
// y * magic is floor(y / d) exactly for every y < 2^56 (the excess of magic over 2^64 / d is below 1, so the error
// of the product is below y, far less than the 2^64 / d that separates a quotient from the next integer)
__device__ __forceinline__ unsigned long long div_ceil(unsigned long long x, uint32_t d, unsigned long long magic) {
    const unsigned long long y = x + d - 1;
    return d == 1 ? x : __umul64hi(y, magic);
}

__device__ __forceinline__ uint32_t side_blocks(unsigned long long s) { return (uint32_t)s & 255u; }
__device__ __forceinline__ uint32_t side_half_fit(unsigned long long s) { return ((uint32_t)s >> 8) & 255u; }
__device__ __forceinline__ uint32_t side_warps(unsigned long long s) { return ((uint32_t)s >> 16) & 255u; }
__device__ __forceinline__ uint32_t side_smem(unsigned long long s) { return (uint32_t)(s >> 24) & ((1u << 20) - 1u); }
__device__ __forceinline__ uint32_t side_regs(unsigned long long s) { return (uint32_t)(s >> 44) & ((1u << 18) - 1u); }

// ---- side records: once per kernel of the library (or of the two profiles of an explicit pair) ---------------
__global__ void __launch_bounds__(256) detailed_side_kernel(DetailedArgs g) {
    const roomie_gpu_spec sp = g.spec;
    for (uint32_t rg = 0; rg < g.n_ranges; ++rg) {
        const SideRange R = g.range[rg];
        for (uint32_t i = blockIdx.x * blockDim.x + threadIdx.x; i < R.count; i += gridDim.x * blockDim.x) {
            const uint4 rec = __ldg(&g.lib.records[R.first_record + i]);
            const uint32_t blocks = rec.w >> 22, b = blocks ? blocks : 1u;
            const uint32_t warps = rec.z >> kWarpShift, regs = rec.z & ((1u << kWarpShift) - 1u),
                           smem = rec.w & ((1u << 22) - 1u);
            const uint32_t wb = div_exact(warps, b), rb = div_exact(regs, b), sb = div_exact(smem, b);
            uint32_t f = min(blocks, sp.blocks_per_sm / 2);
            if (wb) f = min(f, div_floor(sp.threads_per_sm / 64u, wb));
            if (rb) f = min(f, div_floor(sp.regs_per_sm / 2, rb));
            if (sb) f = min(f, div_floor(sp.smem_per_sm / 2, sb));
            g.side[R.first_side + i] = (unsigned long long)b | ((unsigned long long)f << 8) | ((unsigned long long)wb << 16) |
                                       ((unsigned long long)sb << 24) | ((unsigned long long)rb << 44);
        }
    }
}

// ---- plan: which alignments are kept, where they start, how long they may get -----------------------------
__global__ void __launch_bounds__(256) detailed_plan_kernel(DetailedArgs g) {
    __shared__ uint32_t s_hist[kSortBuckets];
    for (int i = threadIdx.x; i < kSortBuckets; i += blockDim.x) s_hist[i] = 0;
    __syncthreads();
    const unsigned long long n_walks = (unsigned long long)g.ps.n_pairs * g.slots;
    for (unsigned long long w = (unsigned long long)blockIdx.x * blockDim.x + threadIdx.x; w < n_walks;
         w += (unsigned long long)gridDim.x * blockDim.x) {
        const uint32_t local = (uint32_t)(w / g.slots), c = (uint32_t)(w % g.slots);
        uint32_t a, b;
        pair_of(g.ps, g.lib.P, local, a, b);
        const uint32_t offa = g.lib.offsets[a], offb = g.lib.offsets[b];
        const uint32_t qa = g.lib.offsets[a + 1] - offa, qb = g.lib.offsets[b + 1] - offb;
        const uint32_t ga = grid_count(qa, g.n_align), gb = grid_count(qb, g.n_align);
        const uint32_t ca = c / gb, cb = c % gb;
        bool keep = ca < ga;
        WalkSeed s;
        s.recA = s.recB = s.nA = s.nB = s.sideA = s.sideB = 0;
        if (keep) {
            const uint32_t si = grid_start(qa, g.n_align, ca), sj = grid_start(qb, g.n_align, cb);
            s.recA = offa + si; s.recB = offb + sj; s.nA = qa - si; s.nB = qb - sj;
            // side records: of the whole library (index = record index) or of the pair's two profiles
            s.sideA = s.recA - g.range[0].first_record + g.range[0].first_side;
            const SideRange& rb = g.range[g.n_ranges - 1];
            s.sideB = s.recB - rb.first_record + rb.first_side;
            if (g.start_filter) {
                const uint4 ra = __ldg(&g.lib.records[s.recA]), rb2 = __ldg(&g.lib.records[s.recB]);
                keep = phi_exceeds(g.lib.cap.lo - ra.z, g.lib.cap.hi - ra.w, rb2.z, rb2.w);
            }
        }
        if (keep) {
            uint32_t k = (s.nA + s.nB) >> g.shift;
            k = kSortBuckets - 1 - (k < (uint32_t)kSortBuckets ? k : (uint32_t)kSortBuckets - 1);   // longest first
            g.seeds[w] = s;
            g.bucket[w] = (uint16_t)k;
            atomicAdd(&s_hist[k], 1u);
        } else {
            WalkInfo wi;
            wi.tile_base = (uint32_t)w; wi.n_tiles = 0; wi.length = 0; wi.valid = 0;
            g.walks[w] = wi;
            g.bucket[w] = 0xffffu;
        }
    }
    __syncthreads();
    for (int i = threadIdx.x; i < kSortBuckets; i += blockDim.x)
        if (s_hist[i]) atomicAdd(&g.hist[i], s_hist[i]);
}

// counts -> first position of every bucket; the total goes behind the table
__global__ void __launch_bounds__(kSortBuckets) detailed_scan_kernel(uint32_t* hist) {
    __shared__ uint32_t s_warp[kSortBuckets / 32];
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    const uint32_t mine = hist[threadIdx.x];
    uint32_t incl = mine;
#pragma unroll
    for (int s = 1; s < 32; s <<= 1) {
        const uint32_t up = __shfl_up_sync(0xffffffffu, incl, s);
        if (lane >= s) incl += up;
    }
    if (lane == 31) s_warp[wid] = incl;
    __syncthreads();
    uint32_t before = 0, total = 0;
    for (int w = 0; w < kSortBuckets / 32; ++w) {
        if (w < wid) before += s_warp[w];
        total += s_warp[w];
    }
    hist[threadIdx.x] = before + incl - mine;
    if (threadIdx.x == 0) { hist[kSortBuckets] = total; hist[kSortBuckets + 1] = 0; }
}

__global__ void __launch_bounds__(256) detailed_scatter_kernel(DetailedArgs g) {
    const unsigned long long n_walks = (unsigned long long)g.ps.n_pairs * g.slots;
    for (unsigned long long w = (unsigned long long)blockIdx.x * blockDim.x + threadIdx.x; w < n_walks;
         w += (unsigned long long)gridDim.x * blockDim.x) {
        const uint32_t k = g.bucket[w];
        if (k != 0xffffu) g.order[atomicAdd(&g.hist[k], 1u)] = (uint32_t)w;     // order inside a bucket is free
    }
}

// One model of the co-run.  The record holds phi at the resident block count: warps = bits 20.. of z, registers
// = low bits of z, shared memory = low bits of w, block slots = bits 22.. of w.
struct CoModel {
    uint4 rec, ahead;                   // active kernel; the one after it (valid while `pending`)
    unsigned long long side, side_ahead;
    uint32_t next_rec, next_side;       // where the kernel after `ahead` is
    uint32_t more;                      // records still to fetch
    uint32_t pending;                   // kernels after the active one, fetched or not
    uint32_t idle;                      // ticks of gap before the active kernel starts
    unsigned long long left;            // block-ticks left
    unsigned long long began;           // tick at which it started
    double lost;                        // delay so far, ticks
    bool alive;                         // the sequence is not exhausted
};

__device__ __forceinline__ void fetch_ahead(CoModel& m, const uint4* __restrict__ records,
                                            const unsigned long long* __restrict__ side) {
    if (m.more) {
        m.ahead = __ldg(&records[m.next_rec]);
        m.side_ahead = __ldg(&side[m.next_side]);
        ++m.next_rec; ++m.next_side; --m.more;
    }
}

__device__ __forceinline__ void open_model(CoModel& m, const uint4* __restrict__ records,
                                           const unsigned long long* __restrict__ side, uint32_t first_rec,
                                           uint32_t first_side, uint32_t n) {
    m.rec = __ldg(&records[first_rec]);
    m.side = __ldg(&side[first_side]);
    m.pending = n - 1; m.more = n - 1;
    m.next_rec = first_rec + 1; m.next_side = first_side + 1;
    fetch_ahead(m, records, side);
    m.idle = 0; m.began = 0; m.lost = 0.0; m.alive = true;
    m.left = (unsigned long long)(m.rec.y - m.rec.x) * side_blocks(m.side);
}

// the active kernel is done: the next one takes its place (after the gap between them), and the one after
// that is fetched
__device__ __forceinline__ void next_kernel(CoModel& m, const uint4* __restrict__ records,
                                            const unsigned long long* __restrict__ side, unsigned long long now) {
    if (m.pending == 0) { m.alive = false; return; }
    const uint32_t ended = m.rec.y;
    m.rec = m.ahead; m.side = m.side_ahead;
    --m.pending;
    fetch_ahead(m, records, side);
    m.idle = m.rec.x - ended;
    m.left = (unsigned long long)(m.rec.y - m.rec.x) * side_blocks(m.side);
    if (m.idle == 0) m.began = now;
}

// blocks of `lo`'s kernel that fit beside all blocks of `hi`'s (what is left of every resource)
__device__ __forceinline__ uint32_t remainder_blocks(uint32_t hi_z, uint32_t hi_w, uint32_t lo_w, unsigned long long lo_side,
                                                     const roomie_gpu_spec& sp) {
    const uint32_t left_w = sp.threads_per_sm / 32u - (hi_z >> kWarpShift);
    const uint32_t left_r = sp.regs_per_sm - (hi_z & ((1u << kWarpShift) - 1u));
    const uint32_t left_s = sp.smem_per_sm - (hi_w & ((1u << 22) - 1u));
    const uint32_t left_b = sp.blocks_per_sm - (hi_w >> 22);
    const uint32_t wb = side_warps(lo_side), rb = side_regs(lo_side), sb = side_smem(lo_side);
    uint32_t f = min(lo_w >> 22, left_b);
    f = min(f, wb ? div_floor(left_w, wb) : f);
    f = min(f, rb ? div_floor(left_r, rb) : f);
    f = min(f, sb ? div_floor(left_s, sb) : f);
    return f;
}

template <int kPolicy>
__global__ void __launch_bounds__(kDetailedThreads) detailed_walk_kernel(DetailedArgs g) {
    __shared__ double s_inv[256];                    // 1 / b: a tick with b~ of b blocks loses (b - b~) / b
    __shared__ unsigned long long s_magic[256];      // ceil(2^64 / d): division by a block count
    for (int i = threadIdx.x; i < 256; i += blockDim.x) {
        s_inv[i] = i ? __ddiv_rn(1.0, (double)i) : 0.0;
        s_magic[i] = i > 1 ? 0xffffffffffffffffull / (unsigned long long)i + 1ull : 0xffffffffffffffffull;
    }
    __syncthreads();
    const uint32_t n_kept = g.hist[kSortBuckets];
    uint32_t* next_walk = g.hist + kSortBuckets + 1;
    const roomie_gpu_spec sp = g.spec;
    const PhiCap cap = g.lib.cap;
    const uint4* __restrict__ records = g.lib.records;
    const unsigned long long* __restrict__ side = g.side;
    const int lane = threadIdx.x & 31;
    const unsigned long long kNever = ~0ull;

    CoModel A, B;
    A.alive = B.alive = false;
    uint32_t slot = 0, events = 0, limit = 0;
    unsigned long long now = 0;
    bool busy = false, drained = false;
    // Every pass of this loop completes one event of each busy lane and hands walks to the idle ones, until
    // the counter has run past the list.  An event ends a gap or completes a kernel of at least one model, so a
    // walk has at most two events per record: a walk that reaches that limit is cut off and reported (it would
    // mean an inconsistent record table), which bounds the loop whatever the data.
    for (;;) {
        const uint32_t want = __ballot_sync(0xffffffffu, !busy && !drained);
        if (want) {
            uint32_t first = 0;
            if (lane == 0) first = atomicAdd(next_walk, (uint32_t)__popc(want));
            first = __shfl_sync(0xffffffffu, first, 0);
            if (!busy && !drained) {
                const uint32_t i = first + (uint32_t)__popc(want & ((1u << lane) - 1u));
                if (i < n_kept) {
                    slot = g.order[i];
                    const WalkSeed s = g.seeds[slot];
                    open_model(A, records, side, s.recA, s.sideA, s.nA);
                    open_model(B, records, side, s.recB, s.sideB, s.nB);
                    now = 0; events = 0; busy = true;
                    limit = 2u * (s.nA + s.nB) + 2u;
                } else drained = true;
            }
        }
        if (__all_sync(0xffffffffu, drained)) break;

        // a few events between two looks at the queue (a lane that finishes in between idles for the rest)
#pragma unroll 1
        for (int rep = 0; rep < kEventsPerLook; ++rep) {
        if (!busy) continue;
        // ---- one event.  Blocks each kernel runs with until something changes: all of its own unless both
        // kernels are active and their combined demand exceeds the SM (Eq. 2) ----
        ++events;
        const uint32_t bA = side_blocks(A.side), bB = side_blocks(B.side);
        const bool actA = A.idle == 0, actB = B.idle == 0;
        const bool contend = actA && actB && phi_exceeds(cap.lo - A.rec.z, cap.hi - A.rec.w, B.rec.z, B.rec.w);
        const bool a_first = kPolicy == ROOMIE_WALK_DETAILED_PRIORITY || A.began <= B.began;
        uint32_t btA, btB;
        if (kPolicy == ROOMIE_WALK_DETAILED_EQUAL) {
            const uint32_t fA = side_half_fit(A.side), fB = side_half_fit(B.side);
            const bool none = fA == 0 && fB == 0;
            btA = fB == 0 ? (none && !a_first ? 0u : bA) : fA;      // the other does not fit: all my blocks
            btB = fA == 0 ? (none && a_first ? 0u : bB) : fB;
        } else {
            const uint32_t rest = remainder_blocks(a_first ? A.rec.z : B.rec.z, a_first ? A.rec.w : B.rec.w,
                                                   a_first ? B.rec.w : A.rec.w, a_first ? B.side : A.side, sp);
            btA = a_first ? bA : rest;
            btB = a_first ? rest : bB;
        }
        btA = contend ? btA : bA;
        btB = contend ? btB : bB;
        // ticks to the next event: a gap ends, or a kernel has done its block-ticks at btX per tick
        const unsigned long long runA = div_ceil(A.left, btA ? btA : 1u, s_magic[btA ? btA : 1u]);
        const unsigned long long runB = div_ceil(B.left, btB ? btB : 1u, s_magic[btB ? btB : 1u]);
        const unsigned long long untilA = actA ? (btA ? runA : kNever) : A.idle;
        const unsigned long long untilB = actB ? (btB ? runB : kNever) : B.idle;
        const unsigned long long step = untilA < untilB ? untilA : untilB;
        now += step;
        // model A
        {
            const bool done = actA && untilA == step;
            if (actA && btA != bA) A.lost = __fma_rn(__ull2double_rn(step * (bA - btA)), s_inv[bA], A.lost);
            if (!actA && A.idle == (uint32_t)step) A.began = now;
            A.idle = actA ? 0u : A.idle - (uint32_t)step;
            A.left -= (actA && !done) ? step * btA : 0ull;
            if (done) next_kernel(A, records, side, now);
        }
        // model B
        {
            const bool done = actB && untilB == step;
            if (actB && btB != bB) B.lost = __fma_rn(__ull2double_rn(step * (bB - btB)), s_inv[bB], B.lost);
            if (!actB && B.idle == (uint32_t)step) B.began = now;
            B.idle = actB ? 0u : B.idle - (uint32_t)step;
            B.left -= (actB && !done) ? step * btB : 0ull;
            if (done) next_kernel(B, records, side, now);
        }
        if (events >= limit && A.alive && B.alive) {
            atomicOr(g.status, ROOMIE_FLAG_WORKSPACE);
            A.alive = false;
        }
        if (!A.alive || !B.alive) {
            WalkInfo wi;
            wi.tile_base = slot; wi.n_tiles = 1; wi.length = events; wi.valid = 1;
            g.walks[slot] = wi;
            TilePartial out;
            out.di = (float)A.lost; out.dj = (float)B.lost; out.V = 0; out.ties = 0; out.pad = 0;
            g.partials[slot] = out;
            busy = false;
        }
        }
    }
}
