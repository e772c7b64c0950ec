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
// longest walk.  Three things keep the lanes busy: (1) the walks of a batch are put in descending order of
// their expected length by a counting sort (plan -> scan -> scatter), so the 32 walks of a warp are alike and
// the longest start first; (2) warps are persistent and every lane pulls its next walk from a shared counter
// when it is done; (3) the record of each model's next kernel is already in registers when the active one
// completes, work left is kept both in block-ticks and in ticks at full occupancy so that an undisturbed
// kernel needs no division, and the divisions that remain go through reciprocals with an integer correction.

constexpr int kSortBuckets = 1024;
constexpr int kDetailedThreads = 128;

struct WalkSeed {              // what a lane needs to start a walk, written by the plan kernel
    uint32_t recA, recB;       // global index of each model's first record of the alignment
    uint32_t nA, nB;           // records from there to the end of each sequence
};

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
};

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
        s.recA = s.recB = s.nA = s.nB = 0;
        if (keep) {
            const uint32_t si = grid_start(qa, g.n_align, ca), sj = grid_start(qb, g.n_align, cb);
            s.recA = offa + si; s.recB = offb + sj; s.nA = qa - si; s.nB = qb - sj;
            if (g.start_filter) {
                const uint4 ra = __ldg(&g.lib.records[s.recA]), rb = __ldg(&g.lib.records[s.recB]);
                keep = phi_exceeds(g.lib.cap.lo - ra.z, g.lib.cap.hi - ra.w, rb.z, rb.w);
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

// ---- arithmetic helpers ---------------------------------------------------------------------------------
// x / d for an exact multiple x < 2^22 of d >= 1: the approximate quotient is within 1/2 of the true one
__device__ __forceinline__ uint32_t div_exact(uint32_t x, uint32_t d) {
    return (uint32_t)__float2int_rn(__fdividef((float)x, (float)d));
}
// floor(x / d) for x < 2^23, d >= 1: approximate quotient, one correction step in integers
__device__ __forceinline__ uint32_t div_floor(uint32_t x, uint32_t d) {
    uint32_t q = (uint32_t)__fdividef((float)x, (float)d);
    const int32_t r = (int32_t)x - (int32_t)(q * d);
    if (r < 0) --q;
    else if ((uint32_t)r >= d) ++q;
    return q;
}
// ceil(x / d) for x < 2^45, 1 <= d <= 255, with inv = the double nearest to 1/d: the product is within 2^-7 of
// the quotient, so its integer part is at most one off
__device__ __forceinline__ unsigned long long div_ceil(unsigned long long x, uint32_t d, double inv) {
    long long q = __double2ll_rz(__dmul_rn(__ull2double_rn(x), inv));
    long long r = (long long)x - q * (long long)d;
    if (r < 0) { --q; r += d; }
    else if (r >= (long long)d) { ++q; r -= d; }
    return (unsigned long long)q + (r != 0 ? 1ull : 0ull);
}

// One model of the co-run.  The record holds phi at the resident block count: warps = bits 20.. of z, registers
// = low bits of z, shared memory = low bits of w, block slots = bits 22.. of w.
struct CoModel {
    const uint4* at;            // record of the NEXT kernel to fetch
    uint32_t more;              // records still to fetch from `at`
    uint4 rec, ahead;           // active kernel; the one after it (valid while `pending`)
    uint32_t pending;           // kernels after the active one, fetched or not
    uint32_t b;                 // blocks of the active kernel alone, at least 1
    uint32_t fit;               // EQUAL: blocks that fit into half an SM; else unused
    uint32_t wb, rg, sm;        // PRIORITY / FCFS: warps, registers, shared memory of one block
    uint32_t idle;              // ticks of gap before the active kernel starts
    uint32_t full;              // ticks it still needs at full occupancy = ceil(left / b)
    unsigned long long left;    // block-ticks left
    unsigned long long began;   // tick at which it started
    double lost;                // delay so far, ticks
    bool alive;                 // the sequence is not exhausted
};

template <int kPolicy>
__device__ __forceinline__ void start_kernel(CoModel& m, const roomie_gpu_spec& sp, unsigned long long now) {
    const uint32_t blocks = m.rec.w >> 22;
    m.b = blocks ? blocks : 1u;
    m.full = m.rec.y - m.rec.x;
    m.left = (unsigned long long)m.full * m.b;
    if (m.idle == 0) m.began = now;
    const uint32_t warps = m.rec.z >> kWarpShift, regs = m.rec.z & ((1u << kWarpShift) - 1u),
                   smem = m.rec.w & ((1u << 22) - 1u);
    const uint32_t wb = div_exact(warps, m.b), rg = div_exact(regs, m.b), sm = div_exact(smem, m.b);
    if (kPolicy == ROOMIE_WALK_DETAILED_EQUAL) {
        uint32_t f = min(blocks, sp.blocks_per_sm / 2);
        if (wb) f = min(f, div_floor(sp.threads_per_sm / 64u, wb));
        if (rg) f = min(f, div_floor(sp.regs_per_sm / 2, rg));
        if (sm) f = min(f, div_floor(sp.smem_per_sm / 2, sm));
        m.fit = f;
    } else {
        m.wb = wb; m.rg = rg; m.sm = sm;
    }
}

// the active kernel is done: the next one takes its place (after the gap between them), and the one after
// that is fetched
template <int kPolicy>
__device__ __forceinline__ void next_kernel(CoModel& m, const roomie_gpu_spec& sp, unsigned long long now) {
    if (m.pending == 0) { m.alive = false; return; }
    const uint32_t ended = m.rec.y;
    m.rec = m.ahead;
    --m.pending;
    if (m.more) { m.ahead = __ldg(m.at); ++m.at; --m.more; }
    m.idle = m.rec.x - ended;
    start_kernel<kPolicy>(m, sp, now);
}

template <int kPolicy>
__device__ __forceinline__ void open_model(CoModel& m, const uint4* first, uint32_t n, const roomie_gpu_spec& sp) {
    m.rec = __ldg(first);
    m.pending = n - 1;
    m.at = first + 1;
    m.more = n - 1;
    if (m.more) { m.ahead = __ldg(m.at); ++m.at; --m.more; }
    m.idle = 0; m.began = 0; m.lost = 0.0; m.alive = true;
    start_kernel<kPolicy>(m, sp, 0);
}

// blocks of `lo`'s kernel that fit beside all blocks of `hi`'s
__device__ __forceinline__ uint32_t remainder_blocks(const CoModel& hi, const CoModel& lo, const roomie_gpu_spec& sp) {
    const uint32_t left_w = sp.threads_per_sm / 32u - (hi.rec.z >> kWarpShift);
    const uint32_t left_r = sp.regs_per_sm - (hi.rec.z & ((1u << kWarpShift) - 1u));
    const uint32_t left_s = sp.smem_per_sm - (hi.rec.w & ((1u << 22) - 1u));
    const uint32_t left_b = sp.blocks_per_sm - (hi.rec.w >> 22);
    uint32_t f = min(lo.rec.w >> 22, left_b);
    if (lo.wb) f = min(f, div_floor(left_w, lo.wb));
    if (lo.rg) f = min(f, div_floor(left_r, lo.rg));
    if (lo.sm) f = min(f, div_floor(left_s, lo.sm));
    return f;
}

// one model's share of an event of `step` ticks during which it ran with `bt` of its blocks (or idled)
template <int kPolicy>
__device__ __forceinline__ void advance(CoModel& m, uint32_t bt, unsigned long long until, unsigned long long step,
                                        unsigned long long now, const double* s_inv, const roomie_gpu_spec& sp) {
    if (m.idle) {
        m.idle -= (uint32_t)step;
        if (m.idle == 0) m.began = now;
        return;
    }
    if (bt != m.b) m.lost = __fma_rn(__ull2double_rn(step * (m.b - bt)), s_inv[m.b], m.lost);
    if (until == step) { next_kernel<kPolicy>(m, sp, now); return; }
    m.left -= step * bt;
    if (bt == m.b) m.full -= (uint32_t)step;
    else m.full = (uint32_t)div_ceil(m.left, m.b, s_inv[m.b]);
}

template <int kPolicy>
__global__ void __launch_bounds__(kDetailedThreads) detailed_walk_kernel(DetailedArgs g) {
    __shared__ double s_inv[256];
    for (int i = threadIdx.x; i < 256; i += blockDim.x) s_inv[i] = i ? __ddiv_rn(1.0, (double)i) : 0.0;
    __syncthreads();
    const uint32_t n_kept = g.hist[kSortBuckets];
    uint32_t* next_walk = g.hist + kSortBuckets + 1;
    const roomie_gpu_spec sp = g.spec;
    const PhiCap cap = g.lib.cap;
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
                    open_model<kPolicy>(A, g.lib.records + s.recA, s.nA, sp);
                    open_model<kPolicy>(B, g.lib.records + s.recB, s.nB, sp);
                    now = 0; events = 0; busy = true;
                    limit = 2u * (s.nA + s.nB) + 2u;
                } else drained = true;
            }
        }
        if (__all_sync(0xffffffffu, drained)) break;
        if (!busy) continue;

        // one event: blocks each kernel runs with until something changes
        ++events;
        uint32_t btA = A.b, btB = B.b;
        if (A.idle == 0 && B.idle == 0 && phi_exceeds(cap.lo - A.rec.z, cap.hi - A.rec.w, B.rec.z, B.rec.w)) {
            if (kPolicy == ROOMIE_WALK_DETAILED_EQUAL) {
                const bool a_first = A.began <= B.began;
                btA = A.fit; btB = B.fit;
                if (btA == 0 && btB == 0) { if (a_first) btA = A.b; else btB = B.b; }
                else if (btA == 0) btB = B.b;
                else if (btB == 0) btA = A.b;
            } else {
                const bool a_first = kPolicy == ROOMIE_WALK_DETAILED_PRIORITY || A.began <= B.began;
                if (a_first) btB = remainder_blocks(A, B, sp);
                else btA = remainder_blocks(B, A, sp);
            }
        }
        const unsigned long long untilA = A.idle ? A.idle : btA == A.b ? A.full : btA ? div_ceil(A.left, btA, s_inv[btA]) : kNever;
        const unsigned long long untilB = B.idle ? B.idle : btB == B.b ? B.full : btB ? div_ceil(B.left, btB, s_inv[btB]) : kNever;
        const unsigned long long step = untilA < untilB ? untilA : untilB;
        now += step;
        advance<kPolicy>(A, btA, untilA, step, now, s_inv, sp);
        advance<kPolicy>(B, btB, untilB, step, now, s_inv, sp);
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
