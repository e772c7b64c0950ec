// Section 3.2 in full (adjusted occupancy, two-phase execution, partition policies) as a third walk
// mode.  Included by roomie_pairs.cu inside namespace roomie.
//
// Unlike the two Algorithm-1 walks, this one is stateful: a kernel slowed down by interference ends
// later, which shifts everything after it, so a walk cannot be cut into independent tiles.  One thread
// simulates one (pair, alignment) walk event by event, in double precision, reading the 16-byte records
// straight from global memory (L2-resident); parallelism comes from the number of walks.
//
// While the two active kernels' combined demand exceeds the SM (Eq. 2) each runs with the blocks b~
// the policy leaves it and progresses at the rate o~/o = b~/b; the interference ends when the first of
// them completes (two-phase execution) and the other carries on with what is left of it.  Gaps are not
// stretched.  The delay of a model is the time lost by its kernels; the run ends when either model
// has completed its last kernel.  Policies: EQUAL (half of every SM resource each), PRIORITY (the first
// model of the pair keeps its blocks, the other gets the remainder), FCFS (priority to the kernel that
// started earlier, the first model on a tie).  A kernel left without a block waits while the other runs
// at full occupancy.

struct DetailedArgs {
    LibView lib;
    PairSet ps;
    uint32_t slots, n_align;
    int start_filter;
    int policy;                 // ROOMIE_WALK_DETAILED_* value
    roomie_gpu_spec spec;
    WalkInfo* walks;
    TilePartial* partials;
};

struct BlockNeed { uint32_t wb, regs, smem, b; };

// b~ / b for b~ <= b <= kRateMax, correctly rounded by the host compiler: the progress rate of a kernel that
// keeps b~ of its b blocks.  One load instead of the double-precision division routine; larger b (more than
// 32 resident blocks per SM) take the division.
constexpr int kRateMax = 32;
struct RateTable {
    double v[(kRateMax + 1) * (kRateMax + 1)];
    constexpr RateTable() : v{} {
        for (int i = 0; i <= kRateMax; ++i)
            for (int j = 1; j <= kRateMax; ++j) v[i * (kRateMax + 1) + j] = (double)i / (double)j;
    }
};
__device__ const RateTable kRates = RateTable();
__device__ __forceinline__ double rate_of(uint32_t kept, uint32_t all) {
    if (all <= (uint32_t)kRateMax) return __ldg(&kRates.v[kept * (kRateMax + 1) + all]);
    return __ddiv_rn((double)kept, (double)all);
}

// floor(a / d) for a < 2^23, d >= 1 without the integer-division routine (about 20 instructions, several
// per simulated event): approximate float quotient, then one exact correction step in integers
__device__ __forceinline__ uint32_t div_floor(uint32_t a, uint32_t d) {
    uint32_t q = (uint32_t)__fdividef((float)a, (float)d);            // within 1 of the true quotient
    const int32_t r = (int32_t)a - (int32_t)(q * d);
    if (r < 0) --q;
    else if ((uint32_t)r >= d) ++q;
    return q;
}

__device__ __forceinline__ BlockNeed need_of(const uint4& r) {
    BlockNeed n;
    n.b = r.w >> 22;
    const uint32_t warps = r.z >> kWarpShift, regs = r.z & ((1u << kWarpShift) - 1u), smem = r.w & ((1u << 22) - 1u);
    n.wb = n.b ? div_floor(warps, n.b) : 0u;
    n.regs = n.b ? div_floor(regs, n.b) : 0u;
    n.smem = n.b ? div_floor(smem, n.b) : 0u;
    return n;
}

// blocks of a kernel that fit into the given amounts of the four resources, at most its own b
__device__ __forceinline__ uint32_t blocks_in(const BlockNeed& n, uint32_t warps, uint32_t regs, uint32_t smem,
                                              uint32_t slots) {
    uint32_t b = n.b;
    if (n.wb) b = min(b, div_floor(warps, n.wb));
    if (n.regs) b = min(b, div_floor(regs, n.regs));
    if (n.smem) b = min(b, div_floor(smem, n.smem));
    return min(b, slots);
}

__global__ void __launch_bounds__(128) detailed_walk_kernel(DetailedArgs g) {
    const unsigned long long w = (unsigned long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (w >= (unsigned long long)g.ps.n_pairs * g.slots) return;
    const uint32_t local = (uint32_t)(w / g.slots), c = (uint32_t)(w % g.slots);
    uint32_t a, b;
    pair_of(g.ps, g.lib.P, local, a, b);
    const uint32_t offa = g.lib.offsets[a], offb = g.lib.offsets[b];
    const uint32_t q[2] = {g.lib.offsets[a + 1] - offa, g.lib.offsets[b + 1] - offb};
    const uint32_t ga = grid_count(q[0], g.n_align), gb = grid_count(q[1], g.n_align);
    WalkInfo wi;
    wi.tile_base = (uint32_t)w; wi.n_tiles = 0; wi.length = 0; wi.valid = 0;
    TilePartial out;
    out.di = 0.0f; out.dj = 0.0f; out.V = 0; out.ties = 0; out.pad = 0;
    const uint32_t ca = c / gb, cb = c % gb;
    if (ca < ga) {
        const uint4* R[2] = {g.lib.records + offa, g.lib.records + offb};
        uint32_t k[2] = {grid_start(q[0], g.n_align, ca), grid_start(q[1], g.n_align, cb)};
        uint4 r[2] = {__ldg(&R[0][k[0]]), __ldg(&R[1][k[1]])};
        bool valid = true;
        if (g.start_filter) valid = phi_exceeds(g.lib.cap.lo - r[0].z, g.lib.cap.hi - r[0].w, r[1].z, r[1].w);
        if (valid) {
            const uint32_t W = g.spec.threads_per_sm / 32u, RG = g.spec.regs_per_sm, SM = g.spec.smem_per_sm,
                           BL = g.spec.blocks_per_sm;
            double work[2] = {(double)(r[0].y - r[0].x), (double)(r[1].y - r[1].x)};
            double gap[2] = {0.0, 0.0}, began[2] = {0.0, 0.0}, lost[2] = {0.0, 0.0}, now = 0.0;
            uint32_t ev = 0;
            while (k[0] < q[0] && k[1] < q[1]) {
                ++ev;
                double rate[2] = {1.0, 1.0};
                if (gap[0] <= 0.0 && gap[1] <= 0.0 &&
                    phi_exceeds(g.lib.cap.lo - r[0].z, g.lib.cap.hi - r[0].w, r[1].z, r[1].w)) {
                    const BlockNeed n0 = need_of(r[0]), n1 = need_of(r[1]);
                    uint32_t b0, b1;
                    if (g.policy == ROOMIE_WALK_DETAILED_EQUAL) {
                        b0 = blocks_in(n0, W / 2, RG / 2, SM / 2, BL / 2);
                        b1 = blocks_in(n1, W / 2, RG / 2, SM / 2, BL / 2);
                        if (b0 == 0 && b1 == 0) { if (began[0] <= began[1]) b0 = n0.b; else b1 = n1.b; }
                        else if (b0 == 0) b1 = n1.b;
                        else if (b1 == 0) b0 = n0.b;
                    } else {
                        const bool first0 = g.policy == ROOMIE_WALK_DETAILED_PRIORITY || began[0] <= began[1];
                        const BlockNeed& hi = first0 ? n0 : n1;
                        const BlockNeed& lo = first0 ? n1 : n0;
                        const uint32_t bl = blocks_in(lo, W - hi.wb * hi.b, RG - hi.regs * hi.b, SM - hi.smem * hi.b,
                                                      BL - hi.b);
                        b0 = first0 ? n0.b : bl;
                        b1 = first0 ? bl : n1.b;
                    }
                    rate[0] = rate_of(b0, n0.b);
                    rate[1] = rate_of(b1, n1.b);
                }
                double t[2];
#pragma unroll
                for (int m = 0; m < 2; ++m)
                    t[m] = gap[m] > 0.0 ? gap[m] : (rate[m] > 0.0 ? __ddiv_rn(work[m], rate[m]) : __longlong_as_double(0x7ff0000000000000LL));
                const double dt = t[0] < t[1] ? t[0] : t[1];
                now = __dadd_rn(now, dt);
#pragma unroll
                for (int m = 0; m < 2; ++m) {
                    if (gap[m] > 0.0) {
                        gap[m] = t[m] <= dt ? 0.0 : __dsub_rn(gap[m], dt);
                        if (gap[m] <= 0.0) began[m] = now;
                        continue;
                    }
                    lost[m] = __dadd_rn(lost[m], __dmul_rn(dt, __dsub_rn(1.0, rate[m])));
                    if (t[m] <= dt) {                               // this kernel completes
                        const uint4 done = r[m];
                        if (++k[m] < q[m]) {
                            r[m] = __ldg(&R[m][k[m]]);
                            gap[m] = (double)r[m].x - (double)done.y;
                            work[m] = (double)(r[m].y - r[m].x);
                            if (gap[m] <= 0.0) { gap[m] = 0.0; began[m] = now; }
                        }
                    } else {
                        work[m] = __dsub_rn(work[m], __dmul_rn(dt, rate[m]));
                    }
                }
            }
            out.di = (float)lost[0]; out.dj = (float)lost[1];
            wi.n_tiles = 1; wi.length = ev; wi.valid = 1;
        }
    }
    g.walks[w] = wi;
    g.partials[w] = out;
}
