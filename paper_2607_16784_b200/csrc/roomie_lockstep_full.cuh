// Algorithm 1 as printed with the FULL alignment set: every pair of start indices (s_i, s_j) of the
// Cartesian product (optionally only those whose start kernels interfere), lock-step walk, median.
// Included by roomie_pairs.cu inside namespace roomie.
//
// The delay of alignment (s_i, s_j) is the sum of the charged terms along the diagonal that starts
// at (s_i, s_j):  delta_i(s_i, s_j) = sum_t hit(s_i+t, s_j+t) * d_{s_i+t} * o_i/(o_i+o_j), so all
// q_i*q_j alignments of a pair are the suffix sums along the q_i+q_j-1 diagonals of one q_i x q_j
// table: q_i*q_j work instead of q_i*q_j*min(q).  The table is never stored: one thread walks four
// neighbouring diagonals from their far ends and the values go
// straight into the histogram of an exact radix select (3 digit passes of 11/11/10 bits over the
// float bits, which order like the non-negative values - the first one also counts the kept
// alignments - plus, for an even count, a pass for the upper middle value).  Every pass recomputes the suffix sums; a suffix sum is accumulated in double
// and ranked as float.
//
// One CTA per pair; both directions (delta_i, delta_j) are selected in the same passes.

constexpr int kFullThreads = 512;
constexpr int kFullBins = 2048;

struct FullArgs {
    LibView lib;
    PairSet ps;
    int start_filter;
    const float* inv_table;       // 1/s, s <= 2W
    uint32_t n_inv;
    float* P_out;
    unsigned long long* evals_out;
};

enum FullPass : int { kPassDigit0 = 0, kPassDigit1 = 1, kPassDigit2 = 2, kPassUpper = 3 };

struct FullSelect {               // state of the radix select of one direction
    uint32_t prefix;              // bits fixed so far
    uint32_t rank;                // rank still to find among the values that share the prefix
    uint32_t value_bits;          // after digit 2: the element of rank k1
    uint32_t count_le;            // pass kPassUpper: values <= value
    uint32_t min_gt;              // pass kPassUpper: smallest value bits above value
};

// walks every diagonal of the pair once; `visit(vi_bits, vj_bits, walk_len)` is called for every
// kept alignment with the float bits of its two delays and the length of its walk.
// One thread takes kDiags neighbouring diagonals at a time and moves up the table row by row: row i
// pairs A[i] with B[i - off - m], m = 0..kDiags-1, and the next row needs only one new record of each
// profile (the B records slide along a register window), so a cell costs half a record load and the
// per-record conversions (duration * warps as float) are done once per record, not once per cell.
constexpr int kDiags = 4;

struct FullRec {                  // what a cell needs of one kernel
    uint32_t lo, hi;              // packed demand
    uint32_t w;                   // resident warps
    float x;                      // duration in ticks * warps
};

__device__ __forceinline__ FullRec full_rec(const uint4& r) {
    FullRec f;
    f.lo = r.z; f.hi = r.w;
    f.w = r.z >> kWarpShift;
    f.x = (float)(r.y - r.x) * small_int_to_float(f.w);
    return f;
}

template <class Visit>
__device__ __forceinline__ void full_walk(const uint4* __restrict__ A, const uint4* __restrict__ B, uint32_t na,
                                          uint32_t nb, PhiCap cap, const float* s_inv, int start_filter,
                                          Visit visit) {
    const int32_t n_diag = (int32_t)(na + nb - 1);
    const int32_t n_groups = (n_diag + kDiags - 1) / kDiags;
    const int32_t last_a = (int32_t)na - 1, last_b = (int32_t)nb - 1;
    for (int32_t grp = (int32_t)threadIdx.x; grp < n_groups; grp += kFullThreads) {
        // diagonal m of the group holds the cells (i, j) with i - j = off + m
        const int32_t off = grp * kDiags - last_b;
        const int32_t i_top = min(last_a, last_b + off + kDiags - 1);      // highest row any of them reaches
        const int32_t i_bot = max(0, off);                                  // lowest row any of them reaches
        double si[kDiags], sj[kDiags];
        uint32_t len[kDiags];
        FullRec rb[kDiags];
#pragma unroll
        for (int m = 0; m < kDiags; ++m) {
            si[m] = 0.0; sj[m] = 0.0; len[m] = 0;
            const int32_t j = i_top - off - m;
            rb[m] = full_rec(__ldg(&B[min(max(j, 0), last_b)]));             // out-of-range cells are skipped below
        }
        for (int32_t i = i_top; i >= i_bot; --i) {
            const FullRec ra = full_rec(__ldg(&A[i]));
#pragma unroll
            for (int m = 0; m < kDiags; ++m) {
                const int32_t j = i - off - m;
                if (j >= 0 && j <= last_b) {                               // cell (i, j) exists (j < 0 also ends short groups)
                    ++len[m];
                    const bool hit = phi_exceeds(cap.lo - ra.lo, cap.hi - ra.hi, rb[m].lo, rb[m].hi);
                    if (hit) {
                        const float inv = s_inv[ra.w + rb[m].w];
                        si[m] += (double)(ra.x * inv);
                        sj[m] += (double)(rb[m].x * inv);
                    }
                    if (!start_filter || hit) visit(__float_as_uint((float)si[m]), __float_as_uint((float)sj[m]), len[m]);
                }
            }
            // next row: diagonal m meets the record diagonal m + 1 met in this row
#pragma unroll
            for (int m = 0; m + 1 < kDiags; ++m) rb[m] = rb[m + 1];
            const int32_t jn = i - 1 - off - (kDiags - 1);
            rb[kDiags - 1] = full_rec(__ldg(&B[min(max(jn, 0), last_b)]));
        }
    }
}

// finds the bin that holds the element of rank `rank` in hist[0..kFullBins); every thread gets the
// bin and the rank inside it.  s_scan: kFullThreads/32 + 2 words of shared scratch.
__device__ __forceinline__ void full_locate(const uint32_t* hist, uint32_t rank, uint32_t* s_scan, uint32_t& bin,
                                            uint32_t& rank_in_bin) {
    constexpr int kPer = kFullBins / kFullThreads;                 // bins per thread
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    uint32_t h[kPer], mine = 0;
#pragma unroll
    for (int k = 0; k < kPer; ++k) { h[k] = hist[threadIdx.x * kPer + k]; mine += h[k]; }
    uint32_t incl = mine;
#pragma unroll
    for (int s = 1; s < 32; s <<= 1) {
        const uint32_t up = __shfl_up_sync(0xffffffffu, incl, s);
        if (lane >= s) incl += up;
    }
    if (lane == 31) s_scan[wid] = incl;
    __syncthreads();
    uint32_t before = incl - mine;
    for (int w = 0; w < wid; ++w) before += s_scan[w];
    if (rank >= before && rank < before + mine) {                  // exactly one thread
        uint32_t r = rank - before;
        int k = 0;
        while (r >= h[k]) { r -= h[k]; ++k; }
        s_scan[kFullThreads / 32] = threadIdx.x * kPer + k;
        s_scan[kFullThreads / 32 + 1] = r;
    }
    __syncthreads();
    bin = s_scan[kFullThreads / 32];
    rank_in_bin = s_scan[kFullThreads / 32 + 1];
    __syncthreads();
}

__global__ void __launch_bounds__(kFullThreads) lockstep_full_kernel(FullArgs g) {
    __shared__ uint32_t s_hist[2][kFullBins];
    __shared__ uint32_t s_scan[kFullThreads / 32 + 2];
    __shared__ uint32_t s_red[4];                    // count_le_i, count_le_j, min_gt_i, min_gt_j
    __shared__ unsigned long long s_ev;
    __shared__ uint32_t s_n;
    extern __shared__ float s_inv[];

    for (uint32_t i = threadIdx.x; i < g.n_inv; i += kFullThreads) s_inv[i] = __ldg(&g.inv_table[i]);
    for (uint32_t local = blockIdx.x; local < g.ps.n_pairs; local += gridDim.x) {
        uint32_t a, b;
        pair_of(g.ps, g.lib.P, local, a, b);
        const uint32_t offa = g.lib.offsets[a], offb = g.lib.offsets[b];
        const uint32_t na = g.lib.offsets[a + 1] - offa, nb = g.lib.offsets[b + 1] - offb;
        const uint4* A = g.lib.records + offa;
        const uint4* B = g.lib.records + offb;
        FullSelect sel[2] = {};
        uint32_t n = 0;
        for (int pass = kPassDigit0; pass <= kPassUpper; ++pass) {
            for (uint32_t i = threadIdx.x; i < 2 * kFullBins; i += kFullThreads) (&s_hist[0][0])[i] = 0;
            if (threadIdx.x == 0) { s_ev = 0; s_n = 0; s_red[0] = s_red[1] = 0; s_red[2] = s_red[3] = 0xffffffffu; }
            __syncthreads();
            if (pass == kPassDigit0) {                                   // first digit, count and walk lengths
                uint32_t cnt = 0;
                unsigned long long ev = 0;
                full_walk(A, B, na, nb, g.lib.cap, s_inv, g.start_filter, [&](uint32_t vi, uint32_t vj, uint32_t len) {
                    ++cnt; ev += len;
                    atomicAdd(&s_hist[0][vi >> 21], 1u);
                    atomicAdd(&s_hist[1][vj >> 21], 1u);
                });
                atomicAdd(&s_n, cnt);
                atomicAdd(&s_ev, ev);
            } else if (pass <= kPassDigit2) {
                const int shift = pass == kPassDigit1 ? 10 : 0;
                const uint32_t mask = pass == kPassDigit2 ? 1023u : 2047u;
                const int pshift = pass == kPassDigit1 ? 21 : 10;        // bits already fixed: v >> pshift
                const uint32_t pi = sel[0].prefix, pj = sel[1].prefix;
                full_walk(A, B, na, nb, g.lib.cap, s_inv, g.start_filter, [&](uint32_t vi, uint32_t vj, uint32_t) {
                    if ((vi >> pshift) == pi) atomicAdd(&s_hist[0][(vi >> shift) & mask], 1u);
                    if ((vj >> pshift) == pj) atomicAdd(&s_hist[1][(vj >> shift) & mask], 1u);
                });
            } else {
                const uint32_t ti = sel[0].value_bits, tj = sel[1].value_bits;
                uint32_t le_i = 0, le_j = 0, gt_i = 0xffffffffu, gt_j = 0xffffffffu;
                full_walk(A, B, na, nb, g.lib.cap, s_inv, g.start_filter, [&](uint32_t vi, uint32_t vj, uint32_t) {
                    if (vi <= ti) ++le_i; else gt_i = min(gt_i, vi);
                    if (vj <= tj) ++le_j; else gt_j = min(gt_j, vj);
                });
                atomicAdd(&s_red[0], le_i); atomicAdd(&s_red[1], le_j);
                atomicMin(&s_red[2], gt_i); atomicMin(&s_red[3], gt_j);
            }
            __syncthreads();
            if (pass == kPassDigit0) {
                n = s_n;
                if (threadIdx.x == 0 && g.evals_out && s_ev) atomicAdd(g.evals_out, s_ev);
                if (n == 0) break;
                sel[0].rank = sel[1].rank = (n - 1) / 2;
            }
            if (pass <= kPassDigit2) {
                const int bits = pass == kPassDigit2 ? 10 : 11;
                for (int dir = 0; dir < 2; ++dir) {
                    uint32_t bin, r;
                    full_locate(s_hist[dir], sel[dir].rank, s_scan, bin, r);
                    sel[dir].prefix = (sel[dir].prefix << bits) | bin;
                    sel[dir].rank = r;
                }
                if (pass == kPassDigit2) {
                    sel[0].value_bits = sel[0].prefix; sel[1].value_bits = sel[1].prefix;
                    sel[0].count_le = sel[1].count_le = n;               // odd count: both middles are this element
                    if (n & 1u) break;
                }
            } else {
                sel[0].count_le = s_red[0]; sel[1].count_le = s_red[1];
                sel[0].min_gt = s_red[2]; sel[1].min_gt = s_red[3];
            }
            __syncthreads();
        }
        if (threadIdx.x == 0) {
            float med[2] = {0.0f, 0.0f};
            if (n > 0) {
                const uint32_t k2 = n / 2;                         // upper middle (equals the lower one for odd n)
                for (int dir = 0; dir < 2; ++dir) {
                    const float lo = __uint_as_float(sel[dir].value_bits);
                    const float hi = k2 < sel[dir].count_le ? lo : __uint_as_float(sel[dir].min_gt);
                    med[dir] = 0.5f * (lo + hi);
                }
            }
            store_pair_values(g.lib, g.ps, g.P_out, a, b, na, nb, med[0], med[1]);
        }
        __syncthreads();
    }
}
