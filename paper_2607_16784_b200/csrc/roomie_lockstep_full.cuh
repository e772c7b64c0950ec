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
// alignments).  For an even count the upper middle value comes out of the last digit pass as well: it is the same
// value, the next occupied bin of the last histogram, or - when the lower middle is the largest value under its
// 22-bit prefix - the smallest value above that prefix, which the pass tracks on the side.  Every pass recomputes the
// suffix sums; a suffix sum is accumulated in double and ranked as float.
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
    unsigned long long max_cells;  // upper bound of q_a * q_b over the pairs of the call (sets the size classes)
};

constexpr int kFullClasses = 4;   // size classes of the launch order, largest tables first

enum FullPass : int { kPassDigit0 = 0, kPassDigit1 = 1, kPassDigit2 = 2 };

struct FullSelect {               // state of the radix select of one direction
    uint32_t prefix;              // bits fixed so far
    uint32_t rank;                // rank still to find among the values that share the prefix
    uint32_t value_bits;          // after digit 2: the element of rank k1 (the lower middle)
    uint32_t upper_bits;          // after digit 2: the element of rank k1 + 1, if the count is even
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
// With `next_bin` the caller also learns whether the element of rank + 1 is in the same bin (next_bin = bin) or which
// is the next occupied bin (kFullBins when there is none).
__device__ __forceinline__ void full_locate(const uint32_t* hist, uint32_t rank, uint32_t* s_scan, uint32_t& bin,
                                            uint32_t& rank_in_bin, uint32_t* next_bin = nullptr) {
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
    if (next_bin) {
        if (rank_in_bin + 1 < hist[bin]) *next_bin = bin;
        else {
            // lowest occupied bin above `bin`: every thread proposes the first of its own bins, the minimum wins
            if (threadIdx.x == 0) s_scan[kFullThreads / 32] = kFullBins;
            __syncthreads();
            uint32_t cand = kFullBins;
#pragma unroll
            for (int k = kPer - 1; k >= 0; --k) {
                const uint32_t b = threadIdx.x * kPer + k;
                if (b > bin && h[k]) cand = b;
            }
            if (cand < (uint32_t)kFullBins) atomicMin(&s_scan[kFullThreads / 32], cand);
            __syncthreads();
            *next_bin = s_scan[kFullThreads / 32];
            __syncthreads();
        }
    }
}

__global__ void __launch_bounds__(kFullThreads) lockstep_full_kernel(FullArgs g) {
    __shared__ uint32_t s_hist[2][kFullBins];
    __shared__ uint32_t s_scan[kFullThreads / 32 + 2];
    __shared__ uint32_t s_gt[2];                     // per direction: smallest value above the 22-bit prefix
    __shared__ unsigned long long s_ev;
    __shared__ uint32_t s_n;
    extern __shared__ float s_inv[];

    // The grid is kFullClasses x n_pairs CTAs: CTA c * n_pairs + p takes pair p if the pair's table falls into size
    // class c (class 0: at least a quarter of the largest possible table, then a factor of four per class) and
    // leaves at once otherwise, so that the largest tables start first and the small ones fill the tail.
    {
        const uint32_t local = blockIdx.x % g.ps.n_pairs, cls = blockIdx.x / g.ps.n_pairs;
        uint32_t a, b;
        pair_of(g.ps, g.lib.P, local, a, b);
        const uint32_t offa = g.lib.offsets[a], offb = g.lib.offsets[b];
        const uint32_t na = g.lib.offsets[a + 1] - offa, nb = g.lib.offsets[b + 1] - offb;
        const unsigned long long cells = (unsigned long long)na * nb;
        uint32_t mine = kFullClasses - 1;
#pragma unroll
        for (int c = kFullClasses - 2; c >= 0; --c)
            if (cells >= (g.max_cells >> (2 * c + 2))) mine = c;
        if (mine != cls) return;
        for (uint32_t i = threadIdx.x; i < g.n_inv; i += kFullThreads) s_inv[i] = __ldg(&g.inv_table[i]);
        const uint4* A = g.lib.records + offa;
        const uint4* B = g.lib.records + offb;
        FullSelect sel[2] = {};
        uint32_t n = 0;
        for (int pass = kPassDigit0; pass <= kPassDigit2; ++pass) {
            for (uint32_t i = threadIdx.x; i < 2 * kFullBins; i += kFullThreads) (&s_hist[0][0])[i] = 0;
            if (threadIdx.x == 0) { s_ev = 0; s_n = 0; s_gt[0] = s_gt[1] = 0xffffffffu; }
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
            } else if (pass == kPassDigit1) {
                const uint32_t pi = sel[0].prefix, pj = sel[1].prefix;
                full_walk(A, B, na, nb, g.lib.cap, s_inv, g.start_filter, [&](uint32_t vi, uint32_t vj, uint32_t) {
                    if ((vi >> 21) == pi) atomicAdd(&s_hist[0][(vi >> 10) & 2047u], 1u);
                    if ((vj >> 21) == pj) atomicAdd(&s_hist[1][(vj >> 10) & 2047u], 1u);
                });
            } else {
                // last digit; on the side, the smallest value whose upper 22 bits lie above the prefix (the upper
                // middle of an even count when the lower middle is the largest value under the prefix)
                const uint32_t pi = sel[0].prefix, pj = sel[1].prefix;
                uint32_t gt_i = 0xffffffffu, gt_j = 0xffffffffu;
                full_walk(A, B, na, nb, g.lib.cap, s_inv, g.start_filter, [&](uint32_t vi, uint32_t vj, uint32_t) {
                    const uint32_t ui = vi >> 10, uj = vj >> 10;
                    if (ui == pi) atomicAdd(&s_hist[0][vi & 1023u], 1u); else if (ui > pi) gt_i = min(gt_i, vi);
                    if (uj == pj) atomicAdd(&s_hist[1][vj & 1023u], 1u); else if (uj > pj) gt_j = min(gt_j, vj);
                });
                if (gt_i != 0xffffffffu) atomicMin(&s_gt[0], gt_i);
                if (gt_j != 0xffffffffu) atomicMin(&s_gt[1], gt_j);
            }
            __syncthreads();
            if (pass == kPassDigit0) {
                n = s_n;
                if (threadIdx.x == 0 && g.evals_out && s_ev) atomicAdd(g.evals_out, s_ev);
                if (n == 0) break;
                sel[0].rank = sel[1].rank = (n - 1) / 2;
            }
            const int bits = pass == kPassDigit2 ? 10 : 11;
            for (int dir = 0; dir < 2; ++dir) {
                uint32_t bin, r, next = 0;
                full_locate(s_hist[dir], sel[dir].rank, s_scan, bin, r, pass == kPassDigit2 ? &next : nullptr);
                const uint32_t group = sel[dir].prefix;                  // the bits fixed before this pass
                sel[dir].prefix = (group << bits) | bin;
                sel[dir].rank = r;
                if (pass == kPassDigit2) {
                    sel[dir].value_bits = sel[dir].prefix;
                    sel[dir].upper_bits = next < (uint32_t)kFullBins ? ((group << 10) | next) : s_gt[dir];
                }
            }
            __syncthreads();
        }
        if (threadIdx.x == 0) {
            float med[2] = {0.0f, 0.0f};
            if (n > 0) {
                for (int dir = 0; dir < 2; ++dir) {
                    const float lo = __uint_as_float(sel[dir].value_bits);
                    const float hi = (n & 1u) ? lo : __uint_as_float(sel[dir].upper_bits);   // odd count: one middle
                    med[dir] = 0.5f * (lo + hi);
                }
            }
            store_pair_values(g.lib, g.ps, g.P_out, a, b, na, nb, med[0], med[1]);
        }
        __syncthreads();
    }
}
