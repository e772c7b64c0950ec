// Algorithm 1 as printed with the FULL alignment set: every pair of start indices (s_i, s_j) of the
// Cartesian product (optionally only those whose start kernels interfere), lock-step walk, median.
// Included by roomie_pairs.cu inside namespace roomie.
//
// The delay of alignment (s_i, s_j) is the sum of the charged terms along the diagonal that starts
// at (s_i, s_j):  delta_i(s_i, s_j) = sum_t hit(s_i+t, s_j+t) * d_{s_i+t} * o_i/(o_i+o_j), so all
// q_i*q_j alignments of a pair are the suffix sums along the q_i+q_j-1 diagonals of one q_i x q_j
// table: q_i*q_j work instead of q_i*q_j*min(q).  The table is never stored: one thread walks four
// neighbouring diagonals from their far ends (a suffix sum is accumulated in double and ranked as float) and the
// values go straight into an exact radix select over the float bits, which order like the non-negative values:
//
//   pass 1 over the table   histogram of the upper 13 bits; it also counts the kept alignments
//   pass 2 over the table   the values that share the median's upper 13 bits (a few per cent of the table, their
//                           number known from pass 1) are appended to a list in the CTA's part of the workspace
//   two passes over the list  the next 10 and the last 9 bits
//
// When the list does not fit (no workspace, or a table dominated by one value) the last two digits are passes over
// the table as well.  For an even count the upper middle value comes out of the last digit pass: it is the same
// value, the next occupied bin of the last histogram, or the smallest value above the prefix, which the passes track
// on the side.
//
// One CTA per pair, both directions (delta_i, delta_j) selected in the same passes.  With a workspace the grid is
// persistent (two CTAs per SM) and takes the pairs from a counter, largest tables first.

constexpr int kFullThreads = 512;
constexpr int kFullBits0 = 13, kFullBits1 = 10, kFullBits2 = 9;   // digits of the select, upper bits first
constexpr int kFullBins = 1 << kFullBits0;                        // the widest histogram
constexpr int kFullClasses = 4;                                   // size classes of the order of work, largest tables first
constexpr uint32_t kFullMinList = 1024;                           // a list shorter than this per CTA and direction is not worth having

struct FullArgs {
    LibView lib;
    PairSet ps;
    int start_filter;
    uint32_t n_inv;               // 2W + 1: the table of 1/s is built on chip
    float* P_out;
    unsigned long long* evals_out;
    unsigned long long max_cells; // upper bound of q_a * q_b over the pairs of the call (sets the size classes)
    uint32_t* work_counter;       // next item of work (zeroed by the host), or null: item = blockIdx.x
    uint32_t* lists;              // [gridDim.x][2][list_cap] float bits, or null
    uint32_t list_cap;
};

struct FullSelect {               // state of the radix select of one direction
    uint32_t prefix;              // bits fixed so far
    uint32_t rank;                // rank still to find among the values that share the prefix
    uint32_t value_bits;          // after the last digit: the element of rank k1 (the lower middle)
    uint32_t upper_bits;          // after the last digit: the element of rank k1 + 1, if the count is even
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
    double x;                     // duration in ticks * warps
};

__device__ __forceinline__ FullRec full_rec(const uint4& r) {
    FullRec f;
    f.lo = r.z; f.hi = r.w;
    f.w = r.z >> kWarpShift;
    f.x = (double)((unsigned long long)(r.y - r.x) * f.w);
    return f;
}

template <class Visit>
__device__ __forceinline__ void full_walk(const uint4* __restrict__ A, const uint4* __restrict__ B, uint32_t na,
                                          uint32_t nb, PhiCap cap, const double* s_inv, int start_filter,
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
                        const double inv = s_inv[ra.w + rb[m].w];
                        si[m] = fma(ra.x, inv, si[m]);
                        sj[m] = fma(rb[m].x, inv, sj[m]);
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

// finds the bin that holds the element of rank `rank` in hist[0 .. 1 << bits); every thread gets the bin, the rank
// inside it and the bin's count.  s_scan: kFullThreads/32 + 3 words of shared scratch.  With `next_bin` the caller
// also learns whether the element of rank + 1 is in the same bin (next_bin = bin) or which is the next occupied
// bin (1 << bits when there is none).
__device__ __forceinline__ void full_locate(const uint32_t* hist, int bits, uint32_t rank, uint32_t* s_scan,
                                            uint32_t& bin, uint32_t& rank_in_bin, uint32_t& count_in_bin,
                                            uint32_t* next_bin = nullptr) {
    const uint32_t nbins = 1u << bits;
    const uint32_t per = (nbins + kFullThreads - 1) / kFullThreads;                // bins per thread
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    const uint32_t first = threadIdx.x * per;
    uint32_t mine = 0;
    for (uint32_t k = 0; k < per; ++k) mine += first + k < nbins ? hist[first + k] : 0u;
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
        uint32_t r = rank - before, k = first;
        while (r >= hist[k]) { r -= hist[k]; ++k; }
        s_scan[kFullThreads / 32] = k;
        s_scan[kFullThreads / 32 + 1] = r;
        s_scan[kFullThreads / 32 + 2] = nbins;                      // next occupied bin, filled in below
    }
    __syncthreads();
    bin = s_scan[kFullThreads / 32];
    rank_in_bin = s_scan[kFullThreads / 32 + 1];
    count_in_bin = hist[bin];
    if (next_bin) {
        if (rank_in_bin + 1 < count_in_bin) *next_bin = bin;
        else {
            // lowest occupied bin above `bin`: every thread proposes the first of its own bins, the minimum wins
            uint32_t cand = nbins;
            for (uint32_t k = per; k-- > 0;) {
                const uint32_t b = first + k;
                if (b < nbins && b > bin && hist[b]) cand = b;
            }
            if (cand < nbins) atomicMin(&s_scan[kFullThreads / 32 + 2], cand);
            __syncthreads();
            *next_bin = s_scan[kFullThreads / 32 + 2];
        }
    }
    __syncthreads();
}

// appends v to the list; the lanes that come here together share one addition to the cursor
__device__ __forceinline__ void full_append(uint32_t* list, uint32_t cap, uint32_t* cursor, uint32_t v) {
    const uint32_t active = __activemask();
    const int lane = threadIdx.x & 31, leader = __ffs(active) - 1;
    uint32_t base = 0;
    if (lane == leader) base = atomicAdd(cursor, (uint32_t)__popc(active));
    base = __shfl_sync(active, base, leader);
    const uint32_t at = base + __popc(active & ((1u << lane) - 1u));
    if (at < cap) list[at] = v;
}

struct FullShared {
    uint32_t hist[2][kFullBins];
    uint32_t scan[kFullThreads / 32 + 3];
    uint32_t gt[2];               // per direction: smallest value above the prefix of the pass
    uint32_t cursor[2];           // lengths of the two lists
    uint32_t n;
    uint32_t item;
    unsigned long long ev;
};

__device__ __forceinline__ void full_clear(FullShared& sh, int bits) {
    for (uint32_t i = threadIdx.x; i < (1u << bits); i += kFullThreads) { sh.hist[0][i] = 0; sh.hist[1][i] = 0; }
    if (threadIdx.x == 0) { sh.gt[0] = sh.gt[1] = 0xffffffffu; sh.cursor[0] = sh.cursor[1] = 0; }
}

// the select of one pair; every thread of the CTA calls it
__device__ __forceinline__ void full_pair(const FullArgs& g, FullShared& sh, const double* s_inv, uint32_t a,
                                          uint32_t b, uint32_t offa, uint32_t offb, uint32_t na, uint32_t nb) {
    const uint4* A = g.lib.records + offa;
    const uint4* B = g.lib.records + offb;
    FullSelect sel[2] = {};
    // ---- pass 1 over the table: first digit, count, walk lengths
    full_clear(sh, kFullBits0);
    if (threadIdx.x == 0) { sh.ev = 0; sh.n = 0; }
    __syncthreads();
    {
        uint32_t cnt = 0;
        unsigned long long ev = 0;
        full_walk(A, B, na, nb, g.lib.cap, s_inv, g.start_filter, [&](uint32_t vi, uint32_t vj, uint32_t len) {
            ++cnt; ev += len;
            atomicAdd(&sh.hist[0][vi >> (32 - kFullBits0)], 1u);
            atomicAdd(&sh.hist[1][vj >> (32 - kFullBits0)], 1u);
        });
        atomicAdd(&sh.n, cnt);
        atomicAdd(&sh.ev, ev);
    }
    __syncthreads();
    const uint32_t n = sh.n;
    if (threadIdx.x == 0 && g.evals_out && sh.ev) atomicAdd(g.evals_out, sh.ev);
    if (n == 0) {                                                  // no alignment kept: both medians are zero
        if (threadIdx.x == 0) store_pair_values(g.lib, g.ps, g.P_out, a, b, na, nb, 0.0f, 0.0f);
        __syncthreads();
        return;
    }
    uint32_t in_bin[2];
    for (int dir = 0; dir < 2; ++dir) {
        uint32_t bin, r;
        full_locate(sh.hist[dir], kFullBits0, (n - 1) / 2, sh.scan, bin, r, in_bin[dir]);
        sel[dir].prefix = bin; sel[dir].rank = r;
    }
    const bool listed = g.lists && in_bin[0] <= g.list_cap && in_bin[1] <= g.list_cap;
    uint32_t* list_i = listed ? g.lists + (size_t)blockIdx.x * 2 * g.list_cap : nullptr;
    uint32_t* list_j = listed ? list_i + g.list_cap : nullptr;
    if (listed) {
        // ---- pass 2 over the table: the values under the first digit's prefix go to the lists
        full_clear(sh, 0);
        __syncthreads();
        const uint32_t pi = sel[0].prefix, pj = sel[1].prefix;
        full_walk(A, B, na, nb, g.lib.cap, s_inv, g.start_filter, [&](uint32_t vi, uint32_t vj, uint32_t) {
            if ((vi >> (32 - kFullBits0)) == pi) full_append(list_i, g.list_cap, &sh.cursor[0], vi);
            if ((vj >> (32 - kFullBits0)) == pj) full_append(list_j, g.list_cap, &sh.cursor[1], vj);
        });
        __syncthreads();
    }
    // ---- the two remaining digits: over the lists, or over the table again
    for (int digit = 1; digit <= 2; ++digit) {
        const int bits = digit == 1 ? kFullBits1 : kFullBits2;
        const int low = digit == 1 ? kFullBits2 : 0;                // bits below this digit
        const uint32_t mask = (1u << bits) - 1u;
        full_clear(sh, bits);
        __syncthreads();
        const uint32_t pi = sel[0].prefix, pj = sel[1].prefix;
        uint32_t gt_i = 0xffffffffu, gt_j = 0xffffffffu;
        if (listed) {
            for (uint32_t e = threadIdx.x; e < in_bin[0]; e += kFullThreads) {
                const uint32_t v = list_i[e], u = v >> (low + bits);
                if (u == pi) atomicAdd(&sh.hist[0][(v >> low) & mask], 1u); else if (u > pi) gt_i = min(gt_i, v);
            }
            for (uint32_t e = threadIdx.x; e < in_bin[1]; e += kFullThreads) {
                const uint32_t v = list_j[e], u = v >> (low + bits);
                if (u == pj) atomicAdd(&sh.hist[1][(v >> low) & mask], 1u); else if (u > pj) gt_j = min(gt_j, v);
            }
        } else {
            full_walk(A, B, na, nb, g.lib.cap, s_inv, g.start_filter, [&](uint32_t vi, uint32_t vj, uint32_t) {
                const uint32_t ui = vi >> (low + bits), uj = vj >> (low + bits);
                if (ui == pi) atomicAdd(&sh.hist[0][(vi >> low) & mask], 1u); else if (ui > pi) gt_i = min(gt_i, vi);
                if (uj == pj) atomicAdd(&sh.hist[1][(vj >> low) & mask], 1u); else if (uj > pj) gt_j = min(gt_j, vj);
            });
        }
        if (gt_i != 0xffffffffu) atomicMin(&sh.gt[0], gt_i);
        if (gt_j != 0xffffffffu) atomicMin(&sh.gt[1], gt_j);
        __syncthreads();
        for (int dir = 0; dir < 2; ++dir) {
            uint32_t bin, r, cnt, next = 0;
            full_locate(sh.hist[dir], bits, sel[dir].rank, sh.scan, bin, r, cnt, digit == 2 ? &next : nullptr);
            const uint32_t group = sel[dir].prefix;                  // the bits fixed before this pass
            sel[dir].prefix = (group << bits) | bin;
            sel[dir].rank = r;
            if (digit == 2) {
                // the element of rank + 1: same value, next occupied bin, smallest value above the prefix of this
                // pass (none: all ones; over the list that is only the part under the first digit, see below)
                sel[dir].value_bits = sel[dir].prefix;
                sel[dir].upper_bits = next <= mask ? ((group << bits) | next) : sh.gt[dir];
            }
        }
        __syncthreads();
    }
    if (listed && !(n & 1u) && (sel[0].upper_bits == 0xffffffffu || sel[1].upper_bits == 0xffffffffu)) {
        // the lower middle is the largest value under its first digit, so the upper middle is not in the list: it is
        // the smallest value of the table above that digit's bin (one more pass; with thousands of values per bin
        // this hardly ever happens)
        full_clear(sh, 0);
        __syncthreads();
        const uint32_t pi = sel[0].value_bits >> (32 - kFullBits0), pj = sel[1].value_bits >> (32 - kFullBits0);
        uint32_t gt_i = 0xffffffffu, gt_j = 0xffffffffu;
        full_walk(A, B, na, nb, g.lib.cap, s_inv, g.start_filter, [&](uint32_t vi, uint32_t vj, uint32_t) {
            if ((vi >> (32 - kFullBits0)) > pi) gt_i = min(gt_i, vi);
            if ((vj >> (32 - kFullBits0)) > pj) gt_j = min(gt_j, vj);
        });
        if (gt_i != 0xffffffffu) atomicMin(&sh.gt[0], gt_i);
        if (gt_j != 0xffffffffu) atomicMin(&sh.gt[1], gt_j);
        __syncthreads();
        for (int dir = 0; dir < 2; ++dir)
            if (sel[dir].upper_bits == 0xffffffffu) sel[dir].upper_bits = sh.gt[dir];
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        float med[2];
        for (int dir = 0; dir < 2; ++dir) {
            const float lo = __uint_as_float(sel[dir].value_bits);
            const float hi = (n & 1u) ? lo : __uint_as_float(sel[dir].upper_bits);   // odd count: one middle
            med[dir] = 0.5f * (lo + hi);
        }
        store_pair_values(g.lib, g.ps, g.P_out, a, b, na, nb, med[0], med[1]);
    }
    __syncthreads();
}

// Items of work: item c * n_pairs + p is pair p if the pair's table falls into size class c (class 0: at least a
// quarter of the largest possible table, then a factor of four per class) and nothing otherwise, so that the largest
// tables start first and the small ones fill the tail.
__global__ void __launch_bounds__(kFullThreads, 2) lockstep_full_kernel(FullArgs g) {
    extern __shared__ __align__(16) unsigned char full_smem[];
    FullShared& sh = *reinterpret_cast<FullShared*>(full_smem);
    double* s_inv = reinterpret_cast<double*>(full_smem + sizeof(FullShared));   // 1/s, s = 1 .. 2W (0 never interferes)
    for (uint32_t i = threadIdx.x; i < g.n_inv; i += kFullThreads) s_inv[i] = i ? 1.0 / (double)i : 0.0;
    __syncthreads();
    const unsigned long long n_items = (unsigned long long)kFullClasses * g.ps.n_pairs;
    for (unsigned long long item = blockIdx.x;; item += gridDim.x) {
        if (g.work_counter) {
            if (threadIdx.x == 0) sh.item = atomicAdd(g.work_counter, 1u);
            __syncthreads();
            item = sh.item;
            __syncthreads();
        }
        if (item >= n_items) break;
        const uint32_t local = (uint32_t)(item % g.ps.n_pairs), cls = (uint32_t)(item / g.ps.n_pairs);
        uint32_t a, b;
        pair_of(g.ps, g.lib.P, local, a, b);
        const uint32_t offa = g.lib.offsets[a], offb = g.lib.offsets[b];
        const uint32_t na = g.lib.offsets[a + 1] - offa, nb = g.lib.offsets[b + 1] - offb;
        const unsigned long long cells = (unsigned long long)na * nb;
        uint32_t mine = kFullClasses - 1;
#pragma unroll
        for (int c = kFullClasses - 2; c >= 0; --c)
            if (cells >= (g.max_cells >> (2 * c + 2))) mine = c;
        if (mine == cls) full_pair(g, sh, s_inv, a, b, offa, offb, na, nb);
    }
}
