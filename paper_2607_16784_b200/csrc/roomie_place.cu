// Greedy multi-model estimate (Algorithm 1, outer loops) and placement (Algorithm 2).
#include "roomie_common.cuh"

namespace roomie {

// ---------------------------------------------------------------------------------------
// K4: performance_drop(M) from the pairwise matrix, one thread per model set.
// All sums are float32 additions in slot order, incoming model last, never contracted.
// ---------------------------------------------------------------------------------------
__global__ void __launch_bounds__(128) multi_estimate_kernel(const float* __restrict__ Pm, uint32_t P,
                                                             const int32_t* __restrict__ ids,
                                                             const uint32_t* __restrict__ count,
                                                             const int32_t* __restrict__ incoming, uint32_t n_sets,
                                                             uint32_t R, float* mu_out, float* mean_out) {
    const uint32_t s = blockIdx.x * blockDim.x + threadIdx.x;
    if (s >= n_sets) return;
    const uint32_t c = min(count[s], R);
    const int32_t* my = ids + (size_t)s * R;
    const int32_t inc = incoming[s];
    float tot = 0.0f;
    for (uint32_t i = 0; i <= c; ++i) {
        const int32_t mi = i < c ? my[i] : inc;
        const float* row = Pm + (size_t)mi * P;
        float mu = 0.0f;
        for (uint32_t j = 0; j <= c; ++j) {
            if (j == i) continue;
            const int32_t mj = j < c ? my[j] : inc;
            mu = __fadd_rn(mu, __ldg(row + mj));
        }
        if (mu_out) mu_out[(size_t)s * (R + 1) + i] = mu;
        tot = __fadd_rn(tot, mu);
    }
    if (mean_out) mean_out[s] = __fdiv_rn(tot, (float)(c + 1));
}

// ---------------------------------------------------------------------------------------
// K5: the arrival stream is a dependent chain (each decision changes the state the next one
// sees), so one CTA walks it with one thread per modelled GPU and the whole state in shared
// memory.  What keeps the chain short:
//   - per GPU and resident, the sum over the other residents is cached (`partial`); adding the
//     arrival's term last reproduces the slot-order float32 sum exactly, so a what-if costs two
//     matrix reads per resident;
//   - the matrix row and column of the arrivals two steps ahead are fetched into a 4-deep
//     shared-memory ring with cp.async while the current arrival is scored (or the whole matrix
//     sits in shared memory when it fits);
//   - the pairwise terms between the residents of a GPU are kept in shared memory, so that a
//     departure re-sums the cached values without touching the matrix;
//   - one barrier per arrival: warp argmin by two redux steps, cross-warp through a
//     double-buffered slot array.
// State arrays are slot-major in shared memory (slot * G + gpu) so that the threads of a warp
// touch consecutive banks.
// ---------------------------------------------------------------------------------------
struct PlaceArgs {
    const float* Pm;
    uint32_t P;
    uint32_t G, R;
    int32_t* ids;
    uint32_t* expiry;
    uint32_t* count;
    uint32_t* tick;
    const int32_t* arr_id;
    const uint32_t* arr_life;
    uint32_t n;
    float lambda;
    int32_t* gpu_out;
    float* mean_out;
    float* mu_arr_out;
    int matrix_mode;        // 0: whole matrix in shared memory, 1: row/column ring, 2: global loads
    int pair_cache;         // 1: resident-resident terms cached in shared memory ([R][R][G] floats)
    uint32_t gpus_per_warp; // fast kernel: GPUs owned by each warp
    int admit_rule;         // 0: mean drop < lambda, 1: largest member drop < lambda
    int objective;          // 0: lowest mean drop, 1: lowest largest drop, 2: lowest drop of the arrival
    uint32_t chunk;         // fast kernel: arrivals staged in shared memory at a time (<= kArrChunk)
    // A long single stream is served by whichever of two kernels suits its admission rate (see place_impl): the
    // kernels are launched in turn, and the one that is running hands the rest of the stream to the next launch
    // when the other kind has become the faster one.
    int32_t* mailbox;        // where a kernel leaves the hand-over for the next launch (the stream's last gpu_out
                             // element, which holds a decision once the stream is done), or null
    int32_t my_kind;         // 0: one lane per modelled GPU, 1: one lane per resident slot
    int32_t first;           // 1: the first launch (starts at arrival 0 without looking at the mailbox)
    int32_t may_hand_over;   // 0: the last launch (finishes the stream whatever the admission rate)
};

constexpr uint32_t kPlaceAdaptiveFrom = 4096;      // arrivals from which a single stream may change kernels
constexpr uint32_t kPlaceWindow = 1024;            // arrivals between two looks at the admission rate
constexpr int kPlaceLaunches = 5;                  // launches of such a stream: kinds 1, 0, 1, 0, 1
// hand-over word: -100 - 2 * (arrivals done / kPlaceWindow) - kind of the kernel that continues (decisions are >= -3)
__device__ __forceinline__ int32_t hand_over_word(uint32_t done, int32_t kind) {
    return -100 - 2 * (int32_t)(done / kPlaceWindow) - kind;
}
// where this launch starts: false = nothing to do (the stream is done, or the hand-over names the other kind)
__device__ __forceinline__ bool place_start(const PlaceArgs& g, uint32_t& k_begin) {
    k_begin = 0;
    if (!g.mailbox || g.first) return true;
    const int32_t m = g.mailbox[0];
    if (m > -100 || ((-100 - m) & 1) != g.my_kind) return false;
    k_begin = (uint32_t)((-100 - m) >> 1) * kPlaceWindow;
    return true;
}
// which kind suits the admissions of the last window: one lane per GPU is the faster one while fewer than about
// half of the arrivals are admitted (its cost grows with the admissions), one lane per slot beyond that
__device__ __forceinline__ int32_t kind_for(uint32_t placed, uint32_t n, int32_t mine) {
    if (placed * 100ull < 45ull * n) return 0;
    if (placed * 100ull > 55ull * n) return 1;
    return mine;
}
// sum of `mine` over the CTA, for thread 0 (s_word: a shared word nobody else uses)
__device__ __forceinline__ uint32_t block_count(uint32_t mine, uint32_t* s_word) {
    if (threadIdx.x == 0) *s_word = 0;
    __syncthreads();
    mine = __reduce_add_sync(0xffffffffu, mine);
    if ((threadIdx.x & 31) == 0 && mine) atomicAdd(s_word, mine);
    __syncthreads();
    return *s_word;
}

constexpr unsigned long long kNoGpu = ~0ull;

// one CTA per independent arrival stream: stream s owns slice s of every per-stream array
__device__ __forceinline__ void select_stream(PlaceArgs& g) {
    const size_t s = blockIdx.x;
    g.ids += s * g.G * g.R; g.expiry += s * g.G * g.R; g.count += s * g.G; g.tick += s;
    g.arr_id += s * g.n; g.arr_life += s * g.n; g.gpu_out += s * g.n;
    if (g.mean_out) g.mean_out += s * g.n;
    if (g.mu_arr_out) g.mu_arr_out += s * g.n;
}

// Algorithm 2 line 7 and the choice criterion (Section 3.4 allows other objectives): returns the bits
// of the score to minimise, or all ones when the GPU is not admissible.  All quantities are >= 0, so
// their float bits order like the floats.
__device__ __forceinline__ uint32_t decision_key(const PlaceArgs& g, float mean, float worst, float mu_inc) {
    const float admit = g.admit_rule == 1 ? worst : mean;
    const float score = g.objective == 1 ? worst : g.objective == 2 ? mu_inc : mean;
    return admit < g.lambda ? __float_as_uint(score) : 0xffffffffu;
}
constexpr uint32_t kArrChunk = 1024;      // arrivals staged in shared memory at a time
constexpr int kRing = 4;      // arrival k+2 is fetched while k is scored and k-1's winner still reads its column

__device__ __forceinline__ void cp_async_4(void* smem_dst, const void* gmem_src) {
    const uint32_t s = (uint32_t)__cvta_generic_to_shared(smem_dst);
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4;\n" ::"r"(s), "l"(gmem_src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::: "memory"); }
template <int kPending>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;\n" ::"n"(kPending) : "memory"); }

// kSlots > 0: compile-time bound of the per-GPU slot loops (fully unrolled, predicated), R <= kSlots;
// kSlots = 0: plain loops for any R
template <int kSlots>
__global__ void __launch_bounds__(1024) place_kernel(PlaceArgs g) {
    select_stream(g);
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const uint32_t G = g.G, R = g.R, P = g.P, GR = G * R;
    int32_t* s_ids = reinterpret_cast<int32_t*>(smem_raw);
    uint32_t* s_exp = reinterpret_cast<uint32_t*>(s_ids + GR);
    float* s_part = reinterpret_cast<float*>(s_exp + GR);
    int32_t* s_arr = reinterpret_cast<int32_t*>(s_part + GR);       // [2][kArrChunk] ids, lifetimes
    float* s_pair = reinterpret_cast<float*>(s_arr + 2 * kArrChunk); // [R][R][G] terms between residents
    float* s_mat = s_pair + (g.pair_cache ? (size_t)GR * R : 0);     // mode 0: P*P, mode 1: ring [kRing][2][P]
    __shared__ unsigned long long s_key[2][32];

    const uint32_t tid = threadIdx.x, lane = tid & 31, wid = tid >> 5, nwarps = blockDim.x >> 5;
    const float* __restrict__ Pm = g.Pm;
    if (g.matrix_mode == 0)
        for (uint32_t i = tid; i < P * P; i += blockDim.x) s_mat[i] = Pm[i];
    for (uint32_t i = tid; i < GR; i += blockDim.x) {                 // [gpu][slot] -> [slot][gpu]
        const uint32_t gpu = i / R, slot = i % R;
        s_ids[slot * G + gpu] = g.ids[i];
        s_exp[slot * G + gpu] = g.expiry[i];
    }
    __syncthreads();

    const bool owner = tid < G;
    {   // a resident id outside the matrix would send the reads below out of bounds: refuse the whole call
        bool bad_id = false;
        for (uint32_t i = tid; i < GR; i += blockDim.x) {
            const uint32_t gpu = i / R, slot = i % R;
            bad_id |= slot < min(g.count[gpu], R) && (uint32_t)g.ids[i] >= P;
        }
        if (__syncthreads_or(bad_id)) {
            for (uint32_t i = tid; i < g.n; i += blockDim.x) {
                g.gpu_out[i] = ROOMIE_PLACE_BAD_ID;
                if (g.mean_out) g.mean_out[i] = 0.0f;
                if (g.mu_arr_out) g.mu_arr_out[i] = 0.0f;
            }
            return;
        }
    }
    auto ID = [&](uint32_t t) -> int32_t& { return s_ids[t * G + tid]; };
    auto EX = [&](uint32_t t) -> uint32_t& { return s_exp[t * G + tid]; };
    auto PA = [&](uint32_t t) -> float& { return s_part[t * G + tid]; };
    // element (i, j) of the matrix for bookkeeping off the fast path
    auto mat = [&](int32_t i, int32_t j) -> float {
        return g.matrix_mode == 0 ? s_mat[(size_t)i * P + j] : __ldg(&Pm[(size_t)i * P + j]);
    };
    auto PT = [&](uint32_t t, uint32_t u) -> float& { return s_pair[(t * R + u) * G + tid]; };   // P[id_t][id_u]
    auto recompute_partials = [&](uint32_t c) {
        for (uint32_t t = 0; t < c; ++t) {
            float s = 0.0f;
            for (uint32_t u = 0; u < c; ++u)
                if (u != t) s = __fadd_rn(s, g.pair_cache ? PT(t, u) : mat(ID(t), ID(u)));
            PA(t) = s;
        }
    };
    uint32_t c = 0, next_exp = 0xffffffffu;
    if (owner) {
        c = min(g.count[tid], R);
        if (g.pair_cache)
            for (uint32_t t = 0; t < c; ++t)
                for (uint32_t u = 0; u < c; ++u) PT(t, u) = mat(ID(t), ID(u));
        recompute_partials(c);
        for (uint32_t s = 0; s < c; ++s)
            if (EX(s) && EX(s) < next_exp) next_exp = EX(s);
    }
    const uint32_t tick0 = *g.tick;

    // ring prefetch of row inc (P[inc][*]) and column inc (P[*][inc]) of arrival k
    auto prefetch = [&](uint32_t k, int32_t inc) {
        float* row = s_mat + (size_t)(k % kRing) * 2 * P;
        float* col = row + P;
        for (uint32_t i = tid; i < P; i += blockDim.x) {
            cp_async_4(row + i, Pm + (size_t)inc * P + i);
            cp_async_4(col + i, Pm + (size_t)i * P + inc);
        }
    };

    for (uint32_t k0 = 0; k0 < g.n; k0 += kArrChunk) {
        const uint32_t kn = min(kArrChunk, g.n - k0);
        __syncthreads();
        for (uint32_t i = tid; i < kn; i += blockDim.x) {
            const int32_t id = g.arr_id[k0 + i];
            s_arr[i] = (uint32_t)id < P ? id : -1;                     // -1: not a profile of this matrix
            s_arr[kArrChunk + i] = (int32_t)g.arr_life[k0 + i];
        }
        __syncthreads();
        if (g.matrix_mode == 1) {                                      // prime the ring: arrivals 0 and 1
            prefetch(0, max(s_arr[0], 0));
            cp_async_commit();
            if (kn > 1) prefetch(1, max(s_arr[1], 0));
            cp_async_commit();
            cp_async_wait<1>();                                        // arrival 0 landed
            __syncthreads();
        }
        for (uint32_t k = 0; k < kn; ++k) {
            const uint32_t now = tick0 + k0 + k;
            const bool bad_arrival = s_arr[k] < 0;                      // scored by nobody, reported as such
            const int32_t inc = max(s_arr[k], 0);
            const float *row_inc, *col_inc;
            uint32_t col_stride;
            if (g.matrix_mode == 1) {
                // arrival k's row and column are in the ring (made visible by the last barrier)
                if (k + 2 < kn) prefetch(k + 2, max(s_arr[k + 2], 0));
                cp_async_commit();
                row_inc = s_mat + (size_t)(k % kRing) * 2 * P; col_inc = row_inc + P; col_stride = 1;
            } else if (g.matrix_mode == 0) {
                row_inc = s_mat + (size_t)inc * P; col_inc = s_mat + inc; col_stride = P;
            } else {
                row_inc = Pm + (size_t)inc * P; col_inc = Pm + inc; col_stride = P;
            }
            unsigned long long key = kNoGpu;
            float mean = 0.0f, mu_inc = 0.0f;
            if (owner) {
                if (next_exp <= now) {                                 // departures, order kept
                    unsigned long long keep = 0;
                    for (uint32_t s = 0; s < c; ++s) {
                        const uint32_t e = EX(s);
                        if (!(e != 0 && e <= now)) keep |= 1ull << s;
                    }
                    uint32_t w = 0;
                    next_exp = 0xffffffffu;
                    for (uint32_t s = 0; s < c; ++s) {
                        if (!((keep >> s) & 1ull)) continue;
                        const uint32_t e = EX(s);
                        ID(w) = ID(s); EX(w) = e;
                        if (e && e < next_exp) next_exp = e;
                        if (g.pair_cache) {                              // survivors' terms, same order
                            uint32_t v = 0;
                            for (uint32_t u = 0; u < c; ++u)
                                if ((keep >> u) & 1ull) { PT(w, v) = PT(s, u); ++v; }
                        }
                        ++w;
                    }
                    for (uint32_t s = w; s < c; ++s) { ID(s) = -1; EX(s) = 0; }
                    c = w;
                    recompute_partials(c);
                }
                if (c < R && !bad_arrival) {                           // what-if: residents + the arrival
                    float tot = 0.0f, worst = 0.0f;
                    if constexpr (kSlots > 0) {
                        float to_inc[kSlots], from_inc[kSlots], part[kSlots];
#pragma unroll
                        for (int t = 0; t < kSlots; ++t) {
                            if ((uint32_t)t < c) {
                                const int32_t id = ID(t);
                                part[t] = PA(t);
                                to_inc[t] = col_inc[(size_t)id * col_stride];   // P[id][inc]
                                from_inc[t] = row_inc[id];                       // P[inc][id]
                            }
                        }
#pragma unroll
                        for (int t = 0; t < kSlots; ++t) {
                            if ((uint32_t)t < c) {
                                const float mu_t = __fadd_rn(part[t], to_inc[t]);
                                worst = fmaxf(worst, mu_t);
                                tot = __fadd_rn(tot, mu_t);
                                mu_inc = __fadd_rn(mu_inc, from_inc[t]);
                            }
                        }
                    } else {
                        for (uint32_t t = 0; t < c; ++t) {
                            const int32_t id = ID(t);
                            const float mu_t = __fadd_rn(PA(t), col_inc[(size_t)id * col_stride]);
                            worst = fmaxf(worst, mu_t);
                            tot = __fadd_rn(tot, mu_t);
                            mu_inc = __fadd_rn(mu_inc, row_inc[id]);
                        }
                    }
                    tot = __fadd_rn(tot, mu_inc);
                    mean = __fdiv_rn(tot, (float)(c + 1));
                    const uint32_t kb = decision_key(g, mean, fmaxf(worst, mu_inc), mu_inc);
                    if (kb != 0xffffffffu) key = ((unsigned long long)kb << 32) | tid;
                }
            }
            // argmin over GPUs, lowest index on equal means (mean >= 0, so its bits order as integers)
            const uint32_t hi = (uint32_t)(key >> 32);
            const uint32_t best_hi = __reduce_min_sync(0xffffffffu, hi);
            const uint32_t best_lo = __reduce_min_sync(0xffffffffu, hi == best_hi ? (uint32_t)key : 0xffffffffu);
            if (lane == 0) s_key[k & 1][wid] = ((unsigned long long)best_hi << 32) | best_lo;
            if (g.matrix_mode == 1) cp_async_wait<1>();                // this thread's share of arrival k+1 landed
            __syncthreads();
            unsigned long long best = s_key[k & 1][0];
            for (uint32_t w = 1; w < nwarps; ++w) {
                const unsigned long long o = s_key[k & 1][w];
                best = o < best ? o : best;
            }
            if (best == kNoGpu) {
                if (tid == 0) {
                    g.gpu_out[k0 + k] = bad_arrival ? ROOMIE_PLACE_BAD_ID : -1;
                    if (g.mean_out) g.mean_out[k0 + k] = 0.0f;
                    if (g.mu_arr_out) g.mu_arr_out[k0 + k] = 0.0f;
                }
            } else if (tid == (uint32_t)(best & 0xffffffffu)) {
                const uint32_t life = (uint32_t)s_arr[kArrChunk + k];
                for (uint32_t t = 0; t < c; ++t) {                     // the what-if sums become the cached ones
                    const float to = col_inc[(size_t)ID(t) * col_stride];
                    PA(t) = __fadd_rn(PA(t), to);
                    if (g.pair_cache) { PT(t, c) = to; PT(c, t) = row_inc[ID(t)]; }
                }
                if (g.pair_cache) PT(c, c) = 0.0f;
                PA(c) = mu_inc;
                ID(c) = inc;
                const uint32_t e = life ? now + life : 0u;
                EX(c) = e;
                if (e && e < next_exp) next_exp = e;
                ++c;
                g.gpu_out[k0 + k] = (int32_t)tid;
                if (g.mean_out) g.mean_out[k0 + k] = mean;
                if (g.mu_arr_out) g.mu_arr_out[k0 + k] = mu_inc;
            }
        }
        if (g.matrix_mode == 1) cp_async_wait<0>();
    }
    if (owner) g.count[tid] = c;
    __syncthreads();
    for (uint32_t i = tid; i < GR; i += blockDim.x) {
        const uint32_t gpu = i / R, slot = i % R;
        g.ids[i] = s_ids[slot * G + gpu];
        g.expiry[i] = s_exp[slot * G + gpu];
    }
    if (tid == 0) *g.tick = tick0 + g.n;
}

// ---------------------------------------------------------------------------------------
// K5, fast variant for up to 8 slots per GPU.  On top of the scheme above it keeps the matrix
// off the critical path entirely, whatever its size:
//   - every resident sits in a fixed *physical* slot; the arrival order of a GPU's residents is a
//     packed nibble list in a register, so a departure moves no shared-memory data and copies in
//     flight never have to follow a resident;
//   - the CTA is split into owner warps (one lane per modelled GPU: departures, what-if sums,
//     argmin, winner update) and as many fetch warps.  While arrival j is decided, the fetch lane
//     of a GPU issues cp.async for the two matrix elements per resident that arrival j+3 will
//     need, into a 4-deep ring indexed by physical slot; it reads the GPU's order list from a
//     64-bit word the owner publishes whenever the list changes;
//   - a resident placed fewer than 5 arrivals ago may have been missed by those fetches (they
//     were issued before, or while, it was placed); its terms depend only on the arrival stream
//     (P[arr_{j-d}][arr_j] and the transpose, d = 1..4) and are fetched on the same schedule.
//   - the what-if loop of an owner lane is a two-stage software pipeline over its residents (the reads
//     for resident t + 1 and t + 2 are in flight while t is summed), and it leaves behind everything
//     the winner's update needs: the new partial sums go into a second copy of the partial-sum array
//     (the winner only switches copies) and the resident-arrival terms into the row and column of the
//     free slot the arrival would take, so the update itself has no loop.
// The owners' critical path per arrival is shared-memory reads, 2c+2 float adds, one division,
// two redux steps and one barrier; no global memory access and no copy wait.
// ---------------------------------------------------------------------------------------
// a / n for 1 <= n <= 9, correctly rounded like the float32 division it replaces (IEEE division is a
// subroutine of a few dozen dependent instructions; this is a conversion, a product and a conversion).
// The double product of a and the double nearest to 1/n is within 2^-52 (relative) of a/n.  A 24-bit a
// divided by n <= 9 is either a float itself or at least 2^-29 (relative) away from every midpoint
// between two neighbouring floats (the distance is a non-zero multiple of half a unit in the last place
// divided by n), so rounding the product to float32 rounds the quotient.
__constant__ double kInvSmall[10] = {0.0, 1.0, 1.0 / 2, 1.0 / 3, 1.0 / 4, 1.0 / 5, 1.0 / 6, 1.0 / 7, 1.0 / 8, 1.0 / 9};
__device__ __forceinline__ float div_small(float a, uint32_t n) {
    return __double2float_rn(__dmul_rn((double)a, kInvSmall[n]));
}

constexpr int kAhead = 3;                     // arrivals fetched ahead
constexpr int kYoungD = kAhead + 1;           // residents this young read the arrival-to-arrival terms
constexpr int kYoungRing = 8;                 // ring depth of the arrival-to-arrival terms
constexpr int kYoungInit = -(1 << 30);        // birth index of initial residents
constexpr int kLead = kYoungD;                // arrival ids staged before / after a chunk

__device__ __forceinline__ void cp_async_4_s(uint32_t smem_addr, const void* gmem_src) {
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4;\n" ::"r"(smem_addr), "l"(gmem_src) : "memory");
}

// kPlain: Algorithm 2 as printed (admit on the mean drop, choose the lowest mean drop); the rule and the
// objective are then compile-time facts and the largest member drop is not tracked
template <bool kPlain>
__global__ void __launch_bounds__(1024) place_fast_kernel(PlaceArgs g) {
    select_stream(g);
    uint32_t k_begin;
    if (!place_start(g, k_begin)) return;                                   // not this launch's turn
    __shared__ uint32_t s_placed;
    uint32_t n_placed = 0;                                                  // admissions since the last look
    uint32_t k_end = g.n;                                                   // where this launch stops
    // one float/int array; every region is addressed by a 32-bit word index
    extern __shared__ __align__(16) float sm[];
    int32_t* smi = reinterpret_cast<int32_t*>(sm);
    uint32_t* smu = reinterpret_cast<uint32_t*>(sm);
    const uint32_t G = g.G, R = g.R, P = g.P, GR = G * R;
    const uint32_t tid = threadIdx.x, lane = tid & 31, wid = tid >> 5, nwarps = blockDim.x >> 5;
    const uint32_t n_owner_warps = nwarps >> 1;
    const bool fetcher = wid >= n_owner_warps;
    const uint32_t gpu = (fetcher ? wid - n_owner_warps : wid) * 32 + lane;
    const bool has_gpu = gpu < G;
    const bool owner = !fetcher && has_gpu;
    // word offsets of the regions; per-GPU arrays are [slot][gpu]
    const uint32_t oID = gpu, oEX = GR + gpu, oPA = 2 * GR + gpu, oBI = 3 * GR + gpu;
    const uint32_t oPT = 4 * GR + gpu;                    // [slot][slot][gpu]
    const uint32_t oRING = 4 * GR + GR * R + gpu;         // [4][2][slot][gpu]
    const uint32_t oYOUNG = 4 * GR + GR * R + 8 * GR;     // [kYoungRing][kYoungD][2]
    const uint32_t oPUB = (oYOUNG + kYoungRing * kYoungD * 2 + 1) & ~1u;   // [G] 64-bit: order list | count << 32
    const uint32_t chunk = g.chunk;
    const uint32_t oARR = oPUB + 2 * G;                   // ids [chunk + 2 kLead], then lifetimes [chunk]
    const uint32_t oLIFE = oARR + chunk + 2 * kLead;
    const uint32_t oOUT = oLIFE + chunk;                  // decisions of the chunk: gpu, mean, mu_arr [3][chunk]
    // cached partial sums, twice: every what-if writes the sums its GPU would have after taking the arrival
    // into the other copy, and the winner just switches copies
    uint32_t pa_cur = oPA, pa_alt = oOUT + 3 * chunk + gpu;
    const uint32_t sm_base = (uint32_t)__cvta_generic_to_shared(sm);
    volatile unsigned long long* pub = reinterpret_cast<volatile unsigned long long*>(sm + oPUB);
    __shared__ unsigned long long s_key[2][32];

    const float* __restrict__ Pm = g.Pm;

    {   // a resident id outside the matrix would send the reads below out of bounds: refuse the whole call
        bool bad_id = false;
        if (owner)
            for (uint32_t p = 0; p < min(g.count[gpu], R); ++p) bad_id |= (uint32_t)g.ids[gpu * R + p] >= P;
        if (__syncthreads_or(bad_id)) {
            for (uint32_t i = tid; i < g.n; i += blockDim.x) {
                g.gpu_out[i] = ROOMIE_PLACE_BAD_ID;
                if (g.mean_out) g.mean_out[i] = 0.0f;
                if (g.mu_arr_out) g.mu_arr_out[i] = 0.0f;
            }
            return;
        }
    }
    // initial state: residents occupy physical slots 0..c-1 in arrival order
    uint32_t c = 0, ord = 0, free_mask = (1u << R) - 1u, next_exp = 0xffffffffu;
    if (owner) {
        c = min(g.count[gpu], R);
        for (uint32_t p = 0; p < R; ++p) {
            smi[oID + p * G] = p < c ? g.ids[gpu * R + p] : -1;
            smu[oEX + p * G] = p < c ? g.expiry[gpu * R + p] : 0u;
            smi[oBI + p * G] = kYoungInit;
        }
        for (uint32_t p = 0; p < c; ++p) {
            ord |= p << (4 * p);
            free_mask &= ~(1u << p);
            const uint32_t e = smu[oEX + p * G];
            if (e && e < next_exp) next_exp = e;
            for (uint32_t q = 0; q < c; ++q)
                sm[oPT + (p * R + q) * G] = __ldg(&Pm[(size_t)smi[oID + p * G] * P + smi[oID + q * G]]);
        }
        for (uint32_t p = 0; p < c; ++p) {
            float s = 0.0f;
            for (uint32_t q = 0; q < c; ++q)
                if (q != p) s = __fadd_rn(s, sm[oPT + (p * R + q) * G]);
            sm[pa_cur + p * G] = s;
        }
        pub[gpu] = (unsigned long long)ord | ((unsigned long long)c << 32);
    }
    const uint32_t tick0 = *g.tick - k_begin;                               // tick of the stream's first arrival

    // fetch warps: what arrival a (staged index a_local, global index a_global) will need
    auto issue = [&](uint32_t a_local, uint32_t a_global) {
        const int32_t inc = max(smi[oARR + a_local], 0);  // an id outside the matrix is staged as -1 and scored by nobody
        const float* row = Pm + (size_t)inc * P;          // P[inc][*]
        const float* col = Pm + inc;                      // P[*][inc]
        if (has_gpu) {
            const unsigned long long pv = pub[gpu];       // one 64-bit read: list and count belong together
            const uint32_t cc = (uint32_t)(pv >> 32);
            const uint32_t ring = oRING + (a_global & 3u) * 2 * GR;
            for (uint32_t t = 0, o = (uint32_t)pv; t < cc; ++t, o >>= 4) {
                const uint32_t p = o & 15u;
                const int32_t id = smi[oID + p * G];
                if (id < 0) continue;                     // just departed
                cp_async_4_s(sm_base + 4u * (ring + p * G), col + (size_t)id * P);
                cp_async_4_s(sm_base + 4u * (ring + GR + p * G), row + id);
            }
        }
        if (wid == n_owner_warps && lane < 2 * kYoungD) {
            const uint32_t d = (lane >> 1) + 1, dir = lane & 1u;
            if (a_local >= d) {
                const int32_t old = max(smi[oARR + a_local - d], 0);
                cp_async_4_s(sm_base + 4u * (oYOUNG + ((a_global & (kYoungRing - 1)) * kYoungD + (d - 1)) * 2 + dir),
                             dir == 0 ? col + (size_t)old * P : row + old);
            }
        }
    };

    for (uint32_t k0 = k_begin; k0 < g.n; k0 += chunk) {
        const uint32_t kn = min(chunk, g.n - k0);
        // stage arrival ids [k0 - kLead, k0 + kn + kLead) and lifetimes [k0, k0 + kn)
        __syncthreads();
        bool saw_bad = false;
        for (uint32_t i = tid; i < kn + 2 * kLead; i += blockDim.x) {
            const long long gi = (long long)k0 + i - kLead;
            int32_t id = 0;
            if (gi >= 0 && gi < (long long)g.n) { id = g.arr_id[gi]; if ((uint32_t)id >= P) { id = -1; saw_bad = true; } }
            smi[oARR + i] = id;
        }
        for (uint32_t i = tid; i < kn; i += blockDim.x) smi[oLIFE + i] = (int32_t)g.arr_life[k0 + i];
        // whether the chunk holds an id outside the matrix at all: the per-arrival look at the staged id would
        // otherwise sit on every arrival's chain
        const bool chunk_bad = __syncthreads_or(saw_bad);
        if (k0 == k_begin) {                                                // prime: the first kAhead arrivals of this launch
            if (fetcher) {
                for (uint32_t a = 0; a < (uint32_t)kAhead; ++a) {
                    if (k_begin + a < g.n) issue(a + kLead, k_begin + a);
                    cp_async_commit();
                }
                cp_async_wait<kAhead - 1>();
            }
            __syncthreads();
        }
        for (uint32_t k = 0; k < kn; ++k) {
            const uint32_t kg = k0 + k, now = tick0 + kg, kl = k + kLead;   // global index, tick, index into the staged ids
            if (fetcher) {
                if (kg + kAhead < g.n) issue(kl + kAhead, kg + kAhead);
                cp_async_commit();
                cp_async_wait<kAhead - 1>();                                 // arrival k+1's terms have landed
                __syncthreads();
                continue;
            }
            if (owner && next_exp <= now) {                                  // departures: drop from the order list
                uint32_t w = 0, nord = 0;
                next_exp = 0xffffffffu;
                for (uint32_t t = 0; t < c; ++t) {
                    const uint32_t p = (ord >> (4 * t)) & 15u, e = smu[oEX + p * G];
                    if (e != 0 && e <= now) { free_mask |= 1u << p; smi[oID + p * G] = -1; smu[oEX + p * G] = 0; continue; }
                    nord |= p << (4 * w); ++w;
                    if (e && e < next_exp) next_exp = e;
                }
                ord = nord; c = w;
                pub[gpu] = (unsigned long long)ord | ((unsigned long long)c << 32);
                for (uint32_t t = 0; t < c; ++t) {                           // re-sum the cached terms, slot order
                    const uint32_t p = (ord >> (4 * t)) & 15u;
                    float s = 0.0f;
                    for (uint32_t u = 0; u < c; ++u)
                        if (u != t) s = __fadd_rn(s, sm[oPT + (p * R + ((ord >> (4 * u)) & 15u)) * G]);
                    sm[pa_cur + p * G] = s;
                }
            }
            // terms of arrival kg: ring (by physical slot) or, for young residents, arrival-to-arrival
            const uint32_t ring_k = oRING + (kg & 3u) * 2 * GR;
            const uint32_t young_k = oYOUNG + (kg & (kYoungRing - 1)) * kYoungD * 2;
            uint32_t key_hi = 0xffffffffu;
            float mean = 0.0f, mu_inc = 0.0f;
            if (owner && c < R) {                                            // what-if: residents + the arrival
                float tot = 0.0f, worst = 0.0f;
                // two-stage pipeline over the residents: while resident t is summed, the terms of t + 1 are on
                // their way and the birth index and cached partial sum of t + 2 are being read (past the end
                // of the list the nibbles are 0: slot 0 is read, a valid address, and the value is dropped)
                const uint32_t pn = __ffs(free_mask) - 1u;                   // lowest free physical slot: the arrival's, if it comes here
                const uint32_t pt_col = oPT + pn * G, pt_row = oPT + pn * R * G;
                uint32_t o = ord, p = o & 15u, p_c = p;
                uint32_t d1 = (uint32_t)((int32_t)kg - smi[oBI + p * G]);    // arrivals since placed, minus 1 (huge if old)
                bool young = d1 < (uint32_t)kYoungD;
                uint32_t i0 = young ? young_k + 2 * d1 : ring_k + p * G;
                float pa = sm[pa_cur + p * G];
                float to = sm[i0];                                            // P[id][inc]
                float from = sm[i0 + (young ? 1u : GR)];                      // P[inc][id]
                o >>= 4; p = o & 15u;
                int32_t bi_n = smi[oBI + p * G];
                float pa_n = sm[pa_cur + p * G];
                for (uint32_t t = 0; t < c; ++t) {
                    const uint32_t p_n = p;
                    d1 = (uint32_t)((int32_t)kg - bi_n);
                    young = d1 < (uint32_t)kYoungD;
                    i0 = young ? young_k + 2 * d1 : ring_k + p * G;
                    const float to_n = sm[i0], from_n = sm[i0 + (young ? 1u : GR)], pa_c = pa_n;
                    o >>= 4; p = o & 15u;
                    bi_n = smi[oBI + p * G];
                    pa_n = sm[pa_cur + p * G];
                    const float mu_t = __fadd_rn(pa, to);
                    if (!kPlain) worst = fmaxf(worst, mu_t);
                    tot = __fadd_rn(tot, mu_t);
                    mu_inc = __fadd_rn(mu_inc, from);
                    // what the winner will need: the new partial sum and the two terms between the
                    // resident and the arrival (the free slot's row and column hold nothing yet)
                    sm[pa_alt + p_c * G] = mu_t;
                    sm[pt_col + p_c * R * G] = to;
                    sm[pt_row + p_c * G] = from;
                    pa = pa_c; to = to_n; from = from_n; p_c = p_n;
                }
                tot = __fadd_rn(tot, mu_inc);
                mean = div_small(tot, c + 1);                                // c + 1 <= 9 in this kernel
                key_hi = kPlain ? (mean < g.lambda ? __float_as_uint(mean) : 0xffffffffu)
                                : decision_key(g, mean, fmaxf(worst, mu_inc), mu_inc);
            }
            // an arrival whose id is outside the matrix (staged as -1, its terms fetched for profile 0) goes nowhere;
            // the look at the staged id is skipped for a chunk without such ids, which keeps it off the chain
            bool bad_arrival = false;
            if (chunk_bad) {
                bad_arrival = smi[oARR + kl] < 0;
                if (bad_arrival) key_hi = 0xffffffffu;
            }
            // warp argmin: lowest key, then the lowest lane (= lowest GPU index of this warp) that holds it
            const uint32_t best_hi = __reduce_min_sync(0xffffffffu, key_hi);
            const uint32_t holders = __ballot_sync(0xffffffffu, key_hi == best_hi);
            const uint32_t best_lo = best_hi != 0xffffffffu ? (wid << 5) + (uint32_t)__ffs(holders) - 1u : 0xffffffffu;
            if (lane == 0) s_key[k & 1][wid] = ((unsigned long long)best_hi << 32) | best_lo;
            __syncthreads();
            unsigned long long best;
            if (n_owner_warps == 2) {                                        // the common shape: both keys at once
                const unsigned long long k0w = s_key[k & 1][0], k1w = s_key[k & 1][1];
                best = k1w < k0w ? k1w : k0w;
            } else {
                best = s_key[k & 1][0];
                for (uint32_t w = 1; w < n_owner_warps; ++w) {
                    const unsigned long long o = s_key[k & 1][w];
                    best = o < best ? o : best;
                }
            }
            // results stay in shared memory until the chunk ends: a global store inside the loop would
            // have to complete before every barrier
            if (best == kNoGpu) {
                if (tid == 0) { smi[oOUT + k] = bad_arrival ? ROOMIE_PLACE_BAD_ID : -1; sm[oOUT + chunk + k] = 0.0f; sm[oOUT + 2 * chunk + k] = 0.0f; }
            } else if (owner && gpu == (uint32_t)(best & 0xffffffffu)) {
                const uint32_t pn = __ffs(free_mask) - 1u;                   // the slot the what-if wrote for
                free_mask &= ~(1u << pn);
                { const uint32_t sw = pa_cur; pa_cur = pa_alt; pa_alt = sw; } // the what-if sums become the cached ones
                sm[oPT + (pn * R + pn) * G] = 0.0f;
                sm[pa_cur + pn * G] = mu_inc;
                smi[oID + pn * G] = smi[oARR + kl];
                const uint32_t life = (uint32_t)smi[oLIFE + k];
                const uint32_t e = life ? now + life : 0u;
                smu[oEX + pn * G] = e;
                smi[oBI + pn * G] = (int32_t)(kg + 1);                       // first arrival that sees this resident
                if (e && e < next_exp) next_exp = e;
                ord |= pn << (4 * c);
                ++c;
                __threadfence_block();                                       // id before the list that names its slot
                pub[gpu] = (unsigned long long)ord | ((unsigned long long)c << 32);
                smi[oOUT + k] = (int32_t)gpu;
                sm[oOUT + chunk + k] = mean;
                sm[oOUT + 2 * chunk + k] = mu_inc;
            }
        }
        __syncthreads();
        for (uint32_t i = tid; i < kn; i += blockDim.x) {
            g.gpu_out[k0 + i] = smi[oOUT + i];
            n_placed += smi[oOUT + i] >= 0 ? 1u : 0u;
            if (g.mean_out) g.mean_out[k0 + i] = sm[oOUT + chunk + i];
            if (g.mu_arr_out) g.mu_arr_out[k0 + i] = sm[oOUT + 2 * chunk + i];
        }
        // a look at the admission rate: should the other kind of kernel take the rest of the stream?
        const uint32_t done = k0 + kn;
        if (g.mailbox && g.may_hand_over && done < g.n && done % kPlaceWindow == 0) {
            const uint32_t placed = block_count(n_placed, &s_placed);
            n_placed = 0;
            if (kind_for(placed, kn, g.my_kind) != g.my_kind) { k_end = done; break; }
        }
    }
    cp_async_wait<0>();
    if (owner) {                                                             // write back in arrival order
        g.count[gpu] = c;
        for (uint32_t t = 0; t < R; ++t) {
            const uint32_t p = (ord >> (4 * t)) & 15u;
            g.ids[gpu * R + t] = t < c ? smi[oID + p * G] : -1;
            g.expiry[gpu * R + t] = t < c ? smu[oEX + p * G] : 0u;
        }
    }
    if (tid == 0) {
        *g.tick = tick0 + k_end;
        if (k_end < g.n) g.mailbox[0] = hand_over_word(k_end, 1 - g.my_kind);
    }
}

#include "roomie_place_slots.cuh"

}  // namespace roomie

using namespace roomie;

extern "C" int roomie_multi_estimate(const float* Pmat, uint32_t P, const int32_t* resident_ids, const uint32_t* count,
                                     const int32_t* incoming, uint32_t n_sets, uint32_t max_residents, float* mu_out,
                                     float* mean_out, void* stream) {
    if (!Pmat || P == 0 || !count || !incoming || (max_residents && !resident_ids) || max_residents > 64)
        return ROOMIE_ERR_INVALID_ARG;
    if (n_sets == 0) return ROOMIE_OK;
    multi_estimate_kernel<<<(n_sets + 127) / 128, 128, 0, static_cast<cudaStream_t>(stream)>>>(
        Pmat, P, resident_ids, count, incoming, n_sets, max_residents, mu_out, mean_out);
    note_launch();
    ROOMIE_CUDA_OK(cudaGetLastError());
    return ROOMIE_OK;
}

static int place_impl(const float* Pmat, uint32_t P, const roomie_cluster_state* state, const int32_t* arr_id,
                      const uint32_t* arr_life, uint32_t n, uint32_t num_streams, const roomie_opts* opts,
                      int32_t* gpu_out, float* mean_out, float* mu_arr_out, void* stream) {
    if (!Pmat || P == 0 || !state || !opts || !state->ids || !state->expiry || !state->count || !state->tick)
        return ROOMIE_ERR_INVALID_ARG;
    if (state->num_gpus == 0 || state->num_gpus > 1024 || state->max_residents == 0 || state->max_residents > 64 ||
        (uint64_t)state->num_gpus * state->max_residents > 8192)
        return ROOMIE_ERR_INVALID_ARG;
    if (n == 0 || num_streams == 0) return ROOMIE_OK;
    if (!arr_id || !arr_life || !gpu_out) return ROOMIE_ERR_INVALID_ARG;
    if (opts->admit_rule < 0 || opts->admit_rule > 1 || opts->objective < 0 || opts->objective > 2)
        return ROOMIE_ERR_INVALID_ARG;
    if (opts->max_residents != 0 && opts->max_residents != state->max_residents) return ROOMIE_ERR_INVALID_ARG;
    PlaceArgs a;
    a.admit_rule = opts->admit_rule; a.objective = opts->objective;
    a.Pm = Pmat; a.P = P; a.G = state->num_gpus; a.R = state->max_residents;
    a.ids = state->ids; a.expiry = state->expiry; a.count = state->count; a.tick = state->tick;
    a.arr_id = arr_id; a.arr_life = arr_life; a.n = n; a.lambda = opts->lambda;
    a.gpu_out = gpu_out; a.mean_out = mean_out; a.mu_arr_out = mu_arr_out;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    a.mailbox = nullptr; a.my_kind = 0; a.first = 1; a.may_hand_over = 0;
    const bool plain = a.admit_rule == 0 && a.objective == 0;
    if (num_streams == 1 && a.R <= (uint32_t)kSlotLanes && a.G <= (1024u - 32u) / kSlotLanes) {
        // One stream, up to 8 slots per GPU.  Two kernels give the same bits: one lane per resident slot (flat in
        // the admission rate, the shorter chain when most arrivals are admitted) and one lane per modelled GPU
        // (cheaper while most arrivals are deferred, dearer with every admission).  A long stream starts on the
        // first kind; every kPlaceWindow arrivals the running kernel looks at the admissions of the window and,
        // when the other kind suits them better, writes the state back, leaves the number of arrivals done and the
        // kind that continues in the stream's last gpu_out element and returns.  The launches alternate between
        // the kinds; one that finds a decision in that element (the stream is done) or a hand-over to the other
        // kind returns at once, and the last one finishes the stream whatever the rate.
        PlaceArgs slots = a, fast = a;
        slots.matrix_mode = 1; slots.pair_cache = 1; slots.gpus_per_warp = 32 / kSlotLanes; slots.chunk = kSlotChunk;
        slots.my_kind = 1;
        const uint32_t s_threads = ((a.G * kSlotLanes + 31) / 32) * 32 + 32;   // one more warp that owns no GPU
        const size_t s_bytes = (size_t)slot_layout(s_threads, a.G).total * sizeof(float);
        auto s_kern = plain ? place_slots_kernel<true> : place_slots_kernel<false>;
        if (s_bytes > 48 * 1024)
            ROOMIE_CUDA_OK(cudaFuncSetAttribute(s_kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)s_bytes));
        fast.matrix_mode = 1; fast.pair_cache = 1; fast.gpus_per_warp = 32; fast.chunk = kArrChunk;
        fast.my_kind = 0;
        const size_t fGR = (size_t)a.G * a.R;
        const size_t f_bytes = fGR * 5 * 4 + fGR * a.R * 4 + 4 * 2 * fGR * 4 + (kYoungRing * kYoungD * 2 + 2) * 4 +
                               2 * a.G * 4 + (5 * fast.chunk + 2 * kLead) * sizeof(int32_t);
        const uint32_t f_threads = 2 * 32 * ((a.G + 31) / 32);
        auto f_kern = plain ? place_fast_kernel<true> : place_fast_kernel<false>;
        const bool adaptive = n >= kPlaceAdaptiveFrom && f_bytes <= 160 * 1024;
        if (adaptive && f_bytes > 48 * 1024)
            ROOMIE_CUDA_OK(cudaFuncSetAttribute(f_kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)f_bytes));
        const int launches = adaptive ? kPlaceLaunches : 1;
        for (int l = 0; l < launches; ++l) {
            PlaceArgs& k = (l & 1) ? fast : slots;
            k.mailbox = adaptive ? gpu_out + n - 1 : nullptr;
            k.first = l == 0; k.may_hand_over = l + 1 < launches;
            if (l & 1) f_kern<<<1, f_threads, f_bytes, st>>>(k);
            else s_kern<<<1, s_threads, s_bytes, st>>>(k);
            note_launch();
            ROOMIE_CUDA_OK(cudaGetLastError());
        }
        return ROOMIE_OK;
    }
    const size_t GR = (size_t)a.G * a.R;
    // many independent streams: a short staging chunk keeps the CTA small enough (44.4 KB) for 5 per SM
    a.chunk = num_streams > 1 ? 32u : kArrChunk;
    const size_t fast_bytes = GR * 5 * 4 + GR * a.R * 4 + 4 * 2 * GR * 4 + (kYoungRing * kYoungD * 2 + 2) * 4 +
                              2 * a.G * 4 + (5 * a.chunk + 2 * kLead) * sizeof(int32_t);
    if (a.R <= 8 && a.G <= 512 && fast_bytes <= 160 * 1024) {
        // up to 8 slots per GPU: matrix elements are fetched three arrivals ahead by fetch warps
        a.matrix_mode = 1; a.pair_cache = 1;
        a.gpus_per_warp = 32;
        const uint32_t threads = 2 * 32 * ((a.G + 31) / 32);                 // owner warps + as many fetch warps
        auto kern = plain ? place_fast_kernel<true> : place_fast_kernel<false>;
        if (fast_bytes > 48 * 1024)
            ROOMIE_CUDA_OK(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)fast_bytes));
        kern<<<num_streams, threads, fast_bytes, st>>>(a);
        note_launch();
        ROOMIE_CUDA_OK(cudaGetLastError());
        return ROOMIE_OK;
    }
    size_t state_bytes = (size_t)a.G * a.R * 12 + 2 * kArrChunk * sizeof(int32_t);
    const size_t pair_bytes = (size_t)a.G * a.R * a.R * sizeof(float);
    a.pair_cache = pair_bytes <= 64 * 1024;
    if (a.pair_cache) state_bytes += pair_bytes;
    const size_t mat_bytes = (size_t)P * P * sizeof(float), ring_bytes = (size_t)kRing * 2 * P * sizeof(float);
    const size_t budget = 200 * 1024;
    size_t smem = state_bytes;
    if (state_bytes + mat_bytes <= budget) { a.matrix_mode = 0; smem += mat_bytes; }
    else if (state_bytes + ring_bytes <= budget) { a.matrix_mode = 1; smem += ring_bytes; }
    else a.matrix_mode = 2;
    uint32_t threads = ((a.G + 31) / 32) * 32;
    if (a.matrix_mode == 1 && threads < 128) threads = 128;          // more lanes to issue the prefetch
    auto kern = a.R <= 16 ? place_kernel<16> : place_kernel<0>;
    if (smem > 48 * 1024)
        ROOMIE_CUDA_OK(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    kern<<<num_streams, threads, smem, st>>>(a);
    note_launch();
    ROOMIE_CUDA_OK(cudaGetLastError());
    return ROOMIE_OK;
}

extern "C" int roomie_place(const float* Pmat, uint32_t P, const roomie_cluster_state* state, const int32_t* arr_id,
                            const uint32_t* arr_life, uint32_t n, const roomie_opts* opts, int32_t* gpu_out,
                            float* mean_out, float* mu_arr_out, void* stream) {
    return place_impl(Pmat, P, state, arr_id, arr_life, n, 1, opts, gpu_out, mean_out, mu_arr_out, stream);
}

extern "C" int roomie_place_batch(const float* Pmat, uint32_t P, const roomie_cluster_state* states,
                                  const int32_t* arr_id, const uint32_t* arr_life, uint32_t n, uint32_t num_streams,
                                  const roomie_opts* opts, int32_t* gpu_out, float* mean_out, float* mu_arr_out,
                                  void* stream) {
    return place_impl(Pmat, P, states, arr_id, arr_life, n, num_streams, opts, gpu_out, mean_out, mu_arr_out, stream);
}
