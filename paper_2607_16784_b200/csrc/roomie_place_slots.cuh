// Algorithm 2 with ONE LANE PER RESIDENT SLOT: clusters of up to 8 slots per modelled GPU and up to 124 GPUs.
// Included by roomie_place.cu inside namespace roomie.
//
// The arrival stream is a dependent chain: what bounds it is the number of instructions one warp executes per
// arrival, times the few cycles a lone warp needs per instruction.  With one lane per modelled GPU every lane loops
// over its GPU's residents (what-if sums, winner update, re-summing after a departure) and the chain pays for the
// longest loop in the warp.  Here the eight lanes of a group own the eight slots of one GPU, so that everything
// about a resident is O(1) work of its own lane:
//   - a lane keeps its resident's id, cached partial sum (sum over the other residents of P[this][other], slot
//     order), birth arrival and expiry tick in registers; the group's arrival order (slot list in nibbles), count
//     and free-slot mask are replicated in all eight lanes and updated identically by them;
//   - a lane fetches ITS OWN two matrix elements for the arrival kAhead steps ahead (P[resident][arrival],
//     P[arrival][resident]; cp.async into a ring stage at its own thread index) and waits only for its own copies:
//     no fetch warps, no published resident lists, no cross-thread wait for data;
//   - a resident placed fewer than kAhead arrivals ago has no such copies yet: its terms depend on the arrival
//     stream alone (P[arrival j][arrival k] and the transpose), are fetched for every arrival and its kAhead
//     predecessors by the first lanes of the CTA, and are visible to everybody after the barrier of the arrival before;
//   - the what-if of a GPU is one add per lane, then every lane of the group collects the (mu, from) pairs of the
//     GPU's residents in arrival order with independent shuffles (as many as the fullest GPU of the warp has
//     residents) and adds them in that order (Algorithm 1's slot order; all eight lanes get the same bits), one
//     division, one key;
//   - argmin: redux + ballot in the warp, one 64-bit word per warp in shared memory, ONE barrier per arrival, then
//     every warp reduces the words of all warps;
//   - the winner's update is one predicated move per lane (the what-if sum becomes the cached one; the lane of the
//     free slot takes the arrival) and two stores into the cache of resident-resident terms;
//   - a departure clears its lane; the group rebuilds the slot list from a ballot, and every surviving lane re-adds
//     its own partial sum from the cached terms (eight independent loads, slot order kept).
// Sums are float32 in slot order with the arrival last and one division, as roomie_multi_estimate defines them.

constexpr int kSlotLanes = 8;                  // lanes (= resident slots) per modelled GPU
constexpr int kSlotAhead = 5;                  // arrivals fetched ahead
constexpr int kSlotStages = 8;                 // ring stages (a power of two > kSlotAhead)
constexpr uint32_t kSlotChunk = 1024;          // arrivals staged in shared memory at a time (= the window between two looks at the admission rate)
constexpr int kSlotLead = kSlotAhead;          // arrival ids staged before and after a chunk
constexpr uint32_t kSlotNever = 0xffffffffu;   // expiry tick of a resident that never leaves
constexpr int32_t kSlotBornLongAgo = -(1 << 30);

struct SlotLayout {                            // word offsets of the shared-memory regions
    uint32_t ring, young, pt, key, arr, life, out, total;
};
__host__ __device__ inline SlotLayout slot_layout(uint32_t threads, uint32_t G) {
    SlotLayout l;
    l.ring = 0;                                              // [stage][to | from][thread]
    l.young = l.ring + kSlotStages * 2 * threads;            // [stage][arrivals back - 1][to | from]
    l.pt = l.young + kSlotStages * kSlotAhead * 2;           // [gpu] x 72: P[id_r][id_u] at r * 9 + u
    l.key = (l.pt + G * 72 + 1) & ~1u;                       // [2][32] 64-bit best key of a warp
    l.arr = l.key + 2 * 2 * 32;                              // arrival ids [chunk + 2 lead]
    l.life = l.arr + kSlotChunk + 2 * kSlotLead;             // lifetimes [chunk]
    l.out = l.life + kSlotChunk;                             // decisions of the chunk: gpu, mean, mu_arr [3][chunk]
    l.total = l.out + 3 * kSlotChunk;
    return l;
}

template <bool kPlain>
__global__ void __launch_bounds__(1024) place_slots_kernel(PlaceArgs g) {
    select_stream(g);
    uint32_t k_begin;
    if (!place_start(g, k_begin)) return;                                 // not this launch's turn
    __shared__ uint32_t s_placed;
    extern __shared__ __align__(16) float sm[];
    int32_t* smi = reinterpret_cast<int32_t*>(sm);
    const uint32_t G = g.G, R = g.R, P = g.P, n = g.n;
    const uint32_t tid = threadIdx.x, lane = tid & 31, wid = tid >> 5, n_warps = blockDim.x >> 5;
    const uint32_t gpu = tid / kSlotLanes, me = tid % kSlotLanes;        // my modelled GPU, my slot
    const uint32_t base = lane & ~(uint32_t)(kSlotLanes - 1);             // first lane of my group
    const bool has_slot = gpu < G && me < R;
    const SlotLayout L = slot_layout(blockDim.x, G);
    const uint32_t sm_base = (uint32_t)__cvta_generic_to_shared(sm);
    const uint32_t kFull = 0xffffffffu;
    const float* __restrict__ Pm = g.Pm;
    const uint32_t oPT = L.pt + min(gpu, G - 1) * 72;                     // + r * 9 + u
    unsigned long long* s_key = reinterpret_cast<unsigned long long*>(sm + L.key);

    {   // a resident id outside the matrix would send reads out of bounds: refuse the whole call
        bool bad_id = has_slot && me < min(g.count[gpu], R) && (uint32_t)g.ids[gpu * R + me] >= P;
        if (__syncthreads_or(bad_id)) {
            for (uint32_t i = tid; i < n; i += blockDim.x) {
                g.gpu_out[i] = ROOMIE_PLACE_BAD_ID;
                if (g.mean_out) g.mean_out[i] = 0.0f;
                if (g.mu_arr_out) g.mu_arr_out[i] = 0.0f;
            }
            return;
        }
    }

    // ---- initial state: residents occupy slots 0 .. c-1 in arrival order ----
    uint32_t c = gpu < G ? min(g.count[gpu], R) : 0u;                     // same in the eight lanes of a group
    uint32_t ord = 0, free_mask = (1u << R) - 1u;
    for (uint32_t p = 0; p < c; ++p) { ord |= p << (4 * p); free_mask &= ~(1u << p); }
    if (gpu >= G) free_mask = 0;
    bool live = has_slot && me < c;
    int32_t id = live ? g.ids[gpu * R + me] : -1;
    uint32_t ex = kSlotNever;
    if (live) { const uint32_t e = g.expiry[gpu * R + me]; ex = e ? e : kSlotNever; }
    int32_t born = kSlotBornLongAgo;
    float pa = 0.0f;
    if (gpu < G) {                                                        // cache of the resident-resident terms
        for (uint32_t u = 0; u < c; ++u) {
            const int32_t other = g.ids[gpu * R + u];
            if (live) sm[oPT + me * 9 + u] = __ldg(&Pm[(size_t)id * P + other]);
        }
        if (live)
            for (uint32_t u = 0; u < c; ++u)
                if (u != me) pa = __fadd_rn(pa, sm[oPT + me * 9 + u]);    // (own stores only: no barrier needed)
    }
    uint32_t cb = __reduce_max_sync(kFull, c);                            // most residents on a GPU of this warp
    const float* my_row = Pm + (size_t)max(id, 0) * P;                    // P[my resident][*]
    const uint32_t tick0 = *g.tick - k_begin;                             // tick of the stream's first arrival
    const uint32_t oRING = L.ring + tid;                                  // + (stage * 2 + dir) * threads

    // what arrival a (staged index a_local) will need of this lane's resident, and of the arrivals just before it
    const uint32_t ring_to0 = sm_base + 4u * oRING, ring_stage = 8u * blockDim.x, ring_from = 4u * blockDim.x;
    const bool helper = wid == n_warps - 1;                               // the last warp owns no GPU: it fetches the shared terms and files the decisions
    const uint32_t young_lane = sm_base + 4u * (L.young + lane);          // its lanes 0 .. 2 kAhead - 1: (back - 1) * 2 + dir
    auto prefetch = [&](uint32_t a_local, uint32_t a_global) {
        const int32_t inc = max(smi[L.arr + a_local], 0);                 // an id outside the matrix is staged as -1
        const uint32_t stage = a_global & (kSlotStages - 1);
        const float* inc_row = Pm + (size_t)inc * P;                      // P[arrival][*]
        if (live) {
            const uint32_t dst = ring_to0 + stage * ring_stage;
            cp_async_4_s(dst, my_row + inc);
            cp_async_4_s(dst + ring_from, inc_row + id);
        }
        if (helper) {                                                     // (warp-uniform)
            if (lane < 2 * kSlotAhead) {
                const uint32_t back = (lane >> 1) + 1;
                const int32_t old = max(smi[L.arr + a_local - back], 0);  // a_local >= kAhead >= back
                cp_async_4_s(young_lane + stage * (8u * kSlotAhead), (lane & 1u) == 0 ? Pm + (size_t)old * P + inc : inc_row + old);
            }
        }
        cp_async_commit();
    };

    uint32_t k_end = n;                                                   // where this launch stops
    for (uint32_t k0 = k_begin; k0 < n; k0 += kSlotChunk) {
        const uint32_t kn = min(kSlotChunk, n - k0);
        // stage arrival ids [k0 - lead, k0 + kn + lead) and lifetimes [k0, k0 + kn)
        __syncthreads();
        for (uint32_t i = tid; i < kn + 2 * kSlotLead; i += blockDim.x) {
            const long long gi = (long long)k0 + i - kSlotLead;
            int32_t v = 0;
            if (gi >= 0 && gi < (long long)n) { v = g.arr_id[gi]; if ((uint32_t)v >= P) v = -1; }
            smi[L.arr + i] = v;
        }
        for (uint32_t i = tid; i < kn; i += blockDim.x) smi[L.life + i] = (int32_t)g.arr_life[k0 + i];
        __syncthreads();
        if (k0 == k_begin) {                                              // prime: the first kAhead arrivals of this launch
            for (uint32_t a = 0; a < (uint32_t)kSlotAhead; ++a) {
                if (k_begin + a < n) prefetch(a + kSlotLead, k_begin + a); else cp_async_commit();
            }
            cp_async_wait<0>();
            __syncthreads();
        }
        for (uint32_t k = 0; k < kn; ++k) {
            const uint32_t kg = k0 + k, now = tick0 + kg, kl = k + kSlotLead;
            // ---- fetch ahead; the copies of arrival kg + 1 (mine and everybody's) have landed after this wait, and
            // this arrival's barrier makes the shared ones visible before they are read ----
            if (kg + kSlotAhead < n) prefetch(kl + kSlotAhead, kg + kSlotAhead); else cp_async_commit();
            cp_async_wait<kSlotAhead - 1>();
            const int32_t inc = smi[L.arr + kl];
            const bool bad_arrival = inc < 0;

            // ---- departures: residents whose expiry tick has come leave, order kept ----
            const bool dying = live && ex <= now;
            const uint32_t dead_all = __ballot_sync(kFull, dying);
            if (dead_all) {
                const uint32_t gone = (dead_all >> base) & 0xffu;         // my group's departures, by slot
                if (gone) {
                    uint32_t nord = 0, nc = 0;
#pragma unroll
                    for (int t = 0; t < kSlotLanes; ++t) {
                        const uint32_t s = (ord >> (4 * t)) & 7u;
                        if ((uint32_t)t < c && !((gone >> s) & 1u)) { nord |= s << (4 * nc); ++nc; }
                    }
                    ord = nord; c = nc; free_mask |= gone;
                    if (dying) { live = false; id = -1; ex = kSlotNever; born = kSlotBornLongAgo; }

                    // the survivors re-add their partial sums in slot order from the cached terms
                    float v[kSlotLanes];
#pragma unroll
                    for (int t = 0; t < kSlotLanes; ++t) v[t] = sm[oPT + me * 9 + ((ord >> (4 * t)) & 7u)];
                    float acc = 0.0f;
#pragma unroll
                    for (int t = 0; t < kSlotLanes; ++t)
                        acc = __fadd_rn(acc, ((uint32_t)t < c && ((ord >> (4 * t)) & 7u) != me) ? v[t] : 0.0f);
                    if (live) pa = acc;
                }
                cb = __reduce_max_sync(kFull, c);
            }

            // ---- what-if: my resident's drop with the arrival added, then the group's slot-order sums ----
            const uint32_t stage = kg & (kSlotStages - 1);
            const uint32_t d1 = kg - (uint32_t)born;                      // arrivals since placed, minus one
            const bool young = d1 < (uint32_t)kSlotAhead;
            const uint32_t a_to = young ? L.young + (stage * kSlotAhead + d1) * 2 : oRING + (stage * 2) * blockDim.x;
            const float to = sm[a_to];                                     // P[resident][arrival]
            const float from = sm[young ? a_to + 1 : a_to + blockDim.x];   // P[arrival][resident]
            const float mu = __fadd_rn(pa, to);
            // every lane of the group collects the (mu, from) pairs of its GPU's residents in arrival order (independent
            // shuffles, as many as the fullest GPU of this warp has residents) and adds them in that order
            float tot = 0.0f, mu_inc = 0.0f, worst = 0.0f;
#pragma unroll
            for (int t = 0; t < kSlotLanes; ++t) {
                if ((uint32_t)t >= cb) break;                             // (warp-uniform)
                const uint32_t src = base + ((ord >> (4 * t)) & 7u);
                const float m_t = __shfl_sync(kFull, mu, src), f_t = __shfl_sync(kFull, from, src);
                const bool in = (uint32_t)t < c;
                tot = __fadd_rn(tot, in ? m_t : 0.0f);
                mu_inc = __fadd_rn(mu_inc, in ? f_t : 0.0f);
                if (!kPlain) worst = fmaxf(worst, in ? m_t : 0.0f);
            }
            tot = __fadd_rn(tot, mu_inc);
            const float mean = div_small(tot, c + 1);                     // c + 1 <= 9
            uint32_t key_hi = 0xffffffffu;
            if (gpu < G && c < R && !bad_arrival)
                key_hi = kPlain ? (mean < g.lambda ? __float_as_uint(mean) : 0xffffffffu)
                                : decision_key(g, mean, fmaxf(worst, mu_inc), mu_inc);

            // ---- argmin: lowest key, lowest GPU index among equals ----
            const uint32_t best_hi = __reduce_min_sync(kFull, key_hi);
            const uint32_t holders = __ballot_sync(kFull, key_hi == best_hi);
            const uint32_t best_gpu = best_hi != 0xffffffffu ? (tid - lane + (uint32_t)__ffs(holders) - 1u) / kSlotLanes : 0xffffffffu;
            if (lane == 0) s_key[(k & 1u) * 32 + wid] = ((unsigned long long)best_hi << 32) | best_gpu;
            __syncthreads();
            unsigned long long best = lane < n_warps ? s_key[(k & 1u) * 32 + lane] : ~0ull;
            {
                const uint32_t hi = (uint32_t)(best >> 32);
                const uint32_t mhi = __reduce_min_sync(kFull, hi);
                const uint32_t mlo = __reduce_min_sync(kFull, hi == mhi ? (uint32_t)best : 0xffffffffu);
                best = ((unsigned long long)mhi << 32) | mlo;
            }
            const bool placed = (uint32_t)(best >> 32) != 0xffffffffu;
            const uint32_t winner = (uint32_t)best;

            // ---- the winner's group takes the arrival ----
            if (placed && gpu == winner) {
                const uint32_t pn = (uint32_t)__ffs(free_mask) - 1u;      // the slot of the arrival
                const uint32_t life = (uint32_t)smi[L.life + k];
                if (live) {
                    pa = mu;                                               // the what-if sum is now the cached one
                    sm[oPT + me * 9 + pn] = to;                            // P[me][new]
                    sm[oPT + pn * 9 + me] = from;                          // P[new][me]
                }
                if (me == pn) {
                    live = true; id = inc; pa = mu_inc; born = (int32_t)(kg + 1);
                    ex = life ? now + life : kSlotNever;
                    my_row = Pm + (size_t)inc * P;
                    sm[oPT + pn * 9 + pn] = 0.0f;
                    sm[L.out + kSlotChunk + k] = mean;
                    sm[L.out + 2 * kSlotChunk + k] = mu_inc;
                }
                ord |= pn << (4 * c);
                ++c;
                free_mask &= ~(1u << pn);
            }
            if (placed && (winner * kSlotLanes) / 32 == wid) cb = max(cb, __shfl_sync(kFull, c, (winner * kSlotLanes) & 31u));
            if (helper && lane == 0) {
                smi[L.out + k] = placed ? (int32_t)winner : (bad_arrival ? ROOMIE_PLACE_BAD_ID : -1);
                if (!placed) { sm[L.out + kSlotChunk + k] = 0.0f; sm[L.out + 2 * kSlotChunk + k] = 0.0f; }
            }
        }
        __syncthreads();
        for (uint32_t i = tid; i < kn; i += blockDim.x) {
            g.gpu_out[k0 + i] = smi[L.out + i];
            if (g.mean_out) g.mean_out[k0 + i] = sm[L.out + kSlotChunk + i];
            if (g.mu_arr_out) g.mu_arr_out[k0 + i] = sm[L.out + 2 * kSlotChunk + i];
        }
        // a look at the admission rate: should the other kind of kernel take the rest of the stream?
        const uint32_t done = k0 + kn;
        if (g.mailbox && g.may_hand_over && done < n && kn == kPlaceWindow) {
            uint32_t mine = 0;
            for (uint32_t i = tid; i < kn; i += blockDim.x) mine += smi[L.out + i] >= 0 ? 1u : 0u;
            if (kind_for(block_count(mine, &s_placed), kn, g.my_kind) != g.my_kind) { k_end = done; break; }
        }
    }
    cp_async_wait<0>();
    // ---- write back in arrival order: position t of the list holds slot s ----
    if (gpu < G) {
        if (me == 0) g.count[gpu] = c;
        if (has_slot && me >= c) { g.ids[gpu * R + me] = -1; g.expiry[gpu * R + me] = 0u; }
#pragma unroll
        for (int t = 0; t < kSlotLanes; ++t)
            if ((uint32_t)t < c && ((ord >> (4 * t)) & 7u) == me) {
                g.ids[gpu * R + t] = id;
                g.expiry[gpu * R + t] = ex == kSlotNever ? 0u : ex;
            }
    }
    if (tid == 0) {
        *g.tick = tick0 + k_end;
        if (k_end < n) g.mailbox[0] = hand_over_word(k_end, 1 - g.my_kind);
    }
}
