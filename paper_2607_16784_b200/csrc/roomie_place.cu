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
// sees), so one CTA walks it with one thread per modelled GPU.  Per GPU and resident the sum
// over the other residents is cached (`partial`); adding the arrival's term last reproduces
// the slot-order float32 sum exactly, so a what-if costs 2 matrix reads per resident.
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
    int matrix_in_smem;
};

constexpr unsigned long long kNoGpu = ~0ull;

__device__ __forceinline__ void recompute_partials(const float* Pm, uint32_t P, const int32_t* ids, float* partial,
                                                   uint32_t c) {
    for (uint32_t t = 0; t < c; ++t) {
        const float* row = Pm + (size_t)ids[t] * P;
        float s = 0.0f;
        for (uint32_t u = 0; u < c; ++u)
            if (u != t) s = __fadd_rn(s, row[ids[u]]);
        partial[t] = s;
    }
}

__global__ void __launch_bounds__(1024) place_kernel(PlaceArgs g) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const uint32_t GR = g.G * g.R;
    int32_t* s_ids = reinterpret_cast<int32_t*>(smem_raw);
    uint32_t* s_exp = reinterpret_cast<uint32_t*>(s_ids + GR);
    float* s_part = reinterpret_cast<float*>(s_exp + GR);
    float* s_P = s_part + GR;
    __shared__ unsigned long long s_key[2][32];

    const uint32_t tid = threadIdx.x, lane = tid & 31, wid = tid >> 5, nwarps = blockDim.x >> 5;
    const float* Pm = g.Pm;
    if (g.matrix_in_smem) {
        for (uint32_t i = tid; i < g.P * g.P; i += blockDim.x) s_P[i] = g.Pm[i];
        Pm = s_P;
    }
    for (uint32_t i = tid; i < GR; i += blockDim.x) { s_ids[i] = g.ids[i]; s_exp[i] = g.expiry[i]; }
    __syncthreads();

    const bool owner = tid < g.G;
    int32_t* my_ids = s_ids + (size_t)tid * g.R;
    uint32_t* my_exp = s_exp + (size_t)tid * g.R;
    float* my_part = s_part + (size_t)tid * g.R;
    uint32_t c = 0, next_exp = 0xffffffffu;
    if (owner) {
        c = min(g.count[tid], g.R);
        recompute_partials(Pm, g.P, my_ids, my_part, c);
        for (uint32_t s = 0; s < c; ++s)
            if (my_exp[s] && my_exp[s] < next_exp) next_exp = my_exp[s];
    }
    const uint32_t tick0 = *g.tick;

    for (uint32_t k = 0; k < g.n; ++k) {
        const uint32_t now = tick0 + k;
        const int32_t inc = __ldg(&g.arr_id[k]);
        unsigned long long key = kNoGpu;
        float mean = 0.0f, mu_inc = 0.0f;
        if (owner) {
            if (next_exp <= now) {                       // departures, order kept
                uint32_t w = 0;
                next_exp = 0xffffffffu;
                for (uint32_t s = 0; s < c; ++s) {
                    const uint32_t e = my_exp[s];
                    if (e != 0 && e <= now) continue;
                    my_ids[w] = my_ids[s]; my_exp[w] = e;
                    if (e && e < next_exp) next_exp = e;
                    ++w;
                }
                for (uint32_t s = w; s < c; ++s) { my_ids[s] = -1; my_exp[s] = 0; }
                c = w;
                recompute_partials(Pm, g.P, my_ids, my_part, c);
            }
            if (c < g.R) {                                // what-if: residents + the arrival
                const float* row_inc = Pm + (size_t)inc * g.P;
                float tot = 0.0f;
                for (uint32_t t = 0; t < c; ++t) {
                    const int32_t id = my_ids[t];
                    const float mu_t = __fadd_rn(my_part[t], Pm[(size_t)id * g.P + inc]);
                    tot = __fadd_rn(tot, mu_t);
                    mu_inc = __fadd_rn(mu_inc, row_inc[id]);
                }
                tot = __fadd_rn(tot, mu_inc);
                mean = __fdiv_rn(tot, (float)(c + 1));
                if (mean < g.lambda)                      // Algorithm 2 line 7; mean >= 0 so its bits order
                    key = ((unsigned long long)__float_as_uint(mean) << 32) | tid;
            }
        }
        // argmin over GPUs, lowest index on equal means
        unsigned long long best = key;
#pragma unroll
        for (int s = 16; s > 0; s >>= 1) {
            const unsigned long long o = __shfl_xor_sync(0xffffffffu, best, s);
            best = o < best ? o : best;
        }
        if (lane == 0) s_key[k & 1][wid] = best;
        __syncthreads();
        best = s_key[k & 1][0];
        for (uint32_t w = 1; w < nwarps; ++w) {
            const unsigned long long o = s_key[k & 1][w];
            best = o < best ? o : best;
        }
        if (best == kNoGpu) {
            if (tid == 0) {
                g.gpu_out[k] = -1;
                if (g.mean_out) g.mean_out[k] = 0.0f;
                if (g.mu_arr_out) g.mu_arr_out[k] = 0.0f;
            }
        } else if (tid == (uint32_t)(best & 0xffffffffu)) {
            const uint32_t life = __ldg(&g.arr_life[k]);
            for (uint32_t t = 0; t < c; ++t)              // the what-if sums become the cached ones
                my_part[t] = __fadd_rn(my_part[t], Pm[(size_t)my_ids[t] * g.P + inc]);
            my_part[c] = mu_inc;
            my_ids[c] = inc;
            const uint32_t e = life ? now + life : 0u;
            my_exp[c] = e;
            if (e && e < next_exp) next_exp = e;
            ++c;
            g.gpu_out[k] = (int32_t)tid;
            if (g.mean_out) g.mean_out[k] = mean;
            if (g.mu_arr_out) g.mu_arr_out[k] = mu_inc;
        }
    }
    if (owner) g.count[tid] = c;
    __syncthreads();
    for (uint32_t i = tid; i < GR; i += blockDim.x) { g.ids[i] = s_ids[i]; g.expiry[i] = s_exp[i]; }
    if (tid == 0) *g.tick = tick0 + g.n;
}

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

extern "C" int roomie_place(const float* Pmat, uint32_t P, const roomie_cluster_state* state, const int32_t* arr_id,
                            const uint32_t* arr_life, uint32_t n, const roomie_opts* opts, int32_t* gpu_out,
                            float* mean_out, float* mu_arr_out, void* stream) {
    if (!Pmat || P == 0 || !state || !opts || !state->ids || !state->expiry || !state->count || !state->tick)
        return ROOMIE_ERR_INVALID_ARG;
    if (state->num_gpus == 0 || state->num_gpus > 1024 || state->max_residents == 0 || state->max_residents > 64 ||
        (uint64_t)state->num_gpus * state->max_residents > 8192)
        return ROOMIE_ERR_INVALID_ARG;
    if (n == 0) return ROOMIE_OK;
    if (!arr_id || !arr_life || !gpu_out) return ROOMIE_ERR_INVALID_ARG;
    PlaceArgs a;
    a.Pm = Pmat; a.P = P; a.G = state->num_gpus; a.R = state->max_residents;
    a.ids = state->ids; a.expiry = state->expiry; a.count = state->count; a.tick = state->tick;
    a.arr_id = arr_id; a.arr_life = arr_life; a.n = n; a.lambda = opts->lambda;
    a.gpu_out = gpu_out; a.mean_out = mean_out; a.mu_arr_out = mu_arr_out;
    const size_t state_bytes = (size_t)a.G * a.R * 12;
    const size_t mat_bytes = (size_t)P * P * sizeof(float);
    a.matrix_in_smem = state_bytes + mat_bytes <= 160 * 1024;
    const size_t smem = state_bytes + (a.matrix_in_smem ? mat_bytes : 0);
    if (smem > 48 * 1024)
        ROOMIE_CUDA_OK(cudaFuncSetAttribute(place_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    const uint32_t threads = ((a.G + 31) / 32) * 32;
    place_kernel<<<1, threads, smem, static_cast<cudaStream_t>(stream)>>>(a);
    note_launch();
    ROOMIE_CUDA_OK(cudaGetLastError());
    return ROOMIE_OK;
}
