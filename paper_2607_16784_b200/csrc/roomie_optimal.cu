// Placement quality (Section 5, "Deployment accuracy evaluation against optimal strategies"): the
// deployment of n models on G identical GPUs with the lowest average predicted drop, by trying every
// assignment - the optimum Algorithm 2's decisions are compared with.
//
// With the pairwise-sum estimate the average drop of a deployment is
//     cost = ( sum over i < j on the same GPU of (P[m_i][m_j] + P[m_j][m_i]) ) / n,
// defined in float32: pair terms are accumulated model by model (j ascending, partners i < j
// ascending), one division at the end.  That order lets the search share work: a thread fixes the
// GPUs of models 1..n-3 (model 0 sits on GPU 0), sums their terms once, and enumerates the last two
// models itself; for each of them one pass over the earlier models yields the sums of all G choices
// (a running sum per GPU, every one taking its members' terms in ascending order).
#include "roomie_common.cuh"

namespace roomie {

constexpr int kOptThreads = 256;
constexpr int kOptMaxModels = 16;
constexpr int kOptMaxGpus = 15;

struct OptArgs {
    const float* Pm;
    uint32_t P;
    const int32_t* models;          // [S][n]
    uint32_t n, S, G, R;
    unsigned long long* best_key;   // [S] (cost bits << 32) | code, smaller is better
    unsigned long long n_prefix;    // G^(n-3): codes of the models a thread does not enumerate itself (1 when n <= 3)
    double inv_n;                   // the double nearest to 1/n
};

// c / n, correctly rounded like the float32 division it stands for, for n <= 16: the double product of c and
// the double nearest to 1/n is within 2^-52 (relative) of c/n, while the quotient of a 24-bit c by such an n
// is either a float or at least 2^-30 (relative) away from the midpoint of two neighbouring floats, so
// rounding the product to float32 rounds the quotient.  Larger n take the division.
__device__ __forceinline__ float div_by_n(float c, double inv_n, float fn) {
    return fn <= 16.0f ? __double2float_rn(__dmul_rn((double)c, inv_n)) : __fdiv_rn(c, fn);
}

// pair sums s[i][j] = P[m_i][m_j] + P[m_j][m_i] of one scenario into shared memory
__device__ __forceinline__ void load_pair_sums(const OptArgs& g, const int32_t* models, float* s_pair) {
    for (uint32_t t = threadIdx.x; t < g.n * g.n; t += blockDim.x) {
        const uint32_t i = t / g.n, j = t % g.n;
        const int32_t mi = models[i], mj = models[j];
        s_pair[t] = __fadd_rn(__ldg(&g.Pm[(size_t)mi * g.P + mj]), __ldg(&g.Pm[(size_t)mj * g.P + mi]));
    }
}

// grid: (CTAs per scenario, S)
__global__ void __launch_bounds__(kOptThreads) optimal_assignment_kernel(OptArgs g) {
    __shared__ float s_pair[kOptMaxModels * kOptMaxModels];
    __shared__ unsigned long long s_best[kOptThreads / 32];
    __shared__ float s_acc[2][kOptMaxGpus * kOptThreads];           // per-GPU running sums of the two tail models
    float* acc1 = s_acc[0] + threadIdx.x;
    float* acc2 = s_acc[1] + threadIdx.x;
    const uint32_t sc = blockIdx.y, n = g.n, G = g.G, R = g.R;
    load_pair_sums(g, g.models + (size_t)sc * n, s_pair);
    __syncthreads();
    unsigned long long best = ~0ull;
    const float fn = (float)n;
    const double inv_n = g.inv_n;
    // A thread fixes the GPUs of models 1 .. n-1-kTail (prefix code pc, model 1 the most significant digit) and
    // tries every choice of the last kTail models below it: kTail = 2 when there are at least three models, so
    // that the prefix's digits, feasibility and pair terms are paid once per G*G assignments, not once per G.
    const uint32_t tail = n >= 3 ? 2u : n - 1u;                     // n = 2: one tail model; n = 1: none
    const uint32_t n_fix = n - tail;                                 // models 0 .. n_fix-1 are fixed by the prefix
    for (unsigned long long pc = (unsigned long long)blockIdx.x * kOptThreads + threadIdx.x; pc < g.n_prefix;
         pc += (unsigned long long)gridDim.x * kOptThreads) {
        // digits of the prefix code; 4 bits per model (its GPU) and per GPU (its load)
        unsigned long long assign = 0, load = 1;                    // model 0 on GPU 0
        if (pc >> 32) {                                             // 64-bit division only for codes that need it
            unsigned long long rest = pc;
            for (int k = (int)n_fix - 1; k >= 1; --k) {
                const uint32_t d = (uint32_t)(rest % G);
                rest /= G;
                assign |= (unsigned long long)d << (4 * k);
                load += 1ull << (4 * d);
            }
        } else {
            uint32_t rest = (uint32_t)pc;
            for (int k = (int)n_fix - 1; k >= 1; --k) {
                const uint32_t q = rest / G, d = rest - q * G;
                rest = q;
                assign |= (unsigned long long)d << (4 * k);
                load += 1ull << (4 * d);
            }
        }
        bool ok = true;
        for (uint32_t d = 0; d < G; ++d) ok = ok && ((load >> (4 * d)) & 15ull) <= R;
        if (!ok) continue;
        float tot = 0.0f;                                           // terms among the fixed models
        for (uint32_t j = 1; j < n_fix; ++j) {
            const uint32_t gj = (uint32_t)(assign >> (4 * j)) & 15u;
            for (uint32_t i = 0; i < j; ++i)
                if (((uint32_t)(assign >> (4 * i)) & 15u) == gj) tot = __fadd_rn(tot, s_pair[i * n + j]);
        }
        if (tail == 0) {
            best = 0ull;                                            // a single model: cost 0, code 0
            continue;
        }
        // One pass over the models gives the sums for all G choices of a tail model at once: every GPU's
        // accumulator starts from the sum so far and takes the terms of its own members in ascending
        // order, which is exactly the order of the definition.  The accumulators live in shared memory
        // ([gpu][thread], so the threads of a warp touch consecutive words).
        if (tail == 2) {                                            // model n_fix
            for (uint32_t d = 0; d < G; ++d) acc2[d * kOptThreads] = tot;
            for (uint32_t i = 0; i < n_fix; ++i) {
                float* a2 = acc2 + ((uint32_t)(assign >> (4 * i)) & 15u) * kOptThreads;
                *a2 = __fadd_rn(*a2, s_pair[i * n + n_fix]);
            }
        }
        const uint32_t g2_count = tail == 2 ? G : 1u;
        for (uint32_t d2 = 0; d2 < g2_count; ++d2) {
            unsigned long long assign2 = assign, load2 = load, code2 = pc;
            float tot2 = tot;
            if (tail == 2) {
                if (((load >> (4 * d2)) & 15ull) >= R) continue;
                tot2 = acc2[d2 * kOptThreads];
                assign2 |= (unsigned long long)d2 << (4 * n_fix);
                load2 += 1ull << (4 * d2);
                code2 = pc * G + d2;
            }
            for (uint32_t d = 0; d < G; ++d) acc1[d * kOptThreads] = tot2;      // the last model
            for (uint32_t i = 0; i + 1 < n; ++i) {
                float* a1 = acc1 + ((uint32_t)(assign2 >> (4 * i)) & 15u) * kOptThreads;
                *a1 = __fadd_rn(*a1, s_pair[i * n + (n - 1)]);
            }
            for (uint32_t d = 0; d < G; ++d) {
                if (((load2 >> (4 * d)) & 15ull) >= R) continue;
                const unsigned long long code = code2 * G + d;
                const unsigned long long key =
                    ((unsigned long long)__float_as_uint(div_by_n(acc1[d * kOptThreads], inv_n, fn)) << 32) | code;
                best = key < best ? key : best;
            }
        }
    }
#pragma unroll
    for (int s = 16; s > 0; s >>= 1) {
        const unsigned long long o = __shfl_xor_sync(0xffffffffu, best, s);
        best = o < best ? o : best;
    }
    if ((threadIdx.x & 31) == 0) s_best[threadIdx.x >> 5] = best;
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int w = 1; w < kOptThreads / 32; ++w) best = s_best[w] < best ? s_best[w] : best;
        if (best != ~0ull) atomicMin(&g.best_key[sc], best);
    }
}

// best_key -> cost and assignment per scenario
__global__ void optimal_unpack_kernel(const unsigned long long* best_key, uint32_t S, uint32_t n, uint32_t G,
                                      float* best_cost, int32_t* best_assign) {
    const uint32_t sc = blockIdx.x * blockDim.x + threadIdx.x;
    if (sc >= S) return;
    const unsigned long long key = best_key[sc];
    if (key == ~0ull) {                                             // no feasible deployment
        best_cost[sc] = -1.0f;
        if (best_assign) for (uint32_t k = 0; k < n; ++k) best_assign[(size_t)sc * n + k] = -1;
        return;
    }
    best_cost[sc] = __uint_as_float((uint32_t)(key >> 32));
    if (best_assign) {
        unsigned long long code = key & 0xffffffffull;
        best_assign[(size_t)sc * n] = 0;
        for (uint32_t k = n - 1; k >= 1; --k) { best_assign[(size_t)sc * n + k] = (int32_t)(code % G); code /= G; }
    }
}

// cost of given deployments, one thread per scenario; gpu_of < 0 = model not deployed
__global__ void assignment_cost_kernel(const float* __restrict__ Pm, uint32_t P, const int32_t* __restrict__ models,
                                       const int32_t* __restrict__ gpu_of, uint32_t n, uint32_t S, float* cost) {
    const uint32_t sc = blockIdx.x * blockDim.x + threadIdx.x;
    if (sc >= S) return;
    const int32_t* m = models + (size_t)sc * n;
    const int32_t* a = gpu_of + (size_t)sc * n;
    float tot = 0.0f;
    for (uint32_t j = 1; j < n; ++j)
        for (uint32_t i = 0; i < j; ++i)
            if (a[i] >= 0 && a[i] == a[j])
                tot = __fadd_rn(tot, __fadd_rn(__ldg(&Pm[(size_t)m[i] * P + m[j]]), __ldg(&Pm[(size_t)m[j] * P + m[i]])));
    cost[sc] = __fdiv_rn(tot, (float)n);
}

}  // namespace roomie

using namespace roomie;

extern "C" size_t roomie_optimal_workspace_bytes(uint32_t num_scenarios) { return 8 * (size_t)num_scenarios + 256; }

extern "C" int roomie_optimal_assignment(const float* Pmat, uint32_t P, const int32_t* models, uint32_t n,
                                         uint32_t num_scenarios, uint32_t num_gpus, uint32_t max_residents,
                                         float* best_cost, int32_t* best_assign, void* workspace,
                                         size_t workspace_bytes, void* stream) {
    if (!Pmat || P == 0 || !models || !best_cost || !workspace || n == 0 || n > kOptMaxModels || num_gpus == 0 ||
        num_gpus > (uint32_t)kOptMaxGpus || max_residents == 0 || max_residents > 15)
        return ROOMIE_ERR_INVALID_ARG;
    if (num_scenarios == 0) return ROOMIE_OK;
    if (workspace_bytes < roomie_optimal_workspace_bytes(num_scenarios)) return ROOMIE_ERR_CAPACITY;
    // the code of an assignment (base-G digits of models 1..n-1) must fit 32 bits
    unsigned long long codes = 1, prefix = 1;
    const uint32_t tail = n >= 3 ? 2u : n - 1u;                     // models enumerated inside a thread
    for (uint32_t k = 1; k < n; ++k) {
        codes *= num_gpus;
        if (k + tail < n) prefix *= num_gpus;
        if (codes > (1ull << 32)) return ROOMIE_ERR_CAPACITY;
    }
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    unsigned long long* keys = static_cast<unsigned long long*>(workspace);
    ROOMIE_CUDA_OK(cudaMemsetAsync(keys, 0xFF, 8 * (size_t)num_scenarios, st));
    OptArgs a;
    a.Pm = Pmat; a.P = P; a.models = models; a.n = n; a.S = num_scenarios; a.G = num_gpus; a.R = max_residents;
    a.best_key = keys; a.n_prefix = prefix; a.inv_n = 1.0 / (double)n;
    unsigned long long ctas = (prefix + kOptThreads - 1) / kOptThreads;
    const unsigned long long cap = (unsigned long long)sm_count() * 8;      // enough CTAs to fill the GPU per scenario
    if (ctas > cap) ctas = cap;
    if (num_scenarios > 65535) return ROOMIE_ERR_CAPACITY;
    optimal_assignment_kernel<<<dim3((unsigned)ctas, num_scenarios), kOptThreads, 0, st>>>(a);
    note_launch();
    ROOMIE_CUDA_OK(cudaGetLastError());
    optimal_unpack_kernel<<<(num_scenarios + 127) / 128, 128, 0, st>>>(keys, num_scenarios, n, num_gpus, best_cost,
                                                                       best_assign);
    note_launch();
    ROOMIE_CUDA_OK(cudaGetLastError());
    return ROOMIE_OK;
}

extern "C" int roomie_assignment_cost(const float* Pmat, uint32_t P, const int32_t* models, const int32_t* gpu_of,
                                      uint32_t n, uint32_t num_scenarios, float* cost_out, void* stream) {
    if (!Pmat || P == 0 || !models || !gpu_of || !cost_out || n == 0) return ROOMIE_ERR_INVALID_ARG;
    if (num_scenarios == 0) return ROOMIE_OK;
    assignment_cost_kernel<<<(num_scenarios + 127) / 128, 128, 0, static_cast<cudaStream_t>(stream)>>>(
        Pmat, P, models, gpu_of, n, num_scenarios, cost_out);
    note_launch();
    ROOMIE_CUDA_OK(cudaGetLastError());
    return ROOMIE_OK;
}
