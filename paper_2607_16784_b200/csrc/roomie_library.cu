// Occupancy (Section 3.1, Eq. 1) and library build: tick timelines + packed walk records.
#include "roomie_common.cuh"

namespace roomie {

// ---------------------------------------------------------------------------------------
// K1: occupancy, one launch over the whole kernel table.  Struct-of-arrays in and out;
// the vector variant moves four kernels per thread with 128-bit loads and stores.
// ---------------------------------------------------------------------------------------
struct OccArgs {
    const uint32_t *grid, *threads, *regs, *smem;
    uint32_t* packed4;
    float *occ, *occ_theo;
    uint32_t* phi;
    uint32_t* n_unlaunchable;
    uint32_t n;
    roomie_gpu_spec spec;
};

__device__ __forceinline__ void occ_store_scalar(const OccArgs& a, uint32_t k, const OccResult& r) {
    if (a.packed4) a.packed4[k] = r.b_lim | (r.b_res << 8) | (r.limiter << 16) | (r.warps << 24);
    if (a.occ) a.occ[k] = r.occ;
    if (a.occ_theo) a.occ_theo[k] = r.occ_theo;
    if (a.phi) {
        a.phi[k] = r.warps;
        a.phi[(size_t)a.n + k] = r.phi_regs;
        a.phi[2 * (size_t)a.n + k] = r.phi_smem;
        a.phi[3 * (size_t)a.n + k] = r.b_res;
    }
}

// kVec: the four input columns and the packed / occ / occ_theo outputs are 16-byte aligned, so the first
// n/4*4 kernels go four per thread with 128-bit accesses (the up to three left over are done one by one).
// Row c of phi starts at phi + c*n, so whether it can take 128-bit stores depends on n as well as on the
// pointer: `phi_rows` has bit c set when that row is 16-byte aligned; the other rows get four scalar stores.
template <bool kVec>
__global__ void __launch_bounds__(256) occupancy_kernel(OccArgs a, uint32_t phi_rows) {
    uint32_t bad = 0;
    const uint32_t n4 = kVec ? a.n / 4 : 0;
    if (kVec) {
        for (uint32_t i = blockIdx.x * blockDim.x + threadIdx.x; i < n4; i += gridDim.x * blockDim.x) {
            const uint4 g = __ldg(reinterpret_cast<const uint4*>(a.grid) + i);
            const uint4 t = __ldg(reinterpret_cast<const uint4*>(a.threads) + i);
            const uint4 r = __ldg(reinterpret_cast<const uint4*>(a.regs) + i);
            const uint4 s = __ldg(reinterpret_cast<const uint4*>(a.smem) + i);
            OccResult o[4];
            o[0] = occupancy_of(g.x, t.x, r.x, s.x, a.spec);
            o[1] = occupancy_of(g.y, t.y, r.y, s.y, a.spec);
            o[2] = occupancy_of(g.z, t.z, r.z, s.z, a.spec);
            o[3] = occupancy_of(g.w, t.w, r.w, s.w, a.spec);
#pragma unroll
            for (int j = 0; j < 4; ++j) bad += (o[j].b_lim == 0);
            if (a.packed4) {
                uint4 p;
                p.x = o[0].b_lim | (o[0].b_res << 8) | (o[0].limiter << 16) | (o[0].warps << 24);
                p.y = o[1].b_lim | (o[1].b_res << 8) | (o[1].limiter << 16) | (o[1].warps << 24);
                p.z = o[2].b_lim | (o[2].b_res << 8) | (o[2].limiter << 16) | (o[2].warps << 24);
                p.w = o[3].b_lim | (o[3].b_res << 8) | (o[3].limiter << 16) | (o[3].warps << 24);
                reinterpret_cast<uint4*>(a.packed4)[i] = p;
            }
            if (a.occ)
                reinterpret_cast<float4*>(a.occ)[i] = make_float4(o[0].occ, o[1].occ, o[2].occ, o[3].occ);
            if (a.occ_theo)
                reinterpret_cast<float4*>(a.occ_theo)[i] =
                    make_float4(o[0].occ_theo, o[1].occ_theo, o[2].occ_theo, o[3].occ_theo);
            if (a.phi) {
                const uint4 rows[4] = {make_uint4(o[0].warps, o[1].warps, o[2].warps, o[3].warps),
                                       make_uint4(o[0].phi_regs, o[1].phi_regs, o[2].phi_regs, o[3].phi_regs),
                                       make_uint4(o[0].phi_smem, o[1].phi_smem, o[2].phi_smem, o[3].phi_smem),
                                       make_uint4(o[0].b_res, o[1].b_res, o[2].b_res, o[3].b_res)};
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    uint32_t* row = a.phi + (size_t)c * a.n + 4 * (size_t)i;
                    if (phi_rows & (1u << c)) *reinterpret_cast<uint4*>(row) = rows[c];
                    else { row[0] = rows[c].x; row[1] = rows[c].y; row[2] = rows[c].z; row[3] = rows[c].w; }
                }
            }
        }
    }
    // everything (scalar variant) or the tail after the last full group of four
    for (uint32_t k = 4 * n4 + blockIdx.x * blockDim.x + threadIdx.x; k < a.n; k += gridDim.x * blockDim.x) {
        const OccResult o = occupancy_of(a.grid[k], a.threads[k], a.regs[k], a.smem[k], a.spec);
        bad += (o.b_lim == 0);
        occ_store_scalar(a, k, o);
    }
    if (a.n_unlaunchable) {
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) bad += __shfl_xor_sync(0xffffffffu, bad, d);
        if ((threadIdx.x & 31) == 0 && bad) atomicAdd(a.n_unlaunchable, bad);
    }
}

// ---------------------------------------------------------------------------------------
// K2: one CTA per profile.  Quantises durations and gaps to ticks, scans them into start
// times, evaluates Eq. 1 for the demand vector and writes the 16-byte walk records.
// ---------------------------------------------------------------------------------------
struct BuildArgs {
    const uint32_t *grid, *threads, *regs, *smem;
    const float *dur_us, *gap_us;
    const uint32_t* offsets;
    uint4* records;
    unsigned long long* T;
    uint32_t* status;
    roomie_gpu_spec spec;
};

constexpr int kBuildThreads = 256;
constexpr int kBuildItems = 4;                       // consecutive kernels per thread and trip

__device__ __forceinline__ uint32_t to_ticks(float us, bool at_least_one, uint32_t& flags) {
    float f = __fmul_rn(us, 1000.0f);
    if (!(f >= 0.0f && f < 2147483648.0f)) { flags |= ROOMIE_FLAG_BAD_TIME; f = 0.0f; }
    uint32_t t = (uint32_t)__float2ll_rn(f);           // round half to even
    return (at_least_one && t < 1u) ? 1u : t;
}

__global__ void __launch_bounds__(kBuildThreads) library_build_kernel(BuildArgs a) {
    __shared__ unsigned long long warp_tot[kBuildThreads / 32];
    __shared__ unsigned long long warp_dur[kBuildThreads / 32];
    const uint32_t m = blockIdx.x;
    const uint32_t lo = a.offsets[m], hi = a.offsets[m + 1];
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    unsigned long long carry = 0, sum_d = 0;
    uint32_t flags = 0;
    for (uint32_t base = lo; base < hi; base += kBuildThreads * kBuildItems) {
        const uint32_t k0 = base + threadIdx.x * kBuildItems;
        uint32_t dt[kBuildItems], gt[kBuildItems];
        unsigned long long mine = 0, d = 0;
#pragma unroll
        for (int j = 0; j < kBuildItems; ++j) {
            dt[j] = gt[j] = 0;
            if (k0 + j < hi) {
                dt[j] = to_ticks(a.dur_us[k0 + j], true, flags);
                gt[j] = to_ticks(a.gap_us[k0 + j], false, flags);
            }
            mine += (unsigned long long)dt[j] + gt[j];
            d += dt[j];
        }
        // inclusive scan of the per-thread sums across the CTA
        unsigned long long v = mine;
#pragma unroll
        for (int s = 1; s < 32; s <<= 1) {
            const unsigned long long up = __shfl_up_sync(0xffffffffu, v, s);
            if (lane >= s) v += up;
        }
#pragma unroll
        for (int s = 16; s > 0; s >>= 1) d += __shfl_xor_sync(0xffffffffu, d, s);
        if (lane == 31) warp_tot[wid] = v;
        if (lane == 0) warp_dur[wid] = d;
        __syncthreads();
        unsigned long long start = carry + v - mine, chunk = 0, chunk_d = 0;
#pragma unroll
        for (int w = 0; w < kBuildThreads / 32; ++w) {
            if (w < wid) start += warp_tot[w];
            chunk += warp_tot[w];
            chunk_d += warp_dur[w];
        }
#pragma unroll
        for (int j = 0; j < kBuildItems; ++j) {
            const uint32_t k = k0 + j;
            if (k < hi) {
                const OccResult o = occupancy_of(a.grid[k], a.threads[k], a.regs[k], a.smem[k], a.spec);
                uint4 rec;
                rec.x = (uint32_t)start;
                rec.y = (uint32_t)(start + dt[j]);
                rec.z = o.phi_regs | (o.warps << kWarpShift);
                rec.w = o.phi_smem | (o.b_res << 22);
                a.records[k] = rec;
                start += (unsigned long long)dt[j] + gt[j];
            }
        }
        carry += chunk;
        sum_d += chunk_d;
        __syncthreads();
    }
    if (carry >= 2147483648ull) flags |= ROOMIE_FLAG_TICK_OVERFLOW;
    if (flags) atomicOr(a.status, flags);
    if (threadIdx.x == 0) a.T[m] = sum_d;
}

static bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Which occupancy kernel a call gets (pointers are only looked at, never dereferenced):
//   bit 0     the 128-bit kernel: n >= 4 and every input column and every packed / occ / occ_theo output
//             (a NULL output counts as aligned) sits on a 16-byte boundary; otherwise the scalar kernel,
//             which has no alignment requirement beyond the element's own;
//   bits 4-7  rows of phi ([4][n]) that take 128-bit stores inside that kernel: row c starts at phi + c*n.
static int occupancy_variant_of(const roomie_kernel_table* t, const roomie_occ_out* o) {
    const bool vec = t->n >= 4 && aligned16(t->grid_blocks) && aligned16(t->block_threads) &&
                     aligned16(t->regs_per_thread) && aligned16(t->smem_per_block) && aligned16(o->packed4) &&
                     aligned16(o->occ) && aligned16(o->occ_theo);
    if (!vec) return 0;
    int rows = 0;
    for (int c = 0; c < 4; ++c)
        if (o->phi && aligned16(o->phi + (size_t)c * t->n)) rows |= 1 << c;
    return 1 | (rows << 4);
}

int validate_spec(const roomie_gpu_spec* s) {
    if (!s) return ROOMIE_ERR_INVALID_ARG;
    if (s->num_sms == 0 || s->threads_per_sm < 32) return ROOMIE_ERR_INVALID_ARG;
    if (s->threads_per_sm / 32u > 255u || s->blocks_per_sm > 255u || s->regs_per_sm >= (1u << 18) ||
        s->smem_per_sm >= (1u << 20))
        return ROOMIE_ERR_RANGE;
    return ROOMIE_OK;
}

}  // namespace roomie

using namespace roomie;

extern "C" int roomie_occupancy(const roomie_kernel_table* table, const roomie_gpu_spec* spec,
                                const roomie_occ_out* out, void* stream) {
    if (!table || !out) return ROOMIE_ERR_INVALID_ARG;
    const int vs = validate_spec(spec);
    if (vs != ROOMIE_OK) return vs;
    if (table->n == 0) return ROOMIE_OK;
    if (!table->grid_blocks || !table->block_threads || !table->regs_per_thread || !table->smem_per_block)
        return ROOMIE_ERR_INVALID_ARG;
    OccArgs a;
    a.grid = table->grid_blocks; a.threads = table->block_threads;
    a.regs = table->regs_per_thread; a.smem = table->smem_per_block;
    a.packed4 = out->packed4; a.occ = out->occ; a.occ_theo = out->occ_theo; a.phi = out->phi;
    a.n_unlaunchable = out->n_unlaunchable;
    a.n = table->n; a.spec = *spec;
    const int variant = occupancy_variant_of(table, out);
    const bool vec = (variant & 1) != 0;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const uint32_t work = vec ? a.n / 4 + 3 : a.n;
    uint32_t blocks = (work + 255) / 256;
    if (blocks > 148 * 16) blocks = 148 * 16;
    if (vec) occupancy_kernel<true><<<blocks, 256, 0, st>>>(a, (uint32_t)variant >> 4);
    else occupancy_kernel<false><<<blocks, 256, 0, st>>>(a, 0u);
    note_launch();
    ROOMIE_CUDA_OK(cudaGetLastError());
    return ROOMIE_OK;
}

extern "C" int roomie_occupancy_variant(const roomie_kernel_table* table, const roomie_occ_out* out) {
    if (!table || !out) return ROOMIE_ERR_INVALID_ARG;
    return occupancy_variant_of(table, out);
}

extern "C" int roomie_library_build(const roomie_library* lib, const roomie_kernel_table* table,
                                    const float* dur_us, const float* gap_us, void* stream) {
    if (!lib || !table || !dur_us || !gap_us) return ROOMIE_ERR_INVALID_ARG;
    const int vs = validate_spec(&lib->spec);
    if (vs != ROOMIE_OK) return vs;
    if (!lib->offsets_host || !lib->offsets || !lib->records || !lib->T || !lib->status)
        return ROOMIE_ERR_INVALID_ARG;
    if (lib->num_profiles == 0 || table->n != lib->num_kernels || lib->offsets_host[0] != 0 ||
        lib->offsets_host[lib->num_profiles] != lib->num_kernels || !aligned16(lib->records))
        return ROOMIE_ERR_INVALID_ARG;
    for (uint32_t m = 0; m < lib->num_profiles; ++m)
        if (lib->offsets_host[m + 1] <= lib->offsets_host[m]) return ROOMIE_ERR_INVALID_ARG;   // empty profile
    if (!table->grid_blocks || !table->block_threads || !table->regs_per_thread || !table->smem_per_block)
        return ROOMIE_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    ROOMIE_CUDA_OK(cudaMemcpyAsync(lib->offsets, lib->offsets_host, sizeof(uint32_t) * (lib->num_profiles + 1),
                                   cudaMemcpyHostToDevice, st));
    BuildArgs a;
    a.grid = table->grid_blocks; a.threads = table->block_threads;
    a.regs = table->regs_per_thread; a.smem = table->smem_per_block;
    a.dur_us = dur_us; a.gap_us = gap_us; a.offsets = lib->offsets;
    a.records = static_cast<uint4*>(lib->records);
    a.T = reinterpret_cast<unsigned long long*>(lib->T);
    a.status = lib->status; a.spec = lib->spec;
    library_build_kernel<<<lib->num_profiles, kBuildThreads, 0, st>>>(a);
    note_launch();
    ROOMIE_CUDA_OK(cudaGetLastError());
    return ROOMIE_OK;
}
