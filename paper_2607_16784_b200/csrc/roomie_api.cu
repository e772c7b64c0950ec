// Status text, CUDA error capture and launch accounting of libroomie.
#include <stdio.h>
#include "roomie_common.cuh"

namespace roomie {

static thread_local uint64_t t_launches = 0;
static thread_local char t_cuda_error[256] = "no CUDA error recorded";

void note_launch() { ++t_launches; }

int check_cuda(cudaError_t e) {
    if (e == cudaSuccess) return ROOMIE_OK;
    snprintf(t_cuda_error, sizeof(t_cuda_error), "%s (%d): %s", cudaGetErrorName(e), (int)e, cudaGetErrorString(e));
    return ROOMIE_ERR_CUDA;
}

int sm_count() {
    static thread_local int cached_dev = -1, cached = 0;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return 148;
    if (dev != cached_dev) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
        cached = n;
        cached_dev = dev;
    }
    return cached;
}

constexpr int kMaxMarks = 256;
static thread_local bool t_prof_on = false;
static thread_local int t_prof_n = 0;              // completed (begin, end) pairs
static thread_local cudaEvent_t t_prof_ev[2 * kMaxMarks];

void profile_mark(cudaStream_t st, bool begin) {
    if (!t_prof_on || t_prof_n >= kMaxMarks) return;
    cudaEventRecord(t_prof_ev[2 * t_prof_n + (begin ? 0 : 1)], st);
    if (!begin) ++t_prof_n;
}

}  // namespace roomie

extern "C" int roomie_profile_enable(int on) {
    using namespace roomie;
    if (on && !t_prof_on) {
        for (int i = 0; i < 2 * kMaxMarks; ++i) ROOMIE_CUDA_OK(cudaEventCreate(&t_prof_ev[i]));
        t_prof_on = true;
        t_prof_n = 0;
    } else if (!on && t_prof_on) {
        for (int i = 0; i < 2 * kMaxMarks; ++i) cudaEventDestroy(t_prof_ev[i]);
        t_prof_on = false;
        t_prof_n = 0;
    }
    return ROOMIE_OK;
}

extern "C" int roomie_profile_walk_ms(float* total_ms, uint32_t* launches) {
    using namespace roomie;
    if (!total_ms || !launches) return ROOMIE_ERR_INVALID_ARG;
    float tot = 0.0f;
    for (int i = 0; i < t_prof_n; ++i) {
        float ms = 0.0f;
        ROOMIE_CUDA_OK(cudaEventSynchronize(t_prof_ev[2 * i + 1]));
        ROOMIE_CUDA_OK(cudaEventElapsedTime(&ms, t_prof_ev[2 * i], t_prof_ev[2 * i + 1]));
        tot += ms;
    }
    *total_ms = tot;
    *launches = (uint32_t)t_prof_n;
    t_prof_n = 0;
    return ROOMIE_OK;
}

extern "C" const char* roomie_strerror(int status) {
    switch (status) {
        case ROOMIE_OK: return "ok";
        case ROOMIE_ERR_INVALID_ARG: return "invalid argument";
        case ROOMIE_ERR_RANGE: return "GPU spec field out of range for the packed demand record";
        case ROOMIE_ERR_CUDA: return "CUDA runtime error";
        case ROOMIE_ERR_CAPACITY: return "workspace too small or too many alignments per pair";
        default: return "unknown status";
    }
}

extern "C" const char* roomie_last_cuda_error(void) { return roomie::t_cuda_error; }
extern "C" uint64_t roomie_launch_count(void) { return roomie::t_launches; }
extern "C" void roomie_reset_launch_count(void) { roomie::t_launches = 0; }
