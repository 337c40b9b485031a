// Library-wide entry points: status handling, error text, version.
#include "common.cuh"

#include <atomic>
#include <cstdio>

namespace distrl {

static std::atomic<int> g_cooperative{1};
bool cooperative_launch_allowed() { return g_cooperative.load(std::memory_order_relaxed) != 0; }

#ifdef DISTRL_BOUNDS_CHECK
int bounds_take_retrace(long long *rec);
int bounds_take_priority(long long *rec);
int bounds_take_sampler(long long *rec);
int bounds_take_batch(long long *rec);
int bounds_take_replay(long long *rec);
#endif

static thread_local char g_cuda_error[256] = "";

int record_cuda_error(cudaError_t e, const char *what) {
    std::snprintf(g_cuda_error, sizeof(g_cuda_error), "%s: %s (%s)", what, cudaGetErrorName(e),
                  cudaGetErrorString(e));
    return DISTRL_ERR_CUDA;
}

} // namespace distrl

using namespace distrl;

extern "C" int distrl_workspace_init(void *workspace, size_t workspace_bytes, void *stream) {
    if (!workspace) return DISTRL_ERR_NULL;
    if (!aligned_to(workspace, 256) || workspace_bytes < kHeaderBytes) return DISTRL_ERR_WORKSPACE;
    DISTRL_CUDA_TRY(cudaMemsetAsync(workspace, 0, workspace_bytes, static_cast<cudaStream_t>(stream)));
    return DISTRL_OK;
}

extern "C" int distrl_get_status(void *workspace, void *stream) {
    if (!workspace) return DISTRL_ERR_NULL;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int status = 0;
    DISTRL_CUDA_TRY(cudaMemcpyAsync(&status, workspace, sizeof(int), cudaMemcpyDeviceToHost, st));
    DISTRL_CUDA_TRY(cudaStreamSynchronize(st));
    if (status != 0) {
        DISTRL_CUDA_TRY(cudaMemsetAsync(workspace, 0, sizeof(int), st));
        DISTRL_CUDA_TRY(cudaStreamSynchronize(st));
    }
    return status;
}

extern "C" const char *distrl_error_string(int code) {
    switch (code) {
    case DISTRL_OK: return "ok";
    case DISTRL_ERR_NULL: return "a required pointer is NULL";
    case DISTRL_ERR_SIZE: return "invalid size";
    case DISTRL_ERR_ALIGN: return "pointer not aligned to its element size";
    case DISTRL_ERR_WORKSPACE: return "workspace too small or not 256-byte aligned";
    case DISTRL_ERR_CUDA: return "CUDA runtime error";
    case DISTRL_ERR_TIMEOUT: return "a bounded device-side wait ran out";
    case DISTRL_ERR_PARAM: return "parameter out of range";
    case DISTRL_ERR_OFFSETS: return "offsets not non-decreasing from 0 to N";
    case DISTRL_ERR_INDEX: return "index outside [0, n)";
    default: return "unknown status";
    }
}

extern "C" int distrl_set_cooperative_launch(int allowed) {
    return g_cooperative.exchange(allowed ? 1 : 0, std::memory_order_relaxed);
}

extern "C" int distrl_bounds_report(int64_t *record4_host) {
    if (!record4_host) return DISTRL_ERR_NULL;
    for (int i = 0; i < 4; ++i) record4_host[i] = 0;
#ifdef DISTRL_BOUNDS_CHECK
    DISTRL_CUDA_TRY(cudaDeviceSynchronize());
    int (*units[])(long long *) = {bounds_take_retrace, bounds_take_priority, bounds_take_sampler, bounds_take_batch,
                                   bounds_take_replay};
    for (auto take : units) {
        long long rec[4] = {0, 0, 0, 0};
        if (take(rec) != 0) return record_cuda_error(cudaGetLastError(), "distrl_bounds_report");
        if (rec[0] && !record4_host[0]) { record4_host[1] = rec[1]; record4_host[2] = rec[2]; record4_host[3] = rec[3]; }
        record4_host[0] += rec[0];
    }
    return 1;
#else
    return 0;
#endif
}

extern "C" const char *distrl_last_cuda_error(void) { return g_cuda_error; }

extern "C" const char *distrl_version(void) { return "distrl-b200 0.1 (sm_100a)"; }
