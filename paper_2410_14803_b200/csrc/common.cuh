// Shared host/device helpers of the CUDA library (sm_100a).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "distrl.h"

namespace distrl {

// ---- host-side helpers ------------------------------------------------------

// Records the text of a failed CUDA call for distrl_last_cuda_error().
int record_cuda_error(cudaError_t e, const char *what);

// Whether kernels whose blocks wait for one another may be launched cooperatively
// (distrl_set_cooperative_launch; on by default).
bool cooperative_launch_allowed();

#define DISTRL_CUDA_TRY(expr)                                              \
    do {                                                                   \
        cudaError_t e__ = (expr);                                          \
        if (e__ != cudaSuccess) return ::distrl::record_cuda_error(e__, #expr); \
    } while (0)

static inline bool aligned_to(const void *p, size_t a) {
    return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0;
}
static inline size_t round_up(size_t x, size_t a) { return (x + a - 1) / a * a; }
static inline int64_t ceil_div(int64_t a, int64_t b) { return (a + b - 1) / b; }

// Launch with programmatic stream serialisation: the grid may be scheduled while the previous kernel of
// the stream is still draining.  Every kernel launched this way calls grid_dependency_wait() before it
// touches global memory, so it observes exactly what an ordinary launch would.
#ifdef __CUDACC__
template <typename... KArgs, typename... Args>
static inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                                     Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}
#endif

// Blocks of one resident wave of `kernel` on the current device: a grid-stride kernel launched with
// more blocks than fit at once ends with a partly filled second wave.
#ifdef __CUDACC__
template <typename K>
static inline int one_wave_blocks(K kernel, int threads, size_t smem = 0) {
    int dev = 0, sms = 0, per_sm = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0)
        sms = 148;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, threads, smem) != cudaSuccess || per_sm <= 0)
        per_sm = 4;
    return sms * per_sm;
}
#endif

// Every workspace starts with this header (256 bytes reserved).
struct WorkspaceHeader {
    int status;          // sticky device-side status word (distrl_status)
    unsigned int ticket; // dynamic tile counter of the scan
    unsigned int qmin;   // (unused)
    unsigned int done;   // finished-block counter (sampler, draws normalised by the last block)
    unsigned int bad_epoch; // call number whose offsets failed validation (scan)
    unsigned int left;      // (unused)
    unsigned int tok_dense; // token-level scan: the steps own too many tokens on average for the pipelined kernel
    unsigned int pad_;
    unsigned long long scan_ticket; // pipelined fp32 scan: (number of the call << 32) | tiles handed out so far
    // sampler, draws whose blocks wait for one another: two words (low half: batch minimum of the sampled
    // masses, high half: blocks counted in) that take turns, and which of them the next call uses
    unsigned long long pair[2];
    unsigned int phase;
};
static_assert(sizeof(WorkspaceHeader) <= 256, "the header has 256 bytes");
constexpr size_t kHeaderBytes = 256;

// ---- device-side helpers ----------------------------------------------------
#ifdef __CUDACC__

__device__ __forceinline__ unsigned int ld_acquire_u32(const unsigned int *p) {
    unsigned int v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void st_release_u32(unsigned int *p, unsigned int v) {
    asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}

// Wait until the kernels this grid depends on have completed and their writes are visible (a no-op for
// an ordinary launch); let the kernel that follows in the stream be scheduled early.
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void grid_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// Records the first device-side error; later ones are dropped.
__device__ __forceinline__ void set_status(int *status, int code) { atomicCAS(status, 0, code); }

// Checked build (-DDISTRL_BOUNDS_CHECK): the stand-in for a memory checker.  Every index that a kernel
// computes from its inputs or from its own tiling goes through DISTRL_IN(i, n) right before the access;
// an index outside [0, n) is recorded (the first one: source line, index, limit; and a count of all) and
// the access is skipped -- nothing traps and nothing is read or written out of bounds.  The record is
// read with distrl_bounds_report().  In the ordinary build the macro is the constant true.
#ifdef DISTRL_BOUNDS_CHECK
// (one record per translation unit: the library is built without relocatable device code)
static __device__ long long g_bounds_record[4]; // violations, line of the first one, its index, its limit
static __device__ __noinline__ bool bounds_violation(long long i, long long n, int line) {
    if (atomicAdd(reinterpret_cast<unsigned long long *>(&g_bounds_record[0]), 1ull) == 0ull) {
        g_bounds_record[1] = line;
        g_bounds_record[2] = i;
        g_bounds_record[3] = n;
    }
    return false;
}
__device__ __forceinline__ bool bounds_ok(long long i, long long n, int line) {
    return (i >= 0 && i < n) ? true : bounds_violation(i, n, line);
}
#define DISTRL_IN(i, n) (::distrl::bounds_ok((long long)(i), (long long)(n), __LINE__))
#else
#define DISTRL_IN(i, n) (true)
#endif

#endif // __CUDACC__

// Each translation unit with kernels names itself once with DISTRL_BOUNDS_UNIT(name, id): in the checked build
// that defines the function through which distrl_bounds_report() collects (and clears) the unit's record; the
// line it reports is id * 100000 + source line.
#if defined(__CUDACC__) && defined(DISTRL_BOUNDS_CHECK)
#define DISTRL_BOUNDS_UNIT(name, id)                                                                   \
    namespace distrl {                                                                                 \
    int bounds_take_##name(long long *rec) {                                                           \
        const long long zero[4] = {0, 0, 0, 0};                                                        \
        if (cudaMemcpyFromSymbol(rec, g_bounds_record, sizeof(zero)) != cudaSuccess) return -1;        \
        if (cudaMemcpyToSymbol(g_bounds_record, zero, sizeof(zero)) != cudaSuccess) return -1;         \
        if (rec[0]) rec[1] += 100000LL * (id);                                                         \
        return 0;                                                                                      \
    }                                                                                                  \
    }
#else
#define DISTRL_BOUNDS_UNIT(name, id)
#endif

#ifdef __CUDACC__

// Streaming 128-bit loads/stores: data that is touched once should not evict
// what the rest of the pass keeps in L2.
__device__ __forceinline__ float4 ldg_stream_f4(const float *p) {
    return __ldcs(reinterpret_cast<const float4 *>(p));
}
__device__ __forceinline__ void stg_stream_f4(float *p, float4 v) {
    __stcs(reinterpret_cast<float4 *>(p), v);
}

#endif // __CUDACC__

} // namespace distrl
