// What the learner takes from a drawn batch: the scalar each transition carries into the actor
// loss of Section 5.1 (w_j * rho_i * A_i), and, for trajectory-level draws (Section 5.3), the
// transition range a trajectory index stands for.  Both are gathers or plain streams: no
// dependency between outputs, so the kernels are sized for coalescing and loads in flight only.
#include "common.cuh"

#include <cmath>

namespace distrl {

constexpr int kBatchThreads = 256;

__device__ __forceinline__ float actor_term(float lp, float lm, float adv) { return expf(lp - lm) * adv; }

// Whole buffer in order: 12 bytes in, 4 out per transition.
template <bool VEC>
__global__ void __launch_bounds__(kBatchThreads) actor_stream_kernel(
    int64_t n, const float *__restrict__ lp, const float *__restrict__ lm, const float *__restrict__ adv,
    const float *__restrict__ w, float *__restrict__ coef) {
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    const int64_t g = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (VEC) {
        const int64_t n4 = n >> 2;
        for (int64_t v = g; v < n4; v += stride) {
            const float4 p = ldg_stream_f4(lp + 4 * v), m = ldg_stream_f4(lm + 4 * v), a = ldg_stream_f4(adv + 4 * v);
            float4 c = make_float4(actor_term(p.x, m.x, a.x), actor_term(p.y, m.y, a.y),
                                   actor_term(p.z, m.z, a.z), actor_term(p.w, m.w, a.w));
            if (w) {
                const float4 ww = ldg_stream_f4(w + 4 * v);
                c = make_float4(ww.x * c.x, ww.y * c.y, ww.z * c.z, ww.w * c.w);
            }
            stg_stream_f4(coef + 4 * v, c);
        }
        for (int64_t t = 4 * n4 + g; t < n; t += stride) {
            const float c = actor_term(lp[t], lm[t], adv[t]);
            coef[t] = w ? w[t] * c : c;
        }
    } else {
        for (int64_t t = g; t < n; t += stride) {
            const float c = actor_term(lp[t], lm[t], adv[t]);
            coef[t] = w ? w[t] * c : c;
        }
    }
}

// Drawn batch: one thread per batch position, three independent 4-byte gathers each.
__global__ void __launch_bounds__(kBatchThreads) actor_gather_kernel(
    int64_t n, int64_t k, const int64_t *__restrict__ idx, const float *__restrict__ lp,
    const float *__restrict__ lm, const float *__restrict__ adv, const float *__restrict__ w,
    float *__restrict__ coef, int *status) {
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (int64_t j = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; j < k; j += stride) {
        const int64_t i = idx[j];
        if (i < 0 || i >= n) {
            if (status) set_status(status, DISTRL_ERR_INDEX);
            coef[j] = nanf("");
            continue;
        }
        const float c = actor_term(lp[i], lm[i], adv[i]);
        coef[j] = w ? w[j] * c : c;
    }
}

__global__ void __launch_bounds__(kBatchThreads) traj_ranges_kernel(
    int64_t m, const int64_t *__restrict__ off, int64_t k, const int64_t *__restrict__ idx,
    int64_t *__restrict__ begin, int64_t *__restrict__ end, int *status) {
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (int64_t j = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; j < k; j += stride) {
        const int64_t t = idx[j];
        if (t < 0 || t >= m) {
            if (status) set_status(status, DISTRL_ERR_INDEX);
            begin[j] = -1;
            end[j] = -1;
            continue;
        }
        if (!DISTRL_IN(t + 1, m + 1)) continue;
        begin[j] = off[t];
        end[j] = off[t + 1];
    }
}

// Trajectory filter: a warp takes 32 consecutive trajectories, whose steps are one contiguous range of
// the buffer, and walks that range in windows of kFilterWindow steps, one 32-step word per lane.  Per
// window the lane of every trajectory that is not retained toggles two bits in the warp's own 128
// bytes of shared memory, one where its steps begin and one where they end (neighbouring dropped
// trajectories cancel at their common boundary); a running parity over the bits then marks exactly the
// steps to clear: inside each word by five shift-and-XOR steps, across words by one ballot.  The warp
// sweeps the window, 32 consecutive steps per instruction, with coalesced stores of zero where a bit is
// set.  Masses of retained trajectories are neither read nor written.  Warps never meet at a block
// barrier; the loads of the next group of trajectories are sent for before the current one is swept.
// I is the type of a position in the buffer: int when n < 2^31.
constexpr int kFilterWindow = 1024;
constexpr int kFilterWarps = kBatchThreads / 32;

template <typename I>
__global__ void __launch_bounds__(kBatchThreads) filter_kernel(
    int64_t n64, int64_t m, const int64_t *__restrict__ off, const float *__restrict__ score, float threshold,
    uint32_t *__restrict__ q, unsigned long long *kept) {
    __shared__ unsigned int s_tog_all[kFilterWarps][32];
    const int lane = threadIdx.x & 31;
    unsigned int *s_tog = s_tog_all[threadIdx.x >> 5];
    const I n = (I)n64;
    auto inside = [&](int64_t x) { return x < 0 ? (I)0 : (x > n64 ? n : (I)x); };
    const int64_t groups = (m + 31) / 32;
    const int64_t warps = ((int64_t)gridDim.x * blockDim.x) >> 5;
    int64_t g = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    unsigned int kept_here = 0; // lane 0: trajectories this warp retained
    // what the lane needs of trajectory 32 g + lane: its two offsets and its score
    auto fetch = [&](int64_t gg, int64_t &ra, int64_t &rb, float &sc) {
        const int64_t j = 32 * gg + lane;
        ra = rb = 0;
        sc = 0.f;
        if (gg < groups && j < m) { ra = __ldg(off + j); rb = __ldg(off + j + 1); sc = __ldg(score + j); }
    };
    int64_t ra, rb;
    float sc;
    fetch(g, ra, rb, sc);
    for (; g < groups; g += warps) { // warp-uniform
        const int64_t j = 32 * g + lane;
        const I a = inside(ra);
        I b = inside(rb);
        if (b < a) b = a;
        const bool valid = j < m;
        const bool keep = valid && sc >= threshold; // NaN: not retained
        fetch(g + warps, ra, rb, sc);                // the next group's loads travel during the sweep
        kept_here += __popc(__ballot_sync(0xffffffffu, keep));
        const bool drop = valid && !keep && b > a;
        const int last_lane = (int)min((int64_t)31, m - 1 - 32 * g);
        const I A = __shfl_sync(0xffffffffu, a, 0);
        I B = __shfl_sync(0xffffffffu, b, last_lane);
        if (B < A) B = A;
        if (!__any_sync(0xffffffffu, drop)) continue; // nothing to clear in this group
        for (I p = A; p < B; p += kFilterWindow) {
            // positions inside a window fit 32 bits: everything below is relative to p
            const int cnt = (int)((B - p < (I)kFilterWindow) ? B - p : (I)kFilterWindow);
            s_tog[lane] = 0u;
            __syncwarp();
            if (drop && b > p && a - p < (I)cnt) {
                const int lo = (a > p) ? (int)(a - p) : 0;                                  // in [0, cnt)
                const int hi = (b - p < (I)cnt) ? (int)(b - p) : kFilterWindow;            // in (lo, cnt) or "to the end"
                atomicXor(&s_tog[lo >> 5], 1u << (lo & 31));
                if (hi < kFilterWindow) atomicXor(&s_tog[hi >> 5], 1u << (hi & 31));
            }
            __syncwarp();
            // running parity: a step is cleared iff an odd number of toggles lies at or before it
            unsigned int x = s_tog[lane];
            x ^= x << 1; x ^= x << 2; x ^= x << 4; x ^= x << 8; x ^= x << 16;
            const unsigned int odd = __ballot_sync(0xffffffffu, x >> 31);    // words that end inside a run
            if (__popc(odd & ((1u << lane) - 1u)) & 1) x = ~x;                // the run of the words before goes on
            // a run that reaches the window's end was left open: nothing beyond the last step
            const int tail = cnt - 32 * lane;
            x = tail >= 32 ? x : (tail > 0 ? x & ((1u << tail) - 1u) : 0u);
            const int words = (cnt + 31) >> 5;
            uint32_t *const qp = q + p + lane;
            for (int wd = 0; wd < words; ++wd) { // 32 consecutive steps per instruction
                const unsigned int mw = __shfl_sync(0xffffffffu, x, wd);
                if (((mw >> lane) & 1u) && DISTRL_IN((int64_t)p + 32 * wd + lane, n64)) qp[32 * wd] = 0u;
            }
            __syncwarp(); // the toggles are cleared for the next window
        }
    }
    if (lane == 0 && kept && kept_here) atomicAdd(kept, (unsigned long long)kept_here);
}

static int batch_grid(int64_t items, int64_t cap) { // cap: one resident wave of the kernel
    int64_t b = ceil_div(items, kBatchThreads);
    if (b < 1) b = 1;
    return (int)(b > cap ? cap : b);
}

} // namespace distrl

using namespace distrl;

extern "C" int distrl_actor_coefficients(int64_t n, const int64_t *idx, int64_t k, const float *logp_target,
                                         const float *logp_behaviour, const float *advantage,
                                         const float *is_weight, float *coef, int *status_out_device,
                                         void *stream) {
    if (n < 0 || n > DISTRL_MAX_N || k < 0 || k > DISTRL_MAX_N) return DISTRL_ERR_SIZE;
    if (k == 0) return DISTRL_OK;
    if (!idx && k != n) return DISTRL_ERR_SIZE;
    if (!logp_target || !logp_behaviour || !advantage || !coef) return DISTRL_ERR_NULL;
    const void *ptrs[] = {logp_target, logp_behaviour, advantage, is_weight, coef, status_out_device};
    bool vec = true;
    for (const void *p : ptrs) {
        if (p && !aligned_to(p, 4)) return DISTRL_ERR_ALIGN;
        if (p && p != status_out_device && !aligned_to(p, 16)) vec = false;
    }
    if (idx && !aligned_to(idx, 8)) return DISTRL_ERR_ALIGN;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (idx) {
        const int grid = batch_grid(k, one_wave_blocks(actor_gather_kernel, kBatchThreads));
        actor_gather_kernel<<<grid, kBatchThreads, 0, st>>>(n, k, idx, logp_target, logp_behaviour, advantage,
                                                            is_weight, coef, status_out_device);
    } else if (vec) {
        const int grid = batch_grid(n / 4 + 1, one_wave_blocks(actor_stream_kernel<true>, kBatchThreads));
        actor_stream_kernel<true><<<grid, kBatchThreads, 0, st>>>(n, logp_target, logp_behaviour, advantage,
                                                                  is_weight, coef);
    } else {
        const int grid = batch_grid(n, one_wave_blocks(actor_stream_kernel<false>, kBatchThreads));
        actor_stream_kernel<false><<<grid, kBatchThreads, 0, st>>>(n, logp_target, logp_behaviour, advantage,
                                                                   is_weight, coef);
    }
    DISTRL_CUDA_TRY(cudaGetLastError());
    return DISTRL_OK;
}

extern "C" int distrl_trajectory_ranges(int64_t m, const int64_t *traj_offsets, const int64_t *idx, int64_t k,
                                        int64_t *begin, int64_t *end, int *status_out_device, void *stream) {
    if (m < 0 || m > DISTRL_MAX_N || k < 0 || k > DISTRL_MAX_N) return DISTRL_ERR_SIZE;
    if (k == 0) return DISTRL_OK;
    if (!traj_offsets || !idx || !begin || !end) return DISTRL_ERR_NULL;
    if (!aligned_to(traj_offsets, 8) || !aligned_to(idx, 8) || !aligned_to(begin, 8) || !aligned_to(end, 8) ||
        (status_out_device && !aligned_to(status_out_device, 4)))
        return DISTRL_ERR_ALIGN;
    const int grid = batch_grid(k, one_wave_blocks(traj_ranges_kernel, kBatchThreads));
    traj_ranges_kernel<<<grid, kBatchThreads, 0, static_cast<cudaStream_t>(stream)>>>(m, traj_offsets, k, idx, begin,
                                                                                     end, status_out_device);
    DISTRL_CUDA_TRY(cudaGetLastError());
    return DISTRL_OK;
}

extern "C" int distrl_filter_trajectories(int64_t n, int64_t m, const int64_t *traj_offsets, const float *traj_score,
                                          float threshold, uint32_t *prio_q, uint64_t *kept_out_device,
                                          void *stream) {
    if (n < 0 || m < 0 || n > DISTRL_MAX_N || m > DISTRL_MAX_N) return DISTRL_ERR_SIZE;
    if (!(threshold == threshold)) return DISTRL_ERR_PARAM;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (kept_out_device) {
        if (!aligned_to(kept_out_device, 8)) return DISTRL_ERR_ALIGN;
        DISTRL_CUDA_TRY(cudaMemsetAsync(kept_out_device, 0, sizeof(uint64_t), st));
    }
    if (m == 0) return DISTRL_OK;
    if (!traj_offsets || !traj_score || (n > 0 && !prio_q)) return DISTRL_ERR_NULL;
    if (!aligned_to(traj_offsets, 8) || !aligned_to(traj_score, 4) || !aligned_to(prio_q, 4)) return DISTRL_ERR_ALIGN;
    if (n < ((int64_t)1 << 31) - kFilterWindow) {
        const int grid = batch_grid(ceil_div(m, 2), one_wave_blocks(filter_kernel<int>, kBatchThreads)); // >= 2 groups per warp
        filter_kernel<int><<<grid, kBatchThreads, 0, st>>>(n, m, traj_offsets, traj_score, threshold, prio_q,
                                                           reinterpret_cast<unsigned long long *>(kept_out_device));
    } else {
        const int grid = batch_grid(ceil_div(m, 2), one_wave_blocks(filter_kernel<int64_t>, kBatchThreads));
        filter_kernel<int64_t><<<grid, kBatchThreads, 0, st>>>(n, m, traj_offsets, traj_score, threshold, prio_q,
                                                               reinterpret_cast<unsigned long long *>(kept_out_device));
    }
    DISTRL_CUDA_TRY(cudaGetLastError());
    return DISTRL_OK;
}

DISTRL_BOUNDS_UNIT(batch, 4)
