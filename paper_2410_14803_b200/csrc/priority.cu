// DPER priorities (Section 5.3): an elementwise streaming kernel that turns
// (delta, log pi, log mu, entropy) into the fp32 sampling mass p^alpha and its
// fixed-point uint32 image, and the trajectory-level form the paper writes
// (means over each trajectory).
#include "priority.cuh"

namespace distrl {

constexpr int kPrioThreads = 256;

template <bool VEC>
__global__ void __launch_bounds__(kPrioThreads) priority_kernel(
    int64_t n, const float *__restrict__ delta, const float *__restrict__ lp, const float *__restrict__ lm,
    const float *__restrict__ ent, PrioCfg c, float *__restrict__ mass_out, uint32_t *__restrict__ q_out) {
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    int64_t g = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (VEC) {
        const int64_t n4 = n >> 2;
        for (int64_t v = g; v < n4; v += stride) {
            float4 d = ldg_stream_f4(delta + 4 * v), p = ldg_stream_f4(lp + 4 * v), m = ldg_stream_f4(lm + 4 * v);
            float4 h = ent ? ldg_stream_f4(ent + 4 * v) : make_float4(-p.x, -p.y, -p.z, -p.w);
            float4 ms = make_float4(prio_mass(d.x, p.x, m.x, h.x, c), prio_mass(d.y, p.y, m.y, h.y, c),
                                    prio_mass(d.z, p.z, m.z, h.z, c), prio_mass(d.w, p.w, m.w, h.w, c));
            if (mass_out) stg_stream_f4(mass_out + 4 * v, ms);
            uint4 q = make_uint4(prio_quantise(ms.x, c), prio_quantise(ms.y, c),
                                 prio_quantise(ms.z, c), prio_quantise(ms.w, c));
            *reinterpret_cast<uint4 *>(q_out + 4 * v) = q; // kept in L2: the sampler build reads it next
        }
        for (int64_t t = 4 * n4 + g; t < n; t += stride) {
            float ms = prio_mass(delta[t], lp[t], lm[t], ent ? ent[t] : -lp[t], c);
            if (mass_out) mass_out[t] = ms;
            q_out[t] = prio_quantise(ms, c);
        }
    } else {
        for (int64_t t = g; t < n; t += stride) {
            float ms = prio_mass(delta[t], lp[t], lm[t], ent ? ent[t] : -lp[t], c);
            if (mass_out) mass_out[t] = ms;
            q_out[t] = prio_quantise(ms, c);
        }
    }
}

// Trajectory means: a block takes kPrioThreads consecutive trajectories, whose steps are one
// contiguous range of the buffer.  All threads stream that range with coalesced loads, a window of
// kTrajWindow steps at a time, and leave the three per-step terms (|delta|, min(rho, clip), H) in
// shared memory; then every thread adds up the part of its own trajectory that lies in the window.
// The formula is applied to the means at the end.
constexpr int kTrajWindow = 2048;

__global__ void __launch_bounds__(kPrioThreads) priority_traj_kernel(
    int64_t n, int64_t m, const int64_t *__restrict__ off, const float *__restrict__ delta,
    const float *__restrict__ lp, const float *__restrict__ lm, const float *__restrict__ ent, PrioCfg c,
    float *__restrict__ mass_out, uint32_t *__restrict__ q_out) {
    __shared__ float s_d[kTrajWindow], s_r[kTrajWindow], s_h[kTrajWindow];
    const int tid = threadIdx.x;
    auto inside = [&](int64_t x) { return x < 0 ? (int64_t)0 : (x > n ? n : x); };
    const int64_t chunks = (m + kPrioThreads - 1) / kPrioThreads;
    for (int64_t chunk = blockIdx.x; chunk < chunks; chunk += gridDim.x) { // block-uniform
        const int64_t j0 = chunk * kPrioThreads, j = j0 + tid;
        const int64_t j1 = (j0 + kPrioThreads < m) ? j0 + kPrioThreads : m;
        int64_t a = 0, b = 0;
        if (j < m) {
            a = inside(off[j]);
            b = inside(off[j + 1]);
            if (b < a) b = a;
        }
        const int64_t A = inside(off[j0]);
        int64_t B = inside(off[j1]);
        if (B < A) B = A;
        float sd = 0.f, sr = 0.f, sh = 0.f;
        for (int64_t p = A; p < B; p += kTrajWindow) {
            const int cnt = (int)((B - p < kTrajWindow) ? B - p : kTrajWindow);
            for (int i0 = tid; i0 < cnt; i0 += 4 * kPrioThreads) { // 16 loads in flight per thread
                float vd[4], vp[4], vm[4], ve[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int i = i0 + u * kPrioThreads;
                    const int64_t t = p + (i < cnt ? i : i0);
                    vd[u] = __ldcs(delta + t);
                    vp[u] = __ldcs(lp + t);
                    vm[u] = __ldcs(lm + t);
                    ve[u] = ent ? __ldcs(ent + t) : 0.f;
                }
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int i = i0 + u * kPrioThreads;
                    if (i < cnt) {
                        s_d[i] = fabsf(vd[u]);
                        s_r[i] = fminf(expf(vp[u] - vm[u]), c.rho_clip);
                        s_h[i] = ent ? ve[u] : -vp[u];
                    }
                }
            }
            __syncthreads();
            const int64_t lo = (a > p) ? a : p, hi = (b < p + cnt) ? b : p + cnt;
            for (int64_t t = lo; t < hi; ++t) {
                sd += s_d[t - p];
                sr += s_r[t - p];
                sh += s_h[t - p];
            }
            __syncthreads();
        }
        if (j < m) {
            float ms = 0.f;
            if (b > a) {
                const float inv = 1.f / (float)(b - a);
                const float pr = c.w_td * (sd * inv) + c.w_rho * (sr * inv) + c.w_ent * (sh * inv);
                ms = (c.alpha == 0.5f) ? sqrtf(pr) : (c.alpha == 1.0f) ? pr : powf(pr, c.alpha);
            }
            if (mass_out) mass_out[j] = ms;
            q_out[j] = prio_quantise(ms, c);
        }
    }
}

static int grid_for(int64_t work_items, int threads, int max_blocks) {
    int64_t b = ceil_div(work_items, threads);
    if (b < 1) b = 1;
    return (int)(b > max_blocks ? max_blocks : b);
}

} // namespace distrl

using namespace distrl;

extern "C" int distrl_compute_priorities(int64_t n, const float *td_delta, const float *lp, const float *lm,
                                         const float *entropy, const distrl_prio_cfg *cfg, float *prio_mass_out,
                                         uint32_t *prio_q, void *stream) {
    if (n < 0 || n > DISTRL_MAX_N) return DISTRL_ERR_SIZE;
    PrioCfg c;
    int rc = check_prio_cfg(cfg, &c);
    if (rc) return rc;
    if (n == 0) return DISTRL_OK;
    if (!td_delta || !lp || !lm || !prio_q) return DISTRL_ERR_NULL;
    const void *ptrs[] = {td_delta, lp, lm, entropy, prio_mass_out, prio_q};
    bool vec = true;
    for (const void *p : ptrs) {
        if (p && !aligned_to(p, 4)) return DISTRL_ERR_ALIGN;
        if (p && !aligned_to(p, 16)) vec = false;
    }
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // 148 SMs x 8 resident blocks of 256 threads
    if (vec)
        priority_kernel<true><<<grid_for(n / 4 + 1, kPrioThreads, 148 * 8), kPrioThreads, 0, st>>>(
            n, td_delta, lp, lm, entropy, c, prio_mass_out, prio_q);
    else
        priority_kernel<false><<<grid_for(n, kPrioThreads, 148 * 8), kPrioThreads, 0, st>>>(
            n, td_delta, lp, lm, entropy, c, prio_mass_out, prio_q);
    DISTRL_CUDA_TRY(cudaGetLastError());
    return DISTRL_OK;
}

extern "C" int distrl_compute_priorities_traj(int64_t n, int64_t m, const int64_t *off, const float *td_delta,
                                              const float *lp, const float *lm, const float *entropy,
                                              const distrl_prio_cfg *cfg, float *prio_mass_out, uint32_t *prio_q,
                                              void *stream) {
    if (n < 0 || m < 0 || n > DISTRL_MAX_N || m > DISTRL_MAX_N) return DISTRL_ERR_SIZE;
    PrioCfg c;
    int rc = check_prio_cfg(cfg, &c);
    if (rc) return rc;
    if (m == 0) return DISTRL_OK;
    if (!off || !td_delta || !lp || !lm || !prio_q) return DISTRL_ERR_NULL;
    const void *ptrs[] = {td_delta, lp, lm, entropy, prio_mass_out, prio_q};
    for (const void *p : ptrs)
        if (p && !aligned_to(p, 4)) return DISTRL_ERR_ALIGN;
    if (!aligned_to(off, 8)) return DISTRL_ERR_ALIGN;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    priority_traj_kernel<<<grid_for(m, kPrioThreads, 148 * 8), kPrioThreads, 0, st>>>(
        n, m, off, td_delta, lp, lm, entropy, c, prio_mass_out, prio_q);
    DISTRL_CUDA_TRY(cudaGetLastError());
    return DISTRL_OK;
}
