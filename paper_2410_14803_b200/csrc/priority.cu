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

// One warp per trajectory: lanes stride over its steps, shuffle-reduce the three
// sums, lane 0 applies the formula to the means.
__global__ void __launch_bounds__(kPrioThreads) priority_traj_kernel(
    int64_t n, int64_t m, const int64_t *__restrict__ off, const float *__restrict__ delta,
    const float *__restrict__ lp, const float *__restrict__ lm, const float *__restrict__ ent, PrioCfg c,
    float *__restrict__ mass_out, uint32_t *__restrict__ q_out) {
    const int lane = threadIdx.x & 31;
    const int64_t warps = ((int64_t)gridDim.x * blockDim.x) >> 5;
    for (int64_t j = (((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5); j < m; j += warps) {
        int64_t a = off[j], b = off[j + 1];
        if (a < 0) a = 0;
        if (b > n) b = n;
        float sd = 0.f, sr = 0.f, sh = 0.f;
        for (int64_t t = a + lane; t < b; t += 32) {
            float p = lp[t];
            sd += fabsf(delta[t]);
            sr += fminf(expf(p - lm[t]), c.rho_clip);
            sh += ent ? ent[t] : -p;
        }
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) {
            sd += __shfl_xor_sync(0xffffffffu, sd, d);
            sr += __shfl_xor_sync(0xffffffffu, sr, d);
            sh += __shfl_xor_sync(0xffffffffu, sh, d);
        }
        if (lane == 0) {
            float ms = 0.f;
            if (b > a) {
                float inv = 1.f / (float)(b - a);
                float p = c.w_td * (sd * inv) + c.w_rho * (sr * inv) + c.w_ent * (sh * inv);
                ms = (c.alpha == 0.5f) ? sqrtf(p) : (c.alpha == 1.0f) ? p : powf(p, c.alpha);
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
    priority_traj_kernel<<<grid_for(m * 32, kPrioThreads, 148 * 8), kPrioThreads, 0, st>>>(
        n, m, off, td_delta, lp, lm, entropy, c, prio_mass_out, prio_q);
    DISTRL_CUDA_TRY(cudaGetLastError());
    return DISTRL_OK;
}
