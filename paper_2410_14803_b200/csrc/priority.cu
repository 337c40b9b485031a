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
// contiguous range of the buffer.  All threads stream that range, a window of kTrajWindow steps at a
// time (16-byte loads when the arrays are 16-byte aligned; windows then start on multiples of four
// steps), and leave one number per step in shared memory; then every thread adds up the part of its
// own trajectory that lies in the window.  The priority is linear in the three means, so the number
// kept per step is the whole combination w_td |delta_t| + w_rho min(rho_t, clip) + w_ent H_t and its
// trajectory mean is the priority: one sum per trajectory instead of three.
constexpr int kTrajWindow = 2048;

template <bool VEC>
__global__ void __launch_bounds__(kPrioThreads) priority_traj_kernel(
    int64_t n, int64_t m, const int64_t *__restrict__ off, const float *__restrict__ delta,
    const float *__restrict__ lp, const float *__restrict__ lm, const float *__restrict__ ent, PrioCfg c,
    float *__restrict__ mass_out, uint32_t *__restrict__ q_out) {
    __shared__ __align__(16) float s_x[kTrajWindow];
    const int tid = threadIdx.x;
    constexpr float kLog2e = 1.4426950408889634f;
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
        auto term = [&](float d, float x, float y, float h) { // h: the entropy, read only if given
            const float rho = fminf(exp2f((x - y) * kLog2e), c.rho_clip);
            return c.w_td * fabsf(d) + c.w_rho * rho + c.w_ent * (ent ? h : -x);
        };
        float sum = 0.f;
        for (int64_t p = VEC ? (A & ~(int64_t)3) : A; p < B; p += kTrajWindow) {
            const int cnt = (int)((B - p < kTrajWindow) ? B - p : kTrajWindow);
            if (VEC) {
                // four consecutive steps per thread and load; a group that reaches past the buffer's
                // end is fetched step by step.  Steps before A or at and after B belong to other
                // blocks: whatever lands in their slots is never added up.
                float4 vd[2], vp[2], vm[2], ve[2];
#pragma unroll
                for (int u = 0; u < 2; ++u) {
                    const int i = 4 * tid + u * 4 * kPrioThreads;
                    const int64_t t = p + i;
                    if (i < cnt && t + 4 <= n) {
                        vd[u] = __ldcs(reinterpret_cast<const float4 *>(delta + t));
                        vp[u] = __ldcs(reinterpret_cast<const float4 *>(lp + t));
                        vm[u] = __ldcs(reinterpret_cast<const float4 *>(lm + t));
                        ve[u] = ent ? __ldcs(reinterpret_cast<const float4 *>(ent + t)) : make_float4(0.f, 0.f, 0.f, 0.f);
                    } else {
                        float q[4][4];
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            const bool ok = i < cnt && t + e < n;
                            q[0][e] = ok ? delta[t + e] : 0.f;
                            q[1][e] = ok ? lp[t + e] : 0.f;
                            q[2][e] = ok ? lm[t + e] : 0.f;
                            q[3][e] = (ok && ent) ? ent[t + e] : 0.f;
                        }
                        vd[u] = make_float4(q[0][0], q[0][1], q[0][2], q[0][3]);
                        vp[u] = make_float4(q[1][0], q[1][1], q[1][2], q[1][3]);
                        vm[u] = make_float4(q[2][0], q[2][1], q[2][2], q[2][3]);
                        ve[u] = make_float4(q[3][0], q[3][1], q[3][2], q[3][3]);
                    }
                }
#pragma unroll
                for (int u = 0; u < 2; ++u) {
                    const int i = 4 * tid + u * 4 * kPrioThreads;
                    if (i < cnt)
                        *reinterpret_cast<float4 *>(s_x + i) = make_float4(
                            term(vd[u].x, vp[u].x, vm[u].x, ve[u].x), term(vd[u].y, vp[u].y, vm[u].y, ve[u].y),
                            term(vd[u].z, vp[u].z, vm[u].z, ve[u].z), term(vd[u].w, vp[u].w, vm[u].w, ve[u].w));
                }
            } else {
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
                        if (i < cnt) s_x[i] = term(vd[u], vp[u], vm[u], ve[u]);
                    }
                }
            }
            __syncthreads();
            const int64_t lo64 = ((a > p) ? a : p) - p, hi64 = ((b < p + cnt) ? b : p + cnt) - p;
            const int lo = (int)(lo64 < cnt ? lo64 : cnt), hi = (int)(hi64 > 0 ? hi64 : 0); // both in [0, cnt]
            for (int t = lo; t < hi; ++t) sum += s_x[t];
            __syncthreads();
        }
        if (j < m) {
            float ms = 0.f;
            if (b > a) {
                const float inv = 1.f / (float)(b - a);
                const float pr = sum * inv;
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
    // one resident wave of blocks, each striding over the buffer
    if (vec)
        priority_kernel<true><<<grid_for(n / 4 + 1, kPrioThreads, one_wave_blocks(priority_kernel<true>, kPrioThreads)),
                                kPrioThreads, 0, st>>>(n, td_delta, lp, lm, entropy, c, prio_mass_out, prio_q);
    else
        priority_kernel<false><<<grid_for(n, kPrioThreads, one_wave_blocks(priority_kernel<false>, kPrioThreads)),
                                 kPrioThreads, 0, st>>>(n, td_delta, lp, lm, entropy, c, prio_mass_out, prio_q);
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
    if (!off || !prio_q) return DISTRL_ERR_NULL;
    if (n > 0 && (!td_delta || !lp || !lm)) return DISTRL_ERR_NULL; // n == 0: only empty trajectories, nothing is read
    const void *ptrs[] = {td_delta, lp, lm, entropy, prio_mass_out, prio_q};
    for (const void *p : ptrs)
        if (p && !aligned_to(p, 4)) return DISTRL_ERR_ALIGN;
    if (!aligned_to(off, 8)) return DISTRL_ERR_ALIGN;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    bool vec = true;
    for (const void *p : {(const void *)td_delta, (const void *)lp, (const void *)lm, (const void *)entropy})
        if (p && !aligned_to(p, 16)) vec = false;
    // one wave: as many blocks as are resident at once, each striding over its share of the chunks
    const int grid = grid_for(m, kPrioThreads, vec ? one_wave_blocks(priority_traj_kernel<true>, kPrioThreads)
                                                   : one_wave_blocks(priority_traj_kernel<false>, kPrioThreads));
    if (vec)
        priority_traj_kernel<true><<<grid, kPrioThreads, 0, st>>>(n, m, off, td_delta, lp, lm, entropy, c,
                                                                  prio_mass_out, prio_q);
    else
        priority_traj_kernel<false><<<grid, kPrioThreads, 0, st>>>(n, m, off, td_delta, lp, lm, entropy, c,
                                                                   prio_mass_out, prio_q);
    DISTRL_CUDA_TRY(cudaGetLastError());
    return DISTRL_OK;
}

DISTRL_BOUNDS_UNIT(priority, 2)
