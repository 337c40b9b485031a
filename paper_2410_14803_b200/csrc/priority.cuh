// DPER priority arithmetic shared by the bulk kernel and the refresh kernel
// (Section 5.3; sampling exponent of App. A "Priority-Based Sampling in DPER").
#pragma once

#include "common.cuh"

#include <cmath>

namespace distrl {

struct PrioCfg {
    float w_td, w_rho, w_ent, rho_clip, alpha;
    double scale;
    int scale_pow2; // scale is 2^k, k >= 0: the product with an fp32 mass is exact in fp32
};

#ifdef __CUDACC__
// mass = (w1 |delta| + w2 min(rho, clip) + w3 H)^alpha, rho = exp(logpi - logmu).
// alpha = 0.5 and alpha = 1 take the correctly rounded sqrt / identity.
template <bool FAST_EXP = false>
__device__ __forceinline__ float prio_mass(float delta, float lp, float lm, float H, const PrioCfg &c) {
    // FAST_EXP: ex2.approx; the ratio only matters up to rho_clip, where its relative error stays near 2^-22
    float rho = FAST_EXP ? __expf(lp - lm) : expf(lp - lm);
    float p = c.w_td * fabsf(delta) + c.w_rho * fminf(rho, c.rho_clip) + c.w_ent * H;
    if (c.alpha == 0.5f) return sqrtf(p);
    if (c.alpha == 1.0f) return p;
    return powf(p, c.alpha);
}

// Fixed-point quantiser Q, a function of the fp32 mass alone: the product with
// the scale is exact in fp64 and the conversion rounds half to even.
__device__ __forceinline__ uint32_t prio_quantise(float mass, const PrioCfg &c) {
    if (c.scale_pow2) { // same result as below without fp64: scaling by 2^k is exact, the convert rounds to even
        const float xf = mass * (float)c.scale;
        if (!(xf > 0.f)) return 1u;
        if (xf >= 4294967296.f) return 4294967295u; // no fp32 lies between 2^32 - 1 and 2^32
        const uint32_t qf = __float2uint_rn(xf);
        return qf < 1u ? 1u : qf;
    }
    const double scale = c.scale;
    double x = (double)mass * scale;
    if (!(x > 0.0)) return 1u;
    if (x >= 4294967295.0) return 4294967295u;
    uint32_t q = __double2uint_rn(x);
    return q < 1u ? 1u : q;
}
#endif

static inline int check_prio_cfg(const distrl_prio_cfg *cfg, PrioCfg *out) {
    if (!cfg) return DISTRL_ERR_NULL;
    if (!(cfg->alpha >= 0.f) || !(cfg->scale > 0.f) || cfg->w_td != cfg->w_td || cfg->w_rho != cfg->w_rho ||
        cfg->w_ent != cfg->w_ent || cfg->rho_clip != cfg->rho_clip)
        return DISTRL_ERR_PARAM;
    out->w_td = cfg->w_td; out->w_rho = cfg->w_rho; out->w_ent = cfg->w_ent;
    out->rho_clip = cfg->rho_clip; out->alpha = cfg->alpha; out->scale = (double)cfg->scale;
    {
        int e = 0;
        const float mant = frexpf(cfg->scale, &e); // scale = mant * 2^e, mant in [0.5, 1)
        out->scale_pow2 = (mant == 0.5f && e >= 1 && e <= 64) ? 1 : 0;
    }
    return DISTRL_OK;
}

} // namespace distrl
