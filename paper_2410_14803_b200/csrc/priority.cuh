// DPER priority arithmetic shared by the bulk kernel and the refresh kernel
// (Section 5.3; sampling exponent of App. A "Priority-Based Sampling in DPER").
#pragma once

#include "common.cuh"

namespace distrl {

struct PrioCfg {
    float w_td, w_rho, w_ent, rho_clip, alpha;
    double scale;
};

#ifdef __CUDACC__
// mass = (w1 |delta| + w2 min(rho, clip) + w3 H)^alpha, rho = exp(logpi - logmu).
// alpha = 0.5 and alpha = 1 take the correctly rounded sqrt / identity.
__device__ __forceinline__ float prio_mass(float delta, float lp, float lm, float H, const PrioCfg &c) {
    float rho = expf(lp - lm);
    float p = c.w_td * fabsf(delta) + c.w_rho * fminf(rho, c.rho_clip) + c.w_ent * H;
    if (c.alpha == 0.5f) return sqrtf(p);
    if (c.alpha == 1.0f) return p;
    return powf(p, c.alpha);
}

// Fixed-point quantiser Q, a function of the fp32 mass alone: the product with
// the scale is exact in fp64 and the conversion rounds half to even.
__device__ __forceinline__ uint32_t prio_quantise(float mass, double scale) {
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
    return DISTRL_OK;
}

} // namespace distrl
