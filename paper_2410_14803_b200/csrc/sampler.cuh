// What the fused Retrace + priority + build pass needs from the sampler's translation unit.
#pragma once

#include "common.cuh"

struct distrl_sampler;

namespace distrl {

// The two lowest levels of the sum tree (level 1: sums of 128 masses, level 2: sums of 32 level-1 entries).
struct TreeBase {
    unsigned long long *lvl1, *lvl2; // lvl2 is null when the tree has a single level
    int64_t n1, n2;
    int levels;
    WorkspaceHeader *hdr;
};

// The words through which the blocks of a normalising draw wait for one another, as a freshly built
// sampler has them (device side; called by whichever kernel builds the tree).
#ifdef __CUDACC__
__device__ __forceinline__ void sampler_handshake_reset(WorkspaceHeader *hdr) {
    hdr->done = 0u;
    hdr->pair[0] = 0xffffffffull; // minimum: none yet; count: 0
    hdr->pair[1] = 0xffffffffull;
    hdr->phase = 0u;
}
#endif

// Validates the arguments and fills a host handle over `workspace`; launches nothing.
int sampler_create(uint32_t *prio_q, int64_t n, void *workspace, size_t workspace_bytes, distrl_sampler **out);
void sampler_tree_base(const distrl_sampler *s, TreeBase *out);
// Levels 3 and above from level 2 (a no-op for trees of one or two levels).
int sampler_build_upper(const distrl_sampler *s, cudaStream_t st);

// What the circular buffer of trajectories needs: the masses of the slots [a, b) replaced by
// src[0 .. b-a) (src null: by zeros), and zeros for a range that only the device knows
// (range_device: int64[2] = begin, end); every partial sum of the tree repaired exactly.
int64_t sampler_size(const distrl_sampler *s);
const uint32_t *sampler_masses(const distrl_sampler *s);
int sampler_overwrite_run(distrl_sampler *s, int64_t a, int64_t b, const uint32_t *src, cudaStream_t st);
int sampler_zero_range(distrl_sampler *s, const int64_t *range_device, cudaStream_t st);

} // namespace distrl
