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

// Validates the arguments and fills a host handle over `workspace`; launches nothing.
int sampler_create(uint32_t *prio_q, int64_t n, void *workspace, size_t workspace_bytes, distrl_sampler **out);
void sampler_tree_base(const distrl_sampler *s, TreeBase *out);
// Levels 3 and above from level 2 (a no-op for trees of one or two levels).
int sampler_build_upper(const distrl_sampler *s, cudaStream_t st);

} // namespace distrl
