// Prioritized proportional sampling over fixed-point masses (App. A,
// "Priority-Based Sampling in DPER": P(i) = p_i^alpha / sum_j p_j^alpha) -- sm_100a.
//
// Data structure: a radix tree of exact uint64 partial sums over the uint32
// masses q.  Level 1 entry g = sum of q[128 g .. 128 g + 127]; level l+1 entry
// g = sum of 32 consecutive level-l entries; the top level has <= 32 entries.
// Integer addition is associative, so descending the tree returns exactly
// min{ i : q_0 + .. + q_i > y }, the answer of a linear scan.
//   build  : one streaming pass over q writes levels 1 and 2, one small block
//            finishes the levels above;
//   sample : one warp per draw; per level one coalesced 256-byte load, a
//            shuffle prefix sum and a ballot; the top levels sit in shared memory;
//   update : for every distinct index the highest batch position wins (what a
//            sequential loop would leave) -- elected per block through a small
//            hash table in shared memory for batches of up to 8192 positions,
//            through a claim word per transition beyond that; the winners store
//            the new mass and add new - old to every ancestor, so the tree stays
//            bit-identical to a rebuild.
#include "priority.cuh"
#include "sampler.cuh"

#include <new>

namespace distrl {

constexpr int kLeaf = 128;      // masses per level-1 entry
constexpr int kFan = 32;        // fan-out above level 1
constexpr int kMaxLevels = 8;   // enough for n <= 2^33
constexpr int kSampleThreads = 512;
constexpr int kTopCap = 4352;                   // tree entries a sampling block caches in shared memory
constexpr int kUpdateThreads = 256;
constexpr int kUpdateChunk = 65536;             // batch positions per pair of update launches
constexpr int kAccCap = 640;                    // tree entries an update block accumulates in shared memory

struct Tree {
    int levels;                     // sum levels 1..levels
    int64_t n;
    int64_t count[kMaxLevels + 1];  // entries of level l (index 0 unused)
    unsigned long long *lvl[kMaxLevels + 1];
    uint32_t *q;
    WorkspaceHeader *hdr;
};

static size_t tree_layout(int64_t n, void *base, Tree *t, size_t *offsets, size_t *claim_off = nullptr,
                          size_t *newq_off = nullptr) {
    int64_t count[kMaxLevels + 1] = {0};
    int levels = 1;
    count[1] = n > 0 ? ceil_div(n, kLeaf) : 1;
    while (count[levels] > kFan && levels < kMaxLevels) {
        count[levels + 1] = ceil_div(count[levels], kFan);
        ++levels;
    }
    size_t o = kHeaderBytes;
    for (int l = 1; l <= levels; ++l) {
        if (offsets) offsets[l] = o;
        if (t) t->lvl[l] = reinterpret_cast<unsigned long long *>(static_cast<char *>(base) + o);
        o = round_up(o + sizeof(unsigned long long) * count[l], 256);
    }
    if (claim_off) *claim_off = o;
    o = round_up(o + sizeof(unsigned int) * (size_t)(n > 0 ? n : 1), 256);      // claim[n]
    if (newq_off) *newq_off = o;
    o = round_up(o + sizeof(uint32_t) * (size_t)kUpdateChunk, 256);             // newq[kUpdateChunk]
    if (t) {
        t->levels = levels;
        t->n = n;
        for (int l = 0; l <= kMaxLevels; ++l) t->count[l] = count[l];
        t->hdr = reinterpret_cast<WorkspaceHeader *>(base);
    }
    return o;
}

// mbarrier + 1-D bulk copy (global -> shared), used to fill the sampling blocks' cache
__device__ __forceinline__ unsigned int smem_addr(const void *p) { return (unsigned int)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint64_t *bar, unsigned int count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_addr(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t *bar, unsigned int bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_addr(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t *bar, unsigned int parity) {
    unsigned int ok;
    asm volatile("{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}"
                 : "=r"(ok) : "r"(smem_addr(bar)), "r"(parity) : "memory");
    return ok != 0;
}
__device__ __forceinline__ void bulk_load(void *dst, const void *src, unsigned int bytes, uint64_t *bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_addr(dst)), "l"(src), "r"(bytes), "r"(smem_addr(bar)) : "memory");
}

__device__ __forceinline__ unsigned long long warp_incl_scan_u64(unsigned long long v, int lane) {
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        unsigned long long o = __shfl_up_sync(0xffffffffu, v, d);
        if (lane >= d) v += o;
    }
    return v;
}
__device__ __forceinline__ unsigned long long warp_sum_u64(unsigned long long v) {
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) v += __shfl_xor_sync(0xffffffffu, v, d);
    return v;
}

// ---------------------------------------------------------------------------
// build, pass 1: block b owns level-2 entry b = leaf groups [32 b, 32 b + 32);
// each of its 8 warps sums 4 leaf groups with the 16 loads issued up front.
// ---------------------------------------------------------------------------
__global__ void __launch_bounds__(256) build_leaf_kernel(Tree t, int vec_ok) {
    __shared__ unsigned long long s_l1[kFan];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    grid_launch_dependents(); // pass 2 may be scheduled now; it waits for this grid before it reads
    if (blockIdx.x == 0 && threadIdx.x == 0) sampler_handshake_reset(t.hdr);
    const int64_t g0 = (int64_t)blockIdx.x * kFan + warp * 4;
    unsigned long long s[4];
    if (vec_ok && (g0 + 4) * kLeaf <= t.n) {
        uint4 v[4];
#pragma unroll
        for (int i = 0; i < 4; ++i)
            v[i] = __ldg(reinterpret_cast<const uint4 *>(t.q + (g0 + i) * kLeaf + 4 * lane));
#pragma unroll
        for (int i = 0; i < 4; ++i)
            s[i] = (unsigned long long)v[i].x + v[i].y + v[i].z + v[i].w;
    } else {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            int64_t p = (g0 + i) * kLeaf + 4 * lane;
            s[i] = 0;
#pragma unroll
            for (int e = 0; e < 4; ++e)
                if (p + e < t.n) s[i] += t.q[p + e];
        }
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        s[i] = warp_sum_u64(s[i]);
        if (lane == 0) {
            if (g0 + i < t.count[1]) t.lvl[1][g0 + i] = s[i];
            s_l1[warp * 4 + i] = (g0 + i < t.count[1]) ? s[i] : 0ull;
        }
    }
    if (t.levels < 2) return;
    __syncthreads();
    if (warp == 0) {
        unsigned long long tot = warp_sum_u64(s_l1[lane]);
        if (lane == 0 && blockIdx.x < t.count[2]) t.lvl[2][blockIdx.x] = tot;
    }
}

// build, pass 2: levels 3.. from level 2, one block, launched with programmatic stream serialisation
// (it is scheduled while pass 1 drains).
// Levels 3 .. levels of the tree from level 2, by the THREADS threads of one block (tid = 0 .. THREADS-1;
// `sync` is a barrier over exactly those threads, `s_lvl` 2 x 128 words of their shared memory).  While a
// level has more than 4096 entries: one warp per parent (32 children, one coalesced load).  From there on
// a single round trip to global memory: every thread loads 4096 / THREADS consecutive children, the
// neighbouring threads that share a parent add up with shuffles, and the levels above (at most 128
// entries) are summed out of shared memory.  Level arrays are 256-byte aligned and padded.
template <int THREADS, typename Sync>
__device__ __forceinline__ void tree_build_upper(const Tree &t, int tid, unsigned long long (*s_lvl)[128], Sync sync) {
    static_assert(THREADS == 128 || THREADS == 256 || THREADS == 512 || THREADS == 1024, "2 .. 32 children per thread");
    constexpr int kPer = 4096 / THREADS;      // children per thread
    constexpr int kShare = kFan / kPer;   // threads per parent
    const int lane = tid & 31, warp = tid >> 5;
    auto warp_sum = [](unsigned long long v) {
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) v += __shfl_xor_sync(0xffffffffu, v, d);
        return v;
    };
    int l = 3;
    for (; l <= t.levels && t.count[l - 1] > 4096; ++l) {
        for (int64_t e = warp; e < t.count[l]; e += THREADS / 32) {
            const int64_t ch = e * kFan + lane;
            unsigned long long v = (ch < t.count[l - 1] && DISTRL_IN(ch, t.count[l - 1])) ? __ldcg(&t.lvl[l - 1][ch]) : 0ull;
            v = warp_sum(v);
            if (lane == 0 && DISTRL_IN(e, t.count[l])) t.lvl[l][e] = v;
        }
        sync();
    }
    if (l > t.levels) return;
    int cur = 0;
    {
        const int64_t c = t.count[l - 1];
        const unsigned long long *src = t.lvl[l - 1] + (int64_t)kPer * tid;
        unsigned long long v = 0ull;
        if ((int64_t)kPer * tid + kPer <= c) {
            ulonglong2 x[kPer / 2];
#pragma unroll
            for (int e = 0; e < kPer / 2; ++e) x[e] = __ldcg(reinterpret_cast<const ulonglong2 *>(src) + e);
#pragma unroll
            for (int e = 0; e < kPer / 2; ++e) v += x[e].x + x[e].y;
        } else {
#pragma unroll
            for (int e = 0; e < kPer; ++e)
                if ((int64_t)kPer * tid + e < c && DISTRL_IN(kPer * tid + e, c)) v += __ldcg(src + e);
        }
#pragma unroll
        for (int d = kShare / 2; d > 0; d >>= 1) v += __shfl_xor_sync(0xffffffffu, v, d);
        if ((tid % kShare) == 0) {
            s_lvl[cur][tid / kShare] = v; // zero beyond the level's last entry
            if (tid / kShare < t.count[l] && DISTRL_IN(tid / kShare, t.count[l])) t.lvl[l][tid / kShare] = v;
        }
        sync();
    }
    for (++l; l <= t.levels; ++l) { // at most 128 children left: one warp per parent
        const int64_t c = t.count[l - 1];
        if (warp < t.count[l]) {
            const int ch = warp * kFan + lane;
            unsigned long long v = (ch < c && ch < 128) ? s_lvl[cur][ch] : 0ull;
            v = warp_sum(v);
            if (lane == 0) {
                s_lvl[cur ^ 1][warp] = v;
                if (DISTRL_IN(warp, t.count[l])) t.lvl[l][warp] = v;
            }
        }
        sync();
        cur ^= 1;
    }
}
constexpr int kUpperThreads = 1024;
__global__ void __launch_bounds__(kUpperThreads) build_upper_kernel(Tree t) {
    __shared__ unsigned long long s_lvl[2][128];
    grid_dependency_wait();
    tree_build_upper<kUpperThreads>(t, (int)threadIdx.x, s_lvl, [] { __syncthreads(); });
}

__global__ void total_kernel(Tree t, unsigned long long *out) {
    const int lane = threadIdx.x;
    unsigned long long v = (lane < t.count[t.levels]) ? t.lvl[t.levels][lane] : 0ull;
    v = warp_sum_u64(v);
    if (lane == 0) *out = v;
}

// ---------------------------------------------------------------------------
// sample: one warp per draw.  The small top levels of the tree are copied into
// shared memory once per block, so a draw pays one global round trip for that
// copy plus one per remaining level and one for the leaf group.
// ---------------------------------------------------------------------------
__device__ __forceinline__ unsigned long long ld_acquire_u64(const unsigned long long *p) {
    unsigned long long v;
    asm volatile("ld.acquire.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
    return v;
}

__device__ __forceinline__ int pick_lane(unsigned long long incl, unsigned long long v, unsigned long long y) {
    unsigned int mask = __ballot_sync(0xffffffffu, incl > y);
    if (mask) return __ffs(mask) - 1;
    // unreachable while y < sum of the children; stay inside the populated part
    unsigned int nz = __ballot_sync(0xffffffffu, v != 0ull);
    return nz ? (31 - __clz(nz)) : 0;
}

struct TopCache {
    int from;                    // levels >= from are cached (levels + 1: none)
    int off[kMaxLevels + 2];     // start of each cached level inside the cache
    int total;                   // cached entries
};

__global__ void __launch_bounds__(kSampleThreads) sample_kernel(
    Tree t, TopCache tc, const unsigned long long *__restrict__ u, int64_t k, float beta, int normalise,
    int64_t *__restrict__ idx_out, float *__restrict__ w_out, int vec_ok, int together) {
    __shared__ __align__(128) unsigned long long s_top[kTopCap];
    __shared__ __align__(8) uint64_t s_bar;
    __shared__ int s_last;
    __shared__ unsigned int s_qmin; // smallest mass drawn by this block
    __shared__ int s_nothing;       // the total mass is zero: no draw is possible (the same in every block)
    const int lane = threadIdx.x & 31;
    grid_dependency_wait();
    grid_launch_dependents();
    // One thread pulls the cached levels in with bulk asynchronous copies (one round trip for all of
    // them); sizes are rounded up to 16 bytes, the slack lies inside the levels' 256-byte padding.
    if (threadIdx.x == 0) {
        s_qmin = 0xffffffffu;
        s_nothing = 0;
        mbar_init(&s_bar, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        unsigned int bytes = 0;
        for (int l = tc.from; l <= t.levels; ++l) bytes += (unsigned int)((t.count[l] + 1) & ~(int64_t)1) * 8u;
        mbar_expect_tx(&s_bar, bytes);
        for (int l = tc.from; l <= t.levels; ++l)
            bulk_load(&s_top[tc.off[l]], t.lvl[l], (unsigned int)((t.count[l] + 1) & ~(int64_t)1) * 8u, &s_bar);
    }
    const int64_t j = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const unsigned long long uj = (j < k) ? __ldg(u + j) : 0ull; // in flight while the cache fills
    // which of the two hand-shake words this call uses (it is flipped only after every block has counted itself in)
    const unsigned int phase = (together && threadIdx.x == 0) ? (__ldcg(&t.hdr->phase) & 1u) : 0u;
    __syncthreads(); // the barrier object is initialised
    {
        unsigned int spins = 0;
        while (!mbar_try_wait(&s_bar, 0u)) {
            if (++spins > (1u << 24)) { // a copy never landed: report, carry on with what is there
                if (threadIdx.x == 0) set_status(&t.hdr->status, DISTRL_ERR_TIMEOUT);
                break;
            }
        }
    }
    uint32_t my_q = 0u; // mass of this warp's draw, in the lane that found it (`together` mode)
    bool mine = false;
    if (j < k) {
        // top level: its entries sum to the total mass
        int l = t.levels;
        unsigned long long v = 0ull;
        if (lane < t.count[l] && (l < tc.from || DISTRL_IN(tc.off[l] + lane, kTopCap)))
            v = (l >= tc.from) ? s_top[tc.off[l] + lane] : __ldcg(&t.lvl[l][lane]);
        unsigned long long incl = warp_incl_scan_u64(v, lane);
        const unsigned long long total = __shfl_sync(0xffffffffu, incl, 31);
        unsigned long long y = __umul64hi(uj, total);
        int64_t node = 0;
        if (total == 0ull) { // every mass is zero (an empty or fully filtered buffer): there is nothing to draw
            if (lane == 0) {
                set_status(&t.hdr->status, DISTRL_ERR_INDEX);
                s_nothing = 1;
                idx_out[j] = -1;
                if (w_out) {
                    w_out[j] = 0.f;
                    if (normalise && together) { my_q = 0xffffffffu; mine = true; }
                }
            }
        } else {
        while (true) {
            int c = pick_lane(incl, v, y);
            y -= __shfl_sync(0xffffffffu, incl - v, c);
            node = node * kFan + c;
            if (--l == 0) break;
            int64_t i = node * kFan + lane;
            if (i < t.count[l] && (l < tc.from || DISTRL_IN(tc.off[l] + i, kTopCap)))
                v = (l >= tc.from) ? s_top[tc.off[l] + (int)i] : __ldcg(&t.lvl[l][i]);
            else v = 0ull;
            incl = warp_incl_scan_u64(v, lane);
        }
        // leaf group `node`: 128 masses, 4 per lane
        const int64_t p = node * kLeaf + 4 * lane;
        uint32_t qv[4];
        if (vec_ok && p + 3 < t.n) {
            uint4 x = __ldcg(reinterpret_cast<const uint4 *>(t.q + p));
            qv[0] = x.x; qv[1] = x.y; qv[2] = x.z; qv[3] = x.w;
        } else {
#pragma unroll
            for (int e = 0; e < 4; ++e) qv[e] = (p + e < t.n) ? __ldcg(t.q + p + e) : 0u;
        }
        v = (unsigned long long)qv[0] + qv[1] + qv[2] + qv[3];
        incl = warp_incl_scan_u64(v, lane);
        int c = pick_lane(incl, v, y);
        y -= __shfl_sync(0xffffffffu, incl - v, c);
        if (lane == c) {
            int e = 0;
#pragma unroll
            for (int f = 0; f < 3; ++f)
                if (e == f && y >= qv[f]) { y -= qv[f]; e = f + 1; }
            int64_t idx = p + e;
            uint32_t qs = (e == 0) ? qv[0] : (e == 1) ? qv[1] : (e == 2) ? qv[2] : qv[3];
            if (idx >= t.n) { idx = t.n - 1; qs = 1u; set_status(&t.hdr->status, DISTRL_ERR_INDEX); }
            idx_out[j] = idx;
            if (w_out) {
                if (normalise && together) {
                    my_q = qs; // stays in the register until the batch minimum is known
                    mine = true;
                } else if (normalise) {
                    w_out[j] = __uint_as_float(qs); // parked here until the batch minimum is known
                } else {
                    w_out[j] = powf((float)((double)t.n * (double)qs / (double)total), -beta);
                }
            }
        }
        }
    }
    if (!(w_out && normalise)) return;
    if (together) {
        // Every block of the grid is resident at once (cooperative launch), so the blocks can wait for one
        // another.  Each adds its smallest mass to a batch minimum and counts itself in; minimum and count are
        // the two halves of one 8-byte word, so a single load tells a waiting block both that everybody has
        // arrived and what the minimum is.  Two such words take turns: the block that arrives last clears the
        // other one and flips the phase for the next call, so nobody has to come back and tidy up.  The
        // largest weight belongs to the smallest sampled mass: w_j = (q_j / q_min)^-beta.  The wait is bounded.
        if (mine) atomicMin(&s_qmin, my_q);
        __syncthreads();
        if (threadIdx.x == 0) {
            unsigned long long *pair = &t.hdr->pair[phase];
            unsigned int *half = reinterpret_cast<unsigned int *>(pair); // [0]: minimum, [1]: blocks counted in
            atomicMin(&half[0], s_qmin);
            unsigned int seen;
            asm volatile("atom.acq_rel.gpu.global.add.u32 %0, [%1], 1;" : "=r"(seen) : "l"(&half[1]) : "memory");
            if (seen + 1u == gridDim.x) {
                // the last to arrive: the other word was read for the last time one call ago
                t.hdr->pair[phase ^ 1u] = 0xffffffffull; // minimum: none yet; count: 0
                st_release_u32(&t.hdr->phase, phase ^ 1u);
            }
            unsigned long long both = ld_acquire_u64(pair);
            unsigned int spins = 0;
            while ((unsigned int)(both >> 32) < gridDim.x) {
                if (++spins > (1u << 22)) { set_status(&t.hdr->status, DISTRL_ERR_TIMEOUT); break; }
                both = ld_acquire_u64(pair);
            }
            s_qmin = (unsigned int)both;
        }
        __syncthreads();
        if (mine) w_out[j] = s_nothing ? 0.f : powf((float)my_q / (float)s_qmin, -beta);
        return;
    }
    // The block that finishes last divides by the batch maximum.  The largest weight belongs to the
    // smallest sampled mass, so w_j = (q_j / q_min)^-beta; that block finds q_min among the parked
    // masses itself, so the other blocks pay a single atomic each.
    __syncthreads();
    if (threadIdx.x == 0) {
        // release: this block's parked masses are visible to whoever sees the count;
        // acquire: the last block sees everybody else's
        unsigned int done;
        asm volatile("atom.acq_rel.gpu.global.add.u32 %0, [%1], 1;" : "=r"(done) : "l"(&t.hdr->done) : "memory");
        s_last = (done == gridDim.x - 1);
    }
    __syncthreads();
    if (!s_last) return;
    if (s_nothing) { // nothing was drawn: the weights stay 0
        if (threadIdx.x == 0) t.hdr->done = 0u;
        return;
    }
    // Up to kTailKeep parked masses per thread stay in registers between the search for the minimum and
    // the rescaling (a batch of 4096 draws is read once); longer batches are read again.
    constexpr int kTailKeep = 8;
    uint32_t kept[kTailKeep];
    unsigned int local_min = 0xffffffffu;
#pragma unroll
    for (int e = 0; e < kTailKeep; ++e) {
        const int64_t i = threadIdx.x + e * (int64_t)blockDim.x;
        kept[e] = (i < k) ? __float_as_uint(__ldcg(w_out + i)) : 0xffffffffu;
        local_min = min(local_min, kept[e]);
    }
    for (int64_t i = threadIdx.x + kTailKeep * (int64_t)blockDim.x; i < k; i += blockDim.x)
        local_min = min(local_min, __float_as_uint(__ldcg(w_out + i)));
    local_min = __reduce_min_sync(0xffffffffu, local_min);
    if (lane == 0) atomicMin(&s_qmin, local_min);
    __syncthreads();
    const double qmin = (double)s_qmin;
#pragma unroll
    for (int e = 0; e < kTailKeep; ++e) {
        const int64_t i = threadIdx.x + e * (int64_t)blockDim.x;
        if (i < k) w_out[i] = powf((float)((double)kept[e] / qmin), -beta);
    }
    for (int64_t i0 = threadIdx.x + kTailKeep * (int64_t)blockDim.x; i0 < k; i0 += 4 * (int64_t)blockDim.x) {
        uint32_t qs[4]; // four loads in flight per thread
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const int64_t i = i0 + e * (int64_t)blockDim.x;
            qs[e] = (i < k) ? __float_as_uint(__ldcg(w_out + i)) : 1u;
        }
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const int64_t i = i0 + e * (int64_t)blockDim.x;
            if (i < k) w_out[i] = powf((float)((double)qs[e] / qmin), -beta);
        }
    }
    if (threadIdx.x == 0) t.hdr->done = 0u; // ready for the next call
}

// ---------------------------------------------------------------------------
// update, in two launches per chunk of batch positions.
//
// A sequential loop over the batch leaves, for an index that occurs several
// times, the value of its highest position.  claim[] has one word per
// transition; position j competes for claim[idx[j]] and the highest one stays.
// The table is never cleared: an entry c counts only if it names a position of
// THIS batch that holds the same index (c < k and idx[c] == i), so whatever an
// earlier call or uninitialised memory left behind is either ignored or is
// itself a correct claim.
//   claim kernel : gathers rho and H, computes the new mass and its fixed-point
//                  image, competes for the claim;
//   apply kernel : the winners store the new mass and add (new - old) to every
//                  ancestor, so the tree equals a rebuild bit for bit.
// ---------------------------------------------------------------------------
struct UpdateWs {
    unsigned int *claim; // [n]
    uint32_t *newq;      // [kUpdateChunk]
};

__global__ void __launch_bounds__(kUpdateThreads) update_claim_kernel(
    Tree t, UpdateWs uw, const int64_t *__restrict__ idx, int k, const float *__restrict__ new_abs_delta,
    const float *__restrict__ lp, const float *__restrict__ lm, const float *__restrict__ ent, PrioCfg c,
    float *__restrict__ mass_out) {
    const int j = blockIdx.x * blockDim.x + threadIdx.x;
    grid_dependency_wait();
    grid_launch_dependents();
    if (j >= k) return;
    const int64_t i = idx[j];
    if (i < 0 || i >= t.n) {
        set_status(&t.hdr->status, DISTRL_ERR_INDEX);
        if (mass_out) mass_out[j] = 0.f;
        return;
    }
    const float p = __ldg(lp + i), m = __ldg(lm + i);
    const float h = ent ? __ldg(ent + i) : -p;
    asm volatile("prefetch.global.L2 [%0];" ::"l"(t.q + i)); // the apply kernel reads it next
    unsigned int *slot = uw.claim + i;
    unsigned int old = *reinterpret_cast<volatile unsigned int *>(slot);
    while (true) {
        const bool legit = old < (unsigned int)k && idx[old] == i;
        if (legit && old >= (unsigned int)j) break;
        const unsigned int prev = atomicCAS(slot, old, (unsigned int)j);
        if (prev == old) break;
        old = prev;
    }
    const float mass = prio_mass(new_abs_delta[j], p, m, h, c);
    if (mass_out) mass_out[j] = mass;
    uw.newq[j] = prio_quantise(mass, c);
}

__global__ void __launch_bounds__(kUpdateThreads) update_apply_kernel(Tree t, UpdateWs uw,
                                                                      const int64_t *__restrict__ idx, int k) {
    __shared__ unsigned long long s_acc[kAccCap]; // pending sums of the small top levels, per block
    __shared__ int s_acc_off[kMaxLevels + 2];
    __shared__ int s_acc_from, s_acc_used;
    grid_dependency_wait();
    grid_launch_dependents();
    if (threadIdx.x == 0) {
        int used = 0, from = t.levels + 1;
        for (int l = t.levels; l >= 1; --l) {
            if (used + t.count[l] > kAccCap) break;
            s_acc_off[l] = used;
            used += (int)t.count[l];
            from = l;
        }
        s_acc_from = from;
        s_acc_used = used;
    }
    __syncthreads();
    const int acc_from = s_acc_from, used = s_acc_used;
    for (int i = threadIdx.x; i < used; i += blockDim.x) s_acc[i] = 0ull;
    __syncthreads();
    const int j = blockIdx.x * blockDim.x + threadIdx.x;
    if (j < k) {
        const int64_t i = idx[j];
        const bool in = (i >= 0 && i < t.n);
        // claim and old mass are fetched together; the old mass is only used by the winner
        const unsigned int cl = in ? __ldcg(uw.claim + i) : 0xffffffffu;
        const uint32_t qo = in ? __ldcg(t.q + i) : 0u;
        if (in && cl == (unsigned int)j) {
            const uint32_t qn = uw.newq[j];
            if (qn != qo) {
                t.q[i] = qn;
                const unsigned long long diff = (unsigned long long)qn - (unsigned long long)qo; // mod 2^64
                int64_t node = i / kLeaf;
                for (int l = 1; l <= t.levels; ++l) {
                    if (!DISTRL_IN(node, t.count[l])) continue;
                    if (l >= acc_from) atomicAdd(&s_acc[s_acc_off[l] + (int)node], diff);
                    else atomicAdd(&t.lvl[l][node], diff);
                    node /= kFan;
                }
            }
        }
    }
    __syncthreads();
    for (int l = acc_from; l <= t.levels; ++l)
        for (int i = threadIdx.x; i < t.count[l]; i += blockDim.x) {
            unsigned long long d = s_acc[s_acc_off[l] + i];
            if (d) atomicAdd(&t.lvl[l][i], d);
        }
}

// ---------------------------------------------------------------------------
// update of a small batch in one launch.  For k <= kSmallBatch the election needs
// no claim table in global memory and no second kernel.  A sequential loop over
// the batch leaves, for an index that occurs several times, the value of its
// highest position; so position j applies its value iff no later position holds
// the same index.  Every block answers that for its own 32 positions: it puts
// their indices into a small hash table in shared memory, then all its threads
// stream the whole batch past that table (one probe per batch entry, almost
// always of an empty slot) and record, per table entry, the highest position at
// which its index occurs.  O(k) work per block, the same for every block.
// ---------------------------------------------------------------------------
constexpr int kSmallBatch = 8192;       // positions the single-launch update serves
constexpr int kSmallThreads = 512;
constexpr int kSmallPerWarp = 2;        // batch positions per warp (one was slower in a chain of rounds, four much slower)
constexpr int kSmallPerBlock = (kSmallThreads / 32) * kSmallPerWarp;
constexpr int kSmallSlots = 4 * kSmallPerBlock;      // hash-table slots of a block (four per position it owns)
constexpr int kSmallKeep = 8;           // batch entries a thread keeps in registers (covers k <= 4096)
constexpr unsigned int kNoIndex = 0xffffffffu; // an empty slot; never a valid index (n < 2^31 on this path)

__device__ __forceinline__ unsigned int slot_of(unsigned int i) { return ((i * 2654435761u) >> 16) & (kSmallSlots - 1); }

__global__ void __launch_bounds__(kSmallThreads) update_small_kernel(
    Tree t, const int64_t *__restrict__ idx, int k, const float *__restrict__ new_abs_delta,
    const float *__restrict__ lp, const float *__restrict__ lm, const float *__restrict__ ent, PrioCfg c,
    float *__restrict__ mass_out) {
    __shared__ unsigned int s_key[kSmallSlots]; // low words of the indices of this block's positions
    __shared__ int s_last[kSmallSlots];         // highest batch position that holds the slot's index
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (int i = threadIdx.x; i < kSmallSlots; i += kSmallThreads) { s_key[i] = kNoIndex; s_last[i] = -1; }
    grid_dependency_wait();
    grid_launch_dependents();
    // Every load that depends on nothing goes out first: this warp's own indices, then the thread's share of
    // the whole batch.  The gathers follow as soon as the own indices are there.
    const int j0 = blockIdx.x * kSmallPerBlock + warp * kSmallPerWarp;
    int64_t my_i[kSmallPerWarp];
#pragma unroll
    for (int u = 0; u < kSmallPerWarp; ++u) my_i[u] = (j0 + u < k) ? idx[j0 + u] : -1;
    int64_t kept[kSmallKeep];
#pragma unroll
    for (int e = 0; e < kSmallKeep; ++e) {
        const int p = threadIdx.x + e * kSmallThreads;
        kept[e] = (p < k) ? idx[p] : -1;
    }
    __syncthreads(); // the table is empty
    float g_val[kSmallPerWarp]; // lane 0: log pi, lane 1: log mu, lane 2: entropy, lane 3: old mass (bits), lane 4: |delta|
    int my_slot[kSmallPerWarp];
#pragma unroll
    for (int u = 0; u < kSmallPerWarp; ++u) {
        const int j = j0 + u;
        g_val[u] = 0.f;
        my_slot[u] = -1;
        if (my_i[u] >= 0 && my_i[u] < t.n) {
            const int64_t i = my_i[u];
            if (lane == 0) g_val[u] = __ldg(lp + i);
            else if (lane == 1) g_val[u] = __ldg(lm + i);
            else if (lane == 2) g_val[u] = ent ? __ldg(ent + i) : 0.f;
            else if (lane == 3) g_val[u] = __uint_as_float(__ldcg(t.q + i));
            else if (lane == 4) g_val[u] = new_abs_delta[j];
            if (lane == 0) { // claim a slot for this index (another position of the block may hold the same one)
                const unsigned int key = (unsigned int)i;
                unsigned int h = slot_of(key);
                for (int probe = 0; probe < kSmallSlots; ++probe) { // the table is a quarter full at most: ends early
                    const unsigned int was = atomicCAS(&s_key[h], kNoIndex, key);
                    if (was == kNoIndex || was == key) { my_slot[u] = (int)h; break; }
                    h = (h + 1) & (kSmallSlots - 1);
                }
            }
        }
    }
    // (the batch entries were sent for before the table was set up: keep them from being fetched only now)
#pragma unroll
    for (int e = 0; e < kSmallKeep; ++e) asm volatile("" : "+l"(kept[e]));
    __syncthreads(); // the table holds this block's indices
    auto note = [&](int p, int64_t i) { // batch position p holds index i: is it one of ours?
        if (i < 0 || i >= t.n) return;
        const unsigned int key = (unsigned int)i;
        unsigned int h = slot_of(key);
        for (int probe = 0; probe < kSmallSlots; ++probe) {
            const unsigned int at = s_key[h];
            if (at == kNoIndex) return;
            if (at == key) { atomicMax(&s_last[h], p); return; }
            h = (h + 1) & (kSmallSlots - 1);
        }
    };
#pragma unroll
    for (int e = 0; e < kSmallKeep; ++e) note(threadIdx.x + e * kSmallThreads, kept[e]);
    for (int p = threadIdx.x + kSmallKeep * kSmallThreads; p < k; p += kSmallThreads) note(p, idx[p]);
    __syncthreads(); // every occurrence has been recorded
#pragma unroll
    for (int u = 0; u < kSmallPerWarp; ++u) {
        const int j = j0 + u;
        if (j >= k) break; // warp-uniform
        const int64_t i = my_i[u];
        if (i < 0 || i >= t.n) {
            if (lane == 0) {
                set_status(&t.hdr->status, DISTRL_ERR_INDEX);
                if (mass_out) mass_out[j] = 0.f;
            }
            continue;
        }
        const float p = __shfl_sync(0xffffffffu, g_val[u], 0), m = __shfl_sync(0xffffffffu, g_val[u], 1);
        const float h_in = __shfl_sync(0xffffffffu, g_val[u], 2);
        const uint32_t qo = __float_as_uint(__shfl_sync(0xffffffffu, g_val[u], 3));
        const float nd = __shfl_sync(0xffffffffu, g_val[u], 4);
        if (lane == 0) {
            const bool later = my_slot[u] >= 0 && s_last[my_slot[u]] > j; // a later position holds the same index
            const float mass = prio_mass(nd, p, m, ent ? h_in : -p, c);
            if (mass_out) mass_out[j] = mass;
            const uint32_t qn = prio_quantise(mass, c);
            if (!later && qn != qo) {
                t.q[i] = qn;
                const unsigned long long diff = (unsigned long long)qn - (unsigned long long)qo; // mod 2^64
                // Plain reductions on every level, the few top entries included: summing those per block in
                // shared memory and flushing after a barrier was measured again (per-kernel +1.1 us, no gain
                // for a round), although the top entries' additions, a quarter of the batch each, do delay the
                // draw that follows by about 1 us.
                int64_t node = i / kLeaf;
                for (int l = 1; l <= t.levels; ++l) {
                    if (DISTRL_IN(node, t.count[l])) atomicAdd(&t.lvl[l][node], diff); // result unused: a reduction the thread does not wait for
                    node /= kFan;
                }
            }
        }
    }
}

// ---------------------------------------------------------------------------
// Circular overwrite (App. A, "Circular Replay Buffer": the write index advances as i <- (i+1) mod N and
// new experiences replace the oldest).  The slots [a, b) receive the masses src[0 .. b-a); one warp per
// touched leaf group stores them, recomputes the group's sum from the masses themselves and adds the
// difference to every ancestor, so the tree again equals a rebuild.
// ---------------------------------------------------------------------------
// One leaf group of the overwrite: slots of [a, b) inside group g receive src[i - a] (src null: 0), the
// group's sum is recomputed from the masses themselves and the difference goes to every ancestor.
__device__ __forceinline__ void overwrite_group(const Tree &t, int64_t g, int64_t a, int64_t b,
                                                const uint32_t *__restrict__ src, int lane) {
    unsigned long long sum = 0;
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        const int64_t i = g * kLeaf + 4 * lane + e;
        uint32_t v = 0u;
        if (i < t.n) {
            if (i >= a && i < b && DISTRL_IN(i, t.n)) { v = src ? src[i - a] : 0u; t.q[i] = v; }
            else v = __ldcg(t.q + i);
        }
        sum += v;
    }
    sum = warp_sum_u64(sum);
    if (lane == 0 && DISTRL_IN(g, t.count[1])) {
        const unsigned long long old = t.lvl[1][g];
        t.lvl[1][g] = sum; // this warp is the only writer of the group at this time
        const unsigned long long diff = sum - old; // mod 2^64
        if (diff) {
            int64_t node = g / kFan;
            for (int l = 2; l <= t.levels; ++l) {
                if (DISTRL_IN(node, t.count[l])) atomicAdd(&t.lvl[l][node], diff);
                node /= kFan;
            }
        }
    }
}

__global__ void __launch_bounds__(256) overwrite_kernel(Tree t, int64_t a, int64_t b, const uint32_t *__restrict__ src) {
    grid_dependency_wait();
    grid_launch_dependents();
    const int lane = threadIdx.x & 31;
    const int64_t g = a / kLeaf + (((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5);
    if (g > (b - 1) / kLeaf) return; // warp-uniform
    overwrite_group(t, g, a, b, src, lane);
}

// Zero masses for a range of slots that only the device knows (range[0] .. range[1]; empty when
// end <= begin): one block, its warps striding over the leaf groups.
__global__ void __launch_bounds__(256) zero_range_kernel(Tree t, const int64_t *__restrict__ range) {
    grid_dependency_wait();
    grid_launch_dependents();
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int64_t a = range[0], b = range[1];
    if (a < 0) a = 0;
    if (b > t.n) b = t.n;
    if (b <= a) return;
    for (int64_t g = a / kLeaf + warp; g <= (b - 1) / kLeaf; g += 8) overwrite_group(t, g, a, b, nullptr, lane);
}

} // namespace distrl

using namespace distrl;

struct distrl_sampler {
    Tree tree;
    TopCache top;
    UpdateWs upd;
    size_t offsets[kMaxLevels + 1];
    int vec_ok;
};

extern "C" size_t distrl_sampler_workspace_bytes(int64_t n) {
    if (n < 0) n = 0;
    return tree_layout(n, nullptr, nullptr, nullptr);
}

namespace distrl {

int sampler_create(uint32_t *prio_q, int64_t n, void *workspace, size_t workspace_bytes, distrl_sampler **out) {
    if (!out) return DISTRL_ERR_NULL;
    *out = nullptr;
    if (n < 0 || n > DISTRL_MAX_N) return DISTRL_ERR_SIZE;
    if (!workspace || (n > 0 && !prio_q)) return DISTRL_ERR_NULL;
    if (!aligned_to(prio_q, 4)) return DISTRL_ERR_ALIGN;
    if (!aligned_to(workspace, 256) || workspace_bytes < tree_layout(n, nullptr, nullptr, nullptr))
        return DISTRL_ERR_WORKSPACE;
    distrl_sampler *s = new (std::nothrow) distrl_sampler();
    if (!s) return DISTRL_ERR_CUDA;
    size_t claim_off = 0, newq_off = 0;
    tree_layout(n, workspace, &s->tree, s->offsets, &claim_off, &newq_off);
    s->upd.claim = reinterpret_cast<unsigned int *>(static_cast<char *>(workspace) + claim_off);
    s->upd.newq = reinterpret_cast<uint32_t *>(static_cast<char *>(workspace) + newq_off);
    {   // which top levels fit the sampling blocks' shared-memory cache
        TopCache &tc = s->top;
        tc.from = s->tree.levels + 1;
        tc.total = 0;
        for (int l = s->tree.levels; l >= 1; --l) {
            const int padded = (int)((s->tree.count[l] + 1) & ~(int64_t)1); // whole 16-byte units
            if (tc.total + padded > kTopCap) break;
            tc.off[l] = tc.total;
            tc.total += padded;
            tc.from = l;
        }
    }
    s->tree.q = prio_q;
    s->vec_ok = aligned_to(prio_q, 16) ? 1 : 0;
    *out = s;
    return DISTRL_OK;
}

void sampler_tree_base(const distrl_sampler *s, TreeBase *out) {
    const Tree &t = s->tree;
    out->lvl1 = t.lvl[1];
    out->n1 = t.count[1];
    out->lvl2 = t.levels >= 2 ? t.lvl[2] : nullptr;
    out->n2 = t.levels >= 2 ? t.count[2] : 0;
    out->levels = t.levels;
    out->hdr = t.hdr;
}

int sampler_build_upper(const distrl_sampler *s, cudaStream_t st) {
    if (s->tree.levels >= 3) {
        DISTRL_CUDA_TRY(launch_pdl(build_upper_kernel, dim3(1), dim3(kUpperThreads), 0, st, s->tree));
    }
    return DISTRL_OK;
}

int64_t sampler_size(const distrl_sampler *s) { return s->tree.n; }
const uint32_t *sampler_masses(const distrl_sampler *s) { return s->tree.q; }

int sampler_overwrite_run(distrl_sampler *s, int64_t a, int64_t b, const uint32_t *src, cudaStream_t st) {
    if (b <= a) return DISTRL_OK;
    const int64_t groups = (b - 1) / kLeaf - a / kLeaf + 1;
    DISTRL_CUDA_TRY(launch_pdl(overwrite_kernel, dim3((unsigned)ceil_div(groups * 32, 256)), dim3(256), 0, st, s->tree,
                               a, b, src));
    return DISTRL_OK;
}

int sampler_zero_range(distrl_sampler *s, const int64_t *range_device, cudaStream_t st) {
    DISTRL_CUDA_TRY(launch_pdl(zero_range_kernel, dim3(1), dim3(256), 0, st, s->tree, range_device));
    return DISTRL_OK;
}

} // namespace distrl

extern "C" int distrl_build_sampler(uint32_t *prio_q, int64_t n, void *workspace, size_t workspace_bytes,
                                    void *stream, distrl_sampler **out) {
    int rc = sampler_create(prio_q, n, workspace, workspace_bytes, out);
    if (rc) return rc;
    if (n == 0) return DISTRL_OK;
    distrl_sampler *s = *out;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const Tree &t = s->tree;
    unsigned grid = (unsigned)(t.levels >= 2 ? t.count[2] : 1);
    build_leaf_kernel<<<grid, 256, 0, st>>>(t, s->vec_ok);
    DISTRL_CUDA_TRY(cudaGetLastError());
    return sampler_build_upper(s, st);
}

extern "C" int distrl_sample(distrl_sampler *s, const uint64_t *u_fix, int64_t k, float beta, int normalise,
                             int64_t *idx_out, float *is_weight_out, void *stream) {
    if (!s) return DISTRL_ERR_NULL;
    if (k < 0 || k > DISTRL_MAX_N) return DISTRL_ERR_SIZE;
    if (!(beta == beta)) return DISTRL_ERR_PARAM;
    if (k == 0) return DISTRL_OK;
    if (s->tree.n == 0) return DISTRL_ERR_SIZE; // nothing to draw from
    if (!u_fix || !idx_out) return DISTRL_ERR_NULL;
    if (!aligned_to(u_fix, 8) || !aligned_to(idx_out, 8) || !aligned_to(is_weight_out, 4)) return DISTRL_ERR_ALIGN;
    const int64_t blocks = ceil_div(k * 32, kSampleThreads);
    // blocks may wait for one another only if the whole grid is resident at once
    static int resident[64] = {0};
    int dev = 0;
    DISTRL_CUDA_TRY(cudaGetDevice(&dev));
    int fit = 0;
    if (dev >= 0 && dev < 64) {
        if (!resident[dev]) {
            int per_sm = 0, sms = 0;
            DISTRL_CUDA_TRY(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, sample_kernel, kSampleThreads, 0));
            DISTRL_CUDA_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
            resident[dev] = per_sm * sms > 0 ? per_sm * sms : -1;
        }
        fit = resident[dev];
    }
    const int together = (normalise && is_weight_out && fit > 0 && blocks <= fit && cooperative_launch_allowed()) ? 1 : 0;
    const unsigned long long *u64 = reinterpret_cast<const unsigned long long *>(u_fix);
    if (together) {
        // Blocks that wait for one another must all be on the GPU at the same time whatever else runs
        // there (another stream's kernels, another sampler's draws): a cooperative launch guarantees
        // that, or fails, in which case the call goes the other way below.
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)blocks);
        cfg.blockDim = dim3(kSampleThreads);
        cfg.stream = static_cast<cudaStream_t>(stream);
        cudaLaunchAttribute attr[2];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        attr[1].id = cudaLaunchAttributeCooperative;
        attr[1].val.cooperative = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 2;
        if (cudaLaunchKernelEx(&cfg, sample_kernel, s->tree, s->top, u64, k, beta, normalise, idx_out, is_weight_out,
                               s->vec_ok, 1) == cudaSuccess)
            return DISTRL_OK;
        (void)cudaGetLastError(); // not launched: fall through to the launch that needs no co-residency
    }
    DISTRL_CUDA_TRY(launch_pdl(sample_kernel, dim3((unsigned)blocks), dim3(kSampleThreads), 0,
                               static_cast<cudaStream_t>(stream), s->tree, s->top, u64, k, beta, normalise, idx_out,
                               is_weight_out, s->vec_ok, 0));
    return DISTRL_OK;
}

extern "C" int distrl_update_priorities(distrl_sampler *s, const int64_t *idx, int64_t k,
                                        const float *new_abs_delta, const float *lp, const float *lm,
                                        const float *entropy, const distrl_prio_cfg *cfg, float *mass_out,
                                        void *stream) {
    if (!s) return DISTRL_ERR_NULL;
    if (k < 0 || k > DISTRL_MAX_N) return DISTRL_ERR_SIZE;
    PrioCfg c;
    int rc = check_prio_cfg(cfg, &c);
    if (rc) return rc;
    if (k == 0) return DISTRL_OK;
    if (!idx || !new_abs_delta || !lp || !lm) return DISTRL_ERR_NULL;
    if (!aligned_to(idx, 8) || !aligned_to(new_abs_delta, 4) || !aligned_to(lp, 4) || !aligned_to(lm, 4) ||
        !aligned_to(entropy, 4) || !aligned_to(mass_out, 4))
        return DISTRL_ERR_ALIGN;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (k <= kSmallBatch && s->tree.n < ((int64_t)1 << 31)) { // one launch: the election happens in shared memory
        DISTRL_CUDA_TRY(launch_pdl(update_small_kernel, dim3((unsigned)ceil_div(k, kSmallPerBlock)), dim3(kSmallThreads), 0,
                                   st, s->tree, idx, (int)k, new_abs_delta, lp, lm, entropy, c, mass_out));
        return DISTRL_OK;
    }
    // chunks run one after another on the stream, so "later position wins" also holds across chunks
    for (int64_t o = 0; o < k; o += kUpdateChunk) {
        const int kc = (int)((k - o < kUpdateChunk) ? (k - o) : kUpdateChunk);
        const unsigned grid = (unsigned)ceil_div(kc, kUpdateThreads);
        DISTRL_CUDA_TRY(launch_pdl(update_claim_kernel, dim3(grid), dim3(kUpdateThreads), 0, st, s->tree, s->upd,
                                   idx + o, kc, new_abs_delta + o, lp, lm, entropy, c,
                                   mass_out ? mass_out + o : nullptr));
        DISTRL_CUDA_TRY(launch_pdl(update_apply_kernel, dim3(grid), dim3(kUpdateThreads), 0, st, s->tree, s->upd,
                                   idx + o, kc));
    }
    return DISTRL_OK;
}

extern "C" int distrl_replay_overwrite(distrl_sampler *s, int64_t head, int64_t k, const uint32_t *new_q,
                                       void *stream) {
    if (!s) return DISTRL_ERR_NULL;
    const int64_t n = s->tree.n;
    if (k < 0 || k > DISTRL_MAX_N) return DISTRL_ERR_SIZE;
    if (k == 0) return DISTRL_OK;
    if (n == 0 || head < 0 || head >= n) return DISTRL_ERR_SIZE;
    if (!new_q) return DISTRL_ERR_NULL;
    if (!aligned_to(new_q, 4)) return DISTRL_ERR_ALIGN;
    if (k > n) { // the buffer wraps more than once: only the last n writes survive
        head = (head + (k - n)) % n;
        new_q += (k - n);
        k = n;
    }
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // at most two contiguous runs of slots; launched one after the other, so a leaf group that both
    // touch (tiny buffers) is still written by one warp at a time
    const int64_t first = (head + k <= n) ? k : n - head;
    const int64_t runs[2][3] = {{head, head + first, 0}, {0, k - first, first}};
    for (int r = 0; r < 2; ++r) {
        const int rc = sampler_overwrite_run(s, runs[r][0], runs[r][1], new_q + runs[r][2], st);
        if (rc) return rc;
    }
    return DISTRL_OK;
}

namespace distrl {
// u_out[j] = floor((j 2^64 + u[j]) / k): a uniform from the j-th of k equal strata (in place is fine)
__global__ void stratify_kernel(const unsigned long long *__restrict__ u, long long k, unsigned long long *__restrict__ out) {
    const long long stride = (long long)gridDim.x * blockDim.x;
    for (long long j = (long long)blockIdx.x * blockDim.x + threadIdx.x; j < k; j += stride) {
        const unsigned __int128 x = ((unsigned __int128)(unsigned long long)j << 64) + u[j];
        out[j] = (unsigned long long)(x / (unsigned __int128)(unsigned long long)k);
    }
}
} // namespace distrl

extern "C" int distrl_stratify_uniforms(const uint64_t *u_fix, int64_t k, uint64_t *u_out, void *stream) {
    if (k < 0 || k > DISTRL_MAX_N) return DISTRL_ERR_SIZE;
    if (k == 0) return DISTRL_OK;
    if (!u_fix || !u_out) return DISTRL_ERR_NULL;
    if (!aligned_to(u_fix, 8) || !aligned_to(u_out, 8)) return DISTRL_ERR_ALIGN;
    int64_t grid = ceil_div(k, 256);
    if (grid > 1184) grid = 1184;
    stratify_kernel<<<(unsigned)grid, 256, 0, static_cast<cudaStream_t>(stream)>>>(
        reinterpret_cast<const unsigned long long *>(u_fix), (long long)k, reinterpret_cast<unsigned long long *>(u_out));
    DISTRL_CUDA_TRY(cudaGetLastError());
    return DISTRL_OK;
}

namespace distrl {
constexpr int kMaxShards = 64;
// One replay over several shards: draw j has the global threshold y = floor(u[j] T / 2^64), T the total
// mass of all shards; it belongs to the shard g whose range of cumulative mass holds y, and inside that
// shard it is the draw with threshold y - (total of the shards before g), which the local uniform
// ceil((y - before) 2^64 / T_g) reproduces exactly.
__global__ void route_draws_kernel(const unsigned long long *__restrict__ u, long long k,
                                   const unsigned long long *__restrict__ totals, int n_shards, int me,
                                   unsigned long long *__restrict__ u_local, unsigned char *__restrict__ mine,
                                   int *__restrict__ owner, int *status) {
    __shared__ unsigned long long s_before[kMaxShards + 1];
    __shared__ int s_bad;
    if (threadIdx.x == 0) {
        unsigned __int128 run = 0;
        for (int g = 0; g < n_shards; ++g) {
            s_before[g] = (unsigned long long)run;
            run += totals[g];
        }
        s_before[n_shards] = (unsigned long long)run;
        s_bad = (run == 0 || (run >> 64) != 0) ? 1 : 0; // nothing to draw from, or a total beyond 64 bits
    }
    __syncthreads();
    const long long stride = (long long)gridDim.x * blockDim.x;
    if (s_bad) {
        if (blockIdx.x == 0 && threadIdx.x == 0 && status) set_status(status, DISTRL_ERR_SIZE);
        for (long long j = (long long)blockIdx.x * blockDim.x + threadIdx.x; j < k; j += stride) {
            u_local[j] = 0ull;
            mine[j] = 0;
            if (owner) owner[j] = -1;
        }
        return;
    }
    const unsigned long long grand = s_before[n_shards];
    for (long long j = (long long)blockIdx.x * blockDim.x + threadIdx.x; j < k; j += stride) {
        const unsigned long long y = __umul64hi(u[j], grand); // < grand
        int g = 0;
        while (g + 1 < n_shards && s_before[g + 1] <= y) ++g; // few shards: a linear walk (empty shards are passed over)
        unsigned long long up = 0ull;
        if (g == me) {
            const unsigned long long t = s_before[g + 1] - s_before[g], y_local = y - s_before[g]; // y_local < t
            const unsigned __int128 num = (unsigned __int128)y_local << 64;
            const unsigned long long quo = (unsigned long long)(num / t);
            up = quo + ((unsigned __int128)quo * t != num ? 1ull : 0ull); // the ceiling: still below 2^64 since y_local < t
        }
        u_local[j] = up;
        mine[j] = (g == me) ? 1 : 0;
        if (owner) owner[j] = g;
    }
}
} // namespace distrl

extern "C" int distrl_route_draws(const uint64_t *u_fix, int64_t k, const uint64_t *shard_totals_device, int n_shards,
                                  int my_shard, uint64_t *u_local_out, uint8_t *mine_out, int *owner_out,
                                  int *status_out_device, void *stream) {
    if (k < 0 || k > DISTRL_MAX_N) return DISTRL_ERR_SIZE;
    if (n_shards < 1 || n_shards > kMaxShards || my_shard < 0 || my_shard >= n_shards) return DISTRL_ERR_PARAM;
    if (k == 0) return DISTRL_OK;
    if (!u_fix || !shard_totals_device || !u_local_out || !mine_out) return DISTRL_ERR_NULL;
    if (!aligned_to(u_fix, 8) || !aligned_to(shard_totals_device, 8) || !aligned_to(u_local_out, 8) ||
        !aligned_to(owner_out, 4) || !aligned_to(status_out_device, 4))
        return DISTRL_ERR_ALIGN;
    int64_t grid = ceil_div(k, 256);
    if (grid > 1184) grid = 1184;
    route_draws_kernel<<<(unsigned)grid, 256, 0, static_cast<cudaStream_t>(stream)>>>(
        reinterpret_cast<const unsigned long long *>(u_fix), (long long)k,
        reinterpret_cast<const unsigned long long *>(shard_totals_device), n_shards, my_shard,
        reinterpret_cast<unsigned long long *>(u_local_out), mine_out, owner_out, status_out_device);
    DISTRL_CUDA_TRY(cudaGetLastError());
    return DISTRL_OK;
}

namespace distrl {
// What a shard contributes to a batch drawn over several shards: for the draws it owns, the global index
// and the un-normalised global weight (N q / T)^-beta = (N_shard q / T_shard)^-beta x ((N / N_shard)(T_shard / T))^-beta;
// -1 and 0 elsewhere, so that an element-wise maximum over the shards assembles the batch.
__global__ void finish_shard_draws_kernel(long long k, const unsigned char *__restrict__ mine,
                                          const long long *__restrict__ idx_local, const float *__restrict__ w_local,
                                          const unsigned long long *__restrict__ totals, int n_shards, int me,
                                          long long n_local, long long n_global, long long index_base, float beta,
                                          long long *__restrict__ idx_out, float *__restrict__ w_out) {
    double grand = 0.0;
    for (int g = 0; g < n_shards; ++g) grand += (double)totals[g];
    const double ratio = ((double)n_global / (double)n_local) * ((double)totals[me] / grand);
    const float factor = (float)pow(ratio, -(double)beta);
    const long long stride = (long long)gridDim.x * blockDim.x;
    for (long long j = (long long)blockIdx.x * blockDim.x + threadIdx.x; j < k; j += stride) {
        const bool own = mine[j] != 0 && idx_local[j] >= 0;
        idx_out[j] = own ? index_base + idx_local[j] : -1;
        if (w_out) w_out[j] = own ? w_local[j] * factor : 0.f;
    }
}

// w[j] /= max_j w[j] (one block; the batch maximum of Section 5.3's importance weights)
__global__ void __launch_bounds__(1024) normalise_weights_kernel(float *__restrict__ w, long long k) {
    __shared__ float s_max[32];
    float m = 0.f;
    for (long long j = threadIdx.x; j < k; j += blockDim.x) m = fmaxf(m, w[j]);
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, d));
    if ((threadIdx.x & 31) == 0) s_max[threadIdx.x >> 5] = m;
    __syncthreads();
    m = (threadIdx.x < 32) ? s_max[threadIdx.x] : 0.f;
    if (threadIdx.x < 32) {
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, d));
        if (threadIdx.x == 0) s_max[0] = m;
    }
    __syncthreads();
    m = s_max[0];
    if (!(m > 0.f)) return; // no weight at all: leave the zeros
    for (long long j = threadIdx.x; j < k; j += blockDim.x) w[j] = w[j] / m;
}
} // namespace distrl

extern "C" int distrl_finish_shard_draws(int64_t k, const uint8_t *mine, const int64_t *idx_local, const float *w_local,
                                         const uint64_t *shard_totals_device, int n_shards, int my_shard,
                                         int64_t n_local, int64_t n_global, int64_t index_base, float beta,
                                         int64_t *idx_global_out, float *w_global_out, void *stream) {
    if (k < 0 || k > DISTRL_MAX_N || n_local <= 0 || n_global < n_local || index_base < 0) return DISTRL_ERR_SIZE;
    if (n_shards < 1 || n_shards > kMaxShards || my_shard < 0 || my_shard >= n_shards || !(beta == beta))
        return DISTRL_ERR_PARAM;
    if (k == 0) return DISTRL_OK;
    if (!mine || !idx_local || !shard_totals_device || !idx_global_out || (w_global_out && !w_local)) return DISTRL_ERR_NULL;
    if (!aligned_to(idx_local, 8) || !aligned_to(idx_global_out, 8) || !aligned_to(shard_totals_device, 8) ||
        !aligned_to(w_local, 4) || !aligned_to(w_global_out, 4))
        return DISTRL_ERR_ALIGN;
    int64_t grid = ceil_div(k, 256);
    if (grid > 1184) grid = 1184;
    finish_shard_draws_kernel<<<(unsigned)grid, 256, 0, static_cast<cudaStream_t>(stream)>>>(
        (long long)k, mine, reinterpret_cast<const long long *>(idx_local), w_local,
        reinterpret_cast<const unsigned long long *>(shard_totals_device), n_shards, my_shard, (long long)n_local,
        (long long)n_global, (long long)index_base, beta, reinterpret_cast<long long *>(idx_global_out), w_global_out);
    DISTRL_CUDA_TRY(cudaGetLastError());
    return DISTRL_OK;
}

extern "C" int distrl_normalise_weights(float *is_weight, int64_t k, void *stream) {
    if (k < 0 || k > DISTRL_MAX_N) return DISTRL_ERR_SIZE;
    if (k == 0) return DISTRL_OK;
    if (!is_weight) return DISTRL_ERR_NULL;
    if (!aligned_to(is_weight, 4)) return DISTRL_ERR_ALIGN;
    normalise_weights_kernel<<<1, 1024, 0, static_cast<cudaStream_t>(stream)>>>(is_weight, (long long)k);
    DISTRL_CUDA_TRY(cudaGetLastError());
    return DISTRL_OK;
}

extern "C" int distrl_sampler_total(distrl_sampler *s, uint64_t *total_out_device, void *stream) {
    if (!s || !total_out_device) return DISTRL_ERR_NULL;
    if (!aligned_to(total_out_device, 8)) return DISTRL_ERR_ALIGN;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (s->tree.n == 0) {
        DISTRL_CUDA_TRY(cudaMemsetAsync(total_out_device, 0, sizeof(uint64_t), st));
        return DISTRL_OK;
    }
    total_kernel<<<1, 32, 0, st>>>(s->tree, reinterpret_cast<unsigned long long *>(total_out_device));
    DISTRL_CUDA_TRY(cudaGetLastError());
    return DISTRL_OK;
}

extern "C" int distrl_sampler_level(const distrl_sampler *s, int level, size_t *offset_bytes, int64_t *count) {
    if (!s) return DISTRL_ERR_NULL;
    if (level >= 1 && level <= s->tree.levels) {
        if (offset_bytes) *offset_bytes = s->offsets[level];
        if (count) *count = s->tree.count[level];
    }
    return s->tree.levels;
}

extern "C" int distrl_destroy_sampler(distrl_sampler *s) {
    delete s;
    return DISTRL_OK;
}

DISTRL_BOUNDS_UNIT(sampler, 3)
