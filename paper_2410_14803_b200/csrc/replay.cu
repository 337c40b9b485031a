// Circular replay buffer of whole trajectories (App. A "Circular Replay Buffer": capacity N, the write
// index advances as i <- (i + 1) mod N and new experiences overwrite the oldest; Section 5.3 prioritises
// and replays trajectories) -- sm_100a.
//
// The buffer is the caller's SoA arrays of N slots plus the masses prio_q.  Its structure lives in two
// bit masks in the workspace, one bit per slot:
//   start : a segment (a live trajectory or a dead stretch) starts at this slot;
//   alive : the slot belongs to a live trajectory.
// From them every ingest rebuilds the CSR offsets the other entry points take (stream compaction of the
// start bits, padded with N up to a fixed capacity so that the caller never has to read a count back),
// and one liveness flag per segment.
//
// An ingest is planned on the host from the lengths of the new trajectories, which the host knows:
// trajectories occupy consecutive slots (the Retrace recursion runs along them), so one that would
// straddle the end of the buffer starts at slot 0 and the slots left at the end are retired.  All new
// rows therefore land in at most two contiguous runs, and the device work is
//   cut    : the stored trajectory that the end of the write region cuts loses its remaining slots too
//            (found by scanning the start bits; masses zeroed with exact repair of the sums),
//   cover  : alive/start bits of the write region,   starts : one start bit per new trajectory,
//   rows   : the new rows into their slots,           masses : new masses with exact repair of the sums,
//   csr    : offsets and liveness flags from the bits.
#include "common.cuh"
#include "sampler.cuh"

#include <new>

namespace distrl {

constexpr int kRingMaxFields = DISTRL_REPLAY_MAX_FIELDS;
constexpr int kRingThreads = 256;
constexpr int kRingWordsPerThread = 4;
constexpr int kRingWordsPerBlock = kRingThreads * kRingWordsPerThread; // 32768 slots

struct RingHeader {
    int status;         // sticky device-side status word (same place as in every workspace)
    int pad_;
    long long segments; // number of segments after the last ingest
    long long kill[2];  // [begin, end) of the slots killed right of the write region
};
static_assert(sizeof(RingHeader) <= kHeaderBytes, "the header has 256 bytes");

struct RingWs {
    RingHeader *hdr;
    unsigned int *start, *alive; // [words]
    long long *block_count;      // [blocks + 1] start bits per block of words, then their exclusive sums
    int64_t words, blocks;
};

static size_t ring_layout(int64_t n, void *base, RingWs *ws) {
    const int64_t words = ceil_div(n > 0 ? n : 1, 32);
    const int64_t blocks = ceil_div(words, kRingWordsPerBlock);
    size_t o = kHeaderBytes;
    char *b = static_cast<char *>(base);
    auto take = [&](size_t bytes) { size_t at = o; o = round_up(o + bytes, 256); return at; };
    const size_t s = take(sizeof(unsigned int) * words);
    const size_t a = take(sizeof(unsigned int) * words);
    const size_t c = take(sizeof(long long) * (blocks + 1));
    if (ws) {
        ws->hdr = reinterpret_cast<RingHeader *>(b);
        ws->start = reinterpret_cast<unsigned int *>(b + s);
        ws->alive = reinterpret_cast<unsigned int *>(b + a);
        ws->block_count = reinterpret_cast<long long *>(b + c);
        ws->words = words;
        ws->blocks = blocks;
    }
    return o;
}

struct FieldPtrs {
    float *dst[kRingMaxFields];
    const float *src[kRingMaxFields];
    int count;
};

__device__ __forceinline__ bool bit_at(const unsigned int *mask, int64_t i) { return (mask[i >> 5] >> (i & 31)) & 1u; }

// bits [a, b) of `mask` set (value != 0) or cleared, word by word with one lane per word
__device__ __forceinline__ void warp_fill_bits(unsigned int *mask, int64_t words, int64_t a, int64_t b, int value, int lane) {
    if (b <= a) return;
    for (int64_t w = (a >> 5) + lane; w <= ((b - 1) >> 5); w += 32) {
        const int64_t lo = w << 5;
        unsigned int m = 0xffffffffu;
        if (a > lo) m &= 0xffffffffu << (int)(a - lo);
        if (b < lo + 32) m &= 0xffffffffu >> (int)(lo + 32 - b);
        if (!DISTRL_IN(w, words)) continue;
        if (value) atomicOr(&mask[w], m);
        else atomicAnd(&mask[w], ~m);
    }
}

// ---------------------------------------------------------------------------
// cut: a stored trajectory that owns slot `right`, the first slot after the write region, without
// starting there reaches out of the region: it loses rows, so its slots from `right` on are killed too
// (alive bits cleared here; the range is left in the header for the kernel that zeroes the masses).
// The other end needs no such care: the write index always sits on the first slot of a segment,
// because every ingest ends by starting one there.  Reads the bits as the previous ingest left them.
// One warp; right = -1: the region ends at the end of the buffer or covers all of it.
// ---------------------------------------------------------------------------
__global__ void __launch_bounds__(32) ring_cut_kernel(RingWs ws, int64_t n, int64_t right) {
    grid_dependency_wait();
    grid_launch_dependents();
    const int lane = threadIdx.x & 31;
    int64_t a = 0, b = 0; // killed range
    if (right > 0 && right < n && bit_at(ws.alive, right) && !bit_at(ws.start, right)) {
        // the nearest start bit above `right`, or the end of the buffer: 32 words at a time
        int64_t w0 = right >> 5;
        int64_t found = n;
        for (;;) {
            const int64_t w = w0 + lane;
            unsigned int v = (w < ws.words) ? ws.start[w] : 0u;
            if (w == (right >> 5)) v &= ((right & 31) == 31) ? 0u : (0xffffffffu << (int)((right & 31) + 1)); // bits above
            const unsigned int hit = __ballot_sync(0xffffffffu, v != 0u);
            if (hit) {
                const int first = __ffs(hit) - 1; // the lowest word that has a bit
                const unsigned int vv = __shfl_sync(0xffffffffu, v, first);
                found = ((w0 + first) << 5) + (__ffs(vv) - 1);
                break;
            }
            w0 += 32;
            if (w0 >= ws.words) break;
        }
        a = right;
        b = found < n ? found : n;
    }
    warp_fill_bits(ws.alive, ws.words, a, b, 0, lane);
    if (lane == 0) {
        ws.hdr->kill[0] = a;
        ws.hdr->kill[1] = b;
    }
}

// cover: up to three runs of slots get their alive bits set or cleared and lose their start bits.
struct CoverRuns {
    int64_t a[3], b[3];
    int alive[3];
};
__global__ void __launch_bounds__(kRingThreads) ring_cover_kernel(RingWs ws, CoverRuns r) {
    grid_dependency_wait();
    grid_launch_dependents();
    const int lane = threadIdx.x & 31;
    const int64_t warp = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int64_t warps = ((int64_t)gridDim.x * blockDim.x) >> 5;
    for (int i = 0; i < 3; ++i) {
        if (r.b[i] <= r.a[i]) continue;
        // a warp takes 1024 slots (32 words) at a time
        for (int64_t c = (r.a[i] >> 10) + warp; c <= ((r.b[i] - 1) >> 10); c += warps) {
            const int64_t lo = c << 10, hi = lo + 1024;
            const int64_t a = r.a[i] > lo ? r.a[i] : lo, b = r.b[i] < hi ? r.b[i] : hi;
            warp_fill_bits(ws.start, ws.words, a, b, 0, lane);
            warp_fill_bits(ws.alive, ws.words, a, b, r.alive[i], lane);
        }
    }
}

// starts: one start bit per new non-empty trajectory, plus up to two more (the retired stretch, the
// slot after the write region).  Rows before `split_row` land at head + row, the others at row - split_row.
__global__ void __launch_bounds__(kRingThreads) ring_starts_kernel(RingWs ws, int64_t n, int64_t k,
                                                                   const int64_t *__restrict__ new_off, int64_t total,
                                                                   int64_t head, int64_t split_row, int64_t extra0,
                                                                   int64_t extra1) {
    grid_dependency_wait();
    grid_launch_dependents();
    const int64_t j = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (j == 0) {
        if (extra0 >= 0 && extra0 < n) atomicOr(&ws.start[extra0 >> 5], 1u << (extra0 & 31));
        if (extra1 >= 0 && extra1 < n) atomicOr(&ws.start[extra1 >> 5], 1u << (extra1 & 31));
        if (new_off[0] != 0 || new_off[k] != total) set_status(&ws.hdr->status, DISTRL_ERR_OFFSETS);
    }
    if (j >= k) return;
    const int64_t row = new_off[j], next = new_off[j + 1];
    if (row < 0 || next < row || next > total) { // not what the host planned with
        set_status(&ws.hdr->status, DISTRL_ERR_OFFSETS);
        return;
    }
    if (next == row) return; // an empty trajectory stores nothing
    const int64_t slot = row < split_row ? head + row : row - split_row;
    if (slot >= 0 && slot < n && DISTRL_IN(slot >> 5, ws.words)) atomicOr(&ws.start[slot >> 5], 1u << (slot & 31));
}

// rows: new row t of every field goes to slot head + t (t < split_row) or t - split_row.
__global__ void __launch_bounds__(kRingThreads) ring_rows_kernel(FieldPtrs f, int64_t n, int64_t total, int64_t head,
                                                                 int64_t split_row) {
    grid_dependency_wait();
    grid_launch_dependents();
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; t < total; t += stride) {
        const int64_t slot = t < split_row ? head + t : t - split_row;
        if (!DISTRL_IN(slot, n)) continue;
        for (int i = 0; i < f.count; ++i) f.dst[i][slot] = __ldcs(f.src[i] + t);
    }
}

// masses without a sampler: plain stores (src null: zeros), and zeros for the killed range
__global__ void __launch_bounds__(kRingThreads) ring_mass_run_kernel(uint32_t *__restrict__ q, int64_t n, int64_t a,
                                                                     int64_t b, const uint32_t *__restrict__ src) {
    grid_dependency_wait();
    grid_launch_dependents();
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (int64_t i = a + (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < b; i += stride)
        if (DISTRL_IN(i, n)) q[i] = src ? src[i - a] : 0u;
}
__global__ void __launch_bounds__(kRingThreads) ring_mass_kill_kernel(uint32_t *__restrict__ q, int64_t n,
                                                                      const long long *__restrict__ kill) {
    grid_dependency_wait();
    grid_launch_dependents();
    int64_t a = kill[0], b = kill[1];
    if (a < 0) a = 0;
    if (b > n) b = n;
    for (int64_t i = a + threadIdx.x; i < b; i += blockDim.x) q[i] = 0u;
}

// ---------------------------------------------------------------------------
// csr: positions of the start bits, in order, are the segment offsets.
//   count : start bits per block of kRingWordsPerBlock words;
//   scan  : one block turns the counts into exclusive sums and records the total M;
//   emit  : every block ranks its own bits and writes offsets[rank] = slot and the segment's liveness;
//           entries M .. m_capacity of the offsets are N (empty segments), liveness 0.
// ---------------------------------------------------------------------------
__global__ void __launch_bounds__(kRingThreads) ring_count_kernel(RingWs ws) {
    grid_dependency_wait();
    grid_launch_dependents();
    __shared__ int s_sum[kRingThreads / 32];
    const int64_t w0 = (int64_t)blockIdx.x * kRingWordsPerBlock + threadIdx.x * kRingWordsPerThread;
    int c = 0;
#pragma unroll
    for (int e = 0; e < kRingWordsPerThread; ++e)
        if (w0 + e < ws.words) c += __popc(ws.start[w0 + e]);
    c = __reduce_add_sync(0xffffffffu, c);
    if ((threadIdx.x & 31) == 0) s_sum[threadIdx.x >> 5] = c;
    __syncthreads();
    if (threadIdx.x == 0) {
        int t = 0;
        for (int i = 0; i < kRingThreads / 32; ++i) t += s_sum[i];
        ws.block_count[blockIdx.x] = t;
    }
}

__global__ void __launch_bounds__(1024) ring_scan_kernel(RingWs ws, int64_t m_capacity, int64_t *m_out) {
    grid_dependency_wait();
    grid_launch_dependents();
    __shared__ long long s_warp[32];
    __shared__ long long s_base;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (threadIdx.x == 0) s_base = 0;
    __syncthreads();
    for (int64_t b0 = 0; b0 < ws.blocks; b0 += 1024) {
        const int64_t b = b0 + threadIdx.x;
        const long long v = (b < ws.blocks) ? ws.block_count[b] : 0;
        long long incl = v;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const long long o = __shfl_up_sync(0xffffffffu, incl, d);
            if (lane >= d) incl += o;
        }
        if (lane == 31) s_warp[warp] = incl;
        __syncthreads();
        long long before = s_base;
        for (int w = 0; w < warp; ++w) before += s_warp[w];
        if (b < ws.blocks) ws.block_count[b] = before + incl - v;
        __syncthreads();
        if (threadIdx.x == 1023) s_base = before + incl;
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        const long long m = s_base;
        ws.block_count[ws.blocks] = m;
        ws.hdr->segments = m;
        if (m_out) *m_out = m;
        if (m > m_capacity) set_status(&ws.hdr->status, DISTRL_ERR_SIZE); // more segments than the offsets array holds
    }
}

__global__ void __launch_bounds__(kRingThreads) ring_emit_kernel(RingWs ws, int64_t n, int64_t *__restrict__ offsets,
                                                                 float *__restrict__ seg_alive, int64_t m_capacity) {
    grid_dependency_wait();
    grid_launch_dependents();
    __shared__ int s_warp[kRingThreads / 32];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t w0 = (int64_t)blockIdx.x * kRingWordsPerBlock + threadIdx.x * kRingWordsPerThread;
    unsigned int sv[kRingWordsPerThread], av[kRingWordsPerThread];
    int c = 0;
#pragma unroll
    for (int e = 0; e < kRingWordsPerThread; ++e) {
        sv[e] = (w0 + e < ws.words) ? ws.start[w0 + e] : 0u;
        av[e] = (w0 + e < ws.words) ? ws.alive[w0 + e] : 0u;
        c += __popc(sv[e]);
    }
    int incl = c;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const int o = __shfl_up_sync(0xffffffffu, incl, d);
        if (lane >= d) incl += o;
    }
    if (lane == 31) s_warp[warp] = incl;
    __syncthreads();
    long long rank = ws.block_count[blockIdx.x] + incl - c;
    for (int w = 0; w < warp; ++w) rank += s_warp[w];
#pragma unroll
    for (int e = 0; e < kRingWordsPerThread; ++e) {
        unsigned int v = sv[e];
        while (v) {
            const int bit = __ffs(v) - 1;
            v &= v - 1u;
            if (rank < m_capacity) {
                offsets[rank] = ((w0 + e) << 5) + bit;
                seg_alive[rank] = ((av[e] >> bit) & 1u) ? 1.f : 0.f;
            }
            ++rank;
        }
    }
    // the tail: empty segments at the end of the buffer
    const long long m = ws.block_count[ws.blocks];
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (int64_t i = (m < m_capacity ? m : m_capacity) + (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i <= m_capacity;
         i += stride) {
        offsets[i] = n;
        if (i < m_capacity) seg_alive[i] = 0.f;
    }
}

__global__ void ring_first_bit_kernel(RingWs ws) {
    grid_dependency_wait();
    grid_launch_dependents();
    if (threadIdx.x == 0 && blockIdx.x == 0) ws.start[0] = 1u; // slot 0 always starts a segment
}

} // namespace distrl

using namespace distrl;

struct distrl_replay {
    int64_t n, m_capacity, head;
    int n_fields;
    float *field[kRingMaxFields];
    uint32_t *q;
    int64_t *offsets;
    float *seg_alive;
    RingWs ws;
};

static int ring_rebuild_csr(distrl_replay *rb, int64_t *m_out_device, cudaStream_t st) {
    DISTRL_CUDA_TRY(launch_pdl(ring_count_kernel, dim3((unsigned)rb->ws.blocks), dim3(kRingThreads), 0, st, rb->ws));
    DISTRL_CUDA_TRY(launch_pdl(ring_scan_kernel, dim3(1), dim3(1024), 0, st, rb->ws, rb->m_capacity, m_out_device));
    DISTRL_CUDA_TRY(launch_pdl(ring_emit_kernel, dim3((unsigned)rb->ws.blocks), dim3(kRingThreads), 0, st, rb->ws, rb->n,
                               rb->offsets, rb->seg_alive, rb->m_capacity));
    return DISTRL_OK;
}

extern "C" size_t distrl_replay_workspace_bytes(int64_t capacity) {
    if (capacity < 0) capacity = 0;
    return ring_layout(capacity, nullptr, nullptr);
}

extern "C" int distrl_replay_create(int64_t capacity, int n_fields, float *const *fields, uint32_t *prio_q,
                                    int64_t *traj_offsets, float *traj_alive, int64_t m_capacity, void *workspace,
                                    size_t workspace_bytes, void *stream, distrl_replay **out) {
    if (!out) return DISTRL_ERR_NULL;
    *out = nullptr;
    if (capacity <= 0 || capacity > DISTRL_MAX_N || m_capacity < 1 || m_capacity > DISTRL_MAX_N) return DISTRL_ERR_SIZE;
    if (n_fields < 0 || n_fields > kRingMaxFields) return DISTRL_ERR_SIZE;
    if ((n_fields > 0 && !fields) || !prio_q || !traj_offsets || !traj_alive || !workspace) return DISTRL_ERR_NULL;
    for (int i = 0; i < n_fields; ++i) {
        if (!fields[i]) return DISTRL_ERR_NULL;
        if (!aligned_to(fields[i], 4)) return DISTRL_ERR_ALIGN;
    }
    if (!aligned_to(prio_q, 4) || !aligned_to(traj_offsets, 8) || !aligned_to(traj_alive, 4)) return DISTRL_ERR_ALIGN;
    if (!aligned_to(workspace, 256) || workspace_bytes < ring_layout(capacity, nullptr, nullptr))
        return DISTRL_ERR_WORKSPACE;
    distrl_replay *rb = new (std::nothrow) distrl_replay();
    if (!rb) return DISTRL_ERR_CUDA;
    rb->n = capacity;
    rb->m_capacity = m_capacity;
    rb->head = 0;
    rb->n_fields = n_fields;
    for (int i = 0; i < n_fields; ++i) rb->field[i] = fields[i];
    rb->q = prio_q;
    rb->offsets = traj_offsets;
    rb->seg_alive = traj_alive;
    const size_t bytes = ring_layout(capacity, workspace, &rb->ws);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    auto fail = [&](int rc) { delete rb; return rc; };
    // an empty buffer: one dead segment [0, N), no mass anywhere, rows zero (dead rows still go through
    // the scan kernels as numbers, so they must be finite)
    if (cudaMemsetAsync(workspace, 0, bytes, st) != cudaSuccess) return fail(record_cuda_error(cudaGetLastError(), "cudaMemsetAsync"));
    if (cudaMemsetAsync(prio_q, 0, sizeof(uint32_t) * (size_t)capacity, st) != cudaSuccess)
        return fail(record_cuda_error(cudaGetLastError(), "cudaMemsetAsync"));
    for (int i = 0; i < n_fields; ++i)
        if (cudaMemsetAsync(fields[i], 0, sizeof(float) * (size_t)capacity, st) != cudaSuccess)
            return fail(record_cuda_error(cudaGetLastError(), "cudaMemsetAsync"));
    ring_first_bit_kernel<<<1, 32, 0, st>>>(rb->ws);
    if (cudaGetLastError() != cudaSuccess) return fail(record_cuda_error(cudaGetLastError(), "ring_first_bit_kernel"));
    const int rc = ring_rebuild_csr(rb, nullptr, st);
    if (rc) return fail(rc);
    *out = rb;
    return DISTRL_OK;
}

extern "C" int distrl_replay_ingest(distrl_replay *rb, distrl_sampler *sampler, int64_t k,
                                    const int64_t *new_offsets_host, const int64_t *new_offsets,
                                    const float *const *new_fields, const uint32_t *new_q,
                                    int64_t *n_segments_out_device, void *stream) {
    if (!rb) return DISTRL_ERR_NULL;
    if (k < 0 || k > DISTRL_MAX_N) return DISTRL_ERR_SIZE;
    if (k == 0) return DISTRL_OK;
    if (!new_offsets_host) return DISTRL_ERR_NULL;
    const int64_t n = rb->n;
    // ---- plan: where the rows go, which slots are retired, how far the write index travels ----
    if (new_offsets_host[0] != 0) return DISTRL_ERR_OFFSETS;
    int64_t h = rb->head, advance = 0, split = -1; // split: first row that lands at slot 0 after the wrap
    for (int64_t j = 0; j < k; ++j) {
        const int64_t T = new_offsets_host[j + 1] - new_offsets_host[j];
        if (T < 0) return DISTRL_ERR_OFFSETS;
        if (T == 0) continue;
        if (h + T > n) {
            if (split >= 0) return DISTRL_ERR_SIZE; // a second lap
            advance += n - h;
            h = 0;
            split = new_offsets_host[j];
        }
        h += T;
        advance += T;
        if (advance > n) return DISTRL_ERR_SIZE; // the call would overwrite its own trajectories
    }
    const int64_t total = new_offsets_host[k];
    if (total == 0) return DISTRL_OK; // nothing but empty trajectories
    if (!new_offsets || !new_q || (rb->n_fields > 0 && !new_fields)) return DISTRL_ERR_NULL;
    if (!aligned_to(new_offsets, 8) || !aligned_to(new_q, 4) || !aligned_to(n_segments_out_device, 8)) return DISTRL_ERR_ALIGN;
    for (int i = 0; i < rb->n_fields; ++i) {
        if (!new_fields[i]) return DISTRL_ERR_NULL;
        if (!aligned_to(new_fields[i], 4)) return DISTRL_ERR_ALIGN;
    }
    if (sampler && (sampler_size(sampler) != rb->n || sampler_masses(sampler) != rb->q)) return DISTRL_ERR_PARAM;
    const bool wrapped = split >= 0;
    const int64_t head0 = rb->head;
    const int64_t split_row = wrapped ? split : total;
    const int64_t end_a = head0 + split_row;               // one past the first run of rows
    const int64_t end_b = wrapped ? total - split_row : 0; // one past the second run (which starts at slot 0)
    const int64_t last = wrapped ? end_b : end_a;          // the slot after the write region (may be N)
    const bool whole = (advance == n);                      // every slot of the buffer is written or retired
    const int64_t cut_right = (!whole && last < n) ? last : -1;
    cudaStream_t st = static_cast<cudaStream_t>(stream);

    DISTRL_CUDA_TRY(launch_pdl(ring_cut_kernel, dim3(1), dim3(32), 0, st, rb->ws, n, cut_right));
    CoverRuns runs = {};
    runs.a[0] = head0; runs.b[0] = end_a; runs.alive[0] = 1;
    runs.a[1] = wrapped ? end_a : 0; runs.b[1] = wrapped ? n : 0; runs.alive[1] = 0; // retired at the end
    runs.a[2] = 0; runs.b[2] = end_b; runs.alive[2] = 1;
    {
        int64_t chunks = 0;
        for (int i = 0; i < 3; ++i)
            if (runs.b[i] > runs.a[i]) chunks += ((runs.b[i] - 1) >> 10) - (runs.a[i] >> 10) + 1;
        int64_t grid = ceil_div(chunks * 32, kRingThreads);
        if (grid > 4096) grid = 4096;
        if (grid < 1) grid = 1;
        DISTRL_CUDA_TRY(launch_pdl(ring_cover_kernel, dim3((unsigned)grid), dim3(kRingThreads), 0, st, rb->ws, runs));
    }
    {
        const int64_t extra0 = (wrapped && end_a < n) ? end_a : -1; // the retired stretch is a segment of its own
        const int64_t extra1 = (!whole && last < n) ? last : -1;    // so is what follows the write region
        DISTRL_CUDA_TRY(launch_pdl(ring_starts_kernel, dim3((unsigned)ceil_div(k, kRingThreads)), dim3(kRingThreads), 0, st,
                                   rb->ws, n, k, new_offsets, total, head0, split_row, extra0, extra1));
    }
    if (rb->n_fields > 0) {
        FieldPtrs f = {};
        f.count = rb->n_fields;
        for (int i = 0; i < rb->n_fields; ++i) { f.dst[i] = rb->field[i]; f.src[i] = new_fields[i]; }
        int64_t grid = ceil_div(total, kRingThreads);
        if (grid > 8 * 148) grid = 8 * 148;
        DISTRL_CUDA_TRY(launch_pdl(ring_rows_kernel, dim3((unsigned)grid), dim3(kRingThreads), 0, st, f, n, total, head0,
                                   split_row));
    }
    // masses: the killed slots, the two runs of new rows, the retired stretch; one launch after the
    // other, so a leaf group that two of them touch is rewritten by one warp at a time
    if (sampler) {
        int rc = sampler_zero_range(sampler, reinterpret_cast<const int64_t *>(rb->ws.hdr->kill), st);
        if (!rc) rc = sampler_overwrite_run(sampler, head0, end_a, new_q, st);
        if (!rc && wrapped) rc = sampler_overwrite_run(sampler, end_a, n, nullptr, st);
        if (!rc && wrapped) rc = sampler_overwrite_run(sampler, 0, end_b, new_q + split_row, st);
        if (rc) return rc;
    } else {
        auto run = [&](int64_t a, int64_t b, const uint32_t *src) -> cudaError_t {
            if (b <= a) return cudaSuccess;
            int64_t grid = ceil_div(b - a, kRingThreads);
            if (grid > 8 * 148) grid = 8 * 148;
            return launch_pdl(ring_mass_run_kernel, dim3((unsigned)grid), dim3(kRingThreads), 0, st, rb->q, n, a, b, src);
        };
        DISTRL_CUDA_TRY(launch_pdl(ring_mass_kill_kernel, dim3(1), dim3(kRingThreads), 0, st, rb->q, n,
                                   (const long long *)rb->ws.hdr->kill));
        DISTRL_CUDA_TRY(run(head0, end_a, new_q));
        if (wrapped) {
            DISTRL_CUDA_TRY(run(end_a, n, nullptr));
            DISTRL_CUDA_TRY(run(0, end_b, new_q + split_row));
        }
    }
    const int rc = ring_rebuild_csr(rb, n_segments_out_device, st);
    if (rc) return rc;
    rb->head = last % n;
    return DISTRL_OK;
}

extern "C" int64_t distrl_replay_head(const distrl_replay *rb) { return rb ? rb->head : -1; }

extern "C" int distrl_replay_destroy(distrl_replay *rb) {
    delete rb;
    return DISTRL_OK;
}

DISTRL_BOUNDS_UNIT(replay, 5)
