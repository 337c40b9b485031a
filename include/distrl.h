/*
 * distrl.h -- C ABI of the B200 (sm_100a) learner hot path of DistRL's A-RIDE
 * algorithm (arXiv 2410.14803): Retrace(lambda) value targets and advantages
 * (Section 5.2), the DPER replay priority (Section 5.3) and prioritized
 * proportional sampling with importance-sampling weights and incremental
 * priority refresh (Section 5.3 and App. A, "Priority-Based Sampling in DPER").
 *
 * General rules, valid for every entry point unless it says otherwise:
 *   - Every data pointer is a DEVICE pointer owned by the caller.  The library
 *     neither allocates nor frees device memory, and keeps no pointer beyond
 *     what a sampler handle documents.  Parameter structs (distrl_batch,
 *     distrl_prio_cfg) and handles live in HOST memory.
 *   - Arrays are dense and contiguous.  fp32 / uint32 arrays need 4-byte
 *     alignment, 64-bit arrays 8-byte alignment; 16-byte alignment of every
 *     array enables the 128-bit load/store path (what torch allocations give).
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream).
 *     Calls enqueue work and return without synchronising.
 *   - Return value: DISTRL_OK (0) or a negative distrl_status.  Nothing throws,
 *     aborts or traps.  Problems that only the device can see (bad offsets, an
 *     index out of range, a bounded wait that ran out) are recorded in the
 *     status word at the start of the workspace: read it with
 *     distrl_get_status().
 *   - Sizes of zero (n = 0, k = 0) are valid and do nothing.
 *   - There is no CPU fallback: without a CUDA device every compute entry
 *     point returns DISTRL_ERR_CUDA.
 */
#ifndef DISTRL_H
#define DISTRL_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    DISTRL_OK = 0,
    DISTRL_ERR_NULL = -1,      /* a required pointer is NULL                                */
    DISTRL_ERR_SIZE = -2,      /* negative size, n > DISTRL_MAX_N, struct_size mismatch     */
    DISTRL_ERR_ALIGN = -3,     /* a pointer breaks its element alignment                    */
    DISTRL_ERR_WORKSPACE = -4, /* workspace too small or not 256-byte aligned               */
    DISTRL_ERR_CUDA = -5,      /* a CUDA runtime call failed (see distrl_last_cuda_error)   */
    DISTRL_ERR_TIMEOUT = -6,   /* device status: a bounded inter-block wait ran out         */
    DISTRL_ERR_PARAM = -7,     /* gamma/lambda outside [0,1], alpha < 0, scale <= 0, NaN    */
    DISTRL_ERR_OFFSETS = -8,   /* device status: offsets decreasing, [0] != 0 or [M] != N   */
    DISTRL_ERR_INDEX = -9      /* device status: a sampled/updated index outside [0, n)     */
} distrl_status;

#define DISTRL_MAX_N ((int64_t)1 << 33) /* largest transition / token count accepted */

/* ---------------------------------------------------------------------------
 * The trajectory buffer: N transitions of M trajectories stored flat,
 * structure-of-arrays.  Trajectory j (Section 3: tau = {(s_t,a_t,r_t,s_t+1)})
 * owns the flat indices [traj_offsets[j], traj_offsets[j+1]); empty
 * trajectories are allowed.  Either the per-step action log-probs are given
 * (logp_*), or, token-level, step t owns the tokens
 * [step_token_offsets[t], step_token_offsets[t+1]) of two bf16 arrays whose
 * per-step sums are the action log-probs (the quantity the ratio
 * rho_t = pi(a_t|s_t)/mu(a_t|s_t) of Section 5.1 needs).
 * ------------------------------------------------------------------------- */
typedef struct {
    uint32_t struct_size;                    /* sizeof(distrl_batch)                       */
    uint32_t reserved;                       /* 0                                          */
    int64_t n_transitions;                   /* N                                          */
    int64_t n_trajectories;                  /* M                                          */
    const int64_t *traj_offsets;             /* [M+1] non-decreasing, [0] = 0, [M] = N     */
    const float *rewards;                    /* [N] r_t                                    */
    const float *values;                     /* [N] V(s_t)                                 */
    const float *bootstrap_values;           /* [M] V(state after the last step); NULL = 0 */
    const float *logp_target;                /* [N] log pi(a_t|s_t); NULL if token-level   */
    const float *logp_behaviour;             /* [N] log mu(a_t|s_t); NULL if token-level   */
    const int64_t *step_token_offsets;       /* [N+1] or NULL; [0] = 0, non-decreasing     */
    const uint16_t *tok_logp_target_bf16;    /* [n_tok] bf16 bit patterns                  */
    const uint16_t *tok_logp_behaviour_bf16; /* [n_tok] bf16 bit patterns                  */
} distrl_batch;

/* Bytes of workspace distrl_retrace_targets needs for N transitions (any M). */
size_t distrl_retrace_workspace_bytes(int64_t n_transitions);

/* Zero-fill a workspace (retrace or sampler).  Call once after allocating it
 * and before its first use: the status word at its start is sticky until
 * distrl_get_status() reads it.  Everything else in a workspace is scratch
 * that each call rewrites. */
int distrl_workspace_init(void *workspace, size_t workspace_bytes, void *stream);

/*
 * Retrace(lambda) targets, Section 5.2, with the TD error of App. A:
 *   rho_t = exp(logpi_t - logmu_t),  c_t = lambda min(1, rho_t)
 *   delta_t = r_t + gamma V(s_{t+1}) - V(s_t)
 *   Delta_t = sum_{k>=t} gamma^(k-t) (prod_{i=t+1..k} c_i) delta_k   (per trajectory)
 *   v_target_t = V(s_t) + Delta_t;  advantage_t = Delta_t;  td_delta_t = delta_t
 * V(s_{t+1}) of a trajectory's last step is bootstrap_values[j], or 0.  (The
 * bootstrap values are read in place while the outputs are written: like every
 * input the array must not alias an output.)
 * Computed in fp32 as a segmented reverse scan; results agree with fp64
 * evaluation of the definition to 1e-4 (1 + |ref|).
 *   v_target, advantage : [N] outputs, required.
 *   td_delta            : [N] output or NULL.
 *   logp_target_out, logp_behaviour_out : [N] outputs or NULL; the per-step
 *       log-probs used (the token sums in token-level mode, a copy otherwise).
 *   workspace : >= distrl_retrace_workspace_bytes(N) bytes, 256-byte aligned,
 *       initialised once by distrl_workspace_init; contents are scratch, it
 *       may be reused by the next call on the same stream, not concurrently.
 * Outputs must not alias inputs.  Offsets are validated on the device
 * (DISTRL_ERR_OFFSETS in the status word; outputs are then unspecified but
 * every access stays in bounds).  Non-finite inputs give unspecified values
 * inside their own trajectory only.
 */
int distrl_retrace_targets(const distrl_batch *batch, float gamma, float lambda,
                           float *v_target, float *advantage, float *td_delta,
                           float *logp_target_out, float *logp_behaviour_out,
                           void *workspace, size_t workspace_bytes, void *stream);

/*
 * distrl_retrace_targets without a workspace argument.  (The paper has no
 * counterpart: this is a convenience of this library.)
 *
 * Meant for callers that cannot allocate device memory when they need the
 * targets -- for instance a learner whose framework has already reserved the
 * whole GPU for its own pool, so that a further cudaMalloc fails or shrinks
 * that pool, or a step loop that must stay clear of cudaMalloc because it
 * stalls the whole device.  The scan's tile bookkeeping lives in a fixed
 * array inside the library image (about 0.75 MB, held by every GPU that loads
 * the library until the process exits), which limits the size:
 *   n_transitions <= DISTRL_STATIC_MAX_N, else DISTRL_ERR_SIZE.
 * Arguments and results are those of distrl_retrace_targets, plus
 *   status_out_device : device int or NULL; receives the device status word of
 *       this call (DISTRL_OK, DISTRL_ERR_OFFSETS, DISTRL_ERR_TIMEOUT).
 * The call allocates nothing (no cudaMalloc / cudaFree, no library allocator).
 * One thing happens once per device all the same: the first call looks up the
 * array's device address, and, if nothing of this library has run on the device
 * yet, the CUDA runtime loads the library's code and the array at that moment
 * (device memory the runtime takes, about 1 MB).  So make one warm-up call per
 * device early -- before a framework reserves what is left of the GPU, and
 * outside any stream capture -- and later calls touch no allocator at all.
 * Arguments are checked before anything is enqueued: a refused call leaves the
 * array as it was.  All calls on a device share the one array: issue them on one
 * stream, or otherwise make sure two of them never run on the GPU at the same
 * time -- overlapping calls race on it.  (Calls of distrl_retrace_targets with
 * their own workspaces are not affected and may run beside it.)  First calls
 * from several host threads at once are safe.
 */
#define DISTRL_STATIC_MAX_N ((int64_t)1 << 22)
int distrl_retrace_targets_static(const distrl_batch *batch, float gamma, float lambda,
                                  float *v_target, float *advantage, float *td_delta,
                                  float *logp_target_out, float *logp_behaviour_out,
                                  int *status_out_device, void *stream);

/*
 * Monte-Carlo return of Section 5.1, G_t = sum_{k>=t} gamma^(k-t) r_k per
 * trajectory, and the label I[G_t > 0] the state-value classifier is trained
 * on.  Same scan as above with coefficient gamma and increment r_t.
 *   mc_return : [N] output or NULL;  label : [N] bytes (0/1) output or NULL.
 * Only traj_offsets, rewards and the sizes of `batch` are read.
 */
int distrl_mc_returns(const distrl_batch *batch, float gamma, float *mc_return,
                      uint8_t *label, void *workspace, size_t workspace_bytes,
                      void *stream);

/* ---------------------------------------------------------------------------
 * DPER priority, Section 5.3, evaluated per transition:
 *   p_t = w_td |delta_t| + w_rho min(rho_t, rho_clip) + w_ent H_t
 *   H_t = entropy[t], or -logpi_t when entropy is NULL (the paper's H_t)
 *   mass_t = p_t^alpha            (App. A: P(i) = p_i^alpha / sum_j p_j^alpha)
 *   q_t = Q(mass_t): x = (double)mass_t * scale; q = 1 if not (x > 0);
 *         q = 2^32-1 if x >= 2^32-1; else max(1, round-half-even(x)).
 * The fixed-point q is what the sampler sums; the floor of 1 keeps every
 * transition reachable.
 * ------------------------------------------------------------------------- */
typedef struct {
    float w_td, w_rho, w_ent; /* w1, w2, w3 of Section 5.3                    */
    float rho_clip;           /* upper clip of the ratio term                  */
    float alpha;              /* prioritisation exponent (0.5 in the paper)    */
    float scale;              /* fixed-point scale, e.g. 2^20                  */
} distrl_prio_cfg;

/*  td_delta, logp_target, logp_behaviour : [n] inputs; entropy : [n] or NULL.
 *  prio_mass : [n] fp32 output or NULL;  prio_q : [n] uint32 output, required.
 *  prio_q[t] equals Q(prio_mass[t]) exactly. */
int distrl_compute_priorities(int64_t n, const float *td_delta, const float *logp_target,
                              const float *logp_behaviour, const float *entropy,
                              const distrl_prio_cfg *cfg, float *prio_mass,
                              uint32_t *prio_q, void *stream);

/*
 * Trajectory-level priority exactly as Section 5.3 writes it: the same formula
 * applied to the trajectory means of |delta|, min(rho, rho_clip) and H.  (The
 * formula is linear in the means, so the kernel averages the per-step
 * combination w_td|delta_t| + w_rho min(rho_t, rho_clip) + w_ent H_t: the same
 * number up to fp32 rounding.)
 *   prio_mass : [M] or NULL;  prio_q : [M] required.  Empty trajectory: q = 1.
 *   With n == 0 (only empty trajectories) the per-step arrays may be NULL.
 */
int distrl_compute_priorities_traj(int64_t n, int64_t m, const int64_t *traj_offsets,
                                   const float *td_delta, const float *logp_target,
                                   const float *logp_behaviour, const float *entropy,
                                   const distrl_prio_cfg *cfg, float *prio_mass,
                                   uint32_t *prio_q, void *stream);

/* ---------------------------------------------------------------------------
 * Prioritized sampling.  The sampler is a radix tree of exact uint64 partial
 * sums over prio_q (leaf groups of 128 masses, fan-out 32 above) kept in the
 * caller's workspace.  Integer sums are associative, so a draw returns exactly
 * the index a linear scan of cumulative masses returns.
 * ------------------------------------------------------------------------- */
typedef struct distrl_sampler distrl_sampler; /* small host-side handle */

size_t distrl_sampler_workspace_bytes(int64_t n);

/*  prio_q : [n] masses; the sampler keeps this pointer, reads it when
 *      sampling and overwrites entries in distrl_update_priorities.
 *  workspace : >= distrl_sampler_workspace_bytes(n), 256-byte aligned,
 *      initialised once by distrl_workspace_init; owned by the caller, must
 *      outlive the handle.  *out receives a host handle (free it with
 *      distrl_destroy_sampler; that frees no device memory). */
int distrl_build_sampler(uint32_t *prio_q, int64_t n, void *workspace,
                         size_t workspace_bytes, void *stream, distrl_sampler **out);

/*
 * k independent draws with replacement, P(i) = q_i / total (App. A).
 *   u_fix : [k] 0.64 fixed-point uniforms (u / 2^64 in [0,1)), device.
 *   Draw j: y = floor(u_j * total / 2^64); idx_j = min{ i : q_0+..+q_i > y }.
 *   idx_out : [k] int64, required.
 *   is_weight_out : [k] fp32 or NULL: w_j = (n q_idx / total)^(-beta)
 *       (importance-sampling weight of prioritized replay, the definition the
 *       paper's replay cites); divided by the batch maximum if normalise != 0.
 * A normalising call whose grid fits the GPU at once (a few thousand draws)
 * lets its thread blocks wait for one another on the device for the batch
 * maximum; it is launched cooperatively, so the blocks are on the GPU together
 * whatever else runs there (if that launch is refused the call takes the path
 * of larger batches, where the last block does the rescaling).  The wait is
 * bounded all the same and reports DISTRL_ERR_TIMEOUT in the status word.
 * Calls on one sampler must not overlap on the GPU (they share words of its
 * workspace); calls on different samplers may.
 */
int distrl_sample(distrl_sampler *s, const uint64_t *u_fix, int64_t k, float beta,
                  int normalise, int64_t *idx_out, float *is_weight_out, void *stream);

/*
 * Stratified draws (the variant of the prioritized replay the paper's DPER cites:
 * the range of cumulative mass is cut into k equal strata and draw j is taken
 * from stratum j).  Turns k uniforms into stratified ones,
 *   u_out[j] = floor((j 2^64 + u_fix[j]) / k)     (0.64 fixed point; in place is fine),
 * which are then given to distrl_sample as they are: sampling itself is unchanged.
 */
int distrl_stratify_uniforms(const uint64_t *u_fix, int64_t k, uint64_t *u_out, void *stream);

/*
 * One prioritized replay over several shards (one per GPU): the proportional
 * draw of App. A ("Priority-Based Sampling": P(i) = p_i^alpha / sum_j p_j^alpha)
 * taken over the concatenation of the shards' masses.  Draw j has the global
 * threshold y = floor(u_fix[j] T / 2^64), T the sum of shard_totals; it belongs to
 * the shard whose range of cumulative mass holds y, and that shard obtains it
 * from its own sampler with the local uniform
 *   u_local = ceil((y - total of the shards before) 2^64 / T_shard),
 * for which floor(u_local T_shard / 2^64) is that local threshold exactly.
 *   shard_totals_device : [n_shards] device array, total mass of every shard in
 *       order (distrl_sampler_total of each, gathered); n_shards <= 64.
 *   u_local_out : [k] the local uniform where this shard (my_shard) owns the
 *       draw, 0 elsewhere;  mine_out : [k] bytes, 1 where it owns the draw;
 *   owner_out : [k] owning shard of every draw, or NULL.
 *   status_out_device : device int or NULL; DISTRL_ERR_SIZE if the totals sum
 *       to 0 or do not fit 64 bits (then nothing is owned).
 * Every shard then calls distrl_sample with u_local_out as it is and keeps the
 * positions it owns; un-normalised local weights become global ones by a factor
 * per shard, ((N / N_shard)(T_shard / T))^-beta.
 */
int distrl_route_draws(const uint64_t *u_fix, int64_t k, const uint64_t *shard_totals_device,
                       int n_shards, int my_shard, uint64_t *u_local_out, uint8_t *mine_out,
                       int *owner_out, int *status_out_device, void *stream);

/*
 * What a shard contributes to a batch drawn over several shards, after it has
 * sampled with distrl_route_draws' uniforms (normalise = 0): for the draws it
 * owns, the global index index_base + idx_local[j] and the un-normalised global
 * weight (n_global q / T)^-beta = w_local[j] ((n_global / n_local)(T_shard / T))^-beta;
 * -1 and 0 for the others, so that an element-wise maximum over the shards (one
 * all-reduce) assembles the batch.  distrl_normalise_weights then divides the
 * assembled weights by their maximum, as distrl_sample does for one shard.
 *   mine, idx_local, w_local : [k] as written by distrl_route_draws / distrl_sample;
 *   index_base : number of transitions in the shards before this one;
 *   w_global_out : [k] or NULL (then w_local may be NULL too).
 */
int distrl_finish_shard_draws(int64_t k, const uint8_t *mine, const int64_t *idx_local,
                              const float *w_local, const uint64_t *shard_totals_device,
                              int n_shards, int my_shard, int64_t n_local, int64_t n_global,
                              int64_t index_base, float beta, int64_t *idx_global_out,
                              float *w_global_out, void *stream);
int distrl_normalise_weights(float *is_weight, int64_t k, void *stream);

/*
 * Priority refresh for sampled indices (Section 5.3: priorities are updated
 * from the latest policy).  For j = 0..k-1 in order:
 *   mass_j = (w_td |new_abs_delta[j]| + w_rho min(rho_i, rho_clip) + w_ent H_i)^alpha,
 *   i = idx[j], rho_i and H_i gathered from the full [n] arrays;
 *   q[i] = Q(mass_j); every partial sum of the tree is repaired exactly.
 * If an index occurs more than once the highest position wins, as a
 * sequential loop would leave it.
 *   mass_out : [k] or NULL, the fp32 mass computed for each position.
 * An index outside [0, n) is skipped and DISTRL_ERR_INDEX recorded.
 */
int distrl_update_priorities(distrl_sampler *s, const int64_t *idx, int64_t k,
                             const float *new_abs_delta, const float *logp_target,
                             const float *logp_behaviour, const float *entropy,
                             const distrl_prio_cfg *cfg, float *mass_out, void *stream);

/*
 * Circular replay buffer (App. A, "Circular Replay Buffer": fixed capacity N, the
 * write index advances as i <- (i+1) mod N and new experiences overwrite the
 * oldest).  Overwrites the masses of the k slots head, head+1, ... (mod n) with
 * new_q[0..k) and repairs every partial sum exactly, so sampling continues as if
 * the sampler had been rebuilt.  The caller copies the transitions themselves
 * into the same slots of its SoA arrays and advances its head to (head+k) mod n.
 *   new_q : [k] device masses, each in [1, 2^32-1] (e.g. from distrl_compute_priorities).
 * If k > n only the last n writes survive, as a sequential loop would leave it.
 */
int distrl_replay_overwrite(distrl_sampler *s, int64_t head, int64_t k, const uint32_t *new_q,
                            void *stream);

/* ---------------------------------------------------------------------------
 * Circular replay buffer of whole trajectories (App. A "Circular Replay Buffer":
 * capacity N, the write index advances as i <- (i+1) mod N and new experiences
 * overwrite the oldest; Section 5.3 prioritises and replays trajectories).
 *
 * The buffer is the caller's SoA arrays of N slots (any fp32 per-transition
 * fields: rewards, values, log-probs, entropy, ...) and the masses prio_q.  The
 * library keeps its structure and, after every ingest, hands back the CSR view
 * the other entry points take:
 *   traj_offsets[0 .. m_capacity] : segment offsets; the flat buffer is cut into
 *       segments, each a live trajectory or a dead stretch; entries past the
 *       last segment are N (empty segments), so a call that takes traj_offsets
 *       may always be given n_trajectories = m_capacity;
 *   traj_alive[0 .. m_capacity)   : 1.0f for a live trajectory, 0.0f otherwise
 *       (a score for distrl_filter_trajectories with threshold 0.5, which
 *       zeroes the masses of dead stretches after priorities were recomputed
 *       for the whole buffer).
 * Rules of an ingest, trajectory by trajectory in the order given:
 *   - a trajectory occupies consecutive slots from the write index on (the
 *     recursion of Section 5.2 runs along it); one that would reach past slot
 *     N-1 starts at slot 0 instead and the slots left at the end are retired;
 *   - every stored trajectory that loses a slot is evicted as a whole: its
 *     remaining slots are dead and their masses 0, so no draw returns them
 *     (their rows stay in place until overwritten);
 *   - an empty trajectory stores nothing.
 * A call whose rows plus retired slots exceed N (it would overwrite its own
 * trajectories) is refused with DISTRL_ERR_SIZE and changes nothing: ingest in
 * smaller batches.  Masses of new rows come from the caller (e.g. Retrace and
 * priorities run on the new batch first); with a sampler over prio_q given,
 * every partial sum is repaired exactly, as if the sampler had been rebuilt.
 * ------------------------------------------------------------------------- */
typedef struct distrl_replay distrl_replay; /* small host-side handle */
#define DISTRL_REPLAY_MAX_FIELDS 8

size_t distrl_replay_workspace_bytes(int64_t capacity);

/*  fields : HOST array of n_fields (<= DISTRL_REPLAY_MAX_FIELDS) device arrays of
 *      `capacity` floats each; prio_q : [capacity]; traj_offsets : [m_capacity+1];
 *      traj_alive : [m_capacity].  All are zero-filled / initialised to the empty
 *      buffer (one dead segment, no mass) on `stream`; dead rows stay finite.
 *  workspace : >= distrl_replay_workspace_bytes(capacity), 256-byte aligned; its
 *      first word is a status word for distrl_get_status (DISTRL_ERR_SIZE: more
 *      segments than m_capacity; DISTRL_ERR_OFFSETS: see distrl_replay_ingest).
 *  The handle keeps the pointers; free it with distrl_replay_destroy (that frees
 *  no device memory).  All calls on one buffer go to one stream. */
int distrl_replay_create(int64_t capacity, int n_fields, float *const *fields, uint32_t *prio_q,
                         int64_t *traj_offsets, float *traj_alive, int64_t m_capacity,
                         void *workspace, size_t workspace_bytes, void *stream, distrl_replay **out);

/*  k new trajectories whose rows are concatenated in new_fields / new_q:
 *  new_offsets_host : HOST array [k+1], non-decreasing from 0 (the learner knows
 *      the lengths of what it received); new_offsets : the same values on the
 *      DEVICE (the batch's own traj_offsets); a mismatch is reported as
 *      DISTRL_ERR_OFFSETS in the status word and leaves the structure unspecified.
 *  new_fields : HOST array of n_fields device arrays of new_offsets_host[k] rows;
 *  new_q : device masses of those rows, each in [1, 2^32-1].
 *  sampler : a sampler built over this buffer's prio_q, or NULL (then only
 *      prio_q is written and the caller rebuilds its sampler).
 *  n_segments_out_device : device int64 or NULL; receives the number of segments. */
int distrl_replay_ingest(distrl_replay *rb, distrl_sampler *sampler, int64_t k,
                         const int64_t *new_offsets_host, const int64_t *new_offsets,
                         const float *const *new_fields, const uint32_t *new_q,
                         int64_t *n_segments_out_device, void *stream);

int64_t distrl_replay_head(const distrl_replay *rb); /* next write index; -1 for NULL */
int distrl_replay_destroy(distrl_replay *rb);

/*
 * Retrace targets (Section 5.2), priorities (Section 5.3) and the sampler's sum
 * tree in ONE pass over the trajectory buffer: what distrl_retrace_targets,
 * distrl_compute_priorities and distrl_build_sampler compute, without writing
 * td_delta and reading it (and both log-prob arrays, and prio_q) back.
 *   entropy     : [N] or NULL (NULL => H_t = -logpi_t).
 *   delta_scale : [N] or NULL; the priority uses |delta_t * delta_scale[t]|.
 *   td_delta    : [N] output or NULL;  prio_mass : [N] output or NULL.
 *   prio_q      : [N] output, kept by the sampler like in distrl_build_sampler.
 * Served only for fp32 per-step log-probs without bootstrap values and with
 * every array 16-byte aligned (DISTRL_ERR_PARAM / DISTRL_ERR_ALIGN otherwise:
 * use the three separate calls).  Results obey the same contracts as theirs.
 */
int distrl_retrace_priorities_build(const distrl_batch *batch, float gamma, float lambda,
                                    const float *entropy, const float *delta_scale,
                                    const distrl_prio_cfg *cfg, float *v_target, float *advantage,
                                    float *td_delta, uint32_t *prio_q, float *prio_mass,
                                    void *retrace_workspace, size_t retrace_workspace_bytes,
                                    void *sampler_workspace, size_t sampler_workspace_bytes,
                                    void *stream, distrl_sampler **out);

/*
 * What a drawn batch carries into the actor loss (Section 5.1, the policy loss;
 * App. A "Policy Update Mechanism"): the update direction is
 * -E_mu[rho_t A(s_t,a_t) grad log pi(a_t|s_t)], so sampled transition i = idx[j]
 * enters with the scalar
 *   coef[j] = is_weight[j] * rho_i * A_i,   rho_i = exp(logp_target[i] - logp_behaviour[i]).
 *   idx       : [k] device indices into the buffer (e.g. from distrl_sample), or
 *               NULL with k == n for the whole buffer in order (k == 0: nothing
 *               is done; any other k with idx NULL is DISTRL_ERR_SIZE).
 *   advantage : [n], e.g. the output of distrl_retrace_targets.
 *   is_weight : [k] importance-sampling weights from distrl_sample, or NULL (= 1).
 *   coef      : [k] output.
 *   status_out_device : device int or NULL; set to DISTRL_ERR_INDEX if some
 *               idx[j] lies outside [0, n) (that coef[j] is then NaN; nothing is
 *               read out of bounds).
 * fp32 arithmetic: one expf, two multiplies.
 */
int distrl_actor_coefficients(int64_t n, const int64_t *idx, int64_t k, const float *logp_target,
                              const float *logp_behaviour, const float *advantage,
                              const float *is_weight, float *coef, int *status_out_device,
                              void *stream);

/*
 * Trajectory-level draws (Section 5.3 prioritises trajectories): with a sampler
 * built over the M masses of distrl_compute_priorities_traj, a drawn index
 * idx[j] stands for the transitions [begin[j], end[j]) =
 * [traj_offsets[idx[j]], traj_offsets[idx[j]+1]) of the flat buffer.
 *   idx outside [0, m): begin = end = -1 and *status_out_device (if given) is set
 *   to DISTRL_ERR_INDEX.
 */
int distrl_trajectory_ranges(int64_t m, const int64_t *traj_offsets, const int64_t *idx, int64_t k,
                             int64_t *begin, int64_t *end, int *status_out_device, void *stream);

/*
 * Trajectory filter (Section 5.1 "Trajectory-Level Value Estimation"; App. A on
 * V_traj: the estimator scores whole trajectories and the replay buffer retains
 * only the high-value ones).  A trajectory is retained iff
 * traj_score[j] >= threshold (a NaN score is not retained).  Every transition of
 * a trajectory that is not retained gets prio_q = 0, so that no draw returns it;
 * the transitions stay where they are until overwritten.  Masses of retained
 * trajectories are left as they are.  Call it between distrl_compute_priorities
 * and distrl_build_sampler (or rebuild the sampler afterwards); at least one
 * retained trajectory must have a transition, or there is nothing to draw
 * (distrl_sample then returns index -1 and weight 0 for every draw and records
 * DISTRL_ERR_INDEX in the sampler's status word).
 *   traj_score : [M] device scores (e.g. V_traj's outputs);  prio_q : [N] in/out.
 *   kept_out_device : device uint64 or NULL; receives the number retained.
 */
int distrl_filter_trajectories(int64_t n, int64_t m, const int64_t *traj_offsets,
                               const float *traj_score, float threshold, uint32_t *prio_q,
                               uint64_t *kept_out_device, void *stream);

/* Writes total = sum_i q_i to *total_out_device (a device uint64). */
int distrl_sampler_total(distrl_sampler *s, uint64_t *total_out_device, void *stream);

/* Tree geometry, for inspection: level 1 holds the sums of 128 consecutive
 * masses, level l+1 the sums of 32 consecutive level-l entries; the top level
 * has at most 32 entries.  Returns the number of levels; for 1 <= level <=
 * levels also the byte offset of that level inside the workspace and its
 * entry count (uint64 entries). */
int distrl_sampler_level(const distrl_sampler *s, int level, size_t *offset_bytes,
                         int64_t *count);

int distrl_destroy_sampler(distrl_sampler *s);

/* Synchronises `stream`, returns the workspace's status word (DISTRL_OK or the
 * first device-side error recorded since the last read) and clears it. */
int distrl_get_status(void *workspace, void *stream);

/* Self-test of the library's bounded device-side waits (no counterpart in the
 * paper): launches one warp that waits, with a limit of about a thousand polls,
 * for a tile that nothing publishes.  Afterwards distrl_get_status(workspace)
 * returns DISTRL_ERR_TIMEOUT; the kernel neither traps nor hangs.  Lets a caller
 * check that its error handling sees device-side timeouts.
 *   workspace : a retrace workspace (>= distrl_retrace_workspace_bytes(1024)). */
int distrl_selftest_bounded_wait(void *workspace, size_t workspace_bytes, void *stream);

/*
 * Library option (no counterpart in the paper).  A normalising distrl_sample whose
 * grid fits the GPU lets its thread blocks wait for one another (batch maximum)
 * and is therefore launched cooperatively: the driver puts the whole grid on the
 * GPU at once, however busy other streams keep it.  With allowed = 0 (or when
 * the driver refuses such a launch) the last block to finish normalises instead:
 * correct under any scheduling, a little slower.  Process-wide; returns the old
 * setting.  (The Retrace scan needs no such launch: its tiles go by ticket, so a
 * block only ever waits for tiles of blocks that are already running.)
 */
int distrl_set_cooperative_launch(int allowed);

/*
 * Checked build (no counterpart in the paper).  A library compiled with
 * -DDISTRL_BOUNDS_CHECK range-checks every index its kernels compute right before
 * the access; an index out of range is recorded and the access skipped (nothing
 * traps, nothing is touched out of bounds).  Returns 1 if this library is such a
 * build, else 0 (record all zero).  Synchronises the device, copies
 * {violations, source line of the first, its index, its limit} to record4_host
 * (host int64[4]) and clears the record.  The ordinary build carries no checks.
 */
int distrl_bounds_report(int64_t *record4_host);

const char *distrl_error_string(int code);
const char *distrl_last_cuda_error(void); /* text of the last failed CUDA call, this thread */
const char *distrl_version(void);

#ifdef __cplusplus
}
#endif
#endif /* DISTRL_H */
