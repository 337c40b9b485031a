/*
 * distrl_oracle.c -- TEST INFRASTRUCTURE ONLY.
 *
 * A plain, slow, single-threaded fp64 CPU statement of what the A-RIDE learner
 * hot path computes (DistRL, arXiv 2410.14803).  It exists so that the CUDA
 * library can be checked against something obviously correct.  It shares no
 * code with the CUDA path, is never called by it, and is not a fallback: only
 * the test-suite, the smoke check and the benchmark's CPU-baseline leg may
 * load this file.
 *
 * Conventions: N transitions stored flat; trajectory j occupies the indices
 * [off[j], off[j+1]); "last" means the final stored step of a trajectory.
 * Every floating-point input arrives already widened to double (the widening
 * of fp32 / bf16 to fp64 is exact), every floating-point result is double.
 *
 * No blocking, fusion or reordering: every routine walks its definition.
 *
 * Pinned by tests/test_oracle_pins.py (closed forms, textbook reductions,
 * brute-force enumeration).  No function here is "parity unpinned".
 */
#include <math.h>
#include <stdint.h>
#include <stddef.h>

/* ------------------------------------------------------------------------- *
 * Token-level action log-probability.
 * The action log-prob that the importance ratio of Eq. (actor loss) needs is
 * the sum of the log-probs of the tokens that spell the action.  Step t owns
 * tokens [sto[t], sto[t+1]).
 * ------------------------------------------------------------------------- */
int oracle_token_logp(int64_t n, const int64_t *sto, const double *tok,
                      double *logp_out)
{
    for (int64_t t = 0; t < n; ++t) {
        double s = 0.0;
        for (int64_t i = sto[t]; i < sto[t + 1]; ++i)
            s += tok[i];
        logp_out[t] = s;
    }
    return 0;
}

/* ------------------------------------------------------------------------- *
 * Retrace(lambda) correction, Section 5.2:
 *   rho_t   = pi(a_t|s_t) / mu(a_t|s_t)            (Section 5.1)
 *   c_t     = lambda * min(1, rho_t)
 *   delta_t = r_t + gamma V(s_{t+1}) - V(s_t)      (Eq. TD error, App. A)
 *   Delta_t = sum_{k=t}^{H} gamma^{k-t} (prod_{i=t+1}^{k} c_i) delta_k
 *   V(s_t) <- V(s_t) + Delta_t
 * evaluated backwards per trajectory through the equivalent recursion
 *   Delta_H = delta_H,   Delta_t = delta_t + gamma c_{t+1} Delta_{t+1}.
 * V(s_{H+1}) is boot[j] when a bootstrap array is given, else 0.
 * Outputs: v_target = V + Delta, advantage = Delta (the corrected advantage,
 * equal to v_target - V), td_delta = delta (the one-step advantage).
 * ------------------------------------------------------------------------- */
int oracle_retrace(int64_t n, int64_t m, const int64_t *off,
                   const double *r, const double *V, const double *boot,
                   const double *logp_pi, const double *logp_mu,
                   double gamma, double lambda,
                   double *v_target, double *advantage, double *td_delta)
{
    (void)n;
    for (int64_t j = 0; j < m; ++j) {
        double Delta_next = 0.0, c_next = 0.0;
        for (int64_t t = off[j + 1] - 1; t >= off[j]; --t) {
            int last = (t == off[j + 1] - 1);
            double rho = exp(logp_pi[t] - logp_mu[t]);
            double c = lambda * fmin(1.0, rho);
            double v_next = last ? (boot ? boot[j] : 0.0) : V[t + 1];
            double delta = r[t] + gamma * v_next - V[t];
            double Delta = last ? delta : delta + gamma * c_next * Delta_next;
            v_target[t] = V[t] + Delta;
            advantage[t] = Delta;
            td_delta[t] = delta;
            Delta_next = Delta;
            c_next = c;
        }
    }
    return 0;
}

/* The same correction written as the printed double sum of Section 5.2,
 * O(T^2) per trajectory, products and powers formed term by term.  Used only
 * to check that the backward recursion above is the same quantity. */
int oracle_retrace_double_sum(int64_t n, int64_t m, const int64_t *off,
                              const double *r, const double *V,
                              const double *boot, const double *logp_pi,
                              const double *logp_mu, double gamma,
                              double lambda, double *Delta_out)
{
    (void)n;
    for (int64_t j = 0; j < m; ++j) {
        int64_t end = off[j + 1]; /* one past the last step H */
        for (int64_t t = off[j]; t < end; ++t) {
            double sum = 0.0;
            for (int64_t k = t; k < end; ++k) {
                double prod = 1.0;
                for (int64_t i = t + 1; i <= k; ++i)
                    prod *= lambda * fmin(1.0, exp(logp_pi[i] - logp_mu[i]));
                double v_next = (k == end - 1) ? (boot ? boot[j] : 0.0) : V[k + 1];
                double delta_k = r[k] + gamma * v_next - V[k];
                sum += pow(gamma, (double)(k - t)) * prod * delta_k;
            }
            Delta_out[t] = sum;
        }
    }
    return 0;
}

/* ------------------------------------------------------------------------- *
 * Monte-Carlo return of Section 5.1, G_t = sum_{k=t}^{H} gamma^{k-t} r_k, and
 * the label I[G_t > 0] the state-value classifier is trained on.
 * ------------------------------------------------------------------------- */
int oracle_mc_return(int64_t n, int64_t m, const int64_t *off, const double *r,
                     double gamma, double *G, uint8_t *label)
{
    (void)n;
    for (int64_t j = 0; j < m; ++j) {
        double g = 0.0;
        for (int64_t t = off[j + 1] - 1; t >= off[j]; --t) {
            g = r[t] + gamma * g;
            G[t] = g;
            label[t] = (g > 0.0) ? 1 : 0;
        }
    }
    return 0;
}

/* ------------------------------------------------------------------------- *
 * DPER priority, Section 5.3, per transition:
 *   p_t = w1 |delta_t| + w2 min(rho_t, rho_clip) + w3 H_t
 * H_t is the supplied entropy, else the paper's surrogate -log pi(a_t|s_t).
 * Sampling mass m_t = p_t^alpha (App. "Priority-Based Sampling", alpha = 0.5
 * in the paper).
 * ------------------------------------------------------------------------- */
int oracle_priority_mass(int64_t n, const double *td_delta,
                         const double *logp_pi, const double *logp_mu,
                         const double *entropy, double w_td, double w_rho,
                         double w_ent, double rho_clip, double alpha,
                         double *mass_out)
{
    for (int64_t t = 0; t < n; ++t) {
        double rho = exp(logp_pi[t] - logp_mu[t]);
        double H = entropy ? entropy[t] : -logp_pi[t];
        double p = w_td * fabs(td_delta[t]) + w_rho * fmin(rho, rho_clip) + w_ent * H;
        mass_out[t] = pow(p, alpha);
    }
    return 0;
}

/* Trajectory-level priority exactly as Section 5.3 states it: the means of
 * |delta|, rho and H over the trajectory's steps.  An empty trajectory gets
 * mass 0 (it can only be reached through the quantiser's floor). */
int oracle_priority_mass_traj(int64_t n, int64_t m, const int64_t *off,
                              const double *td_delta, const double *logp_pi,
                              const double *logp_mu, const double *entropy,
                              double w_td, double w_rho, double w_ent,
                              double rho_clip, double alpha, double *mass_out)
{
    (void)n;
    for (int64_t j = 0; j < m; ++j) {
        int64_t len = off[j + 1] - off[j];
        if (len <= 0) { mass_out[j] = 0.0; continue; }
        double sd = 0.0, sr = 0.0, sh = 0.0;
        for (int64_t t = off[j]; t < off[j + 1]; ++t) {
            sd += fabs(td_delta[t]);
            sr += fmin(exp(logp_pi[t] - logp_mu[t]), rho_clip);
            sh += entropy ? entropy[t] : -logp_pi[t];
        }
        double p = w_td * (sd / (double)len) + w_rho * (sr / (double)len)
                 + w_ent * (sh / (double)len);
        mass_out[j] = pow(p, alpha);
    }
    return 0;
}

/* ------------------------------------------------------------------------- *
 * Fixed-point quantiser.  Q is a function of the fp32 mass value:
 *   x = (double)m * S;  not (x > 0) -> 1;  x >= 2^32-1 -> 2^32-1;
 *   else max(1, round-half-to-even(x)).
 * The floor of 1 keeps every transition reachable (it plays the part of the
 * small epsilon of prioritized replay); NaN maps to 1.
 * ------------------------------------------------------------------------- */
int oracle_quantise(int64_t n, const float *mass_f32, double scale, uint32_t *q_out)
{
    for (int64_t t = 0; t < n; ++t) {
        double x = (double)mass_f32[t] * scale;
        uint32_t q;
        if (!(x > 0.0)) q = 1u;
        else if (x >= 4294967295.0) q = 4294967295u;
        else {
            double rn = nearbyint(x); /* default rounding mode: ties to even */
            q = (rn < 1.0) ? 1u : (uint32_t)rn;
        }
        q_out[t] = q;
    }
    return 0;
}

/* Inclusive cumulative masses C_i = sum_{j<=i} q_j and their total, the
 * normaliser of P(i) = q_i / sum_j q_j (App. "Priority-Based Sampling"). */
int oracle_prefix(int64_t n, const uint32_t *q, uint64_t *C_out, uint64_t *total_out)
{
    uint64_t run = 0;
    for (int64_t i = 0; i < n; ++i) {
        run += q[i];
        if (C_out) C_out[i] = run;
    }
    *total_out = run;
    return 0;
}

/* Proportional sampling by linear scan.  A draw is a 0.64 fixed-point uniform
 * u in [0, 2^64); the threshold is y = floor(u * total / 2^64) and the sample
 * is the first index whose cumulative mass exceeds y. */
int oracle_sample_linear(int64_t n, const uint32_t *q, int64_t k,
                         const uint64_t *u, int64_t *idx_out)
{
    uint64_t total = 0;
    for (int64_t i = 0; i < n; ++i) total += q[i];
    for (int64_t j = 0; j < k; ++j) {
        uint64_t y = (uint64_t)(((unsigned __int128)u[j] * (unsigned __int128)total) >> 64);
        uint64_t run = 0;
        int64_t pick = n - 1;
        for (int64_t i = 0; i < n; ++i) {
            run += q[i];
            if (run > y) { pick = i; break; }
        }
        idx_out[j] = pick;
    }
    return 0;
}

/* Importance-sampling weights of prioritized replay (Schaul et al., cited by
 * the paper for its replay): w_j = (N * P(idx_j))^(-beta), P = q / total,
 * divided by the largest weight of the batch when normalise != 0. */
int oracle_is_weights(int64_t n, const uint32_t *q, int64_t k,
                      const int64_t *idx, double beta, int normalise,
                      double *w_out)
{
    uint64_t total = 0;
    for (int64_t i = 0; i < n; ++i) total += q[i];
    double wmax = 0.0;
    for (int64_t j = 0; j < k; ++j) {
        double P = (double)q[idx[j]] / (double)total;
        w_out[j] = pow((double)n * P, -beta);
        if (w_out[j] > wmax) wmax = w_out[j];
    }
    if (normalise)
        for (int64_t j = 0; j < k; ++j) w_out[j] /= wmax;
    return 0;
}

/* Priority refresh of the sampled indices (Section 5.3, "priorities are
 * periodically updated based on the latest policy"), applied in batch order:
 * a later position overwrites an earlier one that names the same index.
 * The fp32 mass written for position j is returned so that the quantiser can
 * be fed the same value on both sides. */
int oracle_update(int64_t n, uint32_t *q, int64_t k, const int64_t *idx,
                  const double *new_abs_delta, const double *logp_pi,
                  const double *logp_mu, const double *entropy, double w_td,
                  double w_rho, double w_ent, double rho_clip, double alpha,
                  double scale, double *mass_out)
{
    (void)n;
    for (int64_t j = 0; j < k; ++j) {
        int64_t i = idx[j];
        double rho = exp(logp_pi[i] - logp_mu[i]);
        double H = entropy ? entropy[i] : -logp_pi[i];
        double p = w_td * fabs(new_abs_delta[j]) + w_rho * fmin(rho, rho_clip) + w_ent * H;
        double mass = pow(p, alpha);
        float mf = (float)mass;
        if (mass_out) mass_out[j] = mass;
        oracle_quantise(1, &mf, scale, &q[i]);
    }
    return 0;
}

/* The integer half of the refresh on its own: given the fp32 mass chosen for
 * each batch position, requantise and store in batch order (later wins). */
int oracle_update_from_mass(int64_t n, uint32_t *q, int64_t k, const int64_t *idx,
                            const float *mass_f32, double scale)
{
    (void)n;
    for (int64_t j = 0; j < k; ++j)
        oracle_quantise(1, &mass_f32[j], scale, &q[idx[j]]);
    return 0;
}

/* Circular replay buffer of App. A ("Circular Replay Buffer"): the write index advances as
 * i <- (i + 1) mod N and each new experience overwrites the slot it lands on.  Here only the masses
 * are kept; returns the index the next write would use. */
int64_t oracle_replay_overwrite(int64_t n, uint32_t *q, int64_t head, int64_t k, const uint32_t *new_q)
{
    int64_t i = head;
    for (int64_t j = 0; j < k; ++j) {
        q[i] = new_q[j];
        i = (i + 1) % n;
    }
    return i;
}

/* ------------------------------------------------------------------------- *
 * Per-sample coefficient of the actor loss (Section 5.1, the policy loss, and App. A "Policy Update
 * Mechanism"): the update direction is  - E_mu[ rho_t A(s_t,a_t) grad log pi(a_t|s_t) ],  so a
 * sampled transition i enters with the scalar  rho_i A_i,  rho_i = pi(a_i|s_i) / mu(a_i|s_i),
 * times its importance-sampling weight w_j when the batch was drawn by priority.
 *   idx NULL : j runs over the k = n transitions in order;  w NULL : weight 1.
 * ------------------------------------------------------------------------- */
int oracle_actor_coefficients(int64_t n, int64_t k, const int64_t *idx, const double *lp,
                              const double *lm, const double *adv, const double *w, double *coef)
{
    for (int64_t j = 0; j < k; ++j) {
        int64_t i = idx ? idx[j] : j;
        if (i < 0 || i >= n) return -1;
        double rho = exp(lp[i] - lm[i]);
        coef[j] = (w ? w[j] : 1.0) * rho * adv[i];
    }
    return 0;
}

/* Trajectory-level sampling (Section 5.3 prioritises trajectories tau): a drawn trajectory index j
 * stands for the transitions [off[j], off[j+1]) of the flat buffer. */
int oracle_trajectory_ranges(int64_t m, const int64_t *off, int64_t k, const int64_t *idx,
                             int64_t *begin, int64_t *end)
{
    for (int64_t j = 0; j < k; ++j) {
        if (idx[j] < 0 || idx[j] >= m) return -1;
        begin[j] = off[idx[j]];
        end[j] = off[idx[j] + 1];
    }
    return 0;
}

/* Trajectory filter (Section 5.1 "Trajectory-Level Value Estimation", App. A "The trajectory value
 * estimation function"): V_traj scores whole trajectories and the replay buffer retains only the
 * high-value ones.  A trajectory is retained iff score >= threshold; every transition of a
 * trajectory that is not retained gets sampling mass 0, so no proportional draw can return it.
 * Returns the number of retained trajectories. */
int64_t oracle_filter_trajectories(int64_t n, int64_t m, const int64_t *off, const double *score,
                                   double threshold, uint32_t *q)
{
    (void)n;
    int64_t kept = 0;
    for (int64_t j = 0; j < m; ++j) {
        if (score[j] >= threshold) { ++kept; continue; }
        for (int64_t t = off[j]; t < off[j + 1]; ++t) q[t] = 0u;
    }
    return kept;
}

/* ------------------------------------------------------------------------- *
 * Circular replay buffer of whole trajectories (App. A "Circular Replay Buffer": capacity N, the write
 * index advances as i <- (i + 1) mod N, new experiences overwrite the oldest; Section 5.3 prioritises
 * and replays trajectories).  Slots hold transitions; the flat buffer is cut into segments, each a
 * live trajectory or a dead stretch:
 *   start[i] = 1 : a segment starts at slot i (start[0] is always 1);
 *   alive[i] = 1 : slot i belongs to a live trajectory;   q[i] : its sampling mass (0 when dead).
 * A trajectory is stored in consecutive slots, because the Retrace recursion of Section 5.2 runs along
 * it: one that would straddle the end of the buffer starts at slot 0 instead, and the slots left at the
 * end are retired.  A stored trajectory that loses a slot is evicted as a whole: its remaining slots
 * are dead, their masses 0, so no draw returns them.  New trajectories are taken in order; an empty one
 * (length 0) stores nothing.  The call is refused (-1, nothing changed) if the offsets are not
 * non-decreasing from 0, or if the write index would advance by more than N in this one call (rows
 * plus retired slots), i.e. if the call would overwrite its own trajectories.
 * ------------------------------------------------------------------------- */
static void ring_kill_trajectory_at(int64_t n, uint32_t *q, uint8_t *alive, const uint8_t *start, int64_t i)
{
    if (!alive[i]) return;
    int64_t s = i, e = i + 1;
    while (!start[s]) --s;             /* first slot of the trajectory that owns slot i */
    while (e < n && !start[e]) ++e;    /* one past its last slot */
    for (int64_t t = s; t < e; ++t) { alive[t] = 0; q[t] = 0u; }
}

int oracle_ring_ingest(int64_t n, int n_fields, double *const *field, uint32_t *q, uint8_t *alive,
                       uint8_t *start, int64_t *head, int64_t k, const int64_t *new_off,
                       const double *const *new_field, const uint32_t *new_q)
{
    if (k < 0 || (k > 0 && new_off[0] != 0)) return -1;
    {   /* dry run: how far would the write index travel? */
        int64_t h = *head, advance = 0;
        for (int64_t j = 0; j < k; ++j) {
            int64_t T = new_off[j + 1] - new_off[j];
            if (T < 0) return -1;
            if (T == 0) continue;
            if (h + T > n) { advance += n - h; h = 0; }
            h += T;
            advance += T;
            if (advance > n) return -1;
        }
    }
    int64_t h = *head;
    for (int64_t j = 0; j < k; ++j) {
        int64_t T = new_off[j + 1] - new_off[j];
        if (T == 0) continue;
        if (h + T > n) {               /* would straddle the end: retire [h, n), go on at slot 0 */
            for (int64_t i = h; i < n; ++i) ring_kill_trajectory_at(n, q, alive, start, i);
            for (int64_t i = h; i < n; ++i) start[i] = (i == h);
            h = 0;
        }
        /* every stored trajectory that loses a slot goes as a whole */
        for (int64_t i = h; i < h + T; ++i) ring_kill_trajectory_at(n, q, alive, start, i);
        /* what follows the new trajectory starts a segment of its own */
        if (h + T < n) start[h + T] = 1;
        for (int64_t i = 0; i < T; ++i) {
            for (int f = 0; f < n_fields; ++f) field[f][h + i] = new_field[f][new_off[j] + i];
            q[h + i] = new_q[new_off[j] + i];
            alive[h + i] = 1;
            start[h + i] = (i == 0);
        }
        h += T;                        /* h == n wraps at the next write: (h + T) mod n */
    }
    *head = h % n;
    return 0;
}

/* The segments as CSR offsets over the flat buffer, with one liveness flag per segment.
 * Returns the number of segments M; off_out has M + 1 entries, the last one n. */
int64_t oracle_ring_segments(int64_t n, const uint8_t *start, const uint8_t *alive, int64_t *off_out,
                             uint8_t *seg_alive_out)
{
    int64_t m = 0;
    for (int64_t i = 0; i < n; ++i)
        if (start[i]) { off_out[m] = i; seg_alive_out[m] = alive[i]; ++m; }
    off_out[m] = n;
    return m;
}

/* Stratified draws of prioritized replay (Schaul et al., the replay the paper's DPER builds on): the unit
 * interval is cut into k equal strata and draw j takes its uniform from stratum j,
 *   u'_j = (j + u_j) / k     in 0.64 fixed point:  u'_j = floor((j 2^64 + u_j) / k),
 * so that a batch covers the whole range of cumulative mass.  Sampling itself is unchanged. */
int oracle_stratify(int64_t k, const uint64_t *u, uint64_t *u_out)
{
    for (int64_t j = 0; j < k; ++j) {
        unsigned __int128 x = ((unsigned __int128)(uint64_t)j << 64) + u[j];
        u_out[j] = (uint64_t)(x / (unsigned __int128)(uint64_t)k);
    }
    return 0;
}
