/*
 * CPU oracle for DaSGD (Local SGD with Delayed Averaging) -- TEST INFRASTRUCTURE.
 *
 * A plain, slow, single-pass restatement of the paper's update rule, used only to
 * check other implementations.  It is not a product code path and nothing in the
 * library may call it.  It shares no code with the CUDA implementation.
 *
 * What it follows:
 *   - Local step: Eq. 2, "otherwise" branch (Section III-C-1; restated in
 *     Appendix "Update Rule"):  x <- x - eta * g(x).  Momentum and weight decay are
 *     only named as hyper-parameters in Section IV-A (their values, no formula);
 *     the formula used is the usual one of the paper's platform:
 *     g' = g + lambda*w;  m <- mu*m + g' (m_0 = 0);  w <- w - eta*m.
 *   - Snapshot: the bracketed term of Eq. 2, second branch: each worker's weights
 *     right after the local step that closes a tau-block (Fig. 2 narrative:
 *     with tau = 3 the averaging starts once three local updates are done).
 *   - Worker-axis mean: the (1/M) * sum_j of Eq. 2 (right-multiplication by J in
 *     the matrix form of Appendix "Matrix Representation").
 *   - Delayed merge: Eq. 2, second branch, appendix condition (k+1-d) mod tau = 0:
 *     x <- xi*(x - eta*g) + (1-xi)*mean, i.e. a xi-blend applied to the already
 *     locally-stepped weights, d steps after the snapshot.
 *   - A second merge form, w <- w + (mean - snapshot_of_this_worker), is provided
 *     as merge_mode 1.  It is NOT in the paper.
 *
 * Numerics: state (w, m, snapshot, mean) is float32; every element is computed in
 * double from the float32 state and rounded to float32 once, at the store.  In
 * dtype 1 gradients arrive as bfloat16 (widened exactly) and a bfloat16 copy of
 * the weights, rounded to nearest-even, is refreshed after every write of w.
 *
 * Pins (tests marked "not gpu"): hand-worked trajectories derived from Eq. 2,
 * the minibatch-SGD and Local-SGD special cases (Eq. 1, Section II-C-3), the
 * averaged-model recursion of Section III-C-1, the deviation contraction used in
 * the proof of the theorem (Appendix), closed forms for momentum and weight
 * decay, torch.optim.SGD for the momentum/weight-decay local step, torch's
 * bfloat16 cast for the rounding, and the paper's Table II for the delay guideline.
 * Parity unpinned by the paper: schedules with d > tau (the paper assumes
 * d <= tau) -- defined here by pipelining snapshots, checked by invariants only.
 */
#ifndef DASGD_ORACLE_H
#define DASGD_ORACLE_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct oracle_dasgd oracle_dasgd;

enum { ORACLE_F32 = 0, ORACLE_BF16_MASTER_F32 = 1 };
enum { ORACLE_MERGE_XI = 0, ORACLE_MERGE_DELTA = 1 };
enum { ORACLE_OK = 0, ORACLE_ERR_ARG = 1, ORACLE_ERR_STATE = 2 };

/* K workers, P parameters, period tau >= 1, delay d >= 0, blend xi in [0,1]. */
oracle_dasgd *oracle_dasgd_create(int32_t K, int64_t P, int32_t tau, int32_t d, float xi,
                                  float momentum, float weight_decay, int32_t dtype,
                                  int32_t merge_mode);
void oracle_dasgd_destroy(oracle_dasgd *o);
/* Variants of the local step (the paper gives no formula, Section IV-A names only the values):
 *   nesterov:      w <- w - eta*(g' + mu*m) with the freshly updated m   (pinned: torch.optim.SGD(nesterov=True))
 *   decoupled_wd:  g' = g and w <- w - eta*lambda*w - eta*(step direction) (pinned: w*(1-eta*lambda) followed by
 *                  torch.optim.SGD without weight decay, and the closed form (1-eta*lambda)^T for zero gradients) */
int oracle_dasgd_set_variant(oracle_dasgd *o, int32_t nesterov, int32_t decoupled_wd);

/* Momentum averaging (NOT in the paper, which averages weights only): the momentum buffers go through the same
 * three operations as the weights -- copied at the snapshot, averaged over the workers, and blended back d steps
 * later with the same xi (or, in merge_mode 1, m <- m + (mean_m - snapshot_m)).  Needs momentum > 0; may only be
 * switched while no snapshot is pending; not available on a shard of the worker axis.
 * Pinned: identical workers stay identical and follow plain momentum SGD; xi = 1 changes nothing; with xi = 0 and
 * d = 0 every buffer equals the mean of the buffers right after a merge; the worker-mean of the buffers is
 * preserved by a d = 0 merge; a hand-worked trajectory (tests/golden). */
int oracle_dasgd_set_momentum_averaging(oracle_dasgd *o, int32_t on);
/* momentum snapshot [K][P] / its mean [P] of the i-th oldest pending snapshot; either may be NULL */
int oracle_dasgd_get_pending_momentum(const oracle_dasgd *o, int32_t i, float *snap_m, float *mean_m);

/* State access: w, m are [K][P] float32 (row k = worker k); w_lp is [K][P] bf16 bits. */
int oracle_dasgd_set_state(oracle_dasgd *o, const float *w, const float *m);
int oracle_dasgd_get_state(const oracle_dasgd *o, float *w, float *m, uint16_t *w_lp);
int64_t oracle_dasgd_steps_done(const oracle_dasgd *o);
int32_t oracle_dasgd_pending(const oracle_dasgd *o);
/* mean / snapshot of the i-th oldest pending snapshot (0 = oldest); either may be NULL */
int oracle_dasgd_get_pending(const oracle_dasgd *o, int32_t i, int64_t *s, float *snap,
                             float *mean);

/* The four operations of the path; g is [K][P] float32 (dtype 0) or bf16 bits (dtype 1). */
int oracle_dasgd_local_step(oracle_dasgd *o, const void *g, float lr);
int oracle_dasgd_snapshot(oracle_dasgd *o);
int oracle_dasgd_average(oracle_dasgd *o); /* mean of the oldest snapshot not yet averaged */
int oracle_dasgd_merge(oracle_dasgd *o);   /* blend the OLDEST pending mean, then drop it   */

/* Sharded worker axis (the data-parallel setting of Section II-B, where the workers live on several
 * machines and an all-reduce adds their contributions).  After oracle_dasgd_set_shard(o, K_total) the
 * object holds K of the K_total workers of Eq. 2; oracle_dasgd_average and oracle_dasgd_step then
 * fail with ORACLE_ERR_STATE, because the mean needs the other shards.  Instead:
 *   oracle_dasgd_partial_sum      -- sum over this shard's workers of the oldest snapshot that has no
 *                                    mean yet, per parameter, in double ([P]);
 *   (the caller adds the partial sums of all shards)
 *   oracle_dasgd_set_mean_from_sum -- mean = total / K_total, rounded to float32 once; the snapshot
 *                                    then counts as averaged and oracle_dasgd_merge can blend it.
 * Pinned: the shards of a partitioned run reproduce the unsharded oracle (a two-level sum of the same
 * terms), one shard with K_total = K reproduces it bit for bit, and identical shards behave like one. */
int oracle_dasgd_set_shard(oracle_dasgd *o, int32_t K_total);
int oracle_dasgd_partial_sum(const oracle_dasgd *o, double *sum);
int oracle_dasgd_set_mean_from_sum(oracle_dasgd *o, const double *total);

/* One iteration of the schedule: local step; merge if one lands; snapshot+mean if due. */
int oracle_dasgd_step(oracle_dasgd *o, const void *g, float lr);

/* Delay guideline (Section III-D, Eq. 3; Section VI-C and VI-D): the averaging is hidden when
 * t_c < d * t_p, so d is the smallest positive integer with that property, and tau = d + 1.
 * Pinned against every row of the paper's Table II.  Returns ORACLE_ERR_ARG unless t_c >= 0, t_p > 0. */
int oracle_dasgd_delay_guideline(double t_c, double t_p, int32_t *d, int32_t *tau);
/* The same from system parameters (Eq. 3): t_c = m*n_p/BW, t_p = B_l*FLOP/FLOPS. */
int oracle_dasgd_delay_from_system(double m, double n_p, double BW, double B_l, double FLOP, double FLOPS,
                                   int32_t *d, int32_t *tau);

int oracle_dasgd_threads(void); /* OpenMP threads the element loops use (1 if built without) */

#ifdef __cplusplus
}
#endif
#endif
