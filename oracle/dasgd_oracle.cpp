// CPU oracle for DaSGD -- TEST INFRASTRUCTURE, see dasgd_oracle.h.
// Plain loops in the order the paper states them; no blocking, no fusion.
#include "dasgd_oracle.h"

#include <cmath>
#include <cstring>
#include <deque>
#include <new>
#include <vector>
#ifdef _OPENMP
#include <omp.h>
#endif

namespace {

// bfloat16 = the upper 16 bits of a float32; widening is exact.
inline float bf16_to_f32(uint16_t b) {
  uint32_t u = static_cast<uint32_t>(b) << 16;
  float f;
  std::memcpy(&f, &u, 4);
  return f;
}

// float32 -> bfloat16, round to nearest, ties to even; NaN stays NaN.
inline uint16_t f32_to_bf16_rne(float f) {
  uint32_t u;
  std::memcpy(&u, &f, 4);
  if ((u & 0x7F800000u) == 0x7F800000u && (u & 0x007FFFFFu) != 0u)
    return static_cast<uint16_t>((u >> 16) | 0x0040u);
  uint32_t keep = u >> 16, rest = u & 0xFFFFu;
  if (rest > 0x8000u || (rest == 0x8000u && (keep & 1u))) keep += 1;
  return static_cast<uint16_t>(keep);
}

struct Pending {
  int64_t s;                // number of completed local steps when the snapshot was taken
  std::vector<float> snap;  // [K][P]
  std::vector<float> mean;  // [P]
  std::vector<float> snap_m;  // [K][P] momentum buffers at the snapshot (momentum averaging only)
  std::vector<float> mean_m;  // [P]
  bool averaged;
};

}  // namespace

struct oracle_dasgd {
  int32_t K, tau, d, dtype, merge_mode;
  int32_t K_total = 0;  // > 0: this object holds K of the K_total workers (a shard of the worker axis)
  int64_t P;
  float xi, momentum, weight_decay;
  bool nesterov = false, decoupled_wd = false;
  bool average_momentum = false;  // the momentum buffers go through snapshot, mean and merge like the weights
  int64_t t;  // completed local steps
  std::vector<float> w, m;
  std::vector<uint16_t> w_lp;
  std::deque<Pending> pending;  // oldest first
};

extern "C" {

oracle_dasgd *oracle_dasgd_create(int32_t K, int64_t P, int32_t tau, int32_t d, float xi,
                                  float momentum, float weight_decay, int32_t dtype,
                                  int32_t merge_mode) {
  if (K < 1 || P < 1 || tau < 1 || d < 0) return nullptr;
  if (!(xi >= 0.0f && xi <= 1.0f)) return nullptr;
  if (dtype != ORACLE_F32 && dtype != ORACLE_BF16_MASTER_F32) return nullptr;
  if (merge_mode != ORACLE_MERGE_XI && merge_mode != ORACLE_MERGE_DELTA) return nullptr;
  oracle_dasgd *o = new (std::nothrow) oracle_dasgd();
  if (!o) return nullptr;
  o->K = K; o->P = P; o->tau = tau; o->d = d; o->xi = xi;
  o->momentum = momentum; o->weight_decay = weight_decay;
  o->dtype = dtype; o->merge_mode = merge_mode; o->t = 0;
  o->w.assign(static_cast<size_t>(K) * P, 0.0f);
  o->m.assign(static_cast<size_t>(K) * P, 0.0f);
  if (dtype == ORACLE_BF16_MASTER_F32) o->w_lp.assign(static_cast<size_t>(K) * P, 0);
  return o;
}

void oracle_dasgd_destroy(oracle_dasgd *o) { delete o; }

int oracle_dasgd_set_variant(oracle_dasgd *o, int32_t nesterov, int32_t decoupled_wd) {
  if (!o || (nesterov && o->momentum == 0.0f)) return ORACLE_ERR_ARG;
  o->nesterov = nesterov != 0;
  o->decoupled_wd = decoupled_wd != 0;
  return ORACLE_OK;
}

int oracle_dasgd_set_momentum_averaging(oracle_dasgd *o, int32_t on) {
  if (!o || (on && o->momentum == 0.0f) || !o->pending.empty()) return ORACLE_ERR_ARG;
  o->average_momentum = on != 0;
  return ORACLE_OK;
}

int oracle_dasgd_set_state(oracle_dasgd *o, const float *w, const float *m) {
  if (!o || !w) return ORACLE_ERR_ARG;
  const size_t n = static_cast<size_t>(o->K) * o->P;
  std::memcpy(o->w.data(), w, n * sizeof(float));
  if (m) std::memcpy(o->m.data(), m, n * sizeof(float));
  if (o->dtype == ORACLE_BF16_MASTER_F32)
    for (size_t i = 0; i < n; ++i) o->w_lp[i] = f32_to_bf16_rne(o->w[i]);
  return ORACLE_OK;
}

int oracle_dasgd_get_state(const oracle_dasgd *o, float *w, float *m, uint16_t *w_lp) {
  if (!o) return ORACLE_ERR_ARG;
  const size_t n = static_cast<size_t>(o->K) * o->P;
  if (w) std::memcpy(w, o->w.data(), n * sizeof(float));
  if (m) std::memcpy(m, o->m.data(), n * sizeof(float));
  if (w_lp) {
    if (o->dtype != ORACLE_BF16_MASTER_F32) return ORACLE_ERR_ARG;
    std::memcpy(w_lp, o->w_lp.data(), n * sizeof(uint16_t));
  }
  return ORACLE_OK;
}

int64_t oracle_dasgd_steps_done(const oracle_dasgd *o) { return o ? o->t : -1; }
int32_t oracle_dasgd_pending(const oracle_dasgd *o) {
  return o ? static_cast<int32_t>(o->pending.size()) : -1;
}

int oracle_dasgd_get_pending(const oracle_dasgd *o, int32_t i, int64_t *s, float *snap,
                             float *mean) {
  if (!o || i < 0 || i >= static_cast<int32_t>(o->pending.size())) return ORACLE_ERR_ARG;
  const Pending &q = o->pending[i];
  if (s) *s = q.s;
  if (snap) std::memcpy(snap, q.snap.data(), q.snap.size() * sizeof(float));
  if (mean) {
    if (!q.averaged) return ORACLE_ERR_STATE;
    std::memcpy(mean, q.mean.data(), q.mean.size() * sizeof(float));
  }
  return ORACLE_OK;
}

int oracle_dasgd_get_pending_momentum(const oracle_dasgd *o, int32_t i, float *snap_m, float *mean_m) {
  if (!o || !o->average_momentum || i < 0 || i >= static_cast<int32_t>(o->pending.size())) return ORACLE_ERR_ARG;
  const Pending &q = o->pending[i];
  if (snap_m) std::memcpy(snap_m, q.snap_m.data(), q.snap_m.size() * sizeof(float));
  if (mean_m) {
    if (!q.averaged) return ORACLE_ERR_STATE;
    std::memcpy(mean_m, q.mean_m.data(), q.mean_m.size() * sizeof(float));
  }
  return ORACLE_OK;
}

// Eq. 2, first branch, with the momentum / weight-decay form stated in the header.
int oracle_dasgd_local_step(oracle_dasgd *o, const void *g, float lr) {
  if (!o || !g) return ORACLE_ERR_ARG;
  const int64_t P = o->P;
  const double eta = lr, mu = o->momentum, lambda = o->weight_decay;
  const float *g32 = static_cast<const float *>(g);
  const uint16_t *g16 = static_cast<const uint16_t *>(g);
  const bool bf16 = o->dtype == ORACLE_BF16_MASTER_F32;
  for (int32_t k = 0; k < o->K; ++k) {
#pragma omp parallel for schedule(static)
    for (int64_t p = 0; p < P; ++p) {
      const size_t i = static_cast<size_t>(k) * P + p;
      const double gi = bf16 ? static_cast<double>(bf16_to_f32(g16[i])) : static_cast<double>(g32[i]);
      const double w_old = o->w[i];
      const double gp = o->decoupled_wd ? gi : gi + lambda * w_old;
      double dir = gp;  // the direction the weights move along
      if (o->momentum != 0.0f) {
        o->m[i] = static_cast<float>(mu * static_cast<double>(o->m[i]) + gp);
        dir = o->nesterov ? gp + mu * static_cast<double>(o->m[i]) : static_cast<double>(o->m[i]);
      }
      const double decay = o->decoupled_wd ? eta * lambda * w_old : 0.0;
      o->w[i] = static_cast<float>(w_old - decay - eta * dir);
      if (bf16) o->w_lp[i] = f32_to_bf16_rne(o->w[i]);
    }
  }
  o->t += 1;
  return ORACLE_OK;
}

// The bracketed term of Eq. 2's second branch: the just-stepped weights of every worker.
int oracle_dasgd_snapshot(oracle_dasgd *o) {
  if (!o) return ORACLE_ERR_ARG;
  Pending q;
  q.s = o->t;
  q.snap = o->w;
  if (o->average_momentum) q.snap_m = o->m;
  q.averaged = false;
  o->pending.push_back(std::move(q));
  return ORACLE_OK;
}

// (1/M) * sum over workers, Eq. 2 second branch.
int oracle_dasgd_average(oracle_dasgd *o) {
  if (!o) return ORACLE_ERR_ARG;
  if (o->K_total > 0) return ORACLE_ERR_STATE;  // a shard cannot form the mean alone
  Pending *q = nullptr;
  for (auto &cand : o->pending)
    if (!cand.averaged) { q = &cand; break; }  // oldest snapshot that has no mean yet
  if (!q) return ORACLE_ERR_STATE;
  const int64_t P = o->P;
  q->mean.assign(static_cast<size_t>(P), 0.0f);
#pragma omp parallel for schedule(static)
  for (int64_t p = 0; p < P; ++p) {
    double acc = 0.0;
    for (int32_t k = 0; k < o->K; ++k) acc += static_cast<double>(q->snap[static_cast<size_t>(k) * P + p]);
    q->mean[p] = static_cast<float>(acc / static_cast<double>(o->K));
  }
  if (o->average_momentum) {  // the same (1/M) * sum over workers, applied to the momentum buffers
    q->mean_m.assign(static_cast<size_t>(P), 0.0f);
#pragma omp parallel for schedule(static)
    for (int64_t p = 0; p < P; ++p) {
      double acc = 0.0;
      for (int32_t k = 0; k < o->K; ++k) acc += static_cast<double>(q->snap_m[static_cast<size_t>(k) * P + p]);
      q->mean_m[p] = static_cast<float>(acc / static_cast<double>(o->K));
    }
  }
  q->averaged = true;
  return ORACLE_OK;
}

// The worker axis split over several holders (the data-parallel deployment of Section II-B: every
// machine owns some of the M workers and an all-reduce forms the sum).  The (1/M) * sum_j of Eq. 2 is
// then a two-level sum: each holder adds up its own workers, the partial sums are added across
// holders (by the caller), and the total is divided by M = K_total once.
int oracle_dasgd_set_shard(oracle_dasgd *o, int32_t K_total) {
  if (!o || K_total < o->K || o->average_momentum) return ORACLE_ERR_ARG;
  o->K_total = K_total;
  return ORACLE_OK;
}

int oracle_dasgd_partial_sum(const oracle_dasgd *o, double *sum) {
  if (!o || !sum) return ORACLE_ERR_ARG;
  const Pending *q = nullptr;
  for (const auto &cand : o->pending)
    if (!cand.averaged) { q = &cand; break; }  // oldest snapshot that has no mean yet
  if (!q) return ORACLE_ERR_STATE;
  const int64_t P = o->P;
#pragma omp parallel for schedule(static)
  for (int64_t p = 0; p < P; ++p) {
    double acc = 0.0;
    for (int32_t k = 0; k < o->K; ++k) acc += static_cast<double>(q->snap[static_cast<size_t>(k) * P + p]);
    sum[p] = acc;
  }
  return ORACLE_OK;
}

int oracle_dasgd_set_mean_from_sum(oracle_dasgd *o, const double *total) {
  if (!o || !total) return ORACLE_ERR_ARG;
  if (o->K_total < 1) return ORACLE_ERR_STATE;
  Pending *q = nullptr;
  for (auto &cand : o->pending)
    if (!cand.averaged) { q = &cand; break; }
  if (!q) return ORACLE_ERR_STATE;
  const int64_t P = o->P;
  q->mean.assign(static_cast<size_t>(P), 0.0f);
#pragma omp parallel for schedule(static)
  for (int64_t p = 0; p < P; ++p) q->mean[p] = static_cast<float>(total[p] / static_cast<double>(o->K_total));
  q->averaged = true;
  return ORACLE_OK;
}

// Eq. 2, second branch, applied to the already-stepped weights.
int oracle_dasgd_merge(oracle_dasgd *o) {
  if (!o) return ORACLE_ERR_ARG;
  if (o->pending.empty() || !o->pending.front().averaged) return ORACLE_ERR_STATE;
  const Pending &q = o->pending.front();
  const int64_t P = o->P;
  const double xi = o->xi, one_minus_xi = 1.0 - static_cast<double>(o->xi);
  const bool bf16 = o->dtype == ORACLE_BF16_MASTER_F32;
  for (int32_t k = 0; k < o->K; ++k) {
#pragma omp parallel for schedule(static)
    for (int64_t p = 0; p < P; ++p) {
      const size_t i = static_cast<size_t>(k) * P + p;
      const double wi = o->w[i], avg = q.mean[p];
      if (o->merge_mode == ORACLE_MERGE_XI)
        o->w[i] = static_cast<float>(xi * wi + one_minus_xi * avg);
      else
        o->w[i] = static_cast<float>(wi + (avg - static_cast<double>(q.snap[i])));
      if (bf16) o->w_lp[i] = f32_to_bf16_rne(o->w[i]);
      if (o->average_momentum) {  // the same blend on the momentum buffer, with the stale mean of the buffers
        const double mi = o->m[i], avg_m = q.mean_m[p];
        if (o->merge_mode == ORACLE_MERGE_XI)
          o->m[i] = static_cast<float>(xi * mi + one_minus_xi * avg_m);
        else
          o->m[i] = static_cast<float>(mi + (avg_m - static_cast<double>(q.snap_m[i])));
      }
    }
  }
  o->pending.pop_front();
  return ORACLE_OK;
}

// One iteration.  With u = completed steps after the local step:
//   d > 0: the snapshot taken at s = u-d (s a positive multiple of tau) is merged now;
//          then, if u is a multiple of tau, a new snapshot is taken and averaged.
//   d = 0: (Local SGD timing) snapshot, average and merge in the same iteration.
int oracle_dasgd_step(oracle_dasgd *o, const void *g, float lr) {
  int rc = oracle_dasgd_local_step(o, g, lr);
  if (rc) return rc;
  const int64_t u = o->t, tau = o->tau, d = o->d;
  if (d > 0 && u - d >= tau && (u - d) % tau == 0) {
    rc = oracle_dasgd_merge(o);
    if (rc) return rc;
  }
  if (u % tau == 0) {
    rc = oracle_dasgd_snapshot(o);
    if (rc) return rc;
    rc = oracle_dasgd_average(o);
    if (rc) return rc;
    if (d == 0) rc = oracle_dasgd_merge(o);
  }
  return rc;
}

// Eq. 3: d > t_c / t_p, smallest such positive integer; Section VI-D: tau = d + 1.
int oracle_dasgd_delay_guideline(double t_c, double t_p, int32_t *d, int32_t *tau) {
  if (!(t_c >= 0.0) || !(t_p > 0.0) || !d || !tau) return ORACLE_ERR_ARG;
  int32_t k = 1;
  while (!(t_c < static_cast<double>(k) * t_p)) ++k;
  *d = k;
  *tau = k + 1;
  return ORACLE_OK;
}

int oracle_dasgd_delay_from_system(double m, double n_p, double BW, double B_l, double FLOP, double FLOPS,
                                   int32_t *d, int32_t *tau) {
  if (!(BW > 0.0) || !(FLOPS > 0.0)) return ORACLE_ERR_ARG;
  return oracle_dasgd_delay_guideline(m * n_p / BW, B_l * FLOP / FLOPS, d, tau);
}

int oracle_dasgd_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

}  // extern "C"
