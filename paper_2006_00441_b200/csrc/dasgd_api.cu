// Host side of libdasgd: the C ABI declared in include/dasgd.h, the snapshot-slot state machine
// and the two-stream scheduler that lets the worker-axis mean run beside the next local steps.
#include "dasgd.h"
#include "dasgd_kernels.cuh"

#include <chrono>
#include <cstdio>
#include <cstring>
#include <deque>
#include <new>
#include <string>
#include <thread>
#include <vector>

namespace {

using dasgd::kThreads;
using dasgd::Params;

thread_local std::string g_init_error;

enum SlotState { SLOT_FREE = 0, SLOT_SNAPPED = 1, SLOT_AVERAGING = 2 };

struct Slot {
  SlotState state = SLOT_FREE;
  int64_t s = 0;                 // completed local steps when the snapshot was taken
  cudaEvent_t e_snap = nullptr;  // main stream: snapshot written
  cudaEvent_t e_avg = nullptr;   // side stream: mean written
  int stall_sp = -1;             // timing: span whose ev[1] marks "mean complete" (-1: none)
  std::vector<int> stall_sp_c;   // the same per column range
  int buf = -1;                  // index into ctx->pool of the array that holds this snapshot
  bool holds = false;            // this slot still keeps pool[buf] from being overwritten
  // Chunked pipeline (n_chunks > 1): one event pair per column range.  `chunked` says which set the
  // last snapshot of this slot recorded.
  std::vector<cudaEvent_t> e_snap_c, e_avg_c;
  bool chunked = false;
  // Momentum averaging, chunked iterations only: "copy of the buffers written" (main stream) and "mean of the
  // buffers written" (side stream).  Elsewhere e_snap / e_avg cover the buffers as well.
  cudaEvent_t e_msnap = nullptr, e_mavg = nullptr;
};

// A pair of timing events, tagged with what the time between them measures.  For the four kinds of
// kernels the pair brackets the launch on its stream.  For TAG_STALL the pair straddles two streams:
// ev[0] is recorded on the stream that is about to wait for a mean (it completes when that stream has
// nothing else left to do), ev[1] on the side stream right after the mean kernel; ev[1] - ev[0], when
// positive, is how long the mean kept that stream waiting.
enum SpanTag { TAG_STEP = 0, TAG_SNAPSHOT = 1, TAG_MEAN = 2, TAG_MERGE = 3, TAG_STALL = 4, TAG_COUNT = 5 };
struct Span {
  cudaEvent_t ev[2] = {nullptr, nullptr};
  int tag = 0;
  bool open = false;            // in use, not yet harvested
  bool rec[2] = {false, false}; // which of the two events have been recorded
  long long units = 0;          // replica-parameters the timed launch processes
};

// One recorded iteration of the chunked pipeline: every pointer and switch that the launches depend on
// (the gradients and the learning rate come from device memory, so they are not part of the key).
struct GraphKey {
  const void *w, *w_out, *mean, *snap_in, *red_in, *mean_out;
  int mode, vec, s_due, keep_w;
  bool operator==(const GraphKey &o) const {
    return w == o.w && w_out == o.w_out && mean == o.mean && snap_in == o.snap_in && red_in == o.red_in &&
           mean_out == o.mean_out && mode == o.mode && vec == o.vec && s_due == o.s_due && keep_w == o.keep_w;
  }
};
struct GraphEntry {
  GraphKey key;
  cudaGraphExec_t exec = nullptr;
  int64_t kernels = 0;  // kernel launches one replay stands for
};

struct DeviceGuard {
  int prev = -1;
  bool switched = false;
  explicit DeviceGuard(int dev) {
    if (cudaGetDevice(&prev) == cudaSuccess && prev != dev) switched = cudaSetDevice(dev) == cudaSuccess;
  }
  ~DeviceGuard() {
    if (switched) cudaSetDevice(prev);
  }
};

}  // namespace

struct dasgd_ctx {
  dasgd_config cfg;
  cudaStream_t s0, s1;
  int64_t t = 0;
  int64_t launches = 0;
  bool vec = false;  // rows are 16-byte aligned for every array: vector kernels usable
  int epu = 4;       // elements per vector unit
  std::vector<Slot> slots;
  std::deque<int> pending;  // slot indices, oldest snapshot first
  // Weight-sized arrays: pool[0] = cfg.w, pool[1 + i] = the i-th [K][ld] array of cfg.snap.
  // `cur` holds the current weights; frozen[b] counts the pending slots whose snapshot is pool[b] (two
  // snapshots taken with no weight update between them share one array).
  // Copy mode: cur stays 0 and snapshots are copies.  Rotate mode: a snapshot freezes `cur` itself and
  // the next kernel that writes weights writes them into a free array, which becomes `cur`.
  std::vector<float *> pool;
  std::vector<int> frozen;
  int cur = 0;
  bool rotate = false;
  // Chunked pipeline: the parameter axis cut into `chunks` ranges of `chunk_cols` columns (a multiple
  // of the vector kernels' tile, so every range starts on a 16-byte boundary); the last may be shorter.
  int chunks = 1;
  long long chunk_cols = 0;
  // DASGD_FLAG_TWO_LANES: odd column ranges run on this stream, forked from and joined to the main
  // stream inside every chunked iteration, so that the kernel of range i+1 fills the SMs as the kernel
  // of range i drains instead of waiting for the stream's next command.
  // DASGD_FLAG_TWO_SIDE_STREAMS: the means of odd column ranges run on this stream (same priority as the side
  // stream), so that the mean of range i+1 need not wait for the mean of range i; e_cross orders one side stream
  // after the other where the two have to meet (end of a group of ranges, end of the iteration).
  cudaStream_t s1b = nullptr;
  cudaEvent_t e_cross = nullptr;
  std::vector<cudaStream_t> lanes;      // extra lanes (lane 0 is the main stream)
  std::vector<cudaEvent_t> e_joins;     // one per extra lane
  cudaEvent_t e_fork = nullptr;
  // DASGD_FLAG_GRAPH: recorded iterations of the chunked pipeline, their capture-only events and the
  // device block the replayed kernels read the gradients pointer and the learning rate from.
  bool use_graph = false;
  dasgd::DynArgs *dyn_dev = nullptr;
  std::vector<GraphEntry> graphs;
  std::vector<cudaEvent_t> cap_ev;  // per column range, then one per extra lane, then fork and side-stream join
  // Momentum averaging (dasgd_set_momentum_averaging): copies of the momentum buffers per slot and their means.
  float *m_snap = nullptr;  // [n_slots][K][ld]
  float *m_mean = nullptr;  // [n_slots][ld]
  // Sharded worker axis: this context holds cfg.K of K_total workers; `exchange` adds the partial sums of
  // all shards (an all-reduce) on the side stream.  0 / NULL: every worker is here.
  int32_t K_total = 0;
  dasgd_exchange_fn exchange = nullptr;
  void *exchange_user = nullptr;
  // host-gradient staging (dasgd_step_host): a copy stream and, per staging array, an event for
  // "copy landed" (copy stream) and one for "kernels have consumed it" (main stream)
  cudaStream_t s_copy = nullptr;
  std::vector<cudaEvent_t> e_copied, e_consumed;
  std::vector<bool> stage_used;
  int64_t host_calls = 0;
  std::vector<Span> spans;
  int64_t span_n[TAG_COUNT] = {0, 0, 0, 0, 0};
  double span_ms[TAG_COUNT] = {0, 0, 0, 0, 0};
  int64_t span_units[TAG_COUNT] = {0, 0, 0, 0, 0};
  std::string err;
};

namespace {

dasgd_status fail(dasgd_ctx *c, dasgd_status s, const std::string &msg) {
  if (c) c->err = msg; else g_init_error = msg;
  return s;
}

dasgd_status cuda_fail(dasgd_ctx *c, cudaError_t e, const char *what) {
  return fail(c, DASGD_ERR_CUDA, std::string(what) + ": " + cudaGetErrorString(e));
}

#define CU(c, call)                                        \
  do {                                                     \
    cudaError_t e_ = (call);                               \
    if (e_ != cudaSuccess) return cuda_fail(c, e_, #call); \
  } while (0)

bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// The snapshot array of a slot; NULL for a slot that has none (made by the inline-mean schedule).
float *snap_ptr(const dasgd_ctx *c, int slot) {
  const int b = c->slots[slot].buf;
  return b >= 0 && b < (int)c->pool.size() ? c->pool[b] : nullptr;
}
float *mean_ptr(const dasgd_ctx *c, int slot) {
  return static_cast<float *>(c->cfg.mean) + (size_t)slot * c->cfg.ld;
}

Params base_params(const dasgd_ctx *c) {
  Params p{};
  p.w = c->pool[c->cur];
  p.w_out = c->pool[c->cur];
  p.m = static_cast<float *>(c->cfg.m);
  p.w_lp = static_cast<__nv_bfloat16 *>(c->cfg.w_lp);
  p.P = c->cfg.P;
  p.ld = c->cfg.ld;
  p.K = c->cfg.K;
  p.mu = c->cfg.momentum;
  p.lambda = c->cfg.weight_decay;
  p.nesterov = (c->cfg.flags & DASGD_FLAG_NESTEROV) ? 1 : 0;
  p.decoupled_wd = (c->cfg.flags & DASGD_FLAG_DECOUPLED_WD) ? 1 : 0;
  p.xi = c->cfg.xi;
  p.omx = 1.0f - c->cfg.xi;
  p.mean_div = c->K_total > 0 ? (float)c->K_total : 0.0f;
  p.group_tiles = 1;
  return p;
}

unsigned blocks_for(long long n, long long per_block) { return (unsigned)((n + per_block - 1) / per_block); }

// The same operation restricted to the columns [col0, col0 + len) of every row: all pointers move by
// col0 elements, the row stride stays.
Params columns(const dasgd_ctx *c, Params p, long long col0, long long len) {
  const size_t gsz = c->cfg.dtype == DASGD_BF16_MASTER_F32 ? 2 : 4;
  p.w += col0;
  p.w_out += col0;
  if (p.m) p.m += col0;
  if (p.dyn) p.g_off += col0;
  else if (p.g) p.g = static_cast<const char *>(p.g) + (size_t)col0 * gsz;
  if (p.w_lp) p.w_lp += col0;
  if (p.snap_out) p.snap_out += col0;
  if (p.snap_in) p.snap_in += col0;
  if (p.mean) p.mean += col0;
  if (p.mean_out) p.mean_out += col0;
  p.P = len;
  return p;
}

// -------------------------------------------------------------- timing bookkeeping

void harvest(dasgd_ctx *c, bool block) {
  for (Span &sp : c->spans) {
    if (!sp.open || !sp.rec[0] || !sp.rec[1]) continue;
    bool ready = true;
    for (int j = 0; j < 2 && ready; ++j) {
      if (block) {
        ready = cudaEventSynchronize(sp.ev[j]) == cudaSuccess;
      } else if (cudaEventQuery(sp.ev[j]) != cudaSuccess) {
        cudaGetLastError();  // "not ready" is not an error here
        ready = false;
      }
    }
    if (!ready) continue;
    float ms = 0.f;
    if (cudaEventElapsedTime(&ms, sp.ev[0], sp.ev[1]) == cudaSuccess) {
      if (sp.tag == TAG_STALL && ms < 0.f) ms = 0.f;  // the mean was complete before anyone waited
      c->span_n[sp.tag] += 1;
      c->span_ms[sp.tag] += ms;
      c->span_units[sp.tag] += sp.units;
    }
    sp.open = sp.rec[0] = sp.rec[1] = false;
  }
}

// A free span (events created on demand); -1 when timing is off or events cannot be created.
int span_alloc(dasgd_ctx *c, int tag, long long units) {
  if (!(c->cfg.flags & DASGD_FLAG_TIMING)) return -1;
  harvest(c, false);
  int idx = -1;
  for (size_t i = 0; i < c->spans.size(); ++i)
    if (!c->spans[i].open) { idx = (int)i; break; }
  if (idx < 0) {
    Span sp;
    if (cudaEventCreate(&sp.ev[0]) != cudaSuccess || cudaEventCreate(&sp.ev[1]) != cudaSuccess) return -1;
    c->spans.push_back(sp);
    idx = (int)c->spans.size() - 1;
  }
  Span &sp = c->spans[idx];
  sp.tag = tag;
  sp.units = units;
  sp.open = true;
  sp.rec[0] = sp.rec[1] = false;
  return idx;
}

void span_record(dasgd_ctx *c, int idx, int which, cudaStream_t stream) {
  if (idx < 0) return;
  Span &sp = c->spans[idx];
  if (cudaEventRecord(sp.ev[which], stream) == cudaSuccess) sp.rec[which] = true;
  else sp.open = false;
}

// Brackets a launch: records the opening event on `stream`; returns the span, or -1 when timing is off.
int span_begin(dasgd_ctx *c, int tag, cudaStream_t stream, long long units = 0) {
  const int idx = span_alloc(c, tag, units);
  span_record(c, idx, 0, stream);
  return idx;
}

void span_end(dasgd_ctx *c, int idx, cudaStream_t stream) { span_record(c, idx, 1, stream); }

// Stall accounting.  mean_done: called right after a mean kernel has been put on the side stream; the
// returned span is kept in the slot.  about_to_wait: called where `stream` is about to wait for that mean.
int stall_mean_done(dasgd_ctx *c, int old_idx, cudaStream_t side = nullptr) {
  if (old_idx >= 0 && old_idx < (int)c->spans.size() && c->spans[old_idx].open && c->spans[old_idx].tag == TAG_STALL &&
      !c->spans[old_idx].rec[0])
    c->spans[old_idx].open = false;  // the previous mean of this slot was never waited for
  const int idx = span_alloc(c, TAG_STALL, 0);
  span_record(c, idx, 1, side ? side : c->s1);
  return idx;
}

void stall_about_to_wait(dasgd_ctx *c, int &idx, cudaStream_t stream) {
  if (idx >= 0 && idx < (int)c->spans.size() && c->spans[idx].open && c->spans[idx].tag == TAG_STALL && !c->spans[idx].rec[0])
    span_record(c, idx, 0, stream);
  idx = -1;
}

// -------------------------------------------------------------- kernel launchers

// One launch enumerates (row, tile of 4096 columns) pairs in blockIdx.x.
bool fits_one_launch(const Params &p) { return ((p.P + 4095) / 4096) * (long long)p.K <= 0x7FFFFFFFLL; }

template <bool BF16, bool MOM, int MERGE, bool SNAP>
dasgd_status launch_step_t(dasgd_ctx *c, const Params &p, bool vec, cudaStream_t stream) {
  constexpr int EPU = 4;     // elements per unit of the vector step kernel, both dtypes
  constexpr int UNROLL = 4;
  long long done = 0;
  if (vec) {
    const long long units = p.P / EPU;
    if (units > 0) {
      const long long tiles = (units + (long long)kThreads * UNROLL - 1) / ((long long)kThreads * UNROLL);
      dasgd::k_local_step_vec<BF16, MOM, MERGE, SNAP><<<(unsigned)(tiles * p.K), kThreads, 0, stream>>>(p);
      c->launches++;
    }
    done = units * EPU;
  }
  if (done < p.P) {
    dim3 grid(blocks_for(p.P - done, kThreads), (unsigned)p.K);
    dasgd::k_local_step_scalar<BF16, MOM, MERGE, SNAP><<<grid, kThreads, 0, stream>>>(p, done);
    c->launches++;
  }
  CU(c, cudaGetLastError());
  return DASGD_OK;
}

template <bool BF16, bool MOM>
dasgd_status launch_step_m(dasgd_ctx *c, const Params &p, bool vec, int merge, bool snap, cudaStream_t stream) {
  switch (merge * 2 + (snap ? 1 : 0)) {
    case 0: return launch_step_t<BF16, MOM, 0, false>(c, p, vec, stream);
    case 1: return launch_step_t<BF16, MOM, 0, true>(c, p, vec, stream);
    case 2: return launch_step_t<BF16, MOM, 1, false>(c, p, vec, stream);
    case 3: return launch_step_t<BF16, MOM, 1, true>(c, p, vec, stream);
    case 4: return launch_step_t<BF16, MOM, 2, false>(c, p, vec, stream);
    default: return launch_step_t<BF16, MOM, 2, true>(c, p, vec, stream);
  }
}

// merge: 0 none, 1 xi, 2 delta (fused into the step kernel); snap: also write p.snap_out
// `stream`: the main stream, or the second lane of a chunked iteration.
dasgd_status launch_step(dasgd_ctx *c, const Params &p, bool vec, int merge, bool snap, cudaStream_t stream) {
  const bool bf16 = c->cfg.dtype == DASGD_BF16_MASTER_F32;
  const bool mom = c->cfg.momentum != 0.0f;
  if (!fits_one_launch(p)) return fail(c, DASGD_ERR_UNSUPPORTED, "K*P too large for one launch");
  const int sp = span_begin(c, TAG_STEP, stream, (long long)p.K * p.P);
  dasgd_status st;
  if (bf16) st = mom ? launch_step_m<true, true>(c, p, vec, merge, snap, stream) : launch_step_m<true, false>(c, p, vec, merge, snap, stream);
  else st = mom ? launch_step_m<false, true>(c, p, vec, merge, snap, stream) : launch_step_m<false, false>(c, p, vec, merge, snap, stream);
  span_end(c, sp, stream);
  return st;
}

dasgd_status launch_snapshot(dasgd_ctx *c, const Params &p) {
  if (!fits_one_launch(p)) return fail(c, DASGD_ERR_UNSUPPORTED, "K*P too large for one launch");
  const int sp = span_begin(c, TAG_SNAPSHOT, c->s0, (long long)p.K * p.P);
  long long done = 0;
  if (c->vec) {
    const long long units = p.P / 4;
    if (units > 0) {
      const long long tiles = (units + (long long)kThreads * 4 - 1) / ((long long)kThreads * 4);
      dasgd::k_snapshot_vec<<<(unsigned)(tiles * p.K), kThreads, 0, c->s0>>>(p);
      c->launches++;
    }
    done = units * 4;
  }
  if (done < p.P) {
    dim3 grid(blocks_for(p.P - done, kThreads), (unsigned)p.K);
    dasgd::k_snapshot_scalar<<<grid, kThreads, 0, c->s0>>>(p, done);
    c->launches++;
  }
  span_end(c, sp, c->s0);
  CU(c, cudaGetLastError());
  return DASGD_OK;
}

dasgd_status launch_reduce(dasgd_ctx *c, const Params &p, cudaStream_t side) {
  long long done = 0;
  if (c->vec) {
    const long long units = p.P / 4;
    if (units > 0) {
      // Shapes chosen by timing each kernel alone on B200 at P = 25.6M (fraction of the measured copy
      // bandwidth): two columns per thread, four rows per batch, three CTAs per SM: 0.97 at K = 8,
      // 1.02 at K = 16, 1.05 at K = 32; all rows in registers for K <= 4: 0.90 (K = 2) to 0.95 (K = 4).
      if (p.K > 4) dasgd::k_reduce_vec<2, 4, 3><<<blocks_for(units, kThreads * 2), kThreads, 0, side>>>(p);
      else if (p.K > 2) dasgd::k_reduce_small<2, 1><<<blocks_for(units, kThreads * 2), kThreads, 0, side>>>(p);
      else dasgd::k_reduce_small<4, 1><<<blocks_for(units, kThreads * 4), kThreads, 0, side>>>(p);
      c->launches++;
    }
    done = units * 4;
  }
  if (done < p.P) {
    dasgd::k_reduce_scalar<<<blocks_for(p.P - done, kThreads), kThreads, 0, side>>>(p, done);
    c->launches++;
  }
  CU(c, cudaGetLastError());
  return DASGD_OK;
}

// The worker-axis mean of the snapshot p.snap_in into p.mean_out, on the side stream.  With every worker
// in this context: one kernel.  With a sharded worker axis: the kernel writes the plain sum of this
// context's rows (no kernel when there is a single row: the row is its own sum), then the exchange adds
// the sums of all shards in place; the division by the total number of workers happens where the merge
// reads the result.
// `side`: the stream it runs on (the caller's side stream unless stated otherwise).
dasgd_status launch_mean(dasgd_ctx *c, Params p, cudaStream_t side = nullptr) {
  if (!side) side = c->s1;
  const int sp = span_begin(c, TAG_MEAN, side, (long long)p.K * p.P);
  dasgd_status st = DASGD_OK;
  if (c->K_total == 0) {
    st = launch_reduce(c, p, side);
  } else {
    const float *send = p.snap_in;
    if (p.K > 1) {
      p.sum_only = 1;
      st = launch_reduce(c, p, side);
      send = p.mean_out;
    }
    if (st == DASGD_OK) {
      st = c->exchange(c->exchange_user, send, p.mean_out, p.P, side);
      if (st != DASGD_OK) fail(c, st, "average: the exchange of the partial sums failed");
    }
  }
  span_end(c, sp, side);
  return st;
}

float *m_snap_ptr(const dasgd_ctx *c, int slot) { return c->m_snap + (size_t)slot * c->cfg.K * c->cfg.ld; }
float *m_mean_ptr(const dasgd_ctx *c, int slot) { return c->m_mean + (size_t)slot * c->cfg.ld; }

// Momentum averaging, step 1: the buffers as they are now, copied into the slot's array (main stream).
dasgd_status copy_momentum(dasgd_ctx *c, int slot) {
  Params p = base_params(c);
  p.w = p.m;
  p.snap_out = m_snap_ptr(c, slot);
  return launch_snapshot(c, p);
}

// Step 2: their worker-axis mean (side stream; the caller has ordered the side stream after the copy).
dasgd_status mean_momentum(dasgd_ctx *c, int slot) {
  Params p = base_params(c);
  p.snap_in = m_snap_ptr(c, slot);
  p.mean_out = m_mean_ptr(c, slot);
  return launch_mean(c, p);
}

template <bool BF16, int MODE, bool SNAP>
dasgd_status launch_merge_t(dasgd_ctx *c, const Params &p) {
  constexpr int EPU = BF16 ? 8 : 4;
  const int sp = span_begin(c, TAG_MERGE, c->s0, (long long)p.K * p.P);
  long long done = 0;
  if (c->vec) {
    const long long units = p.P / EPU;
    if (units > 0) {
      dasgd::k_merge_vec<BF16, MODE, SNAP><<<blocks_for(units, kThreads), kThreads, 0, c->s0>>>(p);
      c->launches++;
    }
    done = units * EPU;
  }
  if (done < p.P) {
    dasgd::k_merge_scalar<BF16, MODE, SNAP><<<blocks_for(p.P - done, kThreads), kThreads, 0, c->s0>>>(p, done);
    c->launches++;
  }
  span_end(c, sp, c->s0);
  CU(c, cudaGetLastError());
  return DASGD_OK;
}

dasgd_status launch_merge(dasgd_ctx *c, const Params &p, bool snap, bool plain_f32 = false) {
  const bool bf16 = c->cfg.dtype == DASGD_BF16_MASTER_F32 && !plain_f32;
  const bool delta = c->cfg.merge_mode == DASGD_MERGE_DELTA;
  if (bf16) {
    if (delta) return snap ? launch_merge_t<true, 2, true>(c, p) : launch_merge_t<true, 2, false>(c, p);
    return snap ? launch_merge_t<true, 1, true>(c, p) : launch_merge_t<true, 1, false>(c, p);
  }
  if (delta) return snap ? launch_merge_t<false, 2, true>(c, p) : launch_merge_t<false, 2, false>(c, p);
  return snap ? launch_merge_t<false, 1, true>(c, p) : launch_merge_t<false, 1, false>(c, p);
}

template <bool BF16, bool MOM, bool MERGE, bool MEANOUT>
dasgd_status launch_allk_t(dasgd_ctx *c, const Params &p, bool vec) {
  constexpr int EPU = BF16 ? 8 : 4;
  long long done = 0;
  if (vec) {
    const long long units = p.P / EPU;
    if (units > 0) {
      dasgd::k_step_allk_vec<BF16, MOM, MERGE, MEANOUT><<<blocks_for(units, kThreads), kThreads, 0, c->s0>>>(p);
      c->launches++;
    }
    done = units * EPU;
  }
  if (done < p.P) {
    dasgd::k_step_allk_scalar<BF16, MOM, MERGE, MEANOUT>
        <<<blocks_for(p.P - done, kThreads), kThreads, 0, c->s0>>>(p, done);
    c->launches++;
  }
  CU(c, cudaGetLastError());
  return DASGD_OK;
}

template <bool BF16, bool MOM>
dasgd_status launch_allk_m(dasgd_ctx *c, const Params &p, bool vec, bool merge, bool meanout) {
  if (merge) return meanout ? launch_allk_t<BF16, MOM, true, true>(c, p, vec) : launch_allk_t<BF16, MOM, true, false>(c, p, vec);
  return meanout ? launch_allk_t<BF16, MOM, false, true>(c, p, vec) : launch_allk_t<BF16, MOM, false, false>(c, p, vec);
}

dasgd_status launch_allk(dasgd_ctx *c, const Params &p, bool vec, bool merge, bool meanout) {
  const bool bf16 = c->cfg.dtype == DASGD_BF16_MASTER_F32;
  const bool mom = c->cfg.momentum != 0.0f;
  const int sp = span_begin(c, TAG_STEP, c->s0, (long long)p.K * p.P);
  dasgd_status st;
  if (bf16) st = mom ? launch_allk_m<true, true>(c, p, vec, merge, meanout) : launch_allk_m<true, false>(c, p, vec, merge, meanout);
  else st = mom ? launch_allk_m<false, true>(c, p, vec, merge, meanout) : launch_allk_m<false, false>(c, p, vec, merge, meanout);
  span_end(c, sp, c->s0);
  return st;
}

// -------------------------------------------------------------- slot operations

int find_free_slot(const dasgd_ctx *c) {
  for (size_t i = 0; i < c->slots.size(); ++i)
    if (c->slots[i].state == SLOT_FREE) return (int)i;
  return -1;
}

// An array that is neither the current weights nor a pending snapshot; `fallback` (or -1) otherwise.
int find_free_buf(const dasgd_ctx *c, int fallback) {
  for (size_t b = 0; b < c->pool.size(); ++b)
    if ((int)b != c->cur && c->frozen[b] == 0) return (int)b;
  return fallback;
}

// The snapshot array of `slot` if the kernel that merges that slot may overwrite it element by element
// (nobody else still needs it), else -1.
int reusable_buf(const dasgd_ctx *c, int slot) {
  const Slot &sl = c->slots[slot];
  if (sl.buf < 0) return -1;
  const int others = c->frozen[sl.buf] - (sl.holds ? 1 : 0);
  return others == 0 ? sl.buf : -1;
}

// Where the next kernel that writes weights must put them: in place unless the current array is a
// pending snapshot.  `reusable` is an array the same kernel is allowed to overwrite element by
// element after reading it (the snapshot of the slot it merges), or -1.
int pick_w_out(const dasgd_ctx *c, int reusable) {
  if (c->frozen[c->cur] == 0) return c->cur;
  return find_free_buf(c, reusable);
}

// book-keeping after the main stream has been given the work that completes the snapshot in pool[buf]
dasgd_status mark_snapped(dasgd_ctx *c, int slot, int buf) {
  Slot &sl = c->slots[slot];
  if (c->m_snap) {
    dasgd_status st = copy_momentum(c, slot);
    if (st != DASGD_OK) return st;
  }
  CU(c, cudaEventRecord(sl.e_snap, c->s0));
  sl.state = SLOT_SNAPPED;
  sl.chunked = false;
  sl.s = c->t;
  sl.buf = buf;
  c->frozen[buf] += 1;
  sl.holds = true;
  c->pending.push_back(slot);
  return DASGD_OK;
}

// make the main stream wait for the oldest pending average; returns its slot
dasgd_status wait_oldest_average(dasgd_ctx *c, int *slot_out) {
  if (c->pending.empty()) return fail(c, DASGD_ERR_BAD_STATE, "merge: no snapshot is pending");
  const int slot = c->pending.front();
  Slot &sl = c->slots[slot];
  if (sl.state != SLOT_AVERAGING)
    return fail(c, DASGD_ERR_BAD_STATE, "merge: the oldest snapshot has not been given to dasgd_average_async");
  if (sl.chunked) {  // the means of the ranges run in order on the side stream: the last one implies the rest
    const size_t last = sl.e_avg_c.size() - 1;
    stall_about_to_wait(c, sl.stall_sp_c[last], c->s0);
    CU(c, cudaStreamWaitEvent(c->s0, sl.e_avg_c[last], 0));
  } else {
    stall_about_to_wait(c, sl.stall_sp, c->s0);
    CU(c, cudaStreamWaitEvent(c->s0, sl.e_avg, 0));
  }
  // From here on the main stream is ordered after the mean kernel.  The xi-blend no longer needs
  // the snapshot itself, so its array may be overwritten by what the main stream does next.
  if (c->cfg.merge_mode == DASGD_MERGE_XI && sl.holds) {
    c->frozen[sl.buf] -= 1;
    sl.holds = false;
  }
  *slot_out = slot;
  return DASGD_OK;
}

// Momentum averaging, step 3: blend the slot's mean of the buffers into the buffers, on the main stream, after
// the kernels of this iteration that update them.  The same blend as for the weights; no bfloat16 copy exists.
dasgd_status merge_momentum(dasgd_ctx *c, int slot) {
  if (!c->m_snap) return DASGD_OK;
  Slot &sl = c->slots[slot];
  if (sl.chunked) CU(c, cudaStreamWaitEvent(c->s0, sl.e_mavg, 0));  // otherwise e_avg, already waited for, covers it
  Params p = base_params(c);
  p.w = p.m;
  p.w_out = p.m;
  p.w_lp = nullptr;
  p.mean = m_mean_ptr(c, slot);
  p.snap_in = m_snap_ptr(c, slot);
  return launch_merge(c, p, false, true);
}

void release_oldest(dasgd_ctx *c) {
  const int slot = c->pending.front();
  c->pending.pop_front();
  Slot &sl = c->slots[slot];
  if (sl.holds) {
    c->frozen[sl.buf] -= 1;
    sl.holds = false;
  }
  sl.state = SLOT_FREE;
}

void destroy_slot_events(Slot &sl) {
  if (sl.e_snap) cudaEventDestroy(sl.e_snap);
  if (sl.e_avg) cudaEventDestroy(sl.e_avg);
  for (cudaEvent_t e : sl.e_snap_c) if (e) cudaEventDestroy(e);
  for (cudaEvent_t e : sl.e_avg_c) if (e) cudaEventDestroy(e);
  if (sl.e_msnap) cudaEventDestroy(sl.e_msnap);
  if (sl.e_mavg) cudaEventDestroy(sl.e_mavg);
  sl.e_snap = sl.e_avg = sl.e_msnap = sl.e_mavg = nullptr;
  sl.e_snap_c.clear();
  sl.e_avg_c.clear();
}

bool merge_due(const dasgd_ctx *c, int64_t u) {
  const int64_t tau = c->cfg.tau, d = c->cfg.d;
  return d > 0 && u - d >= tau && (u - d) % tau == 0;
}

bool grads_vec_ok(const dasgd_ctx *c, const void *g) { return c->vec && aligned16(g); }

dasgd_status do_average(dasgd_ctx *c) {
  int slot = -1;
  for (int s : c->pending)
    if (c->slots[s].state == SLOT_SNAPPED) { slot = s; break; }
  if (slot < 0) return fail(c, DASGD_ERR_BAD_STATE, "average: no snapshot is waiting for its mean");
  Slot &sl = c->slots[slot];
  CU(c, cudaStreamWaitEvent(c->s1, sl.e_snap, 0));
  Params p = base_params(c);
  p.snap_in = snap_ptr(c, slot);
  p.mean_out = mean_ptr(c, slot);
  dasgd_status st = launch_mean(c, p);
  if (st != DASGD_OK) return st;
  if (c->m_snap) {
    st = mean_momentum(c, slot);
    if (st != DASGD_OK) return st;
  }
  CU(c, cudaEventRecord(sl.e_avg, c->s1));
  sl.stall_sp = stall_mean_done(c, sl.stall_sp);
  sl.state = SLOT_AVERAGING;
  return DASGD_OK;
}

}  // namespace

// ================================================================== C ABI

extern "C" {

const char *dasgd_version(void) { return "0.1"; }

const char *dasgd_strerror(dasgd_status s) {
  switch (s) {
    case DASGD_OK: return "ok";
    case DASGD_ERR_INVALID_ARG: return "invalid argument";
    case DASGD_ERR_BAD_STATE: return "call out of order";
    case DASGD_ERR_NO_SLOT: return "no free snapshot slot";
    case DASGD_ERR_CUDA: return "CUDA error";
    case DASGD_ERR_TIMEOUT: return "timed out";
    case DASGD_ERR_UNSUPPORTED: return "unsupported";
  }
  return "unknown status";
}

const char *dasgd_last_error(const dasgd_ctx *ctx) { return ctx ? ctx->err.c_str() : g_init_error.c_str(); }

dasgd_status dasgd_init(dasgd_ctx **out, const dasgd_config *cfg) {
  if (!out) return fail(nullptr, DASGD_ERR_INVALID_ARG, "init: out is NULL");
  *out = nullptr;
  if (!cfg) return fail(nullptr, DASGD_ERR_INVALID_ARG, "init: cfg is NULL");
  dasgd_config c = *cfg;
  if (c.ld == 0) c.ld = c.P;
  if (c.K < 1 || c.K > 65535) return fail(nullptr, DASGD_ERR_INVALID_ARG, "init: K must be in [1, 65535]");
  if (c.P < 1) return fail(nullptr, DASGD_ERR_INVALID_ARG, "init: P must be >= 1");
  if (c.ld < c.P) return fail(nullptr, DASGD_ERR_INVALID_ARG, "init: ld must be >= P");
  if (c.tau < 1) return fail(nullptr, DASGD_ERR_INVALID_ARG, "init: tau must be >= 1");
  if (c.d < 0) return fail(nullptr, DASGD_ERR_INVALID_ARG, "init: d must be >= 0");
  if (!(c.xi >= 0.0f && c.xi <= 1.0f)) return fail(nullptr, DASGD_ERR_INVALID_ARG, "init: xi must be in [0, 1]");
  if (!(c.momentum >= 0.0f) || !(c.weight_decay >= 0.0f))
    return fail(nullptr, DASGD_ERR_INVALID_ARG, "init: momentum and weight_decay must be >= 0");
  if (c.dtype != DASGD_F32 && c.dtype != DASGD_BF16_MASTER_F32)
    return fail(nullptr, DASGD_ERR_INVALID_ARG, "init: unknown dtype");
  if (c.merge_mode != DASGD_MERGE_XI && c.merge_mode != DASGD_MERGE_DELTA)
    return fail(nullptr, DASGD_ERR_INVALID_ARG, "init: unknown merge_mode");
  const int need = c.d == 0 ? 1 : (c.d + c.tau - 1) / c.tau;
  if (c.n_slots < need)
    return fail(nullptr, DASGD_ERR_INVALID_ARG, "init: n_slots must be >= max(1, ceil(d/tau))");
  if ((c.flags & DASGD_FLAG_NESTEROV) && c.momentum == 0.0f)
    return fail(nullptr, DASGD_ERR_INVALID_ARG, "init: DASGD_FLAG_NESTEROV needs momentum > 0");
  const bool inline_mean = (c.flags & DASGD_FLAG_INLINE_MEAN) != 0;
  if (inline_mean && c.merge_mode != DASGD_MERGE_XI)
    return fail(nullptr, DASGD_ERR_INVALID_ARG, "init: DASGD_FLAG_INLINE_MEAN supports the xi-blend merge only");
  if (!c.w || !c.mean || (!c.snap && !inline_mean))
    return fail(nullptr, DASGD_ERR_INVALID_ARG, "init: w, snap and mean must not be NULL");
  if (c.momentum != 0.0f && !c.m) return fail(nullptr, DASGD_ERR_INVALID_ARG, "init: momentum != 0 needs m");
  if (c.dtype == DASGD_BF16_MASTER_F32 && !c.w_lp)
    return fail(nullptr, DASGD_ERR_INVALID_ARG, "init: bf16 mode needs w_lp");
  const void *ptrs[] = {c.w, c.m, c.w_lp, c.snap, c.mean, c.g_stage};
  for (const void *p : ptrs)
    if (p && !aligned16(p)) return fail(nullptr, DASGD_ERR_INVALID_ARG, "init: device buffers must be 16-byte aligned");
  if (c.main_stream == c.side_stream)
    return fail(nullptr, DASGD_ERR_INVALID_ARG, "init: main_stream and side_stream must differ");
  if (c.sync_timeout_ms == 0) c.sync_timeout_ms = 60000;
  if (c.n_stage < 0 || c.n_stage > 2) return fail(nullptr, DASGD_ERR_INVALID_ARG, "init: n_stage must be 0, 1 or 2");
  if ((c.n_stage > 0) != (c.g_stage != nullptr))
    return fail(nullptr, DASGD_ERR_INVALID_ARG, "init: g_stage and n_stage must be given together");
  if (c.n_chunks < 0 || c.n_chunks > 1024) return fail(nullptr, DASGD_ERR_INVALID_ARG, "init: n_chunks must be in [0, 1024]");
  if (c.n_chunks > 1) {
    const uint32_t need_flags = DASGD_FLAG_ROTATE_SNAPSHOT | DASGD_FLAG_FUSE_MERGE;
    if ((c.flags & need_flags) != need_flags || inline_mean || c.d < 1)
      return fail(nullptr, DASGD_ERR_INVALID_ARG,
                  "init: n_chunks > 1 needs d >= 1, DASGD_FLAG_ROTATE_SNAPSHOT and DASGD_FLAG_FUSE_MERGE, and excludes "
                  "DASGD_FLAG_INLINE_MEAN");
  }

  int ndev = 0;
  cudaError_t e = cudaGetDeviceCount(&ndev);
  if (e != cudaSuccess) return cuda_fail(nullptr, e, "init: cudaGetDeviceCount");
  if (c.device < 0 || c.device >= ndev) return fail(nullptr, DASGD_ERR_INVALID_ARG, "init: no such CUDA device");
  for (const void *p : ptrs) {
    if (!p) continue;
    cudaPointerAttributes at{};
    e = cudaPointerGetAttributes(&at, p);
    if (e != cudaSuccess) {
      cudaGetLastError();
      return cuda_fail(nullptr, e, "init: cudaPointerGetAttributes");
    }
    if (at.type != cudaMemoryTypeDevice && at.type != cudaMemoryTypeManaged)
      return fail(nullptr, DASGD_ERR_INVALID_ARG, "init: w, m, w_lp, snap, mean and g_stage must be device memory");
    if (at.type == cudaMemoryTypeDevice && at.device != c.device)
      return fail(nullptr, DASGD_ERR_INVALID_ARG, "init: a device buffer does not live on cfg.device");
  }

  dasgd_ctx *ctx = new (std::nothrow) dasgd_ctx();
  if (!ctx) return fail(nullptr, DASGD_ERR_INVALID_ARG, "init: out of host memory");
  ctx->cfg = c;
  ctx->s0 = static_cast<cudaStream_t>(c.main_stream);
  ctx->s1 = static_cast<cudaStream_t>(c.side_stream);
  ctx->epu = c.dtype == DASGD_BF16_MASTER_F32 ? 8 : 4;
  ctx->vec = (c.ld % ctx->epu) == 0;
  ctx->rotate = (c.flags & DASGD_FLAG_ROTATE_SNAPSHOT) != 0;
  ctx->pool.push_back(static_cast<float *>(c.w));
  for (int i = 0; c.snap && i < c.n_slots; ++i)
    ctx->pool.push_back(static_cast<float *>(c.snap) + (size_t)i * c.K * c.ld);
  ctx->frozen.assign(ctx->pool.size(), 0);
  if (c.n_chunks > 1 && c.d >= 1) {
    const long long tile = 4096;     // columns per CTA of the vector step kernels, both dtypes
    const long long tiles = (c.P + tile - 1) / tile;
    const long long per = (tiles + c.n_chunks - 1) / c.n_chunks;
    ctx->chunk_cols = per * tile;
    ctx->chunks = (int)((c.P + ctx->chunk_cols - 1) / ctx->chunk_cols);
  }
  DeviceGuard guard(c.device);
  ctx->slots.resize(c.n_slots);
  for (Slot &sl : ctx->slots) {
    bool ok = (e = cudaEventCreateWithFlags(&sl.e_snap, cudaEventDisableTiming)) == cudaSuccess &&
              (e = cudaEventCreateWithFlags(&sl.e_avg, cudaEventDisableTiming)) == cudaSuccess;
    if (ok && ctx->chunks > 1) {
      sl.e_snap_c.assign(ctx->chunks, nullptr);
      sl.e_avg_c.assign(ctx->chunks, nullptr);
      sl.stall_sp_c.assign(ctx->chunks, -1);
      for (int i = 0; ok && i < ctx->chunks; ++i)
        ok = (e = cudaEventCreateWithFlags(&sl.e_snap_c[i], cudaEventDisableTiming)) == cudaSuccess &&
             (e = cudaEventCreateWithFlags(&sl.e_avg_c[i], cudaEventDisableTiming)) == cudaSuccess;
    }
    if (!ok) {
      dasgd_status st = cuda_fail(nullptr, e, "init: cudaEventCreate");
      for (Slot &z : ctx->slots) destroy_slot_events(z);
      delete ctx;
      return st;
    }
  }
  if (ctx->chunks > 1 && (c.flags & DASGD_FLAG_TWO_LANES)) {
    int prio = 0;
    const int extra = 1;  // two lanes; three and four were measured and bring nothing
    bool ok = cudaStreamGetPriority(ctx->s0, &prio) == cudaSuccess &&
              cudaEventCreateWithFlags(&ctx->e_fork, cudaEventDisableTiming) == cudaSuccess;
    for (int i = 0; ok && i < extra; ++i) {
      cudaStream_t st = nullptr;
      cudaEvent_t ev = nullptr;
      ok = cudaStreamCreateWithPriority(&st, cudaStreamNonBlocking, prio) == cudaSuccess &&
           cudaEventCreateWithFlags(&ev, cudaEventDisableTiming) == cudaSuccess;
      if (st) ctx->lanes.push_back(st);
      if (ev) ctx->e_joins.push_back(ev);
    }
    if (!ok) {
      cudaGetLastError();
      dasgd_destroy(ctx);
      return fail(nullptr, DASGD_ERR_CUDA, "init: cannot create the second lane's stream and events");
    }
  }
  if (ctx->chunks > 1 && (c.flags & DASGD_FLAG_TWO_SIDE_STREAMS)) {
    int prio = 0;
    const bool ok = cudaStreamGetPriority(ctx->s1, &prio) == cudaSuccess &&
                    cudaStreamCreateWithPriority(&ctx->s1b, cudaStreamNonBlocking, prio) == cudaSuccess &&
                    cudaEventCreateWithFlags(&ctx->e_cross, cudaEventDisableTiming) == cudaSuccess;
    if (!ok) {
      cudaGetLastError();
      dasgd_destroy(ctx);
      return fail(nullptr, DASGD_ERR_CUDA, "init: cannot create the second side stream");
    }
  }
  if (ctx->chunks > 1 && (c.flags & DASGD_FLAG_GRAPH)) {
    bool ok = cudaMalloc(&ctx->dyn_dev, sizeof(dasgd::DynArgs)) == cudaSuccess;
    const size_t n_ev = (size_t)ctx->chunks + ctx->lanes.size() + 2;
    for (size_t i = 0; ok && i < n_ev; ++i) {
      cudaEvent_t ev = nullptr;
      ok = cudaEventCreateWithFlags(&ev, cudaEventDisableTiming) == cudaSuccess;
      if (ev) ctx->cap_ev.push_back(ev);
    }
    if (!ok) {
      cudaGetLastError();
      dasgd_destroy(ctx);
      return fail(nullptr, DASGD_ERR_CUDA, "init: cannot create the replay's device block and events");
    }
    ctx->use_graph = true;
  }
  if (c.n_stage > 0) {
    bool ok = cudaStreamCreateWithFlags(&ctx->s_copy, cudaStreamNonBlocking) == cudaSuccess;
    ctx->e_copied.assign(c.n_stage, nullptr);
    ctx->e_consumed.assign(c.n_stage, nullptr);
    ctx->stage_used.assign(c.n_stage, false);
    for (int i = 0; ok && i < c.n_stage; ++i)
      ok = cudaEventCreateWithFlags(&ctx->e_copied[i], cudaEventDisableTiming) == cudaSuccess &&
           cudaEventCreateWithFlags(&ctx->e_consumed[i], cudaEventDisableTiming) == cudaSuccess;
    if (!ok) {
      dasgd_destroy(ctx);
      return fail(nullptr, DASGD_ERR_CUDA, "init: cannot create the staging stream and events");
    }
  }
  *out = ctx;
  return DASGD_OK;
}

dasgd_status dasgd_destroy(dasgd_ctx *ctx) {
  if (!ctx) return DASGD_ERR_INVALID_ARG;
  DeviceGuard guard(ctx->cfg.device);
  cudaStreamSynchronize(ctx->s0);
  cudaStreamSynchronize(ctx->s1);
  for (Slot &sl : ctx->slots) destroy_slot_events(sl);
  for (Span &sp : ctx->spans)
    for (int j = 0; j < 2; ++j)
      if (sp.ev[j]) cudaEventDestroy(sp.ev[j]);
  if (ctx->s_copy) {
    cudaStreamSynchronize(ctx->s_copy);
    cudaStreamDestroy(ctx->s_copy);
  }
  for (cudaStream_t st : ctx->lanes) {
    cudaStreamSynchronize(st);
    cudaStreamDestroy(st);
  }
  if (ctx->s1b) {
    cudaStreamSynchronize(ctx->s1b);
    cudaStreamDestroy(ctx->s1b);
  }
  if (ctx->e_cross) cudaEventDestroy(ctx->e_cross);
  for (cudaEvent_t ev : ctx->e_joins) cudaEventDestroy(ev);
  for (GraphEntry &g : ctx->graphs) if (g.exec) cudaGraphExecDestroy(g.exec);
  for (cudaEvent_t ev : ctx->cap_ev) cudaEventDestroy(ev);
  if (ctx->dyn_dev) cudaFree(ctx->dyn_dev);
  if (ctx->e_fork) cudaEventDestroy(ctx->e_fork);
  for (cudaEvent_t e : ctx->e_copied) if (e) cudaEventDestroy(e);
  for (cudaEvent_t e : ctx->e_consumed) if (e) cudaEventDestroy(e);
  delete ctx;
  return DASGD_OK;
}

// ---- the four operations, on the pool of weight arrays -------------------------------------------

namespace {

// Local step, optionally with the merge of `merge_slot` (-1: none) folded in and, in copy mode,
// the snapshot stored into pool[snap_buf] (-1: none).
dasgd_status op_step(dasgd_ctx *c, const void *grads, float lr, int merge_slot, int snap_buf) {
  Params p = base_params(c);
  p.g = grads;
  p.lr = lr;
  int reusable = -1;
  if (merge_slot >= 0) {
    p.mean = mean_ptr(c, merge_slot);
    p.snap_in = snap_ptr(c, merge_slot);
    reusable = reusable_buf(c, merge_slot);
    // One launch over the whole array: walk the rows in runs of 512 tiles (8 MB per array), so that the CTAs in
    // flight stream a few long runs instead of K times as many short ones, while the 8 MB of the mean a group
    // blends with stay in L2 for its K passes.  Measured alone, float32: 6.60 -> 6.78 TB/s at K = 8, 6.65 -> 6.90
    // at K = 32; groups of 128 or 2048 tiles gain less or nothing.  (Column ranges of the pipeline keep 1.)
    p.group_tiles = 512;
  }
  const int out = pick_w_out(c, reusable);
  if (out < 0) return fail(c, DASGD_ERR_NO_SLOT, "step: no free weight array to write into");
  p.w_out = c->pool[out];
  if (snap_buf >= 0) p.snap_out = c->pool[snap_buf];
  const int mode = merge_slot < 0 ? 0 : (c->cfg.merge_mode == DASGD_MERGE_DELTA ? 2 : 1);
  dasgd_status st = launch_step(c, p, grads_vec_ok(c, grads), mode, snap_buf >= 0, c->s0);
  if (st != DASGD_OK) return st;
  c->cur = out;
  c->t += 1;
  return DASGD_OK;
}

// Stand-alone merge of `slot` (already waited for), optionally storing the snapshot into pool[snap_buf].
dasgd_status op_merge(dasgd_ctx *c, int slot, int snap_buf) {
  Params p = base_params(c);
  p.mean = mean_ptr(c, slot);
  p.snap_in = snap_ptr(c, slot);
  const int out = pick_w_out(c, reusable_buf(c, slot));
  if (out < 0) return fail(c, DASGD_ERR_NO_SLOT, "merge: no free weight array to write into");
  p.w_out = c->pool[out];
  if (snap_buf >= 0) p.snap_out = c->pool[snap_buf];
  dasgd_status st = launch_merge(c, p, snap_buf >= 0);
  if (st != DASGD_OK) return st;
  c->cur = out;
  return DASGD_OK;
}

// Snapshot of the current weights.  Rotate mode: no kernel, the current array is frozen.  Copy mode:
// `already_in` >= 0 says a fused kernel has stored the copy into pool[already_in]; otherwise copy now.
dasgd_status op_snapshot(dasgd_ctx *c, int already_in) {
  const int slot = find_free_slot(c);
  if (slot < 0) return fail(c, DASGD_ERR_NO_SLOT, "snapshot: every slot holds a pending average");
  if (c->pool.size() < 2) return fail(c, DASGD_ERR_BAD_STATE, "snapshot: no snapshot arrays were configured (cfg.snap)");
  if (c->rotate) return mark_snapped(c, slot, c->cur);
  int buf = already_in;
  if (buf < 0) {
    buf = find_free_buf(c, -1);
    if (buf < 0) return fail(c, DASGD_ERR_NO_SLOT, "snapshot: no free snapshot array");
    Params p = base_params(c);
    p.snap_out = c->pool[buf];
    dasgd_status st = launch_snapshot(c, p);
    if (st != DASGD_OK) return st;
  }
  return mark_snapped(c, slot, buf);
}

// One iteration of the inline-mean schedule: everything on the main stream, one kernel (two when
// d == 0, because the blend then needs the mean of the very weights this kernel produces).
dasgd_status step_inline(dasgd_ctx *c, const void *grads, float lr, bool m_due, bool s_due) {
  if (c->frozen[c->cur] > 0)
    return fail(c, DASGD_ERR_BAD_STATE, "step: a snapshot taken with dasgd_snapshot is pending; merge it first");
  Params p = base_params(c);
  p.g = grads;
  p.lr = lr;
  if (m_due) {
    if (c->pending.empty()) return fail(c, DASGD_ERR_BAD_STATE, "step: no mean is pending");
    const int ms = c->pending.front();
    if (c->slots[ms].state != SLOT_AVERAGING)
      return fail(c, DASGD_ERR_BAD_STATE, "step: the oldest snapshot has no mean yet");
    if (c->slots[ms].buf >= 0) {  // it came from dasgd_snapshot/dasgd_average_async: order after the side stream
      stall_about_to_wait(c, c->slots[ms].stall_sp, c->s0);
      CU(c, cudaStreamWaitEvent(c->s0, c->slots[ms].e_avg, 0));
    }
    p.mean = mean_ptr(c, ms);
    release_oldest(c);  // its mean is read by this iteration's kernel; the slot may be refilled by it
  }
  int slot = -1;
  if (s_due) {
    slot = find_free_slot(c);
    if (slot < 0) return fail(c, DASGD_ERR_NO_SLOT, "step: no free slot for the mean");
    p.mean_out = mean_ptr(c, slot);
  }
  dasgd_status st = launch_allk(c, p, grads_vec_ok(c, grads), m_due, s_due);
  if (st != DASGD_OK) return st;
  c->t += 1;
  if (s_due) {
    Slot &sl = c->slots[slot];
    sl.state = SLOT_AVERAGING;  // the mean is already on its way, on this same stream
    sl.s = c->t;
    sl.buf = -1;                // no snapshot array belongs to it
    sl.holds = false;
    c->pending.push_back(slot);
    if (c->cfg.d == 0) {        // Local SGD: blend it back at once
      Params q = base_params(c);
      q.mean = mean_ptr(c, slot);
      st = launch_merge(c, q, false);
      if (st != DASGD_OK) return st;
      release_oldest(c);
    }
  }
  return DASGD_OK;
}

// One iteration of the chunked pipeline (d >= 1, rotating snapshots, merge folded into the step kernel).
// Per column range i, on the main stream: wait for range i of the mean that lands (computed one
// iteration ago, so normally long finished), run the step kernel on range i; if a snapshot is due,
// record "range i written" and let the side stream average range i of the new weights while the main
// stream goes on with ranges i+1, ...  With d == 1 the mean of range i thus has the rest of this iteration
// and the first i ranges of the next one as its window (the condition t_c < d*t_p of Eq. 6, per range),
// although the next iteration's kernels consume it directly.  With d >= 2 the window is there anyway; what
// the pipeline still buys is that the mean of a range reads weights that were written a moment ago and
// are largely still in L2.
// The launches of one chunked iteration, enqueued on the main stream, the extra lanes and the side stream.
// Used while a stream capture is active; `ev` are capture-only events.
dasgd_status enqueue_chunked(dasgd_ctx *c, const Params &p, const Params &q, int mode, bool vec, bool s_due) {
  const int n_lanes = 1 + (int)c->lanes.size();
  cudaEvent_t *ev_chunk = c->cap_ev.data();
  cudaEvent_t *ev_lane = ev_chunk + c->chunks;
  cudaEvent_t ev_fork = ev_lane[c->lanes.size()], ev_side = ev_lane[c->lanes.size() + 1];
  CU(c, cudaEventRecord(ev_fork, c->s0));
  for (cudaStream_t st : c->lanes) CU(c, cudaStreamWaitEvent(st, ev_fork, 0));
  for (int i = 0; i < c->chunks; ++i) {
    const long long col0 = (long long)i * c->chunk_cols;
    const long long len = c->cfg.P - col0 < c->chunk_cols ? c->cfg.P - col0 : c->chunk_cols;
    cudaStream_t lane = (i % n_lanes) ? c->lanes[i % n_lanes - 1] : c->s0;
    dasgd_status st = launch_step(c, columns(c, p, col0, len), vec, mode, false, lane);
    if (st != DASGD_OK) return st;
    if (s_due) {
      CU(c, cudaEventRecord(ev_chunk[i], lane));
      CU(c, cudaStreamWaitEvent(c->s1, ev_chunk[i], 0));
      st = launch_mean(c, columns(c, q, col0, len));
      if (st != DASGD_OK) return st;
    }
  }
  for (size_t j = 0; j < c->lanes.size(); ++j) {
    CU(c, cudaEventRecord(ev_lane[j], c->lanes[j]));
    CU(c, cudaStreamWaitEvent(c->s0, ev_lane[j], 0));
  }
  if (s_due) {
    CU(c, cudaEventRecord(ev_side, c->s1));
    CU(c, cudaStreamWaitEvent(c->s0, ev_side, 0));
  }
  return DASGD_OK;
}

// One chunked iteration as the replay of a recorded CUDA graph (recorded on first use of a combination of
// arrays and switches).  The recording holds the step kernels on the lanes and the means on the side stream
// with the same dependencies as the direct launches; gradients pointer and learning rate are read from
// device memory, written by a one-thread kernel just before the replay.  If recording fails, replay is
// switched off for this context (c->use_graph = false) and the caller launches directly.
dasgd_status replay_chunked(dasgd_ctx *c, Params p, const Params &q, const void *grads, float lr, int mode, bool vec,
                            bool m_due, bool s_due, bool per_chunk_wait, int ms) {
  if (m_due && per_chunk_wait)  // the mean that lands was made by direct launches: order after all of it
    CU(c, cudaStreamWaitEvent(c->s0, c->slots[ms].e_avg_c.back(), 0));
  p.g = nullptr;
  p.dyn = c->dyn_dev;
  p.g_off = 0;
  GraphKey key{p.w, p.w_out, p.mean, p.snap_in, q.snap_in, q.mean_out, mode, vec ? 1 : 0, s_due ? 1 : 0, p.keep_w};
  GraphEntry *entry = nullptr;
  for (GraphEntry &g : c->graphs)
    if (g.key == key) { entry = &g; break; }
  if (!entry) {
    const int64_t launches_before = c->launches;
    cudaGraph_t graph = nullptr;
    cudaError_t e = cudaStreamBeginCapture(c->s0, cudaStreamCaptureModeRelaxed);
    dasgd_status st = e == cudaSuccess ? enqueue_chunked(c, p, q, mode, vec, s_due) : DASGD_ERR_CUDA;
    if (e == cudaSuccess) {
      e = cudaStreamEndCapture(c->s0, &graph);  // always ends the capture, also after a failed launch
      if (st == DASGD_OK && e != cudaSuccess) st = DASGD_ERR_CUDA;
    }
    cudaGraphExec_t exec = nullptr;
    if (st == DASGD_OK && cudaGraphInstantiate(&exec, graph, 0) != cudaSuccess) st = DASGD_ERR_CUDA;
    if (graph) cudaGraphDestroy(graph);
    const int64_t kernels = c->launches - launches_before;
    c->launches = launches_before;
    if (st != DASGD_OK) {
      cudaGetLastError();
      c->use_graph = false;
      return DASGD_OK;
    }
    if (c->graphs.size() >= 64) {  // the combinations of a run are few; a long list means something cycles
      cudaGraphExecDestroy(c->graphs.front().exec);
      c->graphs.erase(c->graphs.begin());
    }
    GraphEntry ge;
    ge.key = key;
    ge.exec = exec;
    ge.kernels = kernels;
    c->graphs.push_back(ge);
    entry = &c->graphs.back();
  }
  dasgd::k_set_dyn<<<1, 1, 0, c->s0>>>(c->dyn_dev, grads, lr);
  CU(c, cudaGetLastError());
  CU(c, cudaGraphLaunch(entry->exec, c->s0));
  c->launches += entry->kernels + 1;
  return DASGD_OK;
}

dasgd_status step_chunked(dasgd_ctx *c, const void *grads, float lr, bool m_due, bool s_due) {
  Params p = base_params(c);
  p.g = grads;
  p.lr = lr;
  int ms = -1, ns = -1, reusable = -1;
  bool per_chunk_wait = false;
  if (m_due) {
    if (c->pending.empty()) return fail(c, DASGD_ERR_BAD_STATE, "step: no snapshot is pending for the merge that is due");
    ms = c->pending.front();
    if (c->slots[ms].state != SLOT_AVERAGING)
      return fail(c, DASGD_ERR_BAD_STATE, "step: the oldest snapshot has not been given to dasgd_average_async");
  }
  if (s_due) {
    ns = find_free_slot(c);
    if (ns < 0 && m_due) ns = ms;  // the slot whose mean this iteration consumes is refilled by it
    if (ns < 0) return fail(c, DASGD_ERR_NO_SLOT, "step: every slot holds a pending average");
  }
  if (m_due) {
    Slot &sl = c->slots[ms];
    per_chunk_wait = sl.chunked;
    if (!per_chunk_wait) {  // its mean came from dasgd_average_async: one event for the whole vector
      stall_about_to_wait(c, sl.stall_sp, c->s0);
      CU(c, cudaStreamWaitEvent(c->s0, sl.e_avg, 0));
    }
    // Every kernel below that touches range i is ordered after the mean of range i, so the xi-blend no
    // longer needs the snapshot array: it may be overwritten range by range.
    if (c->cfg.merge_mode == DASGD_MERGE_XI && sl.holds) {
      c->frozen[sl.buf] -= 1;
      sl.holds = false;
    }
    p.mean = mean_ptr(c, ms);
    p.snap_in = snap_ptr(c, ms);
    reusable = reusable_buf(c, ms);
  }
  const int out = pick_w_out(c, reusable);
  if (out < 0) return fail(c, DASGD_ERR_NO_SLOT, "step: no free weight array to write into");
  p.w_out = c->pool[out];
  Params q = base_params(c);  // the mean of the new snapshot = the array this iteration writes
  if (s_due) {
    q.snap_in = c->pool[out];
    q.mean_out = mean_ptr(c, ns);
  }
  const int mode = !m_due ? 0 : (c->cfg.merge_mode == DASGD_MERGE_DELTA ? 2 : 1);
  const bool vec = grads_vec_ok(c, grads);
  // The mean of a range reads the weights its step kernel has just written: store them with the default
  // cache policy so that part of them is still in L2 then (everything else streams through).
  p.keep_w = s_due ? 1 : 0;
  if (c->use_graph && !(c->cfg.flags & DASGD_FLAG_TIMING) && c->K_total == 0 && !c->m_snap) {
    dasgd_status gst = replay_chunked(c, p, q, grads, lr, mode, vec, m_due, s_due, per_chunk_wait, ms);
    if (gst != DASGD_OK) return gst;
    if (c->use_graph) {  // replayed (a failed capture switches replay off and falls through to direct launches)
      c->cur = out;
      c->t += 1;
      if (m_due) release_oldest(c);
      if (s_due) {
        Slot &sl = c->slots[ns];
        CU(c, cudaEventRecord(sl.e_avg, c->s0));  // the replay is complete on the main stream: so is the mean
        sl.state = SLOT_AVERAGING;
        sl.chunked = false;
        sl.s = c->t;
        sl.buf = out;
        c->frozen[out] += 1;
        sl.holds = true;
        c->pending.push_back(ns);
      }
      return DASGD_OK;
    }
  }
  const int n_lanes = 1 + (int)c->lanes.size();
  if (n_lanes > 1) {  // fork: the other lanes start after everything the main stream holds so far
    CU(c, cudaEventRecord(c->e_fork, c->s0));
    for (cudaStream_t st : c->lanes) CU(c, cudaStreamWaitEvent(st, c->e_fork, 0));
  }
  // "Mean of range i complete" is signalled per group of G consecutive ranges (an event after the last mean of
  // the group: the side stream runs them in order), and a lane waits once per group it enters.  A range thus
  // waits for the means of up to G-1 later ranges of the previous iteration, all of which were started at least
  // C-G ranges ago; with G = C/8 that costs nothing and saves most of the event calls.
  const int C = c->chunks;
  const int G = C >= 16 ? C / 8 : 1;
  auto group_end = [&](int i) { const int e = (i / G + 1) * G - 1; return e < C - 1 ? e : C - 1; };
  std::vector<int> waited(n_lanes, -1);
  // An iteration that only merges (no snapshot follows it) has no mean to feed, so the ranges of a group go
  // out as one launch: the group is the granularity of the waits anyway.
  const int stride = s_due ? 1 : G;
  // Two side streams only with every worker here: the exchange of a sharded worker axis is a collective, and the
  // ranks must issue those in one order on one stream.
  const bool two_sides = c->s1b != nullptr && c->K_total == 0;
  for (int i = 0; i < C; i += stride) {
    const int last = i + stride - 1 < C - 1 ? i + stride - 1 : C - 1;   // last range of this launch
    const long long col0 = (long long)i * c->chunk_cols;
    const long long col1 = (long long)(last + 1) * c->chunk_cols < c->cfg.P ? (long long)(last + 1) * c->chunk_cols : c->cfg.P;
    const long long len = col1 - col0;
    const int li = (i / stride) % n_lanes;
    cudaStream_t lane = li ? c->lanes[li - 1] : c->s0;
    if (per_chunk_wait && waited[li] < group_end(last)) {
      const int e = group_end(last);
      stall_about_to_wait(c, c->slots[ms].stall_sp_c[e], lane);
      CU(c, cudaStreamWaitEvent(lane, c->slots[ms].e_avg_c[e], 0));
      waited[li] = e;
    }
    dasgd_status st = launch_step(c, columns(c, p, col0, len), vec, mode, false, lane);
    if (st != DASGD_OK) return st;
    if (s_due) {
      Slot &sl = c->slots[ns];
      cudaStream_t side = (two_sides && (i & 1)) ? c->s1b : c->s1;
      CU(c, cudaEventRecord(sl.e_snap_c[i], lane));
      CU(c, cudaStreamWaitEvent(side, sl.e_snap_c[i], 0));
      st = launch_mean(c, columns(c, q, col0, len), side);
      if (st != DASGD_OK) return st;
      if (i == group_end(i)) {
        if (two_sides) {  // "mean of range i complete" must imply the earlier ranges on the other side stream too
          cudaStream_t other = (i & 1) ? c->s1 : c->s1b;
          CU(c, cudaEventRecord(c->e_cross, other));
          CU(c, cudaStreamWaitEvent(side, c->e_cross, 0));
        }
        CU(c, cudaEventRecord(sl.e_avg_c[i], side));
        sl.stall_sp_c[i] = stall_mean_done(c, sl.stall_sp_c[i], side);
      }
    }
  }
  if (two_sides && s_due) {  // the caller's side stream again comes after everything this iteration averaged
    CU(c, cudaEventRecord(c->e_cross, c->s1b));
    CU(c, cudaStreamWaitEvent(c->s1, c->e_cross, 0));
  }
  if (c->use_graph && (c->cfg.flags & DASGD_FLAG_TIMING) && c->K_total == 0 && !c->m_snap && s_due) {
    // Timing pass of the replayed schedule: a replay ends only when its last mean is complete, so the
    // main stream waits for it here as well (and that wait is accounted as stall like any other).
    Slot &sl = c->slots[ns];
    stall_about_to_wait(c, sl.stall_sp_c[c->chunks - 1], c->s0);
    CU(c, cudaStreamWaitEvent(c->s0, sl.e_avg_c[c->chunks - 1], 0));
  }
  for (size_t j = 0; j < c->lanes.size(); ++j) {  // join: what the caller puts on the main stream next comes after all lanes
    CU(c, cudaEventRecord(c->e_joins[j], c->lanes[j]));
    CU(c, cudaStreamWaitEvent(c->s0, c->e_joins[j], 0));
  }
  if (c->m_snap) {  // momentum averaging: whole-array kernels after the ranges, merge before snapshot as for the weights
    if (m_due) {
      dasgd_status st = merge_momentum(c, ms);
      if (st != DASGD_OK) return st;
    }
    if (s_due) {
      Slot &sl = c->slots[ns];
      dasgd_status st = copy_momentum(c, ns);
      if (st != DASGD_OK) return st;
      CU(c, cudaEventRecord(sl.e_msnap, c->s0));
      CU(c, cudaStreamWaitEvent(c->s1, sl.e_msnap, 0));
      st = mean_momentum(c, ns);
      if (st != DASGD_OK) return st;
      CU(c, cudaEventRecord(sl.e_mavg, c->s1));
    }
  }
  c->cur = out;
  c->t += 1;
  if (m_due) release_oldest(c);
  if (s_due) {
    Slot &sl = c->slots[ns];
    sl.state = SLOT_AVERAGING;
    sl.chunked = true;
    sl.s = c->t;
    sl.buf = out;
    c->frozen[out] += 1;
    sl.holds = true;
    c->pending.push_back(ns);
  }
  return DASGD_OK;
}

}  // namespace

dasgd_status dasgd_local_step(dasgd_ctx *ctx, const void *grads, float lr) {
  if (!ctx) return DASGD_ERR_INVALID_ARG;
  if (!grads) return fail(ctx, DASGD_ERR_INVALID_ARG, "local_step: grads is NULL");
  DeviceGuard guard(ctx->cfg.device);
  return op_step(ctx, grads, lr, -1, -1);
}

dasgd_status dasgd_snapshot(dasgd_ctx *ctx) {
  if (!ctx) return DASGD_ERR_INVALID_ARG;
  DeviceGuard guard(ctx->cfg.device);
  return op_snapshot(ctx, -1);
}

dasgd_status dasgd_average_async(dasgd_ctx *ctx) {
  if (!ctx) return DASGD_ERR_INVALID_ARG;
  DeviceGuard guard(ctx->cfg.device);
  return do_average(ctx);
}

dasgd_status dasgd_merge(dasgd_ctx *ctx) {
  if (!ctx) return DASGD_ERR_INVALID_ARG;
  DeviceGuard guard(ctx->cfg.device);
  int slot = -1;
  dasgd_status st = wait_oldest_average(ctx, &slot);
  if (st != DASGD_OK) return st;
  st = op_merge(ctx, slot, -1);
  if (st != DASGD_OK) return st;
  st = merge_momentum(ctx, slot);
  if (st != DASGD_OK) return st;
  release_oldest(ctx);
  return DASGD_OK;
}

dasgd_status dasgd_step(dasgd_ctx *ctx, const void *grads, float lr) {
  if (!ctx) return DASGD_ERR_INVALID_ARG;
  if (!grads) return fail(ctx, DASGD_ERR_INVALID_ARG, "step: grads is NULL");
  DeviceGuard guard(ctx->cfg.device);
  const dasgd_config &cfg = ctx->cfg;
  const int64_t u = ctx->t + 1;
  const bool m_due = merge_due(ctx, u);
  const bool s_due = (u % cfg.tau) == 0;
  if (cfg.flags & DASGD_FLAG_INLINE_MEAN) return step_inline(ctx, grads, lr, m_due, s_due);
  if (ctx->chunks > 1 && (m_due || s_due)) return step_chunked(ctx, grads, lr, m_due, s_due);
  const bool fuse_merge = m_due && (cfg.flags & DASGD_FLAG_FUSE_MERGE) &&
                          (cfg.d >= 2 || (cfg.d == 1 && (cfg.flags & DASGD_FLAG_FUSE_MERGE_D1)));
  // copy mode only: let the kernel that last writes w in this iteration also store the snapshot
  const bool fuse_snap = s_due && !ctx->rotate && (cfg.flags & DASGD_FLAG_FUSE_SNAPSHOT);
  dasgd_status st;
  int stored_in = -1;  // array a fused kernel has stored this iteration's snapshot into

  // ---- local step (optionally with the merge and/or the snapshot store folded in)
  int merge_slot = -1;
  if (fuse_merge) {
    st = wait_oldest_average(ctx, &merge_slot);
    if (st != DASGD_OK) return st;
  }
  if (fuse_snap && (!m_due || fuse_merge)) {
    // A kernel that merges a slot may store the new snapshot over that slot's old one: each thread
    // reads the old element before it writes the new one.
    stored_in = find_free_buf(ctx, merge_slot >= 0 ? reusable_buf(ctx, merge_slot) : -1);
    if (stored_in < 0) return fail(ctx, DASGD_ERR_NO_SLOT, "step: no free snapshot array");
  }
  st = op_step(ctx, grads, lr, merge_slot, stored_in);
  if (st != DASGD_OK) return st;
  if (fuse_merge) {
    st = merge_momentum(ctx, merge_slot);
    if (st != DASGD_OK) return st;
    release_oldest(ctx);
  }

  // ---- separate merge kernel (d == 1, or fusion off), optionally storing the snapshot
  if (m_due && !fuse_merge) {
    st = wait_oldest_average(ctx, &merge_slot);
    if (st != DASGD_OK) return st;
    if (fuse_snap) {
      stored_in = find_free_buf(ctx, reusable_buf(ctx, merge_slot));
      if (stored_in < 0) return fail(ctx, DASGD_ERR_NO_SLOT, "step: no free snapshot array");
    }
    st = op_merge(ctx, merge_slot, stored_in);
    if (st != DASGD_OK) return st;
    st = merge_momentum(ctx, merge_slot);
    if (st != DASGD_OK) return st;
    release_oldest(ctx);
  }

  // ---- snapshot and its mean
  if (s_due) {
    st = op_snapshot(ctx, stored_in);
    if (st != DASGD_OK) return st;
    st = do_average(ctx);
    if (st != DASGD_OK) return st;
    if (cfg.d == 0) {  // Local SGD: the mean is applied in the same iteration
      int slot = -1;
      st = wait_oldest_average(ctx, &slot);
      if (st != DASGD_OK) return st;
      st = op_merge(ctx, slot, -1);
      if (st != DASGD_OK) return st;
      st = merge_momentum(ctx, slot);
      if (st != DASGD_OK) return st;
      release_oldest(ctx);
    }
  }
  return DASGD_OK;
}

dasgd_status dasgd_step_host(dasgd_ctx *ctx, const void *grads_host, float lr, float *probe_host,
                             int64_t probe_elems) {
  if (!ctx) return DASGD_ERR_INVALID_ARG;
  if (!grads_host) return fail(ctx, DASGD_ERR_INVALID_ARG, "step_host: grads_host is NULL");
  if (!ctx->cfg.g_stage || ctx->cfg.n_stage < 1)
    return fail(ctx, DASGD_ERR_BAD_STATE, "step_host: no gradient staging configured (g_stage, n_stage)");
  if (probe_host && (probe_elems < 0 || probe_elems > ctx->cfg.P))
    return fail(ctx, DASGD_ERR_INVALID_ARG, "step_host: probe_elems must be in [0, P]");
  DeviceGuard guard(ctx->cfg.device);
  const size_t esz = ctx->cfg.dtype == DASGD_BF16_MASTER_F32 ? 2 : 4;
  const size_t bytes = (size_t)ctx->cfg.K * ctx->cfg.ld * esz;
  const int i = (int)(ctx->host_calls % ctx->cfg.n_stage);
  char *stage = static_cast<char *>(ctx->cfg.g_stage) + (size_t)i * bytes;
  // the staging array may be overwritten only after the kernels of its previous use have run
  if (ctx->stage_used[i]) CU(ctx, cudaStreamWaitEvent(ctx->s_copy, ctx->e_consumed[i], 0));
  CU(ctx, cudaMemcpyAsync(stage, grads_host, bytes, cudaMemcpyHostToDevice, ctx->s_copy));
  CU(ctx, cudaEventRecord(ctx->e_copied[i], ctx->s_copy));
  CU(ctx, cudaStreamWaitEvent(ctx->s0, ctx->e_copied[i], 0));
  dasgd_status st = dasgd_step(ctx, stage, lr);
  if (st != DASGD_OK) return st;
  CU(ctx, cudaEventRecord(ctx->e_consumed[i], ctx->s0));
  ctx->stage_used[i] = true;
  ctx->host_calls += 1;
  if (probe_host && probe_elems > 0)
    CU(ctx, cudaMemcpyAsync(probe_host, ctx->pool[ctx->cur], (size_t)probe_elems * sizeof(float),
                            cudaMemcpyDeviceToHost, ctx->s0));
  return DASGD_OK;
}

dasgd_status dasgd_sync(dasgd_ctx *ctx) {
  if (!ctx) return DASGD_ERR_INVALID_ARG;
  DeviceGuard guard(ctx->cfg.device);
  const auto deadline = std::chrono::steady_clock::now() + std::chrono::milliseconds(ctx->cfg.sync_timeout_ms);
  std::vector<cudaStream_t> streams = {ctx->s0, ctx->s1};
  if (ctx->s1b) streams.push_back(ctx->s1b);
  if (ctx->s_copy) streams.push_back(ctx->s_copy);
  for (cudaStream_t st : ctx->lanes) streams.push_back(st);
  for (cudaStream_t s : streams) {
    for (;;) {
      cudaError_t e = cudaStreamQuery(s);
      if (e == cudaSuccess) break;
      if (e != cudaErrorNotReady) return cuda_fail(ctx, e, "sync: cudaStreamQuery");
      if (std::chrono::steady_clock::now() > deadline)
        return fail(ctx, DASGD_ERR_TIMEOUT, "sync: streams still busy after sync_timeout_ms");
      std::this_thread::sleep_for(std::chrono::microseconds(20));
    }
  }
  return DASGD_OK;
}

dasgd_status dasgd_get_step(const dasgd_ctx *ctx, int64_t *t, int32_t *pending) {
  if (!ctx) return DASGD_ERR_INVALID_ARG;
  if (t) *t = ctx->t;
  if (pending) *pending = (int32_t)ctx->pending.size();
  return DASGD_OK;
}

dasgd_status dasgd_get_weights(const dasgd_ctx *ctx, void **w_device) {
  if (!ctx || !w_device) return DASGD_ERR_INVALID_ARG;
  *w_device = ctx->pool[ctx->cur];
  return DASGD_OK;
}

dasgd_status dasgd_get_pending(const dasgd_ctx *ctx, int32_t i, int64_t *s, void **snap_device, void **mean_device) {
  if (!ctx || i < 0 || i >= (int32_t)ctx->pending.size()) return DASGD_ERR_INVALID_ARG;
  const int slot = ctx->pending[i];
  if (s) *s = ctx->slots[slot].s;
  if (snap_device) *snap_device = snap_ptr(ctx, slot);
  if (mean_device) *mean_device = mean_ptr(ctx, slot);
  return DASGD_OK;
}

dasgd_status dasgd_get_timing(dasgd_ctx *ctx, int64_t *n_avg, double *ms_avg, double *ms_stall) {
  if (!ctx) return DASGD_ERR_INVALID_ARG;
  if (!(ctx->cfg.flags & DASGD_FLAG_TIMING)) return fail(ctx, DASGD_ERR_BAD_STATE, "get_timing: DASGD_FLAG_TIMING not set");
  dasgd_status st = dasgd_sync(ctx);
  if (st != DASGD_OK) return st;
  DeviceGuard guard(ctx->cfg.device);
  harvest(ctx, true);
  if (n_avg) *n_avg = ctx->span_n[TAG_MEAN];
  if (ms_avg) *ms_avg = ctx->span_ms[TAG_MEAN];
  if (ms_stall) *ms_stall = ctx->span_ms[TAG_STALL];
  return DASGD_OK;
}

dasgd_status dasgd_get_kernel_timing(dasgd_ctx *ctx, int32_t which, int64_t *n, double *ms) {
  if (!ctx) return DASGD_ERR_INVALID_ARG;
  if (which < 0 || which >= TAG_COUNT) return fail(ctx, DASGD_ERR_INVALID_ARG, "get_kernel_timing: which must be in [0, 4]");
  if (!(ctx->cfg.flags & DASGD_FLAG_TIMING))
    return fail(ctx, DASGD_ERR_BAD_STATE, "get_kernel_timing: DASGD_FLAG_TIMING not set");
  dasgd_status st = dasgd_sync(ctx);
  if (st != DASGD_OK) return st;
  DeviceGuard guard(ctx->cfg.device);
  harvest(ctx, true);
  if (n) *n = ctx->span_n[which];
  if (ms) *ms = ctx->span_ms[which];
  return DASGD_OK;
}

dasgd_status dasgd_reset_timing(dasgd_ctx *ctx) {
  if (!ctx) return DASGD_ERR_INVALID_ARG;
  dasgd_status st = dasgd_sync(ctx);
  if (st != DASGD_OK) return st;
  DeviceGuard guard(ctx->cfg.device);
  harvest(ctx, true);
  for (int i = 0; i < TAG_COUNT; ++i) { ctx->span_n[i] = 0; ctx->span_ms[i] = 0.0; ctx->span_units[i] = 0; }
  return DASGD_OK;
}

namespace {
struct StateHeader {
  uint32_t magic, version;
  int32_t K, tau, d, dtype, merge_mode, n_slots, pool, rotate;
  int64_t P, ld, t;
  int32_t cur, n_pending;
};
struct StatePending { int32_t slot, buf, state, pad; int64_t s; };
constexpr uint32_t kStateMagic = 0x44615347u;  // "DaSG"
}  // namespace

dasgd_status dasgd_export_state(dasgd_ctx *ctx, void *host_buf, int64_t buf_len, int64_t *len) {
  if (!ctx) return DASGD_ERR_INVALID_ARG;
  if (!host_buf || !len) return fail(ctx, DASGD_ERR_INVALID_ARG, "export_state: NULL argument");
  dasgd_status st = dasgd_sync(ctx);
  if (st != DASGD_OK) return st;
  const int64_t need = (int64_t)sizeof(StateHeader) + (int64_t)ctx->pending.size() * (int64_t)sizeof(StatePending);
  *len = need;
  if (buf_len < need) return fail(ctx, DASGD_ERR_INVALID_ARG, "export_state: buffer too small");
  StateHeader h{};
  h.magic = kStateMagic; h.version = 1;
  h.K = ctx->cfg.K; h.tau = ctx->cfg.tau; h.d = ctx->cfg.d; h.dtype = ctx->cfg.dtype;
  h.merge_mode = ctx->cfg.merge_mode; h.n_slots = ctx->cfg.n_slots; h.pool = (int32_t)ctx->pool.size();
  h.rotate = ctx->rotate ? 1 : 0;
  h.P = ctx->cfg.P; h.ld = ctx->cfg.ld; h.t = ctx->t;
  h.cur = ctx->cur; h.n_pending = (int32_t)ctx->pending.size();
  char *out = static_cast<char *>(host_buf);
  std::memcpy(out, &h, sizeof h);
  out += sizeof h;
  for (int slot : ctx->pending) {
    StatePending q{};
    q.slot = slot; q.buf = ctx->slots[slot].buf; q.state = (int32_t)ctx->slots[slot].state; q.s = ctx->slots[slot].s;
    std::memcpy(out, &q, sizeof q);
    out += sizeof q;
  }
  return DASGD_OK;
}

dasgd_status dasgd_import_state(dasgd_ctx *ctx, const void *host_buf, int64_t len) {
  if (!ctx) return DASGD_ERR_INVALID_ARG;
  if (!host_buf || len < (int64_t)sizeof(StateHeader)) return fail(ctx, DASGD_ERR_INVALID_ARG, "import_state: blob too short");
  if (ctx->t != 0 || !ctx->pending.empty())
    return fail(ctx, DASGD_ERR_BAD_STATE, "import_state: the context has already been used");
  StateHeader h;
  std::memcpy(&h, host_buf, sizeof h);
  if (h.magic != kStateMagic || h.version != 1) return fail(ctx, DASGD_ERR_INVALID_ARG, "import_state: not a state blob");
  const dasgd_config &c = ctx->cfg;
  if (h.K != c.K || h.P != c.P || h.ld != c.ld || h.tau != c.tau || h.d != c.d || h.dtype != c.dtype ||
      h.merge_mode != c.merge_mode || h.n_slots != c.n_slots || h.pool != (int32_t)ctx->pool.size() ||
      h.rotate != (ctx->rotate ? 1 : 0))
    return fail(ctx, DASGD_ERR_INVALID_ARG, "import_state: the blob was exported from a different configuration");
  if (h.n_pending < 0 || h.n_pending > c.n_slots || h.cur < 0 || h.cur >= h.pool || h.t < 0 ||
      len < (int64_t)sizeof(StateHeader) + (int64_t)h.n_pending * (int64_t)sizeof(StatePending))
    return fail(ctx, DASGD_ERR_INVALID_ARG, "import_state: corrupt blob");
  std::vector<StatePending> qs(h.n_pending);
  if (h.n_pending) std::memcpy(qs.data(), static_cast<const char *>(host_buf) + sizeof h, qs.size() * sizeof(StatePending));
  std::vector<bool> slot_seen(c.n_slots, false);
  for (const StatePending &q : qs) {
    if (q.slot < 0 || q.slot >= c.n_slots || slot_seen[q.slot] || q.buf < -1 || q.buf >= h.pool ||
        (q.state != SLOT_SNAPPED && q.state != SLOT_AVERAGING))
      return fail(ctx, DASGD_ERR_INVALID_ARG, "import_state: corrupt blob");
    slot_seen[q.slot] = true;
  }
  ctx->t = h.t;
  ctx->cur = h.cur;
  for (const StatePending &q : qs) {
    Slot &sl = ctx->slots[q.slot];
    sl.state = (SlotState)q.state;   // the exporter had synchronised: a started mean is a finished mean,
    sl.s = q.s;                      // so its (never recorded) event makes the later wait a no-op
    sl.buf = q.buf;
    sl.chunked = false;
    sl.holds = q.buf >= 0;
    if (sl.holds) ctx->frozen[q.buf] += 1;
    ctx->pending.push_back(q.slot);
  }
  return DASGD_OK;
}

dasgd_status dasgd_delay_guideline(double t_c, double t_p, int32_t *d, int32_t *tau) {
  if (!d || !tau || !(t_c >= 0.0) || !(t_p > 0.0)) return DASGD_ERR_INVALID_ARG;
  // d > t_c / t_p (Eq. 3): step up from the quotient so that rounding in the division cannot
  // produce a d that violates t_c < d * t_p or is larger than necessary
  double q = t_c / t_p;
  if (q > 1e9) return DASGD_ERR_INVALID_ARG;
  int64_t k = (int64_t)q;  // floor, q >= 0
  if (k < 1) k = 1;
  while (k > 1 && t_c < (double)(k - 1) * t_p) --k;
  while (!(t_c < (double)k * t_p)) ++k;
  *d = (int32_t)k;
  *tau = (int32_t)k + 1;
  return DASGD_OK;
}

dasgd_status dasgd_advise_delay(dasgd_ctx *ctx, double extra_tp_ms, int32_t *d, int32_t *tau, double *t_c_ms,
                                double *t_p_ms) {
  if (!ctx) return DASGD_ERR_INVALID_ARG;
  if (!d || !tau || !(extra_tp_ms >= 0.0)) return fail(ctx, DASGD_ERR_INVALID_ARG, "advise_delay: bad arguments");
  if (!(ctx->cfg.flags & DASGD_FLAG_TIMING)) return fail(ctx, DASGD_ERR_BAD_STATE, "advise_delay: DASGD_FLAG_TIMING not set");
  dasgd_status st = dasgd_sync(ctx);
  if (st != DASGD_OK) return st;
  DeviceGuard guard(ctx->cfg.device);
  harvest(ctx, true);
  if (ctx->span_n[TAG_STEP] < 1 || ctx->span_n[TAG_MEAN] < 1)
    return fail(ctx, DASGD_ERR_BAD_STATE, "advise_delay: needs at least one timed local step and one timed mean");
  const double tc = ctx->span_ms[TAG_MEAN] / (double)ctx->span_n[TAG_MEAN];
  const double tp = ctx->span_ms[TAG_STEP] / (double)ctx->span_n[TAG_STEP] + extra_tp_ms;
  if (t_c_ms) *t_c_ms = tc;
  if (t_p_ms) *t_p_ms = tp;
  if (dasgd_delay_guideline(tc, tp, d, tau) != DASGD_OK) return fail(ctx, DASGD_ERR_INVALID_ARG, "advise_delay: degenerate timings");
  return DASGD_OK;
}

dasgd_status dasgd_get_kernel_units(dasgd_ctx *ctx, int32_t which, int64_t *units) {
  if (!ctx) return DASGD_ERR_INVALID_ARG;
  if (which < 0 || which >= TAG_COUNT || !units)
    return fail(ctx, DASGD_ERR_INVALID_ARG, "get_kernel_units: which must be in [0, 4] and units non-NULL");
  if (!(ctx->cfg.flags & DASGD_FLAG_TIMING))
    return fail(ctx, DASGD_ERR_BAD_STATE, "get_kernel_units: DASGD_FLAG_TIMING not set");
  dasgd_status st = dasgd_sync(ctx);
  if (st != DASGD_OK) return st;
  DeviceGuard guard(ctx->cfg.device);
  harvest(ctx, true);
  *units = ctx->span_units[which];
  return DASGD_OK;
}

dasgd_status dasgd_refresh_lp(dasgd_ctx *ctx) {
  if (!ctx) return DASGD_ERR_INVALID_ARG;
  if (ctx->cfg.dtype != DASGD_BF16_MASTER_F32) return fail(ctx, DASGD_ERR_BAD_STATE, "refresh_lp: float32 mode has no w_lp");
  DeviceGuard guard(ctx->cfg.device);
  Params p = base_params(ctx);
  long long done = 0;
  if (ctx->vec && p.P / 8 > 0) {
    dim3 grid(blocks_for(p.P / 8, kThreads), (unsigned)p.K);
    dasgd::k_refresh_lp_vec<<<grid, kThreads, 0, ctx->s0>>>(p);
    ctx->launches++;
    done = p.P / 8 * 8;
  }
  if (done < p.P) {
    dim3 grid(blocks_for(p.P - done, kThreads), (unsigned)p.K);
    dasgd::k_refresh_lp_scalar<<<grid, kThreads, 0, ctx->s0>>>(p, done);
    ctx->launches++;
  }
  CU(ctx, cudaGetLastError());
  return DASGD_OK;
}

dasgd_status dasgd_set_shard(dasgd_ctx *ctx, int32_t K_total, dasgd_exchange_fn exchange, void *user) {
  if (!ctx) return DASGD_ERR_INVALID_ARG;
  if (K_total < ctx->cfg.K || !exchange)
    return fail(ctx, DASGD_ERR_INVALID_ARG, "set_shard: need K_total >= K and an exchange function");
  if (ctx->cfg.flags & DASGD_FLAG_INLINE_MEAN)
    return fail(ctx, DASGD_ERR_UNSUPPORTED, "set_shard: the inline-mean schedule keeps every worker in one context");
  if (ctx->m_snap) return fail(ctx, DASGD_ERR_UNSUPPORTED, "set_shard: not available together with momentum averaging");
  if (ctx->t != 0 || !ctx->pending.empty())
    return fail(ctx, DASGD_ERR_BAD_STATE, "set_shard: the context has already been used");
  ctx->K_total = K_total;
  ctx->exchange = exchange;
  ctx->exchange_user = user;
  return DASGD_OK;
}

dasgd_status dasgd_set_momentum_averaging(dasgd_ctx *ctx, void *m_snap, void *m_mean) {
  if (!ctx) return DASGD_ERR_INVALID_ARG;
  if (!m_snap || !m_mean || !aligned16(m_snap) || !aligned16(m_mean))
    return fail(ctx, DASGD_ERR_INVALID_ARG, "set_momentum_averaging: m_snap and m_mean must be 16-byte aligned device arrays");
  if (ctx->cfg.momentum == 0.0f || !ctx->cfg.m)
    return fail(ctx, DASGD_ERR_INVALID_ARG, "set_momentum_averaging: the context has no momentum buffers");
  if (ctx->cfg.flags & DASGD_FLAG_INLINE_MEAN)
    return fail(ctx, DASGD_ERR_UNSUPPORTED, "set_momentum_averaging: not available with DASGD_FLAG_INLINE_MEAN");
  if (ctx->K_total > 0) return fail(ctx, DASGD_ERR_UNSUPPORTED, "set_momentum_averaging: not available on a sharded worker axis");
  if (ctx->t != 0 || !ctx->pending.empty())
    return fail(ctx, DASGD_ERR_BAD_STATE, "set_momentum_averaging: the context has already been used");
  DeviceGuard guard(ctx->cfg.device);
  for (void *p : {m_snap, m_mean}) {
    cudaPointerAttributes at{};
    cudaError_t e = cudaPointerGetAttributes(&at, p);
    if (e != cudaSuccess) {
      cudaGetLastError();
      return cuda_fail(ctx, e, "set_momentum_averaging: cudaPointerGetAttributes");
    }
    if ((at.type != cudaMemoryTypeDevice && at.type != cudaMemoryTypeManaged) ||
        (at.type == cudaMemoryTypeDevice && at.device != ctx->cfg.device))
      return fail(ctx, DASGD_ERR_INVALID_ARG, "set_momentum_averaging: m_snap and m_mean must be device memory of cfg.device");
  }
  for (Slot &sl : ctx->slots) {
    if (sl.e_msnap) continue;
    if (cudaEventCreateWithFlags(&sl.e_msnap, cudaEventDisableTiming) != cudaSuccess ||
        cudaEventCreateWithFlags(&sl.e_mavg, cudaEventDisableTiming) != cudaSuccess) {
      cudaGetLastError();
      return fail(ctx, DASGD_ERR_CUDA, "set_momentum_averaging: cannot create events");
    }
  }
  ctx->m_snap = static_cast<float *>(m_snap);
  ctx->m_mean = static_cast<float *>(m_mean);
  return DASGD_OK;
}

dasgd_status dasgd_get_pending_momentum(const dasgd_ctx *ctx, int32_t i, void **m_snap_device, void **m_mean_device) {
  if (!ctx || !ctx->m_snap || i < 0 || i >= (int32_t)ctx->pending.size()) return DASGD_ERR_INVALID_ARG;
  const int slot = ctx->pending[i];
  if (m_snap_device) *m_snap_device = m_snap_ptr(ctx, slot);
  if (m_mean_device) *m_mean_device = m_mean_ptr(ctx, slot);
  return DASGD_OK;
}

// for the other translation units of the library (not exported)
__attribute__((visibility("hidden"))) dasgd_status dasgd_internal_fail(dasgd_ctx *ctx, dasgd_status st, const char *msg) {
  return fail(ctx, st, msg);
}

dasgd_status dasgd_get_launches(const dasgd_ctx *ctx, int64_t *launches) {
  if (!ctx || !launches) return DASGD_ERR_INVALID_ARG;
  *launches = ctx->launches;
  return DASGD_OK;
}

}  // extern "C"
