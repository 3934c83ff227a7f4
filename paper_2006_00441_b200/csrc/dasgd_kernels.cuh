// Device code of libdasgd: the four element-wise / worker-axis kernels of the DaSGD hot path.
//
// Every operation is independent across the parameter index p and moves each byte once, so the
// kernels are HBM-bandwidth bound: the work is laid out for coalesced 128-bit accesses with many
// independent loads in flight per thread, streaming cache hints (nothing is reused inside a
// kernel), and small CTAs so that a higher-priority side-stream kernel can take SM slots as they
// retire.  Tensor cores have no role here (about 0.2 flop per byte).
//
// Weights are read from `w` and written to `w_out`; the two may be the same array (in-place) or
// different ones (the old array then stays intact and serves as the snapshot: no copy is made).
// Each thread reads every element it owns before it writes it, so in-place use is safe.
//
// Arithmetic is float32 with explicit fused multiply-adds, the same expressions in every
// variant, so that fused and unfused schedules give bit-identical results:
//     g' = fma(lambda, w, g);  m = fma(mu, m, g');  w = fma(-lr, m, w)        (local step)
//       Nesterov:            w = fma(-lr, fma(mu, m, g'), w)
//       decoupled decay:     g' = g;  w = fma(-(lr*lambda), w_old, fma(-lr, dir, w_old))
//     w  = fma(xi, w, (1-xi)*mean)                                            (xi merge)
//     w  = w + (mean - snap)                                                  (delta merge)
//     mean = (pairwise sum over k) / K                                        (worker-axis mean)
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace dasgd {

constexpr int kThreads = 256;

// Arguments that change from one iteration to the next, kept in device memory so that a launch recorded
// once (CUDA graph) can be replayed with new values.
struct DynArgs {
  const void *g;  // [K][ld] gradients of this iteration
  float lr;
  int pad;
};

struct Params {
  const float *w;       // [K][ld] weights to read
  float *w_out;         // [K][ld] where the new weights go (== w for an in-place update)
  float *m;             // [K][ld] or nullptr
  const void *g;        // [K][ld] float or bf16
  __nv_bfloat16 *w_lp;  // [K][ld] or nullptr
  float *snap_out;      // [K][ld] snapshot slot to write, or nullptr
  const float *snap_in; // [K][ld] snapshot slot to read (delta merge), or nullptr
  const float *mean;    // [ld] mean slot to read, or nullptr
  float *mean_out;      // [ld] mean slot to write (reduce)
  long long P, ld;
  int K;
  float lr, mu, lambda, xi, omx;
  int nesterov;      // 1: step along g' + mu*m instead of m
  int decoupled_wd;  // 1: weight decay is applied to the weights directly, not added to the gradient
  const DynArgs *dyn;  // non-NULL: take g and lr from there (g_off = first column of this launch)
  long long g_off;
  float mean_div;    // 0: `mean` holds the mean.  Otherwise `mean` holds the SUM over all workers (sharded
                     //    worker axis) and the mean is that sum divided, correctly rounded, by this number
  int sum_only;      // 1: the worker-axis kernel writes the plain sum of its K rows, not their mean
  int group_tiles;   // merging step kernel: tiles per group in the CTA order (1: the K rows of a tile are neighbours)
  int keep_w;        // 1: the new weights are about to be re-read (by the mean of this column range): store
                     //    them with the default cache policy instead of the streaming one
};

// ---------------------------------------------------------------- memory helpers

__device__ __forceinline__ float4 ld_stream(const float4 *p) { return __ldcs(p); }
__device__ __forceinline__ void st_stream(float4 *p, float4 v) { __stcs(p, v); }
__device__ __forceinline__ uint4 ld_stream(const uint4 *p) { return __ldcs(p); }
__device__ __forceinline__ void st_stream(uint4 *p, uint4 v) { __stcs(p, v); }

// 16 bytes from global to shared memory without passing through registers (completion: cp_async_wait_all).
__device__ __forceinline__ void cp_async16(void *smem_dst, const void *gmem_src) {
  const unsigned dst = (unsigned)__cvta_generic_to_shared(smem_dst);
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(gmem_src) : "memory");
}
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_all;" ::: "memory"); }

__device__ __forceinline__ float bf16_bits_to_f32(uint32_t hi16) { return __uint_as_float(hi16 << 16); }

// two float32 -> packed bf16x2, round to nearest even (lo in the low half)
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t *>(&v);
}

// ---------------------------------------------------------------- scalar arithmetic

template <bool MOM>
__device__ __forceinline__ void step_elem(float &w, float &m, float g, const Params &p, float lr) {
  // the two variant switches are uniform across the grid, so the branches cost nothing here
  const float gp = p.decoupled_wd ? g : fmaf(p.lambda, w, g);
  float dir = gp;
  if (MOM) {
    m = fmaf(p.mu, m, gp);
    dir = p.nesterov ? fmaf(p.mu, m, gp) : m;
  }
  const float w_old = w;
  w = fmaf(-lr, dir, w);
  if (p.decoupled_wd) w = fmaf(-__fmul_rn(lr, p.lambda), w_old, w);
}

// The mean as the merge sees it: stored as such, or formed here from the all-worker sum.
__device__ __forceinline__ float mean_of(float v, const Params &p) {
  return p.mean_div != 0.0f ? __fdiv_rn(v, p.mean_div) : v;
}
__device__ __forceinline__ float4 mean_of(float4 v, const Params &p) {
  if (p.mean_div != 0.0f) {
    v.x = __fdiv_rn(v.x, p.mean_div); v.y = __fdiv_rn(v.y, p.mean_div);
    v.z = __fdiv_rn(v.z, p.mean_div); v.w = __fdiv_rn(v.w, p.mean_div);
  }
  return v;
}

// Sum of the K rows -> what the worker-axis kernel stores.
__device__ __forceinline__ float finish_mean(float s, float kf, const Params &p) {
  return p.sum_only ? s : __fdiv_rn(s, kf);
}

__device__ __forceinline__ float blend_xi(float w, float mean, const Params &p) {
  return fmaf(p.xi, w, __fmul_rn(p.omx, mean));
}

__device__ __forceinline__ float blend_delta(float w, float mean, float snap) {
  return __fadd_rn(w, __fsub_rn(mean, snap));
}

#define DASGD_F4_APPLY(dst, expr_x, expr_y, expr_z, expr_w) \
  dst.x = expr_x; dst.y = expr_y; dst.z = expr_z; dst.w = expr_w;

// ---------------------------------------------------------------- local step (vector path)
//
// One CTA = one worker k and one tile of kThreads*UNROLL units; a unit is 4 consecutive parameters in both
// dtypes: the float32 arrays are read and written as one 16-byte access per unit, bfloat16 gradients and the
// bfloat16 weight copy as one 8-byte access per unit, so that every warp-wide access covers a contiguous range
// (with 8-element units each lane would touch two separate halves of a 32-byte sector of the float32 arrays).
// With a fused merge blockIdx.x enumerates groups of group_tiles tiles and, inside a group, (k, tile) with the
// tile fastest: the K passes over a group re-read the same piece of the mean, which is fetched from HBM once and
// then served by L2 (group_tiles = 1: the K CTAs of a tile are neighbours in launch order).  Without a merge rows
// are walked one after the other (k slowest), which keeps every CTA wave on one contiguous address range
// (measured 1.2 % faster).
// MERGE: 0 none, 1 xi-blend, 2 delta.  SNAP: also store the final w into snap_out.

// Three CTAs per SM (at most 80 registers): with a merge folded in the kernel would otherwise take 85-96
// registers and lose a third of its resident warps, i.e. of its loads in flight.
template <bool BF16, bool MOM, int MERGE, bool SNAP>
__global__ void __launch_bounds__(kThreads, 3) k_local_step_vec(const Params p) {
  constexpr int UNROLL = 4;  // units per thread
  const long long units = p.P / 4;
  int k;
  long long tile;
  if (MERGE != 0) {
    // groups of group_tiles tiles: inside a group the rows are walked one after the other, so that every row is
    // read and written in contiguous runs while the K CTAs that share a piece of the mean stay close in time
    const long long tiles = (units + kThreads * UNROLL - 1) / (kThreads * UNROLL);
    const long long per_group = (long long)p.group_tiles * p.K;
    const long long grp = blockIdx.x / per_group;
    const long long r = blockIdx.x - grp * per_group;
    const long long left = tiles - grp * p.group_tiles;
    const long long g_eff = left < p.group_tiles ? left : p.group_tiles;
    k = (int)(r / g_eff);
    tile = grp * p.group_tiles + r % g_eff;
  } else {
    const unsigned tiles = (unsigned)((units + kThreads * UNROLL - 1) / (kThreads * UNROLL));
    k = blockIdx.x / tiles;
    tile = blockIdx.x % tiles;
  }
  const long long row = (long long)k * p.ld;
  const long long u0 = tile * (long long)(kThreads * UNROLL) + threadIdx.x;
  const void *gbase = p.g;
  float lr = p.lr;
  if (p.dyn) {
    gbase = static_cast<const char *>(p.dyn->g) + p.g_off * (BF16 ? 2 : 4);
    lr = p.dyn->lr;
  }

  float4 w4[UNROLL], m4[UNROLL], g4[UNROLL], s4[UNROLL];
  bool ok[UNROLL];
  // The piece of the mean this CTA blends with is staged in shared memory by asynchronous copies: it then holds no
  // registers while in flight (with it in registers the kernel wants 90, and at the 80 that three CTAs per SM
  // allow the compiler can no longer issue all loads before the first use).  Every thread reads back only what it
  // copied itself, so waiting for its own copies is enough; no barrier.
  __shared__ float4 s_mean[MERGE != 0 ? UNROLL : 1][MERGE != 0 ? kThreads : 1];

#pragma unroll
  for (int j = 0; j < UNROLL; ++j) {
    const long long u = u0 + (long long)j * kThreads;
    ok[j] = u < units;
    if (ok[j]) {
      const long long e = u * 4;  // element offset inside the row
      if (BF16) {
        const uint2 gb = __ldcs(reinterpret_cast<const uint2 *>(static_cast<const __nv_bfloat16 *>(gbase) + row + e));
        g4[j] = make_float4(bf16_bits_to_f32(gb.x & 0xFFFFu), bf16_bits_to_f32(gb.x >> 16),
                            bf16_bits_to_f32(gb.y & 0xFFFFu), bf16_bits_to_f32(gb.y >> 16));
      } else {
        g4[j] = ld_stream(reinterpret_cast<const float4 *>(static_cast<const float *>(gbase) + row + e));
      }
      w4[j] = ld_stream(reinterpret_cast<const float4 *>(p.w + row + e));
      if (MOM) m4[j] = ld_stream(reinterpret_cast<const float4 *>(p.m + row + e));
      if (MERGE != 0) cp_async16(&s_mean[j][threadIdx.x], p.mean + e);
      if (MERGE == 2) s4[j] = ld_stream(reinterpret_cast<const float4 *>(p.snap_in + row + e));
    }
  }

  if (MERGE != 0) cp_async_wait_all();
#pragma unroll
  for (int j = 0; j < UNROLL; ++j) {
    if (!ok[j]) continue;
    const long long e = (u0 + (long long)j * kThreads) * 4;
    float4 w = w4[j];
    float4 m = MOM ? m4[j] : make_float4(0.f, 0.f, 0.f, 0.f);
    const float4 g = g4[j];
    step_elem<MOM>(w.x, m.x, g.x, p, lr);
    step_elem<MOM>(w.y, m.y, g.y, p, lr);
    step_elem<MOM>(w.z, m.z, g.z, p, lr);
    step_elem<MOM>(w.w, m.w, g.w, p, lr);
    if (MERGE == 1) {
      const float4 a = mean_of(s_mean[j][threadIdx.x], p);
      DASGD_F4_APPLY(w, blend_xi(w.x, a.x, p), blend_xi(w.y, a.y, p), blend_xi(w.z, a.z, p), blend_xi(w.w, a.w, p))
    } else if (MERGE == 2) {
      const float4 a = mean_of(s_mean[j][threadIdx.x], p), s = s4[j];
      DASGD_F4_APPLY(w, blend_delta(w.x, a.x, s.x), blend_delta(w.y, a.y, s.y), blend_delta(w.z, a.z, s.z),
                     blend_delta(w.w, a.w, s.w))
    }
    if (p.keep_w) *reinterpret_cast<float4 *>(p.w_out + row + e) = w;
    else st_stream(reinterpret_cast<float4 *>(p.w_out + row + e), w);
    if (MOM) st_stream(reinterpret_cast<float4 *>(p.m + row + e), m);
    if (SNAP) st_stream(reinterpret_cast<float4 *>(p.snap_out + row + e), w);
    if (BF16) {
      uint2 o;
      o.x = pack_bf16x2(w.x, w.y);
      o.y = pack_bf16x2(w.z, w.w);
      __stcs(reinterpret_cast<uint2 *>(p.w_lp + row + e), o);
    }
  }
}

// ---------------------------------------------------------------- local step (scalar path)
// Columns [p0, P) of every row, one thread per (k, p).  Used for the ragged end of a row and for
// arrays whose rows are not 16-byte aligned.

template <bool BF16, bool MOM, int MERGE, bool SNAP>
__global__ void __launch_bounds__(kThreads) k_local_step_scalar(const Params p, long long p0) {
  const long long col = p0 + (long long)blockIdx.x * kThreads + threadIdx.x;
  const int k = blockIdx.y;
  if (col >= p.P) return;
  const long long i = (long long)k * p.ld + col;
  float w = p.w[i], m = MOM ? p.m[i] : 0.0f;
  const void *gbase = p.g;
  float lr = p.lr;
  if (p.dyn) {
    gbase = static_cast<const char *>(p.dyn->g) + p.g_off * (BF16 ? 2 : 4);
    lr = p.dyn->lr;
  }
  const float g = BF16 ? __bfloat162float(static_cast<const __nv_bfloat16 *>(gbase)[i])
                       : static_cast<const float *>(gbase)[i];
  step_elem<MOM>(w, m, g, p, lr);
  if (MERGE == 1) w = blend_xi(w, mean_of(p.mean[col], p), p);
  if (MERGE == 2) w = blend_delta(w, mean_of(p.mean[col], p), p.snap_in[i]);
  p.w_out[i] = w;
  if (MOM) p.m[i] = m;
  if (SNAP) p.snap_out[i] = w;
  if (BF16) p.w_lp[i] = __float2bfloat16_rn(w);
}

// ---------------------------------------------------------------- snapshot copy

__global__ void __launch_bounds__(kThreads) k_snapshot_vec(const Params p) {
  constexpr int UNROLL = 4;
  const int k = blockIdx.x % p.K;
  const long long tile = blockIdx.x / p.K;
  const long long units = p.P / 4;
  const long long row = (long long)k * p.ld;
  const long long u0 = tile * (long long)(kThreads * UNROLL) + threadIdx.x;
  float4 v[UNROLL];
#pragma unroll
  for (int j = 0; j < UNROLL; ++j) {
    const long long u = u0 + (long long)j * kThreads;
    if (u < units) v[j] = ld_stream(reinterpret_cast<const float4 *>(p.w + row) + u);
  }
#pragma unroll
  for (int j = 0; j < UNROLL; ++j) {
    const long long u = u0 + (long long)j * kThreads;
    if (u < units) st_stream(reinterpret_cast<float4 *>(p.snap_out + row) + u, v[j]);
  }
}

__global__ void __launch_bounds__(kThreads) k_snapshot_scalar(const Params p, long long p0) {
  const long long col = p0 + (long long)blockIdx.x * kThreads + threadIdx.x;
  if (col >= p.P) return;
  const long long i = (long long)blockIdx.y * p.ld + col;
  p.snap_out[i] = p.w[i];
}

// ---------------------------------------------------------------- worker-axis mean
// One thread owns U units of 4 consecutive parameters and walks the K rows, eight independent
// 16-byte loads at a time.  Summation: four interleaved partial sums (k mod 4) combined pairwise;
// then one correctly rounded division by K.

__device__ __forceinline__ void add4(float4 &a, const float4 &b) {
  a.x = __fadd_rn(a.x, b.x); a.y = __fadd_rn(a.y, b.y); a.z = __fadd_rn(a.z, b.z); a.w = __fadd_rn(a.w, b.w);
}

// U units per thread (columns u, u + kThreads, ...): with few rows more columns per thread keep
// enough loads in flight (K = 2 ran at half the bandwidth with one column per thread).
template <int U, int KC /* rows per batch of loads: a multiple of 4, so k mod 4 == j mod 4 */, int MINB>
__global__ void __launch_bounds__(kThreads, MINB) k_reduce_vec(const Params p) {
  const long long units = p.P / 4;
  const long long u0 = (long long)blockIdx.x * (kThreads * U) + threadIdx.x;
  const float4 *base = reinterpret_cast<const float4 *>(p.snap_in);
  const long long ld4 = p.ld / 4;
  float4 acc[U][4];
#pragma unroll
  for (int c = 0; c < U; ++c)
#pragma unroll
    for (int a = 0; a < 4; ++a) acc[c][a] = make_float4(0.f, 0.f, 0.f, 0.f);
  for (int k0 = 0; k0 < p.K; k0 += KC) {
    float4 v[U][KC];
#pragma unroll
    for (int j = 0; j < KC; ++j)
#pragma unroll
      for (int c = 0; c < U; ++c) {
        const long long u = u0 + (long long)c * kThreads;
        if (k0 + j < p.K && u < units) v[c][j] = ld_stream(base + (long long)(k0 + j) * ld4 + u);
      }
#pragma unroll
    for (int j = 0; j < KC; ++j)
#pragma unroll
      for (int c = 0; c < U; ++c)
        if (k0 + j < p.K && u0 + (long long)c * kThreads < units) add4(acc[c][j & 3], v[c][j]);
  }
  const float kf = (float)p.K;
#pragma unroll
  for (int c = 0; c < U; ++c) {
    const long long u = u0 + (long long)c * kThreads;
    if (u >= units) continue;
    add4(acc[c][0], acc[c][1]);
    add4(acc[c][2], acc[c][3]);
    add4(acc[c][0], acc[c][2]);
    float4 r;
    r.x = finish_mean(acc[c][0].x, kf, p); r.y = finish_mean(acc[c][0].y, kf, p);
    r.z = finish_mean(acc[c][0].z, kf, p); r.w = finish_mean(acc[c][0].w, kf, p);
    reinterpret_cast<float4 *>(p.mean_out)[u] = r;  // re-read by the merge: leave it cacheable
  }
}

// K <= 4: the whole column fits in registers.  Missing rows count as +0, which leaves the pairwise
// tree (r0 + r1) + (r2 + r3) equal to what the general kernel computes.
template <int U, int MINB>
__global__ void __launch_bounds__(kThreads, MINB) k_reduce_small(const Params p) {
  const long long units = p.P / 4;
  const long long u0 = (long long)blockIdx.x * (kThreads * U) + threadIdx.x;
  const float4 *base = reinterpret_cast<const float4 *>(p.snap_in);
  const long long ld4 = p.ld / 4;
  float4 v[U][4];
#pragma unroll
  for (int c = 0; c < U; ++c) {
    const long long u = u0 + (long long)c * kThreads;
#pragma unroll
    for (int j = 0; j < 4; ++j)
      v[c][j] = (j < p.K && u < units) ? ld_stream(base + (long long)j * ld4 + u) : make_float4(0.f, 0.f, 0.f, 0.f);
  }
  const float kf = (float)p.K;
#pragma unroll
  for (int c = 0; c < U; ++c) {
    const long long u = u0 + (long long)c * kThreads;
    if (u >= units) continue;
    add4(v[c][0], v[c][1]);
    add4(v[c][2], v[c][3]);
    add4(v[c][0], v[c][2]);
    float4 r;
    r.x = finish_mean(v[c][0].x, kf, p); r.y = finish_mean(v[c][0].y, kf, p);
    r.z = finish_mean(v[c][0].z, kf, p); r.w = finish_mean(v[c][0].w, kf, p);
    reinterpret_cast<float4 *>(p.mean_out)[u] = r;
  }
}

__global__ void __launch_bounds__(kThreads) k_reduce_scalar(const Params p, long long p0) {
  const long long col = p0 + (long long)blockIdx.x * kThreads + threadIdx.x;
  if (col >= p.P) return;
  float acc[4] = {0.f, 0.f, 0.f, 0.f};
  for (int k = 0; k < p.K; ++k) acc[k & 3] = __fadd_rn(acc[k & 3], p.snap_in[(long long)k * p.ld + col]);
  const float s = __fadd_rn(__fadd_rn(acc[0], acc[1]), __fadd_rn(acc[2], acc[3]));
  p.mean_out[col] = finish_mean(s, (float)p.K, p);
}

// ---------------------------------------------------------------- delayed merge
// One thread owns one unit of the parameter axis, keeps the mean in registers and walks the K
// rows four at a time: the mean is read from HBM once, not K times.

template <bool BF16, int MODE /*1 xi, 2 delta*/, bool SNAP>
__global__ void __launch_bounds__(kThreads) k_merge_vec(const Params p) {
  constexpr int EPU = BF16 ? 8 : 4;
  constexpr int F4 = EPU / 4;
  constexpr int KB = BF16 ? 2 : 4;  // rows in flight
  const long long u = (long long)blockIdx.x * kThreads + threadIdx.x;
  if (u >= p.P / EPU) return;
  const long long e = u * EPU;
  float4 a[F4];
#pragma unroll
  for (int f = 0; f < F4; ++f) a[f] = mean_of(__ldg(reinterpret_cast<const float4 *>(p.mean + e) + f), p);
  for (int k0 = 0; k0 < p.K; k0 += KB) {
    float4 w[KB][F4], s[KB][F4];
#pragma unroll
    for (int j = 0; j < KB; ++j) {
      if (k0 + j >= p.K) continue;
      const long long off = (long long)(k0 + j) * p.ld + e;
#pragma unroll
      for (int f = 0; f < F4; ++f) {
        w[j][f] = ld_stream(reinterpret_cast<const float4 *>(p.w + off) + f);
        if (MODE == 2) s[j][f] = ld_stream(reinterpret_cast<const float4 *>(p.snap_in + off) + f);
      }
    }
#pragma unroll
    for (int j = 0; j < KB; ++j) {
      if (k0 + j >= p.K) continue;
      const long long off = (long long)(k0 + j) * p.ld + e;
#pragma unroll
      for (int f = 0; f < F4; ++f) {
        float4 x = w[j][f];
        if (MODE == 1) {
          DASGD_F4_APPLY(x, blend_xi(x.x, a[f].x, p), blend_xi(x.y, a[f].y, p), blend_xi(x.z, a[f].z, p),
                         blend_xi(x.w, a[f].w, p))
        } else {
          const float4 t = s[j][f];
          DASGD_F4_APPLY(x, blend_delta(x.x, a[f].x, t.x), blend_delta(x.y, a[f].y, t.y),
                         blend_delta(x.z, a[f].z, t.z), blend_delta(x.w, a[f].w, t.w))
        }
        st_stream(reinterpret_cast<float4 *>(p.w_out + off) + f, x);
        if (SNAP) st_stream(reinterpret_cast<float4 *>(p.snap_out + off) + f, x);
        w[j][f] = x;
      }
      if (BF16) {
        uint4 o;
        o.x = pack_bf16x2(w[j][0].x, w[j][0].y);
        o.y = pack_bf16x2(w[j][0].z, w[j][0].w);
        o.z = pack_bf16x2(w[j][F4 - 1].x, w[j][F4 - 1].y);
        o.w = pack_bf16x2(w[j][F4 - 1].z, w[j][F4 - 1].w);
        st_stream(reinterpret_cast<uint4 *>(p.w_lp + off), o);
      }
    }
  }
}

template <bool BF16, int MODE, bool SNAP>
__global__ void __launch_bounds__(kThreads) k_merge_scalar(const Params p, long long p0) {
  const long long col = p0 + (long long)blockIdx.x * kThreads + threadIdx.x;
  if (col >= p.P) return;
  const float a = mean_of(p.mean[col], p);
  for (int k = 0; k < p.K; ++k) {
    const long long i = (long long)k * p.ld + col;
    float w = p.w[i];
    w = (MODE == 1) ? blend_xi(w, a, p) : blend_delta(w, a, p.snap_in[i]);
    p.w_out[i] = w;
    if (SNAP) p.snap_out[i] = w;
    if (BF16) p.w_lp[i] = __float2bfloat16_rn(w);
  }
}

// ---------------------------------------------------------------- whole iteration in one kernel
// "Inline mean" schedule: one thread owns one unit of the parameter axis and walks the K rows doing
// the local step; if a merge lands on this iteration it blends with the stored mean (kept in
// registers); if a snapshot is due it sums the resulting weights of the K rows and writes their mean.
// The mean therefore needs no snapshot array and no second pass over HBM.  Same arithmetic and the
// same summation tree as the separate kernels, so the results are bit-identical to theirs.
// mean (read) and mean_out (written) may be the same array: a thread reads its elements of the old
// mean before it writes the new ones, and no other thread touches them.  Because the array may be
// written by this very kernel, the old mean is fetched with ordinary loads, not through the read-only
// data path (which requires memory that stays unmodified for the whole kernel).

template <bool BF16, bool MOM, bool MERGE, bool MEANOUT>
__global__ void __launch_bounds__(kThreads) k_step_allk_vec(const Params p) {
  constexpr int EPU = BF16 ? 8 : 4;
  constexpr int F4 = EPU / 4;
  constexpr int KB = BF16 ? 2 : 4;  // rows loaded together; rows are taken in groups of 4
  const long long u = (long long)blockIdx.x * kThreads + threadIdx.x;
  if (u >= p.P / EPU) return;
  const long long e = u * EPU;
  float4 a[F4], acc[F4][4];
#pragma unroll
  for (int f = 0; f < F4; ++f) {
    if (MERGE) a[f] = reinterpret_cast<const float4 *>(p.mean + e)[f];
#pragma unroll
    for (int q = 0; q < 4; ++q) acc[f][q] = make_float4(0.f, 0.f, 0.f, 0.f);
  }
  for (int k0 = 0; k0 < p.K; k0 += 4) {
#pragma unroll
    for (int h = 0; h < 4; h += KB) {
      float4 w[KB][F4], m[KB][F4], g[KB][F4];
#pragma unroll
      for (int j = 0; j < KB; ++j) {
        const int k = k0 + h + j;
        if (k >= p.K) continue;
        const long long off = (long long)k * p.ld + e;
        if (BF16) {
          const uint4 gb = ld_stream(reinterpret_cast<const uint4 *>(static_cast<const __nv_bfloat16 *>(p.g) + off));
          g[j][0] = make_float4(bf16_bits_to_f32(gb.x & 0xFFFFu), bf16_bits_to_f32(gb.x >> 16),
                                bf16_bits_to_f32(gb.y & 0xFFFFu), bf16_bits_to_f32(gb.y >> 16));
          g[j][F4 - 1] = make_float4(bf16_bits_to_f32(gb.z & 0xFFFFu), bf16_bits_to_f32(gb.z >> 16),
                                     bf16_bits_to_f32(gb.w & 0xFFFFu), bf16_bits_to_f32(gb.w >> 16));
        } else {
          g[j][0] = ld_stream(reinterpret_cast<const float4 *>(static_cast<const float *>(p.g) + off));
        }
#pragma unroll
        for (int f = 0; f < F4; ++f) {
          w[j][f] = ld_stream(reinterpret_cast<const float4 *>(p.w + off) + f);
          if (MOM) m[j][f] = ld_stream(reinterpret_cast<const float4 *>(p.m + off) + f);
        }
      }
#pragma unroll
      for (int j = 0; j < KB; ++j) {
        const int k = k0 + h + j;
        if (k >= p.K) continue;
        const long long off = (long long)k * p.ld + e;
#pragma unroll
        for (int f = 0; f < F4; ++f) {
          float4 x = w[j][f];
          float4 y = MOM ? m[j][f] : make_float4(0.f, 0.f, 0.f, 0.f);
          const float4 gg = g[j][f];
          step_elem<MOM>(x.x, y.x, gg.x, p, p.lr);
          step_elem<MOM>(x.y, y.y, gg.y, p, p.lr);
          step_elem<MOM>(x.z, y.z, gg.z, p, p.lr);
          step_elem<MOM>(x.w, y.w, gg.w, p, p.lr);
          if (MERGE) {
            DASGD_F4_APPLY(x, blend_xi(x.x, a[f].x, p), blend_xi(x.y, a[f].y, p), blend_xi(x.z, a[f].z, p),
                           blend_xi(x.w, a[f].w, p))
          }
          st_stream(reinterpret_cast<float4 *>(p.w_out + off) + f, x);
          if (MOM) st_stream(reinterpret_cast<float4 *>(p.m + off) + f, y);
          if (MEANOUT) add4(acc[f][h + j], x);   // (k mod 4) == h + j because k0 is a multiple of 4
          w[j][f] = x;
        }
        if (BF16) {
          uint4 o;
          o.x = pack_bf16x2(w[j][0].x, w[j][0].y);
          o.y = pack_bf16x2(w[j][0].z, w[j][0].w);
          o.z = pack_bf16x2(w[j][F4 - 1].x, w[j][F4 - 1].y);
          o.w = pack_bf16x2(w[j][F4 - 1].z, w[j][F4 - 1].w);
          st_stream(reinterpret_cast<uint4 *>(p.w_lp + off), o);
        }
      }
    }
  }
  if (MEANOUT) {
    const float kf = (float)p.K;
#pragma unroll
    for (int f = 0; f < F4; ++f) {
      add4(acc[f][0], acc[f][1]);
      add4(acc[f][2], acc[f][3]);
      add4(acc[f][0], acc[f][2]);
      float4 r;
      r.x = __fdiv_rn(acc[f][0].x, kf); r.y = __fdiv_rn(acc[f][0].y, kf);
      r.z = __fdiv_rn(acc[f][0].z, kf); r.w = __fdiv_rn(acc[f][0].w, kf);
      reinterpret_cast<float4 *>(p.mean_out + e)[f] = r;
    }
  }
}

template <bool BF16, bool MOM, bool MERGE, bool MEANOUT>
__global__ void __launch_bounds__(kThreads) k_step_allk_scalar(const Params p, long long p0) {
  const long long col = p0 + (long long)blockIdx.x * kThreads + threadIdx.x;
  if (col >= p.P) return;
  const float a = MERGE ? p.mean[col] : 0.0f;
  float acc[4] = {0.f, 0.f, 0.f, 0.f};
  for (int k = 0; k < p.K; ++k) {
    const long long i = (long long)k * p.ld + col;
    float w = p.w[i], m = MOM ? p.m[i] : 0.0f;
    const float g = BF16 ? __bfloat162float(static_cast<const __nv_bfloat16 *>(p.g)[i])
                         : static_cast<const float *>(p.g)[i];
    step_elem<MOM>(w, m, g, p, p.lr);
    if (MERGE) w = blend_xi(w, a, p);
    p.w_out[i] = w;
    if (MOM) p.m[i] = m;
    if (BF16) p.w_lp[i] = __float2bfloat16_rn(w);
    if (MEANOUT) acc[k & 3] = __fadd_rn(acc[k & 3], w);
  }
  if (MEANOUT)
    p.mean_out[col] = __fdiv_rn(__fadd_rn(__fadd_rn(acc[0], acc[1]), __fadd_rn(acc[2], acc[3])), (float)p.K);
}

// ---------------------------------------------------------------- per-iteration arguments of a replayed launch

__global__ void k_set_dyn(DynArgs *dyn, const void *g, float lr) {
  dyn->g = g;
  dyn->lr = lr;
}

// ---------------------------------------------------------------- bf16 copy of the master weights
// w_lp <- round-to-nearest-even(w), the same conversion every kernel that writes w applies.

__global__ void __launch_bounds__(kThreads) k_refresh_lp_vec(const Params p) {
  const long long u = (long long)blockIdx.x * kThreads + threadIdx.x;
  const int k = blockIdx.y;
  if (u >= p.P / 8) return;
  const long long off = (long long)k * p.ld + u * 8;
  const float4 a = reinterpret_cast<const float4 *>(p.w + off)[0];
  const float4 b = reinterpret_cast<const float4 *>(p.w + off)[1];
  uint4 o;
  o.x = pack_bf16x2(a.x, a.y);
  o.y = pack_bf16x2(a.z, a.w);
  o.z = pack_bf16x2(b.x, b.y);
  o.w = pack_bf16x2(b.z, b.w);
  *reinterpret_cast<uint4 *>(p.w_lp + off) = o;
}

__global__ void __launch_bounds__(kThreads) k_refresh_lp_scalar(const Params p, long long p0) {
  const long long col = p0 + (long long)blockIdx.x * kThreads + threadIdx.x;
  if (col >= p.P) return;
  const long long i = (long long)blockIdx.y * p.ld + col;
  p.w_lp[i] = __float2bfloat16_rn(p.w[i]);
}

}  // namespace dasgd
