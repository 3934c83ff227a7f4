// dasgd_average_merge_noalloc: the averaging of all replicas in one call, for callers that may not
// allocate device memory.  The mean vector, which every other entry point keeps in a caller-provided
// buffer, lives here in a fixed array that is part of the library image.
#include "dasgd.h"

#include <cuda_runtime.h>

#include <cstdio>
#include <mutex>

namespace {

constexpr int kThreads = 256;

// One mean vector of at most DASGD_NOALLOC_MAX_P float32 values (4 MiB).  It is created on every
// GPU on which this library is loaded and stays there until the process exits.
static __device__ __align__(256) float g_noalloc_mean[DASGD_NOALLOC_MAX_P];

// Variants of the library's mean and merge kernels that take the built-in array as their scratch.
// One thread per parameter; same arithmetic as the vector kernels (four interleaved partial sums
// combined pairwise, one correctly rounded division; blend = fma(xi, w, (1-xi)*mean)).
__global__ void __launch_bounds__(kThreads) k_noalloc_mean(const float *w, float *mean, int K, long long P,
                                                           long long ld) {
  const long long col = (long long)blockIdx.x * kThreads + threadIdx.x;
  if (col >= P) return;
  float acc[4] = {0.f, 0.f, 0.f, 0.f};
  for (int k = 0; k < K; ++k) acc[k & 3] = __fadd_rn(acc[k & 3], w[(long long)k * ld + col]);
  const float s = __fadd_rn(__fadd_rn(acc[0], acc[1]), __fadd_rn(acc[2], acc[3]));
  mean[col] = __fdiv_rn(s, (float)K);
}

__global__ void __launch_bounds__(kThreads) k_noalloc_blend(float *w, const float *mean, int K, long long P,
                                                            long long ld, float xi, float omx) {
  const long long col = (long long)blockIdx.x * kThreads + threadIdx.x;
  if (col >= P) return;
  const float a = __fmul_rn(omx, mean[col]);
  for (int k = 0; k < K; ++k) {
    const long long i = (long long)k * ld + col;
    w[i] = fmaf(xi, w[i], a);
  }
}

constexpr int kMaxDevices = 64;
std::mutex g_mu;
float *g_mean_addr[kMaxDevices] = {};  // device address of g_noalloc_mean, per device ordinal

void say(char *buf, int64_t len, const char *msg) {
  if (buf && len > 0) std::snprintf(buf, (size_t)len, "%s", msg);
}

}  // namespace

extern "C" dasgd_status dasgd_average_merge_noalloc(void *w_device, int32_t K, int64_t P, int64_t ld, float xi,
                                                    int32_t device, void *stream, char *errbuf,
                                                    int64_t errbuf_len) {
  if (ld == 0) ld = P;
  if (!w_device || K < 1 || K > 65535 || P < 1 || ld < P || !(xi >= 0.0f && xi <= 1.0f) || device < 0 ||
      device >= kMaxDevices) {
    say(errbuf, errbuf_len, "average_merge_noalloc: need w != NULL, 1 <= K <= 65535, P >= 1, ld >= P, 0 <= xi <= 1");
    return DASGD_ERR_INVALID_ARG;
  }
  if (P > DASGD_NOALLOC_MAX_P) {
    say(errbuf, errbuf_len, "average_merge_noalloc: P exceeds DASGD_NOALLOC_MAX_P (1048576); "
                            "use dasgd_snapshot/dasgd_average_async/dasgd_merge with caller-provided buffers");
    return DASGD_ERR_UNSUPPORTED;
  }
  if ((reinterpret_cast<uintptr_t>(w_device) & 3u) != 0) {
    say(errbuf, errbuf_len, "average_merge_noalloc: w must be 4-byte aligned");
    return DASGD_ERR_INVALID_ARG;
  }

  int prev = -1;
  cudaError_t e = cudaGetDevice(&prev);
  if (e == cudaSuccess && prev != device) e = cudaSetDevice(device);
  if (e != cudaSuccess) {
    say(errbuf, errbuf_len, cudaGetErrorString(e));
    return DASGD_ERR_CUDA;
  }
  dasgd_status st = DASGD_OK;
  float *mean = nullptr;
  {
    // First call on this device: ask the runtime where the array lives on the device that is
    // current now.  In host code the array's name is only a handle for this query.
    std::lock_guard<std::mutex> lock(g_mu);
    if (!g_mean_addr[device]) {
      void *addr = nullptr;
      e = cudaGetSymbolAddress(&addr, g_noalloc_mean);
      if (e != cudaSuccess || !addr) {
        say(errbuf, errbuf_len, e != cudaSuccess ? cudaGetErrorString(e) : "cudaGetSymbolAddress returned NULL");
        st = DASGD_ERR_CUDA;
      } else {
        g_mean_addr[device] = static_cast<float *>(addr);
      }
    }
    mean = g_mean_addr[device];
  }

  if (st == DASGD_OK) {
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const unsigned blocks = (unsigned)((P + kThreads - 1) / kThreads);
    // every element [0, P) of the array is overwritten by the first kernel before the second reads it
    k_noalloc_mean<<<blocks, kThreads, 0, s>>>(static_cast<const float *>(w_device), mean, K, P, ld);
    k_noalloc_blend<<<blocks, kThreads, 0, s>>>(static_cast<float *>(w_device), mean, K, P, ld, xi, 1.0f - xi);
    e = cudaGetLastError();
    if (e != cudaSuccess) {
      say(errbuf, errbuf_len, cudaGetErrorString(e));
      st = DASGD_ERR_CUDA;
    }
  }
  if (prev >= 0 && prev != device) cudaSetDevice(prev);
  return st;
}
