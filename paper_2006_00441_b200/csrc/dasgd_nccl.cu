// The sharded worker axis over NCCL: the exchange of partial sums is one ncclAllReduce(sum, float32) on the
// side stream.  NCCL is loaded at run time (dlopen), so the library itself has no link-time dependency on
// it and loads on machines without it.  Only the host API is used here: no kernel of this library touches
// another GPU's memory.
#include "dasgd.h"

#include <cuda_runtime.h>
#include <dlfcn.h>
#include <nccl.h>

#include <mutex>
#include <cstring>
#include <string>

extern "C" __attribute__((visibility("hidden"))) dasgd_status dasgd_internal_fail(dasgd_ctx *ctx, dasgd_status st, const char *msg);

namespace {

struct NcclApi {
  void *handle = nullptr;
  ncclResult_t (*GetUniqueId)(ncclUniqueId *) = nullptr;
  ncclResult_t (*CommInitRank)(ncclComm_t *, int, ncclUniqueId, int) = nullptr;
  ncclResult_t (*CommDestroy)(ncclComm_t) = nullptr;
  ncclResult_t (*AllReduce)(const void *, void *, size_t, ncclDataType_t, ncclRedOp_t, ncclComm_t, cudaStream_t) = nullptr;
  const char *(*GetErrorString)(ncclResult_t) = nullptr;
  std::string why;  // why loading failed
};

NcclApi *nccl() {
  static NcclApi api;
  static std::once_flag once;
  std::call_once(once, [] {
    // A process that already carries an NCCL (PyTorch bundles one) gets that copy back: same soname.
    api.handle = dlopen("libnccl.so.2", RTLD_NOW | RTLD_GLOBAL);
    if (!api.handle) {
      const char *e = dlerror();
      api.why = std::string("cannot load libnccl.so.2: ") + (e ? e : "unknown error");
      return;
    }
    auto sym = [&](const char *name) {
      void *p = dlsym(api.handle, name);
      if (!p && api.why.empty()) api.why = std::string("libnccl.so.2 lacks ") + name;
      return p;
    };
    api.GetUniqueId = reinterpret_cast<decltype(api.GetUniqueId)>(sym("ncclGetUniqueId"));
    api.CommInitRank = reinterpret_cast<decltype(api.CommInitRank)>(sym("ncclCommInitRank"));
    api.CommDestroy = reinterpret_cast<decltype(api.CommDestroy)>(sym("ncclCommDestroy"));
    api.AllReduce = reinterpret_cast<decltype(api.AllReduce)>(sym("ncclAllReduce"));
    api.GetErrorString = reinterpret_cast<decltype(api.GetErrorString)>(sym("ncclGetErrorString"));
  });
  return api.why.empty() ? &api : nullptr;
}

dasgd_status unavailable() {
  static NcclApi *dummy = nccl();
  (void)dummy;
  return dasgd_internal_fail(nullptr, DASGD_ERR_UNSUPPORTED, "NCCL is not available (libnccl.so.2 could not be loaded)");
}

dasgd_status nccl_fail(NcclApi *a, ncclResult_t r, const char *what) {
  const std::string msg = std::string(what) + ": " + (a->GetErrorString ? a->GetErrorString(r) : "NCCL error");
  return dasgd_internal_fail(nullptr, DASGD_ERR_CUDA, msg.c_str());
}

dasgd_status nccl_exchange(void *user, const void *send, void *recv, int64_t count, void *stream) {
  NcclApi *a = nccl();
  if (!a) return DASGD_ERR_UNSUPPORTED;
  const ncclResult_t r = a->AllReduce(send, recv, (size_t)count, ncclFloat32, ncclSum, static_cast<ncclComm_t>(user),
                                      static_cast<cudaStream_t>(stream));
  return r == ncclSuccess ? DASGD_OK : nccl_fail(a, r, "ncclAllReduce");
}

}  // namespace

extern "C" {

dasgd_status dasgd_nccl_unique_id(void *id128_host) {
  static_assert(sizeof(ncclUniqueId) == 128, "the id is documented as 128 bytes");
  if (!id128_host) return dasgd_internal_fail(nullptr, DASGD_ERR_INVALID_ARG, "nccl_unique_id: NULL buffer");
  NcclApi *a = nccl();
  if (!a) return unavailable();
  ncclUniqueId id;
  const ncclResult_t r = a->GetUniqueId(&id);
  if (r != ncclSuccess) return nccl_fail(a, r, "ncclGetUniqueId");
  memcpy(id128_host, &id, sizeof id);
  return DASGD_OK;
}

dasgd_status dasgd_nccl_comm_init(void **comm, const void *id128_host, int32_t nranks, int32_t rank, int32_t device) {
  if (!comm || !id128_host || nranks < 1 || rank < 0 || rank >= nranks)
    return dasgd_internal_fail(nullptr, DASGD_ERR_INVALID_ARG, "nccl_comm_init: need comm, id, 0 <= rank < nranks");
  *comm = nullptr;
  NcclApi *a = nccl();
  if (!a) return unavailable();
  int prev = -1;
  cudaError_t e = cudaGetDevice(&prev);
  if (e == cudaSuccess && prev != device) e = cudaSetDevice(device);
  if (e != cudaSuccess) return dasgd_internal_fail(nullptr, DASGD_ERR_CUDA, cudaGetErrorString(e));
  ncclUniqueId id;
  memcpy(&id, id128_host, sizeof id);
  ncclComm_t c = nullptr;
  const ncclResult_t r = a->CommInitRank(&c, nranks, id, rank);
  if (prev >= 0 && prev != device) cudaSetDevice(prev);
  if (r != ncclSuccess) return nccl_fail(a, r, "ncclCommInitRank");
  *comm = c;
  return DASGD_OK;
}

dasgd_status dasgd_nccl_comm_destroy(void *comm) {
  if (!comm) return DASGD_ERR_INVALID_ARG;
  NcclApi *a = nccl();
  if (!a) return unavailable();
  const ncclResult_t r = a->CommDestroy(static_cast<ncclComm_t>(comm));
  return r == ncclSuccess ? DASGD_OK : nccl_fail(a, r, "ncclCommDestroy");
}

dasgd_status dasgd_set_shard_nccl(dasgd_ctx *ctx, int32_t K_total, void *comm) {
  if (!ctx) return DASGD_ERR_INVALID_ARG;
  if (!comm) return dasgd_internal_fail(ctx, DASGD_ERR_INVALID_ARG, "set_shard_nccl: comm is NULL");
  if (!nccl()) return dasgd_internal_fail(ctx, DASGD_ERR_UNSUPPORTED, "set_shard_nccl: NCCL is not available");
  return dasgd_set_shard(ctx, K_total, nccl_exchange, comm);
}

}  // extern "C"
