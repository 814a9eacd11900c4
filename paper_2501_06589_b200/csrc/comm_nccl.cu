// Tensor-parallel exchange over NCCL (paper Sec. 2, Eq. 1: the all-reduce behind the output projection of the
// attention module and the down projection of the MLP module; Algorithm 1 runs it asynchronously).
// One communicator per rank = per process = per GPU.  The NCCL library is looked up at run time (the one the
// process has already loaded, e.g. PyTorch's, else the system's), so the library loads without it and a
// single-GPU user never touches it.  Host code only: the reduction itself is NCCL's kernel on the stream it is given.
#include <cuda_runtime.h>
#include <dlfcn.h>
#if __has_include(<nccl.h>)
#include <nccl.h>
#else
// No NCCL header on the build machine: the handful of declarations this file needs, as NCCL's public interface
// has had them since 2.0 (the library itself is only ever looked up at run time).
typedef struct ncclComm* ncclComm_t;
typedef struct {
  char internal[128];
} ncclUniqueId;
typedef enum { ncclSuccess = 0 } ncclResult_t;
typedef enum { ncclFloat32 = 7 } ncclDataType_t;
typedef enum { ncclSum = 0 } ncclRedOp_t;
#endif

#include <mutex>

#include "../../include/ladder.h"

struct ladder_comm {
  ncclComm_t comm = nullptr;
  int world = 0, rank = 0;
};

namespace {

struct NcclApi {
  void* lib = nullptr;
  ncclResult_t (*get_unique_id)(ncclUniqueId*) = nullptr;
  ncclResult_t (*comm_init_rank)(ncclComm_t*, int, ncclUniqueId, int) = nullptr;
  ncclResult_t (*comm_destroy)(ncclComm_t) = nullptr;
  ncclResult_t (*all_reduce)(const void*, void*, size_t, ncclDataType_t, ncclRedOp_t, ncclComm_t, cudaStream_t) = nullptr;
  bool ok = false;
};

NcclApi* nccl_api() {
  static NcclApi api;
  static std::once_flag once;
  std::call_once(once, [] {
    for (const char* name : {"libnccl.so.2", "libnccl.so"}) {
      api.lib = dlopen(name, RTLD_NOW | RTLD_GLOBAL);
      if (api.lib) break;
    }
    if (!api.lib) return;
    api.get_unique_id = reinterpret_cast<decltype(api.get_unique_id)>(dlsym(api.lib, "ncclGetUniqueId"));
    api.comm_init_rank = reinterpret_cast<decltype(api.comm_init_rank)>(dlsym(api.lib, "ncclCommInitRank"));
    api.comm_destroy = reinterpret_cast<decltype(api.comm_destroy)>(dlsym(api.lib, "ncclCommDestroy"));
    api.all_reduce = reinterpret_cast<decltype(api.all_reduce)>(dlsym(api.lib, "ncclAllReduce"));
    api.ok = api.get_unique_id && api.comm_init_rank && api.comm_destroy && api.all_reduce;
  });
  return api.ok ? &api : nullptr;
}

static_assert(sizeof(ncclUniqueId) == LADDER_COMM_ID_BYTES, "unique id size");

}  // namespace

extern "C" {

ladder_status_t ladder_comm_unique_id(void* id) {
  if (!id) return LADDER_ERR_INVALID_ARG;
  NcclApi* a = nccl_api();
  if (!a) return LADDER_ERR_UNSUPPORTED;
  return a->get_unique_id(static_cast<ncclUniqueId*>(id)) == ncclSuccess ? LADDER_OK : LADDER_ERR_CUDA;
}

ladder_status_t ladder_comm_create(int32_t world, int32_t rank, const void* id, ladder_comm_t** out) {
  if (!id || !out || world < 1 || rank < 0 || rank >= world) return LADDER_ERR_INVALID_ARG;
  *out = nullptr;
  NcclApi* a = nccl_api();
  if (!a) return LADDER_ERR_UNSUPPORTED;
  ladder_comm* c = new ladder_comm();
  c->world = world;
  c->rank = rank;
  if (a->comm_init_rank(&c->comm, world, *static_cast<const ncclUniqueId*>(id), rank) != ncclSuccess) {
    delete c;
    return LADDER_ERR_CUDA;
  }
  *out = c;
  return LADDER_OK;
}

ladder_status_t ladder_comm_destroy(ladder_comm_t* c) {
  if (!c) return LADDER_OK;
  NcclApi* a = nccl_api();
  ladder_status_t s = LADDER_OK;
  if (a && c->comm && a->comm_destroy(c->comm) != ncclSuccess) s = LADDER_ERR_CUDA;
  delete c;
  return s;
}

int32_t ladder_comm_world(const ladder_comm_t* c) { return c ? c->world : 0; }
int32_t ladder_comm_rank(const ladder_comm_t* c) { return c ? c->rank : -1; }

ladder_status_t ladder_comm_all_reduce_sum(void* comm, float* partial, int64_t count, void* cuda_stream) {
  ladder_comm* c = static_cast<ladder_comm*>(comm);
  if (!c || !c->comm || !partial || count < 0) return LADDER_ERR_INVALID_ARG;
  NcclApi* a = nccl_api();
  if (!a) return LADDER_ERR_UNSUPPORTED;
  if (count == 0) return LADDER_OK;
  return a->all_reduce(partial, partial, static_cast<size_t>(count), ncclFloat32, ncclSum, c->comm,
                       static_cast<cudaStream_t>(cuda_stream)) == ncclSuccess
             ? LADDER_OK
             : LADDER_ERR_CUDA;
}

}  // extern "C"
