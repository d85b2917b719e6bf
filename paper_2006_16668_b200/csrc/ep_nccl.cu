// The collectives of the expert-parallel forward through NCCL itself (no callback into the caller's
// language): the AllToAll before and after the expert FFN (Algorithm 2) as grouped point-to-point
// sends and receives of equal slabs, and the all-reduce of the per-rank shares of l_aux.
//
// NCCL is not linked: its entry points are looked up in the process at run time (the framework that
// owns the communicator has loaded it already), by name, with the prototypes of its public header
// restated here.  Every buffer NCCL touches is a device buffer of the CALLING rank's own workspace;
// what crosses NVLink does so inside NCCL's kernels.
#include <dlfcn.h>

#include "kernels.cuh"

namespace gshard {

namespace {

// public NCCL ABI (nccl.h): result code 0 = success; data types ncclUint8 = 1, ncclFloat32 = 7; ncclSum = 0
typedef int (*NcclGroupFn)(void);
typedef int (*NcclSendFn)(const void*, size_t, int, int, void*, cudaStream_t);
typedef int (*NcclRecvFn)(void*, size_t, int, int, void*, cudaStream_t);
typedef int (*NcclAllReduceFn)(const void*, void*, size_t, int, int, void*, cudaStream_t);
constexpr int kNcclUint8 = 1, kNcclFloat32 = 7, kNcclSum = 0;

struct NcclState {          // lives in the caller's gshard_ep_nccl_state
  void* comm;
  int world;
  NcclGroupFn group_start, group_end;
  NcclSendFn send;
  NcclRecvFn recv;
  NcclAllReduceFn all_reduce;
};
static_assert(sizeof(NcclState) <= sizeof(gshard_ep_nccl_state), "state storage too small");

void* nccl_symbol(const char* name) {
  // the copy the process already uses, whatever file it came from; else the system's library
  void* f = dlsym(RTLD_DEFAULT, name);
  if (f) return f;
  static void* handle = dlopen("libnccl.so.2", RTLD_NOW | RTLD_GLOBAL);
  return handle ? dlsym(handle, name) : nullptr;
}

int nccl_all_to_all(void* user, const void* send, void* recv, size_t bytes_per_peer, void* cuda_stream) {
  const NcclState* s = static_cast<const NcclState*>(user);
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  const unsigned char* src = static_cast<const unsigned char*>(send);
  unsigned char* dst = static_cast<unsigned char*>(recv);
  if (s->group_start() != 0) return 1;
  int rc = 0;
  for (int peer = 0; peer < s->world && rc == 0; ++peer) {
    rc = s->send(src + (size_t)peer * bytes_per_peer, bytes_per_peer, kNcclUint8, peer, s->comm, st);
    if (rc == 0) rc = s->recv(dst + (size_t)peer * bytes_per_peer, bytes_per_peer, kNcclUint8, peer, s->comm, st);
  }
  const int rce = s->group_end();
  return (rc == 0 && rce == 0) ? 0 : 1;
}

int nccl_all_reduce_sum_f32(void* user, float* buf, size_t count, void* cuda_stream) {
  const NcclState* s = static_cast<const NcclState*>(user);
  return s->all_reduce(buf, buf, count, kNcclFloat32, kNcclSum, s->comm, static_cast<cudaStream_t>(cuda_stream)) == 0 ? 0 : 1;
}

}  // namespace

}  // namespace gshard

extern "C" int gshard_ep_comm_from_nccl(void* nccl_comm, int world, gshard_ep_nccl_state* state, gshard_ep_comm* comm) {
  using namespace gshard;
  if (!nccl_comm || world < 1 || !state || !comm) return GSHARD_ERR_INVALID_ARG;
  NcclState* s = reinterpret_cast<NcclState*>(state);
  s->comm = nccl_comm;
  s->world = world;
  s->group_start = reinterpret_cast<NcclGroupFn>(nccl_symbol("ncclGroupStart"));
  s->group_end = reinterpret_cast<NcclGroupFn>(nccl_symbol("ncclGroupEnd"));
  s->send = reinterpret_cast<NcclSendFn>(nccl_symbol("ncclSend"));
  s->recv = reinterpret_cast<NcclRecvFn>(nccl_symbol("ncclRecv"));
  s->all_reduce = reinterpret_cast<NcclAllReduceFn>(nccl_symbol("ncclAllReduce"));
  if (!s->group_start || !s->group_end || !s->send || !s->recv || !s->all_reduce) return GSHARD_ERR_INTERNAL;   // no NCCL in the process
  comm->all_to_all = nccl_all_to_all;
  comm->all_reduce_sum_f32 = nccl_all_reduce_sum_f32;
  comm->user = s;
  return GSHARD_OK;
}
