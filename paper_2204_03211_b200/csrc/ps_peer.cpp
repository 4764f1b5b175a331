// Peer buffers: device memory that other processes of the same node can map
// (declarations and contracts: include/ps_b200.h).  A block-sharded deployment
// runs one service per GPU, one process each; a worker's gradient shards live in
// a buffer exported by the worker's process, the owner of a block maps it and
// hands the mapped address to ps_push, and the aggregation kernel reads it in
// place (over NVLink when the two GPUs differ).
#include "../../include/ps_b200.h"

#include <cuda_runtime.h>

#include <cstring>
#include <string>

namespace {

thread_local std::string g_peer_err;

int fail(cudaError_t e) {
  g_peer_err = cudaGetErrorString(e);
  cudaGetLastError();
  return e == cudaErrorMemoryAllocation ? PS_ERR_NOMEM : PS_ERR_CUDA;
}

static_assert(sizeof(cudaIpcMemHandle_t) == PS_PEER_HANDLE_BYTES, "handle size");

}  // namespace

extern "C" {

int ps_peer_alloc(int device, size_t bytes, void** dev_ptr_out, unsigned char* handle_out) {
  if (!dev_ptr_out || !handle_out || bytes == 0 || device < 0) return PS_ERR_BAD_ARG;
  *dev_ptr_out = nullptr;
  cudaError_t e = cudaSetDevice(device);
  if (e != cudaSuccess) return fail(e);
  void* p = nullptr;
  e = cudaMalloc(&p, bytes);                 // its own allocation: the handle names the whole range
  if (e != cudaSuccess) return fail(e);
  cudaIpcMemHandle_t h;
  e = cudaIpcGetMemHandle(&h, p);
  if (e != cudaSuccess) {
    cudaFree(p);
    return fail(e);
  }
  std::memcpy(handle_out, &h, sizeof(h));
  *dev_ptr_out = p;
  return PS_OK;
}

int ps_peer_free(int device, void* dev_ptr) {
  if (!dev_ptr || device < 0) return PS_ERR_BAD_ARG;
  cudaError_t e = cudaSetDevice(device);
  if (e == cudaSuccess) e = cudaFree(dev_ptr);
  return e == cudaSuccess ? PS_OK : fail(e);
}

int ps_peer_open(int device, const unsigned char* handle, void** dev_ptr_out) {
  if (!dev_ptr_out || !handle || device < 0) return PS_ERR_BAD_ARG;
  *dev_ptr_out = nullptr;
  cudaError_t e = cudaSetDevice(device);
  if (e != cudaSuccess) return fail(e);
  cudaIpcMemHandle_t h;
  std::memcpy(&h, handle, sizeof(h));
  void* p = nullptr;
  e = cudaIpcOpenMemHandle(&p, h, cudaIpcMemLazyEnablePeerAccess);
  if (e != cudaSuccess) return fail(e);
  *dev_ptr_out = p;
  return PS_OK;
}

int ps_peer_close(int device, void* dev_ptr) {
  if (!dev_ptr || device < 0) return PS_ERR_BAD_ARG;
  cudaError_t e = cudaSetDevice(device);
  if (e == cudaSuccess) e = cudaIpcCloseMemHandle(dev_ptr);
  return e == cudaSuccess ? PS_OK : fail(e);
}

// Interprocess events: how one process's stream waits for another process's copy
// without either host waiting for its device.
static_assert(sizeof(cudaIpcEventHandle_t) == PS_PEER_HANDLE_BYTES, "event handle size");

int ps_peer_event_create(int device, void** event_out, unsigned char* handle_out) {
  if (!event_out || !handle_out || device < 0) return PS_ERR_BAD_ARG;
  *event_out = nullptr;
  cudaError_t e = cudaSetDevice(device);
  if (e != cudaSuccess) return fail(e);
  cudaEvent_t ev = nullptr;
  e = cudaEventCreateWithFlags(&ev, cudaEventDisableTiming | cudaEventInterprocess);
  if (e != cudaSuccess) return fail(e);
  cudaIpcEventHandle_t h;
  e = cudaIpcGetEventHandle(&h, ev);
  if (e != cudaSuccess) {
    cudaEventDestroy(ev);
    return fail(e);
  }
  std::memcpy(handle_out, &h, sizeof(h));
  *event_out = ev;
  return PS_OK;
}

int ps_peer_event_open(int device, const unsigned char* handle, void** event_out) {
  if (!event_out || !handle || device < 0) return PS_ERR_BAD_ARG;
  *event_out = nullptr;
  cudaError_t e = cudaSetDevice(device);
  if (e != cudaSuccess) return fail(e);
  cudaIpcEventHandle_t h;
  std::memcpy(&h, handle, sizeof(h));
  cudaEvent_t ev = nullptr;
  e = cudaIpcOpenEventHandle(&ev, h);
  if (e != cudaSuccess) return fail(e);
  *event_out = ev;
  return PS_OK;
}

int ps_peer_event_record(void* event, void* stream) {
  if (!event) return PS_ERR_BAD_ARG;
  cudaError_t e = cudaEventRecord(static_cast<cudaEvent_t>(event), static_cast<cudaStream_t>(stream));
  return e == cudaSuccess ? PS_OK : fail(e);
}

int ps_peer_event_wait(void* event, void* stream) {
  if (!event) return PS_ERR_BAD_ARG;
  cudaError_t e = cudaStreamWaitEvent(static_cast<cudaStream_t>(stream), static_cast<cudaEvent_t>(event), 0);
  return e == cudaSuccess ? PS_OK : fail(e);
}

int ps_peer_event_destroy(void* event) {
  if (!event) return PS_ERR_BAD_ARG;
  cudaError_t e = cudaEventDestroy(static_cast<cudaEvent_t>(event));
  return e == cudaSuccess ? PS_OK : fail(e);
}

int ps_peer_copy_many(int n, void* const* dsts, const void* const* srcs, const size_t* bytes, void* stream) {
  if (n < 0 || (n > 0 && (!dsts || !srcs || !bytes))) return PS_ERR_BAD_ARG;
  for (int i = 0; i < n; ++i) {
    if (!bytes[i]) continue;
    if (!dsts[i] || !srcs[i]) return PS_ERR_BAD_ARG;
    // one plain copy per range, by the copy engines: the ranges may lie in a peer's memory
    cudaError_t e = cudaMemcpyAsync(dsts[i], srcs[i], bytes[i], cudaMemcpyDefault, static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) return fail(e);
  }
  return PS_OK;
}

const char* ps_peer_last_error(void) { return g_peer_err.c_str(); }

}  // extern "C"
