// Peer mapping of source blobs for the exchange-free form of cross-GPU resharding: a rank exports
// a handle for each of its saved blobs, the other ranks map them, and their copy kernels then read
// the blobs in place (over NVLink when the owner is another GPU), tile by tile, with the same
// plain bulk loads they use for local memory.  Handles are CUDA IPC memory handles of the
// allocation that contains the pointer, plus the pointer's offset inside it, so buffers carved
// out of a larger pool (a framework's caching allocator) can be exported as they are.
#include <cstring>
#include <mutex>
#include <vector>

#include <cuda.h>

#include "kernels.cuh"
#include "plan.hpp"

namespace {

using namespace bcp;

static_assert(sizeof(cudaIpcMemHandle_t) == 64, "IPC memory handles are 64 bytes");
static_assert(sizeof(bcp_ipc_handle) == 96, "bcp_ipc_handle layout");

struct Mapping {  // one opened allocation of another process
  unsigned char handle[64];
  int device;
  char* base;
  uint64_t bytes;  // size of the mapped allocation
  unsigned refs;
};
std::mutex g_mu;
std::vector<Mapping> g_maps;

typedef CUresult (*AddressRangeFn)(CUdeviceptr*, size_t*, CUdeviceptr);
int address_range_fn(AddressRangeFn* out) {
  static AddressRangeFn fn = nullptr;
  if (!fn) {
    void* sym = nullptr;
    cudaDriverEntryPointQueryResult q;
    cudaError_t e = cudaGetDriverEntryPoint("cuMemGetAddressRange", &sym, cudaEnableDefault, &q);
    if (e != cudaSuccess || q != cudaDriverEntryPointSuccess || !sym) {
      cudaGetLastError();
      return fail(BCP_ERR_CUDA, "cuMemGetAddressRange is not available in this driver");
    }
    fn = reinterpret_cast<AddressRangeFn>(sym);
  }
  *out = fn;
  return BCP_OK;
}

}  // namespace

extern "C" {

int bcp_ipc_export(const void* dev_ptr, bcp_ipc_handle* out) {
  if (!dev_ptr || !out) return fail(BCP_ERR_INVALID, "bcp_ipc_export: NULL argument");
  AddressRangeFn range;
  if (int rc = address_range_fn(&range)) return rc;
  CUdeviceptr base = 0;
  size_t size = 0;
  const CUresult r = range(&base, &size, reinterpret_cast<CUdeviceptr>(dev_ptr));
  if (r != CUDA_SUCCESS) return fail(BCP_ERR_CUDA, "bcp_ipc_export: %p is not inside a device allocation (driver code %d)", dev_ptr, int(r));
  cudaIpcMemHandle_t h;
  const cudaError_t e = cudaIpcGetMemHandle(&h, reinterpret_cast<void*>(base));
  if (e != cudaSuccess) {
    cudaGetLastError();
    return fail(BCP_ERR_CUDA, "cudaIpcGetMemHandle: %s (allocations of a virtual-memory pool cannot be exported this way)", cudaGetErrorString(e));
  }
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) {
    cudaGetLastError();
    return fail(BCP_ERR_CUDA, "cudaGetDevice failed");
  }
  bcp_ipc_handle tmp;
  memset(&tmp, 0, sizeof tmp);
  memcpy(tmp.handle, &h, 64);
  tmp.offset = reinterpret_cast<CUdeviceptr>(dev_ptr) - base;
  tmp.bytes_after = size - tmp.offset;
  tmp.device = dev;
  *out = tmp;
  return BCP_OK;
}

int bcp_ipc_open(const bcp_ipc_handle* h, void** out_ptr) {
  if (!h || !out_ptr) return fail(BCP_ERR_INVALID, "bcp_ipc_open: NULL argument");
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) {
    cudaGetLastError();
    return fail(BCP_ERR_CUDA, "cudaGetDevice failed");
  }
  std::lock_guard<std::mutex> lock(g_mu);
  for (Mapping& m : g_maps)
    if (m.device == dev && memcmp(m.handle, h->handle, 64) == 0) {  // an allocation is mapped once per process and device
      ++m.refs;
      *out_ptr = m.base + h->offset;
      return BCP_OK;
    }
  cudaIpcMemHandle_t ch;
  memcpy(&ch, h->handle, 64);
  void* base = nullptr;
  const cudaError_t e = cudaIpcOpenMemHandle(&base, ch, cudaIpcMemLazyEnablePeerAccess);
  if (e != cudaSuccess || !base) {
    cudaGetLastError();
    return fail(BCP_ERR_CUDA, "cudaIpcOpenMemHandle: %s (a handle cannot be opened by the process that exported it)", cudaGetErrorString(e));
  }
  Mapping m;
  memcpy(m.handle, h->handle, 64);
  m.device = dev;
  m.base = static_cast<char*>(base);
  m.bytes = h->offset + h->bytes_after;
  m.refs = 1;
  g_maps.push_back(m);
  *out_ptr = m.base + h->offset;
  return BCP_OK;
}

int bcp_ipc_close(void* ptr) {
  if (!ptr) return BCP_OK;
  std::lock_guard<std::mutex> lock(g_mu);
  Mapping* best = nullptr;  // the mapped allocation that contains ptr
  for (Mapping& m : g_maps)
    if (m.base <= static_cast<char*>(ptr) && static_cast<char*>(ptr) - m.base < ptrdiff_t(m.bytes ? m.bytes : 1)) best = &m;
  if (!best) return fail(BCP_ERR_INVALID, "bcp_ipc_close: %p was not returned by bcp_ipc_open", ptr);
  if (--best->refs == 0) {
    int cur = 0;
    cudaGetDevice(&cur);
    if (cur != best->device) cudaSetDevice(best->device);
    const cudaError_t e = cudaIpcCloseMemHandle(best->base);
    if (cur != best->device) cudaSetDevice(cur);
    *best = g_maps.back();
    g_maps.pop_back();
    if (e != cudaSuccess) {
      cudaGetLastError();
      return fail(BCP_ERR_CUDA, "cudaIpcCloseMemHandle: %s", cudaGetErrorString(e));
    }
  }
  return BCP_OK;
}

}  // extern "C"
