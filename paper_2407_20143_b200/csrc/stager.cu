// Asynchronous save / load staging through a pinned ping-pong pool.
//
// The paper's save pipeline copies every shard to pinned host memory (a pool with ping-pong
// buffering), then serialises and uploads in the background; only the device-to-host copy
// blocks training (Sec. 4.2).  Here the blocking part shrinks to the device-side pack: a
// rank's tensors are packed into a device slot on the caller's stream (bcp_pack), after which
// the tensors may change again, and the slot is copied to its pinned twin on a side stream.
// Slots alternate, so the pack of blob k+1 overlaps the download of blob k.  Loading is the
// mirror image: pinned slot -> device slot on the side stream, then unpack on the caller's stream.
#include <vector>

#include "kernels.cuh"
#include "plan.hpp"

using namespace bcp;

struct bcp_stager {
  enum State { FREE = 0, SAVING = 1, LOADING = 2, HELD = 3 };
  struct Slot {
    void* dev = nullptr;
    void* host = nullptr;
    cudaEvent_t packed = nullptr;  // device slot written (save) / consumed (load)
    cudaEvent_t moved = nullptr;   // host <-> device copy finished
    State state = FREE;
  };
  uint64_t slot_bytes = 0;
  int device = 0;
  cudaStream_t side = nullptr;
  std::vector<Slot> slots;
  uint32_t next = 0;
};

namespace {

#define BCP_ST_CUDA(call)                                                                    \
  do {                                                                                       \
    cudaError_t e_ = (call);                                                                 \
    if (e_ != cudaSuccess) return fail(BCP_ERR_CUDA, "%s: %s", #call, cudaGetErrorString(e_)); \
  } while (0)

int check_slot(const bcp_stager* s, uint32_t slot, const char* who) {
  if (!s) return fail(BCP_ERR_INVALID, "%s: stager is NULL", who);
  if (slot >= s->slots.size()) return fail(BCP_ERR_INVALID, "%s: slot %u of %zu", who, slot, s->slots.size());
  return BCP_OK;
}

int free_slot(bcp_stager* s, uint32_t* out) {
  for (size_t k = 0; k < s->slots.size(); ++k) {
    const uint32_t i = uint32_t((s->next + k) % s->slots.size());
    if (s->slots[i].state == bcp_stager::FREE) {
      s->next = uint32_t((i + 1) % s->slots.size());
      *out = i;
      return BCP_OK;
    }
  }
  return fail(BCP_ERR_CAPACITY, "every staging slot is in use: release one first");
}

void destroy(bcp_stager* s) {
  if (s->side) cudaStreamSynchronize(s->side);
  for (bcp_stager::Slot& sl : s->slots) {
    if (sl.packed) cudaEventDestroy(sl.packed);
    if (sl.moved) cudaEventDestroy(sl.moved);
    if (sl.dev) cudaFree(sl.dev);
    if (sl.host) cudaFreeHost(sl.host);
  }
  if (s->side) cudaStreamDestroy(s->side);
  cudaGetLastError();
  delete s;
}

int create(bcp_stager* s) {
  BCP_ST_CUDA(cudaGetDevice(&s->device));
  BCP_ST_CUDA(cudaStreamCreateWithFlags(&s->side, cudaStreamNonBlocking));
  for (bcp_stager::Slot& sl : s->slots) {
    BCP_ST_CUDA(cudaMalloc(&sl.dev, s->slot_bytes));
    BCP_ST_CUDA(cudaHostAlloc(&sl.host, s->slot_bytes, cudaHostAllocDefault));
    BCP_ST_CUDA(cudaEventCreateWithFlags(&sl.packed, cudaEventDisableTiming));
    BCP_ST_CUDA(cudaEventCreateWithFlags(&sl.moved, cudaEventDisableTiming));
  }
  return BCP_OK;
}

}  // namespace

extern "C" {

int bcp_stager_create(uint64_t slot_bytes, uint32_t n_slots, bcp_stager_t** out) {
  if (!out) return fail(BCP_ERR_INVALID, "bcp_stager_create: out is NULL");
  if (slot_bytes == 0 || slot_bytes % 256) return fail(BCP_ERR_INVALID, "bcp_stager_create: slot_bytes must be a positive multiple of 256");
  if (n_slots < 1 || n_slots > 16) return fail(BCP_ERR_INVALID, "bcp_stager_create: n_slots must be in [1, 16]");
  bcp_stager* s = new (std::nothrow) bcp_stager;
  if (!s) return fail(BCP_ERR_NOMEM, "out of host memory");
  s->slot_bytes = slot_bytes;
  s->slots.resize(n_slots);
  if (int rc = create(s)) {
    destroy(s);
    return rc;
  }
  *out = s;
  return BCP_OK;
}

int bcp_stager_destroy(bcp_stager_t* s) {
  if (!s) return BCP_OK;
  int cur = 0;
  cudaGetDevice(&cur);
  if (cur != s->device) cudaSetDevice(s->device);
  destroy(s);
  if (cur != s->device) cudaSetDevice(cur);
  return BCP_OK;
}

int bcp_stager_save(bcp_stager_t* s, const void* const* tensors, const bcp_pack_meta* metas, size_t n, uint64_t blob_bytes,
                    void* stream_, uint32_t* out_slot) {
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  if (!s || !out_slot) return fail(BCP_ERR_INVALID, "bcp_stager_save: NULL argument");
  if (blob_bytes > s->slot_bytes)
    return fail(BCP_ERR_CAPACITY, "bcp_stager_save: blob of %llu bytes, slots hold %llu", (unsigned long long)blob_bytes,
                (unsigned long long)s->slot_bytes);
  uint32_t i = 0;
  if (int rc = free_slot(s, &i)) return rc;
  bcp_stager::Slot& sl = s->slots[i];
  // if this slot last carried a load, its unpack (possibly on another stream) must be done reading
  BCP_ST_CUDA(cudaStreamWaitEvent(stream, sl.packed, 0));
  if (int rc = bcp_pack(tensors, metas, n, sl.dev, blob_bytes, stream)) return rc;
  BCP_ST_CUDA(cudaEventRecord(sl.packed, stream));  // from here on the caller's tensors may change again
  BCP_ST_CUDA(cudaStreamWaitEvent(s->side, sl.packed, 0));
  if (blob_bytes) BCP_ST_CUDA(cudaMemcpyAsync(sl.host, sl.dev, blob_bytes, cudaMemcpyDeviceToHost, s->side));
  BCP_ST_CUDA(cudaEventRecord(sl.moved, s->side));
  sl.state = bcp_stager::SAVING;
  *out_slot = i;
  return BCP_OK;
}

int bcp_stager_wait(bcp_stager_t* s, uint32_t slot, void** host_blob) {
  if (int rc = check_slot(s, slot, "bcp_stager_wait")) return rc;
  bcp_stager::Slot& sl = s->slots[slot];
  if (sl.state != bcp_stager::SAVING && sl.state != bcp_stager::HELD)
    return fail(BCP_ERR_INVALID, "bcp_stager_wait: slot %u holds no saved blob", slot);
  BCP_ST_CUDA(cudaEventSynchronize(sl.moved));
  if (host_blob) *host_blob = sl.host;
  return BCP_OK;
}

int bcp_stager_acquire(bcp_stager_t* s, uint32_t* out_slot, void** host_blob) {
  if (!s || !out_slot || !host_blob) return fail(BCP_ERR_INVALID, "bcp_stager_acquire: NULL argument");
  uint32_t i = 0;
  if (int rc = free_slot(s, &i)) return rc;
  // the device twin may still be read by the unpack of the blob this slot carried before
  BCP_ST_CUDA(cudaEventSynchronize(s->slots[i].packed));
  s->slots[i].state = bcp_stager::HELD;
  *out_slot = i;
  *host_blob = s->slots[i].host;
  return BCP_OK;
}

int bcp_stager_load(bcp_stager_t* s, uint32_t slot, uint64_t blob_bytes, const bcp_pack_meta* metas, size_t n,
                    void* const* tensors, void* stream_) {
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  if (int rc = check_slot(s, slot, "bcp_stager_load")) return rc;
  bcp_stager::Slot& sl = s->slots[slot];
  if (sl.state != bcp_stager::HELD) return fail(BCP_ERR_INVALID, "bcp_stager_load: slot %u was not acquired", slot);
  if (blob_bytes > s->slot_bytes) return fail(BCP_ERR_CAPACITY, "bcp_stager_load: blob larger than a slot");
  if (blob_bytes) BCP_ST_CUDA(cudaMemcpyAsync(sl.dev, sl.host, blob_bytes, cudaMemcpyHostToDevice, s->side));
  BCP_ST_CUDA(cudaEventRecord(sl.moved, s->side));
  BCP_ST_CUDA(cudaStreamWaitEvent(stream, sl.moved, 0));
  if (int rc = bcp_unpack(sl.dev, blob_bytes, metas, n, tensors, stream)) return rc;
  BCP_ST_CUDA(cudaEventRecord(sl.packed, stream));
  sl.state = bcp_stager::LOADING;
  return BCP_OK;
}

int bcp_stager_release(bcp_stager_t* s, uint32_t slot) {
  if (int rc = check_slot(s, slot, "bcp_stager_release")) return rc;
  bcp_stager::Slot& sl = s->slots[slot];
  if (sl.state == bcp_stager::FREE) return fail(BCP_ERR_INVALID, "bcp_stager_release: slot %u is not in use", slot);
  // a slot is reusable once its copy has finished (the unpack of a load is awaited at the next acquire)
  BCP_ST_CUDA(cudaEventSynchronize(sl.moved));
  sl.state = bcp_stager::FREE;
  return BCP_OK;
}

}  // extern "C"
