// Shard extract for callers that cannot allocate device memory.
//
// tm_shard_extract needs a small device-resident work list and asks its caller for the scratch to
// hold it.  Some callers have no way to provide that: a recovery hook that runs while the training
// framework's caching allocator already owns the whole GPU, a handler that must not call cudaMalloc
// because that call synchronises the device and may fail exactly when memory is exhausted, or a
// plugin that is handed tensors but no allocator.  For them this file keeps the scratch inside the
// library itself, as a fixed array in device global memory, and exports one extra entry point.
//
// Rules that follow from that choice:
//   * the array is TM_STATIC_SCRATCH_BYTES long on every GPU whose context loads this library and
//     stays resident until the process exits;
//   * a request whose work list does not fit is refused with TM_ERR_CAPACITY, nothing is launched;
//   * all calls on one GPU share the one array and it still holds the previous call's list, so the
//     status block is cleared on every call and two calls whose device work may overlap (different
//     streams) would overwrite each other's list: issue them on one stream;
//   * the host side of a call — clear, two list copies, launch — runs under one lock, so threads that
//     share a stream cannot interleave their sequences;
//   * the list is copied from ordinary (pageable) host memory: the call returns once the stream has
//     taken the copies, which may mean waiting for earlier work in that stream;
//   * the first call on each GPU looks up the array's device address (cudaGetSymbolAddress) with that
//     GPU current; make that first call outside any stream capture.
// No cudaMalloc, cudaFree or other allocating routine is called here.
#include <cuda_runtime.h>

#include <mutex>
#include <new>

#include "tm_internal.h"

// In host code this name is only a handle for the runtime, not a device address: never pass it to a
// kernel.  The address comes from cudaGetSymbolAddress below.
static __device__ __align__(256) unsigned char g_static_scratch[TM_STATIC_SCRATCH_BYTES];

namespace {

constexpr int kMaxDevices = 64;
std::mutex g_mutex;
uint8_t* g_scratch_addr[kMaxDevices] = {nullptr};

// Device address of the scratch array on the current device; looked up once per device.  The caller
// holds g_mutex.
cudaError_t scratch_for_current_device(uint8_t** out) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  if (g_scratch_addr[dev] == nullptr) {
    void* p = nullptr;
    e = cudaGetSymbolAddress(&p, g_static_scratch);
    if (e != cudaSuccess) return e;
    g_scratch_addr[dev] = static_cast<uint8_t*>(p);
  }
  *out = g_scratch_addr[dev];
  return cudaSuccess;
}

}  // namespace

static int extract_static(const tm_desc* plane_descs, uint64_t n_desc, uint32_t r, uint32_t D, void* d_out,
                          uint64_t out_capacity, uint64_t* out_elems, void* stream) {
  uint32_t e = 0;
  uint64_t n_elems = 0;
  int rc = tm_shard_validate(plane_descs, n_desc, r, D, &e, &n_elems);
  if (rc != TM_OK) return rc;
  uint64_t lo = 0, hi = 0;
  rc = tm_bounds_u128(n_elems, r, D, &lo, &hi);
  if (rc != TM_OK) return rc;
  if (out_elems != nullptr) *out_elems = hi - lo;
  if (hi == lo) return TM_OK;
  if (d_out == nullptr) return TM_ERR_ARG;
  if (((uintptr_t)d_out & 1) != 0) return TM_ERR_ALIGN;
  const uint64_t out_bytes = (hi - lo) * e;
  if (out_capacity < out_bytes) return TM_ERR_CAPACITY;
  // refuse oversized requests from the byte count alone, before building any list
  const tms::Tuning opt = tms::tuning();
  const uint64_t min_segs = out_bytes / opt.shard_chunk_bytes;
  if (tms::workspace_layout(min_segs, 1).total > TM_STATIC_SCRATCH_BYTES) return TM_ERR_CAPACITY;
  const uint64_t out_addr = (uint64_t)(uintptr_t)d_out;
  for (uint64_t k = 0; k < n_desc; ++k)
    if (tms::ranges_overlap((uint64_t)(uintptr_t)plane_descs[k].ptr, plane_descs[k].nbytes, out_addr, out_bytes))
      return TM_ERR_OVERLAP;
  tms::WorkList wl;
  tm_shard_worklist(opt, plane_descs, n_desc, e, lo, hi, out_addr, &wl);
  const tms::WorkspaceLayout l = tms::workspace_layout(wl.segs.size(), wl.n_items());
  if (l.total > TM_STATIC_SCRATCH_BYTES) return TM_ERR_CAPACITY;

  // One lock around the address lookup and the whole clear / copy / copy / launch sequence: two threads
  // that issue on the same stream cannot interleave, so each kernel reads the list its own call wrote.
  std::lock_guard<std::mutex> lock(g_mutex);
  uint8_t* scratch = nullptr;
  cudaError_t ce = scratch_for_current_device(&scratch);
  if (ce != cudaSuccess) return tms::cuda_fail((int)ce);
  cudaStream_t st = (cudaStream_t)stream;
  // the array still holds the previous call's status block and list: clear the former, overwrite the latter
  if ((ce = cudaMemsetAsync(scratch, 0, tms::kStatusBlockBytes, st)) != cudaSuccess) return tms::cuda_fail((int)ce);
  if ((ce = cudaMemcpyAsync(scratch + l.segs_off, wl.segs.data(), wl.segs.size() * sizeof(tms::Seg),
                            cudaMemcpyHostToDevice, st)) != cudaSuccess) return tms::cuda_fail((int)ce);
  if ((ce = cudaMemcpyAsync(scratch + l.items_off, wl.item_first.data(), wl.item_first.size() * sizeof(uint32_t),
                            cudaMemcpyHostToDevice, st)) != cudaSuccess) return tms::cuda_fail((int)ce);
  const int err = tms::launch_copy_to_flat((const tms::Seg*)(scratch + l.segs_off),
                                           (const uint32_t*)(scratch + l.items_off), (uint32_t)wl.n_items(),
                                           (uint8_t*)d_out, opt.ctas_per_sm, stream);
  return err == 0 ? TM_OK : tms::cuda_fail(err);
}

extern "C" int tm_shard_extract_static(const tm_desc* plane_descs, uint64_t n_desc, uint32_t r, uint32_t D,
                                       void* d_out, uint64_t out_capacity, uint64_t* out_elems,
                                       void* stream) {
  try {
    return extract_static(plane_descs, n_desc, r, D, d_out, out_capacity, out_elems, stream);
  } catch (const std::bad_alloc&) {
    return TM_ERR_CAPACITY;
  } catch (...) {
    return TM_ERR_ARG;
  }
}
