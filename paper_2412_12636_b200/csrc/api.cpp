// C ABI of the role-state mover (declared in include/tm_state.h): argument validation, work-list
// upload and kernel launches.  Nothing here computes on the CPU what the kernels are for; without
// a CUDA device every operation fails with TM_ERR_CUDA.
#include <cuda_runtime.h>

#include <algorithm>
#include <atomic>
#include <cstring>
#include <mutex>
#include <new>
#include <vector>

#include "tm_internal.h"

int tm_plan_build(tm_plan* p, const tm_desc* descs, uint64_t n_desc, uint64_t bucket_bytes);
int tm_bounds_u128(uint64_t n_elems, uint32_t r, uint32_t D, uint64_t* lo, uint64_t* hi);
int tm_shard_validate(const tm_desc* descs, uint64_t n_desc, uint32_t r, uint32_t D,
                      uint32_t* elem_size, uint64_t* n_elems);
void tm_shard_worklist(const tm_desc* descs, uint64_t n_desc, uint32_t e, uint64_t lo, uint64_t hi,
                       uint64_t d_out, tms::WorkList* wl);
int tm_targets_disjoint(const tm_plan* p);
void tm_shard_append(tms::WorkListBuilder* builder, const tm_desc* descs, uint64_t n_desc, uint32_t e,
                     uint64_t lo, uint64_t hi, uint64_t d_out, uint64_t flat_base, uint32_t bucket_tag);

namespace {

std::atomic<int> g_last_cuda_error{0};

int cuda_fail(int e) {
  g_last_cuda_error.store(e);
  return TM_ERR_CUDA;
}
#define TM_CUDA(call)                              \
  do {                                             \
    cudaError_t e__ = (call);                      \
    if (e__ != cudaSuccess) return cuda_fail((int)e__); \
  } while (0)

bool ranges_overlap(uint64_t a, uint64_t an, uint64_t b, uint64_t bn) {
  return a < b + bn && b < a + an;
}

// Pinned host staging for small work-list uploads: eight 1 MiB slots per device, reused round-robin;
// a slot is free again once the copy that read it has completed (one event per slot).  Host memory
// only.  With it an upload is one truly asynchronous copy instead of a memset plus two copies from
// pageable memory that make the host wait for the stream.
class HostStaging {
 public:
  static constexpr size_t kSlotBytes = 1u << 20;
  static constexpr int kSlots = 8;
  static constexpr int kMaxDevices = 64;

  // Returns a slot for the current device (waiting for its previous copy), or -1 if unavailable.
  int acquire(int dev) {
    if (dev < 0 || dev >= kMaxDevices) return -1;
    Pool& p = pools_[dev];
    if (p.state == 0) {
      p.state = -1;
      uint8_t* base = nullptr;
      if (cudaHostAlloc((void**)&base, kSlotBytes * kSlots, cudaHostAllocPortable) == cudaSuccess) {
        bool ok = true;
        for (int i = 0; i < kSlots && ok; ++i) {
          p.host[i] = base + (size_t)i * kSlotBytes;
          ok = cudaEventCreateWithFlags(&p.ev[i], cudaEventDisableTiming) == cudaSuccess;
        }
        if (ok) p.state = 1;
      }
      (void)cudaGetLastError();
    }
    if (p.state != 1) return -1;
    const int i = p.next;
    p.next = (p.next + 1) % kSlots;
    if (p.busy[i] && cudaEventSynchronize(p.ev[i]) != cudaSuccess) return -1;
    p.busy[i] = false;
    return i;
  }
  uint8_t* host(int dev, int slot) { return pools_[dev].host[slot]; }
  cudaError_t mark(int dev, int slot, cudaStream_t st) {
    pools_[dev].busy[slot] = true;
    return cudaEventRecord(pools_[dev].ev[slot], st);
  }
  std::mutex mutex;

 private:
  struct Pool {
    int state = 0;   // 0 not tried, 1 ready, -1 unavailable
    int next = 0;
    uint8_t* host[kSlots] = {nullptr};
    cudaEvent_t ev[kSlots] = {nullptr};
    bool busy[kSlots] = {false};
  };
  Pool pools_[kMaxDevices];
};
HostStaging g_staging;

int upload_worklist(const tms::WorkList& wl, const tms::WorkspaceLayout& l, uint8_t* d_ws, cudaStream_t st) {
  const size_t items_bytes = wl.item_first.size() * sizeof(uint32_t);
  const size_t segs_bytes = wl.segs.size() * sizeof(tms::Seg);
  const size_t span = l.items_off + items_bytes;   // status block, pieces, items: one contiguous image
  if (span <= HostStaging::kSlotBytes) {
    int dev = 0;
    if (cudaGetDevice(&dev) == cudaSuccess) {
      std::lock_guard<std::mutex> lock(g_staging.mutex);
      const int slot = g_staging.acquire(dev);
      if (slot >= 0) {
        uint8_t* h = g_staging.host(dev, slot);
        std::memset(h, 0, l.segs_off);
        if (segs_bytes != 0) std::memcpy(h + l.segs_off, wl.segs.data(), segs_bytes);
        std::memset(h + l.segs_off + segs_bytes, 0, l.items_off - l.segs_off - segs_bytes);
        std::memcpy(h + l.items_off, wl.item_first.data(), items_bytes);
        TM_CUDA(cudaMemcpyAsync(d_ws, h, span, cudaMemcpyHostToDevice, st));
        TM_CUDA(g_staging.mark(dev, slot, st));
        return TM_OK;
      }
    }
  }
  TM_CUDA(cudaMemsetAsync(d_ws, 0, tms::kStatusBlockBytes, st));
  if (segs_bytes != 0)
    TM_CUDA(cudaMemcpyAsync(d_ws + l.segs_off, wl.segs.data(), segs_bytes, cudaMemcpyHostToDevice, st));
  TM_CUDA(cudaMemcpyAsync(d_ws + l.items_off, wl.item_first.data(), items_bytes, cudaMemcpyHostToDevice, st));
  return TM_OK;
}

int read_status(const void* d_ws, cudaStream_t st, int* device_status) {
  if (d_ws == nullptr || device_status == nullptr) return TM_ERR_ARG;
  int word = 0;
  TM_CUDA(cudaMemcpyAsync(&word, d_ws, sizeof(int), cudaMemcpyDeviceToHost, st));
  TM_CUDA(cudaStreamSynchronize(st));
  *device_status = word;
  return TM_OK;
}

}  // namespace

extern "C" {

int tm_plan_create(const tm_desc* descs, uint64_t n_desc, uint64_t bucket_bytes, tm_plan** out) {
  if (out == nullptr) return TM_ERR_ARG;
  *out = nullptr;
  tm_plan* p = new (std::nothrow) tm_plan();
  if (p == nullptr) return TM_ERR_ARG;
  int rc = tm_plan_build(p, descs, n_desc, bucket_bytes);
  if (rc != TM_OK) {
    delete p;
    return rc;
  }
  *out = p;
  return TM_OK;
}

int tm_plan_query(const tm_plan* plan, uint64_t* total_bytes, uint64_t* n_buckets,
                  uint64_t* workspace_bytes) {
  if (plan == nullptr) return TM_ERR_ARG;
  if (total_bytes != nullptr) *total_bytes = plan->total_bytes;
  if (n_buckets != nullptr) *n_buckets = plan->n_buckets;
  if (workspace_bytes != nullptr) *workspace_bytes = plan->ws_layout.total;
  return TM_OK;
}

int tm_plan_offsets(const tm_plan* plan, uint64_t* offsets) {
  if (plan == nullptr || offsets == nullptr) return TM_ERR_ARG;
  std::memcpy(offsets, plan->offsets.data(), plan->offsets.size() * sizeof(uint64_t));
  return TM_OK;
}

int tm_plan_pieces(const tm_plan* plan, tm_piece* pieces, uint64_t capacity, uint64_t* n_pieces,
                   uint32_t* item_first, uint64_t item_capacity, uint64_t* n_items) {
  if (plan == nullptr) return TM_ERR_ARG;
  static_assert(sizeof(tm_piece) == sizeof(tms::Seg), "tm_piece mirrors the internal piece");
  const uint64_t np = plan->work.segs.size(), ni = plan->work.n_items();
  if (n_pieces != nullptr) *n_pieces = np;
  if (n_items != nullptr) *n_items = ni;
  if (pieces != nullptr) std::memcpy(pieces, plan->work.segs.data(), std::min(np, capacity) * sizeof(tm_piece));
  if (item_first != nullptr)
    std::memcpy(item_first, plan->work.item_first.data(), std::min(ni + 1, item_capacity) * sizeof(uint32_t));
  return TM_OK;
}

int tm_plan_upload(tm_plan* plan, void* d_workspace, uint64_t workspace_bytes, void* stream) {
  if (plan == nullptr || d_workspace == nullptr) return TM_ERR_ARG;
  if (((uintptr_t)d_workspace & 255) != 0) return TM_ERR_ALIGN;
  if (workspace_bytes < plan->ws_layout.total) return TM_ERR_CAPACITY;
  int rc = upload_worklist(plan->work, plan->ws_layout, (uint8_t*)d_workspace, (cudaStream_t)stream);
  if (rc != TM_OK) return rc;
  plan->d_workspace = (uint8_t*)d_workspace;
  return TM_OK;
}

int tm_plan_status(const tm_plan* plan, void* stream, int* device_status) {
  if (plan == nullptr || device_status == nullptr) return TM_ERR_ARG;
  if (plan->d_workspace == nullptr && plan->d_emit_workspace == nullptr) return TM_ERR_STATE;
  int a = 0, b = 0;
  if (plan->d_workspace != nullptr) {
    int rc = read_status(plan->d_workspace, (cudaStream_t)stream, &a);
    if (rc != TM_OK) return rc;
  }
  if (plan->d_emit_workspace != nullptr) {
    int rc = read_status(plan->d_emit_workspace, (cudaStream_t)stream, &b);
    if (rc != TM_OK) return rc;
  }
  *device_status = (a != 0) ? a : b;
  return TM_OK;
}

void tm_plan_destroy(tm_plan* plan) { delete plan; }

int tm_state_pack(const tm_plan* plan, void* d_buckets, uint64_t capacity, uint64_t* d_checksums,
                  void* stream) {
  if (plan == nullptr || d_buckets == nullptr) return TM_ERR_ARG;
  if (plan->d_workspace == nullptr) return TM_ERR_STATE;
  if (((uintptr_t)d_buckets & 255) != 0 || ((uintptr_t)d_checksums & 7) != 0) return TM_ERR_ALIGN;
  if (capacity < plan->total_bytes) return TM_ERR_CAPACITY;
  const uint64_t base = (uint64_t)(uintptr_t)d_buckets;
  for (const tm_desc& d : plan->descs)
    if (ranges_overlap((uint64_t)(uintptr_t)d.ptr, d.nbytes, base, plan->total_bytes)) return TM_ERR_OVERLAP;
  cudaStream_t st = (cudaStream_t)stream;
  if (d_checksums != nullptr)
    TM_CUDA(cudaMemsetAsync(d_checksums, 0, plan->n_buckets * sizeof(uint64_t), st));
  const uint8_t* ws = plan->d_workspace;
  auto pack_fn = tms::tuning().use_ring ? tms::launch_pack_ring : tms::launch_pack;
  int e = pack_fn((const tms::Seg*)(ws + plan->ws_layout.segs_off),
                          (const uint32_t*)(ws + plan->ws_layout.items_off),
                          (uint32_t)plan->work.n_items(), (uint8_t*)d_buckets,
                          (unsigned long long*)d_checksums, (int*)plan->d_workspace, stream);
  return e == 0 ? TM_OK : cuda_fail(e);
}

int tm_state_unpack(const tm_plan* plan, const void* d_buckets, uint64_t nbytes, void* stream) {
  if (plan == nullptr || d_buckets == nullptr) return TM_ERR_ARG;
  if (plan->d_workspace == nullptr) return TM_ERR_STATE;
  if (((uintptr_t)d_buckets & 255) != 0) return TM_ERR_ALIGN;
  if (nbytes < plan->total_bytes) return TM_ERR_CAPACITY;
  const uint64_t base = (uint64_t)(uintptr_t)d_buckets;
  for (const tm_desc& d : plan->descs)
    if (ranges_overlap((uint64_t)(uintptr_t)d.ptr, d.nbytes, base, plan->total_bytes)) return TM_ERR_OVERLAP;
  if (plan->targets_disjoint == 0) plan->targets_disjoint = tm_targets_disjoint(plan);
  if (plan->targets_disjoint < 0) return TM_ERR_OVERLAP;
  const uint8_t* ws = plan->d_workspace;
  auto copy_fn = tms::tuning().use_ring ? tms::launch_copy_ring : tms::launch_copy;
  int e = copy_fn((const tms::Seg*)(ws + plan->ws_layout.segs_off),
                          (const uint32_t*)(ws + plan->ws_layout.items_off),
                          (uint32_t)plan->work.n_items(), (uint8_t*)const_cast<void*>(d_buckets),
                          /*to_tensors=*/true, (int*)plan->d_workspace, stream);
  return e == 0 ? TM_OK : cuda_fail(e);
}

int tm_state_unpack_verify(const tm_plan* plan, const void* d_buckets, uint64_t nbytes, uint64_t* d_checksums,
                           void* stream) {
  if (plan == nullptr || d_buckets == nullptr || d_checksums == nullptr) return TM_ERR_ARG;
  if (plan->d_workspace == nullptr) return TM_ERR_STATE;
  if (((uintptr_t)d_buckets & 255) != 0 || ((uintptr_t)d_checksums & 7) != 0) return TM_ERR_ALIGN;
  if (nbytes < plan->total_bytes) return TM_ERR_CAPACITY;
  const uint64_t base = (uint64_t)(uintptr_t)d_buckets;
  for (const tm_desc& d : plan->descs)
    if (ranges_overlap((uint64_t)(uintptr_t)d.ptr, d.nbytes, base, plan->total_bytes)) return TM_ERR_OVERLAP;
  if (plan->targets_disjoint == 0) plan->targets_disjoint = tm_targets_disjoint(plan);
  if (plan->targets_disjoint < 0) return TM_ERR_OVERLAP;
  TM_CUDA(cudaMemsetAsync(d_checksums, 0, plan->n_buckets * sizeof(uint64_t), (cudaStream_t)stream));
  const uint8_t* ws = plan->d_workspace;
  int e = tms::launch_unpack_verify_ring((const tms::Seg*)(ws + plan->ws_layout.segs_off),
                                         (const uint32_t*)(ws + plan->ws_layout.items_off),
                                         (uint32_t)plan->work.n_items(), (uint8_t*)const_cast<void*>(d_buckets),
                                         (unsigned long long*)d_checksums, (int*)plan->d_workspace, stream);
  return e == 0 ? TM_OK : cuda_fail(e);
}

int tm_plan_attach_shards(tm_plan* plan, const uint64_t* plane_first_desc, const uint64_t* plane_n_desc,
                          uint32_t n_planes, uint32_t r, uint32_t D, void* const* d_outs,
                          const uint64_t* out_capacities, uint64_t* out_elems, void* d_workspace,
                          uint64_t workspace_bytes, uint64_t* workspace_needed, void* stream) {
  if (plan == nullptr || plane_first_desc == nullptr || plane_n_desc == nullptr || n_planes == 0)
    return TM_ERR_ARG;
  if (D == 0 || r >= D) return TM_ERR_RANK;
  const uint64_t n_desc = plan->descs.size();
  struct PlaneInfo { uint64_t first, n; uint32_t e; uint64_t lo, hi; };
  std::vector<PlaneInfo> planes(n_planes);
  uint64_t prev_end = 0;
  for (uint32_t p = 0; p < n_planes; ++p) {
    PlaneInfo& pi = planes[p];
    pi.first = plane_first_desc[p];
    pi.n = plane_n_desc[p];
    if (pi.n == 0 || pi.first < prev_end || pi.first + pi.n > n_desc) return TM_ERR_ARG;   // ascending, disjoint
    prev_end = pi.first + pi.n;
    uint64_t n_elems = 0;
    int rc = tm_shard_validate(plan->descs.data() + pi.first, pi.n, r, D, &pi.e, &n_elems);
    if (rc != TM_OK) return rc;
    rc = tm_bounds_u128(n_elems, r, D, &pi.lo, &pi.hi);
    if (rc != TM_OK) return rc;
    if (out_elems != nullptr) out_elems[p] = pi.hi - pi.lo;
  }
  const bool dry = (d_workspace == nullptr);
  uint64_t base = ~0ull;
  std::vector<std::pair<uint64_t, uint64_t>> outs;
  if (!dry) {
    if (d_outs == nullptr || out_capacities == nullptr) return TM_ERR_ARG;
    if (((uintptr_t)d_workspace & 255) != 0) return TM_ERR_ALIGN;
    for (uint32_t p = 0; p < n_planes; ++p) {
      const uint64_t bytes = (planes[p].hi - planes[p].lo) * planes[p].e;
      if (bytes == 0) continue;
      if (d_outs[p] == nullptr) return TM_ERR_ARG;
      if (((uintptr_t)d_outs[p] & 1) != 0) return TM_ERR_ALIGN;
      if (out_capacities[p] < bytes) return TM_ERR_CAPACITY;
      const uint64_t o = (uint64_t)(uintptr_t)d_outs[p];
      for (const tm_desc& d : plan->descs)
        if (ranges_overlap((uint64_t)(uintptr_t)d.ptr, d.nbytes, o, bytes)) return TM_ERR_OVERLAP;
      for (const auto& q : outs)
        if (ranges_overlap(o, bytes, q.first, q.second)) return TM_ERR_OVERLAP;
      outs.emplace_back(o, bytes);
      base = std::min(base, o);
    }
  }
  if (base == ~0ull) base = 0;
  // one pass over the descriptors: the pack pieces of tensor k, then the emit pieces that read tensor k
  tms::WorkList wl;
  tms::WorkListBuilder builder(&wl);
  size_t cursor = 0;            // next pack piece of the plan
  uint32_t p = 0;               // current plane
  uint64_t start = 0;           // element index, inside plane p, of tensor k's first element
  for (uint64_t k = 0; k < n_desc; ++k) {
    uint64_t seen = 0;
    while (seen < plan->descs[k].nbytes) {
      const tms::Seg& s = plan->work.segs[cursor++];
      builder.add(s);
      seen += s.nbytes;
    }
    while (p < n_planes && k >= planes[p].first + planes[p].n) { ++p; start = 0; }
    if (p < n_planes && k >= planes[p].first) {
      const PlaneInfo& pi = planes[p];
      const uint64_t count = plan->descs[k].nbytes / pi.e;
      const uint64_t a = std::max(pi.lo, start), b = std::min(pi.hi, start + count);
      if (a < b) {
        const uint64_t out = dry ? (uint64_t)256 * (a - pi.lo) : (uint64_t)(uintptr_t)d_outs[p] + (a - pi.lo) * pi.e;
        tm_shard_append(&builder, &plan->descs[k], 1, pi.e, a - start, b - start, out, dry ? 0 : base, 0xffffffffu);
      }
      start += count;
    }
  }
  builder.finish();
  const tms::WorkspaceLayout l = tms::workspace_layout(wl.segs.size() + 2 * n_desc + 8, wl.n_items() + 2 * n_desc + 8);
  if (workspace_needed != nullptr) *workspace_needed = l.total;
  if (dry) return TM_OK;
  const tms::WorkspaceLayout exact = tms::workspace_layout(wl.segs.size(), wl.n_items());
  if (workspace_bytes < exact.total) return TM_ERR_CAPACITY;
  int rc = upload_worklist(wl, exact, (uint8_t*)d_workspace, (cudaStream_t)stream);
  if (rc != TM_OK) return rc;
  plan->emit_work = std::move(wl);
  plan->emit_layout = exact;
  plan->d_emit_workspace = (uint8_t*)d_workspace;
  plan->emit_base = base;
  plan->emit_outs = std::move(outs);
  return TM_OK;
}

int tm_state_pack_emit(const tm_plan* plan, void* d_buckets, uint64_t capacity, uint64_t* d_checksums,
                       void* stream) {
  if (plan == nullptr || d_buckets == nullptr) return TM_ERR_ARG;
  if (plan->d_emit_workspace == nullptr) return TM_ERR_STATE;
  if (((uintptr_t)d_buckets & 255) != 0 || ((uintptr_t)d_checksums & 7) != 0) return TM_ERR_ALIGN;
  if (capacity < plan->total_bytes) return TM_ERR_CAPACITY;
  const uint64_t base = (uint64_t)(uintptr_t)d_buckets;
  for (const tm_desc& d : plan->descs)
    if (ranges_overlap((uint64_t)(uintptr_t)d.ptr, d.nbytes, base, plan->total_bytes)) return TM_ERR_OVERLAP;
  for (const auto& o : plan->emit_outs)
    if (ranges_overlap(o.first, o.second, base, plan->total_bytes)) return TM_ERR_OVERLAP;
  cudaStream_t st = (cudaStream_t)stream;
  if (d_checksums != nullptr)
    TM_CUDA(cudaMemsetAsync(d_checksums, 0, plan->n_buckets * sizeof(uint64_t), st));
  const uint8_t* ws = plan->d_emit_workspace;
  int e = tms::launch_pack_emit_ring((const tms::Seg*)(ws + plan->emit_layout.segs_off),
                                     (const uint32_t*)(ws + plan->emit_layout.items_off),
                                     (uint32_t)plan->emit_work.n_items(), (uint8_t*)d_buckets,
                                     (unsigned long long*)d_checksums, (uint8_t*)(uintptr_t)plan->emit_base,
                                     (int*)plan->d_emit_workspace, stream);
  return e == 0 ? TM_OK : cuda_fail(e);
}

int tm_shard_bounds(uint64_t n_elems, uint32_t r, uint32_t D, uint64_t* lo, uint64_t* hi) {
  if (lo == nullptr || hi == nullptr) return TM_ERR_ARG;
  return tm_bounds_u128(n_elems, r, D, lo, hi);
}

int tm_shard_workspace(const tm_desc* plane_descs, uint64_t n_desc, uint32_t r, uint32_t D,
                       uint64_t* workspace_bytes) {
  if (workspace_bytes == nullptr) return TM_ERR_ARG;
  uint32_t e = 0;
  uint64_t n_elems = 0;
  int rc = tm_shard_validate(plane_descs, n_desc, r, D, &e, &n_elems);
  if (rc != TM_OK) return rc;
  uint64_t lo = 0, hi = 0;
  rc = tm_bounds_u128(n_elems, r, D, &lo, &hi);
  if (rc != TM_OK) return rc;
  // upper bound on pieces: every tensor adds at most two partial pieces to the chunk count
  const uint64_t chunk = tms::tuning().shard_chunk_bytes;
  const uint64_t max_segs = (hi - lo) * e / chunk + 2 * n_desc + 2;
  *workspace_bytes = tms::workspace_layout(max_segs, max_segs).total;
  return TM_OK;
}

// Shared body of shard extract (tensors -> flat) and shard insert (flat -> tensors).
static int shard_run(const tm_desc* plane_descs, uint64_t n_desc, uint32_t r, uint32_t D, void* d_flat,
                     uint64_t flat_capacity, uint64_t* elems, void* d_workspace, uint64_t workspace_bytes,
                     void* stream, bool to_tensors) {
  uint32_t e = 0;
  uint64_t n_elems = 0;
  int rc = tm_shard_validate(plane_descs, n_desc, r, D, &e, &n_elems);
  if (rc != TM_OK) return rc;
  uint64_t lo = 0, hi = 0;
  rc = tm_bounds_u128(n_elems, r, D, &lo, &hi);
  if (rc != TM_OK) return rc;
  if (elems != nullptr) *elems = hi - lo;
  if (hi == lo) return TM_OK;
  if (d_flat == nullptr || d_workspace == nullptr) return TM_ERR_ARG;
  if (((uintptr_t)d_flat & 1) != 0 || ((uintptr_t)d_workspace & 255) != 0) return TM_ERR_ALIGN;
  const uint64_t flat_bytes = (hi - lo) * e;
  if (flat_capacity < flat_bytes) return TM_ERR_CAPACITY;
  const uint64_t flat_addr = (uint64_t)(uintptr_t)d_flat;
  for (uint64_t k = 0; k < n_desc; ++k)
    if (ranges_overlap((uint64_t)(uintptr_t)plane_descs[k].ptr, plane_descs[k].nbytes, flat_addr, flat_bytes))
      return TM_ERR_OVERLAP;
  tms::WorkList wl;
  tm_shard_worklist(plane_descs, n_desc, e, lo, hi, flat_addr, &wl);
  const tms::WorkspaceLayout l = tms::workspace_layout(wl.segs.size(), wl.n_items());
  if (workspace_bytes < l.total) return TM_ERR_CAPACITY;
  rc = upload_worklist(wl, l, (uint8_t*)d_workspace, (cudaStream_t)stream);
  if (rc != TM_OK) return rc;
  const uint8_t* ws = (const uint8_t*)d_workspace;
  auto copy_fn = tms::tuning().use_ring ? tms::launch_copy_ring : tms::launch_copy;
  int err = copy_fn((const tms::Seg*)(ws + l.segs_off), (const uint32_t*)(ws + l.items_off),
                    (uint32_t)wl.n_items(), (uint8_t*)d_flat, to_tensors, (int*)d_workspace, stream);
  return err == 0 ? TM_OK : cuda_fail(err);
}

int tm_shard_extract(const tm_desc* plane_descs, uint64_t n_desc, uint32_t r, uint32_t D, void* d_out,
                     uint64_t out_capacity, uint64_t* out_elems, void* d_workspace,
                     uint64_t workspace_bytes, void* stream) {
  return shard_run(plane_descs, n_desc, r, D, d_out, out_capacity, out_elems, d_workspace, workspace_bytes,
                   stream, /*to_tensors=*/false);
}

int tm_shard_extract_planes(const tm_desc* descs, const uint64_t* plane_n_desc, uint32_t n_planes, uint32_t r,
                            uint32_t D, void* const* d_outs, const uint64_t* out_capacities,
                            uint64_t* out_elems, void* d_workspace, uint64_t workspace_bytes, void* stream) {
  if (descs == nullptr || plane_n_desc == nullptr || n_planes == 0 || d_outs == nullptr ||
      out_capacities == nullptr)
    return TM_ERR_ARG;
  if (d_workspace == nullptr) return TM_ERR_ARG;
  if (((uintptr_t)d_workspace & 255) != 0) return TM_ERR_ALIGN;
  struct PlaneInfo { const tm_desc* d; uint64_t n; uint32_t e; uint64_t lo, hi; };
  std::vector<PlaneInfo> planes(n_planes);
  const tm_desc* cursor = descs;
  uint64_t base = ~0ull;
  for (uint32_t p = 0; p < n_planes; ++p) {
    PlaneInfo& pi = planes[p];
    pi.d = cursor;
    pi.n = plane_n_desc[p];
    uint64_t n_elems = 0;
    int rc = tm_shard_validate(pi.d, pi.n, r, D, &pi.e, &n_elems);
    if (rc != TM_OK) return rc;
    rc = tm_bounds_u128(n_elems, r, D, &pi.lo, &pi.hi);
    if (rc != TM_OK) return rc;
    cursor += pi.n;
    if (pi.hi == pi.lo) continue;
    if (d_outs[p] == nullptr) return TM_ERR_ARG;
    if (((uintptr_t)d_outs[p] & 1) != 0) return TM_ERR_ALIGN;
    if (out_capacities[p] < (pi.hi - pi.lo) * pi.e) return TM_ERR_CAPACITY;
    base = std::min(base, (uint64_t)(uintptr_t)d_outs[p]);
  }
  // no output may overlap a tensor of any plane, nor another output
  const uint64_t n_total = (uint64_t)(cursor - descs);
  for (uint32_t p = 0; p < n_planes; ++p) {
    if (planes[p].hi == planes[p].lo) continue;
    const uint64_t o = (uint64_t)(uintptr_t)d_outs[p], ob = (planes[p].hi - planes[p].lo) * planes[p].e;
    for (uint64_t k = 0; k < n_total; ++k)
      if (ranges_overlap((uint64_t)(uintptr_t)descs[k].ptr, descs[k].nbytes, o, ob)) return TM_ERR_OVERLAP;
    for (uint32_t q = p + 1; q < n_planes; ++q) {
      if (planes[q].hi == planes[q].lo) continue;
      if (ranges_overlap(o, ob, (uint64_t)(uintptr_t)d_outs[q], (planes[q].hi - planes[q].lo) * planes[q].e))
        return TM_ERR_OVERLAP;
    }
  }
  if (out_elems != nullptr)
    for (uint32_t p = 0; p < n_planes; ++p) out_elems[p] = planes[p].hi - planes[p].lo;
  if (base == ~0ull) return TM_OK;   // every shard is empty
  tms::WorkList wl;
  tms::WorkListBuilder builder(&wl);
  for (uint32_t p = 0; p < n_planes; ++p)
    if (planes[p].hi != planes[p].lo)
      tm_shard_append(&builder, planes[p].d, planes[p].n, planes[p].e, planes[p].lo, planes[p].hi,
                      (uint64_t)(uintptr_t)d_outs[p], base, 0);
  builder.finish();
  const tms::WorkspaceLayout l = tms::workspace_layout(wl.segs.size(), wl.n_items());
  if (workspace_bytes < l.total) return TM_ERR_CAPACITY;
  int rc = upload_worklist(wl, l, (uint8_t*)d_workspace, (cudaStream_t)stream);
  if (rc != TM_OK) return rc;
  const uint8_t* ws = (const uint8_t*)d_workspace;
  auto copy_fn = tms::tuning().use_ring ? tms::launch_copy_ring : tms::launch_copy;
  int err = copy_fn((const tms::Seg*)(ws + l.segs_off), (const uint32_t*)(ws + l.items_off),
                    (uint32_t)wl.n_items(), (uint8_t*)(uintptr_t)base, /*to_tensors=*/false,
                    (int*)d_workspace, stream);
  return err == 0 ? TM_OK : cuda_fail(err);
}

int tm_shard_insert(const tm_desc* plane_descs, uint64_t n_desc, uint32_t r, uint32_t D, const void* d_in,
                    uint64_t in_bytes, uint64_t* in_elems, void* d_workspace, uint64_t workspace_bytes,
                    void* stream) {
  return shard_run(plane_descs, n_desc, r, D, const_cast<void*>(d_in), in_bytes, in_elems, d_workspace,
                   workspace_bytes, stream, /*to_tensors=*/true);
}

int tm_selftest_bounded_wait(void* d_workspace, uint64_t limit_ns, void* stream) {
  if (d_workspace == nullptr || limit_ns == 0 || limit_ns > 5000000000ull) return TM_ERR_ARG;
  if (((uintptr_t)d_workspace & 255) != 0) return TM_ERR_ALIGN;
  TM_CUDA(cudaMemsetAsync(d_workspace, 0, tms::kStatusBlockBytes, (cudaStream_t)stream));
  int e = tms::launch_wait_selftest((int*)d_workspace, limit_ns, stream);
  return e == 0 ? TM_OK : cuda_fail(e);
}

int tm_workspace_status(const void* d_workspace, void* stream, int* device_status) {
  return read_status(d_workspace, (cudaStream_t)stream, device_status);
}

int tm_checksum(const void* d_bytes, uint64_t nbytes, uint64_t bucket_bytes, uint64_t* d_checksums,
                void* stream) {
  if (bucket_bytes == 0 || bucket_bytes > (1ull << 35)) return TM_ERR_ARG;
  if (bucket_bytes % 256 != 0) return TM_ERR_ALIGN;
  if (nbytes == 0) return TM_OK;
  if (d_bytes == nullptr || d_checksums == nullptr) return TM_ERR_ARG;
  if (((uintptr_t)d_bytes & 15) != 0 || ((uintptr_t)d_checksums & 7) != 0) return TM_ERR_ALIGN;
  const uint64_t n_buckets = (nbytes + bucket_bytes - 1) / bucket_bytes;
  cudaStream_t st = (cudaStream_t)stream;
  TM_CUDA(cudaMemsetAsync(d_checksums, 0, n_buckets * sizeof(uint64_t), st));
  int e = tms::launch_checksum((const uint8_t*)d_bytes, nbytes, bucket_bytes,
                              (unsigned long long*)d_checksums, stream);
  return e == 0 ? TM_OK : cuda_fail(e);
}

const char* tm_strerror(int status) {
  switch (status) {
    case TM_OK: return "ok";
    case TM_ERR_ARG: return "invalid argument";
    case TM_ERR_ALIGN: return "misaligned address or bucket size";
    case TM_ERR_CAPACITY: return "buffer too small";
    case TM_ERR_OVERLAP: return "buffers overlap";
    case TM_ERR_RANK: return "invalid shard rank";
    case TM_ERR_DTYPE: return "unsupported or mixed element size";
    case TM_ERR_CUDA: return "CUDA runtime error";
    case TM_ERR_TIMEOUT: return "bounded device wait expired";
    case TM_ERR_STATE: return "plan has no uploaded work list";
    default: return "unknown status";
  }
}

int tm_last_cuda_error(void) { return g_last_cuda_error.load(); }

}  // extern "C"
