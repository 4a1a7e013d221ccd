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

namespace {

std::atomic<int> g_last_cuda_error{0};

#define TM_CUDA(call)                                   \
  do {                                                  \
    cudaError_t e__ = (call);                           \
    if (e__ != cudaSuccess) return tms::cuda_fail((int)e__); \
  } while (0)

// No C++ exception may cross the C boundary: host allocations that fail become TM_ERR_CAPACITY.
template <typename F>
int guarded(F&& f) noexcept {
  try {
    return f();
  } catch (const std::bad_alloc&) {
    return TM_ERR_CAPACITY;
  } catch (...) {
    return TM_ERR_ARG;
  }
}

// True when the packed buffer [base, base + nbytes) overlaps a tensor part the plan touches.  The
// plan's address bounding box settles the common case without walking the parts.
bool plan_overlaps(const tm_plan* plan, uint64_t base, uint64_t nbytes) {
  if (plan->box_hi <= plan->box_lo || !tms::ranges_overlap(plan->box_lo, plan->box_hi - plan->box_lo, base, nbytes))
    return false;
  for (const tm_part& q : plan->parts)
    if (tms::ranges_overlap(q.addr, q.nbytes, base, nbytes)) return true;
  return false;
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

}  // namespace

namespace tms {

int cuda_fail(int e) {
  g_last_cuda_error.store(e);
  return TM_ERR_CUDA;
}

int upload_worklist(const WorkList& wl, const std::vector<Emit>* emits, const WorkspaceLayout& l, uint8_t* d_ws,
                    void* stream) {
  cudaStream_t st = (cudaStream_t)stream;
  const size_t items_bytes = wl.item_first.size() * sizeof(uint32_t);
  const size_t segs_bytes = wl.segs.size() * sizeof(Seg);
  const size_t emits_bytes = emits != nullptr ? emits->size() * sizeof(Emit) : 0;
  // status block, pieces, items (, emit records): one contiguous image
  const size_t span = emits != nullptr ? l.emits_off + emits_bytes : l.items_off + items_bytes;
  if (span <= HostStaging::kSlotBytes) {
    int dev = 0;
    if (cudaGetDevice(&dev) == cudaSuccess) {
      std::lock_guard<std::mutex> lock(g_staging.mutex);
      const int slot = g_staging.acquire(dev);
      if (slot >= 0) {
        uint8_t* h = g_staging.host(dev, slot);
        std::memset(h, 0, span);
        if (segs_bytes != 0) std::memcpy(h + l.segs_off, wl.segs.data(), segs_bytes);
        std::memcpy(h + l.items_off, wl.item_first.data(), items_bytes);
        if (emits_bytes != 0) std::memcpy(h + l.emits_off, emits->data(), emits_bytes);
        TM_CUDA(cudaMemcpyAsync(d_ws, h, span, cudaMemcpyHostToDevice, st));
        TM_CUDA(g_staging.mark(dev, slot, st));
        return TM_OK;
      }
    }
  }
  TM_CUDA(cudaMemsetAsync(d_ws, 0, kStatusBlockBytes, st));
  if (segs_bytes != 0)
    TM_CUDA(cudaMemcpyAsync(d_ws + l.segs_off, wl.segs.data(), segs_bytes, cudaMemcpyHostToDevice, st));
  TM_CUDA(cudaMemcpyAsync(d_ws + l.items_off, wl.item_first.data(), items_bytes, cudaMemcpyHostToDevice, st));
  if (emits_bytes != 0)
    TM_CUDA(cudaMemcpyAsync(d_ws + l.emits_off, emits->data(), emits_bytes, cudaMemcpyHostToDevice, st));
  return TM_OK;
}

int read_status_word(const void* d_ws, void* stream, int* device_status) {
  if (d_ws == nullptr || device_status == nullptr) return TM_ERR_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  int word = 0;
  TM_CUDA(cudaMemcpyAsync(&word, d_ws, sizeof(int), cudaMemcpyDeviceToHost, st));
  TM_CUDA(cudaStreamSynchronize(st));
  *device_status = word;
  return TM_OK;
}

}  // namespace tms

namespace {

tms::RingLaunch ring_args(const tm_plan* plan, const uint8_t* ws, const tms::WorkspaceLayout& l, void* d_buckets,
                          uint64_t* d_checksums) {
  tms::RingLaunch a;
  a.d_segs = (const tms::Seg*)(ws + l.segs_off);
  a.d_item_first = (const uint32_t*)(ws + l.items_off);
  a.n_items = (uint32_t)plan->work.n_items();
  a.d_flat = (uint8_t*)d_buckets;
  a.d_checksums = (unsigned long long*)d_checksums;
  a.d_status = (int*)const_cast<uint8_t*>(ws);
  a.wait_limit_ns = plan->opt.wait_limit_ns;
  a.ctas_per_sm = plan->opt.ring_ctas_per_sm;
  return a;
}

// Checks shared by pack, pack_emit, unpack and unpack_verify.
int check_buckets(const tm_plan* plan, const void* d_buckets, uint64_t nbytes, const void* d_checksums) {
  if (plan == nullptr || d_buckets == nullptr) return TM_ERR_ARG;
  if (((uintptr_t)d_buckets & 255) != 0 || ((uintptr_t)d_checksums & 7) != 0) return TM_ERR_ALIGN;
  if (nbytes < plan->total_bytes) return TM_ERR_CAPACITY;
  if (plan_overlaps(plan, (uint64_t)(uintptr_t)d_buckets, plan->total_bytes)) return TM_ERR_OVERLAP;
  return TM_OK;
}

}  // namespace

extern "C" {

int tm_options_get(tm_options* out) {
  if (out == nullptr) return TM_ERR_ARG;
  *out = tms::tuning();
  return TM_OK;
}

int tm_options_set(const tm_options* in) { return tms::set_tuning(in); }

static int plan_create(const tm_desc* descs, uint64_t n_desc, uint64_t bucket_bytes, bool ranged, uint64_t first,
                       uint64_t count, tm_plan** out) {
  if (out == nullptr) return TM_ERR_ARG;
  *out = nullptr;
  return guarded([&]() -> int {
    tm_plan* p = new tm_plan();
    int rc = TM_ERR_CAPACITY;
    try {
      rc = tm_plan_build(p, descs, n_desc, bucket_bytes, ranged, first, count);
    } catch (...) {
      delete p;
      throw;
    }
    if (rc != TM_OK) {
      delete p;
      return rc;
    }
    *out = p;
    return TM_OK;
  });
}

int tm_plan_create(const tm_desc* descs, uint64_t n_desc, uint64_t bucket_bytes, tm_plan** out) {
  return plan_create(descs, n_desc, bucket_bytes, false, 0, 0, out);
}

int tm_plan_create_range(const tm_desc* descs, uint64_t n_desc, uint64_t bucket_bytes, uint64_t first_bucket,
                         uint64_t n_buckets, tm_plan** out) {
  return plan_create(descs, n_desc, bucket_bytes, true, first_bucket, n_buckets, out);
}

int tm_plan_query(const tm_plan* plan, uint64_t* total_bytes, uint64_t* n_buckets,
                  uint64_t* workspace_bytes) {
  if (plan == nullptr) return TM_ERR_ARG;
  if (total_bytes != nullptr) *total_bytes = plan->total_bytes;
  if (n_buckets != nullptr) *n_buckets = plan->n_buckets;
  if (workspace_bytes != nullptr) *workspace_bytes = plan->ws_layout.total;
  return TM_OK;
}

int tm_plan_range(const tm_plan* plan, uint64_t* first_bucket, uint64_t* stream_begin, uint64_t* whole_bytes,
                  uint64_t* whole_buckets) {
  if (plan == nullptr) return TM_ERR_ARG;
  if (first_bucket != nullptr) *first_bucket = plan->first_bucket;
  if (stream_begin != nullptr) *stream_begin = plan->range_begin;
  if (whole_bytes != nullptr) *whole_bytes = plan->whole_bytes;
  if (whole_buckets != nullptr) *whole_buckets = plan->whole_buckets;
  return TM_OK;
}

int tm_plan_offsets(const tm_plan* plan, uint64_t* offsets) {
  if (plan == nullptr || offsets == nullptr) return TM_ERR_ARG;
  std::memcpy(offsets, plan->offsets.data(), plan->offsets.size() * sizeof(uint64_t));
  return TM_OK;
}

static int copy_pieces(const tms::WorkList& wl, tm_piece* pieces, uint64_t capacity, uint64_t* n_pieces,
                       uint32_t* item_first, uint64_t item_capacity, uint64_t* n_items) {
  static_assert(sizeof(tm_piece) == sizeof(tms::Seg), "tm_piece mirrors the internal piece");
  const uint64_t np = wl.segs.size(), ni = wl.n_items();
  if (n_pieces != nullptr) *n_pieces = np;
  if (n_items != nullptr) *n_items = ni;
  if (pieces != nullptr) std::memcpy(pieces, wl.segs.data(), std::min(np, capacity) * sizeof(tm_piece));
  if (item_first != nullptr && !wl.item_first.empty())
    std::memcpy(item_first, wl.item_first.data(), std::min(ni + 1, item_capacity) * sizeof(uint32_t));
  return TM_OK;
}

int tm_plan_pieces(const tm_plan* plan, tm_piece* pieces, uint64_t capacity, uint64_t* n_pieces,
                   uint32_t* item_first, uint64_t item_capacity, uint64_t* n_items) {
  if (plan == nullptr) return TM_ERR_ARG;
  return copy_pieces(plan->work, pieces, capacity, n_pieces, item_first, item_capacity, n_items);
}

int tm_shard_plan_pieces(const tm_shard_plan* sp, tm_piece* pieces, uint64_t capacity, uint64_t* n_pieces,
                         uint32_t* item_first, uint64_t item_capacity, uint64_t* n_items, uint64_t* base) {
  if (sp == nullptr) return TM_ERR_ARG;
  if (base != nullptr) *base = sp->base;
  return copy_pieces(sp->work, pieces, capacity, n_pieces, item_first, item_capacity, n_items);
}

int tm_plan_emits(const tm_plan* plan, tm_emit* emits, uint64_t capacity, uint64_t* n) {
  if (plan == nullptr) return TM_ERR_ARG;
  static_assert(sizeof(tm_emit) == sizeof(tms::Emit), "tm_emit mirrors the internal record");
  if (n != nullptr) *n = plan->emits.size();
  if (emits != nullptr)
    std::memcpy(emits, plan->emits.data(), std::min<uint64_t>(plan->emits.size(), capacity) * sizeof(tm_emit));
  return TM_OK;
}

int tm_plan_upload(tm_plan* plan, void* d_workspace, uint64_t workspace_bytes, void* stream) {
  if (plan == nullptr || d_workspace == nullptr) return TM_ERR_ARG;
  if (((uintptr_t)d_workspace & 255) != 0) return TM_ERR_ALIGN;
  if (workspace_bytes < plan->ws_layout.total) return TM_ERR_CAPACITY;
  int rc = tms::upload_worklist(plan->work, nullptr, plan->ws_layout, (uint8_t*)d_workspace, stream);
  if (rc != TM_OK) return rc;
  plan->d_workspace = (uint8_t*)d_workspace;
  return TM_OK;
}

int tm_plan_status(const tm_plan* plan, void* stream, int* device_status) {
  if (plan == nullptr || device_status == nullptr) return TM_ERR_ARG;
  if (plan->d_workspace == nullptr && plan->d_emit_workspace == nullptr) return TM_ERR_STATE;
  int a = 0, b = 0;
  if (plan->d_workspace != nullptr) {
    int rc = tms::read_status_word(plan->d_workspace, stream, &a);
    if (rc != TM_OK) return rc;
  }
  if (plan->d_emit_workspace != nullptr) {
    int rc = tms::read_status_word(plan->d_emit_workspace, stream, &b);
    if (rc != TM_OK) return rc;
  }
  *device_status = (a != 0) ? a : b;
  return TM_OK;
}

void tm_plan_destroy(tm_plan* plan) { delete plan; }

int tm_state_pack(const tm_plan* plan, void* d_buckets, uint64_t capacity, uint64_t* d_checksums,
                  void* stream) {
  int rc = check_buckets(plan, d_buckets, capacity, d_checksums);
  if (rc != TM_OK) return rc;
  if (plan->d_workspace == nullptr) return TM_ERR_STATE;
  if (d_checksums != nullptr)
    TM_CUDA(cudaMemsetAsync(d_checksums, 0, plan->n_buckets * sizeof(uint64_t), (cudaStream_t)stream));
  int e = tms::launch_ring(tms::kRingPack, ring_args(plan, plan->d_workspace, plan->ws_layout, d_buckets, d_checksums),
                           stream);
  return e == 0 ? TM_OK : tms::cuda_fail(e);
}

static int targets_ok(const tm_plan* plan) {
  if (plan->targets_disjoint == 0) plan->targets_disjoint = tm_parts_disjoint(plan->parts);
  return plan->targets_disjoint < 0 ? TM_ERR_OVERLAP : TM_OK;
}

int tm_state_unpack(const tm_plan* plan, const void* d_buckets, uint64_t nbytes, void* stream) {
  return guarded([&]() -> int {
    int rc = check_buckets(plan, d_buckets, nbytes, nullptr);
    if (rc != TM_OK) return rc;
    if (plan->d_workspace == nullptr) return TM_ERR_STATE;
    if ((rc = targets_ok(plan)) != TM_OK) return rc;
    int e = tms::launch_ring(tms::kRingToTensors,
                             ring_args(plan, plan->d_workspace, plan->ws_layout, const_cast<void*>(d_buckets), nullptr),
                             stream);
    return e == 0 ? TM_OK : tms::cuda_fail(e);
  });
}

int tm_state_unpack_verify(const tm_plan* plan, const void* d_buckets, uint64_t nbytes, uint64_t* d_checksums,
                           void* stream) {
  return guarded([&]() -> int {
    if (d_checksums == nullptr) return TM_ERR_ARG;
    int rc = check_buckets(plan, d_buckets, nbytes, d_checksums);
    if (rc != TM_OK) return rc;
    if (plan->d_workspace == nullptr) return TM_ERR_STATE;
    if ((rc = targets_ok(plan)) != TM_OK) return rc;
    TM_CUDA(cudaMemsetAsync(d_checksums, 0, plan->n_buckets * sizeof(uint64_t), (cudaStream_t)stream));
    int e = tms::launch_ring(tms::kRingToTensorsVerify,
                             ring_args(plan, plan->d_workspace, plan->ws_layout, const_cast<void*>(d_buckets), d_checksums),
                             stream);
    return e == 0 ? TM_OK : tms::cuda_fail(e);
  });
}

}  // extern "C"

// Shard attachment for a plan whose pieces index into `descs` (the plan's own copy, or the one copy a
// transfer endpoint keeps for all of its wave plans).
int tm_attach_shards(tm_plan* plan, const tm_desc* descs, uint64_t n_desc, const uint64_t* plane_first_desc,
                     const uint64_t* plane_n_desc, uint32_t n_planes, uint32_t r, uint32_t D, void* const* d_outs,
                     const uint64_t* out_capacities, uint64_t* out_elems, void* d_workspace,
                     uint64_t workspace_bytes, uint64_t* workspace_needed, void* stream) {
  return guarded([&]() -> int {
    if (plan == nullptr || descs == nullptr || plane_first_desc == nullptr || plane_n_desc == nullptr || n_planes == 0)
      return TM_ERR_ARG;
    if (D == 0 || r >= D) return TM_ERR_RANK;
    struct PlaneInfo { uint64_t first, n; uint32_t e; uint64_t lo, hi; };
    std::vector<PlaneInfo> planes(n_planes);
    uint64_t prev_end = 0;
    for (uint32_t p = 0; p < n_planes; ++p) {
      PlaneInfo& pi = planes[p];
      pi.first = plane_first_desc[p];
      pi.n = plane_n_desc[p];
      if (pi.n == 0 || pi.first < prev_end || pi.n > n_desc || pi.first > n_desc - pi.n) return TM_ERR_ARG;   // ascending, disjoint
      prev_end = pi.first + pi.n;
      uint64_t n_elems = 0;
      int rc = tm_shard_validate(descs + pi.first, pi.n, r, D, &pi.e, &n_elems);
      if (rc != TM_OK) return rc;
      rc = tm_bounds_u128(n_elems, r, D, &pi.lo, &pi.hi);
      if (rc != TM_OK) return rc;
      if (out_elems != nullptr) out_elems[p] = pi.hi - pi.lo;
    }
    const tms::WorkspaceLayout l = tms::workspace_layout(plan->work.segs.size(), plan->work.n_items(), true);
    if (workspace_needed != nullptr) *workspace_needed = l.total;
    if (d_workspace == nullptr && d_outs == nullptr) return TM_OK;   // size query
    if (d_outs == nullptr || out_capacities == nullptr) return TM_ERR_ARG;
    if (((uintptr_t)d_workspace & 255) != 0) return TM_ERR_ALIGN;
    if (d_workspace != nullptr && workspace_bytes < l.total) return TM_ERR_CAPACITY;
    std::vector<std::pair<uint64_t, uint64_t>> outs;
    for (uint32_t p = 0; p < n_planes; ++p) {
      const uint64_t bytes = (planes[p].hi - planes[p].lo) * planes[p].e;
      if (bytes == 0) continue;
      if (d_outs[p] == nullptr) return TM_ERR_ARG;
      if (((uintptr_t)d_outs[p] & 1) != 0) return TM_ERR_ALIGN;
      if (out_capacities[p] < bytes) return TM_ERR_CAPACITY;
      const uint64_t o = (uint64_t)(uintptr_t)d_outs[p];
      if (plan_overlaps(plan, o, bytes)) return TM_ERR_OVERLAP;
      for (const auto& q : outs)
        if (tms::ranges_overlap(o, bytes, q.first, q.second)) return TM_ERR_OVERLAP;
      outs.emplace_back(o, bytes);
    }
    // for every descriptor inside a plane: its plane and the plane-wide index of its first element
    std::vector<int32_t> desc_plane(n_desc, -1);
    std::vector<uint64_t> desc_start(n_desc, 0);
    for (uint32_t p = 0; p < n_planes; ++p) {
      uint64_t start = 0;
      for (uint64_t k = planes[p].first; k < planes[p].first + planes[p].n; ++k) {
        desc_plane[k] = (int32_t)p;
        desc_start[k] = start;
        start += descs[k].nbytes / planes[p].e;
      }
    }
    // one emit record per piece: the piece's bytes that are shard elements, and where they go
    std::vector<tms::Emit> emits(plan->work.segs.size());
    for (size_t i = 0; i < emits.size(); ++i) {
      tms::Emit& em = emits[i];
      em.out = 0;
      em.begin = 0;
      em.len = 0;
      const uint32_t k = plan->piece_desc[i];
      if (desc_plane[k] < 0) continue;
      const PlaneInfo& pi = planes[desc_plane[k]];
      const uint64_t start = desc_start[k], count = descs[k].nbytes / pi.e;
      const uint64_t a = std::max(pi.lo, start), b = std::min(pi.hi, start + count);
      if (a >= b) continue;
      const tms::Seg& s = plan->work.segs[i];
      const uint64_t x = s.tensor - (uint64_t)(uintptr_t)descs[k].ptr;   // piece = tensor bytes [x, x + nbytes)
      const uint64_t sa = (a - start) * pi.e, sb = (b - start) * pi.e;         // shard = tensor bytes [sa, sb)
      const uint64_t lo = std::max(x, sa), hi = std::min(x + s.nbytes, sb);
      if (lo >= hi) continue;
      em.begin = (uint32_t)(lo - x);
      em.len = (uint32_t)(hi - lo);
      em.out = (uint64_t)(uintptr_t)d_outs[desc_plane[k]] + ((start * pi.e + lo) - pi.lo * pi.e);   // plane byte - shard's first byte
    }
    if (d_workspace != nullptr) {   // without a workspace the records are only computed, for inspection on the host
      int rc = tms::upload_worklist(plan->work, &emits, l, (uint8_t*)d_workspace, stream);
      if (rc != TM_OK) return rc;
    }
    plan->emits = std::move(emits);
    plan->emit_layout = l;
    plan->d_emit_workspace = (uint8_t*)d_workspace;
    plan->emit_outs = std::move(outs);
    return TM_OK;
  });
}

extern "C" {

int tm_plan_attach_shards(tm_plan* plan, const uint64_t* plane_first_desc, const uint64_t* plane_n_desc,
                          uint32_t n_planes, uint32_t r, uint32_t D, void* const* d_outs,
                          const uint64_t* out_capacities, uint64_t* out_elems, void* d_workspace,
                          uint64_t workspace_bytes, uint64_t* workspace_needed, void* stream) {
  if (plan == nullptr) return TM_ERR_ARG;
  return tm_attach_shards(plan, plan->descs.data(), plan->descs.size(), plane_first_desc, plane_n_desc, n_planes, r, D,
                          d_outs, out_capacities, out_elems, d_workspace, workspace_bytes, workspace_needed, stream);
}

int tm_state_pack_emit(const tm_plan* plan, void* d_buckets, uint64_t capacity, uint64_t* d_checksums,
                       void* stream) {
  int rc = check_buckets(plan, d_buckets, capacity, d_checksums);
  if (rc != TM_OK) return rc;
  if (plan->d_emit_workspace == nullptr) return TM_ERR_STATE;
  for (const auto& o : plan->emit_outs)
    if (tms::ranges_overlap(o.first, o.second, (uint64_t)(uintptr_t)d_buckets, plan->total_bytes)) return TM_ERR_OVERLAP;
  if (d_checksums != nullptr)
    TM_CUDA(cudaMemsetAsync(d_checksums, 0, plan->n_buckets * sizeof(uint64_t), (cudaStream_t)stream));
  tms::RingLaunch a = ring_args(plan, plan->d_emit_workspace, plan->emit_layout, d_buckets, d_checksums);
  a.d_emits = (const tms::Emit*)(plan->d_emit_workspace + plan->emit_layout.emits_off);
  int e = tms::launch_ring(tms::kRingPackEmit, a, stream);
  return e == 0 ? TM_OK : tms::cuda_fail(e);
}

int tm_state_unpack_emit(const tm_plan* plan, const void* d_buckets, uint64_t nbytes, uint64_t* d_checksums,
                         void* stream) {
  return guarded([&]() -> int {
    if (d_checksums == nullptr) return TM_ERR_ARG;
    int rc = check_buckets(plan, d_buckets, nbytes, d_checksums);
    if (rc != TM_OK) return rc;
    if (plan->d_emit_workspace == nullptr) return TM_ERR_STATE;
    if ((rc = targets_ok(plan)) != TM_OK) return rc;
    for (const auto& o : plan->emit_outs)
      if (tms::ranges_overlap(o.first, o.second, (uint64_t)(uintptr_t)d_buckets, plan->total_bytes)) return TM_ERR_OVERLAP;
    TM_CUDA(cudaMemsetAsync(d_checksums, 0, plan->n_buckets * sizeof(uint64_t), (cudaStream_t)stream));
    tms::RingLaunch a = ring_args(plan, plan->d_emit_workspace, plan->emit_layout, const_cast<void*>(d_buckets), d_checksums);
    a.d_emits = (const tms::Emit*)(plan->d_emit_workspace + plan->emit_layout.emits_off);
    int e = tms::launch_ring(tms::kRingToTensorsVerifyEmit, a, stream);
    return e == 0 ? TM_OK : tms::cuda_fail(e);
  });
}

int tm_selftest_bounded_wait(void* d_workspace, uint64_t limit_ns, void* stream) {
  if (d_workspace == nullptr || limit_ns == 0 || limit_ns > 5000000000ull) return TM_ERR_ARG;
  if (((uintptr_t)d_workspace & 255) != 0) return TM_ERR_ALIGN;
  TM_CUDA(cudaMemsetAsync(d_workspace, 0, tms::kStatusBlockBytes, (cudaStream_t)stream));
  int e = tms::launch_wait_selftest((int*)d_workspace, limit_ns, stream);
  return e == 0 ? TM_OK : tms::cuda_fail(e);
}

int tm_workspace_status(const void* d_workspace, void* stream, int* device_status) {
  return tms::read_status_word(d_workspace, stream, device_status);
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
                              (unsigned long long*)d_checksums, tms::tuning(), stream);
  return e == 0 ? TM_OK : tms::cuda_fail(e);
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
    case TM_ERR_VERIFY: return "checksum mismatch after the last transfer round";
    case TM_ERR_TRANSPORT: return "transport callback failed";
    default: return "unknown status";
  }
}

int tm_last_cuda_error(void) { return g_last_cuda_error.load(); }

}  // extern "C"
