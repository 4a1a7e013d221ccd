// Distributed-optimizer shard calls of the C ABI (include/tm_state.h): the reusable shard plan and
// the one-shot extract / insert calls, which are a plan that lives for one call.
#include <cuda_runtime.h>

#include <algorithm>
#include <new>
#include <vector>

#include "tm_internal.h"

namespace {

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

int plan_build(tm_shard_plan* sp, const tm_desc* descs, const uint64_t* plane_n_desc, uint32_t n_planes, uint32_t r,
               uint32_t D) {
  if (descs == nullptr || plane_n_desc == nullptr || n_planes == 0) return TM_ERR_ARG;
  if (D == 0 || r >= D) return TM_ERR_RANK;
  sp->opt = tms::tuning();
  sp->r = r;
  sp->D = D;
  const tm_desc* cursor = descs;
  for (uint32_t p = 0; p < n_planes; ++p) {
    uint32_t e = 0;
    uint64_t n_elems = 0, lo = 0, hi = 0;
    int rc = tm_shard_validate(cursor, plane_n_desc[p], r, D, &e, &n_elems);
    if (rc != TM_OK) return rc;
    rc = tm_bounds_u128(n_elems, r, D, &lo, &hi);
    if (rc != TM_OK) return rc;
    sp->plane_n.push_back(plane_n_desc[p]);
    sp->elem_size.push_back(e);
    sp->lo.push_back(lo);
    sp->hi.push_back(hi);
    cursor += plane_n_desc[p];
  }
  sp->descs.assign(descs, cursor);
  return TM_OK;
}

// Upper bound on the pieces of one plane's list: every tensor adds at most two partial pieces to
// the chunk count.
uint64_t max_pieces(const tm_shard_plan* sp, uint32_t p) {
  return (sp->hi[p] - sp->lo[p]) * sp->elem_size[p] / sp->opt.shard_chunk_bytes + 2 * sp->plane_n[p] + 2;
}

uint64_t workspace_bound(const tm_shard_plan* sp) {
  uint64_t n = 0;
  for (uint32_t p = 0; p < sp->plane_n.size(); ++p) n += max_pieces(sp, p);
  return tms::workspace_layout(n, n).total;
}

int plan_bind(tm_shard_plan* sp, void* const* d_flats, const uint64_t* capacities, void* d_workspace,
              uint64_t workspace_bytes, void* stream) {
  const uint32_t n_planes = (uint32_t)sp->plane_n.size();
  std::vector<std::pair<uint64_t, uint64_t>> flats(n_planes, {0, 0});
  uint64_t base = ~0ull;
  for (uint32_t p = 0; p < n_planes; ++p) {
    const uint64_t bytes = (sp->hi[p] - sp->lo[p]) * sp->elem_size[p];
    if (bytes == 0) continue;
    if (d_flats == nullptr || capacities == nullptr || d_flats[p] == nullptr) return TM_ERR_ARG;
    if (((uintptr_t)d_flats[p] & 1) != 0) return TM_ERR_ALIGN;
    if (capacities[p] < bytes) return TM_ERR_CAPACITY;
    flats[p] = {(uint64_t)(uintptr_t)d_flats[p], bytes};
    base = std::min(base, flats[p].first);
  }
  sp->d_workspace = nullptr;
  sp->work.segs.clear();
  sp->work.item_first.clear();
  if (base == ~0ull) {   // every shard is empty: nothing to bind, nothing will be launched
    sp->flats = std::move(flats);
    sp->base = 0;
    return TM_OK;
  }
  if (((uintptr_t)d_workspace & 255) != 0) return TM_ERR_ALIGN;
  // no flat buffer may overlap a tensor of any plane, nor another flat buffer
  for (uint32_t p = 0; p < n_planes; ++p) {
    if (flats[p].second == 0) continue;
    for (const tm_desc& d : sp->descs)
      if (tms::ranges_overlap((uint64_t)(uintptr_t)d.ptr, d.nbytes, flats[p].first, flats[p].second)) return TM_ERR_OVERLAP;
    for (uint32_t q = p + 1; q < n_planes; ++q)
      if (flats[q].second != 0 && tms::ranges_overlap(flats[p].first, flats[p].second, flats[q].first, flats[q].second))
        return TM_ERR_OVERLAP;
  }
  uint64_t bound = 0;
  for (uint32_t p = 0; p < n_planes; ++p) {
    if (flats[p].second != 0) bound += max_pieces(sp, p);
    if (bound > tms::kMaxPieces) return TM_ERR_CAPACITY;   // refused before any of the list is built
  }
  tms::WorkList wl;
  tms::WorkListBuilder builder(&wl, sp->opt);
  const tm_desc* cursor = sp->descs.data();
  for (uint32_t p = 0; p < n_planes; ++p) {
    if (flats[p].second != 0)
      tm_shard_append(&builder, sp->opt, cursor, sp->plane_n[p], sp->elem_size[p], sp->lo[p], sp->hi[p], flats[p].first,
                      base);
    cursor += sp->plane_n[p];
  }
  builder.finish();
  const tms::WorkspaceLayout l = tms::workspace_layout(wl.segs.size(), wl.n_items());
  if (d_workspace != nullptr) {   // without a workspace the list is only built, for inspection on the host
    if (workspace_bytes < l.total) return TM_ERR_CAPACITY;
    int rc = tms::upload_worklist(wl, nullptr, l, (uint8_t*)d_workspace, stream);
    if (rc != TM_OK) return rc;
  }
  sp->work = std::move(wl);
  sp->layout = l;
  sp->flats = std::move(flats);
  sp->base = base;
  sp->d_workspace = (uint8_t*)d_workspace;
  return TM_OK;
}

int plan_run(const tm_shard_plan* sp, bool to_tensors, void* stream) {
  bool any = false;
  for (const auto& f : sp->flats) any = any || f.second != 0;
  if (sp->flats.size() != sp->plane_n.size()) return TM_ERR_STATE;   // never bound
  if (!any) return TM_OK;
  if (sp->d_workspace == nullptr) return TM_ERR_STATE;
  tms::RingLaunch a;
  a.d_segs = (const tms::Seg*)(sp->d_workspace + sp->layout.segs_off);
  a.d_item_first = (const uint32_t*)(sp->d_workspace + sp->layout.items_off);
  a.n_items = (uint32_t)sp->work.n_items();
  a.d_flat = (uint8_t*)(uintptr_t)sp->base;
  a.d_status = (int*)sp->d_workspace;
  a.wait_limit_ns = sp->opt.wait_limit_ns;
  a.ctas_per_sm = sp->opt.ring_ctas_per_sm;
  int e = tms::launch_ring(to_tensors ? tms::kRingToTensors : tms::kRingToFlat, a, stream);
  return e == 0 ? TM_OK : tms::cuda_fail(e);
}

// The tensors of every plane must be pairwise disjoint before a flat buffer is scattered into them.
int insert_targets_ok(tm_shard_plan* sp) {
  if (sp->targets_disjoint == 0) {
    std::vector<tm_part> parts;
    parts.reserve(sp->descs.size());
    for (const tm_desc& d : sp->descs) parts.push_back(tm_part{(uint64_t)(uintptr_t)d.ptr, d.nbytes});
    sp->targets_disjoint = tm_parts_disjoint(std::move(parts));
  }
  return sp->targets_disjoint < 0 ? TM_ERR_OVERLAP : TM_OK;
}

// A plan that lives for one call.  The list upload has been enqueued (from pinned staging, or copied
// out of pageable memory before cudaMemcpyAsync returned), so the host object can go right away.
int one_shot(const tm_desc* descs, const uint64_t* plane_n_desc, uint32_t n_planes, uint32_t r, uint32_t D,
             void* const* d_flats, const uint64_t* capacities, uint64_t* elems, void* d_workspace,
             uint64_t workspace_bytes, void* stream, bool to_tensors) {
  return guarded([&]() -> int {
    tm_shard_plan sp;
    int rc = plan_build(&sp, descs, plane_n_desc, n_planes, r, D);
    if (rc != TM_OK) return rc;
    if (elems != nullptr)
      for (uint32_t p = 0; p < n_planes; ++p) elems[p] = sp.hi[p] - sp.lo[p];
    if (to_tensors && (rc = insert_targets_ok(&sp)) != TM_OK) return rc;
    bool any = false;
    for (uint32_t p = 0; p < n_planes; ++p) any = any || sp.hi[p] != sp.lo[p];
    if (any && d_workspace == nullptr) return TM_ERR_ARG;
    rc = plan_bind(&sp, d_flats, capacities, d_workspace, workspace_bytes, stream);
    if (rc != TM_OK) return rc;
    return plan_run(&sp, to_tensors, stream);
  });
}

}  // namespace

extern "C" {

int tm_shard_bounds(uint64_t n_elems, uint32_t r, uint32_t D, uint64_t* lo, uint64_t* hi) {
  if (lo == nullptr || hi == nullptr) return TM_ERR_ARG;
  return tm_bounds_u128(n_elems, r, D, lo, hi);
}

int tm_shard_workspace(const tm_desc* plane_descs, uint64_t n_desc, uint32_t r, uint32_t D,
                       uint64_t* workspace_bytes) {
  if (workspace_bytes == nullptr) return TM_ERR_ARG;
  return guarded([&]() -> int {
    tm_shard_plan sp;
    int rc = plan_build(&sp, plane_descs, &n_desc, 1, r, D);
    if (rc != TM_OK) return rc;
    *workspace_bytes = workspace_bound(&sp);
    return TM_OK;
  });
}

int tm_shard_extract(const tm_desc* plane_descs, uint64_t n_desc, uint32_t r, uint32_t D, void* d_out,
                     uint64_t out_capacity, uint64_t* out_elems, void* d_workspace,
                     uint64_t workspace_bytes, void* stream) {
  void* flats[1] = {d_out};
  return one_shot(plane_descs, &n_desc, 1, r, D, flats, &out_capacity, out_elems, d_workspace, workspace_bytes, stream,
                  /*to_tensors=*/false);
}

int tm_shard_extract_planes(const tm_desc* descs, const uint64_t* plane_n_desc, uint32_t n_planes, uint32_t r,
                            uint32_t D, void* const* d_outs, const uint64_t* out_capacities,
                            uint64_t* out_elems, void* d_workspace, uint64_t workspace_bytes, void* stream) {
  if (d_outs == nullptr || out_capacities == nullptr) return TM_ERR_ARG;
  return one_shot(descs, plane_n_desc, n_planes, r, D, d_outs, out_capacities, out_elems, d_workspace, workspace_bytes,
                  stream, /*to_tensors=*/false);
}

int tm_shard_insert(const tm_desc* plane_descs, uint64_t n_desc, uint32_t r, uint32_t D, const void* d_in,
                    uint64_t in_bytes, uint64_t* in_elems, void* d_workspace, uint64_t workspace_bytes,
                    void* stream) {
  void* flats[1] = {const_cast<void*>(d_in)};
  return one_shot(plane_descs, &n_desc, 1, r, D, flats, &in_bytes, in_elems, d_workspace, workspace_bytes, stream,
                  /*to_tensors=*/true);
}

int tm_shard_plan_create(const tm_desc* descs, const uint64_t* plane_n_desc, uint32_t n_planes, uint32_t r,
                         uint32_t D, tm_shard_plan** out) {
  if (out == nullptr) return TM_ERR_ARG;
  *out = nullptr;
  return guarded([&]() -> int {
    tm_shard_plan* sp = new tm_shard_plan();
    int rc = TM_ERR_CAPACITY;
    try {
      rc = plan_build(sp, descs, plane_n_desc, n_planes, r, D);
    } catch (...) {
      delete sp;
      throw;
    }
    if (rc != TM_OK) {
      delete sp;
      return rc;
    }
    *out = sp;
    return TM_OK;
  });
}

int tm_shard_plan_query(const tm_shard_plan* sp, uint64_t* out_elems, uint64_t* workspace_bytes) {
  if (sp == nullptr) return TM_ERR_ARG;
  if (out_elems != nullptr)
    for (size_t p = 0; p < sp->plane_n.size(); ++p) out_elems[p] = sp->hi[p] - sp->lo[p];
  if (workspace_bytes != nullptr) *workspace_bytes = workspace_bound(sp);
  return TM_OK;
}

int tm_shard_plan_bind(tm_shard_plan* sp, void* const* d_flats, const uint64_t* capacities, void* d_workspace,
                       uint64_t workspace_bytes, void* stream) {
  if (sp == nullptr) return TM_ERR_ARG;
  return guarded([&]() -> int { return plan_bind(sp, d_flats, capacities, d_workspace, workspace_bytes, stream); });
}

int tm_shard_plan_extract(const tm_shard_plan* sp, void* stream) {
  if (sp == nullptr) return TM_ERR_ARG;
  return plan_run(sp, /*to_tensors=*/false, stream);
}

int tm_shard_plan_insert(const tm_shard_plan* sp, void* stream) {
  if (sp == nullptr) return TM_ERR_ARG;
  return guarded([&]() -> int {
    int rc = insert_targets_ok(const_cast<tm_shard_plan*>(sp));
    if (rc != TM_OK) return rc;
    return plan_run(sp, /*to_tensors=*/true, stream);
  });
}

int tm_shard_plan_status(const tm_shard_plan* sp, void* stream, int* device_status) {
  if (sp == nullptr || device_status == nullptr) return TM_ERR_ARG;
  if (sp->d_workspace == nullptr) return TM_ERR_STATE;
  return tms::read_status_word(sp->d_workspace, stream, device_status);
}

void tm_shard_plan_destroy(tm_shard_plan* sp) { delete sp; }

}  // extern "C"
