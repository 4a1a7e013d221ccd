// Host planner: packed-stream layout and device work lists.  Pure host code, no CUDA calls.
//
// The format follows the definitions in tm_state.h (the paper — §7 "State Synchronization" —
// fixes what is moved, not how it is laid out).
#include <algorithm>
#include <cstdlib>
#include <cstring>

#include "tm_internal.h"

namespace tms {

static uint64_t env_u64(const char* name, uint64_t dflt) {
  const char* v = std::getenv(name);
  if (v == nullptr || *v == '\0') return dflt;
  char* end = nullptr;
  unsigned long long x = std::strtoull(v, &end, 10);
  return (end != nullptr && *end == '\0' && x > 0) ? (uint64_t)x : dflt;
}

const Tuning& tuning() {
  static const Tuning t = [] {
    Tuning x;
    x.chunk_bytes = align_up(env_u64("TM_CHUNK_BYTES", 256 * 1024), 256);
    if (x.chunk_bytes > (1ull << 30)) x.chunk_bytes = 1ull << 30;
    x.shard_chunk_bytes = align_up(env_u64("TM_SHARD_CHUNK_BYTES", 64 * 1024), 256);
    if (x.shard_chunk_bytes > (1ull << 30)) x.shard_chunk_bytes = 1ull << 30;
    x.cksum_tile_bytes = align_up(env_u64("TM_CKSUM_TILE_BYTES", 256 * 1024), 256);
    if (x.cksum_tile_bytes > (1ull << 30)) x.cksum_tile_bytes = 1ull << 30;
    x.small_bytes = env_u64("TM_SMALL_BYTES", 8 * 1024);
    x.group_bytes = env_u64("TM_GROUP_BYTES", 64 * 1024);
    x.group_max = (uint32_t)env_u64("TM_GROUP_MAX", 64);
    x.ctas_per_sm = (uint32_t)env_u64("TM_CTAS_PER_SM", 4);
    x.ring_ctas_per_sm = (uint32_t)env_u64("TM_RING_CTAS_PER_SM", 1);
    const char* ring = std::getenv("TM_USE_RING");
    x.use_ring = !(ring != nullptr && ring[0] == '0');
    return x;
  }();
  return t;
}

WorkspaceLayout workspace_layout(uint64_t n_segs, uint64_t n_items) {
  WorkspaceLayout l;
  l.segs_off = kStatusBlockBytes;
  l.items_off = align_up(l.segs_off + n_segs * sizeof(Seg), 256);
  l.total = align_up(l.items_off + (n_items + 1) * sizeof(uint32_t), 256);
  return l;
}

WorkListBuilder::WorkListBuilder(WorkList* wl) : wl_(wl) {
  wl_->segs.clear();
  wl_->item_first.clear();
}

void WorkListBuilder::close_group() {
  open_ = false;
  group_bytes_ = 0;
  group_count_ = 0;
}

void WorkListBuilder::add(const Seg& s) {
  const Tuning& t = tuning();
  const uint64_t span = (uint64_t)s.nbytes + s.pad;
  const uint32_t index = (uint32_t)wl_->segs.size();
  if (span >= t.small_bytes) {          // a block-wide item of its own
    close_group();
    wl_->item_first.push_back(index);
  } else {
    const bool fits = open_ && s.bucket == group_bucket_ && group_bytes_ + span <= t.group_bytes &&
                      group_count_ < t.group_max;
    if (!fits) {
      wl_->item_first.push_back(index);
      open_ = true;
      group_bytes_ = 0;
      group_count_ = 0;
      group_bucket_ = s.bucket;
    }
    group_bytes_ += span;
    group_count_ += 1;
  }
  wl_->segs.push_back(s);
}

void WorkListBuilder::finish() {
  close_group();
  wl_->item_first.push_back((uint32_t)wl_->segs.size());
}

}  // namespace tms

using tms::Seg;

static inline uint64_t align256(uint64_t x) { return (x + 255) & ~(uint64_t)255; }

// Validates the descriptors, computes off_k / T / n_buckets and the pack/unpack work list.
int tm_plan_build(tm_plan* p, const tm_desc* descs, uint64_t n_desc, uint64_t bucket_bytes) {
  if (descs == nullptr || n_desc == 0 || bucket_bytes == 0) return TM_ERR_ARG;
  if (bucket_bytes > (1ull << 35)) return TM_ERR_ARG;
  if (bucket_bytes % 256 != 0) return TM_ERR_ALIGN;
  for (uint64_t k = 0; k < n_desc; ++k) {
    const tm_desc& d = descs[k];
    if (d.elem_size != 2 && d.elem_size != 4 && d.elem_size != 8) return TM_ERR_DTYPE;
    if (d.ptr == nullptr || d.nbytes == 0 || d.nbytes % d.elem_size != 0) return TM_ERR_ARG;
    if (d.nbytes > (1ull << 46)) return TM_ERR_ARG;   // keeps every offset far from 64-bit wrap-around
    if (((uintptr_t)d.ptr & 1) != 0) return TM_ERR_ALIGN;
  }
  if (n_desc > (1ull << 24)) return TM_ERR_ARG;
  p->descs.assign(descs, descs + n_desc);
  p->bucket_bytes = bucket_bytes;
  p->offsets.resize(n_desc);

  const uint64_t chunk = tms::tuning().chunk_bytes;
  tms::WorkListBuilder builder(&p->work);
  uint64_t pos = 0;
  for (uint64_t k = 0; k < n_desc; ++k) {
    const uint64_t off = align256(pos);
    p->offsets[k] = off;
    uint64_t tensor = (uint64_t)(uintptr_t)descs[k].ptr;
    uint64_t cur = off;
    uint64_t remaining = descs[k].nbytes;
    while (remaining > 0) {
      const uint64_t bucket = cur / bucket_bytes;
      const uint64_t bucket_end = (bucket + 1) * bucket_bytes;
      uint64_t len = std::min(remaining, chunk);
      len = std::min(len, bucket_end - cur);
      Seg s;
      s.tensor = tensor;
      s.off = cur;
      s.nbytes = (uint32_t)len;
      s.pad = 0;
      s.bucket = (uint32_t)bucket;
      s.word0 = (uint32_t)((cur - bucket * bucket_bytes) / 8);
      remaining -= len;
      if (remaining == 0) s.pad = (uint32_t)(align256(cur + len) - (cur + len));
      builder.add(s);
      tensor += len;
      cur += len;
    }
    pos = off + descs[k].nbytes;
  }
  builder.finish();
  p->total_bytes = align256(pos);
  p->n_buckets = (p->total_bytes + bucket_bytes - 1) / bucket_bytes;
  if (p->work.segs.size() >= (1ull << 32) - (1u << 20)) return TM_ERR_ARG;   // piece and item indices are 32-bit
  p->ws_layout = tms::workspace_layout(p->work.segs.size(), p->work.n_items());
  return TM_OK;
}

// floor(r*N/D) and floor((r+1)*N/D) with 128-bit products.
int tm_bounds_u128(uint64_t n_elems, uint32_t r, uint32_t D, uint64_t* lo, uint64_t* hi) {
  if (D == 0 || r >= D) return TM_ERR_RANK;
  const unsigned __int128 n = n_elems;
  *lo = (uint64_t)((n * r) / D);
  *hi = (uint64_t)((n * ((unsigned __int128)r + 1)) / D);
  return TM_OK;
}

// Validates a shard plane and returns its element size and element count.
int tm_shard_validate(const tm_desc* descs, uint64_t n_desc, uint32_t r, uint32_t D,
                      uint32_t* elem_size, uint64_t* n_elems) {
  if (descs == nullptr || n_desc == 0 || n_desc > (1ull << 24)) return TM_ERR_ARG;
  if (D == 0 || r >= D) return TM_ERR_RANK;
  const uint32_t e = descs[0].elem_size;
  if (e != 2 && e != 4 && e != 8) return TM_ERR_DTYPE;
  uint64_t total = 0;
  for (uint64_t k = 0; k < n_desc; ++k) {
    const tm_desc& d = descs[k];
    if (d.elem_size != e) return TM_ERR_DTYPE;
    if (d.ptr == nullptr || d.nbytes == 0 || d.nbytes % e != 0 || d.nbytes > (1ull << 46)) return TM_ERR_ARG;
    if (((uintptr_t)d.ptr & 1) != 0) return TM_ERR_ALIGN;
    total += d.nbytes / e;
  }
  *elem_size = e;
  *n_elems = total;
  return TM_OK;
}

// Appends the pieces that gather elements [lo, hi) of one plane into a contiguous output at address
// d_out; piece offsets are relative to `flat_base` (<= d_out).  Pieces after the first of each
// tensor start on a 256-byte boundary of the output.
void tm_shard_append(tms::WorkListBuilder* builder, const tm_desc* descs, uint64_t n_desc, uint32_t e,
                     uint64_t lo, uint64_t hi, uint64_t d_out, uint64_t flat_base, uint32_t bucket_tag) {
  const uint64_t chunk = tms::tuning().shard_chunk_bytes;
  uint64_t start = 0;  // element index of the tensor's first element in the flat plane
  for (uint64_t k = 0; k < n_desc && start < hi; ++k) {
    const uint64_t count = descs[k].nbytes / e;
    const uint64_t a = std::max(lo, start);
    const uint64_t b = std::min(hi, start + count);
    if (a < b) {
      uint64_t tensor = (uint64_t)(uintptr_t)descs[k].ptr + (a - start) * e;
      uint64_t out = (a - lo) * e;
      uint64_t remaining = (b - a) * e;
      while (remaining > 0) {
        uint64_t len = chunk;
        const uint64_t mis = (d_out + out) % 256;
        if (mis != 0) len = chunk - mis;
        len = std::min(len, remaining);
        Seg s;
        s.tensor = tensor;
        s.off = (d_out - flat_base) + out;
        s.nbytes = (uint32_t)len;
        s.pad = 0;
        s.bucket = bucket_tag;
        s.word0 = 0;
        builder->add(s);
        tensor += len;
        out += len;
        remaining -= len;
      }
    }
    start += count;
  }
}

// Work list for one plane, offsets relative to d_out.
void tm_shard_worklist(const tm_desc* descs, uint64_t n_desc, uint32_t e, uint64_t lo, uint64_t hi,
                       uint64_t d_out, tms::WorkList* wl) {
  tms::WorkListBuilder builder(wl);
  tm_shard_append(&builder, descs, n_desc, e, lo, hi, d_out, d_out, 0);
  builder.finish();
}

// 1 when no two tensors of the plan overlap, -1 otherwise.
int tm_targets_disjoint(const tm_plan* p) {
  std::vector<std::pair<uint64_t, uint64_t>> r;
  r.reserve(p->descs.size());
  for (const tm_desc& d : p->descs) r.emplace_back((uint64_t)(uintptr_t)d.ptr, d.nbytes);
  std::sort(r.begin(), r.end());
  for (size_t i = 1; i < r.size(); ++i)
    if (r[i - 1].first + r[i - 1].second > r[i].first) return -1;
  return 1;
}
