// Host planner: packed-stream layout and device work lists.  Pure host code, no CUDA calls.
//
// The format follows the definitions in tm_state.h (the paper — §7 "State Synchronization" —
// fixes what is moved, not how it is laid out).
#include <algorithm>
#include <cstring>
#include <mutex>

#include "tm_internal.h"

namespace tms {

Tuning default_tuning() {
  Tuning x;
  std::memset(&x, 0, sizeof(x));
  x.chunk_bytes = 256 * 1024;
  x.shard_chunk_bytes = 64 * 1024;
  x.small_bytes = 8 * 1024;
  x.group_bytes = 64 * 1024;
  x.cksum_tile_bytes = 256 * 1024;
  x.wait_limit_ns = 2000000000ull;
  x.group_max = 64;
  x.ring_ctas_per_sm = 1;
  x.ctas_per_sm = 4;
  return x;
}

static std::mutex g_tuning_mutex;
static Tuning g_tuning = default_tuning();

Tuning tuning() {
  std::lock_guard<std::mutex> lock(g_tuning_mutex);
  return g_tuning;
}

int set_tuning(const Tuning* t) {
  Tuning x = (t == nullptr) ? default_tuning() : *t;
  const uint64_t kib4 = 4096, gib = 1ull << 30;
  if (x.chunk_bytes < kib4 || x.chunk_bytes > gib || x.shard_chunk_bytes < kib4 || x.shard_chunk_bytes > gib ||
      x.cksum_tile_bytes < kib4 || x.cksum_tile_bytes > gib)
    return TM_ERR_ARG;
  if (x.chunk_bytes % 256 != 0 || x.shard_chunk_bytes % 256 != 0 || x.cksum_tile_bytes % 256 != 0) return TM_ERR_ALIGN;
  if (x.small_bytes == 0 || x.small_bytes > gib || x.group_bytes == 0 || x.group_bytes > gib) return TM_ERR_ARG;
  if (x.wait_limit_ns == 0 || x.wait_limit_ns > 5000000000ull) return TM_ERR_ARG;
  if (x.group_max == 0 || x.group_max > 1024) return TM_ERR_ARG;
  if (x.ring_ctas_per_sm == 0 || x.ring_ctas_per_sm > 2 || x.ctas_per_sm == 0 || x.ctas_per_sm > 8) return TM_ERR_ARG;
  if (x.reserved != 0) return TM_ERR_ARG;
  std::lock_guard<std::mutex> lock(g_tuning_mutex);
  g_tuning = x;
  return TM_OK;
}

WorkspaceLayout workspace_layout(uint64_t n_segs, uint64_t n_items, bool with_emits) {
  WorkspaceLayout l;
  l.segs_off = kStatusBlockBytes;
  l.items_off = align_up(l.segs_off + n_segs * sizeof(Seg), 256);
  l.emits_off = align_up(l.items_off + (n_items + 1) * sizeof(uint32_t), 256);
  l.total = with_emits ? align_up(l.emits_off + n_segs * sizeof(Emit), 256) : l.emits_off;
  return l;
}

WorkListBuilder::WorkListBuilder(WorkList* wl, const Tuning& t) : wl_(wl), t_(t) {
  wl_->segs.clear();
  wl_->item_first.clear();
}

void WorkListBuilder::close_group() {
  open_ = false;
  group_bytes_ = 0;
  group_count_ = 0;
}

void WorkListBuilder::add(const Seg& s) {
  const uint64_t span = (uint64_t)s.nbytes + s.pad;
  const uint32_t index = (uint32_t)wl_->segs.size();
  if (span >= t_.small_bytes) {          // a block-wide item of its own
    close_group();
    wl_->item_first.push_back(index);
  } else {
    const bool fits = open_ && s.bucket == group_bucket_ && group_bytes_ + span <= t_.group_bytes &&
                      group_count_ < t_.group_max;
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

// Validates the descriptors and computes off_k, T and the bucket count of the complete stream.
int tm_layout_build(const tm_desc* descs, uint64_t n_desc, uint64_t bucket_bytes, tm_layout* out) {
  if (descs == nullptr || n_desc == 0 || bucket_bytes == 0) return TM_ERR_ARG;
  if (bucket_bytes > (1ull << 35)) return TM_ERR_ARG;
  if (bucket_bytes % 256 != 0) return TM_ERR_ALIGN;
  if (n_desc > tms::kMaxDescs) return TM_ERR_ARG;
  uint64_t sum = 0;   // running stream length; bounded inside the loop, so it cannot wrap
  for (uint64_t k = 0; k < n_desc; ++k) {
    const tm_desc& d = descs[k];
    if (d.elem_size != 2 && d.elem_size != 4 && d.elem_size != 8) return TM_ERR_DTYPE;
    if (d.ptr == nullptr || d.nbytes == 0 || d.nbytes % d.elem_size != 0) return TM_ERR_ARG;
    if (d.nbytes > tms::kMaxTensorBytes) return TM_ERR_ARG;
    if (((uintptr_t)d.ptr & 1) != 0) return TM_ERR_ALIGN;
    sum = align256(sum) + d.nbytes;
    if (sum > tms::kMaxTotalBytes) return TM_ERR_ARG;
  }
  out->offsets.resize(n_desc);
  uint64_t pos = 0;
  for (uint64_t k = 0; k < n_desc; ++k) {
    out->offsets[k] = align256(pos);
    pos = out->offsets[k] + descs[k].nbytes;
  }
  out->bucket_bytes = bucket_bytes;
  out->whole_bytes = align256(pos);
  out->whole_buckets = (out->whole_bytes + bucket_bytes - 1) / bucket_bytes;
  return TM_OK;
}

// Cuts the part of the stream that the plan covers (all buckets unless `ranged`) into the pack /
// unpack work list.  `cursor` (may be NULL): in, a descriptor index at or before the first tensor
// that reaches into the range; out, the last tensor that does — consecutive ranges of one role are
// then cut in one pass over the descriptors.  The list is refused (TM_ERR_CAPACITY) before any of it
// is built when it would exceed kMaxPieces pieces.
int tm_plan_fill(tm_plan* p, const tm_desc* descs, uint64_t n_desc, const tm_layout& lay, bool ranged,
                 uint64_t first_bucket, uint64_t n_buckets, uint64_t* cursor) {
  if (ranged && n_buckets == 0) return TM_ERR_ARG;
  const uint64_t bucket_bytes = lay.bucket_bytes;
  p->opt = tms::tuning();
  p->bucket_bytes = bucket_bytes;
  p->whole_bytes = lay.whole_bytes;
  p->whole_buckets = lay.whole_buckets;
  uint64_t range_lo = 0, range_hi = p->whole_bytes;
  if (ranged) {
    if (first_bucket >= p->whole_buckets) return TM_ERR_ARG;
    const uint64_t count = std::min(n_buckets, p->whole_buckets - first_bucket);
    range_lo = first_bucket * bucket_bytes;
    range_hi = std::min((first_bucket + count) * bucket_bytes, p->whole_bytes);
    p->first_bucket = first_bucket;
    p->n_buckets = count;
  } else {
    p->first_bucket = 0;
    p->n_buckets = p->whole_buckets;
  }
  p->range_begin = range_lo;
  p->total_bytes = range_hi - range_lo;

  const uint64_t chunk = p->opt.chunk_bytes;
  // first tensor that reaches into the range
  uint64_t k0 = (cursor != nullptr && *cursor < n_desc) ? *cursor : 0;
  while (k0 > 0 && lay.offsets[k0] > range_lo) --k0;
  while (k0 < n_desc && lay.offsets[k0] + descs[k0].nbytes <= range_lo) ++k0;
  // upper bound on the pieces: a part of n bytes is cut at chunk ends and at bucket ends
  uint64_t bound = 0;
  for (uint64_t k = k0; k < n_desc && lay.offsets[k] < range_hi; ++k) {
    const uint64_t a = std::max(lay.offsets[k], range_lo), b = std::min(lay.offsets[k] + descs[k].nbytes, range_hi);
    if (a < b) bound += (b - a) / chunk + (b - a) / bucket_bytes + 2;
    if (bound > tms::kMaxPieces) return TM_ERR_CAPACITY;
  }

  tms::WorkListBuilder builder(&p->work, p->opt);
  p->piece_desc.clear();
  p->parts.clear();
  p->box_lo = ~0ull;
  p->box_hi = 0;
  uint64_t last = k0;
  for (uint64_t k = k0; k < n_desc && lay.offsets[k] < range_hi; ++k) {
    const uint64_t off = lay.offsets[k];
    const uint64_t end = off + descs[k].nbytes;
    const uint64_t a = std::max(off, range_lo), b = std::min(end, range_hi);
    if (a >= b) continue;                                   // the tensor has no byte in the range
    last = k;
    uint64_t tensor = (uint64_t)(uintptr_t)descs[k].ptr + (a - off);
    p->parts.push_back(tm_part{tensor, b - a});
    p->box_lo = std::min(p->box_lo, tensor);
    p->box_hi = std::max(p->box_hi, tensor + (b - a));
    uint64_t cur = a;
    uint64_t remaining = b - a;
    while (remaining > 0) {
      const uint64_t bucket = cur / bucket_bytes;
      const uint64_t bucket_end = (bucket + 1) * bucket_bytes;
      uint64_t len = std::min(remaining, chunk);
      len = std::min(len, bucket_end - cur);
      Seg s;
      s.tensor = tensor;
      s.off = cur - range_lo;
      s.nbytes = (uint32_t)len;
      s.pad = 0;
      s.bucket = (uint32_t)(bucket - p->first_bucket);
      s.word0 = (uint32_t)((cur - bucket * bucket_bytes) / 8);
      remaining -= len;
      // the padding after a tensor's last byte belongs to the piece that holds that byte; it ends on a
      // multiple of 256 and therefore never crosses the end of the range
      if (remaining == 0 && b == end) s.pad = (uint32_t)(align256(end) - end);
      builder.add(s);
      p->piece_desc.push_back((uint32_t)k);
      tensor += len;
      cur += len;
    }
  }
  builder.finish();
  if (cursor != nullptr) *cursor = last;
  if (p->box_lo == ~0ull) p->box_lo = 0;
  p->ws_layout = tms::workspace_layout(p->work.segs.size(), p->work.n_items());
  return TM_OK;
}

// A plan that owns its copy of the descriptors and offsets (what the public plan calls need).
int tm_plan_build(tm_plan* p, const tm_desc* descs, uint64_t n_desc, uint64_t bucket_bytes, bool ranged,
                  uint64_t first_bucket, uint64_t n_buckets) {
  tm_layout lay;
  int rc = tm_layout_build(descs, n_desc, bucket_bytes, &lay);
  if (rc != TM_OK) return rc;
  rc = tm_plan_fill(p, descs, n_desc, lay, ranged, first_bucket, n_buckets, nullptr);
  if (rc != TM_OK) return rc;
  p->descs.assign(descs, descs + n_desc);
  p->offsets = std::move(lay.offsets);
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
  if (descs == nullptr || n_desc == 0 || n_desc > tms::kMaxDescs) return TM_ERR_ARG;
  if (D == 0 || r >= D) return TM_ERR_RANK;
  const uint32_t e = descs[0].elem_size;
  if (e != 2 && e != 4 && e != 8) return TM_ERR_DTYPE;
  uint64_t total = 0, bytes = 0;
  for (uint64_t k = 0; k < n_desc; ++k) {
    const tm_desc& d = descs[k];
    if (d.elem_size != e) return TM_ERR_DTYPE;
    if (d.ptr == nullptr || d.nbytes == 0 || d.nbytes % e != 0 || d.nbytes > tms::kMaxTensorBytes) return TM_ERR_ARG;
    if (((uintptr_t)d.ptr & 1) != 0) return TM_ERR_ALIGN;
    total += d.nbytes / e;
    bytes += d.nbytes;
    if (bytes > tms::kMaxTotalBytes) return TM_ERR_ARG;   // (hi - lo) * e stays far below 2^64
  }
  *elem_size = e;
  *n_elems = total;
  return TM_OK;
}

// Appends the pieces that gather elements [lo, hi) of one plane into a contiguous output at address
// d_out; piece offsets are relative to `flat_base` (<= d_out).  Pieces after the first of each
// tensor start on a 256-byte boundary of the output.
void tm_shard_append(tms::WorkListBuilder* builder, const tms::Tuning& t, const tm_desc* descs, uint64_t n_desc,
                     uint32_t e, uint64_t lo, uint64_t hi, uint64_t d_out, uint64_t flat_base) {
  const uint64_t chunk = t.shard_chunk_bytes;
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
        s.bucket = 0;
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
void tm_shard_worklist(const tms::Tuning& t, const tm_desc* descs, uint64_t n_desc, uint32_t e, uint64_t lo,
                       uint64_t hi, uint64_t d_out, tms::WorkList* wl) {
  tms::WorkListBuilder builder(wl, t);
  tm_shard_append(&builder, t, descs, n_desc, e, lo, hi, d_out, d_out);
  builder.finish();
}

// 1 when no two parts overlap, -1 otherwise.
int tm_parts_disjoint(std::vector<tm_part> r) {
  std::sort(r.begin(), r.end(), [](const tm_part& a, const tm_part& b) { return a.addr < b.addr; });
  for (size_t i = 1; i < r.size(); ++i)
    if (r[i - 1].addr + r[i - 1].nbytes > r[i].addr) return -1;
  return 1;
}
