// Internal declarations shared by the host planner, the kernels and the C ABI.
#ifndef TM_INTERNAL_H
#define TM_INTERNAL_H

#include <cstdint>
#include <utility>
#include <vector>

#include "tm_state.h"

namespace tms {

// One contiguous piece of one tensor and its place in a flat buffer (the packed stream, or a
// shard output).  Pieces never cross a bucket boundary, so a piece belongs to one bucket.
struct alignas(16) Seg {
  uint64_t tensor;  // device address of the piece's first tensor byte (>= 2-byte aligned)
  uint64_t off;     // byte offset of the piece in the flat buffer
  uint32_t nbytes;  // tensor bytes in the piece; even, > 0
  uint32_t pad;     // pack only: zero bytes that follow the piece in the stream (< 256)
  uint32_t bucket;  // pack only: bucket the piece lies in
  uint32_t word0;   // pack only: index, inside that bucket, of the piece's first 8-byte word
};
static_assert(sizeof(Seg) == 32, "Seg is 32 bytes on host and device");

// Optional second destination of a pack piece: bytes [begin, begin + len) of the piece also go to
// the device address `out` (a shard output).  len == 0: nothing to emit.  One record per piece.
struct alignas(16) Emit {
  uint64_t out;
  uint32_t begin;
  uint32_t len;
};
static_assert(sizeof(Emit) == 16, "Emit is 16 bytes on host and device");

// A work list: pieces grouped into items.  Item i owns pieces [item_first[i], item_first[i+1]).
// A large piece is an item of its own (a whole thread block works on it); runs of small pieces
// share an item (one warp per piece).  All pieces of an item lie in one bucket.
struct WorkList {
  std::vector<Seg> segs;
  std::vector<uint32_t> item_first;  // n_items + 1 entries
  uint64_t n_items() const { return item_first.empty() ? 0 : item_first.size() - 1; }
};

// Process-wide tuning values (tm_options_get / tm_options_set); a plan keeps the copy it was built with.
typedef tm_options Tuning;
Tuning tuning();
Tuning default_tuning();
int set_tuning(const Tuning* t);   // validates; nullptr restores the defaults

// Incrementally groups pieces into items.
class WorkListBuilder {
 public:
  WorkListBuilder(WorkList* wl, const Tuning& t);
  void add(const Seg& s);
  void finish();

 private:
  WorkList* wl_;
  Tuning t_;
  uint64_t group_bytes_ = 0;
  uint32_t group_count_ = 0;
  uint32_t group_bucket_ = 0;
  bool open_ = false;
  void close_group();
};

// Byte layout of a work list inside a device workspace.
struct WorkspaceLayout {
  uint64_t segs_off;    // 256: after the status block
  uint64_t items_off;
  uint64_t emits_off;   // one Emit per piece (only lists that emit; otherwise == total)
  uint64_t total;
};
WorkspaceLayout workspace_layout(uint64_t n_segs, uint64_t n_items, bool with_emits = false);
constexpr uint64_t kStatusBlockBytes = 256;  // word 0: device status (0 ok, else tm_status)

inline uint64_t align_up(uint64_t x, uint64_t a) { return (x + a - 1) / a * a; }
inline bool ranges_overlap(uint64_t a, uint64_t an, uint64_t b, uint64_t bn) { return a < b + bn && b < a + an; }

// Sizes beyond these are refused: with them no sum of sizes or offsets formed by the planner can
// reach 2^63.
constexpr uint64_t kMaxTensorBytes = 1ull << 46;
constexpr uint64_t kMaxDescs = 1ull << 24;
constexpr uint64_t kMaxTotalBytes = 1ull << 56;
// Longest work list that is built (pieces): 16 M pieces are 512 MiB of host memory and, at the default
// piece sizes, 4 TiB of stream or 1 TiB of shard.  Longer lists are refused before anything is allocated.
constexpr uint64_t kMaxPieces = 1ull << 24;

// ---- kernel launchers.  Each returns a cudaError_t as int. -----------------------------------
// What a ring launch does with the pieces of its list.
enum RingMode {
  kRingPack,          // tensors -> stream, zero padding, per-bucket checksums
  kRingPackEmit,      // the same, and every piece's emit span also goes to its shard output
  kRingToFlat,        // tensors -> flat buffer (shard extract)
  kRingToTensors,     // flat buffer -> tensors (unpack, shard insert)
  kRingToTensorsVerify,  // unpack that also accumulates the checksums of the stream as read
  kRingToTensorsVerifyEmit  // the same, and every piece's emit span also goes to its shard output
};
struct RingLaunch {
  const Seg* d_segs = nullptr;
  const uint32_t* d_item_first = nullptr;
  const Emit* d_emits = nullptr;
  uint32_t n_items = 0;
  uint8_t* d_flat = nullptr;
  unsigned long long* d_checksums = nullptr;
  int* d_status = nullptr;
  unsigned long long wait_limit_ns = 0;
  uint32_t ctas_per_sm = 1;
};
int launch_ring(RingMode mode, const RingLaunch& a, void* stream);
// register-path copy tensors -> flat (used by the entry point that owns its scratch)
int launch_copy_to_flat(const Seg* d_segs, const uint32_t* d_item_first, uint32_t n_items, uint8_t* d_flat,
                        uint32_t ctas_per_sm, void* stream);
int launch_wait_selftest(int* d_status, unsigned long long limit_ns, void* stream);
int launch_checksum(const uint8_t* d_bytes, uint64_t nbytes, uint64_t bucket_bytes,
                    unsigned long long* d_checksums, const Tuning& t, void* stream);
int device_sm_count(int* sms);
void count_launch();

// ---- shared host helpers (api.cpp) ------------------------------------------------------------
int cuda_fail(int cuda_error);   // records the error for tm_last_cuda_error(), returns TM_ERR_CUDA
// Uploads status block + pieces + items (+ emits) as one image; asynchronous on `stream`.
int upload_worklist(const WorkList& wl, const std::vector<Emit>* emits, const WorkspaceLayout& l, uint8_t* d_ws,
                    void* stream);
int read_status_word(const void* d_ws, void* stream, int* device_status);

}  // namespace tms

// One part of a tensor that a plan touches (a range plan touches only part of the role).
struct tm_part {
  uint64_t addr;
  uint64_t nbytes;
};

struct tm_plan {
  std::vector<tm_desc> descs;
  std::vector<uint64_t> offsets;     // off_k in the complete stream
  tms::Tuning opt{};
  uint64_t bucket_bytes = 0;
  uint64_t whole_bytes = 0;          // T of the complete stream
  uint64_t whole_buckets = 0;
  uint64_t first_bucket = 0;         // range plans: first bucket covered
  uint64_t range_begin = 0;          // = first_bucket * bucket_bytes
  uint64_t total_bytes = 0;          // bytes this plan packs / unpacks (the whole stream, or the range)
  uint64_t n_buckets = 0;            // buckets this plan covers
  tms::WorkList work;
  std::vector<uint32_t> piece_desc;  // descriptor index of every piece
  std::vector<tm_part> parts;        // tensor parts touched by the plan
  uint64_t box_lo = 0, box_hi = 0;   // address bounding box of `parts`
  tms::WorkspaceLayout ws_layout{};
  // set by tm_plan_upload
  uint8_t* d_workspace = nullptr;
  // set by tm_plan_attach_shards: the same work list with one emit record per piece
  std::vector<tms::Emit> emits;
  tms::WorkspaceLayout emit_layout{};
  uint8_t* d_emit_workspace = nullptr;
  std::vector<std::pair<uint64_t, uint64_t>> emit_outs;   // (address, bytes) of every non-empty shard output
  // lazily computed: 0 unknown, 1 targets disjoint, -1 targets overlap
  mutable int targets_disjoint = 0;
};

// Reusable shard plan: the same [lo, hi) of one or several planes, bound to flat buffers.
struct tm_shard_plan {
  std::vector<tm_desc> descs;
  std::vector<uint64_t> plane_n;
  std::vector<uint32_t> elem_size;
  std::vector<uint64_t> lo, hi;
  tms::Tuning opt{};
  uint32_t r = 0, D = 0;
  // set by tm_shard_plan_bind
  tms::WorkList work;
  tms::WorkspaceLayout layout{};
  std::vector<std::pair<uint64_t, uint64_t>> flats;   // (address, bytes) per plane (0 bytes: empty shard)
  uint64_t base = 0;                                   // lowest flat address; piece offsets are relative to it
  uint8_t* d_workspace = nullptr;
  int targets_disjoint = 0;
};

// Layout of a complete stream: off_k of every descriptor, T and the bucket count.
struct tm_layout {
  std::vector<uint64_t> offsets;
  uint64_t bucket_bytes = 0, whole_bytes = 0, whole_buckets = 0;
};

// planner (plan.cpp)
int tm_layout_build(const tm_desc* descs, uint64_t n_desc, uint64_t bucket_bytes, tm_layout* out);
int tm_plan_fill(tm_plan* p, const tm_desc* descs, uint64_t n_desc, const tm_layout& lay, bool ranged,
                 uint64_t first_bucket, uint64_t n_buckets, uint64_t* cursor);
int tm_plan_build(tm_plan* p, const tm_desc* descs, uint64_t n_desc, uint64_t bucket_bytes, bool ranged,
                  uint64_t first_bucket, uint64_t n_buckets);
int tm_attach_shards(tm_plan* plan, const tm_desc* descs, uint64_t n_desc, const uint64_t* plane_first_desc,
                     const uint64_t* plane_n_desc, uint32_t n_planes, uint32_t r, uint32_t D, void* const* d_outs,
                     const uint64_t* out_capacities, uint64_t* out_elems, void* d_workspace,
                     uint64_t workspace_bytes, uint64_t* workspace_needed, void* stream);   // api.cpp
int tm_bounds_u128(uint64_t n_elems, uint32_t r, uint32_t D, uint64_t* lo, uint64_t* hi);
int tm_shard_validate(const tm_desc* descs, uint64_t n_desc, uint32_t r, uint32_t D, uint32_t* elem_size,
                      uint64_t* n_elems);
void tm_shard_append(tms::WorkListBuilder* builder, const tms::Tuning& t, const tm_desc* descs, uint64_t n_desc,
                     uint32_t e, uint64_t lo, uint64_t hi, uint64_t d_out, uint64_t flat_base);
void tm_shard_worklist(const tms::Tuning& t, const tm_desc* descs, uint64_t n_desc, uint32_t e, uint64_t lo,
                       uint64_t hi, uint64_t d_out, tms::WorkList* wl);
int tm_parts_disjoint(std::vector<tm_part> parts);   // 1 disjoint, -1 overlap

#endif  // TM_INTERNAL_H
