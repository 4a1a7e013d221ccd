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

// A work list: pieces grouped into items.  Item i owns pieces [item_first[i], item_first[i+1]).
// A large piece is an item of its own (a whole thread block works on it); runs of small pieces
// share an item (one warp per piece).  All pieces of an item lie in one bucket.
struct WorkList {
  std::vector<Seg> segs;
  std::vector<uint32_t> item_first;  // n_items + 1 entries
  uint64_t n_items() const { return item_first.empty() ? 0 : item_first.size() - 1; }
};

// Incrementally groups pieces into items.
class WorkListBuilder {
 public:
  explicit WorkListBuilder(WorkList* wl);
  void add(const Seg& s);
  void finish();

 private:
  WorkList* wl_;
  uint64_t group_bytes_ = 0;
  uint32_t group_count_ = 0;
  uint32_t group_bucket_ = 0;
  bool open_ = false;
  void close_group();
};

struct Tuning {
  uint64_t chunk_bytes;    // largest piece of a pack / unpack plan; multiple of 256
  uint64_t shard_chunk_bytes;  // largest piece of a shard list (smaller: a shard is a fraction of a role)
  uint64_t small_bytes;    // pieces below this share items
  uint64_t group_bytes;    // byte budget of a shared item
  uint32_t group_max;      // piece budget of a shared item
  uint64_t cksum_tile_bytes;   // tile of the stand-alone checksum kernel; multiple of 256
  uint32_t ctas_per_sm;    // persistent grid = SMs * ctas_per_sm (register-path kernels)
  uint32_t ring_ctas_per_sm;  // same for the bulk-copy ring kernels (96 KiB of shared memory each)
  bool use_ring;           // pack / unpack / shard through the bulk-copy ring kernels
};
const Tuning& tuning();

// Byte layout of a work list inside a device workspace.
struct WorkspaceLayout {
  uint64_t segs_off;    // 256: after the status block
  uint64_t items_off;
  uint64_t total;
};
WorkspaceLayout workspace_layout(uint64_t n_segs, uint64_t n_items);
constexpr uint64_t kStatusBlockBytes = 256;  // word 0: device status (0 ok, else tm_status)

inline uint64_t align_up(uint64_t x, uint64_t a) { return (x + a - 1) / a * a; }

// ---- kernel launchers (kernels.cu).  Each returns a cudaError_t as int. -----------------------
int launch_pack(const Seg* d_segs, const uint32_t* d_item_first, uint32_t n_items, uint8_t* d_stream,
                unsigned long long* d_checksums, int* d_status, void* stream);
// flat -> tensors when to_tensors, tensors -> flat otherwise (no checksum, no padding)
int launch_copy(const Seg* d_segs, const uint32_t* d_item_first, uint32_t n_items, uint8_t* d_flat,
                bool to_tensors, int* d_status, void* stream);
// bulk-copy ring versions (ring_kernels.cu); d_status receives TM_ERR_TIMEOUT if a bounded wait expires
int launch_pack_ring(const Seg* d_segs, const uint32_t* d_item_first, uint32_t n_items, uint8_t* d_stream,
                     unsigned long long* d_checksums, int* d_status, void* stream);
int launch_copy_ring(const Seg* d_segs, const uint32_t* d_item_first, uint32_t n_items, uint8_t* d_flat,
                     bool to_tensors, int* d_status, void* stream);
int launch_unpack_verify_ring(const Seg* d_segs, const uint32_t* d_item_first, uint32_t n_items, uint8_t* d_stream,
                              unsigned long long* d_checksums, int* d_status, void* stream);
int launch_pack_emit_ring(const Seg* d_segs, const uint32_t* d_item_first, uint32_t n_items, uint8_t* d_stream,
                          unsigned long long* d_checksums, uint8_t* d_emit_base, int* d_status, void* stream);
int launch_wait_selftest(int* d_status, unsigned long long limit_ns, void* stream);
int launch_checksum(const uint8_t* d_bytes, uint64_t nbytes, uint64_t bucket_bytes,
                    unsigned long long* d_checksums, void* stream);
int device_sm_count(int* sms);
void count_launch();

}  // namespace tms

struct tm_plan {
  std::vector<tm_desc> descs;
  std::vector<uint64_t> offsets;
  uint64_t bucket_bytes = 0;
  uint64_t total_bytes = 0;
  uint64_t n_buckets = 0;
  tms::WorkList work;
  tms::WorkspaceLayout ws_layout{};
  // set by tm_plan_upload
  uint8_t* d_workspace = nullptr;
  // set by tm_plan_attach_shards: pack pieces interleaved with the emit pieces of the attached shards
  tms::WorkList emit_work;
  tms::WorkspaceLayout emit_layout{};
  uint8_t* d_emit_workspace = nullptr;
  uint64_t emit_base = 0;                      // lowest shard output address; emit offsets are relative to it
  std::vector<std::pair<uint64_t, uint64_t>> emit_outs;   // (address, bytes) of every non-empty shard output
  // lazily computed: 0 unknown, 1 targets disjoint, -1 targets overlap
  mutable int targets_disjoint = 0;
};

#endif  // TM_INTERNAL_H
