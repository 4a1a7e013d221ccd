/*
 * tm_state.h — C ABI of the role-state mover.
 *
 * The operation family implemented here is the bulk state hand-over that
 * TrainMover performs in its switching phase (paper §7 "Implementation",
 * paragraph "State Synchronization"): a leaver sends its latest training
 * state — model parameters and optimizer states — to the joiner that takes
 * over its role, and with a distributed (ZeRO-style) optimizer a joiner needs
 * the slice of the optimizer state that belongs to its data-parallel rank.
 * §8.5 "Zero Memory Overhead Workflow" adds that the state travels through a
 * staging channel (the leaver's recycled gradient buffer), which is why the
 * state is first packed into flat, fixed-size transfer buckets.  The paper
 * fixes no wire format; the format below (256-byte alignment, fixed-size
 * buckets, floor shard bounds, weighted 64-bit word checksum) is this
 * library's definition.
 *
 * Definitions (all arithmetic on byte offsets is exact, uint64):
 *
 *   align256(x)   = (x + 255) & ~255
 *   Packed stream : descriptors are taken in the order given (never sorted).
 *                   off_0 = 0, off_k = align256(off_{k-1} + nbytes_{k-1}),
 *                   T = align256(off_last + nbytes_last).  Stream byte
 *                   off_k + j is byte j of tensor k; every other byte of
 *                   [0, T) is 0x00.
 *   Buckets       : bucket_bytes = B, a positive multiple of 256.  Bucket j is
 *                   stream bytes [j*B, min((j+1)*B, T)); n_buckets =
 *                   ceil(T / B).  Tensors may straddle buckets.  The packed
 *                   buffer is the contiguous stream, bucket j at byte j*B.
 *   Checksum      : for a bucket of L bytes, n = ceil(L / 8) little-endian
 *                   uint64 words w_i (missing bytes read as zero);
 *                   C = sum_{i=0}^{n-1} w_i * (2*i + 1)  mod 2^64.
 *                   i restarts at 0 in every bucket.
 *   Shard         : a plane is an ordered list of tensors with one common
 *                   elem_size e, viewed as one flat array of N elements
 *                   (concatenated WITHOUT padding).  The shard of data-parallel
 *                   rank r of D is elements [floor(r*N/D), floor((r+1)*N/D)),
 *                   written contiguously.  The products are formed in 128 bits.
 *
 * Conventions
 *   - Every pointer whose name starts with d_ is a DEVICE pointer; tm_desc.ptr
 *     is a device pointer; everything else is a HOST pointer.
 *   - The caller owns all device memory (tensors, packed buffer, checksum
 *     array, workspace) and the stream.  The library allocates no device
 *     memory.  A tm_plan owns host memory only, plus the contents it wrote
 *     into the workspace handed to tm_plan_upload.  The library keeps 8 MiB
 *     of pinned host memory per GPU for uploading small work lists.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default
 *     stream).  All device work is enqueued on it and the call returns without
 *     waiting; the caller synchronises.  The device of the stream/pointers must
 *     be the current device.
 *   - Every argument is validated on the host before anything is launched.
 *     Functions return TM_OK (0) or a negative tm_status.  On an argument error
 *     nothing has been enqueued.  A TM_ERR_CUDA return means a runtime call failed
 *     part-way: no kernel of the call has been launched, but a clearing memset or
 *     a work-list upload may already sit in the stream.  There is no CPU fallback:
 *     without a usable CUDA device the operations return TM_ERR_CUDA.
 *   - Calls are thread-safe with respect to one another, but one plan object must
 *     not be used by two threads at the same time.  tm_shard_extract_static has a
 *     rule of its own (see there).
 *   - An address named d_... only has to be readable / writable by the GPU: the
 *     packed buffer (and, for that matter, the tensors) may live in mapped pinned
 *     host memory, in which case the kernels move the bytes over PCIe themselves
 *     (the "remote CPU memory checkpoint" tier of §7).  Checksum arrays and
 *     workspaces should stay in device memory (the kernels update them with atomics).
 *   - Tensor addresses need only 2-byte alignment.  To serve such tensors at
 *     full speed the kernels read whole 16-byte-aligned lines: a line that
 *     holds at least one byte of a tensor may be read in full (it lies in the
 *     same memory page as that byte), but bytes outside the tensor are never
 *     used and never written.
 */
#ifndef TM_STATE_H
#define TM_STATE_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum tm_status {
  TM_OK           =  0,
  TM_ERR_ARG      = -1,  /* NULL pointer, zero count/size, odd nbytes, nbytes % elem_size != 0 */
  TM_ERR_ALIGN    = -2,  /* odd tensor address, bucket_bytes % 256 != 0, packed buffer not 256-byte aligned */
  TM_ERR_CAPACITY = -3,  /* output, input or workspace buffer smaller than required; work list too long to build; out of host memory */
  TM_ERR_OVERLAP  = -4,  /* a tensor overlaps the packed/output buffer, or two unpack targets overlap */
  TM_ERR_RANK     = -5,  /* D == 0 or r >= D */
  TM_ERR_DTYPE    = -6,  /* elem_size not in {2,4,8}, or mixed elem_size inside one shard plane */
  TM_ERR_CUDA     = -7,  /* a CUDA runtime call failed (tm_last_cuda_error() gives its code) */
  TM_ERR_TIMEOUT  = -8,  /* a bounded device-side wait expired (reported by tm_plan_status / tm_workspace_status) */
  TM_ERR_STATE    = -9,  /* the plan has no uploaded work list (tm_plan_upload / bind not called) */
  TM_ERR_VERIFY   = -10, /* a transfer still had buckets with a checksum mismatch after the last round */
  TM_ERR_TRANSPORT = -11 /* a transport or hook callback of a transfer returned non-zero */
} tm_status;

/* One tensor of a role's training state. */
typedef struct tm_desc {
  void*    ptr;        /* device address, >= 2-byte aligned; source for pack and shard, destination for unpack */
  uint64_t nbytes;     /* numel * elem_size; > 0 */
  uint32_t elem_size;  /* 2 (bf16), 4 (fp32) or 8 (int64) */
  uint32_t plane;      /* caller's label: 0 bf16 param, 1 fp32 master, 2 Adam m, 3 Adam v, 4 other; not interpreted */
} tm_desc;

typedef struct tm_plan tm_plan;  /* opaque */

/* ---- tuning ------------------------------------------------------------------------------- */

/* Process-wide tuning values.  A plan keeps the values in force when it was created; launches read
 * the rest from the plan.  The defaults are what every published number was measured with. */
typedef struct tm_options {
  uint64_t chunk_bytes;        /* largest piece of a pack / unpack plan; multiple of 256, 4 KiB .. 1 GiB; default 256 KiB */
  uint64_t shard_chunk_bytes;  /* largest piece of a shard list (a shard is a fraction of a role); default 64 KiB */
  uint64_t small_bytes;        /* pieces below this share a work item, one warp per piece; default 8 KiB */
  uint64_t group_bytes;        /* byte budget of a shared item; default 64 KiB */
  uint64_t cksum_tile_bytes;   /* tile of the stand-alone checksum kernel; multiple of 256; default 256 KiB */
  uint64_t wait_limit_ns;      /* bound of every device-side wait of the ring kernels; 1 .. 5e9; default 2e9.  Below 1024 (the timer's resolution) a wait that is not satisfied at once gives up at once: a diagnostic setting that makes launches end with TM_ERR_TIMEOUT and incomplete output */
  uint32_t group_max;          /* piece budget of a shared item; 1 .. 1024; default 64 */
  uint32_t ring_ctas_per_sm;   /* persistent blocks per SM of the ring kernels (96 KiB of shared memory each, 192 KiB in pack and unpack, where a second block does not fit); 1 .. 2; default 1 */
  uint32_t ctas_per_sm;        /* persistent blocks per SM of the checksum kernel; 1 .. 8; default 4 */
  uint32_t reserved;           /* must be 0 */
} tm_options;

/* Reads the values in force. */
int tm_options_get(tm_options* out);
/* Replaces them (TM_ERR_ARG / TM_ERR_ALIGN if a value is out of range); NULL restores the defaults.
 * Existing plans keep what they were built with. */
int tm_options_set(const tm_options* in);

/* ---- plan: layout of a role's tensors in the packed stream ------------------------------- */

/* Computes the packed-stream layout (off_k, T, buckets; definitions above) for `n_desc`
 * descriptors and cuts it into the device work list.  Host only: no CUDA call is made.
 * `descs` is copied; it may be freed after the call.  *out receives a plan to be released with
 * tm_plan_destroy.  Errors: TM_ERR_ARG (NULL, n_desc == 0, nbytes == 0, nbytes % elem_size != 0,
 * bucket_bytes == 0 or > 2^35, nbytes > 2^46, n_desc > 2^24, T > 2^56), TM_ERR_DTYPE, TM_ERR_ALIGN
 * (odd ptr, bucket_bytes % 256 != 0), TM_ERR_CAPACITY (out of host memory, or a work list of more than
 * 2^24 pieces — 4 TiB of stream at the default piece size, far less with tiny buckets; such a role is
 * planned in ranges).  The same piece limit applies to a bound shard plan and to all waves of a
 * transfer endpoint together. */
int tm_plan_create(const tm_desc* descs, uint64_t n_desc, uint64_t bucket_bytes, tm_plan** out);

/* Plan for a run of whole buckets of the same stream — the unit in which a role travels through a
 * bounded staging ring instead of a full second copy (§8.5 "Zero Memory Overhead Workflow": the
 * channel is a recycled buffer, not a role-sized allocation).  The layout is computed for the
 * complete descriptor list exactly as by tm_plan_create; the plan then covers stream bytes
 * [first_bucket * B, min((first_bucket + n_buckets) * B, T)) only.  For such a plan the packed
 * buffer passed to tm_state_pack / tm_state_unpack(_verify) / tm_state_pack_emit is a staging slot
 * that holds just this range (its byte 0 is stream byte first_bucket * B; capacity >= the range's
 * length, reported as total_bytes by tm_plan_query), and the checksum array has one entry per
 * bucket of the range.  Buckets are independent units (each checksum restarts its word index), so the
 * slots of consecutive ranges concatenate to the complete stream and their checksum arrays to the
 * complete list.  Tensors outside the range are never touched (their ptr must still be non-NULL and
 * even); a tensor that straddles a range boundary is split there.  first_bucket + n_buckets may
 * exceed the bucket count (the range is clipped); first_bucket >= the bucket count is TM_ERR_ARG. */
int tm_plan_create_range(const tm_desc* descs, uint64_t n_desc, uint64_t bucket_bytes, uint64_t first_bucket,
                         uint64_t n_buckets, tm_plan** out);

/* Any of the three outputs may be NULL.  total_bytes = T, n_buckets = ceil(T/B),
 * workspace_bytes = size the caller must provide to tm_plan_upload. */
int tm_plan_query(const tm_plan* plan, uint64_t* total_bytes, uint64_t* n_buckets,
                  uint64_t* workspace_bytes);

/* Where the plan sits in the complete stream (all outputs may be NULL): its first bucket, the stream
 * offset of its first byte, and T and the bucket count of the complete stream.  For a plan made by
 * tm_plan_create: 0, 0, and the same values as tm_plan_query. */
int tm_plan_range(const tm_plan* plan, uint64_t* first_bucket, uint64_t* stream_begin, uint64_t* whole_bytes,
                  uint64_t* whole_buckets);

/* Writes off_k (offset in the complete stream) for every descriptor into host array `offsets`
 * (n_desc entries). */
int tm_plan_offsets(const tm_plan* plan, uint64_t* offsets);

/* Copies the work list into caller-owned device memory `d_workspace` (256-byte aligned, at
 * least workspace_bytes from tm_plan_query) on `stream`.  The workspace must stay untouched
 * while the plan is in use.  Calling it again re-targets the plan to another workspace. */
int tm_plan_upload(tm_plan* plan, void* d_workspace, uint64_t workspace_bytes, void* stream);

/* Synchronises `stream`, then reads the plan's device status word: *device_status = TM_OK, or
 * TM_ERR_TIMEOUT if any kernel launched with this plan gave up a bounded wait (its output is
 * then incomplete).  Returns TM_ERR_CUDA if the synchronisation itself failed. */
int tm_plan_status(const tm_plan* plan, void* stream, int* device_status);

void tm_plan_destroy(tm_plan* plan);

/* ---- the four operations ------------------------------------------------------------------- */

/* Pack (leaver side of "State Synchronization", §7; bucket staging per §8.5).
 * Gathers every tensor of the plan into d_buckets[0, T) following the packed-stream definition,
 * writes all padding bytes as zero, and — in the same pass over the data — accumulates the
 * checksum of each bucket.  d_buckets: device, 256-byte aligned, `capacity` >= T bytes, must not
 * overlap any tensor.  d_checksums: device array of n_buckets uint64 (8-byte aligned) that
 * receives the checksums, or NULL to skip them.  Enqueues on `stream`. */
int tm_state_pack(const tm_plan* plan, void* d_buckets, uint64_t capacity,
                  uint64_t* d_checksums, void* stream);

/* Unpack (joiner side: the received state overwrites the sandbox-warmed state, §7 and §4.2).
 * Copies nbytes_k bytes from d_buckets + off_k into tensor k for every k; padding is ignored.
 * `nbytes` = valid bytes at d_buckets, must be >= T.  d_buckets 256-byte aligned.  The tensors
 * must not overlap the packed buffer or one another. */
int tm_state_unpack(const tm_plan* plan, const void* d_buckets, uint64_t nbytes, void* stream);

/* Unpack and verify in one pass (joiner side: checking the received buckets and overwriting the
 * sandbox-warmed state are both part of "State Synchronization", §7; the paper has no integrity check,
 * the checksum is this library's).  Does what tm_state_unpack does and, while the buckets stream
 * through, accumulates the checksum of every bucket exactly as tm_checksum(d_buckets, T, B) defines it
 * — over the bytes as received, padding included — into d_checksums (n_buckets uint64, 8-byte
 * aligned, required).  The caller compares them with the sender's after synchronising; the tensors
 * have been written by then, so a mismatch means the unpacked state must be discarded. */
int tm_state_unpack_verify(const tm_plan* plan, const void* d_buckets, uint64_t nbytes,
                           uint64_t* d_checksums, void* stream);

/* Pack that also emits shards (the leaver, or a stayer holding a replica, hands a joiner both the
 * packed role and the slice of the optimizer state its data-parallel rank owns — §7 "State
 * Synchronization" — and reads every tensor from memory once for both).
 *
 * tm_plan_attach_shards prepares it: planes are runs of the plan's own descriptors — plane p is
 * descriptors [plane_first_desc[p], + plane_n_desc[p]), runs ascending and disjoint, one elem_size
 * per plane — and each is sliced with the same r and D exactly as by tm_shard_extract, into
 * d_outs[p] (capacity out_capacities[p]; the buffer receives the complete shard, element lo first).
 * Every pack piece that holds shard elements gets a second destination for that sub-range; the
 * kernel writes it from the same staged copy of the piece that feeds the stream and the checksum.
 * (Pieces under 8 KiB are not staged; their few bytes are re-read through the caches.)  With a
 * range plan only the part of each shard that lies in the plan's buckets is written, at its place in
 * d_outs[p]; the plans of all ranges together fill the shard.  The list (pieces, items and emit
 * records) is uploaded once to d_workspace on `stream`.  With d_workspace == NULL nothing is uploaded:
 * *workspace_needed (may be NULL otherwise) and out_elems (n_planes entries, may be NULL) are filled,
 * and if d_outs is given the emit records are computed for inspection (tm_plan_emits) while
 * tm_state_pack_emit keeps returning TM_ERR_STATE.  The outputs must not overlap the tensors, one
 * another, or the packed buffer used later.
 *
 * tm_state_pack_emit then does what tm_state_pack does (same arguments, same results) and fills the
 * attached shard outputs in the same launch. */
int tm_plan_attach_shards(tm_plan* plan, const uint64_t* plane_first_desc, const uint64_t* plane_n_desc,
                          uint32_t n_planes, uint32_t r, uint32_t D, void* const* d_outs,
                          const uint64_t* out_capacities, uint64_t* out_elems, void* d_workspace,
                          uint64_t workspace_bytes, uint64_t* workspace_needed, void* stream);
int tm_state_pack_emit(const tm_plan* plan, void* d_buckets, uint64_t capacity, uint64_t* d_checksums,
                       void* stream);

/* The receiving side's counterpart (a joiner that is sent a whole role and keeps, under the distributed
 * optimizer, its own slice of the optimizer state as flat buffers — §7 "State Synchronization"): does
 * what tm_state_unpack_verify does (same arguments, same results, d_checksums required) and, from the
 * same staged copy of every piece, also fills the shard outputs attached with tm_plan_attach_shards —
 * one read of the received buckets gives the tensors, the checksums and the shards. */
int tm_state_unpack_emit(const tm_plan* plan, const void* d_buckets, uint64_t nbytes, uint64_t* d_checksums,
                         void* stream);

/* Host helper: floor shard bounds lo = floor(r*N/D), hi = floor((r+1)*N/D) in 128-bit arithmetic. */
int tm_shard_bounds(uint64_t n_elems, uint32_t r, uint32_t D, uint64_t* lo, uint64_t* hi);

/* Workspace size tm_shard_extract needs for a plane of n_desc tensors and the given bounds.
 * Returns the size in *workspace_bytes. */
int tm_shard_workspace(const tm_desc* plane_descs, uint64_t n_desc, uint32_t r, uint32_t D,
                       uint64_t* workspace_bytes);

/* Shard extract (state for a joiner under the distributed optimizer, §7 "State
 * Synchronization": no replica holds the shard, so it is cut out of the flat plane).
 * plane_descs: host array of n_desc tensors with one common elem_size (TM_ERR_DTYPE otherwise),
 * viewed as one flat array without padding.  Copies elements [lo, hi) (definition above) to
 * d_out (device, >= 2-byte aligned, out_capacity bytes >= (hi-lo)*elem_size, no overlap with the
 * tensors).  *out_elems (host, may be NULL) receives hi - lo, which may be 0 (nothing is then
 * launched).  d_workspace: caller-owned device scratch, 256-byte aligned, at least
 * tm_shard_workspace() bytes; it must stay untouched until the enqueued work has finished.
 * Errors: TM_ERR_RANK for D == 0 or r >= D. */
int tm_shard_extract(const tm_desc* plane_descs, uint64_t n_desc, uint32_t r, uint32_t D,
                     void* d_out, uint64_t out_capacity, uint64_t* out_elems,
                     void* d_workspace, uint64_t workspace_bytes, void* stream);

/* Shard extract of several planes in one launch (a joiner needs the same [lo, hi) of the fp32
 * master weights, Adam m and Adam v — §7 "State Synchronization").  `descs` is the concatenation of
 * the planes' descriptor lists, plane p having plane_n_desc[p] entries; each plane is validated and
 * sliced exactly as by tm_shard_extract with the same r and D (its own elem_size and element count),
 * and written contiguously to d_outs[p] (capacity out_capacities[p] bytes).  out_elems (host array of
 * n_planes entries, may be NULL) receives each plane's hi - lo.  Outputs must not overlap any tensor
 * or one another.  Workspace: the sum of tm_shard_workspace() over the planes is enough. */
int tm_shard_extract_planes(const tm_desc* descs, const uint64_t* plane_n_desc, uint32_t n_planes,
                            uint32_t r, uint32_t D, void* const* d_outs, const uint64_t* out_capacities,
                            uint64_t* out_elems, void* d_workspace, uint64_t workspace_bytes, void* stream);

/* Shard insert: the inverse of tm_shard_extract (a joiner that fetched its slice of the optimizer
 * state from a peer or from storage — §7 "State Synchronization", the no-redundancy case — puts it
 * into its own flat plane).  Elements [lo, hi) of the plane (same definition and bounds as
 * tm_shard_extract) are overwritten with the (hi - lo) elements at d_in (device, >= 2-byte aligned,
 * `in_bytes` >= (hi-lo)*elem_size, no overlap with the tensors); all other elements stay as they
 * are.  *in_elems (host, may be NULL) receives hi - lo.  Workspace: as for tm_shard_extract
 * (tm_shard_workspace gives the size).  The tensors of the plane must not overlap one another. */
int tm_shard_insert(const tm_desc* plane_descs, uint64_t n_desc, uint32_t r, uint32_t D,
                    const void* d_in, uint64_t in_bytes, uint64_t* in_elems,
                    void* d_workspace, uint64_t workspace_bytes, void* stream);

/* Reusable shard plan.  The one-shot calls above validate, build the work list on the host and
 * upload it on every call; a plan does that once, after which extract and insert are single kernel
 * launches with no host work (the joiner slices the same [lo, hi) out of master, m and v every time
 * it is assigned a rank — §7 "State Synchronization").
 *
 * tm_shard_plan_create: `descs` is the concatenation of the planes' descriptor lists (plane p has
 * plane_n_desc[p] entries, one elem_size per plane); validation and bounds as tm_shard_extract_planes.
 * Host only.  tm_shard_plan_query: out_elems (n_planes entries, may be NULL) = hi - lo per plane;
 * workspace_bytes (may be NULL) = device scratch tm_shard_plan_bind needs.
 * tm_shard_plan_bind: fixes the flat buffers (d_flats[p], >= 2-byte aligned, capacities[p] >= the
 * shard's bytes, no overlap with the tensors or one another; entries of empty shards are ignored),
 * builds the list and uploads it to d_workspace (256-byte aligned) on `stream`.  May be called again
 * to bind other buffers.  With d_workspace == NULL the list is only built (tm_shard_plan_pieces shows
 * it) and extract / insert return TM_ERR_STATE.  tm_shard_plan_extract copies elements [lo, hi) of every plane to its flat
 * buffer; tm_shard_plan_insert writes the flat buffers into elements [lo, hi) of the planes (the
 * tensors of a plane must then not overlap one another: TM_ERR_OVERLAP).  Both are one launch, or none
 * when every shard is empty. */
typedef struct tm_shard_plan tm_shard_plan;
int tm_shard_plan_create(const tm_desc* descs, const uint64_t* plane_n_desc, uint32_t n_planes, uint32_t r,
                         uint32_t D, tm_shard_plan** out);
int tm_shard_plan_query(const tm_shard_plan* sp, uint64_t* out_elems, uint64_t* workspace_bytes);
int tm_shard_plan_bind(tm_shard_plan* sp, void* const* d_flats, const uint64_t* capacities, void* d_workspace,
                       uint64_t workspace_bytes, void* stream);
int tm_shard_plan_extract(const tm_shard_plan* sp, void* stream);
int tm_shard_plan_insert(const tm_shard_plan* sp, void* stream);
/* Status word of the plan's workspace (same meaning as tm_plan_status). */
int tm_shard_plan_status(const tm_shard_plan* sp, void* stream, int* device_status);
void tm_shard_plan_destroy(tm_shard_plan* sp);

/* Size of the library-resident scratch array used by tm_shard_extract_static. */
#define TM_STATIC_SCRATCH_BYTES (1u << 20)

/* Shard extract without caller scratch.  (The paper has no counterpart: this entry point exists
 * for the library's users, not for the method.)  It is for callers that are handed tensors but
 * cannot allocate on the device: a recovery hook running while the framework's allocator owns the
 * whole GPU, code that must avoid cudaMalloc because it synchronises the device and can fail when
 * memory is full, or a plugin with no allocator.  Same arguments, checks, results and errors as
 * tm_shard_extract, minus the workspace: the work list goes into a fixed array of
 * TM_STATIC_SCRATCH_BYTES (1 MiB) of device global memory that is part of the library image; every
 * GPU that loads the library holds that array until the process exits.  A shard whose list does
 * not fit (with the default 64 KiB pieces: more than about 1.8 GiB of output, or more than about
 * 29 000 tensor pieces) is refused with TM_ERR_CAPACITY and nothing is launched.  The call makes no
 * device allocation and frees none.  The first call on each GPU resolves the array's device address
 * once, with that GPU current; make that call before starting any stream capture.  All calls on a
 * GPU share the array, which keeps the previous call's contents: the part that must start from zero
 * (the status block) is cleared on every call.  The host side of a call (clear, two list copies,
 * launch) runs under a lock, so calls from several threads on ONE stream are safe; calls whose
 * device work can overlap in time (different streams) race on the list — issue them on one stream.
 * The list is copied from ordinary host memory, so the call returns only after the stream has taken
 * the copies (it may wait for earlier work in that stream). */
int tm_shard_extract_static(const tm_desc* plane_descs, uint64_t n_desc, uint32_t r, uint32_t D,
                            void* d_out, uint64_t out_capacity, uint64_t* out_elems, void* stream);

/* Status word of a raw workspace used by tm_shard_extract (same meaning as tm_plan_status). */
int tm_workspace_status(const void* d_workspace, void* stream, int* device_status);

/* Checksum (integrity check of received buckets; the paper has no integrity check, the formula
 * is this library's, see "Checksum" above).  Treats d_bytes[0, nbytes) as ceil(nbytes /
 * bucket_bytes) buckets and writes one uint64 per bucket to d_checksums.  d_bytes must be
 * 16-byte aligned; nbytes may be any value (the last word is zero-extended); nbytes == 0 writes
 * nothing.  bucket_bytes: positive multiple of 256, <= 2^35. */
int tm_checksum(const void* d_bytes, uint64_t nbytes, uint64_t bucket_bytes,
                uint64_t* d_checksums, void* stream);

/* Self-test of the device-side failure reporting.  The kernels' only waits (mbarrier waits of the
 * bulk-copy ring) are bounded in time; a wait that expires makes the kernel record TM_ERR_TIMEOUT in
 * the status word of its workspace and return, leaving the context usable.  This call launches one
 * thread that waits, for at most limit_ns (1 .. 5e9), on a barrier that nothing will ever complete,
 * so that the reporting path can be checked without a fault or a hang: afterwards
 * tm_workspace_status(d_workspace) yields TM_ERR_TIMEOUT.  d_workspace: >= 256 bytes, 256-byte aligned. */
int tm_selftest_bounded_wait(void* d_workspace, uint64_t limit_ns, void* stream);

/* ---- leaver -> joiner transfer through a bounded ring of staging slots ------------------------- */

/* §7 "State Synchronization" delivers a role's state one-to-one from a leaver to its joiner, and
 * §8.5 "Zero Memory Overhead Workflow" sends it through a per-pair channel that is created for the
 * transfer and recycled, not through a second role-sized buffer.  Here the role is cut into waves of
 * `buckets_per_wave` whole buckets (range plans); wave j of a round travels in slot j mod n_slots of a
 * ring on each side.  Sender: pack wave -> slot (with the checksums of its buckets), hand slot and
 * checksums to the transport, reuse the slot once the transport has read it.  Receiver: take a wave
 * into a free slot, unpack + verify it (tm_state_unpack_verify), reuse the slot.  At the end of a
 * round the receiver compares the checksums it recomputed with the sender's, bucket by bucket, and
 * reports the waves that hold a mismatch; the sender packs and sends those again (the leaver's
 * tensors are still there), up to max_rounds rounds in all.  Packing, sending, receiving and
 * unpacking of different waves overlap: each side runs on two streams and only the slot hand-overs
 * are ordered (events).  The integrity check and the re-request are this library's; the paper has
 * none. */

/* How bytes and control messages travel between the two sides.  All functions return 0 on success;
 * anything else ends the transfer with that value if it is a negative tm_status, else with
 * TM_ERR_TRANSPORT.  send / recv enqueue on `stream` (they may block the host until the peer has posted
 * the matching call, as a rendezvous transport does) and move `nbytes` bytes of a slot plus
 * `n_checksums` uint64 values; the data must land in the receiver's own memory.  Reports are small
 * host-side messages: the list of waves to send again (n == 0: the round was clean). */
typedef struct tm_transport {
  void* ctx;
  int (*send)(void* ctx, uint32_t wave, const void* d_slot, uint64_t nbytes, const uint64_t* d_checksums,
              uint64_t n_checksums, void* stream);
  int (*recv)(void* ctx, uint32_t wave, void* d_slot, uint64_t nbytes, uint64_t* d_checksums, uint64_t n_checksums,
              void* stream);
  int (*send_report)(void* ctx, const uint32_t* waves, uint32_t n);
  int (*recv_report)(void* ctx, uint32_t* waves, uint32_t capacity, uint32_t* n);
} tm_transport;

typedef struct tm_xfer_stats {
  uint32_t rounds;        /* rounds run (1 = nothing had to be sent again) */
  uint32_t waves;         /* waves packed and sent / received and unpacked, all rounds */
  uint32_t waves_again;   /* of those, in rounds after the first */
  uint32_t bad_buckets;   /* receiver: buckets whose checksums differed, all rounds */
  uint64_t first_bad_bucket;  /* receiver: the first of them (bucket index in the complete stream); ~0 if none */
  uint64_t bytes;         /* slot bytes moved, all rounds */
} tm_xfer_stats;

/* The protocol itself, free of CUDA: the order of steps, the slot assignment (wave j of a round uses
 * slot j mod n_slots), the rounds and the re-request.  tm_xfer_send / tm_xfer_receive run it with
 * the library's kernels and a tm_transport; a harness can run the same loops over any other
 * implementation of the steps (the CPU tests drive two processes over a host transport this way).
 * Every hook returns 0 on success.  Sender hooks: pack, send, recv_report.  Receiver hooks: recv,
 * unpack_verify, bad_waves (waits for the round's work, then lists which of `waves` arrived damaged),
 * send_report.  Unused hooks may be NULL. */
typedef struct tm_xfer_hooks {
  void* ctx;
  int (*pack)(void* ctx, uint32_t wave, uint32_t slot);
  int (*send)(void* ctx, uint32_t wave, uint32_t slot);
  int (*recv_report)(void* ctx, uint32_t* waves, uint32_t capacity, uint32_t* n);
  int (*recv)(void* ctx, uint32_t wave, uint32_t slot);
  int (*unpack_verify)(void* ctx, uint32_t wave, uint32_t slot);
  int (*bad_waves)(void* ctx, const uint32_t* waves, uint32_t n_waves, uint32_t* bad, uint32_t* n_bad);
  int (*send_report)(void* ctx, const uint32_t* waves, uint32_t n);
} tm_xfer_hooks;

/* Return TM_OK when a round ended clean, TM_ERR_VERIFY when waves were still damaged after
 * max_rounds rounds, TM_ERR_TRANSPORT (or the hook's own negative status) when a hook failed or a
 * report named a wave that was not sent in that round.  `stats` may be NULL. */
int tm_xfer_run_sender(uint32_t n_waves, uint32_t n_slots, uint32_t max_rounds, const tm_xfer_hooks* hooks,
                       tm_xfer_stats* stats);
int tm_xfer_run_receiver(uint32_t n_waves, uint32_t n_slots, uint32_t max_rounds, const tm_xfer_hooks* hooks,
                         tm_xfer_stats* stats);

/* One side of a transfer: the role's tensors (sources on the sender, destinations on the receiver),
 * cut into waves.  Host only; `descs` is copied. */
typedef struct tm_xfer tm_xfer;
int tm_xfer_create(const tm_desc* descs, uint64_t n_desc, uint64_t bucket_bytes, uint64_t buckets_per_wave,
                   uint32_t n_slots, tm_xfer** out);
/* All outputs may be NULL: number of waves, bytes of one slot (buckets_per_wave * bucket_bytes), bytes
 * of the ring (n_slots slots — the whole staging footprint of this side), device scratch for the
 * waves' work lists, bucket count of the complete stream. */
int tm_xfer_query(const tm_xfer* x, uint32_t* n_waves, uint64_t* slot_bytes, uint64_t* ring_bytes,
                  uint64_t* workspace_bytes, uint64_t* n_buckets);
/* Gives the side its memory (caller-owned, 256-byte aligned): the ring, the scratch (work lists are
 * uploaded on `stream`), d_checksums (n_buckets uint64: filled by packing on the sender, recomputed
 * from what arrived on the receiver) and, on the receiver, d_peer_checksums (n_buckets uint64: the
 * sender's values as received; NULL on the sender).  Creates the events that order slot hand-overs. */
int tm_xfer_bind(tm_xfer* x, void* d_ring, uint64_t ring_bytes, void* d_workspace, uint64_t workspace_bytes,
                 uint64_t* d_checksums, uint64_t* d_peer_checksums, void* stream);
/* Optional: shards filled during the transfer.  Planes, r, D, outputs and the size query (d_workspace
 * == NULL) as for tm_plan_attach_shards, applied to every wave; afterwards the sender packs with
 * tm_state_pack_emit and the receiver unpacks with tm_state_unpack_emit, so that a joiner under the
 * distributed optimizer has its flat slices of master weights, m and v when the last wave has been
 * verified (§7 "State Synchronization"), from the same read that scatters the tensors.  A wave that is
 * sent again rewrites its part of the shards.  Call after tm_xfer_bind; d_workspace is further
 * caller-owned scratch (256-byte aligned) that must stay untouched while the endpoint is in use. */
int tm_xfer_attach_shards(tm_xfer* x, const uint64_t* plane_first_desc, const uint64_t* plane_n_desc, uint32_t n_planes,
                          uint32_t r, uint32_t D, void* const* d_outs, const uint64_t* out_capacities,
                          uint64_t* out_elems, void* d_workspace, uint64_t workspace_bytes,
                          uint64_t* workspace_needed, void* stream);

/* Run one side to the end.  Packing (unpacking) is enqueued on the first stream, the transport's
 * send (recv) on the second; the two must differ for the steps to overlap.  The calls block the host
 * until the last round's report has been exchanged; the receiver's tensors are complete when
 * tm_xfer_receive returns TM_OK. */
int tm_xfer_send(tm_xfer* x, const tm_transport* transport, void* pack_stream, void* send_stream,
                 uint32_t max_rounds, tm_xfer_stats* stats);
int tm_xfer_receive(tm_xfer* x, const tm_transport* transport, void* unpack_stream, void* recv_stream,
                    uint32_t max_rounds, tm_xfer_stats* stats);
void tm_xfer_destroy(tm_xfer* x);

/* Transport between two sides that live in one process on one GPU (two host threads): send waits for
 * the matching recv to be posted, then copies slot and checksums device-to-device on its stream into
 * the receiver's slot; reports go through a mailbox.  It stands in for a link between two GPUs, whose
 * transport (for example NCCL send / recv of whole slots) implements the same four functions.  A
 * posted call that finds no partner within 60 s fails with TM_ERR_TRANSPORT.  *transport is filled
 * with functions and a context that stay valid until tm_loopback_destroy. */
typedef struct tm_loopback tm_loopback;
int tm_loopback_create(tm_loopback** out, tm_transport* transport);
void tm_loopback_destroy(tm_loopback* lb);

/* One piece of a plan's work list, as the kernels see it (for inspection and host-side checks). */
typedef struct tm_piece {
  uint64_t tensor;   /* device address of the piece's first tensor byte */
  uint64_t off;      /* offset of the piece in the packed stream */
  uint32_t nbytes;   /* tensor bytes in the piece */
  uint32_t pad;      /* zero bytes that follow it in the stream */
  uint32_t bucket;   /* bucket the piece lies in */
  uint32_t word0;    /* index of its first 8-byte word inside that bucket */
} tm_piece;

/* Copies the plan's work list to host arrays: up to `capacity` pieces into `pieces` and, for every
 * item, the index of its first piece into `item_first` (n_items + 1 entries, the last one = number
 * of pieces; `item_capacity` entries available).  Either array may be NULL.  *n_pieces / *n_items
 * (may be NULL) receive the full counts.  Host only. */
int tm_plan_pieces(const tm_plan* plan, tm_piece* pieces, uint64_t capacity, uint64_t* n_pieces,
                   uint32_t* item_first, uint64_t item_capacity, uint64_t* n_items);

/* Emit record of a piece after tm_plan_attach_shards: bytes [begin, begin + len) of the piece also go
 * to device address `out`; len == 0 for pieces that hold no shard element. */
typedef struct tm_emit {
  uint64_t out;
  uint32_t begin;
  uint32_t len;
} tm_emit;

/* Copies the emit records (one per piece, in piece order) to `emits` (up to `capacity`); *n (may be
 * NULL) receives the count — 0 before tm_plan_attach_shards.  Host only. */
int tm_plan_emits(const tm_plan* plan, tm_emit* emits, uint64_t capacity, uint64_t* n);

/* Work list of a bound shard plan, as tm_plan_pieces gives it for a plan; a piece's `off` is relative
 * to *base (the lowest bound flat address; may be NULL), pad / bucket / word0 are 0.  Host only. */
int tm_shard_plan_pieces(const tm_shard_plan* sp, tm_piece* pieces, uint64_t capacity, uint64_t* n_pieces,
                         uint32_t* item_first, uint64_t item_capacity, uint64_t* n_items, uint64_t* base);

/* ---- diagnostics ----------------------------------------------------------------------------- */

const char* tm_strerror(int status);

/* cudaError_t value of the most recent failed CUDA runtime call made by this library (0 if none). */
int tm_last_cuda_error(void);

/* Number of kernels this library has launched since it was loaded (all streams, all threads). */
uint64_t tm_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* TM_STATE_H */
