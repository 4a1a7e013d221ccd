// Bulk-copy ("TMA") ring kernels for sm_100a: the same pack / copy work as kernels.cu, but large
// pieces travel global -> shared memory with cp.async.bulk issued by one producer thread into a
// ring of stages guarded by mbarriers.  When source and destination are both 16-byte aligned the
// stage goes straight back out, shared memory -> global, with a bulk store issued by one store
// thread, and the eight consumer warps only read the stage to accumulate the checksum.  When the
// source sits at a 2-byte-granular address the consumers re-align the stage in registers.  In pack
// and unpack they write the aligned vectors into a second ring of "out" stages in shared memory and
// the store thread sends those out with bulk stores as well (bulk stores keep DRAM busier than
// 16-byte stores from registers: +1.5 % on a role whose tensors are all misaligned).  The plain
// gather into a flat buffer (shard extract: short launches, where the extra hand-over costs more
// than it gains) stores the re-aligned vectors from registers.  The producer runs ahead across
// piece and item boundaries, so the loads of the next pieces are in flight while the current one is
// consumed.
//
// Misaligned sources cost no extra global traffic here: the producer fetches the aligned superset
// of the source span (one extra 16-byte vector per stage) and the consumers shift in registers.
// The superset stays inside 16-byte lines that hold at least one byte of the tensor.
//
// Every wait is bounded in time.  If one expires the waiter records TM_ERR_TIMEOUT in the status
// word, raises a block-wide abort flag that all roles poll, and the producer waits (bounded) for its
// own copies in flight before the block exits; the context stays usable.
//
// Small pieces (items that group several pieces, or single pieces below kBulkMinVectors) are
// copied by the consumer warps with the register routines of device_util.cuh.
//
// Pack-and-emit: a pack piece may carry a second destination for a sub-range of its bytes (the part
// of the tensor that falls into a distributed-optimizer shard).  The consumer warps write that
// sub-range to the shard output from the same shared-memory stage that feeds the stream and the
// checksum, so the tensor is read from HBM once for all three results.
#include <cuda_runtime.h>

#include <cstdint>

#include "device_util.cuh"
#include "tm_internal.h"

namespace tms {

constexpr int kRingStages = 3;
constexpr uint32_t kStageBytes = 32 * 1024;
constexpr uint32_t kStageVectors = kStageBytes / 16;
constexpr uint32_t kStageStride = kStageBytes + 128;   // room for the one extra vector of a shifted source
#ifndef TM_OUT_STAGES
#define TM_OUT_STAGES 3
#endif
constexpr int kOutStages = TM_OUT_STAGES;              // re-aligned stages waiting for their bulk store
#ifndef TM_CONS_WARPS
#define TM_CONS_WARPS 8
#endif
constexpr int kConsWarps = TM_CONS_WARPS;
constexpr int kConsThreads = kConsWarps * 32;
constexpr int kRingThreads = kConsThreads + 64;     // + one producer warp + one store warp
constexpr uint32_t kBulkMinVectors = 128;           // pieces below 2 KiB are not worth a stage
constexpr unsigned long long kDrainLimitNs = 2000000000ull;   // bound of the producer's final wait for its own loads

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint64_t* b, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(b)), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* b, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(b)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* b) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(b)) : "memory");
}
__device__ __forceinline__ bool mbar_try(uint64_t* b, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n.reg .pred p;\nmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\nselp.u32 %0, 1, 0, p;\n}"
      : "=r"(ok)
      : "r"(smem_u32(b)), "r"(parity)
      : "memory");
  return ok != 0;
}
__device__ __forceinline__ unsigned long long global_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
// Non-blocking probe of a barrier phase.
__device__ __forceinline__ bool mbar_test(uint64_t* b, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n.reg .pred p;\nmbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\nselp.u32 %0, 1, 0, p;\n}"
      : "=r"(ok)
      : "r"(smem_u32(b)), "r"(parity)
      : "memory");
  return ok != 0;
}
constexpr unsigned long long kTimerResolutionNs = 1024;   // limits below this cannot be measured with %globaltimer
// Waits for the phase with the given parity; gives up after limit_ns or when the block aborts.  A
// limit below the timer's resolution means "do not wait at all": the wait fails unless the phase has
// already completed (used to drive the give-up paths of the kernels on purpose).
__device__ __forceinline__ bool mbar_wait(uint64_t* b, uint32_t parity, volatile int* abort_flag,
                                          unsigned long long limit_ns) {
  if (mbar_test(b, parity)) return true;
  if (limit_ns < kTimerResolutionNs) return false;
  if (mbar_try(b, parity)) return true;
  const unsigned long long t0 = global_ns();
  for (;;) {
#pragma unroll 1
    for (int i = 0; i < 64; ++i)
      if (mbar_try(b, parity)) return true;
    if (*abort_flag != 0) return false;
    if (global_ns() - t0 > limit_ns) return false;
  }
}
// 1-D bulk copy global -> this block's own shared memory (single destination block), completion on an mbarrier.
__device__ __forceinline__ void bulk_g2s(void* smem, const void* g, uint32_t bytes, uint64_t* bar) {
  asm volatile("cp.async.bulk.shared::cta.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                   smem_u32(smem)),
               "l"(g), "r"(bytes), "r"(smem_u32(bar))
               : "memory");
}
// Bulk store this block's shared memory -> global, tracked by the issuing thread's bulk groups.
__device__ __forceinline__ void bulk_s2g(void* g, const void* smem, uint32_t bytes) {
  asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(g), "r"(smem_u32(smem)),
               "r"(bytes)
               : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
// Waits until all but the newest N bulk stores of this thread have finished READING shared memory.
template <int N>
__device__ __forceinline__ void bulk_wait_read() {
  asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory");
}
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }

// How one piece is cut into ring stages.  Destination vectors are 16-byte aligned; `head` bytes
// before the first aligned destination vector and `rem` bytes after the last full one are copied
// directly.  Stage t carries destination vectors [t*V, t*V + cnt) and is loaded from the aligned
// source address sa + 16*t*V, (cnt + extra) vectors long, extra = 1 when the source is shifted.
struct BulkPlan {
  const uint8_t* src;   // after the head
  uint8_t* dst;         // after the head, 16-byte aligned
  const uint8_t* sa;    // src rounded down to 16 bytes
  uint32_t a;           // src - sa, even, 0..14
  uint32_t head, nfull, rem, V, ntiles;
  bool straight;        // source and destination both aligned: stages are stored back by bulk stores
};

template <bool TO_TENSORS>
__device__ __forceinline__ bool plan_bulk(const Seg& s, uint8_t* flat, BulkPlan& p) {
  uint8_t* tensor = reinterpret_cast<uint8_t*>(s.tensor);
  uint8_t* f = flat + s.off;
  const uint8_t* src = TO_TENSORS ? f : tensor;
  uint8_t* dst = TO_TENSORS ? tensor : f;
  uint32_t n = s.nbytes;
  uint32_t head = (uint32_t)((0 - (uintptr_t)dst) & 15);
  if (head > n) head = n;
  p.head = head;
  p.src = src + head;
  p.dst = dst + head;
  n -= head;
  p.nfull = n >> 4;
  p.rem = n & 15;
  p.a = (uint32_t)((uintptr_t)p.src & 15);
  p.sa = p.src - p.a;
  p.V = kStageVectors;
  p.ntiles = (p.nfull + p.V - 1) / p.V;
  p.straight = (p.a == 0);   // the destination is aligned by construction (head bytes are cut off)
  return p.nfull >= kBulkMinVectors;
}

struct RingShared {
  uint64_t full[kRingStages];
  uint64_t empty[kRingStages];
  uint64_t out_full[kOutStages];    // the consumer warps have written a re-aligned stage
  uint64_t out_empty[kOutStages];   // its bulk store has finished reading it
  int abort_flag;
};

// Makes this thread's ordinary shared-memory writes visible to the bulk-copy engine.
__device__ __forceinline__ void fence_smem_for_bulk() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

__device__ __forceinline__ void raise_timeout(int* status, RingShared* sh) {
  if (status != nullptr) atomicExch(status, (int)TM_ERR_TIMEOUT);
  atomicExch(&sh->abort_flag, 1);
}

// Adds a per-thread value, summed over the warp by shuffles, to *target: one atomic per warp.  The
// consumer warps do not meet at a block barrier for this, so a bucket change never stalls the ring;
// integer addition mod 2^64 commutes, so the result does not depend on the order of the atomics.
__device__ __forceinline__ void consumer_flush(u64 value, u64* target) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) value += __shfl_xor_sync(0xffffffffu, value, o);
  if ((threadIdx.x & 31) == 0 && value != 0) atomicAdd(target, value);
}

// Copies n bytes (even) from shared memory `s` to global memory `d`, both at any even alignment, with
// threads c, c + C, ...: 2-byte copies up to the first 16-byte boundary of the destination, aligned
// 16-byte stores re-aligned from two aligned shared-memory vectors, 2-byte copies for the tail.
// Reads at most one aligned 16-byte vector past the last source byte (inside the stage's slack).
__device__ __forceinline__ void smem_to_global(uint8_t* d, const uint8_t* s, uint32_t n, uint32_t c, uint32_t C) {
  uint32_t head = (uint32_t)((0 - (uintptr_t)d) & 15);
  if (head > n) head = n;
  if (2 * c < head) st2(d + 2 * c, (uint32_t)(*reinterpret_cast<const uint16_t*>(s + 2 * c)));
  d += head;
  s += head;
  n -= head;
  const uint32_t nfull = n >> 4, rem = n & 15;
  const uint32_t a = smem_u32(s) & 15;
  const uint4* sa = reinterpret_cast<const uint4*>(s - a);
  if (a == 0) {
    for (uint32_t v = c; v < nfull; v += C) st16(d + (size_t)v * 16u, sa[v]);
  } else {
    const uint32_t ws = a >> 2, bs = (a & 3) * 8;
    for (uint32_t v = c; v < nfull; v += C) st16(d + (size_t)v * 16u, shift_pair(sa[v], sa[v + 1], ws, bs));
  }
  const size_t tl = (size_t)nfull * 16u;
  const uint32_t gt = C - 1 - c;
  if (2 * gt < rem) st2(d + tl + 2 * gt, (uint32_t)(*reinterpret_cast<const uint16_t*>(s + tl + 2 * gt)));
}

// Emits the part of piece bytes [lo, hi) (hi - lo <= 16) that lies inside the emit span, straight
// from the tensor: the few bytes of a bulk piece that do not travel through the ring.
__device__ __forceinline__ void emit_direct(const Emit& em, const uint8_t* piece_src, uint32_t lo, uint32_t hi,
                                            uint32_t c) {
  const uint32_t b = lo > em.begin ? lo : em.begin;
  const uint32_t e = hi < em.begin + em.len ? hi : em.begin + em.len;
  if (b + 2 * c < e) st2(reinterpret_cast<uint8_t*>(em.out) + (b - em.begin) + 2 * c, ld2(piece_src + b + 2 * c));
}

// PACK: tensors -> stream with padding and checksums.  Otherwise a plain copy of pieces, direction
// given by TO_TENSORS (PACK implies TO_TENSORS == false).  VERIFY (with TO_TENSORS): the unpack also
// accumulates the per-bucket checksums of the stream it reads — data and padding bytes as they
// arrived — so that a receiver checks and scatters in one pass over the buckets.
// EMIT (with PACK, or with TO_TENSORS + VERIFY): emits[i] gives piece i an optional second destination
// for a sub-range of its bytes; the consumers write it from the stage in shared memory (bulk pieces)
// or re-read the few KiB of a small piece they have just copied (served by L1 / L2).
template <bool PACK, bool TO_TENSORS, bool VERIFY, bool EMIT>
__global__ void __launch_bounds__(kRingThreads, 1)
ring_kernel(const Seg* __restrict__ segs, const uint32_t* __restrict__ item_first, uint32_t n_items,
            uint8_t* __restrict__ flat, u64* __restrict__ checksums, int* __restrict__ status,
            const Emit* __restrict__ emits, unsigned long long wait_limit_ns) {
  extern __shared__ __align__(128) uint8_t ring[];
  __shared__ RingShared sh;
  const uint32_t warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    for (int s = 0; s < kRingStages; ++s) {
      mbar_init(&sh.full[s], 1);
      mbar_init(&sh.empty[s], kConsWarps + 1);   // consumer warps + the store thread
    }
    for (int s = 0; s < kOutStages; ++s) {
      mbar_init(&sh.out_full[s], kConsWarps);
      mbar_init(&sh.out_empty[s], 1);
    }
    sh.abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  volatile int* abort_flag = &sh.abort_flag;
  // re-aligned stages leave through the out ring (bulk stores) in pack and unpack, from registers otherwise
  constexpr bool RESTAGE = PACK || TO_TENSORS;
  uint8_t* const out_ring = ring + (size_t)kRingStages * kStageStride;

  if (warp == kConsWarps) {
    // ---------------- producer: one thread issues every bulk load of this block, in item order
    if (lane != 0) return;
    uint32_t stage = 0, phase = 0, issued = 0;
    bool ok = true;
    for (uint32_t item = blockIdx.x; ok && item < n_items; item += gridDim.x) {
      const uint32_t first = item_first[item];
      if (item_first[item + 1] - first != 1) continue;
      const Seg s = segs[first];
      BulkPlan p;
      if (!plan_bulk<TO_TENSORS>(s, flat, p)) continue;
      const uint32_t extra = p.a != 0 ? 1u : 0u;
      for (uint32_t t = 0; t < p.ntiles; ++t) {
        if (!mbar_wait(&sh.empty[stage], phase ^ 1u, abort_flag, wait_limit_ns)) {
          raise_timeout(status, &sh);
          ok = false;
          break;
        }
        uint32_t cnt = p.nfull - t * p.V;
        if (cnt > p.V) cnt = p.V;
        const uint32_t bytes = (cnt + extra) * 16u;
        mbar_expect_tx(&sh.full[stage], bytes);
        bulk_g2s(ring + (size_t)stage * kStageStride, p.sa + (size_t)t * p.V * 16u, bytes, &sh.full[stage]);
        ++issued;
        if (++stage == kRingStages) { stage = 0; phase ^= 1u; }
      }
    }
    // Leave no copy in flight, whatever the other roles do: the newest load of every stage must have
    // landed before this thread — and with it possibly the block — exits.  try_wait only observes the
    // phase, so the consumers' own waits on the same barriers are not disturbed.  The bound here is a
    // constant of its own; a shortened wait_limit_ns does not shorten it.
    {
      uint32_t n = issued < (uint32_t)kRingStages ? issued : (uint32_t)kRingStages;
      uint32_t st = stage, ph = phase;
      for (uint32_t k = 0; k < n; ++k) {
        if (st == 0) { st = kRingStages; ph ^= 1u; }
        --st;
        if (mbar_try(&sh.full[st], ph)) continue;
        const unsigned long long t0 = global_ns();
        while (!mbar_try(&sh.full[st], ph) && global_ns() - t0 < kDrainLimitNs) {}
      }
    }
    return;
  }

  if (warp == kConsWarps + 1) {
    // ---------------- store thread: sends every stage back out with bulk stores, in item order —
    // straight from the load stage when source and destination are aligned alike, else from the out
    // stage the consumers have re-aligned it into
    if (lane != 0) return;
    uint32_t stage = 0, phase = 0, ostage = 0, ophase = 0;
    uint64_t* pending = nullptr;   // barrier to release once the newest bulk store has finished reading shared memory
    bool ok = true;
    for (uint32_t item = blockIdx.x; ok && item < n_items; item += gridDim.x) {
      const uint32_t first = item_first[item];
      if (item_first[item + 1] - first != 1) continue;
      const Seg s = segs[first];
      BulkPlan p;
      if (!plan_bulk<TO_TENSORS>(s, flat, p)) continue;
      for (uint32_t t = 0; t < p.ntiles; ++t) {
        if (!mbar_wait(&sh.full[stage], phase, abort_flag, wait_limit_ns)) {
          raise_timeout(status, &sh);
          ok = false;
          break;
        }
        uint32_t cnt = p.nfull - t * p.V;
        if (cnt > p.V) cnt = p.V;
        const uint8_t* from;
        uint64_t* release;
        if (p.straight) {
          from = ring + (size_t)stage * kStageStride;
          release = &sh.empty[stage];
        } else {
          mbar_arrive(&sh.empty[stage]);   // the consumers read this stage; the store thread does not
          if (!RESTAGE) {                  // ... and write its data themselves
            if (pending != nullptr) {
              bulk_wait_read<0>();
              mbar_arrive(pending);
              pending = nullptr;
            }
            if (++stage == kRingStages) { stage = 0; phase ^= 1u; }
            continue;
          }
          if (!mbar_wait(&sh.out_full[ostage], ophase, abort_flag, wait_limit_ns)) {
            raise_timeout(status, &sh);
            ok = false;
            break;
          }
          from = out_ring + (size_t)ostage * kStageBytes;
          release = &sh.out_empty[ostage];
          if (++ostage == kOutStages) { ostage = 0; ophase ^= 1u; }
        }
        bulk_s2g(p.dst + (size_t)t * p.V * 16u, from, cnt * 16u);
        bulk_commit();
        if (pending != nullptr) {
          bulk_wait_read<1>();
          mbar_arrive(pending);
        }
        pending = release;
        if (++stage == kRingStages) { stage = 0; phase ^= 1u; }
      }
    }
    bulk_wait_read<0>();
    if (pending != nullptr) mbar_arrive(pending);
    bulk_wait_all();
    return;
  }

  // ---------------- consumers
  const uint32_t c = threadIdx.x;   // 0 .. kConsThreads-1
  Cksum ck;
  u64 total = 0;
  uint32_t cur = 0xffffffffu;
  uint32_t stage = 0, phase = 0, ostage = 0, ophase = 0;
  bool ok = true;
  for (uint32_t item = blockIdx.x; item < n_items; item += gridDim.x) {
    const uint32_t first = item_first[item], last = item_first[item + 1];
    if (PACK || VERIFY) {
      const uint32_t bucket = segs[first].bucket;
      if (bucket != cur) {   // uniform over the consumers
        if (cur != 0xffffffffu && checksums != nullptr) consumer_flush(total, checksums + cur);
        total = 0;
        cur = bucket;
      }
    }
    const bool single = (last - first == 1);
    BulkPlan p;
    Seg s0;
    bool bulk = false;
    if (single) {
      s0 = segs[first];
      bulk = plan_bulk<TO_TENSORS>(s0, flat, p);
    }
    if (!bulk) {
      if (!ok) continue;
      const uint32_t g = single ? c : lane, G = single ? (uint32_t)kConsThreads : 32u;
      for (uint32_t i = first + (single ? 0u : warp); i < last; i += (single ? 1u : (uint32_t)kConsWarps)) {
        const Seg s = segs[i];
        if (PACK) {
          pack_piece(s, flat, g, G, ck);
          total += ck.finish(s.word0);
          if (EMIT) {
            const Emit em = emits[i];
            if (em.len != 0)
              copy_piece(reinterpret_cast<uint8_t*>(em.out), reinterpret_cast<const uint8_t*>(s.tensor) + em.begin,
                         em.len, g, G);
          }
        } else {
          uint8_t* t = reinterpret_cast<uint8_t*>(s.tensor);
          uint8_t* f = flat + s.off;
          copy_piece(TO_TENSORS ? t : f, TO_TENSORS ? f : t, s.nbytes, g, G);
          if (EMIT) {
            const Emit em = emits[i];
            if (em.len != 0)
              copy_piece(reinterpret_cast<uint8_t*>(em.out), (TO_TENSORS ? f : t) + em.begin, em.len, g, G);
          }
          if (VERIFY) {   // the piece's span of the stream, padding included, in aligned vectors
            const uint32_t nvec = (s.nbytes + s.pad) >> 4;
            for (uint32_t v = g; v < nvec; v += G) ck.add(ld16_cached(f + (size_t)v * 16u), v);
            total += ck.finish(s.word0);
          }
        }
      }
      continue;
    }
    // After a timeout the consumers only walk the rest of the item list, touching no memory.
    if (!ok) continue;
    // bulk piece: head bytes directly, full vectors through the ring, tail (and padding) directly
    if (2 * c < p.head) st2(p.dst - p.head + 2 * c, ld2(p.src - p.head + 2 * c));
    Emit em;
    em.out = 0; em.begin = 0; em.len = 0;
    if (EMIT) {
      em = emits[first];
      if (em.len != 0) {   // piece bytes outside the ring's share: before the first and after the last full vector
        const uint8_t* piece_src = p.src - p.head;
        if (p.head != 0) emit_direct(em, piece_src, 0, p.head, c);
        if (p.rem != 0) emit_direct(em, piece_src, p.head + p.nfull * 16u, s0.nbytes, c);
      }
    }
    const uint32_t ws = p.a >> 2, bs = (p.a & 3) * 8;
    for (uint32_t t = 0; t < p.ntiles; ++t) {
      // the vote keeps the warp together: either all of its lanes go on or none does
      if (!__all_sync(0xffffffffu, mbar_wait(&sh.full[stage], phase, abort_flag, wait_limit_ns))) {
        raise_timeout(status, &sh);
        ok = false;
        break;
      }
      uint32_t cnt = p.nfull - t * p.V;
      if (cnt > p.V) cnt = p.V;
      const uint8_t* stage_base = ring + (size_t)stage * kStageStride;
      const uint4* sp = reinterpret_cast<const uint4*>(stage_base);
      const uint32_t vbase = t * p.V;
      // VERIFY: the stream piece starts 256-byte aligned, so stage vector v is stream vector vbase + v
      if (p.straight) {
        if (PACK || VERIFY) {   // the store thread moves the data; only the checksum is left to do
#pragma unroll 4
          for (uint32_t v = c; v < cnt; v += kConsThreads) ck.add(sp[v], vbase + v);
        }
      } else if (!RESTAGE) {
        uint8_t* d = p.dst + (size_t)vbase * 16u;
#pragma unroll 2
        for (uint32_t v = c; v < cnt; v += kConsThreads) st16(d + (size_t)v * 16u, shift_pair(sp[v], sp[v + 1], ws, bs));
      } else {
        // re-align into an out stage whose previous bulk store has finished reading it
        if (!__all_sync(0xffffffffu, mbar_wait(&sh.out_empty[ostage], ophase ^ 1u, abort_flag, wait_limit_ns))) {
          raise_timeout(status, &sh);
          ok = false;
          break;
        }
        uint4* op = reinterpret_cast<uint4*>(out_ring + (size_t)ostage * kStageBytes);
#pragma unroll 2
        for (uint32_t v = c; v < cnt; v += kConsThreads) {
          const uint4 lo = sp[v];
          const uint4 x = shift_pair(lo, sp[v + 1], ws, bs);
          op[v] = x;
          if (PACK) ck.add(x, vbase + v);
          if (VERIFY) ck.add(lo, vbase + v);
        }
        fence_smem_for_bulk();
        __syncwarp();
        if (lane == 0) mbar_arrive(&sh.out_full[ostage]);
        if (++ostage == kOutStages) { ostage = 0; ophase ^= 1u; }
      }
      if (EMIT && em.len != 0) {
        // this stage holds piece bytes [s_lo, s_hi), byte b at stage_base + a + (b - s_lo)
        const uint32_t s_lo = p.head + vbase * 16u, s_hi = s_lo + cnt * 16u;
        const uint32_t b = s_lo > em.begin ? s_lo : em.begin;
        const uint32_t e = s_hi < em.begin + em.len ? s_hi : em.begin + em.len;
        if (b < e)
          smem_to_global(reinterpret_cast<uint8_t*>(em.out) + (b - em.begin), stage_base + p.a + (b - s_lo), e - b, c,
                         (uint32_t)kConsThreads);
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(&sh.empty[stage]);
      if (++stage == kRingStages) { stage = 0; phase ^= 1u; }
    }
    if (!ok) continue;
    if (PACK) {
      // the vector with the tensor's last (n mod 16) bytes, then whole vectors of zero padding
      const uint32_t nvec = (s0.nbytes + s0.pad) >> 4;
      for (uint32_t v = p.nfull + c; v < nvec; v += kConsThreads) {
        uint32_t w[4] = {0u, 0u, 0u, 0u};
        if (v == p.nfull && p.rem != 0) {
          const uint8_t* tl = p.src + (size_t)p.nfull * 16u;
#pragma unroll
          for (uint32_t h = 0; h < 7; ++h)
            if (2 * h < p.rem) w[h >> 1] |= ld2(tl + 2 * h) << ((h & 1) * 16);
        }
        const uint4 x = make_uint4(w[0], w[1], w[2], w[3]);
        st16(p.dst + (size_t)v * 16u, x);
        ck.add(x, v);
      }
      total += ck.finish(s0.word0);
    } else {
      const size_t tl = (size_t)p.nfull * 16u;
      const uint32_t gt = kConsThreads - 1 - c;
      if (2 * gt < p.rem) st2(p.dst + tl + 2 * gt, ld2(p.src + tl + 2 * gt));
      if (VERIFY) {   // stream vectors behind the ring's share: end of the data and the padding
        const uint8_t* f = flat + s0.off;
        const uint32_t nvec = (s0.nbytes + s0.pad) >> 4;
        for (uint32_t v = p.nfull + c; v < nvec; v += kConsThreads) ck.add(ld16_cached(f + (size_t)v * 16u), v);
        total += ck.finish(s0.word0);
      }
    }
  }
  if ((PACK || VERIFY) && cur != 0xffffffffu && checksums != nullptr) consumer_flush(total, checksums + cur);
}

// Exercises the bounded wait on purpose: one thread waits for a barrier phase that nobody will ever
// complete, gives up after limit_ns and reports TM_ERR_TIMEOUT through the status word, exactly as
// the ring kernels do.  The kernel returns normally; nothing is left in flight.
__global__ void wait_selftest_kernel(int* status, unsigned long long limit_ns) {
  __shared__ RingShared sh;
  if (threadIdx.x == 0) {
    mbar_init(&sh.full[0], 1);
    sh.abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    if (!mbar_wait(&sh.full[0], 0, &sh.abort_flag, limit_ns)) raise_timeout(status, &sh);
  }
}

// ---- host side ------------------------------------------------------------------------------------

int launch_wait_selftest(int* d_status, unsigned long long limit_ns, void* stream) {
  wait_selftest_kernel<<<1, 32, 0, (cudaStream_t)stream>>>(d_status, limit_ns);
  count_launch();
  return (int)cudaGetLastError();
}

constexpr int kMaxDevices = 64;

// The ring needs more dynamic shared memory than the default limit; the attribute is set once per
// kernel and device.
template <typename K>
static cudaError_t ensure_smem(K kernel, size_t smem, int dev, bool* done) {
  if (dev >= 0 && dev < kMaxDevices && done[dev]) return cudaSuccess;
  cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e == cudaSuccess && dev >= 0 && dev < kMaxDevices) done[dev] = true;
  return e;
}

template <bool PACK, bool TO_TENSORS, bool VERIFY, bool EMIT>
static int launch_ring_t(const RingLaunch& a, void* stream) {
  static bool attr_done[kMaxDevices] = {false};
  int sms = 0;
  int rc = device_sm_count(&sms);
  if (rc != 0) return rc;
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return (int)e;
  const size_t smem = (size_t)kRingStages * kStageStride + ((PACK || TO_TENSORS) ? (size_t)kOutStages * kStageBytes : 0);
  auto kernel = ring_kernel<PACK, TO_TENSORS, VERIFY, EMIT>;
  e = ensure_smem(kernel, smem, dev, attr_done);
  if (e != cudaSuccess) return (int)e;
  uint64_t grid = (uint64_t)sms * (a.ctas_per_sm == 0 ? 1u : a.ctas_per_sm);
  if (grid > a.n_items) grid = a.n_items;
  if (grid == 0) grid = 1;
  kernel<<<(uint32_t)grid, kRingThreads, smem, (cudaStream_t)stream>>>(a.d_segs, a.d_item_first, a.n_items, a.d_flat,
                                                                    a.d_checksums, a.d_status, a.d_emits,
                                                                    a.wait_limit_ns);
  count_launch();
  return (int)cudaGetLastError();
}

int launch_ring(RingMode mode, const RingLaunch& a, void* stream) {
  switch (mode) {
    case kRingPack: return launch_ring_t<true, false, false, false>(a, stream);
    case kRingPackEmit: return launch_ring_t<true, false, false, true>(a, stream);
    case kRingToFlat: return launch_ring_t<false, false, false, false>(a, stream);
    case kRingToTensors: return launch_ring_t<false, true, false, false>(a, stream);
    case kRingToTensorsVerify: return launch_ring_t<false, true, true, false>(a, stream);
    case kRingToTensorsVerifyEmit: return launch_ring_t<false, true, true, true>(a, stream);
  }
  return (int)cudaErrorInvalidValue;
}

}  // namespace tms
