// Register-path kernels of the role-state mover for sm_100a: the stand-alone checksum
// (checksum_kernel, the one every tm_checksum call runs) and copy_to_flat_kernel, a load/store
// gather of pieces into a flat buffer that serves tm_shard_extract_static.  Pack, unpack and the
// other shard calls run on the bulk-copy ring in ring_kernels.cu.
// Everything here is HBM-bound byte movement with one 64-bit multiply-add per 8 bytes; there is no
// contraction, so no tensor cores.
//
// Work distribution: a persistent grid walks the item or tile list with a grid stride.  An item with
// one piece is copied by the whole block; an item with several small pieces gives one warp per
// piece.  All global accesses of the main loops are 16-byte vectors, consecutive lanes on
// consecutive vectors.  A piece whose tensor address is not 16-byte aligned is read as aligned
// vectors and re-aligned in registers (funnel shifts), so stores stay aligned to the flat buffer.
#include <cuda_runtime.h>

#include <atomic>
#include <cstdint>

#include "device_util.cuh"
#include "tm_internal.h"

namespace tms {

// Block-wide sum of a per-thread value, added to *target by one thread.
__device__ __forceinline__ void block_flush(u64 value, u64* target, u64* smem) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) value += __shfl_xor_sync(0xffffffffu, value, o);
  const int warp = threadIdx.x >> 5;
  if ((threadIdx.x & 31) == 0) smem[warp] = value;
  __syncthreads();
  if (threadIdx.x == 0) {
    u64 total = 0;
#pragma unroll
    for (int w = 0; w < kWarps; ++w) total += smem[w];
    if (total != 0) atomicAdd(target, total);
  }
  __syncthreads();
}

__global__ void __launch_bounds__(kThreads, kMinBlocks)
copy_to_flat_kernel(const Seg* __restrict__ segs, const uint32_t* __restrict__ item_first, uint32_t n_items,
                    uint8_t* __restrict__ flat) {
  const uint32_t warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  for (uint32_t item = blockIdx.x; item < n_items; item += gridDim.x) {
    const uint32_t first = item_first[item], last = item_first[item + 1];
    const bool single = (last - first == 1);
    const uint32_t g = single ? threadIdx.x : lane, G = single ? kThreads : 32u;
    for (uint32_t i = first + (single ? 0u : warp); i < last; i += (single ? 1u : (uint32_t)kWarps)) {
      const Seg s = segs[i];
      copy_piece(flat + s.off, reinterpret_cast<const uint8_t*>(s.tensor), s.nbytes, g, G);
    }
  }
}

// Stand-alone checksum.  Tile t covers bytes [tile_bytes * (t % tiles_per_bucket), +tile_bytes) of
// bucket t / tiles_per_bucket (tile_bytes: a multiple of 256, at most 1 GiB).  The input is 16-byte aligned; only the very last vector of the
// input can be partial.

__global__ void __launch_bounds__(kThreads, kMinBlocks)
checksum_kernel(const uint8_t* __restrict__ bytes, u64 nbytes, u64 bucket_bytes, uint32_t tiles_per_bucket,
                u64 n_tiles, uint32_t tile_bytes, u64* __restrict__ checksums) {
  __shared__ u64 red[kWarps];
  Cksum ck;
  u64 total = 0;
  u64 cur = ~0ull;
  for (u64 t = blockIdx.x; t < n_tiles; t += gridDim.x) {
    const u64 bucket = t / tiles_per_bucket;
    const u64 in_bucket = (t - bucket * tiles_per_bucket) * (u64)tile_bytes;
    const u64 begin = bucket * bucket_bytes + in_bucket;
    u64 end = begin + tile_bytes;
    const u64 bucket_end = (bucket + 1) * bucket_bytes;
    if (end > bucket_end) end = bucket_end;
    if (end > nbytes) end = nbytes;
    if (in_bucket >= bucket_bytes || begin >= end) continue;   // uniform over the block
    if (bucket != cur) {
      if (cur != ~0ull) block_flush(total, checksums + cur, red);
      total = 0;
      cur = bucket;
    }
    const uint8_t* p = bytes + begin;
    const uint32_t n = (uint32_t)(end - begin);
    const uint32_t nfull = n >> 4;
    for (uint32_t v0 = threadIdx.x; v0 < nfull; v0 += kThreads * kUnroll) {
      uint4 x[kUnroll];
#pragma unroll
      for (int u = 0; u < kUnroll; ++u) {
        const uint32_t v = v0 + u * kThreads;
        if (v < nfull) x[u] = ld16(p + (size_t)v * 16);
      }
#pragma unroll
      for (int u = 0; u < kUnroll; ++u) {
        const uint32_t v = v0 + u * kThreads;
        if (v < nfull) ck.add(x[u], v);
      }
    }
    const uint32_t rem = n & 15;
    if (rem != 0 && threadIdx.x == 0) {   // ragged end of the input: assemble the last bytes
      u64 w0 = 0, w1 = 0;
      const uint8_t* q = p + (size_t)nfull * 16;
      for (uint32_t b = 0; b < rem; ++b) {
        if (b < 8) w0 |= (u64)q[b] << (8 * b);
        else w1 |= (u64)q[b] << (8 * (b - 8));
      }
      ck.add(make_uint4((uint32_t)w0, (uint32_t)(w0 >> 32), (uint32_t)w1, (uint32_t)(w1 >> 32)), nfull);
    }
    total += ck.finish((uint32_t)(in_bucket / 8));
  }
  if (cur != ~0ull) block_flush(total, checksums + cur, red);
}

// ---- host side ------------------------------------------------------------------------------------

static std::atomic<uint64_t> g_launches{0};
void count_launch() { g_launches.fetch_add(1, std::memory_order_relaxed); }
uint64_t launches() { return g_launches.load(std::memory_order_relaxed); }

int device_sm_count(int* sms) {
  static int cached[64] = {0};
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return (int)e;
  if (dev >= 0 && dev < 64 && cached[dev] > 0) {
    *sms = cached[dev];
    return 0;
  }
  int n = 0;
  e = cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev);
  if (e != cudaSuccess) return (int)e;
  if (dev >= 0 && dev < 64) cached[dev] = n;
  *sms = n;
  return 0;
}

static int grid_for(uint64_t n_items, uint32_t ctas_per_sm, uint32_t* grid) {
  int sms = 0;
  int rc = device_sm_count(&sms);
  if (rc != 0) return rc;
  uint64_t g = (uint64_t)sms * (ctas_per_sm == 0 ? 1u : ctas_per_sm);
  if (g > n_items) g = n_items;
  if (g == 0) g = 1;
  *grid = (uint32_t)g;
  return 0;
}

int launch_copy_to_flat(const Seg* d_segs, const uint32_t* d_item_first, uint32_t n_items, uint8_t* d_flat,
                        uint32_t ctas_per_sm, void* stream) {
  uint32_t grid = 0;
  int rc = grid_for(n_items, ctas_per_sm, &grid);
  if (rc != 0) return rc;
  copy_to_flat_kernel<<<grid, kThreads, 0, (cudaStream_t)stream>>>(d_segs, d_item_first, n_items, d_flat);
  count_launch();
  return (int)cudaGetLastError();
}

int launch_checksum(const uint8_t* d_bytes, uint64_t nbytes, uint64_t bucket_bytes,
                    unsigned long long* d_checksums, const Tuning& t, void* stream) {
  const uint64_t n_buckets = (nbytes + bucket_bytes - 1) / bucket_bytes;
  const uint32_t tile = (uint32_t)t.cksum_tile_bytes;
  const uint64_t tpb = (bucket_bytes + tile - 1) / tile;
  const uint64_t n_tiles = n_buckets * tpb;
  uint32_t grid = 0;
  int rc = grid_for(n_tiles, t.ctas_per_sm, &grid);
  if (rc != 0) return rc;
  checksum_kernel<<<grid, kThreads, 0, (cudaStream_t)stream>>>(d_bytes, nbytes, bucket_bytes, (uint32_t)tpb,
                                                              n_tiles, tile, d_checksums);
  count_launch();
  return (int)cudaGetLastError();
}

}  // namespace tms

extern "C" uint64_t tm_launch_count(void) { return tms::launches(); }
