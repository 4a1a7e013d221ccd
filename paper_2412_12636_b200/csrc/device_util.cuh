// Device helpers shared by the kernels: streaming 16-byte accesses, re-alignment of 2-byte-granular
// sources, the running checksum, and the per-piece copy routines of the register path.
#ifndef TM_DEVICE_UTIL_CUH
#define TM_DEVICE_UTIL_CUH

#include <cuda_runtime.h>

#include <cstdint>

#include "tm_internal.h"

namespace tms {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;
constexpr int kUnroll = 4;         // independent 16-byte loads in flight per thread, aligned sources
constexpr int kUnrollShifted = 2;  // same for sources that need re-alignment (two loads per vector)
constexpr int kMinBlocks = 4;  // resident blocks per SM the register budget is held to

typedef unsigned long long u64;

// ---- streaming 16-byte accesses -----------------------------------------------------------------
// Data is touched once: loads bypass L1 allocation, stores are marked streaming.
__device__ __forceinline__ uint4 ld16(const uint8_t* p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
               : "l"(p));
  return v;
}
// Lines that neighbouring threads read twice (misaligned sources) may stay in L1.
__device__ __forceinline__ uint4 ld16_cached(const uint8_t* p) {
  uint4 v;
  asm volatile("ld.global.nc.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
               : "l"(p));
  return v;
}
__device__ __forceinline__ void st16(uint8_t* p, uint4 v) {
  asm volatile("st.global.cs.v4.u32 [%0], {%1,%2,%3,%4};" ::"l"(p), "r"(v.x), "r"(v.y), "r"(v.z),
               "r"(v.w)
               : "memory");
}
__device__ __forceinline__ uint32_t ld2(const uint8_t* p) {
  return (uint32_t)(*reinterpret_cast<const uint16_t*>(p));
}
__device__ __forceinline__ void st2(uint8_t* p, uint32_t v) {
  *reinterpret_cast<uint16_t*>(p) = (uint16_t)v;
}

// Bytes [a, a + 16) of the 32-byte pair lo|hi, a = 4*ws + bs/8 (even, 2..14): a barrel shifter,
// whole words by ws (two select stages), then bits by bs with funnel shifts.
__device__ __forceinline__ uint4 shift_pair(const uint4 lo, const uint4 hi, uint32_t ws, uint32_t bs) {
  uint32_t c0 = lo.x, c1 = lo.y, c2 = lo.z, c3 = lo.w, c4 = hi.x, c5 = hi.y, c6 = hi.z, c7 = hi.w;
  if (ws & 2) { c0 = c2; c1 = c3; c2 = c4; c3 = c5; c4 = c6; c5 = c7; }
  if (ws & 1) { c0 = c1; c1 = c2; c2 = c3; c3 = c4; c4 = c5; }
  uint4 r;
  r.x = __funnelshift_r(c0, c1, bs);
  r.y = __funnelshift_r(c1, c2, bs);
  r.z = __funnelshift_r(c2, c3, bs);
  r.w = __funnelshift_r(c3, c4, bs);
  return r;
}

// Vector v of a source that starts `a` bytes (even, 2..14) after the aligned address `sa`: bytes
// [16v + a, 16v + a + 16) of the aligned stream, taken from two aligned vectors.
__device__ __forceinline__ uint4 ld16_shifted(const uint8_t* sa, uint32_t v, uint32_t ws, uint32_t bs) {
  const uint4 lo = ld16_cached(sa + (size_t)v * 16);
  const uint4 hi = ld16_cached(sa + (size_t)v * 16 + 16);
  return shift_pair(lo, hi, ws, bs);
}

// Running checksum state of one thread.  Within a piece the weight of local word j is 2j+1
// (fits 32 bits: pieces are < 4 GiB); the piece's position in its bucket enters once at the end:
//   sum_j w_j * (2*(word0 + j) + 1) = sum_j w_j * (2j+1) + 2*word0 * sum_j w_j.
struct Cksum {
  u64 acc = 0;  // sum of w_j * (2j+1)
  u64 sw = 0;   // sum of w_j
  __device__ __forceinline__ void add(uint4 x, uint32_t v) {
    const u64 w0 = (u64)x.x | ((u64)x.y << 32);
    const u64 w1 = (u64)x.z | ((u64)x.w << 32);
    const uint32_t k = 4u * v + 1u;  // weight of local word 2v; word 2v+1 has k + 2
    acc += w0 * (u64)k + w1 * (u64)(k + 2u);
    sw += w0 + w1;
  }
  __device__ __forceinline__ u64 finish(uint32_t word0) {
    const u64 r = acc + 2ull * (u64)word0 * sw;
    acc = 0;
    sw = 0;
    return r;
  }
};

// Copies full vectors [0, nfull) from src (any even alignment) to dst (16-byte aligned) with
// threads g, g+G, ...; optionally accumulates the checksum of what is stored.
template <bool CKSUM, bool ALIGNED>
__device__ __forceinline__ void copy_vectors(uint8_t* dst, const uint8_t* src, uint32_t nfull, uint32_t g,
                                             uint32_t G, uint32_t ws, uint32_t bs, Cksum& ck) {
  constexpr int U = ALIGNED ? kUnroll : kUnrollShifted;
  const uint8_t* sa = src - (ALIGNED ? 0 : ((uintptr_t)src & 15));
  for (uint32_t v0 = g; v0 < nfull; v0 += G * U) {
    uint4 x[U];
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const uint32_t v = v0 + u * G;
      if (v < nfull) x[u] = ALIGNED ? ld16(sa + (size_t)v * 16) : ld16_shifted(sa, v, ws, bs);
    }
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const uint32_t v = v0 + u * G;
      if (v < nfull) {
        st16(dst + (size_t)v * 16, x[u]);
        if (CKSUM) ck.add(x[u], v);
      }
    }
  }
}

template <bool CKSUM>
__device__ __forceinline__ void copy_vectors_any(uint8_t* dst, const uint8_t* src, uint32_t nfull,
                                                 uint32_t g, uint32_t G, Cksum& ck) {
  const uint32_t a = (uint32_t)((uintptr_t)src & 15);   // uniform over the group
  if (a == 0) copy_vectors<CKSUM, true>(dst, src, nfull, g, G, 0, 0, ck);
  else copy_vectors<CKSUM, false>(dst, src, nfull, g, G, a >> 2, (a & 3) * 8, ck);
}

// Pack one piece: tensor -> stream, zero padding, checksum.  dst is 256-byte aligned.
__device__ __forceinline__ void pack_piece(const Seg& s, uint8_t* stream, uint32_t g, uint32_t G, Cksum& ck) {
  uint8_t* dst = stream + s.off;
  const uint8_t* src = reinterpret_cast<const uint8_t*>(s.tensor);
  const uint32_t n = s.nbytes;
  const uint32_t nfull = n >> 4;
  copy_vectors_any<true>(dst, src, nfull, g, G, ck);
  // the vector that holds the tensor's last (n mod 16) bytes, then whole vectors of padding
  const uint32_t nvec = (n + s.pad) >> 4;
  const uint32_t rem = n & 15;
  for (uint32_t v = nfull + g; v < nvec; v += G) {
    uint32_t w[4] = {0u, 0u, 0u, 0u};
    if (v == nfull && rem != 0) {
      const uint8_t* t = src + (size_t)nfull * 16;
#pragma unroll
      for (uint32_t h = 0; h < 7; ++h)
        if (2 * h < rem) w[h >> 1] |= ld2(t + 2 * h) << ((h & 1) * 16);
    }
    const uint4 x = make_uint4(w[0], w[1], w[2], w[3]);
    st16(dst + (size_t)v * 16, x);
    ck.add(x, v);
  }
}

// Copy one piece between a tensor and the flat buffer, both at any even alignment.
__device__ __forceinline__ void copy_piece(uint8_t* dst, const uint8_t* src, uint32_t n, uint32_t g, uint32_t G) {
  Cksum unused;
  uint32_t head = (uint32_t)((0 - (uintptr_t)dst) & 15);
  if (head > n) head = n;
  if (2 * g < head) st2(dst + 2 * g, ld2(src + 2 * g));
  dst += head;
  src += head;
  n -= head;
  const uint32_t nfull = n >> 4;
  copy_vectors_any<false>(dst, src, nfull, g, G, unused);
  const uint32_t rem = n & 15;
  const size_t t = (size_t)nfull * 16;
  // the last G/… threads are as good as any; use the group's tail so the head threads differ
  const uint32_t gt = G - 1 - g;
  if (2 * gt < rem) st2(dst + t + 2 * gt, ld2(src + t + 2 * gt));
}

}  // namespace tms

#endif  // TM_DEVICE_UTIL_CUH
