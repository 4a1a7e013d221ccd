// tm_oracle.cpp — TEST INFRASTRUCTURE ONLY.
//
// Plain, single-threaded, deliberately slow CPU statement of what the role-state mover
// computes: the packed stream, its buckets and checksums, the reverse unpack, and the
// distributed-optimizer shard.  It exists so that tests can compare the CUDA library against
// it; it shares no code, header, table or helper with that library and must never be called
// from the product path.  Only tests, the smoke check and the CPU-baseline legs of the benchmark
// may load it.
//
// What it follows.  The paper (§7 "Implementation", paragraph "State Synchronization") only says
// WHAT is moved — the leaver's model parameters and optimizer states go to the joiner, and with
// the distributed optimizer a joiner needs its own slice of the optimizer state — and §8.5
// "Zero Memory Overhead Workflow" says the state travels through a staging buffer.  The paper
// gives no format; the definitions below are the format of this project, written out literally:
//
//   align256(x) = smallest multiple of 256 that is >= x
//   off_0 = 0 ; off_k = align256(off_{k-1} + nbytes_{k-1}) ; T = align256(off_last + nbytes_last)
//   stream[off_k + j] = tensor_k[j] ; every other byte of [0,T) is 0
//   bucket j = stream[j*B, min((j+1)*B, T)) ; n_buckets = ceil(T/B) ; B % 256 == 0
//   checksum of L bytes: n = ceil(L/8), w_i = sum_b byte[8i+b] << (8b) (missing bytes 0),
//                        C = sum_i w_i * (2i+1) mod 2^64, i from 0 in every bucket
//   shard r of D of a plane with N elements: elements [floor(r*N/D), floor((r+1)*N/D))
//
// Every loop below is per byte or per element, in the order of the definition.  Nothing is
// blocked, vectorised or parallelised by hand.  All functions take HOST pointers.
//
// Pins: every function here is pinned by tests/test_oracle_pins.py (closed forms, hand-computed
// golden values, round trip, exact shard tiling, Python big-integer brute force).  Nothing is
// "parity unpinned".

#include <cstdint>
#include <cstddef>

namespace {

const int ORC_OK = 0;
const int ORC_ERR_ARG = -1;
const int ORC_ERR_ALIGN = -2;
const int ORC_ERR_CAPACITY = -3;
const int ORC_ERR_RANK = -5;
const int ORC_ERR_DTYPE = -6;

uint64_t round_up_256(uint64_t x) {
  uint64_t rem = x % 256;
  if (rem == 0) return x;
  return x + (256 - rem);
}

// Offsets of the packed stream.  off may be NULL.
int layout(const uint64_t* nbytes, uint64_t n, uint64_t B, uint64_t* off, uint64_t* total,
           uint64_t* n_buckets) {
  if (nbytes == NULL || n == 0) return ORC_ERR_ARG;
  if (B == 0) return ORC_ERR_ARG;
  if (B % 256 != 0) return ORC_ERR_ALIGN;
  uint64_t pos = 0;
  for (uint64_t k = 0; k < n; ++k) {
    if (nbytes[k] == 0 || nbytes[k] % 2 != 0) return ORC_ERR_ARG;
    pos = round_up_256(pos);
    if (off != NULL) off[k] = pos;
    pos += nbytes[k];
  }
  uint64_t T = round_up_256(pos);
  if (total != NULL) *total = T;
  if (n_buckets != NULL) *n_buckets = (T + B - 1) / B;
  return ORC_OK;
}

// Checksum of one bucket of L bytes, by the definition.
uint64_t checksum_one(const uint8_t* bytes, uint64_t L) {
  uint64_t n = (L + 7) / 8;
  uint64_t C = 0;
  for (uint64_t i = 0; i < n; ++i) {
    uint64_t w = 0;
    for (uint64_t b = 0; b < 8; ++b) {
      uint64_t idx = 8 * i + b;
      uint64_t byte = (idx < L) ? (uint64_t)bytes[idx] : 0;
      w |= byte << (8 * b);
    }
    C += w * (2 * i + 1);  // uint64 arithmetic wraps mod 2^64
  }
  return C;
}

}  // namespace

extern "C" {

int oracle_layout(const uint64_t* nbytes, uint64_t n, uint64_t bucket_bytes, uint64_t* off,
                  uint64_t* total, uint64_t* n_buckets) {
  return layout(nbytes, n, bucket_bytes, off, total, n_buckets);
}

// One checksum per bucket of `bucket_bytes` over bytes[0, nbytes).
int oracle_checksum(const uint8_t* bytes, uint64_t nbytes, uint64_t bucket_bytes, uint64_t* out) {
  if (bucket_bytes == 0) return ORC_ERR_ARG;
  if (bucket_bytes % 256 != 0) return ORC_ERR_ALIGN;
  if (nbytes == 0) return ORC_OK;
  if (bytes == NULL || out == NULL) return ORC_ERR_ARG;
  uint64_t nb = (nbytes + bucket_bytes - 1) / bucket_bytes;
  for (uint64_t j = 0; j < nb; ++j) {
    uint64_t begin = j * bucket_bytes;
    uint64_t end = begin + bucket_bytes;
    if (end > nbytes) end = nbytes;
    out[j] = checksum_one(bytes + begin, end - begin);
  }
  return ORC_OK;
}

// Whole packed stream into out[0, T), then the per-bucket checksums (checksums may be NULL).
int oracle_pack(const uint8_t* const* ptrs, const uint64_t* nbytes, uint64_t n,
                uint64_t bucket_bytes, uint8_t* out, uint64_t capacity, uint64_t* checksums) {
  uint64_t T = 0, nb = 0;
  int rc = layout(nbytes, n, bucket_bytes, NULL, &T, &nb);
  if (rc != ORC_OK) return rc;
  if (ptrs == NULL || out == NULL) return ORC_ERR_ARG;
  if (capacity < T) return ORC_ERR_CAPACITY;
  for (uint64_t i = 0; i < T; ++i) out[i] = 0;
  uint64_t pos = 0;
  for (uint64_t k = 0; k < n; ++k) {
    pos = round_up_256(pos);
    const uint8_t* src = ptrs[k];
    if (src == NULL) return ORC_ERR_ARG;
    for (uint64_t j = 0; j < nbytes[k]; ++j) out[pos + j] = src[j];
    pos += nbytes[k];
  }
  if (checksums != NULL) return oracle_checksum(out, T, bucket_bytes, checksums);
  return ORC_OK;
}

// Stream bytes [lo, hi) only (for sampling one bucket of a layout too large to pack whole).
// ptrs[k] may be NULL for a tensor that does not intersect [lo, hi).
int oracle_pack_range(const uint8_t* const* ptrs, const uint64_t* nbytes, uint64_t n,
                      uint64_t lo, uint64_t hi, uint8_t* out) {
  uint64_t T = 0;
  int rc = layout(nbytes, n, 256, NULL, &T, NULL);
  if (rc != ORC_OK) return rc;
  if (ptrs == NULL || lo > hi || hi > T) return ORC_ERR_ARG;
  if (lo == hi) return ORC_OK;
  if (out == NULL) return ORC_ERR_ARG;
  for (uint64_t i = 0; i < hi - lo; ++i) out[i] = 0;
  uint64_t pos = 0;
  for (uint64_t k = 0; k < n; ++k) {
    pos = round_up_256(pos);
    bool intersects = (pos < hi) && (pos + nbytes[k] > lo);  // tensors wholly outside are skipped
    if (intersects) {
      if (ptrs[k] == NULL) return ORC_ERR_ARG;
      for (uint64_t j = 0; j < nbytes[k]; ++j) {
        uint64_t s = pos + j;
        if (s >= lo && s < hi) out[s - lo] = ptrs[k][j];
      }
    }
    pos += nbytes[k];
  }
  return ORC_OK;
}

// Inverse of oracle_pack: tensor_k[j] = stream[off_k + j].
int oracle_unpack(uint8_t* const* ptrs, const uint64_t* nbytes, uint64_t n,
                  const uint8_t* stream, uint64_t stream_bytes) {
  uint64_t T = 0;
  int rc = layout(nbytes, n, 256, NULL, &T, NULL);
  if (rc != ORC_OK) return rc;
  if (ptrs == NULL || stream == NULL) return ORC_ERR_ARG;
  if (stream_bytes < T) return ORC_ERR_CAPACITY;
  uint64_t pos = 0;
  for (uint64_t k = 0; k < n; ++k) {
    pos = round_up_256(pos);
    uint8_t* dst = ptrs[k];
    if (dst == NULL) return ORC_ERR_ARG;
    for (uint64_t j = 0; j < nbytes[k]; ++j) dst[j] = stream[pos + j];
    pos += nbytes[k];
  }
  return ORC_OK;
}

// lo = floor(r*N/D), hi = floor((r+1)*N/D); products in 128 bits.
int oracle_shard_bounds(uint64_t N, uint32_t r, uint32_t D, uint64_t* lo, uint64_t* hi) {
  if (D == 0 || r >= D) return ORC_ERR_RANK;
  if (lo == NULL || hi == NULL) return ORC_ERR_ARG;
  unsigned __int128 a = (unsigned __int128)r * (unsigned __int128)N;
  unsigned __int128 b = ((unsigned __int128)r + 1) * (unsigned __int128)N;
  *lo = (uint64_t)(a / D);
  *hi = (uint64_t)(b / D);
  return ORC_OK;
}

// Shard r of D of the plane (ptrs, nbytes) with common element size e: walk every element of
// the flat array in order and keep those whose global index is in [lo, hi).
int oracle_shard(const uint8_t* const* ptrs, const uint64_t* nbytes, uint64_t n, uint32_t e,
                 uint32_t r, uint32_t D, uint8_t* out, uint64_t capacity, uint64_t* out_elems) {
  if (ptrs == NULL || nbytes == NULL || n == 0) return ORC_ERR_ARG;
  if (e != 2 && e != 4 && e != 8) return ORC_ERR_DTYPE;
  uint64_t N = 0;
  for (uint64_t k = 0; k < n; ++k) {
    if (nbytes[k] == 0 || nbytes[k] % e != 0) return ORC_ERR_ARG;
    N += nbytes[k] / e;
  }
  uint64_t lo = 0, hi = 0;
  int rc = oracle_shard_bounds(N, r, D, &lo, &hi);
  if (rc != ORC_OK) return rc;
  if (out_elems != NULL) *out_elems = hi - lo;
  if (hi == lo) return ORC_OK;
  if (out == NULL) return ORC_ERR_ARG;
  if (capacity < (hi - lo) * e) return ORC_ERR_CAPACITY;
  uint64_t g = 0;  // global element index of the flat array
  for (uint64_t k = 0; k < n; ++k) {
    uint64_t count = nbytes[k] / e;
    for (uint64_t idx = 0; idx < count; ++idx, ++g) {
      if (g >= lo && g < hi) {
        if (ptrs[k] == NULL) return ORC_ERR_ARG;
        for (uint32_t b = 0; b < e; ++b) out[(g - lo) * e + b] = ptrs[k][idx * e + b];
      }
    }
  }
  return ORC_OK;
}

// Inverse of oracle_shard: element g of the flat plane, for g in [lo, hi), is overwritten with
// element g - lo of `in`; every other element of every tensor is left as it is.
int oracle_shard_insert(uint8_t* const* ptrs, const uint64_t* nbytes, uint64_t n, uint32_t e,
                        uint32_t r, uint32_t D, const uint8_t* in, uint64_t in_bytes,
                        uint64_t* in_elems) {
  if (ptrs == NULL || nbytes == NULL || n == 0) return ORC_ERR_ARG;
  if (e != 2 && e != 4 && e != 8) return ORC_ERR_DTYPE;
  uint64_t N = 0;
  for (uint64_t k = 0; k < n; ++k) {
    if (nbytes[k] == 0 || nbytes[k] % e != 0) return ORC_ERR_ARG;
    N += nbytes[k] / e;
  }
  uint64_t lo = 0, hi = 0;
  int rc = oracle_shard_bounds(N, r, D, &lo, &hi);
  if (rc != ORC_OK) return rc;
  if (in_elems != NULL) *in_elems = hi - lo;
  if (hi == lo) return ORC_OK;
  if (in == NULL) return ORC_ERR_ARG;
  if (in_bytes < (hi - lo) * e) return ORC_ERR_CAPACITY;
  uint64_t g = 0;
  for (uint64_t k = 0; k < n; ++k) {
    uint64_t count = nbytes[k] / e;
    for (uint64_t idx = 0; idx < count; ++idx, ++g) {
      if (g >= lo && g < hi) {
        if (ptrs[k] == NULL) return ORC_ERR_ARG;
        for (uint32_t b = 0; b < e; ++b) ptrs[k][idx * e + b] = in[(g - lo) * e + b];
      }
    }
  }
  return ORC_OK;
}

}  // extern "C"
