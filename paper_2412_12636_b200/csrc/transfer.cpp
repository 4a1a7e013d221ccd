// Leaver -> joiner transfer of a role through a bounded ring of staging slots (declared in
// include/tm_state.h): the protocol loops (no CUDA), the CUDA implementation of their steps on top of
// range plans, and a same-GPU loopback transport.
#include <cuda_runtime.h>

#include <algorithm>
#include <chrono>
#include <condition_variable>
#include <cstring>
#include <mutex>
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

// A hook's or transport's return value as a status of this library.
int hook_status(int rc) {
  if (rc == 0) return TM_OK;
  return (rc < 0 && rc >= TM_ERR_TRANSPORT) ? rc : TM_ERR_TRANSPORT;
}

#define TM_HOOK(call)                         \
  do {                                        \
    int rc__ = hook_status(call);             \
    if (rc__ != TM_OK) return rc__;           \
  } while (0)

#define TM_CUDA(call)                                        \
  do {                                                       \
    cudaError_t e__ = (call);                                \
    if (e__ != cudaSuccess) return tms::cuda_fail((int)e__); \
  } while (0)

void stats_init(tm_xfer_stats* s) {
  if (s == nullptr) return;
  std::memset(s, 0, sizeof(*s));
  s->first_bad_bucket = ~0ull;
}

// Every reported wave must have been part of the round it answers, and appear once.
bool report_is_valid(const std::vector<uint32_t>& pending, const uint32_t* bad, uint32_t n, uint32_t n_waves) {
  std::vector<char> in_round(n_waves, 0);
  for (uint32_t w : pending) in_round[w] = 1;
  for (uint32_t i = 0; i < n; ++i) {
    if (bad[i] >= n_waves || in_round[bad[i]] != 1) return false;
    in_round[bad[i]] = 2;
  }
  return true;
}

}  // namespace

extern "C" int tm_xfer_run_sender(uint32_t n_waves, uint32_t n_slots, uint32_t max_rounds, const tm_xfer_hooks* h,
                                  tm_xfer_stats* stats) {
  if (n_waves == 0 || n_slots == 0 || max_rounds == 0 || h == nullptr) return TM_ERR_ARG;
  if (h->pack == nullptr || h->send == nullptr || h->recv_report == nullptr) return TM_ERR_ARG;
  stats_init(stats);
  return guarded([&]() -> int {
    std::vector<uint32_t> pending(n_waves), bad(n_waves);
    for (uint32_t w = 0; w < n_waves; ++w) pending[w] = w;
    for (uint32_t round = 0; round < max_rounds; ++round) {
      for (uint32_t j = 0; j < pending.size(); ++j) {
        const uint32_t slot = j % n_slots;
        TM_HOOK(h->pack(h->ctx, pending[j], slot));
        TM_HOOK(h->send(h->ctx, pending[j], slot));
      }
      if (stats != nullptr) {
        stats->rounds = round + 1;
        stats->waves += (uint32_t)pending.size();
        if (round > 0) stats->waves_again += (uint32_t)pending.size();
      }
      uint32_t n_bad = 0;
      TM_HOOK(h->recv_report(h->ctx, bad.data(), n_waves, &n_bad));
      if (n_bad > n_waves || !report_is_valid(pending, bad.data(), n_bad, n_waves)) return TM_ERR_TRANSPORT;
      if (n_bad == 0) return TM_OK;
      pending.assign(bad.begin(), bad.begin() + n_bad);
    }
    return TM_ERR_VERIFY;
  });
}

extern "C" int tm_xfer_run_receiver(uint32_t n_waves, uint32_t n_slots, uint32_t max_rounds, const tm_xfer_hooks* h,
                                    tm_xfer_stats* stats) {
  if (n_waves == 0 || n_slots == 0 || max_rounds == 0 || h == nullptr) return TM_ERR_ARG;
  if (h->recv == nullptr || h->unpack_verify == nullptr || h->bad_waves == nullptr || h->send_report == nullptr)
    return TM_ERR_ARG;
  stats_init(stats);
  return guarded([&]() -> int {
    std::vector<uint32_t> pending(n_waves), bad(n_waves);
    for (uint32_t w = 0; w < n_waves; ++w) pending[w] = w;
    for (uint32_t round = 0; round < max_rounds; ++round) {
      for (uint32_t j = 0; j < pending.size(); ++j) {
        const uint32_t slot = j % n_slots;
        TM_HOOK(h->recv(h->ctx, pending[j], slot));
        TM_HOOK(h->unpack_verify(h->ctx, pending[j], slot));
      }
      if (stats != nullptr) {
        stats->rounds = round + 1;
        stats->waves += (uint32_t)pending.size();
        if (round > 0) stats->waves_again += (uint32_t)pending.size();
      }
      uint32_t n_bad = 0;
      TM_HOOK(h->bad_waves(h->ctx, pending.data(), (uint32_t)pending.size(), bad.data(), &n_bad));
      if (n_bad > pending.size() || !report_is_valid(pending, bad.data(), n_bad, n_waves)) return TM_ERR_TRANSPORT;
      TM_HOOK(h->send_report(h->ctx, bad.data(), n_bad));
      if (n_bad == 0) return TM_OK;
      pending.assign(bad.begin(), bad.begin() + n_bad);
    }
    return TM_ERR_VERIFY;
  });
}

// ---- one side of a transfer on the GPU -------------------------------------------------------------

struct tm_xfer {
  std::vector<tm_desc> descs;           // the role's descriptors (one copy for all waves)
  bool emits = false;                   // shards attached: packing / unpacking also fills them
  std::vector<tm_plan*> waves;          // one range plan per wave
  std::vector<uint64_t> ws_off;         // each plan's place in the workspace
  uint64_t bucket_bytes = 0, per_wave = 0, n_buckets = 0, slot_bytes = 0, workspace_bytes = 0;
  uint32_t n_slots = 0;
  // set by tm_xfer_bind
  uint8_t* d_ring = nullptr;
  uint64_t* d_checksums = nullptr;
  uint64_t* d_peer = nullptr;
  std::vector<cudaEvent_t> filled, drained;   // per slot: contents complete / contents consumed
  std::vector<char> used;
  // per run
  const tm_transport* transport = nullptr;
  cudaStream_t work_stream = nullptr, wire_stream = nullptr;
  tm_xfer_stats* stats = nullptr;
  std::vector<uint64_t> host_mine, host_peer;

  ~tm_xfer() {
    for (tm_plan* p : waves) delete p;
    for (cudaEvent_t e : filled) cudaEventDestroy(e);
    for (cudaEvent_t e : drained) cudaEventDestroy(e);
  }
  uint8_t* slot_ptr(uint32_t slot) const { return d_ring + (uint64_t)slot * slot_bytes; }
};

namespace {

int check_wave(const tm_xfer* x, uint32_t wave, uint32_t slot) {
  return (wave < x->waves.size() && slot < x->n_slots) ? TM_OK : TM_ERR_ARG;
}

// sender steps
int hook_pack(void* ctx, uint32_t wave, uint32_t slot) {
  tm_xfer* x = static_cast<tm_xfer*>(ctx);
  if (check_wave(x, wave, slot) != TM_OK) return TM_ERR_ARG;
  const tm_plan* p = x->waves[wave];
  if (x->used[slot]) TM_CUDA(cudaStreamWaitEvent(x->work_stream, x->drained[slot], 0));   // the transport has read the slot
  int rc = x->emits
      ? tm_state_pack_emit(p, x->slot_ptr(slot), x->slot_bytes, x->d_checksums + p->first_bucket, x->work_stream)
      : tm_state_pack(p, x->slot_ptr(slot), x->slot_bytes, x->d_checksums + p->first_bucket, x->work_stream);
  if (rc != TM_OK) return rc;
  TM_CUDA(cudaEventRecord(x->filled[slot], x->work_stream));
  return TM_OK;
}

int hook_send(void* ctx, uint32_t wave, uint32_t slot) {
  tm_xfer* x = static_cast<tm_xfer*>(ctx);
  if (check_wave(x, wave, slot) != TM_OK) return TM_ERR_ARG;
  const tm_plan* p = x->waves[wave];
  TM_CUDA(cudaStreamWaitEvent(x->wire_stream, x->filled[slot], 0));
  int rc = hook_status(x->transport->send(x->transport->ctx, wave, x->slot_ptr(slot), p->total_bytes,
                                          x->d_checksums + p->first_bucket, p->n_buckets, x->wire_stream));
  if (rc != TM_OK) return rc;
  TM_CUDA(cudaEventRecord(x->drained[slot], x->wire_stream));
  x->used[slot] = 1;
  if (x->stats != nullptr) x->stats->bytes += p->total_bytes;
  return TM_OK;
}

int hook_recv_report(void* ctx, uint32_t* waves, uint32_t capacity, uint32_t* n) {
  tm_xfer* x = static_cast<tm_xfer*>(ctx);
  return hook_status(x->transport->recv_report(x->transport->ctx, waves, capacity, n));
}

// receiver steps
int hook_recv(void* ctx, uint32_t wave, uint32_t slot) {
  tm_xfer* x = static_cast<tm_xfer*>(ctx);
  if (check_wave(x, wave, slot) != TM_OK) return TM_ERR_ARG;
  const tm_plan* p = x->waves[wave];
  if (x->used[slot]) TM_CUDA(cudaStreamWaitEvent(x->wire_stream, x->drained[slot], 0));   // the previous wave has been unpacked
  int rc = hook_status(x->transport->recv(x->transport->ctx, wave, x->slot_ptr(slot), p->total_bytes,
                                          x->d_peer + p->first_bucket, p->n_buckets, x->wire_stream));
  if (rc != TM_OK) return rc;
  TM_CUDA(cudaEventRecord(x->filled[slot], x->wire_stream));
  if (x->stats != nullptr) x->stats->bytes += p->total_bytes;
  return TM_OK;
}

int hook_unpack_verify(void* ctx, uint32_t wave, uint32_t slot) {
  tm_xfer* x = static_cast<tm_xfer*>(ctx);
  if (check_wave(x, wave, slot) != TM_OK) return TM_ERR_ARG;
  const tm_plan* p = x->waves[wave];
  TM_CUDA(cudaStreamWaitEvent(x->work_stream, x->filled[slot], 0));
  int rc = x->emits
      ? tm_state_unpack_emit(p, x->slot_ptr(slot), p->total_bytes, x->d_checksums + p->first_bucket, x->work_stream)
      : tm_state_unpack_verify(p, x->slot_ptr(slot), p->total_bytes, x->d_checksums + p->first_bucket, x->work_stream);
  if (rc != TM_OK) return rc;
  TM_CUDA(cudaEventRecord(x->drained[slot], x->work_stream));
  x->used[slot] = 1;
  return TM_OK;
}

// Waits for the round's device work, then compares, bucket by bucket, the checksums recomputed from
// what arrived with the sender's; a wave whose kernel gave up a bounded wait counts as damaged too.
int hook_bad_waves(void* ctx, const uint32_t* waves, uint32_t n_waves, uint32_t* bad, uint32_t* n_bad) {
  tm_xfer* x = static_cast<tm_xfer*>(ctx);
  TM_CUDA(cudaStreamSynchronize(x->wire_stream));
  TM_CUDA(cudaStreamSynchronize(x->work_stream));
  x->host_mine.resize(x->n_buckets);
  x->host_peer.resize(x->n_buckets);
  TM_CUDA(cudaMemcpy(x->host_mine.data(), x->d_checksums, x->n_buckets * sizeof(uint64_t), cudaMemcpyDeviceToHost));
  TM_CUDA(cudaMemcpy(x->host_peer.data(), x->d_peer, x->n_buckets * sizeof(uint64_t), cudaMemcpyDeviceToHost));
  uint32_t count = 0;
  for (uint32_t i = 0; i < n_waves; ++i) {
    if (waves[i] >= x->waves.size()) return TM_ERR_ARG;
    const tm_plan* p = x->waves[waves[i]];
    bool damaged = false;
    for (uint64_t b = p->first_bucket; b < p->first_bucket + p->n_buckets; ++b) {
      if (x->host_mine[b] == x->host_peer[b]) continue;
      damaged = true;
      if (x->stats != nullptr) {
        x->stats->bad_buckets += 1;
        if (x->stats->first_bad_bucket == ~0ull) x->stats->first_bad_bucket = b;
      }
    }
    int device_status = 0;
    int rc = tm_plan_status(p, x->work_stream, &device_status);
    if (rc != TM_OK) return rc;
    if (device_status != 0) damaged = true;
    if (damaged) bad[count++] = waves[i];
  }
  *n_bad = count;
  return TM_OK;
}

int hook_send_report(void* ctx, const uint32_t* waves, uint32_t n) {
  tm_xfer* x = static_cast<tm_xfer*>(ctx);
  return hook_status(x->transport->send_report(x->transport->ctx, waves, n));
}

int run_side(tm_xfer* x, const tm_transport* t, void* work_stream, void* wire_stream, uint32_t max_rounds,
             tm_xfer_stats* stats, bool sender) {
  if (x == nullptr || t == nullptr || max_rounds == 0) return TM_ERR_ARG;
  if (x->d_ring == nullptr) return TM_ERR_STATE;
  if (sender ? (t->send == nullptr || t->recv_report == nullptr) : (t->recv == nullptr || t->send_report == nullptr))
    return TM_ERR_ARG;
  if (!sender && x->d_peer == nullptr) return TM_ERR_ARG;
  x->transport = t;
  x->work_stream = (cudaStream_t)work_stream;
  x->wire_stream = (cudaStream_t)wire_stream;
  x->stats = stats;
  std::fill(x->used.begin(), x->used.end(), 0);
  tm_xfer_hooks h;
  std::memset(&h, 0, sizeof(h));
  h.ctx = x;
  h.pack = hook_pack;
  h.send = hook_send;
  h.recv_report = hook_recv_report;
  h.recv = hook_recv;
  h.unpack_verify = hook_unpack_verify;
  h.bad_waves = hook_bad_waves;
  h.send_report = hook_send_report;
  // the loops reset *stats first; the hooks then add bytes and bad buckets to it
  const uint32_t n_waves = (uint32_t)x->waves.size();
  int rc = sender ? tm_xfer_run_sender(n_waves, x->n_slots, max_rounds, &h, stats)
                  : tm_xfer_run_receiver(n_waves, x->n_slots, max_rounds, &h, stats);
  x->stats = nullptr;
  x->transport = nullptr;
  return rc;
}

}  // namespace

extern "C" {

int tm_xfer_create(const tm_desc* descs, uint64_t n_desc, uint64_t bucket_bytes, uint64_t buckets_per_wave,
                   uint32_t n_slots, tm_xfer** out) {
  if (out == nullptr) return TM_ERR_ARG;
  *out = nullptr;
  if (buckets_per_wave == 0 || n_slots == 0 || n_slots > 64) return TM_ERR_ARG;
  if (bucket_bytes != 0 && buckets_per_wave > (1ull << 40) / bucket_bytes) return TM_ERR_ARG;   // a slot is at most 1 TiB
  return guarded([&]() -> int {
    tm_xfer* x = new tm_xfer();
    int rc = TM_OK;
    try {
      if (descs != nullptr && n_desc <= tms::kMaxDescs) x->descs.assign(descs, descs + n_desc);
      x->bucket_bytes = bucket_bytes;
      x->per_wave = buckets_per_wave;
      x->n_slots = n_slots;
      // one pass over the descriptors for the layout, one more for all waves together: the wave plans
      // hold their pieces only, not a copy of the role's descriptor list each
      tm_layout lay;
      rc = tm_layout_build(descs, n_desc, bucket_bytes, &lay);
      if (rc == TM_OK) {
        x->n_buckets = lay.whole_buckets;
        if ((lay.whole_buckets + buckets_per_wave - 1) / buckets_per_wave > (1u << 20)) rc = TM_ERR_ARG;   // more waves than any ring is driven with
        // all waves together hold the pieces of the whole stream: refuse an over-long list before building any
        const uint64_t bound = lay.whole_bytes / tms::tuning().chunk_bytes + lay.whole_bytes / bucket_bytes;
        if (rc == TM_OK && bound > tms::kMaxPieces) rc = TM_ERR_CAPACITY;
      }
      uint64_t first = 0, cursor = 0, pieces = 0;
      while (rc == TM_OK && first < x->n_buckets) {
        tm_plan* p = new tm_plan();
        x->waves.push_back(p);
        rc = tm_plan_fill(p, descs, n_desc, lay, /*ranged=*/true, first, buckets_per_wave, &cursor);
        if (rc != TM_OK) break;
        pieces += p->work.segs.size();
        if (pieces > tms::kMaxPieces) rc = TM_ERR_CAPACITY;
        x->ws_off.push_back(x->workspace_bytes);
        x->workspace_bytes += p->ws_layout.total;
        first += buckets_per_wave;
      }
    } catch (...) {
      delete x;
      throw;
    }
    if (rc != TM_OK) {
      delete x;
      return rc;
    }
    x->slot_bytes = buckets_per_wave * bucket_bytes;
    *out = x;
    return TM_OK;
  });
}

int tm_xfer_query(const tm_xfer* x, uint32_t* n_waves, uint64_t* slot_bytes, uint64_t* ring_bytes,
                  uint64_t* workspace_bytes, uint64_t* n_buckets) {
  if (x == nullptr) return TM_ERR_ARG;
  if (n_waves != nullptr) *n_waves = (uint32_t)x->waves.size();
  if (slot_bytes != nullptr) *slot_bytes = x->slot_bytes;
  if (ring_bytes != nullptr) *ring_bytes = x->slot_bytes * x->n_slots;
  if (workspace_bytes != nullptr) *workspace_bytes = x->workspace_bytes;
  if (n_buckets != nullptr) *n_buckets = x->n_buckets;
  return TM_OK;
}

int tm_xfer_bind(tm_xfer* x, void* d_ring, uint64_t ring_bytes, void* d_workspace, uint64_t workspace_bytes,
                 uint64_t* d_checksums, uint64_t* d_peer_checksums, void* stream) {
  if (x == nullptr || d_ring == nullptr || d_workspace == nullptr || d_checksums == nullptr) return TM_ERR_ARG;
  if (((uintptr_t)d_ring & 255) != 0 || ((uintptr_t)d_workspace & 255) != 0 || ((uintptr_t)d_checksums & 7) != 0 ||
      ((uintptr_t)d_peer_checksums & 7) != 0)
    return TM_ERR_ALIGN;
  if (ring_bytes < x->slot_bytes * x->n_slots || workspace_bytes < x->workspace_bytes) return TM_ERR_CAPACITY;
  return guarded([&]() -> int {
    for (size_t w = 0; w < x->waves.size(); ++w) {
      int rc = tm_plan_upload(x->waves[w], (uint8_t*)d_workspace + x->ws_off[w], x->waves[w]->ws_layout.total, stream);
      if (rc != TM_OK) return rc;
    }
    while (x->filled.size() < x->n_slots) {
      cudaEvent_t e = nullptr;
      TM_CUDA(cudaEventCreateWithFlags(&e, cudaEventDisableTiming));
      x->filled.push_back(e);
    }
    while (x->drained.size() < x->n_slots) {
      cudaEvent_t e = nullptr;
      TM_CUDA(cudaEventCreateWithFlags(&e, cudaEventDisableTiming));
      x->drained.push_back(e);
    }
    x->used.assign(x->n_slots, 0);
    x->d_ring = (uint8_t*)d_ring;
    x->d_checksums = d_checksums;
    x->d_peer = d_peer_checksums;
    return TM_OK;
  });
}

int tm_xfer_attach_shards(tm_xfer* x, const uint64_t* plane_first_desc, const uint64_t* plane_n_desc, uint32_t n_planes,
                          uint32_t r, uint32_t D, void* const* d_outs, const uint64_t* out_capacities,
                          uint64_t* out_elems, void* d_workspace, uint64_t workspace_bytes,
                          uint64_t* workspace_needed, void* stream) {
  if (x == nullptr) return TM_ERR_ARG;
  if (((uintptr_t)d_workspace & 255) != 0) return TM_ERR_ALIGN;
  return guarded([&]() -> int {
    // size pass: every wave's list with its emit records
    uint64_t need = 0;
    std::vector<uint64_t> off(x->waves.size());
    for (size_t w = 0; w < x->waves.size(); ++w) {
      uint64_t n = 0;
      int rc = tm_attach_shards(x->waves[w], x->descs.data(), x->descs.size(), plane_first_desc, plane_n_desc, n_planes, r, D,
                                nullptr, nullptr, w == 0 ? out_elems : nullptr, nullptr, 0, &n, stream);
      if (rc != TM_OK) return rc;
      off[w] = need;
      need += n;
    }
    if (workspace_needed != nullptr) *workspace_needed = need;
    if (d_workspace == nullptr) return TM_OK;
    if (workspace_bytes < need) return TM_ERR_CAPACITY;
    for (size_t w = 0; w < x->waves.size(); ++w) {
      const uint64_t span = (w + 1 < off.size() ? off[w + 1] : need) - off[w];
      int rc = tm_attach_shards(x->waves[w], x->descs.data(), x->descs.size(), plane_first_desc, plane_n_desc, n_planes, r, D,
                                d_outs, out_capacities, nullptr, (uint8_t*)d_workspace + off[w], span, nullptr, stream);
      if (rc != TM_OK) return rc;
    }
    x->emits = true;
    return TM_OK;
  });
}

int tm_xfer_send(tm_xfer* x, const tm_transport* transport, void* pack_stream, void* send_stream,
                 uint32_t max_rounds, tm_xfer_stats* stats) {
  return run_side(x, transport, pack_stream, send_stream, max_rounds, stats, /*sender=*/true);
}

int tm_xfer_receive(tm_xfer* x, const tm_transport* transport, void* unpack_stream, void* recv_stream,
                    uint32_t max_rounds, tm_xfer_stats* stats) {
  return run_side(x, transport, unpack_stream, recv_stream, max_rounds, stats, /*sender=*/false);
}

void tm_xfer_destroy(tm_xfer* x) { delete x; }

}  // extern "C"

// ---- loopback transport: both sides in one process, on one GPU ---------------------------------------

struct tm_loopback {
  std::mutex m;
  std::condition_variable cv;
  // one posted receive at a time; `posts` and `taken` count the receives posted and the receives whose
  // stream has been made to wait for the sender's copy (a sender waits for "its" receive by number: the
  // receiver may already have posted the next one when the sender wakes up)
  bool posted = false, matched = false;
  uint64_t posts = 0, taken = 0;
  int match_rc = TM_OK;
  uint32_t wave = 0;
  void* d_slot = nullptr;
  uint64_t nbytes = 0;
  uint64_t* d_cks = nullptr;
  uint64_t n_cks = 0;
  cudaEvent_t slot_ready = nullptr;   // recorded by the receiver: its slot may be overwritten
  cudaEvent_t data_ready = nullptr;   // recorded by the sender: slot and checksums have been copied
  // one report at a time
  bool report_posted = false;
  std::vector<uint32_t> report;

  ~tm_loopback() {
    if (slot_ready != nullptr) cudaEventDestroy(slot_ready);
    if (data_ready != nullptr) cudaEventDestroy(data_ready);
  }
};

namespace {

constexpr std::chrono::seconds kPartnerTimeout(60);

int lb_recv(void* ctx, uint32_t wave, void* d_slot, uint64_t nbytes, uint64_t* d_cks, uint64_t n_cks, void* stream) {
  tm_loopback* lb = static_cast<tm_loopback*>(ctx);
  std::unique_lock<std::mutex> lock(lb->m);
  if (!lb->cv.wait_for(lock, kPartnerTimeout, [&] { return !lb->posted; })) return TM_ERR_TRANSPORT;
  TM_CUDA(cudaEventRecord(lb->slot_ready, (cudaStream_t)stream));
  lb->wave = wave;
  lb->d_slot = d_slot;
  lb->nbytes = nbytes;
  lb->d_cks = d_cks;
  lb->n_cks = n_cks;
  lb->matched = false;
  lb->posted = true;
  lb->posts += 1;
  lb->cv.notify_all();
  const bool met = lb->cv.wait_for(lock, kPartnerTimeout, [&] { return lb->matched; });
  int rc = met ? lb->match_rc : TM_ERR_TRANSPORT;
  if (rc == TM_OK && cudaStreamWaitEvent((cudaStream_t)stream, lb->data_ready, 0) != cudaSuccess) rc = TM_ERR_CUDA;
  lb->posted = false;
  lb->matched = false;
  lb->taken += 1;
  lb->cv.notify_all();
  return rc;
}

int lb_send(void* ctx, uint32_t wave, const void* d_slot, uint64_t nbytes, const uint64_t* d_cks, uint64_t n_cks,
            void* stream) {
  tm_loopback* lb = static_cast<tm_loopback*>(ctx);
  cudaStream_t st = (cudaStream_t)stream;
  std::unique_lock<std::mutex> lock(lb->m);
  if (!lb->cv.wait_for(lock, kPartnerTimeout, [&] { return lb->posted && !lb->matched; })) return TM_ERR_TRANSPORT;
  int rc = TM_OK;
  if (lb->wave != wave || lb->nbytes != nbytes || lb->n_cks != n_cks) {
    rc = TM_ERR_TRANSPORT;   // the two sides disagree about what travels now
  } else {
    cudaError_t e = cudaStreamWaitEvent(st, lb->slot_ready, 0);
    if (e == cudaSuccess) e = cudaMemcpyAsync(lb->d_slot, d_slot, nbytes, cudaMemcpyDeviceToDevice, st);
    if (e == cudaSuccess) e = cudaMemcpyAsync(lb->d_cks, d_cks, n_cks * sizeof(uint64_t), cudaMemcpyDeviceToDevice, st);
    if (e == cudaSuccess) e = cudaEventRecord(lb->data_ready, st);
    if (e != cudaSuccess) rc = tms::cuda_fail((int)e);
  }
  lb->match_rc = rc;
  lb->matched = true;
  const uint64_t mine = lb->posts;
  lb->cv.notify_all();
  // data_ready must not be recorded again before the receiver has made its stream wait on this record
  if (!lb->cv.wait_for(lock, kPartnerTimeout, [&] { return lb->taken >= mine; })) return TM_ERR_TRANSPORT;
  return rc;
}

int lb_send_report(void* ctx, const uint32_t* waves, uint32_t n) {
  tm_loopback* lb = static_cast<tm_loopback*>(ctx);
  std::unique_lock<std::mutex> lock(lb->m);
  if (!lb->cv.wait_for(lock, kPartnerTimeout, [&] { return !lb->report_posted; })) return TM_ERR_TRANSPORT;
  lb->report.assign(waves, waves + n);
  lb->report_posted = true;
  lb->cv.notify_all();
  return TM_OK;
}

int lb_recv_report(void* ctx, uint32_t* waves, uint32_t capacity, uint32_t* n) {
  tm_loopback* lb = static_cast<tm_loopback*>(ctx);
  std::unique_lock<std::mutex> lock(lb->m);
  // the receiver reports only after its device work of the round has finished: allow for a long round
  if (!lb->cv.wait_for(lock, 10 * kPartnerTimeout, [&] { return lb->report_posted; })) return TM_ERR_TRANSPORT;
  if (lb->report.size() > capacity) return TM_ERR_TRANSPORT;
  std::copy(lb->report.begin(), lb->report.end(), waves);
  *n = (uint32_t)lb->report.size();
  lb->report_posted = false;
  lb->cv.notify_all();
  return TM_OK;
}

}  // namespace

extern "C" {

int tm_loopback_create(tm_loopback** out, tm_transport* transport) {
  if (out == nullptr || transport == nullptr) return TM_ERR_ARG;
  *out = nullptr;
  return guarded([&]() -> int {
    tm_loopback* lb = new tm_loopback();
    cudaError_t e = cudaEventCreateWithFlags(&lb->slot_ready, cudaEventDisableTiming);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&lb->data_ready, cudaEventDisableTiming);
    if (e != cudaSuccess) {
      delete lb;
      return tms::cuda_fail((int)e);
    }
    transport->ctx = lb;
    transport->send = lb_send;
    transport->recv = lb_recv;
    transport->send_report = lb_send_report;
    transport->recv_report = lb_recv_report;
    *out = lb;
    return TM_OK;
  });
}

void tm_loopback_destroy(tm_loopback* lb) { delete lb; }

}  // extern "C"
