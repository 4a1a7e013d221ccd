/* Compiled as C99 by tests/test_host_api.py: the header must be plain C, and the host-only entry
 * points must work without a GPU when called from C. */
#include <stdio.h>
#include <string.h>
#include "tm_state.h"

/* A sender and a receiver of the transfer protocol, played in one thread over a tiny in-memory "wire":
 * the sender's steps only record what they were asked to do, the reports come from a script. */
static uint32_t packed[16], n_packed, report_calls;
static int c_pack(void* ctx, uint32_t wave, uint32_t slot) { (void)ctx; packed[n_packed++] = wave * 10 + slot; return 0; }
static int c_send(void* ctx, uint32_t wave, uint32_t slot) { (void)ctx; (void)wave; (void)slot; return 0; }
static int c_recv_report(void* ctx, uint32_t* waves, uint32_t capacity, uint32_t* n) {
  (void)ctx;
  if (capacity < 1) return 1;
  if (report_calls++ == 0) { waves[0] = 2; *n = 1; } else { *n = 0; }   /* first round: wave 2 again */
  return 0;
}

int main(void) {
  tm_desc d[3];
  memset(d, 0, sizeof d);
  d[0].ptr = (void*)0x7f0000000000ull; d[0].nbytes = 2;    d[0].elem_size = 2; d[0].plane = 0;
  d[1].ptr = (void*)0x7f0000100000ull; d[1].nbytes = 258;  d[1].elem_size = 2; d[1].plane = 0;
  d[2].ptr = (void*)0x7f0000200000ull; d[2].nbytes = 1000; d[2].elem_size = 4; d[2].plane = 1;
  tm_plan* plan = NULL;
  if (tm_plan_create(d, 3, 512, &plan) != TM_OK || plan == NULL) return 1;
  uint64_t total = 0, nb = 0, ws = 0, off[3] = {0, 0, 0};
  if (tm_plan_query(plan, &total, &nb, &ws) != TM_OK) return 2;
  if (tm_plan_offsets(plan, off) != TM_OK) return 3;
  /* off = 0, 256, 768; end = 1768 -> T = 1792; ceil(1792 / 512) = 4 buckets */
  if (off[0] != 0 || off[1] != 256 || off[2] != 768 || total != 1792 || nb != 4 || ws < 512) return 4;
  if (tm_state_pack(plan, (void*)0x7f1000000000ull, 1792, NULL, NULL) != TM_ERR_STATE) return 5;
  tm_plan_destroy(plan);
  uint64_t lo = 0, hi = 0;
  if (tm_shard_bounds(10, 2, 3, &lo, &hi) != TM_OK || lo != 6 || hi != 10) return 6;
  if (tm_shard_bounds(10, 3, 3, &lo, &hi) != TM_ERR_RANK) return 7;
  if (tm_plan_create(d, 3, 500, &plan) != TM_ERR_ALIGN) return 8;
  if (strcmp(tm_strerror(TM_ERR_OVERLAP), "buffers overlap") != 0) return 9;
  /* range plan: buckets 1..2 of the same stream: bytes [512, 1536) */
  uint64_t first = 0, begin = 0, wt = 0, wn = 0;
  if (tm_plan_create_range(d, 3, 512, 1, 2, &plan) != TM_OK) return 10;
  if (tm_plan_query(plan, &total, &nb, &ws) != TM_OK || total != 1024 || nb != 2) return 11;
  if (tm_plan_range(plan, &first, &begin, &wt, &wn) != TM_OK || first != 1 || begin != 512 || wt != 1792 || wn != 4) return 12;
  tm_plan_destroy(plan);
  if (tm_plan_create_range(d, 3, 512, 4, 1, &plan) != TM_ERR_ARG) return 13;
  /* options */
  tm_options o;
  if (tm_options_get(&o) != TM_OK || o.chunk_bytes != 256 * 1024 || o.wait_limit_ns != 2000000000ull) return 14;
  o.chunk_bytes = 4096 + 1;
  if (tm_options_set(&o) != TM_ERR_ALIGN) return 15;
  if (tm_options_set(NULL) != TM_OK) return 16;
  /* the protocol loop with C callbacks: 3 waves over 2 slots, wave 2 is requested again */
  tm_xfer_hooks h;
  tm_xfer_stats st;
  memset(&h, 0, sizeof h);
  h.pack = c_pack; h.send = c_send; h.recv_report = c_recv_report;
  if (tm_xfer_run_sender(3, 2, 3, &h, &st) != TM_OK) return 17;
  if (st.rounds != 2 || st.waves != 4 || st.waves_again != 1) return 18;
  if (n_packed != 4 || packed[0] != 0 || packed[1] != 11 || packed[2] != 20 || packed[3] != 20) return 19;
  if (tm_xfer_run_receiver(3, 2, 3, &h, &st) != TM_ERR_ARG) return 20;   /* receiver steps missing */
  printf("c abi ok, %llu launches\n", (unsigned long long)tm_launch_count());
  return 0;
}
