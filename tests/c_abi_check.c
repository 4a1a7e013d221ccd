/* Compiled as C99 by tests/test_host_api.py: the header must be plain C, and the host-only entry
 * points must work without a GPU when called from C. */
#include <stdio.h>
#include <string.h>
#include "tm_state.h"

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
  printf("c abi ok, %llu launches\n", (unsigned long long)tm_launch_count());
  return 0;
}
