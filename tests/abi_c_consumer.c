/* A plain C99 consumer of the library: includes the public header, links against libkvrebuild.so and calls the
 * entry points that need no device (Eq. (1), the window selection of Algorithm 1, status strings).  Built and
 * run by tests/test_abi_host.py to show that the boundary is usable without C++ or Python. */
#include "kvrebuild.h"

#include <stddef.h>
#include <stdio.h>
#include <string.h>

int main(void) {
  kv_window_inputs in;
  kv_window_eval best;
  int32_t trigger = -1;
  memset(&in, 0, sizeof(in));
  in.k_curr = 4096.0;
  in.r_p = 20000.0;
  in.r_d = 50.0;
  in.goodput = 37.5e6;
  in.s_kv = (double)kv_bytes_per_token(64, 8, 128, 2);
  in.t0 = 0.015;
  in.alpha = 0.8;
  in.t_remain = 5.0;
  if (in.s_kv != 262144.0) return 2;
  if (kv_window_select(&in, 3.0, 0.05, &best, &trigger) != KV_OK) return 3;
  if (trigger != 0 && trigger != 1) return 4;
  if (best.t_w < 0.0 || best.t_w > 3.0) return 5;
  if (kv_window_select(NULL, 3.0, 0.05, &best, &trigger) != KV_ERR_ARG) return 6;
  if (kv_status_string(KV_ERR_GAP) == NULL || strlen(kv_status_string(KV_ERR_GAP)) == 0) return 7;
  if (kv_pack_blocks(NULL, NULL, 0, NULL, 0, KV_WIRE_BLOCK_MAJOR, NULL) != KV_ERR_ARG) return 8;
  printf("t_w=%.3f t_sit=%.4f trigger=%d\n", best.t_w, best.t_sit, (int)trigger);
  return 0;
}
