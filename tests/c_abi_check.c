/* The header is plain C: compile with a C compiler, link against libastro.so, exercise the host-only part of
 * the ABI (no device is touched).  Exit code 0 on success. */
#include <stdio.h>
#include <string.h>

#include "astro.h"

#define CHECK(cond)                                            \
  do {                                                         \
    if (!(cond)) {                                             \
      fprintf(stderr, "check failed: %s (line %d)\n", #cond, __LINE__); \
      return 1;                                                \
    }                                                          \
  } while (0)

int main(void) {
  astro_kvcache_desc_t d;
  astro_kvcache_t* cache = NULL;
  astro_kvcache_state_t st;
  int sink = -1, win = -1;
  int64_t seen = -1;
  d.cache_batch = 2; d.heads = 12; d.head_dim = 128; d.tokens_per_frame = 1560; d.sink_frames = 3; d.window_frames = 12;
  CHECK(astro_kvcache_storage_bytes(&d) == (size_t)2 * 12 * 15 * 1560 * 128 * 2);
  CHECK(astro_kvcache_create(&d, (void*)0x1000, (void*)0x2000, (size_t)1 << 40, &cache) == ASTRO_OK);
  CHECK(astro_kvcache_query(cache, &sink, &win, &seen) == ASTRO_OK && sink == 0 && win == 0 && seen == 0);
  CHECK(astro_kvcache_evict(cache, 1, NULL) == ASTRO_ERR_UNDERFLOW);
  CHECK(astro_kvcache_append(cache, (void*)0x3000, (void*)0x4000, 16, NULL) == ASTRO_ERR_CAPACITY);
  st.sink_held = 3; st.window_head = 5; st.window_held = 7; st.frames_seen = 40;
  CHECK(astro_kvcache_set_state(cache, &st) == ASTRO_OK);
  memset(&st, 0, sizeof(st));
  CHECK(astro_kvcache_get_state(cache, &st) == ASTRO_OK && st.window_head == 5 && st.frames_seen == 40);
  CHECK(astro_chunk_attn_fwd(cache, (void*)0x5000, NULL, NULL, 3, 12, 128, 4680, 0, 0.088f, (void*)0x6000, NULL, NULL)
        == ASTRO_ERR_SHAPE); /* batch 3 against a cache of 2 */
  CHECK(astro_chunk_attn_bwd_workspace_bytes(2, 12, 4680, 128) >= (size_t)2 * 12 * 4680 * 4);
  CHECK(strcmp(astro_status_string(ASTRO_OK), "ok") == 0);
  CHECK(astro_kvcache_destroy(cache) == ASTRO_OK);
  printf("c abi ok\n");
  return 0;
}
