/* A plain C99 translation unit against the public header and the shared library: the declarations parse as C,
 * the symbols link, and the entry points that need no GPU behave as documented.  Built and run by
 * tests/test_boundary_cpu.py. */
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include "pdattn.h"

#define CHECK(cond)                                                      \
  do {                                                                   \
    if (!(cond)) {                                                       \
      fprintf(stderr, "abi_check: %s failed (line %d)\n", #cond, __LINE__); \
      return 1;                                                          \
    }                                                                    \
  } while (0)

int main(void) {
  size_t n = 0, pinned = 1;
  CHECK(pdattn_workspace_size(256, 28, 4, 128, 16, 8192, &n, &pinned) == PDATTN_OK);
  CHECK(n > 0 && n % 256 == 0 && pinned == 0);
  CHECK(pdattn_workspace_size(256, 28, 4, 96, 16, 8192, &n, NULL) == PDATTN_UNSUPPORTED);
  CHECK(strcmp(pdattn_status_string(PDATTN_OK), "ok") == 0);

  /* the host partitioner: three sequences of 100, 1000 and 10 tokens, two KV heads, four CTAs */
  {
    const int32_t lens[3] = {100, 1000, 10};
    int32_t spans[4 * (4 + 1)];
    pdattn_plan plan;
    int i, tiles = 0;
    CHECK(pdattn_plan_host(lens, 3, 2, 4, 0, 4, spans, &plan) == PDATTN_OK);
    CHECK(plan.n_static == 4 && plan.n_dynamic == 0);
    CHECK(plan.total_tiles == 2 * (2 + 16 + 1));          /* ceil(L / 64) tiles per unit, two units per sequence */
    for (i = 0; i < 4; ++i) {
      CHECK(spans[4 * (i + 1) + 2] >= spans[4 * i + 2]);  /* flat tile numbers ascend */
      tiles += spans[4 * (i + 1) + 2] - spans[4 * i + 2];
    }
    CHECK(tiles == plan.total_tiles && spans[2] == 0);
  }

  /* argument checks come before any CUDA call */
  CHECK(pdattn_decode_ex(NULL, NULL) == PDATTN_INVALID_ARG);
  CHECK(pdattn_set_merge_mode(7) == PDATTN_INVALID_ARG && pdattn_set_merge_mode(-1) == PDATTN_OK);
  printf("abi_check: ok\n");
  return 0;
}
