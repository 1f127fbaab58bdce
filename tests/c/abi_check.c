/* The public header must be plain C99 and the library usable without Python: plan a tiny
 * reshard on the host (no GPU needed) and print what came out. */
#include <stdio.h>
#include <string.h>

#include "bcp.h"

int main(void) {
  int64_t lengths[2] = {3, 2};
  int64_t off[4][BCP_MAX_NDIM], len[4][BCP_MAX_NDIM];
  size_t n = 0;
  if (bcp_decompose(lengths, 2, 0, 3, off, len, 4, &n) != BCP_OK || n != 2) return 1;
  if (off[1][0] != 1 || off[1][1] != 0 || len[1][0] != 1 || len[1][1] != 1) return 2;

  bcp_shard_meta src[2], dst[1];
  memset(src, 0, sizeof src);
  memset(dst, 0, sizeof dst);
  for (int i = 0; i < 2; ++i) { /* a (4, 6) fp32 tensor saved as two row blocks */
    src[i].fqn = "w";
    src[i].itemsize = 4;
    src[i].dtype_tag = 2;
    src[i].ndim = 2;
    src[i].kind = BCP_BOX;
    src[i].global_shape[0] = 4, src[i].global_shape[1] = 6;
    src[i].offsets[0] = 2 * i, src[i].lengths[0] = 2, src[i].lengths[1] = 6;
    src[i].buf_index = (uint32_t)i;
    src[i].byte_length = 48;
  }
  dst[0] = src[0]; /* wanted: columns 2..5 of all rows */
  dst[0].offsets[0] = 0, dst[0].lengths[0] = 4;
  dst[0].offsets[1] = 2, dst[0].lengths[1] = 4;
  dst[0].buf_index = 0;
  dst[0].byte_length = 64;
  uint64_t sb[2] = {48, 48}, db[1] = {64};
  bcp_plan_t* plan = NULL;
  if (bcp_plan(src, 2, sb, 2, dst, 1, db, 1, NULL, &plan) != BCP_OK) {
    printf("plan failed: %s\n", bcp_last_error());
    return 3;
  }
  bcp_plan_stats_t st;
  if (bcp_plan_stats(plan, &st) != BCP_OK || st.bytes_copied != 64 || st.n_intersections != 2) return 4;
  bcp_tile tiles[8];
  if (bcp_plan_tiles(plan, tiles, 8, &n) != BCP_OK || n != 2) return 5;
  /* each unit: 2 rows of 16 bytes, source pitch 24, target pitch 16 */
  for (size_t i = 0; i < n; ++i)
    if (tiles[i].rows != 2 || tiles[i].row_bytes != 16 || tiles[i].src_pitch != 24 || tiles[i].dst_pitch != 16) return 6;
  dst[0].byte_length = 60; /* wrong length: rejected with a message, nothing created */
  bcp_plan_t* bad = NULL;
  if (bcp_plan(src, 2, sb, 2, dst, 1, db, 1, NULL, &bad) != BCP_ERR_INVALID || bad != NULL || !bcp_last_error()[0]) return 7;
  bcp_plan_destroy(plan);
  printf("abi ok, version %d\n", bcp_version());
  return 0;
}
