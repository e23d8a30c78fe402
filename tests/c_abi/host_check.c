/* A plain C program against the C ABI: the header must compile as C, the library must link from C,
 * and the host-only calls must work without a GPU.  Prints "ok" and exits 0 on success. */
#include <stdio.h>
#include <string.h>

#include "distdl.h"

#define CHECK(cond)                                                         \
    do {                                                                    \
        if (!(cond)) {                                                      \
            printf("failed: %s (line %d): %s\n", #cond, __LINE__, distdl_last_error()); \
            return 1;                                                       \
        }                                                                   \
    } while (0)

int main(void) {
    /* Fig. B2 of the paper's appendix: kernel 5, no padding, 11 inputs on 3 workers */
    int32_t lo[3], hi[3], ulo[3], uhi[3];
    CHECK(distdl_halo_widths_1d(11, 3, 5, 1, 1, 0, 0, lo, hi, ulo, uhi) == DISTDL_OK);
    CHECK(lo[0] == 0 && lo[1] == 1 && lo[2] == 3 && hi[0] == 3 && hi[1] == 1 && hi[2] == 0);

    const int64_t shape[3] = {512, 512, 512};
    const int32_t workers[3] = {4, 4, 4}, h[3] = {4, 4, 4};
    distdl_partition_t *p = NULL;
    /* without a GPU the partition is host-only: geometry and plan sizes work */
    const distdl_status_t st = distdl_partition_create(3, shape, workers, h, h, DISTDL_F32, &p);
    CHECK(st == DISTDL_OK);
    CHECK(distdl_partition_num_workers(p) == 64);
    int64_t start[3], bulk[3], padded[3];
    int32_t wlo[3], whi[3];
    CHECK(distdl_partition_shard_extents(p, 21, start, bulk, padded, wlo, whi) == DISTDL_OK);   /* worker (1, 1, 1) */
    CHECK(start[0] == 128 && start[1] == 128 && start[2] == 128 && bulk[0] == 128 && padded[2] == 136 && wlo[1] == 4);
    int64_t boxes, tiles, bytes;
    CHECK(distdl_partition_halo_stats(p, 0, &boxes, &tiles, &bytes) == DISTDL_OK);
    CHECK(boxes == 64 * 26 && bytes == 186177536);
    CHECK(distdl_partition_halo_stats(p, 1, NULL, NULL, &bytes) == DISTDL_OK && bytes == 330205184);
    distdl_partition_destroy(p);

    /* error reporting */
    const int32_t too_many[3] = {1024, 1, 1};
    CHECK(distdl_partition_create(3, shape, too_many, NULL, NULL, DISTDL_F32, &p) == DISTDL_ERR_SHAPE ||
          distdl_partition_create(3, shape, too_many, NULL, NULL, DISTDL_F32, &p) == DISTDL_ERR_UNSUPPORTED);
    CHECK(strlen(distdl_last_error()) > 0);
    printf("ok\n");
    return 0;
}
