/* Runs the library's host-only entry points (layout validation, the Stage-2 rebalancer) in a build
 * of runtime.cu and epilogue.cu whose host code is instrumented with -fsanitize=address,undefined.
 * No device is needed: none of these calls touches the CUDA runtime. */
#include <math.h>
#include <stdio.h>
#include <string.h>

#include "cobalt.h"

#define CHECK(cond)                                                          \
    do {                                                                     \
        if (!(cond)) {                                                       \
            fprintf(stderr, "%s:%d: check failed: %s\n", __FILE__, __LINE__, #cond); \
            return 1;                                                        \
        }                                                                    \
    } while (0)

int main(void)
{
    /* Fig. 1 layout and its faulty variants */
    const int32_t fig1[8] = {0, 1, 2, 0, 1, 2, 3, 0};
    const int32_t primary[4] = {0, 4, 2, 6};
    CHECK(cobalt_layout_check(2, 2, 2, 4, fig1, primary) == COBALT_OK);
    CHECK(cobalt_layout_check(2, 2, 2, 4, fig1, NULL) == COBALT_OK);
    const int32_t missing[8] = {0, 1, 2, 0, 1, 2, 0, 0}, twice[8] = {0, 0, 2, 1, 1, 2, 3, 0};
    const int32_t range[8] = {0, 1, 2, 0, 1, 2, 3, 4}, bad_primary[4] = {1, 4, 2, 6};
    CHECK(cobalt_layout_check(2, 2, 2, 4, missing, NULL) == COBALT_ERR_INVALID_ARG);
    CHECK(cobalt_layout_check(2, 2, 2, 4, twice, NULL) == COBALT_ERR_INVALID_ARG);
    CHECK(cobalt_layout_check(2, 2, 2, 4, range, NULL) == COBALT_ERR_INVALID_ARG);
    CHECK(cobalt_layout_check(2, 2, 2, 4, fig1, bad_primary) == COBALT_ERR_INVALID_ARG);
    CHECK(cobalt_layout_check(9, 2, 2, 4, fig1, NULL) == COBALT_ERR_UNSUPPORTED);
    CHECK(cobalt_layout_check(2, 2, 2, 4, NULL, NULL) == COBALT_ERR_INVALID_ARG);

    /* the largest layout of the envelope: N = 8, D = 4096, E = 1024, every expert four times */
    static int32_t big[4096];
    for (int d = 0; d < 4096; ++d) big[d] = (d % 64) * 16 + (d / 64) % 16;      /* rank r = d / 64 holds 64 distinct experts */
    CHECK(cobalt_layout_check(8, 8, 64, 1024, big, NULL) == COBALT_OK);

    /* rebalancer: hand cases (10,7,5,3 over two ranks -> 13/12), a dead end, empty slots, bad loads */
    int32_t out[8], moved[8], kept = -1;
    const int32_t four[4] = {0, 1, 2, 3};
    const float load4[4] = {10.f, 7.f, 5.f, 3.f};
    CHECK(cobalt_rebalance_intra_node(1, 2, 2, 4, four, load4, out, moved, &kept) == COBALT_OK);
    CHECK(out[0] == 0 && out[1] == 3 && out[2] == 1 && out[3] == 2 && kept == 0);
    CHECK(moved[0] == 0 && moved[1] == 3 && moved[2] == 1 && moved[3] == 2);
    const int32_t dead[4] = {0, 1, 2, 0};
    const float load_dead[4] = {10.f, 9.f, 8.f, 1.f};
    CHECK(cobalt_rebalance_intra_node(1, 2, 2, 3, dead, load_dead, out, NULL, &kept) == COBALT_OK);
    CHECK(kept == 1 && memcmp(out, dead, sizeof(dead)) == 0);
    const float load_fig1[8] = {5.f, 1.f, 2.f, 2.f, 4.f, 4.f, 0.f, 3.f};
    CHECK(cobalt_rebalance_intra_node(2, 2, 2, 4, fig1, load_fig1, out, moved, NULL) == COBALT_OK);
    CHECK(cobalt_layout_check(2, 2, 2, 4, out, NULL) == COBALT_OK);
    const float load_nan[4] = {10.f, NAN, 5.f, 3.f};
    CHECK(cobalt_rebalance_intra_node(1, 2, 2, 4, four, load_nan, out, moved, &kept) == COBALT_ERR_INVALID_ARG);
    CHECK(cobalt_rebalance_intra_node(1, 2, 2, 4, four, NULL, out, moved, &kept) == COBALT_ERR_INVALID_ARG);
    static float big_load[4096];
    static int32_t big_out[4096], big_moved[4096];
    for (int d = 0; d < 4096; ++d) big_load[d] = (float)((d * 37) % 11);
    CHECK(cobalt_rebalance_intra_node(8, 8, 64, 1024, big, big_load, big_out, big_moved, &kept) == COBALT_OK);
    CHECK(cobalt_layout_check(8, 8, 64, 1024, big_out, NULL) == COBALT_OK);

    CHECK(strcmp(cobalt_status_string(COBALT_ERR_HOST_ALLOC), "unknown status") != 0);
    CHECK(cobalt_version() == COBALT_VERSION);
    printf("host entry points ok under the sanitizers\n");
    return 0;
}
