/* A plain C11 client of the library: includes the public header as C, links libcobalt.so, and
 * (when a CUDA device is present) routes a tiny batch over the Fig. 1 layout through the four
 * stages with raw device pointers obtained from the CUDA runtime, checking the values that the
 * paper's figure fixes by hand.  Exit code 0 = ok, 77 = no device (host-side checks still ran). */
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <cuda_runtime_api.h>

#include "cobalt.h"

#define CHECK(cond)                                                        \
    do {                                                                   \
        if (!(cond)) {                                                     \
            fprintf(stderr, "check failed at line %d: %s\n", __LINE__, #cond); \
            return 1;                                                      \
        }                                                                  \
    } while (0)

int main(void)
{
    /* Fig. 1: GPU0 {a,b} GPU1 {c,a} | GPU2 {b,c} GPU3 {d,a}; a b c d = 0 1 2 3 */
    const int32_t slot_expert[8] = {0, 1, 2, 0, 1, 2, 3, 0};
    const int32_t primary[4] = {0, 4, 2, 6};
    CHECK(cobalt_version() == COBALT_VERSION);
    CHECK(cobalt_layout_check(2, 2, 2, 4, slot_expert, primary) == COBALT_OK);
    const int32_t twice[8] = {0, 0, 2, 1, 1, 2, 3, 0};
    CHECK(cobalt_layout_check(2, 2, 2, 4, twice, NULL) == COBALT_ERR_INVALID_ARG);
    CHECK(strcmp(cobalt_status_string(COBALT_ERR_WORKSPACE_TOO_SMALL), "workspace too small") == 0);

    int n_dev = 0;
    if (cudaGetDeviceCount(&n_dev) != cudaSuccess || n_dev == 0) {
        printf("c_abi_check: host-side checks ok, no CUDA device\n");
        return 77;
    }

    enum { T = 12, K = 2, E = 4, D = 8, H = 8, P = T * K };
    const int32_t ids_h[P] = {0, 1, 0, 2, 0, 3, 1, 2, 1, 3, 2, 3, 0, 1, 0, 2, 0, 3, 1, 2, 1, 3, 2, 3};
    const int32_t src_h[T] = {0, 0, 0, 0, 0, 0, 2, 2, 2, 2, 2, 2};
    float w_h[P];
    uint16_t x_h[T * H];
    for (int i = 0; i < P; ++i) w_h[i] = 0.5f;
    for (int i = 0; i < T * H; ++i) x_h[i] = (uint16_t)(0x3F80 + (i % 64));   /* bf16 values in [1, 2) */

    cobalt_layout_t* layout = NULL;
    CHECK(cobalt_layout_create(&layout, 2, 2, 2, E, slot_expert, primary) == COBALT_OK);
    CHECK(cobalt_layout_num_dests(layout) == D);

    const size_t ws_bytes = 1 << 20;
    int32_t *ids, *src, *slots, *rop, *por;
    uint32_t *coact, *load, *slot_load, *counts, *offsets;
    uint8_t* remote;
    uint64_t* totals;
    float* w;
    uint16_t *x, *send, *y;
    void* ws;
    CHECK(cudaMalloc((void**)&ids, sizeof ids_h) == cudaSuccess);
    CHECK(cudaMalloc((void**)&src, sizeof src_h) == cudaSuccess);
    CHECK(cudaMalloc((void**)&slots, sizeof(int32_t) * P) == cudaSuccess);
    CHECK(cudaMalloc((void**)&rop, sizeof(int32_t) * P) == cudaSuccess);
    CHECK(cudaMalloc((void**)&por, sizeof(int32_t) * P) == cudaSuccess);
    CHECK(cudaMalloc((void**)&coact, sizeof(uint32_t) * E * E) == cudaSuccess);
    CHECK(cudaMalloc((void**)&load, sizeof(uint32_t) * E) == cudaSuccess);
    CHECK(cudaMalloc((void**)&slot_load, sizeof(uint32_t) * D) == cudaSuccess);
    CHECK(cudaMalloc((void**)&counts, sizeof(uint32_t) * D) == cudaSuccess);
    CHECK(cudaMalloc((void**)&offsets, sizeof(uint32_t) * (D + 1)) == cudaSuccess);
    CHECK(cudaMalloc((void**)&remote, T) == cudaSuccess);
    CHECK(cudaMalloc((void**)&totals, sizeof(uint64_t) * 2) == cudaSuccess);
    CHECK(cudaMalloc((void**)&w, sizeof w_h) == cudaSuccess);
    CHECK(cudaMalloc((void**)&x, sizeof x_h) == cudaSuccess);
    CHECK(cudaMalloc((void**)&send, sizeof(uint16_t) * P * H) == cudaSuccess);
    CHECK(cudaMalloc((void**)&y, sizeof x_h) == cudaSuccess);
    CHECK(cudaMalloc(&ws, ws_bytes) == cudaSuccess);
    CHECK(cudaMemcpy(ids, ids_h, sizeof ids_h, cudaMemcpyHostToDevice) == cudaSuccess);
    CHECK(cudaMemcpy(src, src_h, sizeof src_h, cudaMemcpyHostToDevice) == cudaSuccess);
    CHECK(cudaMemcpy(w, w_h, sizeof w_h, cudaMemcpyHostToDevice) == cudaSuccess);
    CHECK(cudaMemcpy(x, x_h, sizeof x_h, cudaMemcpyHostToDevice) == cudaSuccess);

    CHECK(cobalt_coact_stats(ids, T, K, E, coact, load, 0, ws, ws_bytes, NULL) == COBALT_OK);
    CHECK(cobalt_assign(layout, ids, src, 0, T, K, 36959u, slots, slot_load, remote, totals, 0, ws, ws_bytes, NULL) ==
          COBALT_OK);
    CHECK(cobalt_permute(slots, T, K, D, x, H, send, counts, offsets, rop, por, 0, ws, ws_bytes, NULL) == COBALT_OK);
    CHECK(cobalt_combine(send, rop, w, T, K, H, y, 0, NULL) == COBALT_OK);
    uint32_t err_bits = 1;
    CHECK(cobalt_read_and_clear_device_error(&err_bits, NULL) == COBALT_OK);
    CHECK(err_bits == 0);

    uint32_t coact_h[E * E], load_h[E], offsets_h[D + 1];
    uint64_t totals_h[2];
    uint8_t remote_h[T];
    int32_t slots_h[P];
    uint16_t y_h[T * H];
    CHECK(cudaMemcpy(coact_h, coact, sizeof coact_h, cudaMemcpyDeviceToHost) == cudaSuccess);
    CHECK(cudaMemcpy(load_h, load, sizeof load_h, cudaMemcpyDeviceToHost) == cudaSuccess);
    CHECK(cudaMemcpy(offsets_h, offsets, sizeof offsets_h, cudaMemcpyDeviceToHost) == cudaSuccess);
    CHECK(cudaMemcpy(totals_h, totals, sizeof totals_h, cudaMemcpyDeviceToHost) == cudaSuccess);
    CHECK(cudaMemcpy(remote_h, remote, sizeof remote_h, cudaMemcpyDeviceToHost) == cudaSuccess);
    CHECK(cudaMemcpy(slots_h, slots, sizeof slots_h, cudaMemcpyDeviceToHost) == cudaSuccess);
    CHECK(cudaMemcpy(y_h, y, sizeof y_h, cudaMemcpyDeviceToHost) == cudaSuccess);

    /* every expert is selected 6 times, every pair twice; V = 3 against 10 for the naive rule */
    for (int i = 0; i < E; ++i)
        for (int j = 0; j < E; ++j) CHECK(coact_h[i * E + j] == (i == j ? 6u : 2u));
    for (int i = 0; i < E; ++i) CHECK(load_h[i] == 6u);
    CHECK(totals_h[0] == 3 && totals_h[1] == 10);
    const uint8_t want_remote[T] = {0, 0, 1, 0, 1, 1, 0, 0, 0, 0, 0, 0};
    CHECK(memcmp(remote_h, want_remote, T) == 0);
    for (int p = 0; p < P; ++p) CHECK(slot_expert[slots_h[p]] == ids_h[p]);   /* the replica holds its expert */
    CHECK(offsets_h[0] == 0 && offsets_h[D] == (uint32_t)P);
    /* identity experts and weights 0.5 + 0.5: y = x exactly */
    CHECK(memcmp(y_h, x_h, sizeof x_h) == 0);

    CHECK(cobalt_layout_destroy(layout) == COBALT_OK);
    printf("c_abi_check: ok (V = %llu, naive %llu)\n", (unsigned long long)totals_h[0],
           (unsigned long long)totals_h[1]);
    return 0;
}
