/* Runs the C oracle over the Fig. 1 example and a ragged random case in a build instrumented with
 * -fsanitize=address,undefined: any out-of-bounds access, use of freed memory, signed overflow or
 * misaligned access in the oracle aborts this program.  The expected values are the hand-derived ones
 * of tests/golden/fig1_example.txt (V = 3 against 10 for the naive rule). */
#include <stdint.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

int oracle_layout_tables(int32_t N, int32_t Q, int32_t S, int32_t E, const int32_t* slot_expert,
                         const int32_t* primary_in, uint32_t* nodes_mask, int32_t* r_count, int32_t* r_list,
                         int32_t* primary);
int oracle_coact_stats(const int32_t* topk_ids, int64_t T, int32_t K, int32_t E, uint32_t* coact, uint32_t* load);
int oracle_assign(int32_t N, int32_t Q, int32_t S, int32_t E, const int32_t* slot_expert, const int32_t* primary_in,
                  const int32_t* topk_ids, const int32_t* src_rank, int64_t T, int32_t K, uint64_t seed,
                  uint32_t flags, int32_t* assigned_slot, uint32_t* slot_load, uint8_t* remote_nodes,
                  uint64_t* totals);
int oracle_traffic(int32_t N, int32_t Q, int32_t S, int32_t E, const int32_t* slot_expert, const int32_t* topk_ids,
                   const int32_t* src_rank, const int32_t* assigned_slot, int64_t T, int32_t K, uint8_t* per_token,
                   uint64_t* V_out);
int oracle_permute(const int32_t* assigned_slot, int64_t T, int32_t K, int32_t D, const uint16_t* x, int32_t H,
                   uint16_t* send, uint32_t* dest_counts, uint32_t* dest_offsets, int32_t* row_of_pair,
                   int32_t* pair_of_row);
int oracle_combine(const uint16_t* expert_out, const int32_t* row_of_pair, const float* gate_w, int64_t T, int32_t K,
                   int32_t H, const int64_t* tokens, int64_t n_tokens, float* y);

#define CHECK(cond)                                                          \
    do {                                                                     \
        if (!(cond)) {                                                       \
            fprintf(stderr, "%s:%d: check failed: %s\n", __FILE__, __LINE__, #cond); \
            return 1;                                                        \
        }                                                                    \
    } while (0)

static int run_case(int32_t N, int32_t Q, int32_t S, int32_t E, const int32_t* slot_expert, const int32_t* primary,
                    const int32_t* ids, const int32_t* src, int64_t T, int32_t K, int32_t H, uint64_t* totals)
{
    const int32_t D = N * Q * S;
    const int64_t P = T * K;
    /* every buffer has exactly the size the oracle documents, so that one element too far is caught */
    uint32_t* coact = malloc(sizeof(uint32_t) * (size_t)E * E);
    uint32_t* load = malloc(sizeof(uint32_t) * (size_t)E);
    int32_t* slots = malloc(sizeof(int32_t) * (size_t)(P > 0 ? P : 1));
    uint32_t* slot_load = malloc(sizeof(uint32_t) * (size_t)D);
    uint8_t* remote = malloc((size_t)(T > 0 ? T : 1));
    uint16_t* x = malloc(sizeof(uint16_t) * (size_t)(T > 0 ? T : 1) * H);
    uint16_t* send = malloc(sizeof(uint16_t) * (size_t)(P > 0 ? P : 1) * H);
    uint32_t* counts = malloc(sizeof(uint32_t) * (size_t)D);
    uint32_t* offsets = malloc(sizeof(uint32_t) * (size_t)(D + 1));
    int32_t* row_of_pair = malloc(sizeof(int32_t) * (size_t)(P > 0 ? P : 1));
    int32_t* pair_of_row = malloc(sizeof(int32_t) * (size_t)(P > 0 ? P : 1));
    float* gate = malloc(sizeof(float) * (size_t)(P > 0 ? P : 1));
    float* y = malloc(sizeof(float) * (size_t)(T > 0 ? T : 1) * H);
    for (int64_t i = 0; i < T * H; ++i) x[i] = (uint16_t)(0x3F80u + (i % 7));      /* bf16 values near 1 */
    for (int64_t p = 0; p < P; ++p) gate[p] = 1.0f / (float)K;
    CHECK(oracle_coact_stats(ids, T, K, E, coact, load) == 0);
    for (uint32_t flags = 0; flags < 3; ++flags) {
        CHECK(oracle_assign(N, Q, S, E, slot_expert, primary, ids, src, T, K, 36959u, flags, slots, slot_load, remote,
                            totals) == 0);
        uint64_t V = 0;
        CHECK(oracle_traffic(N, Q, S, E, slot_expert, ids, src, slots, T, K, NULL, &V) == 0);
        CHECK(V == totals[0]);
    }
    CHECK(oracle_assign(N, Q, S, E, slot_expert, primary, ids, src, T, K, 36959u, 0, slots, slot_load, remote,
                        totals) == 0);
    CHECK(oracle_permute(slots, T, K, D, x, H, send, counts, offsets, row_of_pair, pair_of_row) == 0);
    CHECK(offsets[D] == (uint32_t)P);
    for (int32_t d = 0; d < D; ++d) CHECK(counts[d] == slot_load[d]);
    CHECK(oracle_combine(send, row_of_pair, gate, T, K, H, NULL, 0, y) == 0);
    free(coact); free(load); free(slots); free(slot_load); free(remote); free(x); free(send); free(counts);
    free(offsets); free(row_of_pair); free(pair_of_row); free(gate); free(y);
    return 0;
}

int main(void)
{
    /* Fig. 1: GPU0 {a,b} GPU1 {c,a} | GPU2 {b,c} GPU3 {d,a}; every 2-subset from node 0 and from node 1 */
    const int32_t slot_expert[8] = {0, 1, 2, 0, 1, 2, 3, 0};
    const int32_t primary[4] = {0, 4, 2, 6};
    int32_t ids[24], src[12];
    int n = 0;
    for (int s = 0; s < 2; ++s)
        for (int a = 0; a < 4; ++a)
            for (int b = a + 1; b < 4; ++b) {
                ids[2 * n] = a;
                ids[2 * n + 1] = b;
                src[n] = 2 * s;
                ++n;
            }
    uint64_t totals[2] = {0, 0};
    if (run_case(2, 2, 2, 4, slot_expert, primary, ids, src, 12, 2, 8, totals)) return 1;
    CHECK(totals[0] == 3 && totals[1] == 10);

    /* a ragged case with eight nodes, empty slots and K = 5 (sizes that are multiples of nothing) */
    enum { N = 8, Q = 3, S = 2, E = 19, K = 5, T = 37 };
    int32_t lay[N * Q * S];
    for (int d = 0; d < N * Q * S; ++d) lay[d] = (d % 5 == 4) ? -1 : (d * 7) % E;
    for (int r = 0; r < N * Q; ++r)
        if (lay[r * S] == lay[r * S + 1]) lay[r * S + 1] = -1;
    int32_t ids2[T * K], src2[T];
    uint32_t x = 12345u;
    for (int t = 0; t < T; ++t) {
        src2[t] = (t * 5) % (N * Q);
        int32_t first = (int32_t)((x = x * 1664525u + 1013904223u) >> 8) % E;
        int32_t step = 1 + (int32_t)((x = x * 1664525u + 1013904223u) >> 8) % 3;
        for (int k = 0; k < K; ++k) ids2[t * K + k] = (first + step * k) % E;      /* distinct: step * K < E */
    }
    uint32_t mask[E];
    int32_t r_count[E * N], r_list[E * N * Q], prim[E];
    int rc = oracle_layout_tables(N, Q, S, E, lay, NULL, mask, r_count, r_list, prim);
    if (rc == 0) {
        if (run_case(N, Q, S, E, lay, NULL, ids2, src2, T, K, 24, totals)) return 1;
        CHECK(totals[0] <= totals[1]);
    } else {
        /* some expert got no slot: the oracle must say so rather than read past its tables */
        CHECK(rc == -1);
    }
    /* inputs the oracle must refuse: an id outside [0, E), a duplicate, a source rank outside [0, G) */
    int32_t bad_ids[2] = {0, 4}, dup_ids[2] = {1, 1}, one_src[1] = {0}, bad_src[1] = {4}, out[2];
    CHECK(oracle_assign(2, 2, 2, 4, slot_expert, primary, bad_ids, one_src, 1, 2, 1u, 0, out, NULL, NULL, NULL) == -2);
    CHECK(oracle_assign(2, 2, 2, 4, slot_expert, primary, dup_ids, one_src, 1, 2, 1u, 0, out, NULL, NULL, NULL) == -2);
    CHECK(oracle_assign(2, 2, 2, 4, slot_expert, primary, ids, bad_src, 1, 2, 1u, 0, out, NULL, NULL, NULL) == -2);
    printf("oracle ok under the sanitizers (V = %llu, naive %llu on Fig. 1)\n", 3ull, 10ull);
    return 0;
}
