/*
 * CPU oracle for the per-step token-routing path of Cobalt (co-activation-aware MoE training).
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain, single-threaded statement of what
 * the path computes, written from the paper's definitions.  It shares no code, header, table
 * or helper with the CUDA library and must never be linked into or called from the product
 * path; only the test-suite, the smoke check and the bench's CPU-baseline leg use it.
 *
 * Every function cites the passage it follows.  Where the paper leaves a choice open (the
 * bit <-> node map of RemoteMask, how "random" picks are drawn, the order inside R_{e,n}),
 * the reading taken is stated at the function.  Build: gcc -O2 -ffp-contract=off -std=c11.
 *
 * Parity pins (tests, CPU only): Fig. 1 worked example, Eq. 1 by exhaustive enumeration,
 * indicator-matrix product for the statistics, library stable sort for the permutation,
 * closed forms for the combine.  "parity unpinned": the *magnitude* of the traffic reduction
 * on the synthetic workloads (the paper's 75.74%-99.26% depends on its planner and models).
 *
 * Symbols follow Table 1: E experts, K per token, G ranks on N nodes (Q = G/N per node),
 * T tokens, D_t selected experts, s_t source rank, P_r experts on rank r, r_te assigned rank.
 * A layout is slot_expert[G*S]: global slot d = r*S + j of rank r holds that expert id, or -1.
 * r_te is reported as the global slot id (rank = d / S, node = d / (S*Q)).
 */
#include <stddef.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORACLE_OK 0
#define ORACLE_ERR_LAYOUT (-1)   /* violates Eq. 2's first constraint, or an expert twice on a rank */
#define ORACLE_ERR_INPUT (-2)    /* id out of range, duplicate id in a token, bad source rank ... */
#define ORACLE_ERR_ALLOC (-3)

/* ------------------------------------------------------------------------------------------
 * Counter hash used wherever Algorithm 1 says "random" (RandomNode, UniformChoice).
 * The paper fixes only the distribution (uniform); to make both implementations reproducible
 * the draw is a pure function of (seed, token, expert, stream): stream 0 = node pick,
 * stream 1 = replica pick.  All arithmetic is modulo 2^32.
 * ---------------------------------------------------------------------------------------- */
uint32_t oracle_hash(uint64_t seed, uint32_t t, uint32_t e, uint32_t stream)
{
    uint32_t seed_lo = (uint32_t)(seed & 0xFFFFFFFFu);
    uint32_t seed_hi = (uint32_t)(seed >> 32);
    uint32_t x = seed_lo ^ 0x6A09E667u;
    x = (x ^ t) * 0x9E3779B9u;
    x ^= x >> 16;
    x = (x ^ seed_hi) * 0xBB67AE85u;
    x ^= x >> 15;
    x = (x ^ (2u * e + stream)) * 0x9E3779B9u;
    x ^= x >> 16;
    x = x * 0xBB67AE85u;
    x ^= x >> 15;
    x = x * 0x6A09E667u;
    x ^= x >> 16;
    return x;
}

/* index in [0, n) from a hash value: floor(x * n / 2^32) */
uint32_t oracle_hash_index(uint32_t x, uint32_t n)
{
    return (uint32_t)(((uint64_t)x * (uint64_t)n) >> 32);
}

static int popcount32(uint32_t v)
{
    int c = 0;
    while (v) { c += (int)(v & 1u); v >>= 1; }
    return c;
}

/* ------------------------------------------------------------------------------------------
 * Layout tables (Section 3.3, Step 1): R_{e,n} = ranks of node n holding e, N_e = nodes
 * holding e.  Here R is kept as global slot ids in ascending order (an expert sits at most
 * once on a rank, so this is also ascending rank order).
 *   nodes_mask[e]        bit n set  <=>  n in N_e
 *   r_count[e*N + n]     |R_{e,n}|
 *   r_list[(e*N+n)*Q+i]  i-th slot of R_{e,n}
 *   primary[e]           primary_in[e] if given (must hold e), else the lowest slot holding e
 * Rejected (Eq. 2, first constraint; Section 3.2 Stage 2 "two replicas of the same expert
 * cannot reside on one rank"): an expert without replica, an expert twice on a rank, an id
 * outside [-1, E).
 * ---------------------------------------------------------------------------------------- */
int oracle_layout_tables(int32_t N, int32_t Q, int32_t S, int32_t E,
                         const int32_t* slot_expert, const int32_t* primary_in,
                         uint32_t* nodes_mask, int32_t* r_count, int32_t* r_list, int32_t* primary)
{
    if (N < 1 || N > 32 || Q < 1 || S < 1 || E < 1) return ORACLE_ERR_LAYOUT;
    int32_t G = N * Q;
    for (int32_t e = 0; e < E; ++e) { nodes_mask[e] = 0; primary[e] = -1; }
    for (int64_t i = 0; i < (int64_t)E * N; ++i) r_count[i] = 0;
    for (int64_t i = 0; i < (int64_t)E * N * Q; ++i) r_list[i] = -1;
    for (int32_t r = 0; r < G; ++r) {
        int32_t n = r / Q;
        for (int32_t j = 0; j < S; ++j) {
            int32_t d = r * S + j;
            int32_t e = slot_expert[d];
            if (e == -1) continue;
            if (e < 0 || e >= E) return ORACLE_ERR_LAYOUT;
            for (int32_t j2 = 0; j2 < j; ++j2)
                if (slot_expert[r * S + j2] == e) return ORACLE_ERR_LAYOUT;
            int64_t en = (int64_t)e * N + n;
            r_list[en * Q + r_count[en]] = d;
            r_count[en] += 1;
            nodes_mask[e] |= (1u << n);
            if (primary[e] < 0) primary[e] = d;
        }
    }
    for (int32_t e = 0; e < E; ++e) {
        if (nodes_mask[e] == 0) return ORACLE_ERR_LAYOUT;
        if (primary_in) {
            int32_t d = primary_in[e];
            if (d < 0 || d >= G * S || slot_expert[d] != e) return ORACLE_ERR_LAYOUT;
            primary[e] = d;
        }
    }
    return ORACLE_OK;
}

/* ------------------------------------------------------------------------------------------
 * Per-step raw statistics (Section 3.2, Stage 1): load[e] = number of tasks of expert e
 * (tokens selecting e); coact[i][j] = number of tokens selecting both i and j.  The diagonal
 * "both i and i" is the load.  The EMAs w^_e, c^_ij are taken over these per-step counts.
 * Overwrites its outputs.
 * ---------------------------------------------------------------------------------------- */
int oracle_coact_stats(const int32_t* topk_ids, int64_t T, int32_t K, int32_t E,
                       uint32_t* coact, uint32_t* load)
{
    memset(coact, 0, sizeof(uint32_t) * (size_t)E * (size_t)E);
    memset(load, 0, sizeof(uint32_t) * (size_t)E);
    for (int64_t t = 0; t < T; ++t) {
        const int32_t* D_t = topk_ids + t * K;
        for (int32_t a = 0; a < K; ++a) {
            if (D_t[a] < 0 || D_t[a] >= E) return ORACLE_ERR_INPUT;
            for (int32_t b = 0; b < a; ++b)
                if (D_t[b] == D_t[a]) return ORACLE_ERR_INPUT;   /* D_t is a set */
        }
        for (int32_t a = 0; a < K; ++a) {
            load[D_t[a]] += 1;
            for (int32_t b = 0; b < K; ++b)
                coact[(size_t)D_t[a] * E + D_t[b]] += 1;
        }
    }
    return ORACLE_OK;
}

/* ------------------------------------------------------------------------------------------
 * Communication-aware task assignment (Section 3.3, Algorithm 1), token by token.
 *
 * Step 1 (node per expert).  Experts with a replica on the source node N(s_t) run there.  The
 * others form U_t; each has a mask m_{t,e} over the N-1 remote nodes that hold it, and the
 * token must reach a set of remote nodes b that meets every mask.  The paper finds the set with
 * the fewest nodes by trying every (N-1)-bit mask.  Readings: bit j of a mask stands for the j-th
 * remote node in ascending node id with the source node skipped; among covers of the minimum
 * size the numerically smallest mask wins (the paper scans masks in ascending order and only
 * replaces its candidate on a strictly smaller node count).  An expert of U_t then picks a node
 * uniformly among the nodes of b* that hold it: the i-th set bit of b* & m_{t,e} counted from
 * bit 0, i = floor(hash(stream 0) * popcount / 2^32).
 * Step 2 (replica inside the node).  Uniform over R_{e,n} in ascending slot order with hash
 * stream 1; the source rank gets no preference inside its node.  The hash key is (token, expert),
 * not the position k.
 *
 * Outputs: assigned_slot[t*K+k] (r_te as global slot id); optional slot_load[d] = w_er
 * (Section 3.1); optional remote_nodes[t] = number of nodes in b* (0 when U_t is empty) = the
 * token's term of Eq. 1; optional totals[0] = V of this assignment, totals[1] = V of the naive rule.
 * flags bit0: use the naive primary-replica rule (every task goes to primary[e]) instead.
 * flags bit1: round-robin replica pick.  Step 1 is unchanged; in Step 2 the tasks of a group
 *   (expert e, node n) are dealt to R_{e,n} in turn: walking the pairs in ascending p = t*K + k,
 *   the j-th task of the group (j from 0) goes to R_{e,n}[j mod |R_{e,n}|].  Where the paper's
 *   uniform pick balances the replicas of a group only on average (Section 3.3, Step 2), this
 *   makes their loads differ by at most one.  Not in the paper; an optional mode of this repository.
 * ---------------------------------------------------------------------------------------- */

/* m_{t,e}: which remote nodes (all nodes but n_s, ascending, bit j = j-th of them) hold an expert
 * whose node set is `held`; 0 if the source node itself holds it (the expert is not in U_t). */
static uint32_t remote_mask(uint32_t held, int32_t n_s, int32_t N)
{
    if (held & (1u << n_s)) return 0u;
    uint32_t m = 0;
    int32_t j = 0;
    for (int32_t n = 0; n < N; ++n) {
        if (n == n_s) continue;
        if (held & (1u << n)) m |= 1u << j;
        ++j;
    }
    return m;
}

/* b*: the smallest set of remote nodes that meets every non-zero mask (a minimum set cover by
 * exhaustive search, sizes in increasing order, masks of one size in ascending value).  The empty
 * set covers an empty U_t; the set of all remote nodes covers anything, so the search ends. */
static uint32_t smallest_cover(const uint32_t* m, int32_t K, int32_t n_remote)
{
    for (int32_t size = 0; size <= n_remote; ++size) {
        for (uint32_t b = 0; b < (1u << n_remote); ++b) {
            if (popcount32(b) != size) continue;
            int covers = 1;
            for (int32_t a = 0; a < K; ++a)
                if (m[a] != 0 && (b & m[a]) == 0) covers = 0;
            if (covers) return b;
        }
    }
    return 0u;   /* not reached */
}

/* Position of the i-th set bit of c, counting set bits from bit 0 (i < popcount(c)). */
static int32_t nth_set_bit(uint32_t c, uint32_t i)
{
    for (int32_t bit = 0; bit < 32; ++bit) {
        if (!(c & (1u << bit))) continue;
        if (i == 0) return bit;
        --i;
    }
    return -1;
}

/* Node id of remote-mask bit j as seen from source node n_s. */
static int32_t remote_node(int32_t j, int32_t n_s) { return j < n_s ? j : j + 1; }

int oracle_assign(int32_t N, int32_t Q, int32_t S, int32_t E,
                  const int32_t* slot_expert, const int32_t* primary_in,
                  const int32_t* topk_ids, const int32_t* src_rank, int64_t T, int32_t K,
                  uint64_t seed, uint32_t flags,
                  int32_t* assigned_slot, uint32_t* slot_load, uint8_t* remote_nodes,
                  uint64_t* totals)
{
    int32_t G = N * Q, D = G * S;
    uint32_t* nodes_mask = (uint32_t*)malloc(sizeof(uint32_t) * (size_t)E);
    int32_t* r_count = (int32_t*)malloc(sizeof(int32_t) * (size_t)E * N);
    int32_t* r_list = (int32_t*)malloc(sizeof(int32_t) * (size_t)E * N * Q);
    int32_t* primary = (int32_t*)malloc(sizeof(int32_t) * (size_t)E);
    uint32_t* m = (uint32_t*)malloc(sizeof(uint32_t) * (size_t)(K > 0 ? K : 1));
    int32_t* n_te = (int32_t*)malloc(sizeof(int32_t) * (size_t)(K > 0 ? K : 1));
    uint32_t* dealt = (uint32_t*)calloc((size_t)E * N, sizeof(uint32_t));   /* tasks seen per (e, n) group */
    int rc = ORACLE_ERR_ALLOC;
    if (!nodes_mask || !r_count || !r_list || !primary || !m || !n_te || !dealt) goto done;
    rc = oracle_layout_tables(N, Q, S, E, slot_expert, primary_in, nodes_mask, r_count, r_list, primary);
    if (rc != ORACLE_OK) goto done;

    if (slot_load) memset(slot_load, 0, sizeof(uint32_t) * (size_t)D);
    uint64_t V = 0, V_naive = 0;

    for (int64_t t = 0; t < T; ++t) {
        const int32_t* D_t = topk_ids + t * K;
        int32_t s_t = src_rank[t];
        if (s_t < 0 || s_t >= G) { rc = ORACLE_ERR_INPUT; goto done; }
        int32_t n_s = s_t / Q;                                  /* N(s_t) */
        for (int32_t a = 0; a < K; ++a) {
            if (D_t[a] < 0 || D_t[a] >= E) { rc = ORACLE_ERR_INPUT; goto done; }
            for (int32_t b = 0; b < a; ++b)
                if (D_t[b] == D_t[a]) { rc = ORACLE_ERR_INPUT; goto done; }
        }

        /* the naive rule's term of Eq. 1: distinct nodes of the primaries, source excluded */
        uint32_t naive_nodes = 0;
        for (int32_t a = 0; a < K; ++a)
            naive_nodes |= 1u << (primary[D_t[a]] / (S * Q));
        naive_nodes &= ~(1u << n_s);
        V_naive += (uint64_t)popcount32(naive_nodes);

        if (flags & 1u) {
            for (int32_t a = 0; a < K; ++a) {
                int32_t d = primary[D_t[a]];
                assigned_slot[t * K + a] = d;
                if (slot_load) slot_load[d] += 1;
            }
            if (remote_nodes) remote_nodes[t] = (uint8_t)popcount32(naive_nodes);
            V += (uint64_t)popcount32(naive_nodes);
            continue;
        }

        /* Step 1: masks of the experts that are not on the source node, the smallest cover b*, and
         * a node for every expert */
        int any_remote = 0;
        for (int32_t a = 0; a < K; ++a) {
            m[a] = remote_mask(nodes_mask[D_t[a]], n_s, N);
            if (m[a] != 0) any_remote = 1;
        }
        uint32_t b_star = smallest_cover(m, K, N - 1);
        for (int32_t a = 0; a < K; ++a) {
            n_te[a] = n_s;
            if (m[a] != 0) {
                uint32_t c = b_star & m[a];
                uint32_t i = oracle_hash_index(oracle_hash(seed, (uint32_t)t, (uint32_t)D_t[a], 0u),
                                               (uint32_t)popcount32(c));
                n_te[a] = remote_node(nth_set_bit(c, i), n_s);
            }
        }

        /* Step 2: a replica of the expert inside its node */
        for (int32_t a = 0; a < K; ++a) {
            int64_t en = (int64_t)D_t[a] * N + n_te[a];
            uint32_t i;
            if (flags & 2u) {
                i = dealt[en] % (uint32_t)r_count[en];
                dealt[en] += 1;
            } else {
                i = oracle_hash_index(oracle_hash(seed, (uint32_t)t, (uint32_t)D_t[a], 1u),
                                      (uint32_t)r_count[en]);
            }
            int32_t d = r_list[en * Q + i];
            assigned_slot[t * K + a] = d;
            if (slot_load) slot_load[d] += 1;
        }

        int32_t cost = any_remote ? popcount32(b_star) : 0;
        if (remote_nodes) remote_nodes[t] = (uint8_t)cost;
        V += (uint64_t)cost;
    }
    if (totals) { totals[0] = V; totals[1] = V_naive; }
    rc = ORACLE_OK;
done:
    free(nodes_mask); free(r_count); free(r_list); free(primary); free(m); free(n_te); free(dealt);
    return rc;
}

/* ------------------------------------------------------------------------------------------
 * Eq. 1 evaluated straight from an assignment: V = sum_t | {N(r_te) : e in D_t} \ {N(s_t)} |.
 * Independent of how the assignment was produced; also checks the third constraint of Eq. 2
 * (the assigned slot holds the task's expert).  per_token (optional) receives each term.
 * ---------------------------------------------------------------------------------------- */
int oracle_traffic(int32_t N, int32_t Q, int32_t S, int32_t E, const int32_t* slot_expert,
                   const int32_t* topk_ids, const int32_t* src_rank, const int32_t* assigned_slot,
                   int64_t T, int32_t K, uint8_t* per_token, uint64_t* V_out)
{
    int32_t D = N * Q * S;
    (void)E;
    uint64_t V = 0;
    for (int64_t t = 0; t < T; ++t) {
        uint32_t dest_nodes = 0;
        for (int32_t k = 0; k < K; ++k) {
            int32_t d = assigned_slot[t * K + k];
            if (d < 0 || d >= D || slot_expert[d] != topk_ids[t * K + k]) return ORACLE_ERR_INPUT;
            dest_nodes |= 1u << (d / (S * Q));
        }
        dest_nodes &= ~(1u << (src_rank[t] / Q));
        int c = popcount32(dest_nodes);
        if (per_token) per_token[t] = (uint8_t)c;
        V += (uint64_t)c;
    }
    *V_out = V;
    return ORACLE_OK;
}

/* ------------------------------------------------------------------------------------------
 * Dispatch-side local permutation (Fig. 1, "Dispatch"; Section 1: tokens are sent to their
 * assigned replicas).  Pairs p = t*K + k are grouped by destination slot; inside one
 * destination they keep ascending p (stable).  Plain definition, one serial pass each:
 *   dest_counts[d]  = #{p : slot_p = d}           (equals w_er of Section 3.1)
 *   dest_offsets    = exclusive scan, length D+1, last entry = P
 *   row_of_pair[p]  = dest_offsets[slot_p] + #{q < p : slot_q = slot_p}
 *   pair_of_row     = inverse permutation
 *   send[row_of_pair[p]] = x[p / K]  (bit copy of the 16-bit elements; skipped if x == NULL)
 * ---------------------------------------------------------------------------------------- */
int oracle_permute(const int32_t* assigned_slot, int64_t T, int32_t K, int32_t D,
                   const uint16_t* x, int32_t H, uint16_t* send,
                   uint32_t* dest_counts, uint32_t* dest_offsets,
                   int32_t* row_of_pair, int32_t* pair_of_row)
{
    int64_t P = T * K;
    memset(dest_counts, 0, sizeof(uint32_t) * (size_t)D);
    for (int64_t p = 0; p < P; ++p) {
        int32_t d = assigned_slot[p];
        if (d < 0 || d >= D) return ORACLE_ERR_INPUT;
        dest_counts[d] += 1;
    }
    dest_offsets[0] = 0;
    for (int32_t d = 0; d < D; ++d) dest_offsets[d + 1] = dest_offsets[d] + dest_counts[d];
    uint32_t* cursor = (uint32_t*)malloc(sizeof(uint32_t) * (size_t)(D > 0 ? D : 1));
    if (!cursor) return ORACLE_ERR_ALLOC;
    memcpy(cursor, dest_offsets, sizeof(uint32_t) * (size_t)D);
    for (int64_t p = 0; p < P; ++p) {
        int32_t d = assigned_slot[p];
        int32_t row = (int32_t)cursor[d];
        cursor[d] += 1;
        row_of_pair[p] = row;
        if (pair_of_row) pair_of_row[row] = (int32_t)p;
        if (x && send)
            memcpy(send + (size_t)row * H, x + (size_t)(p / K) * H, sizeof(uint16_t) * (size_t)H);
    }
    free(cursor);
    return ORACLE_OK;
}

static float f32_from_bf16(uint16_t b)
{
    uint32_t u = (uint32_t)b << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return f;
}

/* ------------------------------------------------------------------------------------------
 * Combine-side inverse permutation and gate-weighted sum (Fig. 1, "Weighted sum"; Section 1:
 * the MoE layer "merges the results from these experts"):
 *   y[t][h] = sum_{k=0..K-1} g[t][k] * out[row_of_pair[t*K+k]][h]
 * accumulated in fp32 in ascending k, product and sum rounded separately; the result is
 * left in fp32 (no final rounding to bf16).  `tokens` (optional, n_tokens entries) restricts
 * the computation to a list of tokens; y then has n_tokens rows in list order.
 * ---------------------------------------------------------------------------------------- */
int oracle_combine(const uint16_t* expert_out, const int32_t* row_of_pair, const float* gate_w,
                   int64_t T, int32_t K, int32_t H, const int64_t* tokens, int64_t n_tokens,
                   float* y)
{
    int64_t n = tokens ? n_tokens : T;
    for (int64_t i = 0; i < n; ++i) {
        int64_t t = tokens ? tokens[i] : i;
        if (t < 0 || t >= T) return ORACLE_ERR_INPUT;
        for (int32_t h = 0; h < H; ++h) {
            float acc = 0.0f;
            for (int32_t k = 0; k < K; ++k) {
                int64_t row = row_of_pair[t * K + k];
                float prod = gate_w[t * K + k] * f32_from_bf16(expert_out[(size_t)row * H + h]);
                acc = acc + prod;
            }
            y[(size_t)i * H + h] = acc;
        }
    }
    return ORACLE_OK;
}

/* ------------------------------------------------------------------------------------------
 * Backward of the two row stages (the method is a training method: Section 1, "MoE training").
 * With rows r(t,k) = row_of_pair[t*K+k], the forward maps are linear:
 *   dispatch  send[r(t,k)] = x[t]                       combine  y[t] = sum_k g[t][k] * out[r(t,k)]
 * so their adjoints are
 *   grad_x[t]        = sum_k grad_send[r(t,k)]           (permute backward)
 *   grad_out[r(t,k)] = g[t][k] * grad_y[t]               (combine backward, data)
 *   grad_g[t][k]     = sum_h grad_y[t][h] * out[r(t,k)][h]   (combine backward, gate weights)
 * Inputs are 16-bit bfloat patterns; results are left in double precision (no rounding), so
 * that tolerances against them measure the CUDA path alone.
 * ---------------------------------------------------------------------------------------- */
int oracle_permute_backward(const uint16_t* grad_send, const int32_t* row_of_pair, int64_t T, int32_t K,
                            int32_t H, double* grad_x)
{
    for (int64_t t = 0; t < T; ++t)
        for (int32_t h = 0; h < H; ++h) {
            double acc = 0.0;
            for (int32_t k = 0; k < K; ++k)
                acc += (double)f32_from_bf16(grad_send[(size_t)row_of_pair[t * K + k] * H + h]);
            grad_x[(size_t)t * H + h] = acc;
        }
    return ORACLE_OK;
}

int oracle_combine_backward(const uint16_t* grad_y, const uint16_t* expert_out, const int32_t* row_of_pair,
                            const float* gate_w, int64_t T, int32_t K, int32_t H, double* grad_out,
                            double* grad_gate_w)
{
    for (int64_t t = 0; t < T; ++t)
        for (int32_t k = 0; k < K; ++k) {
            size_t row = (size_t)row_of_pair[t * K + k];
            double g = (double)gate_w[t * K + k];
            double dot = 0.0;
            for (int32_t h = 0; h < H; ++h) {
                double gy = (double)f32_from_bf16(grad_y[(size_t)t * H + h]);
                grad_out[row * H + h] = g * gy;
                dot += gy * (double)f32_from_bf16(expert_out[row * H + h]);
            }
            grad_gate_w[t * K + k] = dot;
        }
    return ORACLE_OK;
}
