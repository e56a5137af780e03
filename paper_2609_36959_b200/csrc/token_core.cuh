// Per-token device routines shared by the statistics, assignment and fused route kernels:
// loading and checking a token's K expert ids, and Algorithm 1 for one token.
#pragma once

#ifdef __CUDACC__
#include <cooperative_groups.h>
#endif

#include "common.cuh"

namespace cobalt {

#ifdef __CUDACC__

template <int KT>
struct TokenShape {
    static constexpr int KMAX = (KT > 0) ? KT : COBALT_MAX_TOPK;
};

// ids of token t into registers (16/8-byte loads when K allows)
template <int KT>
__device__ __forceinline__ void load_token_ids(const int32_t* __restrict__ ids, int64_t t, int K,
                                               int32_t (&id)[TokenShape<KT>::KMAX])
{
    constexpr int KMAX = TokenShape<KT>::KMAX;
    const int32_t* row = ids + t * K;
    if (KT > 0 && KT % 4 == 0) {
#pragma unroll
        for (int a = 0; a < KT / 4; ++a) {
            const int4 v = __ldg(reinterpret_cast<const int4*>(row) + a);
            id[4 * a] = v.x; id[4 * a + 1] = v.y; id[4 * a + 2] = v.z; id[4 * a + 3] = v.w;
        }
    } else if (KT > 0 && KT % 2 == 0) {
#pragma unroll
        for (int a = 0; a < KT / 2; ++a) {
            const int2 v = __ldg(reinterpret_cast<const int2*>(row) + a);
            id[2 * a] = v.x; id[2 * a + 1] = v.y;
        }
    } else {
#pragma unroll
        for (int a = 0; a < KMAX; ++a)
            if (a < K) id[a] = __ldg(row + a);
    }
}

// COBALT_DEVERR_* bits for ids outside [0, E) or listed twice (D_t must be a set); 0 if fine
template <int KT>
__device__ __forceinline__ uint32_t check_token_ids(const int32_t (&id)[TokenShape<KT>::KMAX], int K, int E)
{
    constexpr int KMAX = TokenShape<KT>::KMAX;
    uint32_t bad = 0;
#pragma unroll
    for (int a = 0; a < KMAX; ++a) {
        if (a < K) {
            if (id[a] < 0 || id[a] >= E) bad |= COBALT_DEVERR_BAD_EXPERT_ID;
#pragma unroll
            for (int b = 0; b < a; ++b)
                if (id[b] == id[a]) bad |= COBALT_DEVERR_DUPLICATE_ID;
        }
    }
    return bad;
}

template <int KT>
__device__ __forceinline__ void store_token_slots(int32_t* __restrict__ dst, const int32_t (&out)[TokenShape<KT>::KMAX],
                                                  int K)
{
    constexpr int KMAX = TokenShape<KT>::KMAX;
    if (KT > 0 && KT % 4 == 0) {
#pragma unroll
        for (int a = 0; a < KT / 4; ++a)
            reinterpret_cast<int4*>(dst)[a] = make_int4(out[4 * a], out[4 * a + 1], out[4 * a + 2], out[4 * a + 3]);
    } else if (KT > 0 && KT % 2 == 0) {
#pragma unroll
        for (int a = 0; a < KT / 2; ++a)
            reinterpret_cast<int2*>(dst)[a] = make_int2(out[2 * a], out[2 * a + 1]);
    } else {
#pragma unroll
        for (int a = 0; a < KMAX; ++a)
            if (a < K) dst[a] = out[a];
    }
}

// The K ids of a token in ascending order (a compare-exchange network, fully unrolled; entries past K
// are padded with a value above every id so that they stay at the end).  K = 8 takes the 19-exchange
// network, the other sizes an odd-even transposition sort.
template <int KT>
__device__ __forceinline__ void sort_token_ids(const int32_t (&id)[TokenShape<KT>::KMAX], int K,
                                               int32_t (&s)[TokenShape<KT>::KMAX])
{
    constexpr int KMAX = TokenShape<KT>::KMAX;
#pragma unroll
    for (int a = 0; a < KMAX; ++a) s[a] = (a < K) ? id[a] : 0x7FFFFFFF;
    auto exchange = [&](int a, int b) {
        const int32_t lo = min(s[a], s[b]), hi = max(s[a], s[b]);
        s[a] = lo;
        s[b] = hi;
    };
    if (KT == 8) {
        constexpr int net[19][2] = {{0, 1}, {2, 3}, {4, 5}, {6, 7}, {0, 2}, {1, 3}, {4, 6}, {5, 7}, {1, 2}, {5, 6},
                                    {0, 4}, {3, 7}, {1, 5}, {2, 6}, {1, 4}, {3, 6}, {2, 4}, {3, 5}, {3, 4}};
#pragma unroll
        for (int i = 0; i < 19; ++i) exchange(net[i][0], net[i][1]);
    } else {
#pragma unroll
        for (int pass = 0; pass < KMAX; ++pass) {
#pragma unroll
            for (int a = pass & 1; a + 1 < KMAX; a += 2) exchange(a, a + 1);
        }
    }
}

// The same checks as check_token_ids on ids that are already sorted: the range is decided by the two
// ends, a repeated id by its neighbour.
template <int KT>
__device__ __forceinline__ uint32_t check_sorted_ids(const int32_t (&s)[TokenShape<KT>::KMAX], int K, int E)
{
    constexpr int KMAX = TokenShape<KT>::KMAX;
    uint32_t bad = 0;
    bool high = false, twice = false;
#pragma unroll
    for (int a = 0; a < KMAX; ++a) {
        if (a < K) {
            high = high || s[a] >= E;
            if (a > 0) twice = twice || s[a] == s[a - 1];
        }
    }
    if (s[0] < 0 || high) bad |= COBALT_DEVERR_BAD_EXPERT_ID;
    if (twice) bad |= COBALT_DEVERR_DUPLICATE_ID;
    return bad;
}

// Layout tables staged in shared memory (see LayoutView for the word layout).
struct TableView {
    const uint32_t* ent;
    const uint32_t* primary;
    const uint32_t* rlist;
    const uint8_t* cover;
    int N, G, E;
    uint32_t q_inverse;
};

__device__ __forceinline__ uint32_t ent_count(uint32_t w) { return w & ((1u << kEntCountBits) - 1u); }
__device__ __forceinline__ uint32_t ent_offset(uint32_t w) { return (w >> kEntCountBits) & ((1u << kEntOffsetBits) - 1u); }
__device__ __forceinline__ uint32_t ent_remote_mask(uint32_t w) { return (w >> kEntMaskShift) & 0x7Fu; }
__device__ __forceinline__ uint32_t ent_primary_node(uint32_t w) { return w >> kEntPrimaryNodeShift; }

// The view of tables that are (or will be) staged at `tab`.
__device__ __forceinline__ TableView table_view(const LayoutView& lv, const uint32_t* tab)
{
    TableView tv;
    tv.ent = tab + lv.ent_off();
    tv.primary = tab + lv.primary_off();
    tv.rlist = tab + lv.rlist_off();
    tv.cover = reinterpret_cast<const uint8_t*>(tab + lv.cover_off());
    tv.N = lv.N; tv.G = lv.G; tv.E = lv.E;
    tv.q_inverse = lv.q_inverse;
    return tv;
}

__device__ __forceinline__ TableView stage_tables(const LayoutView& lv, uint32_t* tab)
{
    // the blob is padded to whole 16-byte vectors
    const uint4* src = reinterpret_cast<const uint4*>(lv.blob);
    uint4* dst = reinterpret_cast<uint4*>(tab);
    const int n_vec = (lv.words + 3) / 4;
#pragma unroll 4
    for (int i = threadIdx.x; i < n_vec; i += blockDim.x) dst[i] = __ldg(src + i);
    return table_view(lv, tab);
}

// What assign_token writes per task.
enum AssignMode {
    kAssignSlot = 0,      // Algorithm 1 with the hashed uniform replica pick (Step 2)
    kAssignNaive = 1,     // every task to its expert's primary replica
    kAssignGroupKey = 2,  // Step 1 only: out = e * N + n_te (the replica is picked later, in task order)
};

// Algorithm 1 for one token (ids already checked, s_t in range).  Writes out[a] for each of the K
// tasks and returns the token's term of Eq. 1 in `cost`, the naive rule's term in `naive_cost`.
template <int KT, int MODE>
__device__ __forceinline__ void assign_token(const TableView& tv, const int32_t (&id)[TokenShape<KT>::KMAX], int K,
                                             int32_t s_t, uint32_t t, uint32_t seed_lo, uint32_t seed_hi,
                                             int32_t (&out)[TokenShape<KT>::KMAX], uint32_t& cost,
                                             uint32_t& naive_cost)
{
    constexpr int KMAX = TokenShape<KT>::KMAX;
    const int N = tv.N;
    const int n_s = static_cast<int>(__umulhi(static_cast<uint32_t>(s_t) << 12, tv.q_inverse));   // N(s_t) = s_t / Q
    const uint32_t src_bit = 1u << n_s;

    // One table word per expert, read for the token's own source node: the remote mask m_{t,e} (0 if
    // the expert is present on the source node, i.e. not in U_t), the replicas on the source node,
    // and the node of the primary replica (for the naive rule's term of Eq. 1).
    uint32_t w[KMAX];
    uint32_t naive_nodes = 0;
#pragma unroll
    for (int a = 0; a < KMAX; ++a) {
        if (a < K) {
            w[a] = tv.ent[id[a] * N + n_s];
            naive_nodes |= 1u << ent_primary_node(w[a]);
        }
    }
    naive_cost = __popc(naive_nodes & ~src_bit);

    if (MODE == kAssignNaive) {
#pragma unroll
        for (int a = 0; a < KMAX; ++a)
            if (a < K) out[a] = static_cast<int32_t>(tv.primary[id[a]]);
        cost = naive_cost;
        return;
    }

    // b*: the fewest remote nodes that meet every mask, the numerically smallest among equals (the
    // outcome of scanning all (N-1)-bit masks in ascending order and replacing the candidate only on
    // a strictly smaller node count).  Up to four nodes a mask is one of seven values, and the answer
    // for every set of values present is looked up in a table built once per layout by that very
    // scan.  Beyond that: a single node covers U_t iff every mask has its bit, and the lowest such
    // bit is the smallest one-bit candidate; only otherwise are the candidates with two or more bits
    // scanned.
    uint32_t b_star = 0;
    if (N <= 4) {
        uint32_t present = 0;
#pragma unroll
        for (int a = 0; a < KMAX; ++a)
            if (a < K) present |= 1u << ent_remote_mask(w[a]);
        b_star = tv.cover[present >> 1];                 // bit 0 (mask 0: a local expert) drops out
    } else {
        uint32_t any_remote = 0, common = 0xFFFFFFFFu;
#pragma unroll
        for (int a = 0; a < KMAX; ++a) {
            if (a < K) {
                const uint32_t m = ent_remote_mask(w[a]);
                any_remote |= m;
                if (m) common &= m;
            }
        }
        if (any_remote) {
            if (common) {
                b_star = common & (0u - common);
            } else {
                const uint32_t full = (1u << (N - 1)) - 1u;
                b_star = full;
                int best = N - 1;
                for (uint32_t b = 3; b < full; ++b) {
                    const int pc = __popc(b);
                    if (pc >= best) continue;
                    bool feasible = true;
#pragma unroll
                    for (int a = 0; a < KMAX; ++a) {
                        if (a < K) {
                            const uint32_t m = ent_remote_mask(w[a]);
                            feasible = feasible && (m == 0 || (b & m) != 0);
                        }
                    }
                    if (feasible) {
                        b_star = b;
                        best = pc;
                        if (pc == 2) break;  // one node is known not to suffice
                    }
                }
            }
        }
    }
    cost = __popc(b_star);

    // Node per expert (Step 1), then a replica inside the node (Step 2).  Written without branches, so
    // that the K experts' chains (table loads, hashes) are independent straight-line code that the
    // scheduler can interleave: a draw among one candidate is floor(x * 1 / 2^32) = 0 whatever x is, and
    // an expert that stays local simply reads its own table word again.
    const bool few_nodes = N <= 4;                       // at most three remote nodes: two bits to drop at most
#pragma unroll
    for (int a = 0; a < KMAX; ++a) {
        if (a < K) {
            const uint32_t m = ent_remote_mask(w[a]);
            // RandomNode: the i-th set bit of b* & m, i uniform over the candidates
            uint32_t c = b_star & m;
            const uint32_t i = hash_index(route_hash(seed_lo, seed_hi, t, id[a], 0u), __popc(c));
            if (few_nodes) {
#pragma unroll
                for (uint32_t j = 0; j < 2; ++j) c = (j < i) ? (c & (c - 1u)) : c;
            } else {
#pragma unroll
                for (uint32_t j = 0; j < COBALT_MAX_NODES - 2; ++j) c = (j < i) ? (c & (c - 1u)) : c;
            }
            const int bit = __ffs(c) - 1;
            const int node = (m != 0) ? bit + (bit >= n_s ? 1 : 0) : n_s;
            if (MODE == kAssignGroupKey) {
                out[a] = id[a] * N + node;
            } else {
                // UniformChoice over R_{e,node}
                const uint32_t e_n = tv.ent[id[a] * N + node];
                const uint32_t r = hash_index(route_hash(seed_lo, seed_hi, t, id[a], 1u), ent_count(e_n));
                out[a] = static_cast<int32_t>(tv.rlist[ent_offset(e_n) + r]);
            }
        }
    }
}

// Adds the K(K+1)/2 unordered pairs of one token (diagonal included) to a lower-triangle tile, from
// ids in ascending order: entry (s[b], s[a]) with a <= b sits at s[b](s[b]+1)/2 + s[a].
template <int KT, bool kPacked>
__device__ __forceinline__ void add_sorted_token_to_triangle(uint32_t* tri, const int32_t (&s)[TokenShape<KT>::KMAX], int K)
{
    constexpr int KMAX = TokenShape<KT>::KMAX;
#pragma unroll
    for (int b = 0; b < KMAX; ++b) {
        if (b < K) {
            const int row = s[b] * (s[b] + 1) / 2;
#pragma unroll
            for (int a = 0; a <= b; ++a) {
                const int idx = row + s[a];
                if (kPacked) atomicAdd(&tri[idx >> 1], (idx & 1) ? 0x10000u : 1u);
                else atomicAdd(&tri[idx], 1u);
            }
        }
    }
}

// Adds the K(K+1)/2 unordered pairs of one token (diagonal included) to a lower-triangle tile.
// kPacked: two 16-bit counters per word (entry idx in the low or high half of word idx / 2); the
// caller guarantees that no counter of the tile, nor its sum over the cluster, reaches 65536.
// kSplit: the tile holds only the entries [first, first + count) of the flat triangle; pairs outside
// are skipped (another CTA, fed the same tokens, holds them).
template <int KT, bool kPacked = false, bool kSplit = false>
__device__ __forceinline__ void add_token_to_triangle(uint32_t* tri, const int32_t (&id)[TokenShape<KT>::KMAX], int K,
                                                      int first = 0, int count = 0)
{
    constexpr int KMAX = TokenShape<KT>::KMAX;
#pragma unroll
    for (int a = 0; a < KMAX; ++a) {
#pragma unroll
        for (int b = a; b < KMAX; ++b) {
            if (b < K) {
                const int hi = max(id[a], id[b]), lo = min(id[a], id[b]);
                int idx = hi * (hi + 1) / 2 + lo;
                if (kSplit) {
                    idx -= first;
                    if (static_cast<unsigned>(idx) >= static_cast<unsigned>(count)) continue;
                }
                if (kPacked) atomicAdd(&tri[idx >> 1], (idx & 1) ? 0x10000u : 1u);
                else atomicAdd(&tri[idx], 1u);
            }
        }
    }
}

__host__ __device__ inline size_t tri_entries(int E) { return static_cast<size_t>(E) * (E + 1) / 2; }

// Row of the lower triangle that holds flat index idx (row hi starts at hi*(hi+1)/2).
__device__ __forceinline__ int tri_row(int idx)
{
    int hi = static_cast<int>((sqrtf(8.0f * static_cast<float>(idx) + 1.0f) - 1.0f) * 0.5f);
    while (hi * (hi + 1) / 2 > idx) --hi;
    while ((hi + 1) * (hi + 2) / 2 <= idx) ++hi;
    return hi;
}

// After a cluster barrier: every CTA owns a contiguous slice of the flat triangle, sums it over
// all tiles of the cluster with 16-byte distributed-shared-memory loads and merges the sums into
// coact and load (the diagonal) with global integer reductions.  Entry (hi, lo) goes out straight
// from the registers, lanes running along lo.  Its mirror (lo, hi) would put the 32 lanes of such a
// reduction on 32 different rows of coact, so the sums are also written back into this CTA's own
// tile (no peer reads that slice) and the mirrors are issued in a second walk whose lanes run along
// hi, i.e. along a row of coact.
// The caller must hold a second cluster barrier before any CTA exits.
// parts > 1: the tiles are split (see add_token_to_triangle); CTA rank r of the cluster holds part
// r mod parts, `part_entries` entries (a multiple of the entries of a 16-byte vector) starting at
// flat entry part * part_entries, and is merged with the cluster's other CTAs of the same part.
// kStore: the grid is this one cluster and the outputs are to be overwritten: every entry (zeros
// included) is stored instead of added, so the outputs need no clearing beforehand.
template <bool kPacked = false, bool kStore = false>
__device__ __forceinline__ void merge_triangle_over_cluster(uint32_t* tri, int E, uint32_t* __restrict__ coact,
                                                            uint32_t* __restrict__ load, int parts = 1,
                                                            int part_entries = 0)
{
    namespace cg = cooperative_groups;
    cg::cluster_group cluster = cg::this_cluster();
    constexpr int kPerWord = kPacked ? 2 : 1;            // triangle entries per 32-bit word
    const int n_tri = static_cast<int>(tri_entries(E));
    const int part = static_cast<int>(cluster.block_rank()) % parts;
    const int entry0 = part * part_entries;              // flat entry held by word 0 of this tile
    const int n_here = parts > 1 ? max(0, min(part_entries, n_tri - entry0)) : n_tri;
    const int n_words = (n_here + kPerWord - 1) / kPerWord;
    const int n_vec = (n_words + 3) / 4;
    const int csize = static_cast<int>(cluster.num_blocks()) / parts;     // CTAs holding this part
    const int crank = static_cast<int>(cluster.block_rank()) / parts;     // this CTA's index among them
    const int per = (n_vec + csize - 1) / csize;
    const int v0 = min(n_vec, crank * per), v1 = min(n_vec, v0 + per);
    for (int v = v0 + threadIdx.x; v < v1; v += blockDim.x) {
        uint4 s = make_uint4(0, 0, 0, 0);
#pragma unroll 4
        for (int i = 0; i < csize; ++i) {
            // every CTA starts at its own tile, so the CTAs of a cluster do not all read one peer at once
            const int r = ((crank + i) % csize) * parts + part;
            const uint4 q = reinterpret_cast<const uint4*>(cluster.map_shared_rank(tri, r))[v];
            s.x += q.x; s.y += q.y; s.z += q.z; s.w += q.w;    // packed halves cannot carry (see above)
        }
        reinterpret_cast<uint4*>(tri)[v] = s;
        const uint32_t word[4] = {s.x, s.y, s.z, s.w};
        const int first = entry0 + 4 * kPerWord * v;             // first triangle entry of this vector
        int hi = tri_row(first);
        int lo = first - hi * (hi + 1) / 2;
#pragma unroll
        for (int c = 0; c < 4 * kPerWord; ++c) {
            const uint32_t val = kPacked ? ((word[c >> 1] >> (16 * (c & 1))) & 0xFFFFu) : word[c];
            if (kStore) {
                if (first + c < n_tri) {
                    coact[static_cast<size_t>(hi) * E + lo] = val;
                    if (lo == hi) load[hi] = val;
                }
            } else if (first + c < n_tri && val) {
                atomicAdd(&coact[static_cast<size_t>(hi) * E + lo], val);
                if (lo == hi) atomicAdd(&load[hi], val);
            }
            if (++lo > hi) { ++hi; lo = 0; }
        }
    }
    __syncthreads();
    // mirrors of the slice [f0, f1): it covers (parts of) rows a..b of the triangle
    const int f0 = entry0 + 4 * kPerWord * v0, f1 = min(entry0 + n_here, entry0 + 4 * kPerWord * v1);
    if (f0 >= f1) return;
    const int a = tri_row(f0), b = tri_row(f1 - 1);
    const int n_rows = b - a + 1;
    const int n_walk = n_rows * b;                       // lo in [0, b), hi in [a, b]
    for (int j = threadIdx.x; j < n_walk; j += blockDim.x) {
        const int lo = j / n_rows;
        const int hi = a + (j - lo * n_rows);
        const int flat = hi * (hi + 1) / 2 + lo;
        if (lo < hi && flat >= f0 && flat < f1) {
            const int at = flat - entry0;
            const uint32_t val = kPacked ? ((tri[at >> 1] >> (16 * (at & 1))) & 0xFFFFu) : tri[at];
            if (kStore) coact[static_cast<size_t>(lo) * E + hi] = val;
            else if (val) atomicAdd(&coact[static_cast<size_t>(lo) * E + hi], val);
        }
    }
}

#else

inline size_t tri_entries(int E) { return static_cast<size_t>(E) * (E + 1) / 2; }

#endif  // __CUDACC__

}  // namespace cobalt
