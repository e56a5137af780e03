// Fused index pass: statistics (stage 1), assignment (stage 2) and the per-chunk destination
// histograms of the permutation (first kernel of stage 3) in ONE pass over the top-k ids.
//
// The separate entry points read the ids three times and launch six kernels before the scan;
// for the few megabytes involved those launches, not the bytes, set the time.  Here one
// cluster-launched kernel keeps, per CTA, the co-activation triangle, the layout tables and the
// chunk histograms in shared memory; every thread owns one token per round: it adds the token's
// K(K+1)/2 pairs to the triangle, runs Algorithm 1, stores the K slots and counts them in the
// histogram of its permutation chunk (256 consecutive tokens = 8 warps).  The triangle is then
// merged over the cluster exactly as in the stand-alone statistics kernel; the scan and rank
// kernels of the permutation follow.  Batches of at most 16 chunks run in a second kernel that does
// all of it, scan and rank included, in one cluster (route_small_kernel).  Results are bit-identical
// to the separate calls.
#include <cooperative_groups.h>

#include <algorithm>
#include <map>
#include <mutex>
#include <tuple>
#include <utility>

#include "permute_index.cuh"
#include "token_core.cuh"

namespace cg = cooperative_groups;

namespace cobalt {

constexpr int kRouteThreads = 1024;
constexpr int kRouteChunkTokens = 256;                              // tokens per permutation chunk
constexpr int kRouteChunksPerRound = kRouteThreads / kRouteChunkTokens;
constexpr size_t kRouteMaxSmem = 220 * 1024;

struct RouteSmem {
    size_t tri_words, tab_words, hist_words;
    size_t bytes() const { return (tri_words + tab_words + hist_words) * sizeof(uint32_t); }
};

static RouteSmem route_smem(const LayoutView& lv, bool packed)
{
    RouteSmem r;
    r.tri_words = ((packed ? (tri_entries(lv.E) + 1) / 2 : tri_entries(lv.E)) + 3) / 4 * 4;
    r.tab_words = static_cast<size_t>(lv.words + 3) / 4 * 4;
    r.hist_words = static_cast<size_t>(kRouteChunksPerRound) * lv.D;
    return r;
}

// kPacked: 16-bit counters in the triangle (see the statistics kernel); the launcher allows it only
// while one cluster sees at most 65535 tokens.
template <int KT, bool kPacked>
__global__ void __launch_bounds__(kRouteThreads)
route_fused_kernel(LayoutView lv, const int32_t* __restrict__ topk_ids, const int32_t* __restrict__ src_rank,
                   int32_t src_uniform, int64_t T, int32_t K_rt, uint32_t seed_lo, uint32_t seed_hi,
                   uint32_t* __restrict__ coact, uint32_t* __restrict__ load, int32_t* __restrict__ assigned_slot,
                   uint8_t* __restrict__ remote_nodes, unsigned long long* __restrict__ totals,
                   uint32_t* __restrict__ chunk_ws, int n_chunks, int tri_words, int tab_words,
                   int chunks_per_cta, const unsigned long long* __restrict__ seed_on_device,
                   uint32_t* __restrict__ err_word)
{
    if (seed_on_device) {                               // the seed of this run, not of the capture
        const unsigned long long sd = __ldg(seed_on_device);
        seed_lo = static_cast<uint32_t>(sd);
        seed_hi = static_cast<uint32_t>(sd >> 32);
    }
    extern __shared__ __align__(16) uint32_t smem[];
    uint32_t* tri = smem;
    uint32_t* tab = smem + tri_words;
    uint32_t* chist = tab + tab_words;            // [kRouteChunksPerRound][D]
    __shared__ unsigned long long cta_totals[2];
    constexpr int KMAX = TokenShape<KT>::KMAX;
    const int K = (KT > 0) ? KT : K_rt;
    const int D = lv.D;
    cg::cluster_group cluster = cg::this_cluster();

    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // the scan kernel may be scheduled early
    // a CTA owns chunks_per_cta consecutive chunks of 256 tokens (the batch cut evenly over the grid)
    // and takes them in rounds of up to four, one token per thread
    const int chunk_lo = min(n_chunks, static_cast<int>(blockIdx.x) * chunks_per_cta);
    const int chunk_hi = min(n_chunks, chunk_lo + chunks_per_cta);
    const int n_rounds = (chunk_hi - chunk_lo + kRouteChunksPerRound - 1) / kRouteChunksPerRound;
    // the first round's loads go out before the shared-memory set-up so that the two overlap
    int32_t id[KMAX], out[KMAX];
    int32_t s_t = src_uniform;
    {
        const int64_t t0 = static_cast<int64_t>(chunk_lo) * kRouteChunkTokens + threadIdx.x;
        if (static_cast<int>(threadIdx.x) < (chunk_hi - chunk_lo) * kRouteChunkTokens && t0 < T) {
            load_token_ids<KT>(topk_ids, t0, K, id);
            if (src_rank) s_t = __ldg(src_rank + t0);
        }
    }
    for (int i = threadIdx.x; i < tri_words / 4; i += blockDim.x) reinterpret_cast<uint4*>(tri)[i] = make_uint4(0, 0, 0, 0);
    for (int i = threadIdx.x; i < kRouteChunksPerRound * D; i += blockDim.x) chist[i] = 0;
    if (threadIdx.x < 2) cta_totals[threadIdx.x] = 0;
    const TableView tv = stage_tables(lv, tab);
    __syncthreads();

    uint32_t cost_sum = 0, naive_sum = 0;
    for (int round = 0; round < n_rounds; ++round) {
        const int first_chunk = chunk_lo + round * kRouteChunksPerRound;
        const int chunks_this_round = min(kRouteChunksPerRound, chunk_hi - first_chunk);
        const int64_t t = static_cast<int64_t>(first_chunk) * kRouteChunkTokens + threadIdx.x;
        if (static_cast<int>(threadIdx.x) < chunks_this_round * kRouteChunkTokens && t < T) {
            if (round > 0) {
                load_token_ids<KT>(topk_ids, t, K, id);
                if (src_rank) s_t = __ldg(src_rank + t);
            }
            const uint32_t bad_ids = check_token_ids<KT>(id, K, lv.E);
            uint32_t bad = bad_ids;
            if (s_t < 0 || s_t >= lv.G) bad |= COBALT_DEVERR_BAD_SRC_RANK;
            if (bad) flag_error(err_word, bad);
            // the statistics only need valid ids, as in the stand-alone statistics call
            if (!bad_ids) add_token_to_triangle<KT, kPacked>(tri, id, K);
            uint32_t cost = 0, naive_cost = 0;
            if (bad) {
#pragma unroll
                for (int a = 0; a < KMAX; ++a) out[a] = -1;
            } else {
                assign_token<KT, kAssignSlot>(tv, id, K, s_t, static_cast<uint32_t>(t), seed_lo, seed_hi, out, cost,
                                              naive_cost);
                uint32_t* mine = chist + (threadIdx.x / kRouteChunkTokens) * D;
#pragma unroll
                for (int a = 0; a < KMAX; ++a)
                    if (a < K) atomicAdd(&mine[out[a]], 1u);
            }
            store_token_slots<KT>(assigned_slot + t * K, out, K);
            if (remote_nodes) remote_nodes[t] = static_cast<uint8_t>(cost);
            cost_sum += cost;
            naive_sum += naive_cost;
        }
        __syncthreads();
        // hand this round's chunk histograms to the scan (every chunk row is written, zeros included)
        for (int i = threadIdx.x; i < chunks_this_round * D; i += blockDim.x) {
            const int g = i / D, d = i - g * D;
            chunk_ws[static_cast<size_t>(d) * n_chunks + first_chunk + g] = chist[i];
            chist[i] = 0;
        }
        __syncthreads();
    }

    if (totals) {
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) {
            cost_sum += __shfl_xor_sync(0xFFFFFFFFu, cost_sum, off);
            naive_sum += __shfl_xor_sync(0xFFFFFFFFu, naive_sum, off);
        }
        if ((threadIdx.x & 31) == 0) {
            if (cost_sum) atomicAdd(&cta_totals[0], static_cast<unsigned long long>(cost_sum));
            if (naive_sum) atomicAdd(&cta_totals[1], static_cast<unsigned long long>(naive_sum));
        }
    }
    cluster.sync();            // every triangle of the cluster is complete (also orders cta_totals)
    wait_for_prior_kernel();   // coact / load / totals may still be being cleared by the kernel before this one
    merge_triangle_over_cluster<kPacked>(tri, lv.E, coact, load);
    if (totals && threadIdx.x < 2 && cta_totals[threadIdx.x])
        atomicAdd(&totals[threadIdx.x], cta_totals[threadIdx.x]);
    cluster.sync();            // no CTA may exit while a peer still reads its triangle
}

// ---- batches of at most 16 chunks: everything in ONE kernel, one cluster --------------------------
// Every CTA owns one chunk of 256 tokens.  The per-chunk destination histograms are exchanged through
// distributed shared memory instead of a workspace in global memory, so the scan across chunks and
// the stable rank run in the same kernel (two cluster barriers, no further launches), and with a
// single cluster the statistics can be stored instead of added, so nothing is cleared beforehand.
constexpr int kSmallMaxChunks = 16;
constexpr int kSmallMaxDests = 992;        // one destination per thread in the scan over d; the last warp sums the totals
constexpr int kSmallWarps = kRouteThreads / 32;

struct SmallSmem {
    size_t tri_words, tab_words, dest_words, slot_words, rank_words;
    size_t bytes() const { return (tri_words + tab_words + 2 * dest_words + slot_words + rank_words) * sizeof(uint32_t); }
};

static SmallSmem small_smem(const LayoutView& lv, int K)
{
    SmallSmem r;
    // 16-bit counters (a cluster sees at most 4096 tokens): the merge is bound by the bytes that cross
    // distributed shared memory, and these are half as many
    r.tri_words = ((tri_entries(lv.E) + 1) / 2 + 3) / 4 * 4;
    r.tab_words = static_cast<size_t>(lv.words + 3) / 4 * 4;
    r.dest_words = static_cast<size_t>(lv.D + 3) / 4 * 4;                   // chist, and the totals per destination
    r.slot_words = static_cast<size_t>(kRouteChunkTokens) * K;              // this chunk's slots, in pair order
    r.rank_words = static_cast<size_t>(1 + kSmallWarps) * r.dest_words;     // base[d] and the per-warp counters
    return r;
}

template <int KT, bool kAccumulate>
__global__ void __launch_bounds__(kRouteThreads)
route_small_kernel(LayoutView lv, const int32_t* __restrict__ topk_ids, const int32_t* __restrict__ src_rank,
                   int32_t src_uniform, int64_t T, uint32_t seed_lo, uint32_t seed_hi, uint32_t* __restrict__ coact,
                   uint32_t* __restrict__ load, int32_t* __restrict__ assigned_slot, uint8_t* __restrict__ remote_nodes,
                   unsigned long long* __restrict__ totals, uint32_t* __restrict__ dest_counts,
                   uint32_t* __restrict__ dest_offsets, int32_t* __restrict__ row_of_pair,
                   int32_t* __restrict__ pair_of_row, int tri_words, int tab_words, int dest_words, int key_bits,
                   const unsigned long long* __restrict__ seed_on_device, uint32_t* __restrict__ err_word)
{
    if (seed_on_device) {                               // the seed of this run, not of the capture
        const unsigned long long sd = __ldg(seed_on_device);
        seed_lo = static_cast<uint32_t>(sd);
        seed_hi = static_cast<uint32_t>(sd >> 32);
    }
    extern __shared__ __align__(16) uint32_t smem[];
    uint32_t* tri = smem;
    uint32_t* tab = tri + tri_words;
    uint32_t* chist = tab + tab_words;             // [D] this chunk's pairs per destination
    uint32_t* tot = chist + dest_words;            // [D] all chunks' pairs per destination
    int32_t* slots = reinterpret_cast<int32_t*>(tot + dest_words);      // [256 * K]
    uint32_t* base = reinterpret_cast<uint32_t*>(slots) + kRouteChunkTokens * KT;   // [D]
    uint32_t* wcnt = base + dest_words;            // [kSmallWarps][dest_words]
    __shared__ unsigned long long cta_totals[2];
    __shared__ uint32_t warp_sums[kSmallWarps];
    constexpr int K = KT;
    const int D = lv.D;
    cg::cluster_group cluster = cg::this_cluster();
    const int chunk = static_cast<int>(cluster.block_rank());
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

    // threads 0..255 run Algorithm 1 for the chunk's tokens, threads 256..511 add the same tokens to
    // the triangle: two short instruction chains side by side instead of one long one
    const int64_t t = static_cast<int64_t>(chunk) * kRouteChunkTokens + (tid & (kRouteChunkTokens - 1));
    const bool has_token = tid < kRouteChunkTokens && t < T;
    const bool counts_token = tid >= kRouteChunkTokens && tid < 2 * kRouteChunkTokens && t < T;
    int32_t id[K], out[K];
    int32_t s_t = src_uniform;
    if (has_token || counts_token) {
        load_token_ids<KT>(topk_ids, t, K, id);
        if (has_token && src_rank) s_t = __ldg(src_rank + t);
    }
    for (int i = tid; i < tri_words / 4; i += blockDim.x) reinterpret_cast<uint4*>(tri)[i] = make_uint4(0, 0, 0, 0);
    for (int i = tid; i < dest_words; i += blockDim.x) chist[i] = 0;
    for (int i = tid; i < kSmallWarps * dest_words; i += blockDim.x) wcnt[i] = 0;
    if (tid < 2) cta_totals[tid] = 0;
    const TableView tv = stage_tables(lv, tab);
    __syncthreads();

    uint32_t cost = 0, naive_cost = 0;
    if (has_token) {
        const uint32_t bad_ids = check_token_ids<KT>(id, K, lv.E);
        uint32_t bad = bad_ids;
        if (s_t < 0 || s_t >= lv.G) bad |= COBALT_DEVERR_BAD_SRC_RANK;
        if (bad) flag_error(err_word, bad);
        if (bad) {
#pragma unroll
            for (int a = 0; a < K; ++a) out[a] = -1;
        } else {
            assign_token<KT, kAssignSlot>(tv, id, K, s_t, static_cast<uint32_t>(t), seed_lo, seed_hi, out, cost, naive_cost);
#pragma unroll
            for (int a = 0; a < K; ++a) atomicAdd(&chist[out[a]], 1u);
        }
        store_token_slots<KT>(assigned_slot + t * K, out, K);
#pragma unroll
        for (int a = 0; a < K; ++a) slots[tid * K + a] = out[a];
        if (remote_nodes) remote_nodes[t] = static_cast<uint8_t>(cost);
    } else if (counts_token) {
        // the statistics only need valid ids, as in the stand-alone statistics call
        if (!check_token_ids<KT>(id, K, lv.E)) add_token_to_triangle<KT, true>(tri, id, K);
    }
    if (totals && tid < kRouteChunkTokens) {      // the first eight warps hold the tokens
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) {
            cost += __shfl_xor_sync(0xFFFFFFFFu, cost, off);
            naive_cost += __shfl_xor_sync(0xFFFFFFFFu, naive_cost, off);
        }
        if (lane == 0) {
            if (cost) atomicAdd(&cta_totals[0], static_cast<unsigned long long>(cost));
            if (naive_cost) atomicAdd(&cta_totals[1], static_cast<unsigned long long>(naive_cost));
        }
    }
    cluster.sync();            // every triangle, chunk histogram and cost sum of the cluster is complete

    merge_triangle_over_cluster<true, !kAccumulate>(tri, lv.E, coact, load);
    // scan across chunks, one destination per thread: pairs of lower chunks, and of all chunks
    // (the cluster always has kSmallMaxChunks CTAs: all remote loads are issued before the first is used)
    uint32_t mine_total = 0;
    if (tid < D) {
        uint32_t c[kSmallMaxChunks];
#pragma unroll
        for (int r = 0; r < kSmallMaxChunks; ++r) c[r] = cluster.map_shared_rank(chist, r)[tid];
        uint32_t before = 0;
#pragma unroll
        for (int r = 0; r < kSmallMaxChunks; ++r) {
            if (r < chunk) before += c[r];
            mine_total += c[r];
        }
        base[tid] = before;
        tot[tid] = mine_total;
    } else if (totals && chunk == 0 && tid >= kSmallMaxDests && tid < kSmallMaxDests + 2) {
        const int which = tid - kSmallMaxDests;
        unsigned long long part[kSmallMaxChunks];
#pragma unroll
        for (int r = 0; r < kSmallMaxChunks; ++r) part[r] = cluster.map_shared_rank(cta_totals, r)[which];
        unsigned long long sum = 0;
#pragma unroll
        for (int r = 0; r < kSmallMaxChunks; ++r) sum += part[r];
        totals[which] = sum;
    }
    cluster.sync();            // no CTA may exit, nor may shared memory change, while a peer still reads it
    // exclusive scan of the totals over d (one destination per thread, D <= blockDim.x)
    uint32_t incl = mine_total;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const uint32_t up = __shfl_up_sync(0xFFFFFFFFu, incl, off);
        if (lane >= off) incl += up;
    }
    if (lane == 31) warp_sums[warp] = incl;
    __syncthreads();
    uint32_t offset = incl - mine_total;
    for (int w = 0; w < warp; ++w) offset += warp_sums[w];
    if (tid < D) {
        base[tid] += offset;                    // first row of this chunk inside destination d
        if (chunk == 0) {
            dest_counts[tid] = mine_total;
            dest_offsets[tid] = offset;
            if (tid == D - 1) dest_offsets[D] = offset + mine_total;
        }
    }
    __syncthreads();

    // stable rank of the chunk's pairs: each warp owns 8 K consecutive pairs (at most four 32-pair steps)
    const int n_tok = static_cast<int>(min(static_cast<int64_t>(kRouteChunkTokens),
                                           max(static_cast<int64_t>(0), T - static_cast<int64_t>(chunk) * kRouteChunkTokens)));
    const int n_pairs = n_tok * K;
    constexpr int kSub = kRouteChunkTokens * K / kSmallWarps;
    constexpr int kSteps = (kSub + 31) / 32;
    const int w0 = warp * kSub, w1 = min(n_pairs, w0 + kSub);
    const int64_t p0 = static_cast<int64_t>(chunk) * kRouteChunkTokens * K;
    uint32_t* mine = wcnt + warp * dest_words;
    int32_t dreg[kSteps];
    uint32_t preg[kSteps];
#pragma unroll
    for (int st = 0; st < kSteps; ++st) {
        const int p = w0 + st * 32 + lane;
        const int32_t d = (st * 32 + lane < kSub && p < w1) ? slots[p] : -1;
        const uint32_t key = static_cast<uint32_t>(d < 0 ? D : d);
        uint32_t peers = 0xFFFFFFFFu;
        for (int b = 0; b < key_bits; ++b) {
            const uint32_t bit = (key >> b) & 1u;
            const uint32_t vote = __ballot_sync(0xFFFFFFFFu, bit);
            peers &= bit ? vote : ~vote;
        }
        dreg[st] = d;
        preg[st] = peers;
        if (d >= 0 && (peers >> lane) == 1u) mine[d] += __popc(peers);   // highest lane of the group
        __syncwarp();
    }
    __syncthreads();
    if (tid < D) {                              // per destination: per-warp counts -> starting rows, in warp order
        uint32_t run = base[tid];
#pragma unroll 8
        for (int w = 0; w < kSmallWarps; ++w) {
            const uint32_t c = wcnt[w * dest_words + tid];
            wcnt[w * dest_words + tid] = run;
            run += c;
        }
    }
    __syncthreads();
#pragma unroll
    for (int st = 0; st < kSteps; ++st) {
        const int p = w0 + st * 32 + lane;
        const bool in_range = st * 32 + lane < kSub && p < w1;
        const int32_t d = dreg[st];
        const uint32_t peers = preg[st];
        if (d >= 0) {
            const uint32_t row = mine[d] + __popc(peers & ((1u << lane) - 1u));
            row_of_pair[p0 + p] = static_cast<int32_t>(row);
            if (pair_of_row) pair_of_row[row] = static_cast<int32_t>(p0 + p);
        } else if (in_range) {
            row_of_pair[p0 + p] = -1;
        }
        __syncwarp();
        if (d >= 0 && (peers >> lane) == 1u) mine[d] += __popc(peers);
        __syncwarp();
    }
}

struct RouteLaunch {
    int cluster;
    int ctas;
};

template <int KT, bool kPacked>
static int pick_route_launch(const LayoutView& lv, int64_t T, size_t smem, int n_sm, RouteLaunch* out)
{
    auto kernel = route_fused_kernel<KT, kPacked>;
    static std::mutex cache_lock;
    static std::map<std::tuple<int, int, int, int64_t>, RouteLaunch> cache;
    int dev = 0;
    COBALT_CUDA_TRY(cudaGetDevice(&dev));
    int64_t want = (T + kRouteChunkTokens - 1) / kRouteChunkTokens;   // one chunk per CTA while CTAs last
    if (want < 16) want = 16;      // a full cluster at least: CTAs without tokens still share the merge
    if (want > n_sm) want = n_sm;
    const auto key = std::make_tuple(dev, static_cast<int>(smem), lv.D, want);
    {
        std::lock_guard<std::mutex> guard(cache_lock);
        auto it = cache.find(key);
        if (it != cache.end()) {
            *out = it->second;
            return COBALT_OK;
        }
    }
    int rc_attr = ensure_kernel_attributes(reinterpret_cast<const void*>(kernel), smem, true);
    if (rc_attr != COBALT_OK) return rc_attr;
    cudaLaunchConfig_t cfg = {};
    cudaLaunchAttribute attr[1];
    cfg.blockDim = dim3(kRouteThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    int cand_cs[5], cand_cta[5], n_cand = 0, most = 0;
    for (int cs = 16; cs >= 1; cs >>= 1) {
        if (cs > want) continue;
        attr[0].val.clusterDim.x = cs;
        cfg.gridDim = dim3(cs);
        int max_clusters = 0;
        if (cudaOccupancyMaxActiveClusters(&max_clusters, kernel, &cfg) != cudaSuccess) {
            (void)cudaGetLastError();
            continue;
        }
        int n_cta = static_cast<int>(want) / cs * cs;
        if (n_cta > max_clusters * cs) n_cta = max_clusters * cs;
        if (n_cta < cs) continue;
        cand_cs[n_cand] = cs;
        cand_cta[n_cand] = n_cta;
        ++n_cand;
        if (n_cta > most) most = n_cta;
    }
    RouteLaunch best = {0, 0};
    for (int i = 0; i < n_cand; ++i) {
        if (cand_cta[i] * 4 >= most * 3) {
            best.cluster = cand_cs[i];
            best.ctas = cand_cta[i];
            break;
        }
    }
    if (best.cluster == 0) return COBALT_ERR_UNSUPPORTED;
    {
        std::lock_guard<std::mutex> guard(cache_lock);
        cache[key] = best;
    }
    *out = best;
    return COBALT_OK;
}

struct RouteArgs {
    const LayoutView* lv;
    const int32_t* ids;
    const int32_t* src;
    int32_t src_uniform;
    int64_t T;
    int32_t K;
    uint64_t seed;
    const unsigned long long* seed_on_device;
    uint32_t* coact;
    uint32_t* load;
    int32_t* assigned_slot;
    uint8_t* remote_nodes;
    uint64_t* totals;
    uint32_t* chunk_ws;
    int n_chunks;
    uint32_t* err_word;
    ZeroList zero;
    int n_sm;
    cudaStream_t stream;
};

// *launched stays false (and nothing has been enqueued) when 16-bit counters would be needed but one
// cluster would see more than 65535 tokens: the caller then takes the separate calls.
template <int KT, bool kPacked>
static int launch_route(const RouteArgs& a, bool* launched)
{
    *launched = false;
    const LayoutView& lv = *a.lv;
    const RouteSmem sm = route_smem(lv, kPacked);
    RouteLaunch how;
    int rc = pick_route_launch<KT, kPacked>(lv, a.T, sm.bytes(), a.n_sm, &how);
    if (rc != COBALT_OK) return rc;
    const int chunks_per_cta = (a.n_chunks + how.ctas - 1) / how.ctas;
    if (kPacked && static_cast<int64_t>(chunks_per_cta) * kRouteChunkTokens * how.cluster > 65535) return COBALT_OK;
    bool after_zeroing = false;
    rc = launch_zero_list(a.zero, a.stream, &after_zeroing);
    if (rc != COBALT_OK) return rc;
    auto kernel = route_fused_kernel<KT, kPacked>;
    rc = ensure_kernel_attributes(reinterpret_cast<const void*>(kernel), sm.bytes(), true);
    if (rc != COBALT_OK) return rc;
    cudaLaunchConfig_t cfg = {};
    cudaLaunchAttribute attr[2];
    cfg.blockDim = dim3(kRouteThreads);
    cfg.gridDim = dim3(static_cast<unsigned>(how.ctas));
    cfg.dynamicSmemBytes = sm.bytes();
    cfg.stream = a.stream;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = how.cluster;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    set_programmatic_launch(&attr[1], after_zeroing);
    COBALT_CUDA_TRY(cudaLaunchKernelEx(&cfg, kernel, lv, a.ids, a.src, a.src_uniform, a.T, a.K,
                                       static_cast<uint32_t>(a.seed & 0xFFFFFFFFu),
                                       static_cast<uint32_t>(a.seed >> 32), a.coact, a.load, a.assigned_slot,
                                       a.remote_nodes, reinterpret_cast<unsigned long long*>(a.totals), a.chunk_ws,
                                       a.n_chunks, static_cast<int>(sm.tri_words), static_cast<int>(sm.tab_words),
                                       chunks_per_cta, a.seed_on_device, a.err_word));
    *launched = true;
    return COBALT_OK;
}

struct SmallArgs {
    uint32_t* dest_counts;
    uint32_t* dest_offsets;
    int32_t* row_of_pair;
    int32_t* pair_of_row;
    bool accumulate;
};

// *launched stays false (nothing enqueued) when the batch, the layout or the device does not qualify.
template <int KT>
static int launch_route_small(const RouteArgs& a, const SmallArgs& b, bool* launched)
{
    *launched = false;
    const LayoutView& lv = *a.lv;
    if (a.T < 1 || a.n_chunks > kSmallMaxChunks || lv.D > kSmallMaxDests) return COBALT_OK;
    const SmallSmem sm = small_smem(lv, KT);
    if (sm.bytes() > kRouteMaxSmem) return COBALT_OK;
    // always a full cluster: CTAs without tokens still take their share of the clearing and the merge
    const int cluster = kSmallMaxChunks;
    using Kernel = void (*)(LayoutView, const int32_t*, const int32_t*, int32_t, int64_t, uint32_t, uint32_t, uint32_t*,
                            uint32_t*, int32_t*, uint8_t*, unsigned long long*, uint32_t*, uint32_t*, int32_t*, int32_t*,
                            int, int, int, int, const unsigned long long*, uint32_t*);
    Kernel kernel = b.accumulate ? route_small_kernel<KT, true> : route_small_kernel<KT, false>;
    int rc = ensure_kernel_attributes(reinterpret_cast<const void*>(kernel), sm.bytes(), true);
    if (rc != COBALT_OK) return rc;
    cudaLaunchConfig_t cfg = {};
    cudaLaunchAttribute attr[1];
    cfg.blockDim = dim3(kRouteThreads);
    cfg.gridDim = dim3(static_cast<unsigned>(cluster));
    cfg.dynamicSmemBytes = sm.bytes();
    cfg.stream = a.stream;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = cluster;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    {   // can the device hold one such cluster at all?  asked once per (device, kernel, cluster, bytes)
        static std::mutex lock;
        static std::map<std::tuple<int, const void*, int, size_t>, bool> fits;
        int dev = 0;
        COBALT_CUDA_TRY(cudaGetDevice(&dev));
        const auto key = std::make_tuple(dev, reinterpret_cast<const void*>(kernel), cluster, sm.bytes());
        bool known = false, ok = false;
        {
            std::lock_guard<std::mutex> guard(lock);
            auto it = fits.find(key);
            if (it != fits.end()) { known = true; ok = it->second; }
        }
        if (!known) {
            int max_clusters = 0;
            if (cudaOccupancyMaxActiveClusters(&max_clusters, kernel, &cfg) != cudaSuccess) {
                (void)cudaGetLastError();
                max_clusters = 0;
            }
            ok = max_clusters >= 1;
            std::lock_guard<std::mutex> guard(lock);
            fits[key] = ok;
        }
        if (!ok) return COBALT_OK;
    }
    int key_bits = 1;
    while ((1 << key_bits) <= lv.D) ++key_bits;          // keys 0..D
    COBALT_CUDA_TRY(cudaLaunchKernelEx(&cfg, kernel, lv, a.ids, a.src, a.src_uniform, a.T,
                                       static_cast<uint32_t>(a.seed & 0xFFFFFFFFu), static_cast<uint32_t>(a.seed >> 32),
                                       a.coact, a.load, a.assigned_slot, a.remote_nodes,
                                       reinterpret_cast<unsigned long long*>(a.totals), b.dest_counts, b.dest_offsets,
                                       b.row_of_pair, b.pair_of_row, static_cast<int>(sm.tri_words),
                                       static_cast<int>(sm.tab_words), static_cast<int>(sm.dest_words), key_bits,
                                       a.seed_on_device, a.err_word));
    *launched = true;
    return COBALT_OK;
}

template <int KT>
static int launch_route_any(const RouteArgs& a, bool packed, bool* launched)
{
    return packed ? launch_route<KT, true>(a, launched) : launch_route<KT, false>(a, launched);
}

static ChunkPlan route_chunks(int64_t T, int32_t K)
{
    ChunkPlan c;
    c.P = T * K;
    c.chunk = kRouteChunkTokens * K;
    c.n_chunks = static_cast<int>((T + kRouteChunkTokens - 1) / kRouteChunkTokens);
    if (c.n_chunks < 1) c.n_chunks = 1;
    return c;
}

// 0: the triangle does not fit beside the tables, 1: it fits with 32-bit counters, 2: with 16-bit ones
static int fused_mode(const LayoutView& lv, uint32_t tile_flags)
{
    // from about 180 experts on the 16-bit triangle is taken even where the 32-bit one fits: the merge
    // is bound by the bytes that cross distributed shared memory
    const bool large_tile = tri_entries(lv.E) * sizeof(uint32_t) >= 64 * 1024;
    if (large_tile && !(tile_flags & COBALT_STATS_TILE32) && route_smem(lv, true).bytes() <= kRouteMaxSmem) return 2;
    if (route_smem(lv, false).bytes() <= kRouteMaxSmem) return 1;
    if (route_smem(lv, true).bytes() <= kRouteMaxSmem) return 2;
    return 0;
}

}  // namespace cobalt

using namespace cobalt;

extern "C" {

size_t cobalt_route_index_workspace_bytes(const cobalt_layout_t* layout, int64_t T, int32_t K)
{
    if (!layout || T < 0 || K < 1 || K > COBALT_MAX_TOPK || T * static_cast<int64_t>(K) >= (1ll << 31)) return 0;
    const LayoutView& lv = layout->view;
    const int mode = fused_mode(lv, 0);
    if (mode == 0 || T == 0) return cobalt_permute_workspace_bytes(T, K, lv.D);
    const ChunkPlan c = route_chunks(T, K);
    const size_t fused = round_up(sizeof(uint32_t) * static_cast<size_t>(lv.D) * c.n_chunks, 256);
    // the call may still take the separate calls (K without a compiled variant, 16-bit counters not
    // allowed for this T): room for them as well
    return std::max(fused, cobalt_permute_workspace_bytes(T, K, lv.D));
}

int cobalt_route_index(const cobalt_layout_t* layout, const int32_t* topk_ids, const int32_t* src_rank,
                       int32_t src_rank_uniform, int64_t T, int32_t K, uint64_t seed, uint32_t* coact,
                       uint32_t* load, int32_t* assigned_slot, uint8_t* remote_nodes, uint64_t* totals,
                       uint32_t* dest_counts, uint32_t* dest_offsets, int32_t* row_of_pair,
                       int32_t* pair_of_row, uint32_t flags, void* workspace, size_t workspace_bytes,
                       cobalt_stream_t stream)
{
    if (!layout || T < 0 || K < 1 || !coact || !load || !dest_counts || !dest_offsets) return COBALT_ERR_INVALID_ARG;
    if (K > COBALT_MAX_TOPK || T * static_cast<int64_t>(K) >= (1ll << 31)) return COBALT_ERR_UNSUPPORTED;
    const LayoutView& lv = layout->view;
    if (K > lv.E) return COBALT_ERR_INVALID_ARG;
    if (!src_rank && (src_rank_uniform < 0 || src_rank_uniform >= lv.G)) return COBALT_ERR_INVALID_ARG;
    if (T > 0 && (!topk_ids || !assigned_slot || !row_of_pair)) return COBALT_ERR_INVALID_ARG;
    if (!aligned16(topk_ids) || !aligned16(src_rank) || !aligned16(coact) || !aligned16(load) ||
        !aligned16(assigned_slot) || !aligned16(totals) || !aligned16(dest_counts) || !aligned16(dest_offsets) ||
        !aligned16(row_of_pair) || !aligned16(pair_of_row) || !aligned16(workspace))
        return COBALT_ERR_INVALID_ARG;
    if (flags & ~(COBALT_STATS_ACCUMULATE | COBALT_SEED_ON_DEVICE | COBALT_STATS_TILE32 | COBALT_ROUTE_GENERAL_KERNELS))
        return COBALT_ERR_INVALID_ARG;
    const bool seed_on_device = (flags & COBALT_SEED_ON_DEVICE) != 0;
    if (seed_on_device && (seed == 0 || (seed & 7u) != 0)) return COBALT_ERR_INVALID_ARG;
    const size_t need = cobalt_route_index_workspace_bytes(layout, T, K);
    if (!workspace || workspace_bytes < need) return COBALT_ERR_WORKSPACE_TOO_SMALL;
    int dev = 0;
    COBALT_CUDA_TRY(cudaGetDevice(&dev));
    if (dev != layout->device) return COBALT_ERR_INVALID_ARG;

    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const int mode = fused_mode(lv, flags & COBALT_STATS_TILE32);
    bool launched = false;
    const ChunkPlan c = route_chunks(T, K);
    // The kernel is compiled for K = 1, 2, 4, 6, 8, 10, 12, 16 with the K ids of a token in registers; its variant
    // for any other K (loops to 16, spills) measured slower than the separate calls (K = 10: 85 us
    // against 58 us at T = 65536, E = 256), so those take the separate calls.
    const bool k_compiled = K == 1 || K == 2 || K == 4 || K == 6 || K == 8 || K == 10 || K == 12 || K == 16;
    if (mode != 0 && T > 0 && k_compiled) {
        RouteArgs a;
        a.zero = ZeroList{{nullptr, nullptr, reinterpret_cast<uint32_t*>(totals), nullptr}, {0, 0, 4, 0}};
        if (!(flags & COBALT_STATS_ACCUMULATE)) {
            a.zero.ptr[0] = coact; a.zero.n[0] = lv.E * lv.E;
            a.zero.ptr[1] = load;  a.zero.n[1] = lv.E;
        }
        a.lv = &lv; a.ids = topk_ids; a.src = src_rank; a.src_uniform = src_rank_uniform; a.T = T; a.K = K;
        a.seed = seed_on_device ? 0 : seed;
        a.seed_on_device = seed_on_device ? reinterpret_cast<const unsigned long long*>(static_cast<uintptr_t>(seed)) : nullptr;
        a.coact = coact; a.load = load; a.assigned_slot = assigned_slot; a.remote_nodes = remote_nodes; a.totals = totals;
        a.chunk_ws = static_cast<uint32_t*>(workspace); a.n_chunks = c.n_chunks; a.stream = s;
        int rc = device_error_word(&a.err_word);
        if (rc != COBALT_OK) return rc;
        rc = sm_count(&a.n_sm);
        if (rc != COBALT_OK) return rc;
        if (!(flags & COBALT_ROUTE_GENERAL_KERNELS) && K <= 8) {
            const SmallArgs b = {dest_counts, dest_offsets, row_of_pair, pair_of_row, (flags & COBALT_STATS_ACCUMULATE) != 0};
            bool small = false;
            switch (K) {
                case 1: rc = launch_route_small<1>(a, b, &small); break;
                case 2: rc = launch_route_small<2>(a, b, &small); break;
                case 4: rc = launch_route_small<4>(a, b, &small); break;
                case 6: rc = launch_route_small<6>(a, b, &small); break;
                default: rc = launch_route_small<8>(a, b, &small);
            }
            if (rc != COBALT_OK || small) return rc;     // the single kernel has done everything
        }
        auto launch_general = [&](bool packed) {
            switch (K) {
                case 1: return launch_route_any<1>(a, packed, &launched);
                case 2: return launch_route_any<2>(a, packed, &launched);
                case 4: return launch_route_any<4>(a, packed, &launched);
                case 6: return launch_route_any<6>(a, packed, &launched);
                case 8: return launch_route_any<8>(a, packed, &launched);
                case 10: return launch_route_any<10>(a, packed, &launched);
                case 12: return launch_route_any<12>(a, packed, &launched);
                case 16: return launch_route_any<16>(a, packed, &launched);
                default: return static_cast<int>(COBALT_ERR_UNSUPPORTED);
            }
        };
        rc = launch_general(mode == 2);
        // 16-bit counters refused for this many tokens: the 32-bit triangle, if it fits
        if (rc == COBALT_OK && !launched && mode == 2 && route_smem(lv, false).bytes() <= kRouteMaxSmem)
            rc = launch_general(false);
        if (rc != COBALT_OK) return rc;
    }
    if (!launched) {
        // the co-activation triangle does not fit beside the tables (or there is nothing to route):
        // same results from the separate calls
        int rc = cobalt_coact_stats(topk_ids, T, K, lv.E, coact, load, flags & COBALT_STATS_ACCUMULATE, nullptr, 0, stream);
        if (rc != COBALT_OK) return rc;
        rc = cobalt_assign(layout, topk_ids, src_rank, src_rank_uniform, T, K, seed, assigned_slot, nullptr,
                           remote_nodes, totals, flags & COBALT_SEED_ON_DEVICE, nullptr, 0, stream);
        if (rc != COBALT_OK) return rc;
        return cobalt_permute_index(assigned_slot, T, K, lv.D, dest_counts, dest_offsets, row_of_pair, pair_of_row,
                                    workspace, workspace_bytes, stream);
    }
    return launch_scan_and_rank(assigned_slot, T * K, lv.D, c, static_cast<uint32_t*>(workspace), dest_counts, dest_offsets,
                                row_of_pair, pair_of_row, 0, s);
}

}  // extern "C"
