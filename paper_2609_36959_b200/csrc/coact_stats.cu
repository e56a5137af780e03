// Stage 1: per-step co-activation counts and expert loads (Section 3.2, Stage 1).
//
// coact[i][j] = #tokens selecting both i and j is symmetric with the load on its diagonal,
// so each CTA histograms only the lower triangle (hi >= lo) of its tokens into a private
// shared-memory tile: K(K+1)/2 shared-memory integer adds per token.  CTAs are grouped in
// thread-block clusters; after a cluster barrier each CTA sums its share of the tile rows over
// all CTAs of the cluster through distributed shared memory and merges the result into global
// memory with integer reductions, mirroring (hi, lo) to (lo, hi) and writing the diagonal to
// `load` as well.  Only integer adds are used, so the result is independent of scheduling.
// Expert counts whose triangle does not fit in one CTA's shared memory take 16-bit counters, two per
// word (E <= 452, while a cluster sees at most 65535 tokens); beyond that the triangle is split
// over 2 to 8 CTAs that are fed the same tokens; few tokens over a large matrix go straight to
// global memory.
#include <cooperative_groups.h>

#include <algorithm>
#include <map>
#include <mutex>
#include <tuple>
#include <utility>

#include "token_core.cuh"

namespace cg = cooperative_groups;

namespace cobalt {

constexpr int kStatsThreads = 1024;
constexpr size_t kStatsMaxTileBytes = 200 * 1024;

// kPacked: 16-bit counters, two per word.  The launcher selects it only when one CLUSTER sees at
// most 65535 tokens, so that neither a tile nor the sum of a cluster's tiles can overflow a half.
// kSplit (E > 452): the triangle is cut into `parts` runs of part_entries flat entries; `parts`
// consecutive CTAs form a group that is fed the same tokens, each CTA adding only the pairs that
// fall into its own run.  All adds stay in the CTA's own shared memory.
// kStore: the grid is a single cluster and the outputs are overwritten: the merge stores every entry
// instead of adding to cleared outputs, and no clearing kernel runs before this one.
template <int KT, bool kPacked, bool kSplit, bool kStore>
__global__ void __launch_bounds__(kStatsThreads)
coact_tile_kernel(const int32_t* __restrict__ topk_ids, int64_t T, int K_rt, int E, int tokens_per_cta, int parts,
                  int part_entries, uint32_t* __restrict__ coact, uint32_t* __restrict__ load,
                  uint32_t* __restrict__ err_word)
{
    extern __shared__ __align__(16) uint32_t tri[];   // lower triangle, padded to whole uint4
    constexpr int KMAX = TokenShape<KT>::KMAX;
    const int K = (KT > 0) ? KT : K_rt;
    cg::cluster_group cluster = cg::this_cluster();

    // A CTA takes tokens_per_cta consecutive tokens (the batch cut evenly over the grid, so that no
    // cluster is left with a second pass over a remainder while the others wait at the barrier).
    // The first token's ids are requested before the tile is cleared so that the two overlap.
    const int64_t group = kSplit ? blockIdx.x / parts : blockIdx.x;     // CTAs of a group share their tokens
    const int first = kSplit ? static_cast<int>(blockIdx.x % parts) * part_entries : 0;
    const int count = kSplit ? min(part_entries, static_cast<int>(tri_entries(E)) - first) : static_cast<int>(tri_entries(E));
    const int64_t t_end = min(T, (group + 1) * tokens_per_cta);
    int64_t t = group * tokens_per_cta + threadIdx.x;
    int32_t id[KMAX];
    if (t < t_end) load_token_ids<KT>(topk_ids, t, K, id);
    const int n_vec = ((kSplit ? part_entries : count) + (kPacked ? 7 : 3)) / (kPacked ? 8 : 4);
    for (int i = threadIdx.x; i < n_vec; i += blockDim.x) reinterpret_cast<uint4*>(tri)[i] = make_uint4(0, 0, 0, 0);
    __syncthreads();

    while (t < t_end) {
        const uint32_t bad = check_token_ids<KT>(id, K, E);
        if (bad) flag_error(err_word, bad);
        else add_token_to_triangle<KT, kPacked, kSplit>(tri, id, K, first, count);
        t += blockDim.x;
        if (t < t_end) load_token_ids<KT>(topk_ids, t, K, id);
    }

    cluster.sync();            // every tile of the cluster is complete
    wait_for_prior_kernel();   // the outputs may still be being cleared by the kernel before this one
    merge_triangle_over_cluster<kPacked, kStore>(tri, E, coact, load, kSplit ? parts : 1, part_entries);
    cluster.sync();            // no CTA may exit while a peer still reads its tile
}

// Every pair straight to global memory: few pairs over a large matrix, and the last resort.
__global__ void __launch_bounds__(256)
coact_global_kernel(const int32_t* __restrict__ topk_ids, int64_t T, int K, int E,
                    uint32_t* __restrict__ coact, uint32_t* __restrict__ load, uint32_t* __restrict__ err_word)
{
    wait_for_prior_kernel();
    const int64_t stride = static_cast<int64_t>(gridDim.x) * blockDim.x;
    for (int64_t t = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x; t < T; t += stride) {
        int32_t id[COBALT_MAX_TOPK];
        load_token_ids<0>(topk_ids, t, K, id);
        const uint32_t bad = check_token_ids<0>(id, K, E);
        if (bad) {
            flag_error(err_word, bad);
            continue;
        }
        for (int a = 0; a < K; ++a) {
            atomicAdd(&load[id[a]], 1u);
            for (int b = 0; b < K; ++b) atomicAdd(&coact[static_cast<size_t>(id[a]) * E + id[b]], 1u);
        }
    }
}

static size_t tile_bytes(int E, bool packed)
{
    return round_up((packed ? (tri_entries(E) + 1) / 2 : tri_entries(E)) * sizeof(uint32_t), 16);
}

// Split tiles (16-bit counters): the fewest parts, a power of two up to 8, whose runs fit one CTA.
static int split_parts(int E, int* part_entries)
{
    for (int parts = 2; parts <= 8; parts *= 2) {
        const size_t per = round_up((tri_entries(E) + parts - 1) / parts, 8);     // whole 16-byte vectors
        if (per * 2 <= kStatsMaxTileBytes) {
            *part_entries = static_cast<int>(per);
            return parts;
        }
    }
    return 0;
}

template <int KT, bool kPacked, bool kSplit>
static int launch_tile(const int32_t* ids, int64_t T, int K, int E, uint32_t* coact, uint32_t* load,
                       uint32_t* err_word, int n_sm, bool clear, cudaStream_t stream, bool* launched)
{
    static_assert(kPacked || !kSplit, "split tiles use 16-bit counters");
    *launched = false;
    auto kernel = coact_tile_kernel<KT, kPacked, kSplit, false>;
    int part_entries = 0;
    const int parts = kSplit ? split_parts(E, &part_entries) : 1;
    if (parts == 0) return COBALT_OK;
    const size_t smem = kSplit ? static_cast<size_t>(part_entries) * 2 : tile_bytes(E, kPacked);
    int rc_attr = ensure_kernel_attributes(reinterpret_cast<const void*>(kernel), smem, true);
    if (rc_attr != COBALT_OK) return rc_attr;

    // never more CTAs than can be co-resident (a second wave of
    // clusters would double the run time), clusters as large as the device schedules well
    // sized for 256 tokens per CTA until the co-resident clusters run out (measured: T = 16384 takes
    // 15.4 us on 64 CTAs, 19.2 us on 16)
    int64_t want = (T + 255) / 256;
    // small batches still get one full cluster: CTAs without tokens take their share of the merge
    // (T = 64 on one CTA: 31 us), at no extra global reductions
    if (want < 16) want = 16;
    want *= parts;                      // `parts` CTAs per group of tokens
    if (want > n_sm) want = n_sm;
    if (want < parts) want = parts;

    cudaLaunchConfig_t cfg = {};
    cudaLaunchAttribute attr[2];
    cfg.blockDim = dim3(kStatsThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;

    // candidates: cluster sizes 16 (non-portable), 8, 4, 2, 1 -> CTAs that can be co-resident
    struct Candidates { int n = 0, cs[5], cta[5]; };
    static std::mutex cache_lock;
    static std::map<std::tuple<int, int, int>, Candidates> cache;   // (dev, E, want); per <KT, kPacked>
    int dev = 0;
    COBALT_CUDA_TRY(cudaGetDevice(&dev));
    const auto key = std::make_tuple(dev, E, static_cast<int>(want));
    Candidates cand;
    bool cached = false;
    {
        std::lock_guard<std::mutex> guard(cache_lock);
        auto it = cache.find(key);
        if (it != cache.end()) {
            cand = it->second;
            cached = true;
        }
    }
    if (!cached) {
        for (int cs = 16; cs >= 1; cs >>= 1) {
            if (cs > want || cs % parts != 0) continue;
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
            cand.cs[cand.n] = cs;
            cand.cta[cand.n] = n_cta;
            ++cand.n;
        }
        std::lock_guard<std::mutex> guard(cache_lock);
        cache[key] = cand;
    }
    // 16-bit tiles: a cluster may see at most 65535 tokens (its CTAs x the tokens of one CTA), which
    // rules out the larger clusters when T is large
    bool legal[5];
    int most = 0;
    auto tokens_per_cta = [T, parts](int n_cta) {      // tokens of one group of `parts` CTAs
        const int groups = n_cta / parts;
        return static_cast<int64_t>(round_up((T + groups - 1) / groups, 32));
    };
    for (int i = 0; i < cand.n; ++i) {
        legal[i] = !kPacked || tokens_per_cta(cand.cta[i]) * (cand.cs[i] / parts) <= 65535;
        if (legal[i] && cand.cta[i] > most) most = cand.cta[i];
    }
    // the largest cluster that keeps at least 3/4 of the best CTA count: the merge (distributed
    // shared memory reads and global reductions, ~10 us of a 23 us kernel at E = 256) shrinks with
    // the number of clusters, the per-token work (~4 us) grows only mildly with fewer CTAs
    int best_cs = 0, best_cta = 0;
    for (int i = 0; i < cand.n; ++i) {
        if (legal[i] && cand.cta[i] * 4 >= most * 3) {
            best_cs = cand.cs[i];
            best_cta = cand.cta[i];
            break;
        }
    }
    if (best_cs == 0) return kPacked ? COBALT_OK : COBALT_ERR_UNSUPPORTED;   // packed: caller takes another kernel
    attr[0].val.clusterDim.x = best_cs;
    cfg.gridDim = dim3(static_cast<unsigned>(best_cta));
    // one cluster in all: it can store its sums, and the outputs need no clearing first
    const bool store = clear && !kSplit && best_cta == best_cs;
    bool after_zeroing = false;
    if (clear && !store) {
        const int rc = launch_zero_words(coact, E * E, load, E, stream, &after_zeroing);
        if (rc != COBALT_OK) return rc;
    }
    if (store) {
        kernel = coact_tile_kernel<KT, kPacked, kSplit, !kSplit>;
        const int rc = ensure_kernel_attributes(reinterpret_cast<const void*>(kernel), smem, true);
        if (rc != COBALT_OK) return rc;
    }
    set_programmatic_launch(&attr[1], after_zeroing);
    cfg.numAttrs = 2;
    COBALT_CUDA_TRY(cudaLaunchKernelEx(&cfg, kernel, ids, T, K, E, static_cast<int>(tokens_per_cta(best_cta)), parts,
                                       part_entries, coact, load, err_word));
    *launched = true;
    return COBALT_OK;
}

// The 16-bit tile when it is allowed and wanted, else the 32-bit tile when it fits, else split
// 16-bit tiles.
template <int KT>
static int launch_tiles(const int32_t* ids, int64_t T, int K, int E, uint32_t* coact, uint32_t* load,
                        uint32_t* err_word, int n_sm, bool clear, uint32_t tile_flags, cudaStream_t stream,
                        bool* launched)
{
    *launched = false;
    const bool fits32 = tile_bytes(E, false) <= kStatsMaxTileBytes;
    const bool fits16 = tile_bytes(E, true) <= kStatsMaxTileBytes;
    // the merge is bound by the bytes that cross distributed shared memory: from about 180 experts on
    // the halved tile wins (E = 256: 19.5 -> 17.4 us), below that the unpacking costs more (E = 64)
    const bool large_tile = tile_bytes(E, false) >= 64 * 1024;
    const bool want16 = (tile_flags & COBALT_STATS_TILE16) != 0 ||
                        (!(tile_flags & COBALT_STATS_TILE32) && (!fits32 || large_tile));
    if (fits16 && want16) {
        const int rc = launch_tile<KT, true, false>(ids, T, K, E, coact, load, err_word, n_sm, clear, stream,
                                                    launched);
        if (rc != COBALT_OK || *launched) return rc;
    }
    if (fits32)
        return launch_tile<KT, false, false>(ids, T, K, E, coact, load, err_word, n_sm, clear, stream, launched);
    return launch_tile<KT, true, true>(ids, T, K, E, coact, load, err_word, n_sm, clear, stream, launched);
}

}  // namespace cobalt

using namespace cobalt;

extern "C" {

size_t cobalt_coact_stats_workspace_bytes(int64_t T, int32_t K, int32_t E)
{
    (void)T; (void)K; (void)E;
    return 0;  // privatised tiles live in shared memory
}

int cobalt_coact_stats(const int32_t* topk_ids, int64_t T, int32_t K, int32_t E, uint32_t* coact,
                       uint32_t* load, uint32_t flags, void* workspace, size_t workspace_bytes,
                       cobalt_stream_t stream)
{
    (void)workspace; (void)workspace_bytes;
    if (T < 0 || K < 1 || E < 1 || !coact || !load) return COBALT_ERR_INVALID_ARG;
    if (K > E) return COBALT_ERR_INVALID_ARG;
    if (K > COBALT_MAX_TOPK || E > COBALT_MAX_EXPERTS || T * static_cast<int64_t>(K) >= (1ll << 31))
        return COBALT_ERR_UNSUPPORTED;
    if (T > 0 && !topk_ids) return COBALT_ERR_INVALID_ARG;
    if (!aligned16(topk_ids) || !aligned16(coact) || !aligned16(load)) return COBALT_ERR_INVALID_ARG;

    if (flags & ~(COBALT_STATS_ACCUMULATE | COBALT_STATS_TILE16 | COBALT_STATS_TILE32)) return COBALT_ERR_INVALID_ARG;
    const uint32_t tile_flags = flags & (COBALT_STATS_TILE16 | COBALT_STATS_TILE32);
    if (tile_flags == (COBALT_STATS_TILE16 | COBALT_STATS_TILE32)) return COBALT_ERR_INVALID_ARG;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    int rc = COBALT_OK;
    const bool clear = !(flags & COBALT_STATS_ACCUMULATE);
    bool after_zeroing = false;
    if (T == 0) return clear ? launch_zero_words(coact, E * E, load, E, s, &after_zeroing) : COBALT_OK;

    uint32_t* err_word = nullptr;
    rc = device_error_word(&err_word);
    if (rc != COBALT_OK) return rc;
    int n_sm = 0;
    rc = sm_count(&n_sm);
    if (rc != COBALT_OK) return rc;

    // Few pairs over a large matrix (the split tiles' merge costs about 20 us + 22 us (E/1024)^2 whatever
    // the batch, a global atomic about 1/45 ns): every pair straight to global memory.
    const bool large = tile_bytes(E, true) > kStatsMaxTileBytes;
    const int64_t adds = T * static_cast<int64_t>(K) * K;
    const bool sparse = large && adds < (2 << 20) && (E > 896 || adds < (300 << 10));
    bool launched = false;
    if (!sparse) {
        switch (K) {
            case 1: rc = launch_tiles<1>(topk_ids, T, K, E, coact, load, err_word, n_sm, clear, tile_flags, s, &launched); break;
            case 2: rc = launch_tiles<2>(topk_ids, T, K, E, coact, load, err_word, n_sm, clear, tile_flags, s, &launched); break;
            case 4: rc = launch_tiles<4>(topk_ids, T, K, E, coact, load, err_word, n_sm, clear, tile_flags, s, &launched); break;
            case 6: rc = launch_tiles<6>(topk_ids, T, K, E, coact, load, err_word, n_sm, clear, tile_flags, s, &launched); break;
            case 8: rc = launch_tiles<8>(topk_ids, T, K, E, coact, load, err_word, n_sm, clear, tile_flags, s, &launched); break;
            case 10: rc = launch_tiles<10>(topk_ids, T, K, E, coact, load, err_word, n_sm, clear, tile_flags, s, &launched); break;
            case 12: rc = launch_tiles<12>(topk_ids, T, K, E, coact, load, err_word, n_sm, clear, tile_flags, s, &launched); break;
            case 16: rc = launch_tiles<16>(topk_ids, T, K, E, coact, load, err_word, n_sm, clear, tile_flags, s, &launched); break;
            default: rc = launch_tiles<0>(topk_ids, T, K, E, coact, load, err_word, n_sm, clear, tile_flags, s, &launched);
        }
        if (rc != COBALT_OK || launched) return rc;
    }
    // also the last resort when no cluster shape can be scheduled
    if (clear) {
        rc = launch_zero_words(coact, E * E, load, E, s, &after_zeroing);
        if (rc != COBALT_OK) return rc;
    }
    int64_t want = (T + 255) / 256;
    const unsigned grid = static_cast<unsigned>(want > 8 * n_sm ? 8 * n_sm : want);
    cudaLaunchConfig_t cfg = {};
    cudaLaunchAttribute attr[1];
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(256);
    cfg.stream = s;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    set_programmatic_launch(&attr[0], after_zeroing);
    COBALT_CUDA_TRY(cudaLaunchKernelEx(&cfg, coact_global_kernel, topk_ids, T, static_cast<int>(K),
                                       static_cast<int>(E), coact, load, err_word));
    return COBALT_OK;
}

}  // extern "C"
