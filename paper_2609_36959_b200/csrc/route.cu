// Fused index pass: statistics (stage 1), assignment (stage 2) and the index half of the permutation
// (stage 3) in ONE kernel and one pass over the top-k ids.
//
// The separate entry points read the ids three times and launch seven kernels; for the few megabytes
// involved those launches and the dependent-latency chains between them, not the bytes, set the time.
// Here a grid of at most one CTA per SM (1024 threads, launched cooperatively so that all of it is
// resident) does everything:
//
//   phase 1  every CTA owns a contiguous range of tokens, one token per thread and round: the
//            token's K(K+1)/2 pairs go into the CTA's private co-activation triangle in shared
//            memory, Algorithm 1 picks its K slots (stored, and counted per destination).
//   publish  the CTA writes its triangle and its destination counts to the workspace (plain
//            coalesced stores) and adds the counts and its Eq. 1 sums to grid-wide totals there
//            (atomic adds).  Then ONE grid-wide barrier (bounded wait).
//   phase 2  every CTA sums a slice of the triangle over all CTAs' partials and STORES coact / load
//            (no atomics on the outputs, nothing to clear beforehand); it derives, from the totals
//            and from the counts of at most half of the other CTAs, the offsets and the first row
//            of its own tokens inside every destination; and ranks its pairs.  A token sends at most one pair to a destination
//            (its experts, hence its slots, are distinct), so the rows of one destination inside a
//            warp's 32 tokens are ordered by lane: each lane ORs its bit into a per-destination lane
//            mask, and a pair's rank is the popcount of the lower lanes -- no sorting, no position
//            atomics, and the result is the stable order by construction.  The inverse map is
//            staged in shared memory in row order, so that its stores run along rows.
//
// Results are bit-identical to cobalt_coact_stats + cobalt_assign + cobalt_permute_index.
#include <algorithm>
#include <atomic>
#include <map>
#include <mutex>
#include <utility>

#include "permute_index.cuh"
#include "token_core.cuh"

namespace cobalt {

constexpr int kRouteThreads = 1024;
constexpr int kRouteWarps = kRouteThreads / 32;
constexpr size_t kRouteMaxSmem = 220 * 1024;
constexpr int kRouteMaxCtas = 160;                  // the workspace is sized for grids up to this
constexpr int kRouteMaxDests = kRouteThreads;       // one destination per thread in the scans over d
constexpr uint32_t kBarrierSpinLimit = 1u << 22;    // polls of the grid barrier before giving up (about a second)

// Shared memory of one CTA, in 32-bit words.
struct RouteSmem {
    size_t tri_words;     // co-activation triangle (16- or 32-bit counters), whole 16-byte vectors; after the
                          // grid barrier: the sums of this CTA's slice, then partial destination sums
    size_t stage_words;   // the inverse map of one round in row order (1024 K entries)
    size_t tab_words;     // layout tables
    size_t dest_words;    // D rounded up to a multiple of 8
    size_t lane_stride;   // entries per warp of the lane-mask table: D rounded up to an odd number
    // tri | stage | tab | cnt[dest] | base[dest] | excl[dest] | mask[warps][lane_stride] | pre[warps][lane_stride]
    size_t words() const { return tri_words + stage_words + tab_words + 3 * dest_words + 2 * kRouteWarps * lane_stride; }
    size_t bytes() const { return words() * sizeof(uint32_t); }
};

static RouteSmem route_smem(const LayoutView& lv, int K, bool packed)
{
    RouteSmem r;
    r.tri_words = ((packed ? (tri_entries(lv.E) + 1) / 2 : tri_entries(lv.E)) + 3) / 4 * 4;
    r.stage_words = static_cast<size_t>(kRouteThreads) * K;
    r.tab_words = static_cast<size_t>(lv.words + 3) / 4 * 4;
    r.dest_words = static_cast<size_t>(lv.D + 7) / 8 * 8;
    r.lane_stride = static_cast<size_t>(lv.D) | 1u;
    return r;
}

// Grid-wide sums kept in the workspace behind the destination totals, cleared with them: the two 64-bit
// sums of Eq. 1 (V_cobalt, V_naive), as 32-bit words.
constexpr int kGridSumWords = 4;

// Workspace of the fused kernel (byte offsets, 256-byte aligned).
struct RouteWorkspace {
    size_t barrier_off, cnt_off, dtot_off, tri_off, total;
};

static RouteWorkspace route_workspace(const LayoutView& lv, bool packed)
{
    const RouteSmem sm = route_smem(lv, 1, packed);
    RouteWorkspace w;
    size_t off = 0;
    w.barrier_off = off; off += 256;
    w.cnt_off = off;     off += round_up(sizeof(uint16_t) * kRouteMaxCtas * sm.dest_words, 256);
    w.dtot_off = off;    off += round_up(sizeof(uint32_t) * (sm.dest_words + kGridSumWords), 256);
    w.tri_off = off;     off += round_up(sizeof(uint32_t) * kRouteMaxCtas * sm.tri_words, 256);
    w.total = off;
    return w;
}

__device__ __forceinline__ unsigned long long ld_relaxed_u64(const unsigned long long* p)
{
    unsigned long long v;
    asm volatile("ld.relaxed.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
    return v;
}

__device__ __forceinline__ unsigned long long ld_acquire_u64(const unsigned long long* p)
{
    unsigned long long v;
    asm volatile("ld.acquire.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
    return v;
}

// Grid-wide barrier on one 64-bit word of the workspace: epoch (high half) and arrival count.
// The word may hold anything when the kernel starts.  CTA 0 sets it to (epoch, 0) once it has cleared
// the grid-wide totals; a CTA adds to those totals, and arrives, only after it has seen the epoch
// (grid_epoch_seen), so neither can be lost to the clearing.  Arrival is one atomic add; the wait polls
// until the count reaches the number of CTAs.  Every CTA of the grid is
// resident (cooperative launch), so the wait ends as soon as the slowest CTA has arrived; it is
// bounded all the same, and a wait that runs out reports COBALT_DEVERR_WAIT_TIMEOUT and makes the
// CTA return.  After the wait every CTA signs off on the same word and the last one clears it, so
// that a replay of a captured launch (same epoch) starts from a word that differs from its epoch.
// Arrival and wait are separate calls (work that needs no other CTA goes in between); all are called by
// all threads of the CTA.
//
// grid_barrier_init: the last warp of CTA 0 does the work (the one most likely to have no token), the
// rest of the CTA does not wait for it.
__device__ __forceinline__ void grid_barrier_init(unsigned long long* word, uint32_t epoch, uint32_t* grid_sums,
                                                  int n_words)
{
    if (blockIdx.x != 0 || threadIdx.x < blockDim.x - 32) return;
    const int lane = threadIdx.x & 31;
    for (int i = lane; i < n_words; i += 32) grid_sums[i] = 0;
    __syncwarp();
    if (lane == 0) {
        __threadfence();                   // the cleared words are visible before the epoch is
        atomicExch(word, static_cast<unsigned long long>(epoch) << 32);
    }
}

// Thread 0 of a CTA: has CTA 0 published this launch's epoch (and with it the cleared totals)?  `first`
// is an earlier acquire load of the word, issued where its latency hides.  Bounded like the barrier's wait.
__device__ __forceinline__ bool grid_epoch_seen(const unsigned long long* word, unsigned long long first, uint32_t epoch)
{
    if ((first >> 32) == epoch) return true;
    for (uint32_t spin = 0; spin < kBarrierSpinLimit; ++spin) {
        if ((ld_acquire_u64(word) >> 32) == epoch) return true;
        __nanosleep(40);
    }
    return false;
}

// Arrival (after grid_epoch_seen): nothing comes back, so the arriving thread goes on with whatever lies
// between this call and the wait while the atomic travels.
__device__ __forceinline__ void grid_arrive(unsigned long long* word)
{
    __syncthreads();                       // this CTA's writes are done ...
    if (threadIdx.x == 0) {
        __threadfence();                   // ... and visible to the grid before the arrival is
        atomicAdd(word, 1ull);
    }
}

// Returns false on a timeout.  `*signed_off` (thread 0) receives what the sign-off atomic returned;
// grid_leave looks at it when the CTA is done, so nobody waits for it.
__device__ __forceinline__ bool grid_wait(unsigned long long* word, uint32_t epoch, uint32_t n_ctas, uint32_t* err_word,
                                          unsigned long long* signed_off)
{
    __shared__ int barrier_ok;
    if (threadIdx.x == 0) {
        const unsigned long long target = (static_cast<unsigned long long>(epoch) << 32) | n_ctas;
        bool ok = false;
        for (uint32_t spin = 0; spin < kBarrierSpinLimit; ++spin) {
            const unsigned long long v = ld_relaxed_u64(word);
            if ((v >> 32) == epoch && v >= target) {
                ok = true;
                break;
            }
            if (spin >= 4096) __nanosleep(40);      // a barrier that is about to open is polled back to back
        }
        __threadfence();                            // what the other CTAs published is read after this
        if (ok) *signed_off = atomicAdd(word, 1ull);
        else flag_error(err_word, COBALT_DEVERR_WAIT_TIMEOUT);
        barrier_ok = ok ? 1 : 0;
    }
    __syncthreads();
    return barrier_ok != 0;
}

// Thread 0, when the CTA is done: the last CTA to have signed off leaves the word cleared.
__device__ __forceinline__ void grid_leave(unsigned long long* word, unsigned long long signed_off, uint32_t n_ctas)
{
    if (threadIdx.x == 0 && static_cast<uint32_t>(signed_off) + 1u == 2u * n_ctas) atomicExch(word, 0ull);
}

struct RouteParams {
    LayoutView lv;
    const int32_t* topk_ids;
    const int32_t* src_rank;
    int32_t src_uniform;
    int64_t T;
    int32_t K_rt;
    uint32_t seed_lo, seed_hi;
    const unsigned long long* seed_on_device;
    uint32_t* coact;
    uint32_t* load;
    int32_t* assigned_slot;
    uint8_t* remote_nodes;
    unsigned long long* totals;
    uint32_t* dest_counts;
    uint32_t* dest_offsets;
    int32_t* row_of_pair;
    int32_t* pair_of_row;
    // workspace
    unsigned long long* barrier;
    uint16_t* ws_cnt;                  // [CTAs][dest_words], 16-bit: a CTA sends at most one pair per token to a destination
    uint32_t* ws_dtot;                 // [dest_words] pairs per destination over the whole grid (atomic adds),
                                       // then the two sums of Eq. 1 (64-bit each)
    uint32_t* ws_tri;                  // [CTAs][tri_words]
    uint32_t epoch;
    int tri_words, stage_words, tab_words, dest_words, lane_stride;
    int tokens_per_cta;                // a multiple of 32
    int accumulate;                    // add to coact / load instead of overwriting them
    uint32_t* err_word;
};

// Exclusive scan over d of one value per thread (threads >= D pass 0); returns the sum of the
// values of lower threads.  `total` receives the sum of all values.  Two block barriers.
__device__ __forceinline__ uint32_t block_exclusive_scan(uint32_t value, uint32_t* warp_sums, uint32_t* total)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    uint32_t incl = value;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const uint32_t up = __shfl_up_sync(0xFFFFFFFFu, incl, off);
        if (lane >= off) incl += up;
    }
    __syncthreads();                      // warp_sums may still be read from the previous scan
    if (lane == 31) warp_sums[warp] = incl;
    __syncthreads();
    uint32_t before = incl - value, all = 0;
#pragma unroll
    for (int w = 0; w < kRouteWarps; ++w) {
        const uint32_t s = warp_sums[w];
        if (w < warp) before += s;
        all += s;
    }
    *total = all;
    return before;
}

// One entry of the staged inverse map / of a thread's saved ranks: destination in the low bits, the
// rest above it.
constexpr int kDestBits = 10;
static_assert(kRouteMaxDests <= (1 << kDestBits), "destinations must fit the packed entry");
static_assert(kRouteThreads * COBALT_MAX_TOPK <= (1 << (32 - kDestBits - 1)), "a round's pairs must fit the packed entry");

// Barrier among the 512 threads of one half of the CTA (named barrier 1 for the lower half, 2 for the upper).
__device__ __forceinline__ void half_barrier(int id)
{
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(kRouteThreads / 2) : "memory");
}

// Exclusive scan over d with two consecutive destinations per thread of the lower half (threads
// 0 .. 511, D <= 1024); `before` receives the sum of the values below destination 2 * tid.  Uses half
// barriers only.
__device__ __forceinline__ uint32_t half_exclusive_scan2(uint32_t pair_sum, uint32_t* warp_sums, uint32_t* total)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    uint32_t incl = pair_sum;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const uint32_t up = __shfl_up_sync(0xFFFFFFFFu, incl, off);
        if (lane >= off) incl += up;
    }
    if (lane == 31) warp_sums[warp] = incl;
    half_barrier(1);
    uint32_t before = incl - pair_sum, all = 0;
#pragma unroll
    for (int w = 0; w < kRouteWarps / 2; ++w) {
        const uint32_t s = warp_sums[w];
        if (w < warp) before += s;
        all += s;
    }
    *total = all;
    return before;
}

template <int KT, bool kPacked>
__global__ void __launch_bounds__(kRouteThreads)
route_fused_kernel(const RouteParams p)
{
    extern __shared__ __align__(16) uint32_t smem[];
    uint32_t* tri = smem;                                      // later: acc (phase 2a), part (phase 2b)
    uint32_t* stage = tri + p.tri_words;                       // [1024 K] the pairs of one round by place (destination-major)
    uint32_t* tab = stage + p.stage_words;
    uint32_t* cnt = tab + p.tab_words;                         // [D] pairs of this CTA per destination (several rounds only)
    uint32_t* base = cnt + p.dest_words;                       // [D] first row of the CTA's (round's) pairs inside d; with
                                                               // one round: that minus the place of the first of them
    uint32_t* excl = base + p.dest_words;                      // [D] place of d's first pair (one round); several rounds:
                                                               // the round's shift from place to row
    uint32_t* mask = excl + p.dest_words;                      // [warps][lane_stride] lanes (tokens) of the warp that send to d
    uint32_t* pre = mask + kRouteWarps * p.lane_stride;        // [warps][lane_stride] place of the warp's first pair to d
    __shared__ unsigned long long cta_totals[2];
    __shared__ uint32_t warp_sums[kRouteWarps];
    __shared__ int epoch_ok;

    constexpr int KMAX = TokenShape<KT>::KMAX;
    const int K = (KT > 0) ? KT : p.K_rt;
    const int D = p.lv.D, E = p.lv.E;
    const int dest_words = p.dest_words;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int cta = static_cast<int>(blockIdx.x), n_ctas = static_cast<int>(gridDim.x);
    uint32_t* my_mask = mask + warp * p.lane_stride;
    const uint32_t* my_pre = pre + warp * p.lane_stride;
    const uint32_t lower_lanes = (1u << lane) - 1u;

    uint32_t seed_lo = p.seed_lo, seed_hi = p.seed_hi;
    if (p.seed_on_device) {                                   // the seed of this run, not of the capture
        const unsigned long long sd = __ldg(p.seed_on_device);
        seed_lo = static_cast<uint32_t>(sd);
        seed_hi = static_cast<uint32_t>(sd >> 32);
    }

    const int64_t t_lo = min(p.T, static_cast<int64_t>(cta) * p.tokens_per_cta);
    const int64_t t_hi = min(p.T, t_lo + p.tokens_per_cta);
    const int n_rounds = static_cast<int>((t_hi - t_lo + kRouteThreads - 1) / kRouteThreads);
    // One round (at most 1024 tokens per CTA): the lane masks that rank the pairs are built while the
    // slots are assigned, and everything about the ranks that needs no other CTA is done before the
    // grid barrier is waited for.  More rounds: the slots are counted, and the ranks are worked out
    // round by round after the barrier.
    const bool single = n_rounds <= 1;

    // the first round's loads go out before the shared-memory set-up so that the two overlap
    int32_t id[KMAX], out[KMAX];
    int32_t s_t = p.src_uniform;
    if (t_lo + tid < t_hi) {
        load_token_ids<KT>(p.topk_ids, t_lo + tid, K, id);
        if (p.src_rank) s_t = __ldg(p.src_rank + t_lo + tid);
    }
    // the layout tables travel to shared memory asynchronously, behind the clearing of the other arrays
    {
        const uint4* src = reinterpret_cast<const uint4*>(p.lv.blob);
        const int n_vec = (p.lv.words + 3) / 4;
        for (int i = tid; i < n_vec; i += kRouteThreads)
            asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(static_cast<uint32_t>(__cvta_generic_to_shared(
                             reinterpret_cast<uint4*>(tab) + i))),
                         "l"(src + i)
                         : "memory");
        asm volatile("cp.async.commit_group;" ::: "memory");
    }
    for (int i = tid; i < p.tri_words / 4; i += kRouteThreads) reinterpret_cast<uint4*>(tri)[i] = make_uint4(0, 0, 0, 0);
    for (int i = tid; i < dest_words / 4; i += kRouteThreads) reinterpret_cast<uint4*>(cnt)[i] = make_uint4(0, 0, 0, 0);
    for (int i = tid; i < kRouteWarps * p.lane_stride / 4; i += kRouteThreads)      // 32 x stride words: whole vectors
        reinterpret_cast<uint4*>(mask)[i] = make_uint4(0, 0, 0, 0);
    if (tid < 2) cta_totals[tid] = 0;
    const TableView tv = table_view(p.lv, tab);
    asm volatile("cp.async.wait_all;" ::: "memory");      // the tables have arrived behind the clearing
    __syncthreads();
    grid_barrier_init(p.barrier, p.epoch, p.ws_dtot, dest_words + kGridSumWords);   // no CTA looks before it publishes

    // ---- phase 1: statistics, Algorithm 1, destination counts ---------------------------------
    uint32_t cost_sum = 0, naive_sum = 0;
    for (int round = 0; round < n_rounds; ++round) {
        const int64_t t = t_lo + static_cast<int64_t>(round) * kRouteThreads + tid;
        const bool has_token = t < t_hi;
        uint32_t bad = 0;
        if (has_token) {
            if (round > 0) {
                load_token_ids<KT>(p.topk_ids, t, K, id);
                if (p.src_rank) s_t = __ldg(p.src_rank + t);
            }
            int32_t sorted[KMAX];
            sort_token_ids<KT>(id, K, sorted);
            const uint32_t bad_ids = check_sorted_ids<KT>(sorted, K, E);
            bad = bad_ids;
            if (s_t < 0 || s_t >= p.lv.G) bad |= COBALT_DEVERR_BAD_SRC_RANK;
            if (bad) flag_error(p.err_word, bad);
            // the statistics only need valid ids, as in the stand-alone statistics call
            if (!bad_ids) add_sorted_token_to_triangle<KT, kPacked>(tri, sorted, K);
        }
        if (has_token) {
            uint32_t cost = 0, naive_cost = 0;
            if (bad) {
#pragma unroll
                for (int a = 0; a < KMAX; ++a) out[a] = -1;
            } else {
                assign_token<KT, kAssignSlot>(tv, id, K, s_t, static_cast<uint32_t>(t), seed_lo, seed_hi, out, cost,
                                              naive_cost);
                if (single) {
#pragma unroll
                    for (int a = 0; a < KMAX; ++a)
                        if (a < K) atomicOr(&my_mask[out[a]], 1u << lane);
                } else {
#pragma unroll
                    for (int a = 0; a < KMAX; ++a)
                        if (a < K) atomicAdd(&cnt[out[a]], 1u);
                }
            }
            store_token_slots<KT>(p.assigned_slot + t * K, out, K);
            if (p.remote_nodes) p.remote_nodes[t] = static_cast<uint8_t>(cost);
            cost_sum += cost;
            naive_sum += naive_cost;
        }
    }
    if (p.totals) {
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) {
            cost_sum += __shfl_xor_sync(0xFFFFFFFFu, cost_sum, off);
            naive_sum += __shfl_xor_sync(0xFFFFFFFFu, naive_sum, off);
        }
        if (lane == 0) {
            if (cost_sum) atomicAdd(&cta_totals[0], static_cast<unsigned long long>(cost_sum));
            if (naive_sum) atomicAdd(&cta_totals[1], static_cast<unsigned long long>(naive_sum));
        }
    }
    __syncthreads();

    // The ranks of a round's pairs come from the lane masks in three steps.  (1) count_dests: thread d
    // adds up the pairs the 32 warps send to destination d (consecutive threads, consecutive words: no
    // bank conflicts).  (2) A scan of those counts over d gives the place of d's first pair in the round's
    // destination-major order, and prefix_dests walks down the warps once more and leaves in pre[w][d] the
    // place of warp w's first pair to d.  (3) rank_round: a pair's place is pre[w][d] plus the lower lanes
    // of its warp that send to d; the pair goes into the staged inverse map at that place, and the place
    // (packed with d into out[], -1 for a pair without a destination) is kept for write_round.
    auto count_dests = [&]() -> uint32_t {
        uint32_t sum = 0;
        if (tid < D) {
#pragma unroll 8
            for (int w = 0; w < kRouteWarps; ++w) sum += __popc(mask[w * p.lane_stride + tid]);
        }
        return sum;
    };
    auto prefix_dests = [&](uint32_t first) {
        if (tid < D) {
            uint32_t run = first;
#pragma unroll 8
            for (int w = 0; w < kRouteWarps; ++w) {
                const uint32_t c = __popc(mask[w * p.lane_stride + tid]);
                pre[w * p.lane_stride + tid] = run;
                run += c;
            }
        }
    };
    auto rank_round = [&](bool has_token) {
        if (!has_token) return;
#pragma unroll
        for (int a = 0; a < KMAX; ++a) {
            if (a < K && out[a] >= 0) {
                const uint32_t d = static_cast<uint32_t>(out[a]);
                const uint32_t r = my_pre[d] + __popc(my_mask[d] & lower_lanes);
                if (p.pair_of_row) stage[r] = d | (static_cast<uint32_t>(tid * K + a) << kDestBits);
                out[a] = static_cast<int32_t>(d | (r << kDestBits));
            }
        }
    };
    // Rows of the thread's pairs and the round's part of the inverse map in row order (consecutive
    // threads write consecutive rows of a destination): a pair's row is its place in the round plus
    // shift[d], the first row of the round's pairs inside d minus the place of the first of them.
    auto write_round = [&](bool has_token, int64_t t_round, uint32_t round_pairs, const uint32_t* shift) {
        if (has_token) {
            int32_t row[KMAX];
#pragma unroll
            for (int a = 0; a < KMAX; ++a) {
                row[a] = -1;
                if (a < K && out[a] >= 0)
                    row[a] = static_cast<int32_t>(shift[out[a] & ((1 << kDestBits) - 1)] + (static_cast<uint32_t>(out[a]) >> kDestBits));
            }
            store_token_slots<KT>(p.row_of_pair + (t_round + tid) * K, row, K);
        }
        if (p.pair_of_row) {
            for (uint32_t j = tid; j < round_pairs; j += kRouteThreads) {
                const uint32_t v = stage[j];
                p.pair_of_row[shift[v & ((1u << kDestBits) - 1u)] + j] = static_cast<int32_t>(t_round * K + (v >> kDestBits));
            }
        }
    };

    // ---- publish this CTA's partial results ------------------------------------------------------
    // The triangle goes first (9.7 MB over the grid: the stores drain while the counts are worked out).
    unsigned long long word_now = 0;
    if (tid == 0) word_now = ld_acquire_u64(p.barrier);     // looked at below: has CTA 0 cleared the grid's totals?
    {
        uint4* dst = reinterpret_cast<uint4*>(p.ws_tri + static_cast<size_t>(cta) * p.tri_words);
        for (int v = tid; v < p.tri_words / 4; v += kRouteThreads) dst[v] = reinterpret_cast<const uint4*>(tri)[v];
    }
    // this CTA's pairs to destination tid: from the lane masks (one round) or as counted in phase 1
    uint32_t my_cnt = 0, first_place = 0, round_pairs = 0;
    if (single) my_cnt = count_dests();
    else if (tid < D) my_cnt = cnt[tid];
    if (tid == 0) {
        epoch_ok = grid_epoch_seen(p.barrier, word_now, p.epoch) ? 1 : 0;
        if (!epoch_ok) flag_error(p.err_word, COBALT_DEVERR_WAIT_TIMEOUT);
    }
    if (single) first_place = block_exclusive_scan(my_cnt, warp_sums, &round_pairs);
    else __syncthreads();
    if (!epoch_ok) return;
    {
        // 16-bit counts, two to a word: the even thread takes its neighbour's along
        const uint32_t next_cnt = __shfl_down_sync(0xFFFFFFFFu, my_cnt, 1);
        if (!(tid & 1) && tid < dest_words)
            reinterpret_cast<uint32_t*>(p.ws_cnt + static_cast<size_t>(cta) * dest_words)[tid >> 1] = my_cnt | (next_cnt << 16);
        if (my_cnt) atomicAdd(p.ws_dtot + tid, my_cnt);
        if (p.totals && tid < 2 && cta_totals[tid])
            atomicAdd(reinterpret_cast<unsigned long long*>(p.ws_dtot + dest_words) + tid, cta_totals[tid]);
    }
    // what the ranks need from this CTA alone: the prefixes before the arrival (the additions above travel
    // meanwhile), the ranks between arrival and wait
    if (single) {
        prefix_dests(first_place);
        if (tid < D) excl[tid] = first_place;
    }
    grid_arrive(p.barrier);
    if (single) rank_round(t_lo + tid < t_hi);
    unsigned long long signed_off = 0;
    if (!grid_wait(p.barrier, p.epoch, static_cast<uint32_t>(n_ctas), p.err_word, &signed_off)) return;

    // ---- phase 2a and 2b side by side: both wait on loads of what the other CTAs published, so the
    // upper half of the CTA's warps sums this CTA's slice of the triangle over all partials (2a) while
    // the lower half sums the destination counts of all CTAs (2b) ---------------------------------
    constexpr int kHalf = kRouteThreads / 2;
    constexpr int kPerWord = kPacked ? 2 : 1;
    const int n_tri = static_cast<int>(tri_entries(E));
    const int n_vec = p.tri_words / 4;                                // 16-byte vectors of a triangle
    const int slice = (n_vec + n_ctas - 1) / n_ctas;                  // vectors of a CTA's slice
    const int v0 = min(n_vec, cta * slice), v1 = min(n_vec, v0 + slice);
    const int n_mine = v1 - v0;
    const int n_acc = 4 * n_mine * kPerWord;                          // sums of the slice, 32 bits each
    // 2b: the pairs of the lower CTAs per destination.  The grid's totals are there already (atomic
    // adds before the barrier), so a CTA of the lower half of the grid sums the counts of the CTAs below
    // it and one of the upper half those from itself upwards, which it takes off the total: at most half
    // of the CTAs' counts either way.  They are split over `parts` groups of threads; a thread sums eight
    // consecutive destinations of its share of the CTAs and leaves its sums where the triangle was,
    // behind the sums of the slice; one thread per destination adds them up.
    const bool from_below = 2 * cta <= n_ctas;
    const int c_begin = from_below ? 0 : cta, c_end = from_below ? cta : n_ctas;
    const int octs = dest_words / 8;
    int parts = max(1, kHalf / octs);
    parts = min(parts, max(1, (n_ctas + 1) / 2));
    if (parts > 1) parts = max(1, min(parts, (p.tri_words - n_acc) / dest_words));
    uint32_t* acc = tri;
    uint32_t* part_sum = tri + (n_acc + 3) / 4 * 4;                   // [parts][dest_words]
    if ((n_acc + 3) / 4 * 4 + parts * dest_words > p.tri_words) {     // a tiny triangle: one group, sums straight into base
        parts = 1;
        part_sum = base;
    }
    for (int i = tid; i < n_acc; i += kRouteThreads) acc[i] = 0;
    __syncthreads();
    if (tid >= kHalf) {
        // 2a: `groups` threads share a vector of the slice, each summing every groups-th partial in
        // registers (loads in flight together, lanes along consecutive vectors), then shared-memory adds
        constexpr int kBatch = 9;
        const int ht = tid - kHalf;
        if (n_mine > 0) {
            const int groups = max(1, kHalf / n_mine);
            for (int j = ht; j < groups * n_mine; j += kHalf) {          // one pass unless n_mine > 512
                const int g = j / n_mine, v = j - g * n_mine;
                const uint4* src = reinterpret_cast<const uint4*>(p.ws_tri) + v0 + v;
                uint32_t sum[4 * kPerWord];
#pragma unroll
                for (int i = 0; i < 4 * kPerWord; ++i) sum[i] = 0;
                for (int c = g; c < n_ctas; c += groups * kBatch) {
                    uint4 q[kBatch];
#pragma unroll
                    for (int u = 0; u < kBatch; ++u) {
                        const int cc = c + u * groups;
                        q[u] = (cc < n_ctas) ? __ldcg(src + static_cast<size_t>(cc) * n_vec) : make_uint4(0, 0, 0, 0);
                    }
#pragma unroll
                    for (int u = 0; u < kBatch; ++u) {
                        const uint32_t word[4] = {q[u].x, q[u].y, q[u].z, q[u].w};
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            if (kPacked) {
                                sum[2 * i] += word[i] & 0xFFFFu;
                                sum[2 * i + 1] += word[i] >> 16;
                            } else {
                                sum[i] += word[i];
                            }
                        }
                    }
                }
#pragma unroll
                for (int i = 0; i < 4 * kPerWord; ++i)
                    if (sum[i]) atomicAdd(&acc[4 * kPerWord * v + i], sum[i]);
            }
        }
        if (p.totals && cta == 0 && ht < 2)
            p.totals[ht] = __ldcg(reinterpret_cast<const unsigned long long*>(p.ws_dtot + dest_words) + ht);
    } else {
        constexpr int kBatch = 6;
        const int part = tid / octs, oct = tid - part * octs;
        if (part < parts) {
            const uint4* src = reinterpret_cast<const uint4*>(p.ws_cnt) + oct;
            uint32_t sum[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) sum[i] = 0;
            for (int c = c_begin + part; c < c_end; c += parts * kBatch) {
                uint4 q[kBatch];
#pragma unroll
                for (int u = 0; u < kBatch; ++u) {
                    const int cc = c + u * parts;
                    q[u] = (cc < c_end) ? __ldcg(src + static_cast<size_t>(cc) * octs) : make_uint4(0, 0, 0, 0);
                }
#pragma unroll
                for (int u = 0; u < kBatch; ++u) {
                    const uint32_t word[4] = {q[u].x, q[u].y, q[u].z, q[u].w};
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        sum[2 * i] += word[i] & 0xFFFFu;
                        sum[2 * i + 1] += word[i] >> 16;
                    }
                }
            }
            uint4* dst = reinterpret_cast<uint4*>(part_sum + part * dest_words + 8 * oct);
            dst[0] = make_uint4(sum[0], sum[1], sum[2], sum[3]);
            dst[1] = make_uint4(sum[4], sum[5], sum[6], sum[7]);
        }
    }
    // (the two halves go on separately: each only waits for its own half until the rows are written)
    if (tid >= kHalf) {
        half_barrier(2);
        // 2a: the sums of the slice go out to coact / load (plain stores unless accumulating)
        for (int i = tid - kHalf; i < n_acc; i += kHalf) {
            const int flat = 4 * v0 * kPerWord + i;
            if (flat >= n_tri) continue;
            const int hi = tri_row(flat), lo = flat - hi * (hi + 1) / 2;
            const uint32_t v = acc[i];
            if (p.accumulate) {
                if (v) {
                    atomicAdd(&p.coact[static_cast<size_t>(hi) * E + lo], v);
                    if (lo != hi) atomicAdd(&p.coact[static_cast<size_t>(lo) * E + hi], v);
                    else atomicAdd(&p.load[hi], v);
                }
            } else {
                p.coact[static_cast<size_t>(hi) * E + lo] = v;
                if (lo != hi) p.coact[static_cast<size_t>(lo) * E + hi] = v;
                else p.load[hi] = v;
            }
        }
    } else {
        // 2b: totals over all CTAs, their exclusive scan over d (the offsets), first row of this CTA;
        // two consecutive destinations per thread
        uint32_t mine[2] = {0, 0}, lower[2] = {0, 0};
        if (2 * tid < D) {                       // dest_words is even: the pair is inside the array
            const uint2 both = __ldcg(reinterpret_cast<const uint2*>(p.ws_dtot) + tid);
            mine[0] = both.x;
            mine[1] = (2 * tid + 1 < D) ? both.y : 0u;
        }
        half_barrier(1);
#pragma unroll
        for (int j = 0; j < 2; ++j) {
            const int d = 2 * tid + j;
            if (d < D) {
                uint32_t s = 0;
                for (int g = 0; g < parts; ++g) s += part_sum[g * dest_words + d];
                lower[j] = from_below ? s : mine[j] - s;
            }
        }
        uint32_t total = 0;
        uint32_t before = half_exclusive_scan2(mine[0] + mine[1], warp_sums, &total);
        half_barrier(1);                         // the part buffers have been read: base may be written (it can be one of them)
#pragma unroll
        for (int j = 0; j < 2; ++j) {
            const int d = 2 * tid + j;
            if (d < D) {
                if (cta == 0) {
                    p.dest_counts[d] = mine[j];
                    p.dest_offsets[d] = before;
                }
                // one round: its pairs' places are known already, so what is kept is the shift from place to row
                base[d] = before + lower[j] - (single ? excl[d] : 0u);
            }
            before += mine[j];
        }
        if (cta == 0 && tid == 0) p.dest_offsets[D] = total;
    }
    __syncthreads();

    // ---- phase 2c: rows of this CTA's pairs ------------------------------------------------------
    if (single) {
        write_round(t_lo + tid < t_hi, t_lo, round_pairs, base);
        grid_leave(p.barrier, signed_off, static_cast<uint32_t>(n_ctas));
        return;
    }
    for (int round = 0; round < n_rounds; ++round) {
        const int64_t t_round = t_lo + static_cast<int64_t>(round) * kRouteThreads;
        const int64_t t = t_round + tid;
        const bool has_token = t < t_hi;
        if (has_token) {
            // the slots come back from memory (this thread wrote them in phase 1)
            const int32_t* slots = p.assigned_slot + t * K;
            if (KT > 0 && KT % 4 == 0) {
#pragma unroll
                for (int a = 0; a < KT / 4; ++a) {
                    const int4 v = reinterpret_cast<const int4*>(slots)[a];
                    out[4 * a] = v.x; out[4 * a + 1] = v.y; out[4 * a + 2] = v.z; out[4 * a + 3] = v.w;
                }
            } else {
#pragma unroll
                for (int a = 0; a < KMAX; ++a)
                    if (a < K) out[a] = slots[a];
            }
#pragma unroll
            for (int a = 0; a < KMAX; ++a)
                if (a < K && out[a] >= 0) atomicOr(&my_mask[out[a]], 1u << lane);
        }
        __syncthreads();
        const uint32_t round_total = count_dests();
        const uint32_t round_first = block_exclusive_scan(round_total, warp_sums, &round_pairs);
        prefix_dests(round_first);
        if (tid < D) excl[tid] = base[tid] - round_first;        // the round's shift from place to row
        // the masks are cleared through the still unpacked slots before rank_round packs them
        __syncthreads();
        uint32_t touched[KMAX];
#pragma unroll
        for (int a = 0; a < KMAX; ++a) touched[a] = (has_token && a < K && out[a] >= 0) ? static_cast<uint32_t>(out[a]) : 0xFFFFFFFFu;
        rank_round(has_token);
        __syncthreads();
        write_round(has_token, t_round, round_pairs, excl);
        __syncthreads();
#pragma unroll
        for (int a = 0; a < KMAX; ++a)
            if (touched[a] != 0xFFFFFFFFu) my_mask[touched[a]] = 0;
        if (tid < D) base[tid] += round_total;
        __syncthreads();
    }
    grid_leave(p.barrier, signed_off, static_cast<uint32_t>(n_ctas));
}

// The grid the device can hold for this kernel and shared-memory size (one CTA per SM in practice),
// asked once per (device, kernel, bytes); 0 if the device cannot launch it cooperatively.
template <int KT, bool kPacked>
static int max_resident_ctas(size_t smem, int* out)
{
    auto kernel = route_fused_kernel<KT, kPacked>;
    static std::mutex cache_lock;
    static std::map<std::pair<int, size_t>, int> cache;
    int dev = 0;
    COBALT_CUDA_TRY(cudaGetDevice(&dev));
    const auto key = std::make_pair(dev, smem);
    {
        std::lock_guard<std::mutex> guard(cache_lock);
        auto it = cache.find(key);
        if (it != cache.end()) {
            *out = it->second;
            return COBALT_OK;
        }
    }
    int rc_attr = ensure_kernel_attributes(reinterpret_cast<const void*>(kernel), smem, false);
    if (rc_attr != COBALT_OK) return rc_attr;
    int best = 0, cooperative = 0, n_sm = 0, per_sm = 0;
    COBALT_CUDA_TRY(cudaDeviceGetAttribute(&cooperative, cudaDevAttrCooperativeLaunch, dev));
    rc_attr = sm_count(&n_sm);
    if (rc_attr != COBALT_OK) return rc_attr;
    if (cooperative &&
        cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, kRouteThreads, smem) == cudaSuccess && per_sm >= 1)
        best = std::min(n_sm, kRouteMaxCtas);          // one CTA per SM: more would only share the SM's issue slots
    else
        (void)cudaGetLastError();
    {
        std::lock_guard<std::mutex> guard(cache_lock);
        cache[key] = best;
    }
    *out = best;
    return COBALT_OK;
}

struct RouteArgs {
    RouteParams p;
    int K;
    void* workspace;
    cudaStream_t stream;
};

// Epochs of the grid barrier: distinct for consecutive launches and never 0 (a cleared word).
static uint32_t next_epoch()
{
    static std::atomic<uint32_t> counter{0};
    uint32_t x = counter.fetch_add(1) + 1u;
    x *= 0x9E3779B9u;                 // odd multiplier: a bijection, so consecutive launches differ
    return x ? x : 0x5bd1e995u;
}

// *launched stays false (and nothing has been enqueued) when the kernel does not fit this layout,
// batch or device: the caller then takes the separate calls.
template <int KT, bool kPacked>
static int launch_route(RouteArgs a, bool* launched)
{
    *launched = false;
    RouteParams& p = a.p;
    if (p.lv.D > kRouteMaxDests) return COBALT_OK;
    const RouteSmem sm = route_smem(p.lv, a.K, kPacked);
    if (sm.bytes() > kRouteMaxSmem) return COBALT_OK;
    int max_ctas = 0;
    int rc = max_resident_ctas<KT, kPacked>(sm.bytes(), &max_ctas);
    if (rc != COBALT_OK) return rc;
    if (max_ctas < 1) return COBALT_OK;
    // 256 tokens per CTA until the resident CTAs run out
    int64_t want = (p.T + 255) / 256;
    if (want > max_ctas) want = max_ctas;
    // with 16-bit counters the sums of a slice (32-bit) are kept where the triangle was: at least two slices
    const int min_ctas = kPacked ? 2 : 1;
    if (want < min_ctas) want = min_ctas;
    if (want > max_ctas) return COBALT_OK;
    const int n_ctas = static_cast<int>(want);
    const int64_t per = static_cast<int64_t>(round_up(static_cast<size_t>((p.T + n_ctas - 1) / n_ctas), 32));
    if (per > 0x7FFFFFFFll) return COBALT_OK;
    if (per > 65535) return COBALT_OK;     // the CTA's 16-bit counters (destination counts, packed triangle) could overflow
    p.tokens_per_cta = static_cast<int>(per);
    p.tri_words = static_cast<int>(sm.tri_words);
    p.stage_words = static_cast<int>(sm.stage_words);
    p.tab_words = static_cast<int>(sm.tab_words);
    p.dest_words = static_cast<int>(sm.dest_words);
    p.lane_stride = static_cast<int>(sm.lane_stride);
    const RouteWorkspace w = route_workspace(p.lv, kPacked);
    uint8_t* ws = static_cast<uint8_t*>(a.workspace);
    p.barrier = reinterpret_cast<unsigned long long*>(ws + w.barrier_off);
    p.ws_cnt = reinterpret_cast<uint16_t*>(ws + w.cnt_off);
    p.ws_dtot = reinterpret_cast<uint32_t*>(ws + w.dtot_off);
    p.ws_tri = reinterpret_cast<uint32_t*>(ws + w.tri_off);
    p.epoch = next_epoch();

    auto kernel = route_fused_kernel<KT, kPacked>;
    cudaLaunchConfig_t cfg = {};
    cudaLaunchAttribute attr[1];
    cfg.blockDim = dim3(kRouteThreads);
    cfg.gridDim = dim3(static_cast<unsigned>(n_ctas));
    cfg.dynamicSmemBytes = sm.bytes();
    cfg.stream = a.stream;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    attr[0].id = cudaLaunchAttributeCooperative;     // all CTAs resident together: the grid barrier cannot starve
    attr[0].val.cooperative = 1;
    COBALT_CUDA_TRY(cudaLaunchKernelEx(&cfg, kernel, p));
    *launched = true;
    return COBALT_OK;
}

// 0: the triangle does not fit beside the other arrays, 1: it fits with 32-bit counters, 2: with 16-bit ones
static int fused_mode(const LayoutView& lv, int K, uint32_t tile_flags)
{
    // from about 180 experts on the 16-bit triangle is taken even where the 32-bit one fits: the
    // exchange is bound by the bytes of the partial triangles
    const bool large_tile = tri_entries(lv.E) * sizeof(uint32_t) >= 64 * 1024;
    if (large_tile && !(tile_flags & COBALT_STATS_TILE32) && route_smem(lv, K, true).bytes() <= kRouteMaxSmem) return 2;
    if (route_smem(lv, K, false).bytes() <= kRouteMaxSmem) return 1;
    if (route_smem(lv, K, true).bytes() <= kRouteMaxSmem) return 2;
    return 0;
}

template <int KT>
static int launch_route_any(const RouteArgs& a, bool packed, bool* launched)
{
    return packed ? launch_route<KT, true>(a, launched) : launch_route<KT, false>(a, launched);
}

static int dispatch_route(const RouteArgs& a, bool packed, bool* launched)
{
    switch (a.K) {
        case 1: return launch_route_any<1>(a, packed, launched);
        case 2: return launch_route_any<2>(a, packed, launched);
        case 3: return launch_route_any<3>(a, packed, launched);
        case 4: return launch_route_any<4>(a, packed, launched);
        case 5: return launch_route_any<5>(a, packed, launched);
        case 6: return launch_route_any<6>(a, packed, launched);
        case 7: return launch_route_any<7>(a, packed, launched);
        case 8: return launch_route_any<8>(a, packed, launched);
        case 9: return launch_route_any<9>(a, packed, launched);
        case 10: return launch_route_any<10>(a, packed, launched);
        case 11: return launch_route_any<11>(a, packed, launched);
        case 12: return launch_route_any<12>(a, packed, launched);
        case 13: return launch_route_any<13>(a, packed, launched);
        case 14: return launch_route_any<14>(a, packed, launched);
        case 15: return launch_route_any<15>(a, packed, launched);
        case 16: return launch_route_any<16>(a, packed, launched);
        default: *launched = false; return COBALT_OK;
    }
}

}  // namespace cobalt

using namespace cobalt;

extern "C" {

size_t cobalt_route_index_workspace_bytes(const cobalt_layout_t* layout, int64_t T, int32_t K)
{
    if (!layout || T < 0 || K < 1 || K > COBALT_MAX_TOPK || T * static_cast<int64_t>(K) >= (1ll << 31)) return 0;
    const LayoutView& lv = layout->view;
    // room for the separate calls as well: the pass falls back to them when the fused kernel does not
    // fit the layout, the batch or the device
    size_t need = cobalt_permute_workspace_bytes(T, K, lv.D);
    if (route_smem(lv, K, false).bytes() <= kRouteMaxSmem) need = std::max(need, route_workspace(lv, false).total);
    if (route_smem(lv, K, true).bytes() <= kRouteMaxSmem) need = std::max(need, route_workspace(lv, true).total);
    return need;
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
    if (flags & ~(COBALT_STATS_ACCUMULATE | COBALT_SEED_ON_DEVICE | COBALT_STATS_TILE32 | COBALT_ROUTE_SEPARATE_KERNELS))
        return COBALT_ERR_INVALID_ARG;
    const bool seed_on_device = (flags & COBALT_SEED_ON_DEVICE) != 0;
    if (seed_on_device && (seed == 0 || (seed & 7u) != 0)) return COBALT_ERR_INVALID_ARG;
    const size_t need = cobalt_route_index_workspace_bytes(layout, T, K);
    if (!workspace || workspace_bytes < need) return COBALT_ERR_WORKSPACE_TOO_SMALL;
    int dev = 0;
    COBALT_CUDA_TRY(cudaGetDevice(&dev));
    if (dev != layout->device) return COBALT_ERR_INVALID_ARG;

    const int mode = fused_mode(lv, K, flags & COBALT_STATS_TILE32);
    bool launched = false;
    if (mode != 0 && T > 0 && !(flags & COBALT_ROUTE_SEPARATE_KERNELS)) {
        RouteArgs a;
        RouteParams& p = a.p;
        p.lv = lv;
        p.topk_ids = topk_ids; p.src_rank = src_rank; p.src_uniform = src_rank_uniform; p.T = T; p.K_rt = K;
        p.seed_lo = seed_on_device ? 0u : static_cast<uint32_t>(seed & 0xFFFFFFFFu);
        p.seed_hi = seed_on_device ? 0u : static_cast<uint32_t>(seed >> 32);
        p.seed_on_device = seed_on_device ? reinterpret_cast<const unsigned long long*>(static_cast<uintptr_t>(seed)) : nullptr;
        p.coact = coact; p.load = load; p.assigned_slot = assigned_slot; p.remote_nodes = remote_nodes;
        p.totals = reinterpret_cast<unsigned long long*>(totals);
        p.dest_counts = dest_counts; p.dest_offsets = dest_offsets; p.row_of_pair = row_of_pair; p.pair_of_row = pair_of_row;
        p.accumulate = (flags & COBALT_STATS_ACCUMULATE) ? 1 : 0;
        a.K = K; a.workspace = workspace; a.stream = static_cast<cudaStream_t>(stream);
        int rc = device_error_word(&p.err_word);
        if (rc != COBALT_OK) return rc;
        rc = dispatch_route(a, mode == 2, &launched);
        // 16-bit counters refused for this many tokens: the 32-bit triangle, if it fits
        if (rc == COBALT_OK && !launched && mode == 2 && route_smem(lv, K, false).bytes() <= kRouteMaxSmem)
            rc = dispatch_route(a, false, &launched);
        if (rc != COBALT_OK || launched) return rc;
    }
    // the fused kernel does not fit (or there is nothing to route, or the caller asked for it): the
    // same results from the separate calls
    int rc = cobalt_coact_stats(topk_ids, T, K, lv.E, coact, load, flags & (COBALT_STATS_ACCUMULATE | COBALT_STATS_TILE32),
                                nullptr, 0, stream);
    if (rc != COBALT_OK) return rc;
    rc = cobalt_assign(layout, topk_ids, src_rank, src_rank_uniform, T, K, seed, assigned_slot, nullptr,
                       remote_nodes, totals, flags & COBALT_SEED_ON_DEVICE, nullptr, 0, stream);
    if (rc != COBALT_OK) return rc;
    return cobalt_permute_index(assigned_slot, T, K, lv.D, dest_counts, dest_offsets, row_of_pair, pair_of_row,
                                workspace, workspace_bytes, stream);
}

}  // extern "C"
