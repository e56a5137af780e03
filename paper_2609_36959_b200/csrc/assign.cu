// Stage 2: communication-aware task assignment (Section 3.3, Algorithm 1), one thread per token.
//
// The layout tables (R_{e,n}, N_e, primaries; a few KB) are staged once per CTA in shared
// memory.  Each thread keeps its token's K ids and remote masks in registers, finds b* (lines
// 5-8), draws the node and the replica with the counter hash, and writes its K slots with
// 8/16-byte stores.  Per-slot loads w_er are histogrammed in shared memory and merged with one
// integer reduction per slot and CTA; the Eq. 1 totals are reduced per warp and added once per
// CTA.  Integer adds commute, so the result does not depend on scheduling.
//
// Round-robin replica pick (COBALT_ASSIGN_ROUND_ROBIN): Step 1 is unchanged, but the j-th task
// of a group (expert, node) in ascending pair order goes to replica j mod |R_{e,n}|.  That
// depends on a running count, reproduced exactly without a serial pass: the kernel writes the
// group key e*N + n_te per task, the permutation-index machinery (chunk histograms, scan,
// stable rank) yields each task's rank inside its group, and a last kernel maps rank to slot.
#include "permute_index.cuh"
#include "token_core.cuh"

namespace cobalt {

constexpr int kAssignThreads = 512;       // the most a launch uses; small batches take half
constexpr int kRoundRobinThreads = 256;

template <int KT, int MODE>
__global__ void __launch_bounds__(kAssignThreads)
assign_kernel(LayoutView lv, const int32_t* __restrict__ topk_ids, const int32_t* __restrict__ src_rank,
              int32_t src_uniform, int64_t T, int32_t K_rt, uint32_t seed_lo, uint32_t seed_hi,
              int32_t* __restrict__ assigned_slot, uint32_t* __restrict__ slot_load,
              uint8_t* __restrict__ remote_nodes, unsigned long long* __restrict__ totals,
              const unsigned long long* __restrict__ seed_on_device, uint32_t* __restrict__ err_word)
{
    extern __shared__ __align__(16) uint32_t smem[];
    if (seed_on_device) {                               // the seed of this run, not of the capture
        const unsigned long long sd = __ldg(seed_on_device);
        seed_lo = static_cast<uint32_t>(sd);
        seed_hi = static_cast<uint32_t>(sd >> 32);
    }
    uint32_t* tab = smem;                               // lv.words, padded to a multiple of 4
    uint32_t* hist = smem + (lv.words + 3) / 4 * 4;     // lv.D (only when slot_load != nullptr)
    __shared__ unsigned long long cta_totals[2];
    constexpr int KMAX = TokenShape<KT>::KMAX;
    constexpr bool kCountSlots = (MODE != kAssignGroupKey);   // group keys are not slots yet

    const int K = (KT > 0) ? KT : K_rt;
    // the token's own loads go out first so that their latency overlaps the table staging
    const int64_t t = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    int32_t id[KMAX], out[KMAX];
    int32_t s_t = src_uniform;
    if (t < T) {
        load_token_ids<KT>(topk_ids, t, K, id);
        if (src_rank) s_t = __ldg(src_rank + t);
    }
    const TableView tv = stage_tables(lv, tab);
    if (kCountSlots && slot_load)
        for (int i = threadIdx.x; i < lv.D; i += blockDim.x) hist[i] = 0;
    if (threadIdx.x < 2) cta_totals[threadIdx.x] = 0;
    __syncthreads();

    uint32_t cost = 0, naive_cost = 0;
    if (t < T) {
        uint32_t bad = check_token_ids<KT>(id, K, lv.E);
        if (s_t < 0 || s_t >= lv.G) bad |= COBALT_DEVERR_BAD_SRC_RANK;
        if (bad) {
            flag_error(err_word, bad);
#pragma unroll
            for (int a = 0; a < KMAX; ++a) out[a] = -1;
        } else {
            assign_token<KT, MODE>(tv, id, K, s_t, static_cast<uint32_t>(t), seed_lo, seed_hi, out, cost, naive_cost);
            if (kCountSlots && slot_load) {
#pragma unroll
                for (int a = 0; a < KMAX; ++a)
                    if (a < K) atomicAdd(&hist[out[a]], 1u);
            }
        }
        store_token_slots<KT>(assigned_slot + t * K, out, K);
        if (remote_nodes) remote_nodes[t] = static_cast<uint8_t>(cost);
    }

    if (totals) {
        uint32_t c = cost, n = naive_cost;
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) {
            c += __shfl_xor_sync(0xFFFFFFFFu, c, off);
            n += __shfl_xor_sync(0xFFFFFFFFu, n, off);
        }
        if ((threadIdx.x & 31) == 0) {
            if (c) atomicAdd(&cta_totals[0], static_cast<unsigned long long>(c));
            if (n) atomicAdd(&cta_totals[1], static_cast<unsigned long long>(n));
        }
    }
    __syncthreads();
    wait_for_prior_kernel();   // slot_load / totals may still be being cleared by the kernel before this one
    if (kCountSlots && slot_load)
        for (int i = threadIdx.x; i < lv.D; i += blockDim.x)
            if (hist[i]) atomicAdd(&slot_load[i], hist[i]);
    if (totals && threadIdx.x < 2 && cta_totals[threadIdx.x])
        atomicAdd(&totals[threadIdx.x], cta_totals[threadIdx.x]);
}

// Round-robin pick, last step: key = e*N + n, rank = position of the task inside its group.
__global__ void __launch_bounds__(kRoundRobinThreads)
assign_round_robin_kernel(LayoutView lv, const int32_t* __restrict__ group_rank, int64_t P,
                          int32_t* __restrict__ key_to_slot, uint32_t* __restrict__ slot_load)
{
    extern __shared__ __align__(16) uint32_t smem[];
    uint32_t* tab = smem;
    uint32_t* hist = smem + (lv.words + 3) / 4 * 4;
    const TableView tv = stage_tables(lv, tab);
    if (slot_load)
        for (int i = threadIdx.x; i < lv.D; i += blockDim.x) hist[i] = 0;
    __syncthreads();
    const int64_t stride = static_cast<int64_t>(gridDim.x) * blockDim.x;
    for (int64_t p = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x; p < P; p += stride) {
        const int32_t key = key_to_slot[p];
        if (key < 0) continue;                       // a token that failed its checks
        const uint32_t e_n = tv.ent[key];
        const uint32_t j = static_cast<uint32_t>(__ldg(group_rank + p)) % ent_count(e_n);
        const int32_t slot = static_cast<int32_t>(tv.rlist[ent_offset(e_n) + j]);
        key_to_slot[p] = slot;
        if (slot_load) atomicAdd(&hist[slot], 1u);
    }
    __syncthreads();
    if (slot_load)
        for (int i = threadIdx.x; i < lv.D; i += blockDim.x)
            if (hist[i]) atomicAdd(&slot_load[i], hist[i]);
}

struct AssignArgs {
    const LayoutView* lv;
    const int32_t* ids;
    const int32_t* src;
    int32_t src_uniform;
    int64_t T;
    int32_t K;
    uint64_t seed;
    const unsigned long long* seed_on_device;
    int32_t* assigned_slot;
    uint32_t* slot_load;
    uint8_t* remote_nodes;
    uint64_t* totals;
    uint32_t* err_word;
    bool after_zeroing;
    cudaStream_t stream;
};

static size_t table_smem_bytes(const LayoutView& lv, bool with_hist)
{
    return (static_cast<size_t>(lv.words + 3) / 4 * 4 + (with_hist ? lv.D : 0)) * sizeof(uint32_t);
}

template <int KT, int MODE>
static int launch_assign(const AssignArgs& a)
{
    const LayoutView& lv = *a.lv;
    const size_t smem = table_smem_bytes(lv, a.slot_load != nullptr && MODE != kAssignGroupKey);
    auto kernel = assign_kernel<KT, MODE>;
    if (smem > 48 * 1024)
        COBALT_CUDA_TRY(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             static_cast<int>(smem)));
    cudaLaunchConfig_t cfg = {};
    cudaLaunchAttribute attr[1];
    // 512 threads per CTA once that still gives every SM a CTA (the tables are staged half as often and
    // the grid is one wave: 13.4 us against 15.5 us at 131 072 tokens); 256 below (9.6 us against 11.3 us
    // at 4 096 tokens)
    int n_sm = 0;
    const int rc_sm = sm_count(&n_sm);
    if (rc_sm != COBALT_OK) return rc_sm;
    const int threads = (a.T >= static_cast<int64_t>(kAssignThreads) * n_sm) ? kAssignThreads : kAssignThreads / 2;
    cfg.gridDim = dim3(static_cast<unsigned>((a.T + threads - 1) / threads));
    cfg.blockDim = dim3(threads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = a.stream;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    set_programmatic_launch(&attr[0], a.after_zeroing);
    COBALT_CUDA_TRY(cudaLaunchKernelEx(&cfg, kernel, lv, a.ids, a.src, a.src_uniform, a.T, a.K,
                                       static_cast<uint32_t>(a.seed & 0xFFFFFFFFu),
                                       static_cast<uint32_t>(a.seed >> 32), a.assigned_slot, a.slot_load,
                                       a.remote_nodes, reinterpret_cast<unsigned long long*>(a.totals),
                                       a.seed_on_device, a.err_word));
    return COBALT_OK;
}

template <int MODE>
static int dispatch_assign(const AssignArgs& a)
{
    switch (a.K) {
        case 1: return launch_assign<1, MODE>(a);
        case 2: return launch_assign<2, MODE>(a);
        case 4: return launch_assign<4, MODE>(a);
        case 6: return launch_assign<6, MODE>(a);
        case 8: return launch_assign<8, MODE>(a);
        case 10: return launch_assign<10, MODE>(a);
        case 12: return launch_assign<12, MODE>(a);
        case 16: return launch_assign<16, MODE>(a);
        default: return launch_assign<0, MODE>(a);
    }
}

// workspace layout of the round-robin mode
struct RoundRobinPlan {
    ChunkPlan chunks;
    int n_groups;             // E * N keys
    size_t rank_off, counts_off, offsets_off, err_off, hist_off, total;
};

static RoundRobinPlan plan_round_robin(const LayoutView& lv, int64_t T, int32_t K)
{
    RoundRobinPlan r;
    r.chunks = plan_chunks(T * K);
    r.n_groups = lv.E * lv.N;
    size_t off = 0;
    r.rank_off = off;    off += round_up(sizeof(int32_t) * static_cast<size_t>(T) * K, 256);
    r.counts_off = off;  off += round_up(sizeof(uint32_t) * r.n_groups, 256);
    r.offsets_off = off; off += round_up(sizeof(uint32_t) * (r.n_groups + 1), 256);
    r.err_off = off;     off += 256;
    r.hist_off = off;    off += round_up(sizeof(uint32_t) * static_cast<size_t>(r.n_groups) * r.chunks.n_chunks, 256);
    r.total = off;
    return r;
}

}  // namespace cobalt

using namespace cobalt;

extern "C" {

size_t cobalt_assign_workspace_bytes(const cobalt_layout_t* layout, int64_t T, int32_t K)
{
    // only the round-robin mode needs scratch (group ranks and the scan tables); the size is
    // reported for it so that one workspace serves every mode
    if (!layout || T < 0 || K < 1 || K > COBALT_MAX_TOPK || T * static_cast<int64_t>(K) >= (1ll << 31)) return 0;
    if (layout->view.E * layout->view.N > COBALT_MAX_DESTS) return 0;
    return plan_round_robin(layout->view, T, K).total;
}

int cobalt_assign(const cobalt_layout_t* layout, const int32_t* topk_ids, const int32_t* src_rank,
                  int32_t src_rank_uniform, int64_t T, int32_t K, uint64_t seed, int32_t* assigned_slot,
                  uint32_t* slot_load, uint8_t* remote_nodes, uint64_t* totals, uint32_t flags,
                  void* workspace, size_t workspace_bytes, cobalt_stream_t stream)
{
    if (!layout || T < 0 || K < 1) return COBALT_ERR_INVALID_ARG;
    if (K > COBALT_MAX_TOPK || T * static_cast<int64_t>(K) >= (1ll << 31)) return COBALT_ERR_UNSUPPORTED;
    const LayoutView& lv = layout->view;
    if (K > lv.E) return COBALT_ERR_INVALID_ARG;
    if (!src_rank && (src_rank_uniform < 0 || src_rank_uniform >= lv.G)) return COBALT_ERR_INVALID_ARG;
    if (T > 0 && (!topk_ids || !assigned_slot)) return COBALT_ERR_INVALID_ARG;
    if (!aligned16(topk_ids) || !aligned16(assigned_slot) || !aligned16(src_rank) || !aligned16(slot_load) ||
        !aligned16(totals) || !aligned16(workspace))
        return COBALT_ERR_INVALID_ARG;
    const bool seed_on_device = (flags & COBALT_SEED_ON_DEVICE) != 0;
    if (seed_on_device && (seed == 0 || (seed & 7u) != 0)) return COBALT_ERR_INVALID_ARG;
    const bool naive = (flags & COBALT_ASSIGN_NAIVE) != 0;
    const bool round_robin = (flags & COBALT_ASSIGN_ROUND_ROBIN) != 0 && !naive;
    RoundRobinPlan rr = {};
    if (round_robin) {
        if (lv.E * lv.N > COBALT_MAX_DESTS) return COBALT_ERR_UNSUPPORTED;
        rr = plan_round_robin(lv, T, K);
        if (!workspace || workspace_bytes < rr.total) return COBALT_ERR_WORKSPACE_TOO_SMALL;
    }
    int dev = 0;
    COBALT_CUDA_TRY(cudaGetDevice(&dev));
    if (dev != layout->device) return COBALT_ERR_INVALID_ARG;

    cudaStream_t s = static_cast<cudaStream_t>(stream);
    AssignArgs a;
    a.after_zeroing = false;
    int rc = launch_zero_words(slot_load, lv.D, reinterpret_cast<uint32_t*>(totals), 4, s, &a.after_zeroing);
    if (rc != COBALT_OK) return rc;
    if (T == 0) return COBALT_OK;

    a.lv = &lv; a.ids = topk_ids; a.src = src_rank; a.src_uniform = src_rank_uniform; a.T = T; a.K = K;
    a.seed = seed_on_device ? 0 : seed;
    a.seed_on_device = seed_on_device ? reinterpret_cast<const unsigned long long*>(static_cast<uintptr_t>(seed)) : nullptr;
    a.assigned_slot = assigned_slot; a.slot_load = slot_load; a.remote_nodes = remote_nodes;
    a.totals = totals; a.stream = s;
    rc = device_error_word(&a.err_word);
    if (rc != COBALT_OK) return rc;

    if (naive) return dispatch_assign<kAssignNaive>(a);
    if (!round_robin) return dispatch_assign<kAssignSlot>(a);

    // round robin: group keys -> rank inside the group (in pair order) -> replica rank mod |R|
    rc = dispatch_assign<kAssignGroupKey>(a);
    if (rc != COBALT_OK) return rc;
    uint8_t* ws = static_cast<uint8_t*>(workspace);
    int32_t* group_rank = reinterpret_cast<int32_t*>(ws + rr.rank_off);
    uint32_t* counts = reinterpret_cast<uint32_t*>(ws + rr.counts_off);
    uint32_t* offsets = reinterpret_cast<uint32_t*>(ws + rr.offsets_off);
    uint32_t* hist = reinterpret_cast<uint32_t*>(ws + rr.hist_off);
    // Tokens that failed their checks carry key -1; the histogram kernel skips such keys and
    // reports them in the error word it is given.  They were already reported by the kernel
    // above with the precise reason, so this second report goes to a scratch word.
    uint32_t* scratch_err = reinterpret_cast<uint32_t*>(ws + rr.err_off);
    const int64_t P = T * K;
    rc = launch_chunk_histograms(assigned_slot, P, rr.n_groups, rr.chunks, hist, scratch_err, s);
    if (rc != COBALT_OK) return rc;
    rc = launch_scan_and_rank(assigned_slot, P, rr.n_groups, rr.chunks, hist, counts, offsets, group_rank, nullptr, 1, s);
    if (rc != COBALT_OK) return rc;
    const size_t smem = table_smem_bytes(lv, slot_load != nullptr);
    if (smem > 48 * 1024)
        COBALT_CUDA_TRY(cudaFuncSetAttribute(assign_round_robin_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             static_cast<int>(smem)));
    int n_sm = 0;
    rc = sm_count(&n_sm);
    if (rc != COBALT_OK) return rc;
    int64_t grid = (P + kRoundRobinThreads - 1) / kRoundRobinThreads;
    if (grid > 8ll * n_sm) grid = 8ll * n_sm;
    assign_round_robin_kernel<<<static_cast<unsigned>(grid), kRoundRobinThreads, smem, s>>>(lv, group_rank, P, assigned_slot,
                                                                                       slot_load);
    COBALT_CUDA_TRY(cudaGetLastError());
    return COBALT_OK;
}

}  // extern "C"
