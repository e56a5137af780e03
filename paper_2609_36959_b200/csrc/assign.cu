// Stage 2: communication-aware task assignment (Section 3.3, Algorithm 1), one thread per token.
//
// The layout tables (R_{e,n}, N_e, primaries; a few KB) are staged once per CTA in shared
// memory.  Each thread keeps its token's K ids and remote masks in registers, finds b* by the
// ascending enumeration of (N-1)-bit masks (lines 5-8), draws the node and the replica with
// the counter hash, and writes its K slots with 8/16-byte stores.  Per-slot loads w_er are
// histogrammed in shared memory and merged with one integer reduction per slot and CTA; the
// Eq. 1 totals are reduced per warp and added once per CTA.  Integer adds commute, so the
// result does not depend on scheduling.
#include "common.cuh"

namespace cobalt {

constexpr int kAssignThreads = 256;

template <int KT>
__global__ void __launch_bounds__(kAssignThreads)
assign_kernel(LayoutView lv, const int32_t* __restrict__ topk_ids, const int32_t* __restrict__ src_rank,
              int32_t src_uniform, int64_t T, int32_t K_rt, uint32_t seed_lo, uint32_t seed_hi,
              int32_t* __restrict__ assigned_slot, uint32_t* __restrict__ slot_load,
              uint8_t* __restrict__ remote_nodes, unsigned long long* __restrict__ totals,
              uint32_t naive, uint32_t* __restrict__ err_word)
{
    extern __shared__ __align__(16) uint32_t smem[];
    uint32_t* tab = smem;                               // lv.words, padded to a multiple of 4
    uint32_t* hist = smem + (lv.words + 3) / 4 * 4;     // lv.D (only when slot_load != nullptr)
    __shared__ unsigned long long cta_totals[2];

    const int K = (KT > 0) ? KT : K_rt;
    {   // the blob is padded to whole 16-byte vectors
        const uint4* src = reinterpret_cast<const uint4*>(lv.blob);
        uint4* dst = reinterpret_cast<uint4*>(tab);
        const int n_vec = (lv.words + 3) / 4;
#pragma unroll 4
        for (int i = threadIdx.x; i < n_vec; i += blockDim.x) dst[i] = __ldg(src + i);
    }
    if (slot_load)
        for (int i = threadIdx.x; i < lv.D; i += blockDim.x) hist[i] = 0;
    if (threadIdx.x < 2) cta_totals[threadIdx.x] = 0;
    __syncthreads();

    const uint32_t* ent = tab + lv.ent_off();
    const uint32_t* primary = tab + lv.primary_off();
    const uint32_t* rlist = tab + lv.rlist_off();
    const uint32_t* nodes = tab + lv.nodes_off();
    const int N = lv.N;

    const int64_t t = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    uint32_t cost = 0, naive_cost = 0;

    if (t < T) {
        constexpr int KMAX = (KT > 0) ? KT : COBALT_MAX_TOPK;
        int32_t id[KMAX];
        const int32_t* row = topk_ids + t * K;
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

        const int32_t s_t = src_rank ? __ldg(src_rank + t) : src_uniform;
        uint32_t bad = 0;
        if (s_t < 0 || s_t >= lv.G) bad |= COBALT_DEVERR_BAD_SRC_RANK;
#pragma unroll
        for (int a = 0; a < KMAX; ++a) {
            if (a < K) {
                if (id[a] < 0 || id[a] >= lv.E) bad |= COBALT_DEVERR_BAD_EXPERT_ID;
#pragma unroll
                for (int b = 0; b < a; ++b)
                    if (id[b] == id[a]) bad |= COBALT_DEVERR_DUPLICATE_ID;
            }
        }

        int32_t out[KMAX];
        if (bad) {
            flag_error(err_word, bad);
#pragma unroll
            for (int a = 0; a < KMAX; ++a) out[a] = -1;
        } else {
            const int n_s = s_t / lv.Q;                       // N(s_t)
            const uint32_t src_bit = 1u << n_s;
            const uint32_t low = src_bit - 1u;

            // the naive rule's term of Eq. 1: distinct nodes of the primaries, source excluded
            uint32_t naive_nodes = 0;
#pragma unroll
            for (int a = 0; a < KMAX; ++a)
                if (a < K) naive_nodes |= 1u << (primary[id[a]] >> 24);
            naive_cost = __popc(naive_nodes & ~src_bit);

            if (naive) {
#pragma unroll
                for (int a = 0; a < KMAX; ++a)
                    if (a < K) out[a] = static_cast<int32_t>(primary[id[a]] & 0xFFFFFFu);
                cost = naive_cost;
            } else {
                // line 3-4: U_t and the remote masks; bit j <-> j-th node after skipping n_s.
                // m[a] == 0 marks an expert that is present on the source node.
                uint32_t m[KMAX];
                uint32_t any_remote = 0, common = 0xFFFFFFFFu;
#pragma unroll
                for (int a = 0; a < KMAX; ++a) {
                    if (a < K) {
                        const uint32_t held = nodes[id[a]];
                        m[a] = (held & src_bit) ? 0u : (((held >> (n_s + 1)) << n_s) | (held & low));
                        any_remote |= m[a];
                        if (m[a]) common &= m[a];
                    }
                }
                // lines 5-8: ascending b, strictly smaller popcount replaces b*.  A single node
                // covers U_t iff every mask has its bit, and the lowest such bit is the smallest
                // one-bit b; only otherwise are the masks with two or more bits enumerated.
                uint32_t b_star = 0;
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
                            for (int a = 0; a < KMAX; ++a)
                                if (a < K) feasible = feasible && (m[a] == 0 || (b & m[a]) != 0);
                            if (feasible) {
                                b_star = b;
                                best = pc;
                                if (pc == 2) break;  // one node is known not to suffice
                            }
                        }
                    }
                    cost = __popc(b_star);
                }
                // lines 9-16: node per expert, then a replica inside the node
#pragma unroll
                for (int a = 0; a < KMAX; ++a) {
                    if (a < K) {
                        int node = n_s;
                        if (m[a] != 0) {
                            // RandomNode: the i-th set bit of b* & m; a single candidate needs no draw
                            uint32_t c = b_star & m[a];
                            const uint32_t n_c = __popc(c);
                            if (n_c > 1) {
                                const uint32_t i = hash_index(
                                    route_hash(seed_lo, seed_hi, static_cast<uint32_t>(t), id[a], 0u), n_c);
                                for (uint32_t j = 0; j < i; ++j) c &= c - 1u;   // drop the i lowest set bits
                            }
                            const int bit = __ffs(c) - 1;
                            node = bit + (bit >= n_s ? 1 : 0);
                        }
                        // UniformChoice over R_{e,node}; floor(x * 1 / 2^32) = 0, so one replica needs no draw
                        const uint32_t e_n = ent[id[a] * N + node];
                        const uint32_t n_r = e_n & 0xFFu;
                        const uint32_t i = (n_r > 1) ? hash_index(
                            route_hash(seed_lo, seed_hi, static_cast<uint32_t>(t), id[a], 1u), n_r) : 0u;
                        out[a] = static_cast<int32_t>(rlist[(e_n >> 8) + i]);
                    }
                }
            }
            if (slot_load) {
#pragma unroll
                for (int a = 0; a < KMAX; ++a)
                    if (a < K) atomicAdd(&hist[out[a]], 1u);
            }
        }

        int32_t* dst = assigned_slot + t * K;
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
    if (slot_load)
        for (int i = threadIdx.x; i < lv.D; i += blockDim.x)
            if (hist[i]) atomicAdd(&slot_load[i], hist[i]);
    if (totals && threadIdx.x < 2 && cta_totals[threadIdx.x])
        atomicAdd(&totals[threadIdx.x], cta_totals[threadIdx.x]);
}

template <int KT>
static int launch_assign(const LayoutView& lv, const int32_t* ids, const int32_t* src, int32_t src_uniform,
                         int64_t T, int32_t K, uint64_t seed, int32_t* assigned_slot, uint32_t* slot_load,
                         uint8_t* remote_nodes, uint64_t* totals, uint32_t naive, uint32_t* err_word,
                         bool after_zeroing, cudaStream_t stream)
{
    const size_t smem = (static_cast<size_t>(lv.words + 3) / 4 * 4 + (slot_load ? lv.D : 0)) * sizeof(uint32_t);
    auto kernel = assign_kernel<KT>;
    if (smem > 48 * 1024)
        COBALT_CUDA_TRY(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             static_cast<int>(smem)));
    const unsigned grid = static_cast<unsigned>((T + kAssignThreads - 1) / kAssignThreads);
    cudaLaunchConfig_t cfg = {};
    cudaLaunchAttribute attr[1];
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(kAssignThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    set_programmatic_launch(&attr[0], after_zeroing);
    COBALT_CUDA_TRY(cudaLaunchKernelEx(&cfg, kernel, lv, ids, src, src_uniform, T, K,
                                       static_cast<uint32_t>(seed & 0xFFFFFFFFu), static_cast<uint32_t>(seed >> 32),
                                       assigned_slot, slot_load, remote_nodes,
                                       reinterpret_cast<unsigned long long*>(totals), naive, err_word));
    return COBALT_OK;
}

}  // namespace cobalt

using namespace cobalt;

extern "C" {

size_t cobalt_assign_workspace_bytes(const cobalt_layout_t* layout, int64_t T, int32_t K)
{
    (void)layout; (void)T; (void)K;
    return 0;  // the assignment keeps all temporaries on chip
}

int cobalt_assign(const cobalt_layout_t* layout, const int32_t* topk_ids, const int32_t* src_rank,
                  int32_t src_rank_uniform, int64_t T, int32_t K, uint64_t seed, int32_t* assigned_slot,
                  uint32_t* slot_load, uint8_t* remote_nodes, uint64_t* totals, uint32_t flags,
                  void* workspace, size_t workspace_bytes, cobalt_stream_t stream)
{
    (void)workspace; (void)workspace_bytes;
    if (!layout || T < 0 || K < 1) return COBALT_ERR_INVALID_ARG;
    if (K > COBALT_MAX_TOPK || T * static_cast<int64_t>(K) >= (1ll << 31)) return COBALT_ERR_UNSUPPORTED;
    const LayoutView& lv = layout->view;
    if (K > lv.E) return COBALT_ERR_INVALID_ARG;
    if (!src_rank && (src_rank_uniform < 0 || src_rank_uniform >= lv.G)) return COBALT_ERR_INVALID_ARG;
    if (T > 0 && (!topk_ids || !assigned_slot)) return COBALT_ERR_INVALID_ARG;
    if (!aligned16(topk_ids) || !aligned16(assigned_slot) || !aligned16(src_rank) || !aligned16(slot_load) ||
        !aligned16(totals))
        return COBALT_ERR_INVALID_ARG;
    int dev = 0;
    COBALT_CUDA_TRY(cudaGetDevice(&dev));
    if (dev != layout->device) return COBALT_ERR_INVALID_ARG;

    cudaStream_t s = static_cast<cudaStream_t>(stream);
    bool after_zeroing = false;
    int rc = launch_zero_words(slot_load, lv.D, reinterpret_cast<uint32_t*>(totals), 4, s, &after_zeroing);
    if (rc != COBALT_OK) return rc;
    if (T == 0) return COBALT_OK;

    uint32_t* err_word = nullptr;
    rc = device_error_word(&err_word);
    if (rc != COBALT_OK) return rc;
    const uint32_t naive = (flags & COBALT_ASSIGN_NAIVE) ? 1u : 0u;
#define COBALT_ASSIGN_CASE(KT)                                                                          \
    case KT:                                                                                            \
        return launch_assign<KT>(lv, topk_ids, src_rank, src_rank_uniform, T, K, seed, assigned_slot,   \
                                 slot_load, remote_nodes, totals, naive, err_word, after_zeroing, s)
    switch (K) {
        COBALT_ASSIGN_CASE(1);
        COBALT_ASSIGN_CASE(2);
        COBALT_ASSIGN_CASE(4);
        COBALT_ASSIGN_CASE(6);
        COBALT_ASSIGN_CASE(8);
        default:
            return launch_assign<0>(lv, topk_ids, src_rank, src_rank_uniform, T, K, seed, assigned_slot,
                                    slot_load, remote_nodes, totals, naive, err_word, after_zeroing, s);
    }
#undef COBALT_ASSIGN_CASE
}

}  // extern "C"
