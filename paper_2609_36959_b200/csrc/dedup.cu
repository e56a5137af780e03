// Node-deduplicated send layout (Section 3.1, Eq. 1; Section 1 on node-level deduplication).
//
// With node-level deduplication a token crosses the network once per destination NODE and is
// forwarded to the ranks inside it, so the buffer that goes on the wire needs one row per
// (token, destination node), not one per (token, expert).  cobalt_dedup_index builds that layout
// from the assignment: a kernel marks, per token, the nodes its K slots live on as keys
// t*N + n -> n (or -1); the permutation-index kernels (chunk histograms, scan, stable rank) group
// those keys by node in ascending token order; a last kernel points every (token, expert) pair at
// the row it is forwarded from.  The rows themselves are moved by cobalt_permute_rows_block with
// N "copies" per token (absent nodes are skipped), and cobalt_forward_rows is the receiving
// node's expansion back to one row per pair.
#include "permute_index.cuh"

namespace cobalt {

constexpr int kDedupThreads = 256;

__global__ void __launch_bounds__(kDedupThreads)
dedup_keys_kernel(const int32_t* __restrict__ assigned_slot, const int32_t* __restrict__ src_rank,
                  int32_t src_uniform, int64_t T, int K, int N, int Q, int slots_per_node, int D,
                  int32_t* __restrict__ keys, unsigned long long* __restrict__ cross_rows,
                  uint32_t* __restrict__ err_word)
{
    const int64_t t = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    uint32_t cross = 0;
    if (t < T) {
        uint32_t mask = 0;
        bool bad = false;
        for (int k = 0; k < K; ++k) {
            const int32_t d = __ldg(assigned_slot + t * K + k);
            if (d >= 0 && d < D) mask |= 1u << (d / slots_per_node);
            else bad = true;
        }
        if (bad) flag_error(err_word, COBALT_DEVERR_BAD_SLOT);
        for (int n = 0; n < N; ++n) keys[t * N + n] = ((mask >> n) & 1u) ? n : -1;
        const int32_t s_t = src_rank ? __ldg(src_rank + t) : src_uniform;
        if (s_t >= 0 && s_t < N * Q) mask &= ~(1u << (s_t / Q));
        else flag_error(err_word, COBALT_DEVERR_BAD_SRC_RANK);
        cross = __popc(mask);
    }
    if (cross_rows) {
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) cross += __shfl_xor_sync(0xFFFFFFFFu, cross, off);
        wait_for_prior_kernel();   // the counter may still be being cleared by the kernel before this one
        if ((threadIdx.x & 31) == 0 && cross) atomicAdd(cross_rows, static_cast<unsigned long long>(cross));
    }
}

__global__ void __launch_bounds__(kDedupThreads)
dedup_forward_index_kernel(const int32_t* __restrict__ assigned_slot, const int32_t* __restrict__ node_row,
                           int64_t P, int K, int N, int slots_per_node, int D, int32_t* __restrict__ fwd_src_row)
{
    const int64_t stride = static_cast<int64_t>(gridDim.x) * blockDim.x;
    for (int64_t p = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x; p < P; p += stride) {
        const int32_t d = __ldg(assigned_slot + p);
        fwd_src_row[p] = (d >= 0 && d < D) ? __ldg(node_row + (p / K) * N + d / slots_per_node) : -1;
    }
}

struct DedupPlan {
    ChunkPlan chunks;
    size_t keys_off, err_off, hist_off, total;
};

static DedupPlan plan_dedup(int64_t T, int32_t N)
{
    DedupPlan d;
    d.chunks = plan_chunks(T * N);
    size_t off = 0;
    d.keys_off = off; off += round_up(sizeof(int32_t) * static_cast<size_t>(T) * N, 256);
    d.err_off = off;  off += 256;
    d.hist_off = off; off += round_up(sizeof(uint32_t) * static_cast<size_t>(N) * d.chunks.n_chunks, 256);
    d.total = off;
    return d;
}

}  // namespace cobalt

using namespace cobalt;

extern "C" {

size_t cobalt_dedup_workspace_bytes(int64_t T, int32_t K, int32_t num_nodes)
{
    if (T < 0 || K < 1 || num_nodes < 1 || num_nodes > COBALT_MAX_NODES || T * static_cast<int64_t>(K) >= (1ll << 31))
        return 0;
    return plan_dedup(T, num_nodes).total;
}

int cobalt_dedup_index(const int32_t* assigned_slot, const int32_t* src_rank, int32_t src_rank_uniform, int64_t T,
                       int32_t K, int32_t num_nodes, int32_t ranks_per_node, int32_t slots_per_rank,
                       uint32_t* node_counts, uint32_t* node_offsets, int32_t* node_row_of_token,
                       int32_t* fwd_src_row, uint64_t* cross_node_rows, void* workspace, size_t workspace_bytes,
                       cobalt_stream_t stream)
{
    const int32_t N = num_nodes, Q = ranks_per_node, S = slots_per_rank;
    if (T < 0 || K < 1 || N < 1 || Q < 1 || S < 1 || !node_counts || !node_offsets) return COBALT_ERR_INVALID_ARG;
    if (N > COBALT_MAX_NODES || K > COBALT_MAX_TOPK || static_cast<int64_t>(N) * Q * S > COBALT_MAX_DESTS ||
        T * static_cast<int64_t>(K) >= (1ll << 31) || T * static_cast<int64_t>(N) >= (1ll << 31))
        return COBALT_ERR_UNSUPPORTED;
    if (!src_rank && (src_rank_uniform < 0 || src_rank_uniform >= N * Q)) return COBALT_ERR_INVALID_ARG;
    if (T > 0 && (!assigned_slot || !node_row_of_token || !fwd_src_row)) return COBALT_ERR_INVALID_ARG;
    if (!aligned16(assigned_slot) || !aligned16(src_rank) || !aligned16(node_counts) || !aligned16(node_offsets) ||
        !aligned16(node_row_of_token) || !aligned16(fwd_src_row) || !aligned16(cross_node_rows) || !aligned16(workspace))
        return COBALT_ERR_INVALID_ARG;
    const DedupPlan plan = plan_dedup(T, N);
    if (!workspace || workspace_bytes < plan.total) return COBALT_ERR_WORKSPACE_TOO_SMALL;

    cudaStream_t s = static_cast<cudaStream_t>(stream);
    uint8_t* ws = static_cast<uint8_t*>(workspace);
    int32_t* keys = reinterpret_cast<int32_t*>(ws + plan.keys_off);
    uint32_t* scratch_err = reinterpret_cast<uint32_t*>(ws + plan.err_off);   // absent nodes are not errors
    uint32_t* hist = reinterpret_cast<uint32_t*>(ws + plan.hist_off);
    uint32_t* err_word = nullptr;
    int rc = device_error_word(&err_word);
    if (rc != COBALT_OK) return rc;
    bool after_zeroing = false;
    rc = launch_zero_words(reinterpret_cast<uint32_t*>(cross_node_rows), 2, nullptr, 0, s, &after_zeroing);
    if (rc != COBALT_OK) return rc;

    const int D = N * Q * S;
    if (T > 0) {
        cudaLaunchConfig_t cfg = {};
        cudaLaunchAttribute attr[1];
        set_programmatic_launch(&attr[0], after_zeroing);
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        cfg.stream = s;
        cfg.blockDim = dim3(kDedupThreads);
        cfg.gridDim = dim3(static_cast<unsigned>((T + kDedupThreads - 1) / kDedupThreads));
        COBALT_CUDA_TRY(cudaLaunchKernelEx(&cfg, dedup_keys_kernel, assigned_slot, src_rank, src_rank_uniform, T,
                                           static_cast<int>(K), static_cast<int>(N), static_cast<int>(Q),
                                           static_cast<int>(S * Q), D, keys,
                                           reinterpret_cast<unsigned long long*>(cross_node_rows), err_word));
    }
    rc = launch_chunk_histograms(keys, T * N, N, plan.chunks, hist, scratch_err, s);
    if (rc != COBALT_OK) return rc;
    rc = launch_scan_and_rank(keys, T * N, N, plan.chunks, hist, node_counts, node_offsets, node_row_of_token, nullptr,
                              0, s);
    if (rc != COBALT_OK) return rc;
    if (T > 0) {
        const int64_t P = T * K;
        int n_sm = 0;
        rc = sm_count(&n_sm);
        if (rc != COBALT_OK) return rc;
        int64_t grid = (P + kDedupThreads - 1) / kDedupThreads;
        if (grid > 16ll * n_sm) grid = 16ll * n_sm;
        dedup_forward_index_kernel<<<static_cast<unsigned>(grid), kDedupThreads, 0, s>>>(
            assigned_slot, node_row_of_token, P, K, N, S * Q, D, fwd_src_row);
        COBALT_CUDA_TRY(cudaGetLastError());
    }
    return COBALT_OK;
}

int cobalt_forward_rows(const void* dedup_send, const int32_t* fwd_src_row, const int32_t* row_of_pair, int64_t P,
                        int32_t H, void* recv, int64_t src_rows, int64_t dst_rows, cobalt_stream_t stream)
{
    if (P < 0 || H < 1 || src_rows < 0 || dst_rows < 0) return COBALT_ERR_INVALID_ARG;
    if (H % 8 != 0 || P >= (1ll << 31) || src_rows >= (1ll << 31) || dst_rows >= (1ll << 31)) return COBALT_ERR_UNSUPPORTED;
    if (P == 0) return COBALT_OK;
    if (!dedup_send || !fwd_src_row || !row_of_pair || !recv) return COBALT_ERR_INVALID_ARG;
    if (!aligned16(dedup_send) || !aligned16(recv) || !aligned16(fwd_src_row) || !aligned16(row_of_pair))
        return COBALT_ERR_INVALID_ARG;
    return launch_row_gather_scatter(dedup_send, fwd_src_row, row_of_pair, P, src_rows, dst_rows, H, recv,
                                     static_cast<cudaStream_t>(stream));
}

}  // extern "C"
