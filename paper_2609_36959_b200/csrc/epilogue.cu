// Statistics epilogue (Section 3.2): exponential moving averages of the per-step counts, the
// Ochiai similarity of expert pairs (footnote of Section 1), and Stage 2 of the layout planner,
// the per-step intra-node greedy rebalancing of replicas (host code: the paper runs it on the
// CPU, overlapped with model computation; it touches a few hundred numbers).
#include <algorithm>
#include <cmath>
#include <new>
#include <vector>

#include "common.cuh"

namespace cobalt {

__global__ void __launch_bounds__(256)
ema_update_kernel(const uint32_t* __restrict__ counts, float* __restrict__ ema, int64_t n, float decay,
                  float one_minus_decay, int initialise)
{
    const int64_t stride = static_cast<int64_t>(gridDim.x) * blockDim.x;
    for (int64_t i = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x; i < n; i += stride) {
        const float c = static_cast<float>(counts[i]);
        ema[i] = initialise ? c : fmaf(decay, ema[i], one_minus_decay * c);
    }
}

__global__ void __launch_bounds__(256)
ochiai_kernel(const uint32_t* __restrict__ coact, int E, float* __restrict__ ochiai)
{
    const int64_t n = static_cast<int64_t>(E) * E;
    const int64_t stride = static_cast<int64_t>(gridDim.x) * blockDim.x;
    for (int64_t idx = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x; idx < n; idx += stride) {
        const int i = static_cast<int>(idx / E), j = static_cast<int>(idx - static_cast<int64_t>(i) * E);
        const float a = static_cast<float>(__ldg(coact + static_cast<size_t>(i) * E + i));
        const float b = static_cast<float>(__ldg(coact + static_cast<size_t>(j) * E + j));
        const float c = static_cast<float>(coact[idx]);
        // |A n B| / sqrt(|A| |B|); the square roots are taken separately so that the product cannot overflow
        ochiai[idx] = (a > 0.0f && b > 0.0f) ? c / (sqrtf(a) * sqrtf(b)) : 0.0f;
    }
}

static unsigned small_grid(int64_t n)
{
    int64_t g = (n + 255) / 256;
    if (g < 1) g = 1;
    if (g > 1184) g = 1184;
    return static_cast<unsigned>(g);
}

}  // namespace cobalt

using namespace cobalt;

extern "C" {

int cobalt_ema_update(const uint32_t* counts, float* ema, int64_t n, float decay, uint32_t flags,
                      cobalt_stream_t stream)
{
    if (n < 0 || !(decay >= 0.0f && decay <= 1.0f)) return COBALT_ERR_INVALID_ARG;
    if (n == 0) return COBALT_OK;
    if (!counts || !ema || !aligned16(counts) || !aligned16(ema)) return COBALT_ERR_INVALID_ARG;
    ema_update_kernel<<<small_grid(n), 256, 0, static_cast<cudaStream_t>(stream)>>>(
        counts, ema, n, decay, 1.0f - decay, (flags & COBALT_EMA_INITIALISE) ? 1 : 0);
    COBALT_CUDA_TRY(cudaGetLastError());
    return COBALT_OK;
}

int cobalt_ochiai(const uint32_t* coact, int32_t E, float* ochiai, cobalt_stream_t stream)
{
    if (E < 1 || !coact || !ochiai || !aligned16(coact) || !aligned16(ochiai)) return COBALT_ERR_INVALID_ARG;
    if (E > COBALT_MAX_EXPERTS) return COBALT_ERR_UNSUPPORTED;
    ochiai_kernel<<<small_grid(static_cast<int64_t>(E) * E), 256, 0, static_cast<cudaStream_t>(stream)>>>(coact, E,
                                                                                                         ochiai);
    COBALT_CUDA_TRY(cudaGetLastError());
    return COBALT_OK;
}

int cobalt_rebalance_intra_node(int32_t N, int32_t Q, int32_t S, int32_t E, const int32_t* slot_expert_host,
                                const float* slot_load_host, int32_t* new_slot_expert_host,
                                int32_t* moved_from_host, int32_t* nodes_kept_host)
{
    int rc = cobalt_layout_check(N, Q, S, E, slot_expert_host, nullptr);
    if (rc != COBALT_OK) return rc;
    if (!slot_load_host || !new_slot_expert_host) return COBALT_ERR_INVALID_ARG;
    // loads of occupied slots must be finite and non-negative: a NaN would leave the sort below
    // without a strict weak order
    for (int32_t d = 0; d < N * Q * S; ++d)
        if (slot_expert_host[d] >= 0 && !(slot_load_host[d] >= 0.0f && std::isfinite(slot_load_host[d])))
            return COBALT_ERR_INVALID_ARG;
    try {
    struct Replica {
        int32_t slot, expert;
        float load;
    };
    int32_t kept = 0;
    std::vector<Replica> replicas;
    std::vector<double> rank_load(Q);
    std::vector<std::vector<int32_t>> rank_has(Q);
    std::vector<int32_t> placed_rank, placed_pos;
    for (int32_t n = 0; n < N; ++n) {
        const int32_t lo = n * Q * S, hi = (n + 1) * Q * S;
        replicas.clear();
        for (int32_t d = lo; d < hi; ++d)
            if (slot_expert_host[d] >= 0) replicas.push_back({d, slot_expert_host[d], slot_load_host[d]});
        // longest first; ties by lower expert id, then lower old slot
        std::sort(replicas.begin(), replicas.end(), [](const Replica& a, const Replica& b) {
            if (a.load != b.load) return a.load > b.load;
            if (a.expert != b.expert) return a.expert < b.expert;
            return a.slot < b.slot;
        });
        std::fill(rank_load.begin(), rank_load.end(), 0.0);
        for (auto& h : rank_has) h.clear();
        placed_rank.assign(replicas.size(), -1);
        placed_pos.assign(replicas.size(), -1);
        bool ok = true;
        for (size_t i = 0; i < replicas.size() && ok; ++i) {
            int best = -1;
            for (int q = 0; q < Q; ++q) {
                if (static_cast<int32_t>(rank_has[q].size()) >= S) continue;   // (1+rho)E/G slots per rank
                if (std::find(rank_has[q].begin(), rank_has[q].end(), replicas[i].expert) != rank_has[q].end())
                    continue;                                                  // an expert at most once per rank
                if (best < 0 || rank_load[q] < rank_load[best]) best = q;
            }
            if (best < 0) {
                ok = false;
                break;
            }
            placed_rank[i] = best;
            placed_pos[i] = static_cast<int32_t>(rank_has[best].size());
            rank_has[best].push_back(replicas[i].expert);
            rank_load[best] += static_cast<double>(replicas[i].load);
        }
        for (int32_t d = lo; d < hi; ++d) {
            new_slot_expert_host[d] = ok ? -1 : slot_expert_host[d];
            if (moved_from_host) moved_from_host[d] = (ok || slot_expert_host[d] < 0) ? -1 : d;
        }
        if (!ok) {
            kept += 1;   // a replica found no admissible rank: this node keeps its placement
            continue;
        }
        for (size_t i = 0; i < replicas.size(); ++i) {
            const int32_t slot = (n * Q + placed_rank[i]) * S + placed_pos[i];
            new_slot_expert_host[slot] = replicas[i].expert;
            if (moved_from_host) moved_from_host[slot] = replicas[i].slot;
        }
    }
    if (nodes_kept_host) *nodes_kept_host = kept;
    } catch (const std::bad_alloc&) {
        return COBALT_ERR_HOST_ALLOC;
    }
    return COBALT_OK;
}

}  // extern "C"
