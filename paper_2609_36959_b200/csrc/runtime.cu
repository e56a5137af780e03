// Status codes, the device error word and the expert-layout handle.
#include <stdlib.h>

#include <map>
#include <mutex>
#include <new>
#include <utility>
#include <vector>

#include "common.cuh"

namespace cobalt {

static thread_local int g_last_cuda_error = 0;

int record_cuda_error(cudaError_t err)
{
    g_last_cuda_error = static_cast<int>(err);
    (void)cudaGetLastError();  // clear the sticky-free error state of the runtime
    return COBALT_ERR_CUDA;
}

// One error word per device: kernels OR COBALT_DEVERR_* bits into it instead of trapping.
__device__ uint32_t g_device_error_word = 0;

int device_error_word(uint32_t** out)
{
    static uint32_t* cached[64] = {nullptr};      // the symbol's address on each device
    int dev = 0;
    COBALT_CUDA_TRY(cudaGetDevice(&dev));
    if (dev >= 0 && dev < 64 && cached[dev]) {
        *out = cached[dev];
        return COBALT_OK;
    }
    void* p = nullptr;
    COBALT_CUDA_TRY(cudaGetSymbolAddress(&p, g_device_error_word));
    if (dev >= 0 && dev < 64) cached[dev] = static_cast<uint32_t*>(p);
    *out = static_cast<uint32_t*>(p);
    return COBALT_OK;
}

int ensure_kernel_attributes(const void* kernel, size_t bytes, bool non_portable_cluster)
{
    static std::mutex lock;
    static std::map<std::pair<const void*, int>, size_t> granted;   // (kernel, device) -> bytes + 1 once set up
    int dev = 0;
    COBALT_CUDA_TRY(cudaGetDevice(&dev));
    const auto key = std::make_pair(kernel, dev);
    {
        std::lock_guard<std::mutex> guard(lock);
        auto it = granted.find(key);
        if (it != granted.end() && it->second > bytes) return COBALT_OK;
    }
    if (bytes > 48 * 1024)
        COBALT_CUDA_TRY(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(bytes)));
    if (non_portable_cluster)
        COBALT_CUDA_TRY(cudaFuncSetAttribute(kernel, cudaFuncAttributeNonPortableClusterSizeAllowed, 1));
    std::lock_guard<std::mutex> guard(lock);
    size_t& have = granted[key];
    if (have < bytes + 1) have = bytes + 1;
    return COBALT_OK;
}

int sm_count(int* out)
{
    static int cached[64] = {0};
    int dev = 0;
    COBALT_CUDA_TRY(cudaGetDevice(&dev));
    if (dev >= 0 && dev < 64 && cached[dev] > 0) {
        *out = cached[dev];
        return COBALT_OK;
    }
    int n = 0;
    COBALT_CUDA_TRY(cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev));
    if (dev >= 0 && dev < 64) cached[dev] = n;
    *out = n;
    return COBALT_OK;
}

// Host-side validation + table construction shared by cobalt_layout_check / _create.
// Fills `blob` (see LayoutView) when it is non-null.
static int build_tables(int32_t N, int32_t Q, int32_t S, int32_t E, const int32_t* slot_expert,
                        const int32_t* primary_in, LayoutView* view, std::vector<uint32_t>* blob)
{
    if (!slot_expert || N < 1 || Q < 1 || S < 1 || E < 1) return COBALT_ERR_INVALID_ARG;
    if (N > COBALT_MAX_NODES || E > COBALT_MAX_EXPERTS || Q > COBALT_MAX_RANKS_PER_NODE) return COBALT_ERR_UNSUPPORTED;
    const int64_t D64 = static_cast<int64_t>(N) * Q * S;
    if (D64 > COBALT_MAX_DESTS) return COBALT_ERR_UNSUPPORTED;
    const int32_t G = N * Q, D = static_cast<int32_t>(D64);

    // group sizes |R_{e,n}| and the duplicate-on-rank check
    std::vector<int32_t> count(static_cast<size_t>(E) * N, 0);
    int32_t n_replicas = 0;
    for (int32_t r = 0; r < G; ++r) {
        for (int32_t j = 0; j < S; ++j) {
            const int32_t e = slot_expert[r * S + j];
            if (e == -1) continue;
            if (e < 0 || e >= E) return COBALT_ERR_INVALID_ARG;
            for (int32_t j2 = 0; j2 < j; ++j2)
                if (slot_expert[r * S + j2] == e) return COBALT_ERR_INVALID_ARG;
            count[static_cast<size_t>(e) * N + r / Q] += 1;
            n_replicas += 1;
        }
    }
    std::vector<int32_t> offset(static_cast<size_t>(E) * N, 0);
    int32_t running = 0;
    for (int32_t e = 0; e < E; ++e) {
        int32_t total = 0;
        for (int32_t n = 0; n < N; ++n) {
            offset[static_cast<size_t>(e) * N + n] = running;
            running += count[static_cast<size_t>(e) * N + n];
            total += count[static_cast<size_t>(e) * N + n];
        }
        if (total == 0) return COBALT_ERR_INVALID_ARG;  // Eq. 2: at least one replica per expert
    }
    if (primary_in) {
        for (int32_t e = 0; e < E; ++e) {
            const int32_t d = primary_in[e];
            if (d < 0 || d >= D || slot_expert[d] != e) return COBALT_ERR_INVALID_ARG;
        }
    }

    view->N = N; view->Q = Q; view->S = S; view->E = E; view->G = G; view->D = D;
    view->n_replicas = n_replicas;
    view->words = E * N + E + n_replicas + kCoverTableWords;
    view->blob = nullptr;
    // s / Q by multiplication, verified for every source rank
    view->q_inverse = (1u << 20) / static_cast<uint32_t>(Q) + 1u;
    for (int32_t s = 0; s < G; ++s)
        if (static_cast<int32_t>((static_cast<uint64_t>(s) * view->q_inverse) >> 20) != s / Q) return COBALT_ERR_UNSUPPORTED;
    if (!blob) return COBALT_OK;

    blob->assign(static_cast<size_t>(view->words + 3) / 4 * 4, 0u);   // whole 16-byte vectors
    uint32_t* ent = blob->data() + view->ent_off();
    uint32_t* primary = blob->data() + view->primary_off();
    uint32_t* rlist = blob->data() + view->rlist_off();
    uint8_t* cover = reinterpret_cast<uint8_t*>(blob->data() + view->cover_off());
    std::vector<int32_t> fill(static_cast<size_t>(E) * N, 0);
    std::vector<uint32_t> nodes(static_cast<size_t>(E), 0u);          // N_e as a bitmask over nodes
    for (int32_t e = 0; e < E; ++e) primary[e] = 0xFFFFFFFFu;
    for (int32_t d = 0; d < D; ++d) {  // ascending slot id => every R_{e,n} list is ascending
        const int32_t e = slot_expert[d];
        if (e < 0) continue;
        const int32_t n = d / (S * Q);
        const size_t en = static_cast<size_t>(e) * N + n;
        rlist[offset[en] + fill[en]] = static_cast<uint32_t>(d);
        fill[en] += 1;
        nodes[e] |= 1u << n;
        if (primary[e] == 0xFFFFFFFFu) primary[e] = static_cast<uint32_t>(d);
    }
    if (primary_in)
        for (int32_t e = 0; e < E; ++e) primary[e] = static_cast<uint32_t>(primary_in[e]);
    for (int32_t e = 0; e < E; ++e) {
        const uint32_t primary_node = primary[e] / static_cast<uint32_t>(S * Q);
        for (int32_t n = 0; n < N; ++n) {
            // the remote mask of e for a token whose source node is n: the nodes holding e with node n
            // taken out of the numbering; 0 when n holds e (the expert then runs on the source node)
            uint32_t m = 0;
            if (!(nodes[e] & (1u << n))) m = ((nodes[e] >> (n + 1)) << n) | (nodes[e] & ((1u << n) - 1u));
            const size_t en = static_cast<size_t>(e) * N + n;
            ent[en] = static_cast<uint32_t>(count[en]) | (static_cast<uint32_t>(offset[en]) << kEntCountBits) |
                      (m << kEntMaskShift) | (primary_node << kEntPrimaryNodeShift);
        }
    }
    // Smallest cover for every set of mask values (N <= 4: values 1 .. 2^(N-1)-1, at most seven), found
    // with Algorithm 1's own search: candidates b ascend from 0, a candidate replaces the best so far
    // only when it covers every mask of the set with strictly fewer nodes; the search starts from the
    // set of all remote nodes.
    if (N <= 4) {
        const uint32_t full = (1u << (N - 1)) - 1u;
        for (uint32_t present = 0; present < 128u; ++present) {
            uint32_t best = full;
            for (uint32_t b = 0; b < full; ++b) {
                bool covers = true;
                for (uint32_t v = 1; v <= 7u; ++v)
                    if ((present & (1u << (v - 1))) && v <= full && (b & v) == 0) covers = false;
                if (covers && __builtin_popcount(b) < __builtin_popcount(best)) best = b;
            }
            cover[present] = static_cast<uint8_t>(best);
        }
    }
    return COBALT_OK;
}

}  // namespace cobalt

using namespace cobalt;

extern "C" {

const char* cobalt_status_string(int status)
{
    switch (status) {
        case COBALT_OK: return "ok";
        case COBALT_ERR_INVALID_ARG: return "invalid argument";
        case COBALT_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
        case COBALT_ERR_UNSUPPORTED: return "outside the supported size envelope";
        case COBALT_ERR_CUDA: return "CUDA runtime error";
        case COBALT_ERR_SCRATCH_LIMIT: return "problem exceeds the built-in scratch of the no-allocation entry point";
        case COBALT_ERR_HOST_ALLOC: return "host memory allocation failed";
        default: return "unknown status";
    }
}

int cobalt_version(void) { return COBALT_VERSION; }

int cobalt_last_cuda_error(void) { return g_last_cuda_error; }

int cobalt_layout_check(int32_t N, int32_t Q, int32_t S, int32_t E, const int32_t* slot_expert_host,
                        const int32_t* primary_slot_host)
{
    LayoutView view;
    try {
        return build_tables(N, Q, S, E, slot_expert_host, primary_slot_host, &view, nullptr);
    } catch (const std::bad_alloc&) {
        return COBALT_ERR_HOST_ALLOC;
    }
}

int cobalt_layout_create(cobalt_layout_t** out, int32_t N, int32_t Q, int32_t S, int32_t E,
                         const int32_t* slot_expert_host, const int32_t* primary_slot_host)
{
    if (!out) return COBALT_ERR_INVALID_ARG;
    *out = nullptr;
    LayoutView view;
    std::vector<uint32_t> blob;
    int rc = COBALT_OK;
    try {
        rc = build_tables(N, Q, S, E, slot_expert_host, primary_slot_host, &view, &blob);
    } catch (const std::bad_alloc&) {
        return COBALT_ERR_HOST_ALLOC;
    }
    if (rc != COBALT_OK) return rc;
    int dev = 0;
    COBALT_CUDA_TRY(cudaGetDevice(&dev));
    void* dptr = nullptr;
    COBALT_CUDA_TRY(cudaMalloc(&dptr, blob.size() * sizeof(uint32_t)));
    cudaError_t err = cudaMemcpy(dptr, blob.data(), blob.size() * sizeof(uint32_t), cudaMemcpyHostToDevice);
    if (err != cudaSuccess) {
        cudaFree(dptr);
        return record_cuda_error(err);
    }
    cobalt_layout* h = static_cast<cobalt_layout*>(malloc(sizeof(cobalt_layout)));
    if (!h) {
        cudaFree(dptr);
        return COBALT_ERR_HOST_ALLOC;
    }
    view.blob = static_cast<const uint32_t*>(dptr);
    h->view = view;
    h->device = dev;
    *out = h;
    return COBALT_OK;
}

int cobalt_layout_destroy(cobalt_layout_t* layout)
{
    if (!layout) return COBALT_OK;
    cudaError_t err = cudaFree(const_cast<uint32_t*>(layout->view.blob));
    free(layout);
    if (err != cudaSuccess) return record_cuda_error(err);
    return COBALT_OK;
}

int32_t cobalt_layout_num_dests(const cobalt_layout_t* layout) { return layout ? layout->view.D : 0; }

int cobalt_read_and_clear_device_error(uint32_t* out_bits_host, cobalt_stream_t stream)
{
    if (!out_bits_host) return COBALT_ERR_INVALID_ARG;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    uint32_t* word = nullptr;
    int rc = device_error_word(&word);
    if (rc != COBALT_OK) return rc;
    COBALT_CUDA_TRY(cudaMemcpyAsync(out_bits_host, word, sizeof(uint32_t), cudaMemcpyDeviceToHost, s));
    COBALT_CUDA_TRY(cudaMemsetAsync(word, 0, sizeof(uint32_t), s));
    COBALT_CUDA_TRY(cudaStreamSynchronize(s));
    return COBALT_OK;
}

}  // extern "C"
