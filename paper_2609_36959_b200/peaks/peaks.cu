// Measurement kernels: the shared-memory atomic rate and the instruction issue rate of an SM
// (see cobalt_peaks.h).  Separate from the routing library; only the benchmark loads this.
#include <cuda_runtime.h>
#include <stdint.h>

#include <algorithm>
#include <vector>

#include "cobalt_peaks.h"

namespace {

constexpr int kThreads = 1024;
constexpr int kMaxK = 16;

#define PEAKS_TRY(expr)                                  \
    do {                                                 \
        cudaError_t err__ = (expr);                      \
        if (err__ != cudaSuccess) return static_cast<int>(err__); \
    } while (0)

// pattern 0: lane l of every warp adds to word (warp * 32 + l): its own bank, its own address
__global__ void __launch_bounds__(kThreads) atomics_conflict_free_kernel(int repeats, long long* cycles, uint32_t* sink)
{
    __shared__ uint32_t tile[kThreads];
    tile[threadIdx.x] = 0;
    __syncthreads();
    const long long t0 = clock64();
    for (int r = 0; r < repeats; ++r) {
#pragma unroll
        for (int i = 0; i < 32; ++i) atomicAdd(&tile[(threadIdx.x + 32 * i) & (kThreads - 1)], 1u);
    }
    __syncthreads();
    const long long t1 = clock64();
    if (threadIdx.x == 0) cycles[blockIdx.x] = t1 - t0;
    if (tile[threadIdx.x] == 0xFFFFFFFFu) sink[0] = 1;
}

// pattern 1: the statistics kernel's adds (sorted ids, triangle of 16-bit counters, two per word)
template <int K>
__global__ void __launch_bounds__(kThreads)
atomics_stats_pattern_kernel(const int32_t* __restrict__ ids, long long T, int E, int tokens_per_cta, int repeats,
                             long long* cycles, uint32_t* sink)
{
    extern __shared__ __align__(16) uint32_t tri[];
    const int n_words = (E * (E + 1) / 2 + 1) / 2;
    for (int i = threadIdx.x; i < n_words; i += kThreads) tri[i] = 0;
    // the CTA's tokens in registers first, so that only the adds are inside the timed region
    const long long t_lo = static_cast<long long>(blockIdx.x) * tokens_per_cta;
    const long long t = t_lo + threadIdx.x;
    const bool has = threadIdx.x < tokens_per_cta && t < T;
    int s[K];
#pragma unroll
    for (int a = 0; a < K; ++a) s[a] = has ? ids[t * K + a] : 0;
#pragma unroll
    for (int pass = 0; pass < K; ++pass)
#pragma unroll
        for (int a = pass & 1; a + 1 < K; a += 2) {
            const int lo = min(s[a], s[a + 1]), hi = max(s[a], s[a + 1]);
            s[a] = lo;
            s[a + 1] = hi;
        }
    __syncthreads();
    const long long t0 = clock64();
    for (int r = 0; r < repeats; ++r) {
        if (has) {
#pragma unroll
            for (int b = 0; b < K; ++b) {
                const int row = s[b] * (s[b] + 1) / 2;
#pragma unroll
                for (int a = 0; a <= b; ++a) {
                    const int idx = row + s[a];
                    atomicAdd(&tri[idx >> 1], (idx & 1) ? 0x10000u : 1u);
                }
            }
        }
    }
    __syncthreads();
    const long long t1 = clock64();
    if (threadIdx.x == 0) cycles[blockIdx.x] = t1 - t0;
    if (tri[threadIdx.x % n_words] == 0xFFFFFFFFu && repeats < 0) sink[0] = 1;
}

// eight independent chains of integer arithmetic per thread, no memory access.
// kMix 0: add, logic, shift only (three instructions per step): the issue rate itself.
// kMix 1: multiply-add, shift, logic (three per step): the hashing of Algorithm 1's draws, where every
//         third instruction is a 32-bit multiply.
template <int kMix>
__global__ void __launch_bounds__(kThreads) issue_rate_kernel(int repeats, long long* cycles, uint32_t* sink)
{
    uint32_t x[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) x[i] = threadIdx.x * 2654435761u + i;
    __syncthreads();
    const long long t0 = clock64();
    for (int r = 0; r < repeats; ++r) {
#pragma unroll
        for (int u = 0; u < 8; ++u) {
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                if (kMix == 1) x[i] = x[i] * 0x9E3779B9u + 0x7F4A7C15u;   // multiply-add
                else x[i] = x[i] + 0x7F4A7C15u;                           // add
                x[i] ^= x[i] >> 15;                                       // shift, logic
            }
        }
    }
    __syncthreads();
    const long long t1 = clock64();
    if (threadIdx.x == 0) cycles[blockIdx.x] = t1 - t0;
    uint32_t acc = 0;
#pragma unroll
    for (int i = 0; i < 8; ++i) acc ^= x[i];
    if (acc == 0x12345678u) sink[0] = acc;
}

struct Scratch {
    long long* cycles = nullptr;
    uint32_t* sink = nullptr;
    int n_sm = 0;
    ~Scratch()
    {
        if (cycles) cudaFree(cycles);
        if (sink) cudaFree(sink);
    }
};

int make_scratch(Scratch* s)
{
    int dev = 0;
    PEAKS_TRY(cudaGetDevice(&dev));
    PEAKS_TRY(cudaDeviceGetAttribute(&s->n_sm, cudaDevAttrMultiProcessorCount, dev));
    PEAKS_TRY(cudaMalloc(&s->cycles, sizeof(long long) * s->n_sm));
    PEAKS_TRY(cudaMalloc(&s->sink, sizeof(uint32_t)));
    return 0;
}

int slowest_cta(const Scratch& s, long long* out)
{
    std::vector<long long> h(s.n_sm);
    PEAKS_TRY(cudaMemcpy(h.data(), s.cycles, sizeof(long long) * s.n_sm, cudaMemcpyDeviceToHost));
    *out = *std::max_element(h.begin(), h.end());
    return 0;
}

template <int K>
int run_stats_pattern(const int32_t* ids, int64_t T, int E, int repeats, const Scratch& s, double* out)
{
    const size_t smem = (static_cast<size_t>(E) * (E + 1) / 2 + 1) / 2 * sizeof(uint32_t);
    auto kernel = atomics_stats_pattern_kernel<K>;
    if (smem > 48 * 1024)
        PEAKS_TRY(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem)));
    // the tokens of one CTA of the routing kernels: T spread over the SMs, at most one per thread
    int per_cta = static_cast<int>(std::min<int64_t>(kThreads, (T + s.n_sm - 1) / s.n_sm));
    if (per_cta < 1) per_cta = 1;
    long long best = 0;
    for (int it = 0; it < 5; ++it) {                     // the last (warm) run counts
        kernel<<<s.n_sm, kThreads, smem>>>(ids, T, E, per_cta, repeats, s.cycles, s.sink);
        PEAKS_TRY(cudaGetLastError());
        PEAKS_TRY(cudaDeviceSynchronize());
        int rc = slowest_cta(s, &best);
        if (rc) return rc;
    }
    const int64_t tokens = std::min<int64_t>(T, static_cast<int64_t>(per_cta) * s.n_sm);
    const double adds_per_sm = static_cast<double>(tokens) / s.n_sm * (K * (K + 1) / 2) * repeats;
    *out = adds_per_sm / static_cast<double>(best);
    return 0;
}

}  // namespace

extern "C" {

int cobalt_peak_shared_atomics(int pattern, const int32_t* topk_ids, int64_t T, int32_t K, int32_t E, int32_t repeats,
                               double* adds_per_clock_host)
{
    if (!adds_per_clock_host || repeats < 1) return static_cast<int>(cudaErrorInvalidValue);
    Scratch s;
    int rc = make_scratch(&s);
    if (rc) return rc;
    if (pattern == 0) {
        long long best = 0;
        for (int it = 0; it < 5; ++it) {
            atomics_conflict_free_kernel<<<s.n_sm, kThreads>>>(repeats, s.cycles, s.sink);
            PEAKS_TRY(cudaGetLastError());
            PEAKS_TRY(cudaDeviceSynchronize());
            rc = slowest_cta(s, &best);
            if (rc) return rc;
        }
        *adds_per_clock_host = static_cast<double>(kThreads) * 32.0 * repeats / static_cast<double>(best);
        return 0;
    }
    if (pattern != 1 || !topk_ids || T < 1 || K < 1 || K > kMaxK || E < K || E > 600)
        return static_cast<int>(cudaErrorInvalidValue);
    switch (K) {
        case 1: return run_stats_pattern<1>(topk_ids, T, E, repeats, s, adds_per_clock_host);
        case 2: return run_stats_pattern<2>(topk_ids, T, E, repeats, s, adds_per_clock_host);
        case 4: return run_stats_pattern<4>(topk_ids, T, E, repeats, s, adds_per_clock_host);
        case 6: return run_stats_pattern<6>(topk_ids, T, E, repeats, s, adds_per_clock_host);
        case 8: return run_stats_pattern<8>(topk_ids, T, E, repeats, s, adds_per_clock_host);
        default: return static_cast<int>(cudaErrorInvalidValue);      // the benchmark configs use these K
    }
}

int cobalt_peak_issue_rate(int32_t mix, int32_t repeats, double* warp_instructions_per_clock_host)
{
    if (!warp_instructions_per_clock_host || repeats < 1 || mix < 0 || mix > 1) return static_cast<int>(cudaErrorInvalidValue);
    Scratch s;
    int rc = make_scratch(&s);
    if (rc) return rc;
    long long best = 0;
    for (int it = 0; it < 5; ++it) {
        if (mix == 1) issue_rate_kernel<1><<<s.n_sm, kThreads>>>(repeats, s.cycles, s.sink);
        else issue_rate_kernel<0><<<s.n_sm, kThreads>>>(repeats, s.cycles, s.sink);
        PEAKS_TRY(cudaGetLastError());
        PEAKS_TRY(cudaDeviceSynchronize());
        rc = slowest_cta(s, &best);
        if (rc) return rc;
    }
    // per thread and repeat: 8 x 8 x three instructions = 192; 32 warps per SM
    *warp_instructions_per_clock_host = 192.0 * repeats * (kThreads / 32) / static_cast<double>(best);
    return 0;
}

}  // extern "C"
