// Stage 4: inverse permutation + gate-weighted sum (Fig. 1, "Weighted sum").
//
//   y[t][h] = bf16( sum_{k<K} g[t][k] * float(out[row_of_pair[t*K+k]][h]) )
//
// Read-dominated streaming kernel: a thread owns one 16-byte vector (8 bf16 columns) of a
// token, issues its K gathered row loads back to back (K * 16 bytes in flight per thread),
// accumulates in fp32 in ascending k and stores one 16-byte vector.  Rows are read once and
// written once, so both directions bypass L1 allocation.
#include <cuda_bf16.h>

#include "common.cuh"

namespace cobalt {

constexpr int kCombineThreads = 256;

__device__ __forceinline__ void fma_bf16x2(float& a0, float& a1, uint32_t packed, float w)
{
    a0 = fmaf(w, __uint_as_float(packed << 16), a0);
    a1 = fmaf(w, __uint_as_float(packed & 0xFFFF0000u), a1);
}

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi)
{
    const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<const uint32_t*>(&v);
}

// kUnit: no gate weights, the plain sum of the K rows (the adjoint of the dispatch gather).
template <int KT, bool kUnit>
__global__ void __launch_bounds__(kCombineThreads)
combine_kernel(const uint4* __restrict__ out, const int32_t* __restrict__ row_of_pair,
               const float* __restrict__ gate_w, int64_t T, int K_rt, int n_vec, int64_t P,
               uint4* __restrict__ y, uint32_t* __restrict__ err_word)
{
    constexpr int KMAX = (KT > 0) ? KT : COBALT_MAX_TOPK;
    const int K = (KT > 0) ? KT : K_rt;
    for (int64_t t = blockIdx.x; t < T; t += gridDim.x) {
        int64_t row[KMAX];
        float w[KMAX];
#pragma unroll
        for (int k = 0; k < KMAX; ++k) {
            if (k < K) {
                const int32_t r = __ldg(row_of_pair + t * K + k);
                const bool valid = (r >= 0 && r < P);
                row[k] = valid ? static_cast<int64_t>(r) * n_vec : -1;
                w[k] = valid ? (kUnit ? 1.0f : __ldg(gate_w + t * K + k)) : 0.0f;
                if (!valid && threadIdx.x == 0) flag_error(err_word, COBALT_DEVERR_BAD_SLOT);
            }
        }
        for (int v = threadIdx.x; v < n_vec; v += blockDim.x) {
            uint4 val[KMAX];
#pragma unroll
            for (int k = 0; k < KMAX; ++k)
                if (k < K) val[k] = (row[k] >= 0) ? ld_stream16(out + row[k] + v) : make_uint4(0, 0, 0, 0);
            float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
#pragma unroll
            for (int k = 0; k < KMAX; ++k) {
                if (k < K) {
                    fma_bf16x2(acc[0], acc[1], val[k].x, w[k]);
                    fma_bf16x2(acc[2], acc[3], val[k].y, w[k]);
                    fma_bf16x2(acc[4], acc[5], val[k].z, w[k]);
                    fma_bf16x2(acc[6], acc[7], val[k].w, w[k]);
                }
            }
            uint4 o;
            o.x = pack_bf16x2(acc[0], acc[1]);
            o.y = pack_bf16x2(acc[2], acc[3]);
            o.z = pack_bf16x2(acc[4], acc[5]);
            o.w = pack_bf16x2(acc[6], acc[7]);
            st_stream16(y + t * n_vec + v, o);
        }
    }
}

// Backward of the combine for one token per CTA: grad_out[r(t,k)] = g[t][k] * grad_y[t] (bf16, one
// rounding) and grad_g[t][k] = <grad_y[t], out[r(t,k)]> (fp32; per-thread partial sums, then a fixed
// warp-shuffle tree and a fixed-order sum over the warps, so the result does not depend on timing).
template <int KT>
__global__ void __launch_bounds__(kCombineThreads)
combine_backward_kernel(const uint4* __restrict__ grad_y, const uint4* __restrict__ out,
                        const int32_t* __restrict__ row_of_pair, const float* __restrict__ gate_w, int64_t T,
                        int K_rt, int n_vec, int64_t P, uint4* __restrict__ grad_out, float* __restrict__ grad_w,
                        uint32_t* __restrict__ err_word)
{
    constexpr int KMAX = (KT > 0) ? KT : COBALT_MAX_TOPK;
    constexpr int kWarps = kCombineThreads / 32;
    const int K = (KT > 0) ? KT : K_rt;
    __shared__ float partial[kWarps][KMAX];
    const int64_t t = blockIdx.x;
    if (t >= T) return;

    int64_t row[KMAX];
    float w[KMAX], dot[KMAX];
#pragma unroll
    for (int k = 0; k < KMAX; ++k) {
        dot[k] = 0.0f;
        if (k < K) {
            const int32_t r = __ldg(row_of_pair + t * K + k);
            const bool valid = (r >= 0 && r < P);
            row[k] = valid ? static_cast<int64_t>(r) * n_vec : -1;
            w[k] = __ldg(gate_w + t * K + k);
            if (!valid && threadIdx.x == 0) flag_error(err_word, COBALT_DEVERR_BAD_SLOT);
        }
    }
    for (int v = threadIdx.x; v < n_vec; v += blockDim.x) {
        const uint4 g = ld_stream16(grad_y + t * n_vec + v);
        const uint32_t gw[4] = {g.x, g.y, g.z, g.w};
        float gf[8];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            gf[2 * i] = __uint_as_float(gw[i] << 16);
            gf[2 * i + 1] = __uint_as_float(gw[i] & 0xFFFF0000u);
        }
        if (grad_w) {
            uint4 val[KMAX];
#pragma unroll
            for (int k = 0; k < KMAX; ++k)
                if (k < K) val[k] = (row[k] >= 0) ? ld_stream16(out + row[k] + v) : make_uint4(0, 0, 0, 0);
#pragma unroll
            for (int k = 0; k < KMAX; ++k) {
                if (k < K) {
                    const uint32_t ow[4] = {val[k].x, val[k].y, val[k].z, val[k].w};
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        dot[k] = fmaf(gf[2 * i], __uint_as_float(ow[i] << 16), dot[k]);
                        dot[k] = fmaf(gf[2 * i + 1], __uint_as_float(ow[i] & 0xFFFF0000u), dot[k]);
                    }
                }
            }
        }
        if (grad_out) {
#pragma unroll
            for (int k = 0; k < KMAX; ++k) {
                if (k < K && row[k] >= 0) {
                    uint4 o;
                    o.x = pack_bf16x2(w[k] * gf[0], w[k] * gf[1]);
                    o.y = pack_bf16x2(w[k] * gf[2], w[k] * gf[3]);
                    o.z = pack_bf16x2(w[k] * gf[4], w[k] * gf[5]);
                    o.w = pack_bf16x2(w[k] * gf[6], w[k] * gf[7]);
                    st_stream16(grad_out + row[k] + v, o);
                }
            }
        }
    }
    if (grad_w) {
        const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
        for (int k = 0; k < KMAX; ++k) {
            if (k < K) {
                float d = dot[k];
#pragma unroll
                for (int off = 16; off > 0; off >>= 1) d += __shfl_xor_sync(0xFFFFFFFFu, d, off);
                if (lane == 0) partial[warp][k] = d;
            }
        }
        __syncthreads();
        if (threadIdx.x < K) {
            float d = 0.0f;
#pragma unroll
            for (int wi = 0; wi < kWarps; ++wi) d += partial[wi][threadIdx.x];
            grad_w[t * K + threadIdx.x] = d;
        }
    }
}

// grad_expert_out alone (no gate-weight gradient wanted): one warp per (token, k).  The token's grad_y
// row is staged in shared memory once, then warp k writes row r(t,k) of grad_expert_out from end to
// end, so that every warp produces one long contiguous run instead of the K rows being interleaved
// 512 bytes at a time (measured at T = 131072, K = 8, H = 7168: 2.63 ms against 2.81 ms).  With the dot
// products in the same kernel the interleaved form above is the faster one (5.09 ms against 5.16 ms).
__global__ void __launch_bounds__(kCombineThreads)
combine_backward_scatter_kernel(const uint4* __restrict__ grad_y, const int32_t* __restrict__ row_of_pair,
                                const float* __restrict__ gate_w, int64_t T, int K, int n_vec, int64_t P,
                                uint4* __restrict__ grad_out, uint32_t* __restrict__ err_word)
{
    extern __shared__ __align__(16) uint4 g_row[];             // [n_vec] the token's grad_y row
    constexpr int kWarps = kCombineThreads / 32;
    const int64_t t = blockIdx.x;
    if (t >= T) return;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (int v = threadIdx.x; v < n_vec; v += kCombineThreads) g_row[v] = ld_stream16(grad_y + t * n_vec + v);
    __syncthreads();
    for (int k = warp; k < K; k += kWarps) {
        const int32_t r = __ldg(row_of_pair + t * K + k);
        if (r < 0 || r >= P) {
            if (lane == 0) flag_error(err_word, COBALT_DEVERR_BAD_SLOT);
            continue;
        }
        const float w = __ldg(gate_w + t * K + k);
        uint4* dst = grad_out + static_cast<int64_t>(r) * n_vec;
#pragma unroll 4
        for (int v = lane; v < n_vec; v += 32) {
            const uint4 g = g_row[v];
            uint4 o;
            o.x = pack_bf16x2(w * __uint_as_float(g.x << 16), w * __uint_as_float(g.x & 0xFFFF0000u));
            o.y = pack_bf16x2(w * __uint_as_float(g.y << 16), w * __uint_as_float(g.y & 0xFFFF0000u));
            o.z = pack_bf16x2(w * __uint_as_float(g.z << 16), w * __uint_as_float(g.z & 0xFFFF0000u));
            o.w = pack_bf16x2(w * __uint_as_float(g.w << 16), w * __uint_as_float(g.w & 0xFFFF0000u));
            st_stream16(dst + v, o);
        }
    }
}

// Argument checks and launch shared by the combine and by the backward of the dispatch gather.
// gate_w == nullptr selects unit weights (the plain sum of the K rows); the public combine entries
// reject it before they get here.
static int launch_combine(const void* expert_out, const int32_t* row_of_pair, const float* gate_w, int64_t T,
                          int32_t K, int32_t H, void* y, int64_t total_rows, uint32_t flags,
                          cobalt_stream_t stream)
{
    if (T < 0 || K < 1 || H < 1 || total_rows < 0) return COBALT_ERR_INVALID_ARG;
    if (K > COBALT_MAX_TOPK || H % 8 != 0 || T * static_cast<int64_t>(K) >= (1ll << 31) ||
        total_rows >= (1ll << 31))
        return COBALT_ERR_UNSUPPORTED;
    if (T == 0) return COBALT_OK;
    if (!expert_out || !row_of_pair || !y) return COBALT_ERR_INVALID_ARG;
    if (!aligned16(expert_out) || !aligned16(y) || !aligned16(row_of_pair) || !aligned16(gate_w))
        return COBALT_ERR_INVALID_ARG;
    const uint32_t impl = flags & COBALT_IMPL_MASK;
    if (impl != 0 && impl != COBALT_IMPL_VECTOR) return COBALT_ERR_INVALID_ARG;

    uint32_t* err_word = nullptr;
    int rc = device_error_word(&err_word);
    if (rc != COBALT_OK) return rc;

    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const int n_vec = H / 8;
    const int64_t P = total_rows;      // bound on the row indices (rows of the whole expert_out buffer)
    // one CTA per token: the block scheduler overlaps the per-token index loads of one CTA with
    // the row streaming of the others (measured faster than a persistent grid-stride grid)
    const unsigned grid = static_cast<unsigned>(T < 0x7FFFFFFFll ? T : 0x7FFFFFFFll);
    const uint4* src = static_cast<const uint4*>(expert_out);
    uint4* dst = static_cast<uint4*>(y);
#define COBALT_COMBINE_CASE(KT)                                                                         \
    case KT:                                                                                            \
        if (gate_w)                                                                                     \
            combine_kernel<KT, false><<<grid, kCombineThreads, 0, s>>>(src, row_of_pair, gate_w, T, K, n_vec, P, dst, \
                                                                       err_word);                       \
        else                                                                                            \
            combine_kernel<KT, true><<<grid, kCombineThreads, 0, s>>>(src, row_of_pair, gate_w, T, K, n_vec, P, dst,  \
                                                                      err_word);                        \
        break
    switch (K) {
        COBALT_COMBINE_CASE(1);
        COBALT_COMBINE_CASE(2);
        COBALT_COMBINE_CASE(4);
        COBALT_COMBINE_CASE(6);
        COBALT_COMBINE_CASE(8);
        COBALT_COMBINE_CASE(10);
        COBALT_COMBINE_CASE(12);
        COBALT_COMBINE_CASE(16);
        default:
            if (gate_w)
                combine_kernel<0, false><<<grid, kCombineThreads, 0, s>>>(src, row_of_pair, gate_w, T, K, n_vec, P, dst,
                                                                          err_word);
            else
                combine_kernel<0, true><<<grid, kCombineThreads, 0, s>>>(src, row_of_pair, gate_w, T, K, n_vec, P, dst,
                                                                         err_word);
    }
#undef COBALT_COMBINE_CASE
    COBALT_CUDA_TRY(cudaGetLastError());
    return COBALT_OK;
}

}  // namespace cobalt

using namespace cobalt;

extern "C" {

int cobalt_combine_block(const void* expert_out, const int32_t* row_of_pair, const float* gate_w, int64_t T,
                         int32_t K, int32_t H, void* y, int64_t total_rows, uint32_t flags,
                         cobalt_stream_t stream)
{
    if (T > 0 && !gate_w) return COBALT_ERR_INVALID_ARG;
    return launch_combine(expert_out, row_of_pair, gate_w, T, K, H, y, total_rows, flags, stream);
}

int cobalt_combine(const void* expert_out, const int32_t* row_of_pair, const float* gate_w, int64_t T,
                   int32_t K, int32_t H, void* y, uint32_t flags, cobalt_stream_t stream)
{
    if (T < 0 || K < 1) return COBALT_ERR_INVALID_ARG;
    return cobalt_combine_block(expert_out, row_of_pair, gate_w, T, K, H, y, T * static_cast<int64_t>(K), flags,
                                stream);
}

int cobalt_permute_backward(const void* grad_send, const int32_t* row_of_pair, int64_t T, int32_t K, int32_t H,
                            void* grad_x, uint32_t flags, cobalt_stream_t stream)
{
    if (T < 0 || K < 1) return COBALT_ERR_INVALID_ARG;
    // the adjoint of the gather is the sum of the token's K rows: the combine with unit weights
    return launch_combine(grad_send, row_of_pair, nullptr, T, K, H, grad_x, T * static_cast<int64_t>(K), flags, stream);
}

int cobalt_combine_backward(const void* grad_y, const void* expert_out, const int32_t* row_of_pair,
                            const float* gate_w, int64_t T, int32_t K, int32_t H, void* grad_expert_out,
                            float* grad_gate_w, uint32_t flags, cobalt_stream_t stream)
{
    if (T < 0 || K < 1 || H < 1) return COBALT_ERR_INVALID_ARG;
    if (K > COBALT_MAX_TOPK || H % 8 != 0 || T * static_cast<int64_t>(K) >= (1ll << 31)) return COBALT_ERR_UNSUPPORTED;
    if ((flags & COBALT_IMPL_MASK) != 0 && (flags & COBALT_IMPL_MASK) != COBALT_IMPL_VECTOR) return COBALT_ERR_INVALID_ARG;
    if (!grad_expert_out && !grad_gate_w) return COBALT_ERR_INVALID_ARG;
    if (T == 0) return COBALT_OK;
    if (!grad_y || !row_of_pair || !gate_w || (grad_gate_w && !expert_out)) return COBALT_ERR_INVALID_ARG;
    if (!aligned16(grad_y) || !aligned16(expert_out) || !aligned16(row_of_pair) || !aligned16(gate_w) ||
        !aligned16(grad_expert_out) || !aligned16(grad_gate_w))
        return COBALT_ERR_INVALID_ARG;
    uint32_t* err_word = nullptr;
    int rc = device_error_word(&err_word);
    if (rc != COBALT_OK) return rc;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const int n_vec = H / 8;
    const int64_t P = T * K;
    const unsigned grid = static_cast<unsigned>(T);
    const uint4* gy = static_cast<const uint4*>(grad_y);
    const uint4* out = static_cast<const uint4*>(expert_out);
    uint4* go = static_cast<uint4*>(grad_expert_out);
    if (!grad_gate_w && (flags & COBALT_IMPL_MASK) != COBALT_IMPL_VECTOR && static_cast<size_t>(n_vec) * sizeof(uint4) <= 96 * 1024) {
        const size_t smem = sizeof(uint4) * static_cast<size_t>(n_vec);
        int rc_attr = ensure_kernel_attributes(reinterpret_cast<const void*>(combine_backward_scatter_kernel), smem, false);
        if (rc_attr != COBALT_OK) return rc_attr;
        combine_backward_scatter_kernel<<<grid, kCombineThreads, smem, s>>>(gy, row_of_pair, gate_w, T, K, n_vec, P, go, err_word);
        COBALT_CUDA_TRY(cudaGetLastError());
        return COBALT_OK;
    }
#define COBALT_CBWD_CASE(KT)                                                                                   \
    case KT:                                                                                                   \
        combine_backward_kernel<KT><<<grid, kCombineThreads, 0, s>>>(gy, out, row_of_pair, gate_w, T, K, n_vec, P, go, \
                                                                     grad_gate_w, err_word);                   \
        break
    switch (K) {
        COBALT_CBWD_CASE(1);
        COBALT_CBWD_CASE(2);
        COBALT_CBWD_CASE(4);
        COBALT_CBWD_CASE(6);
        COBALT_CBWD_CASE(8);
        COBALT_CBWD_CASE(10);
        COBALT_CBWD_CASE(12);
        COBALT_CBWD_CASE(16);
        default:
            combine_backward_kernel<0><<<grid, kCombineThreads, 0, s>>>(gy, out, row_of_pair, gate_w, T, K, n_vec, P, go,
                                                                        grad_gate_w, err_word);
    }
#undef COBALT_CBWD_CASE
    COBALT_CUDA_TRY(cudaGetLastError());
    return COBALT_OK;
}

}  // extern "C"
