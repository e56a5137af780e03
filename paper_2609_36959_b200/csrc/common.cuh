// Shared host/device helpers of the sm_100a token-routing library (not part of the C ABI).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "cobalt.h"

namespace cobalt {

// ---- host side ---------------------------------------------------------------------------
// Records a failed runtime call for cobalt_last_cuda_error() and maps it to COBALT_ERR_CUDA.
int record_cuda_error(cudaError_t err);

#define COBALT_CUDA_TRY(expr)                                        \
    do {                                                             \
        cudaError_t cobalt_err__ = (expr);                           \
        if (cobalt_err__ != cudaSuccess)                             \
            return ::cobalt::record_cuda_error(cobalt_err__);        \
    } while (0)

// Address of the current device's error word (kernels receive it as an argument).
int device_error_word(uint32_t** out);

// Number of SMs of the current device (cached per device).
int sm_count(int* out);

// Lets `kernel` be launched with up to `bytes` of dynamic shared memory (and, if asked, with a
// cluster size above 8) on the current device.  The runtime calls are made only the first time
// and when a larger size is asked for; later calls cost a map lookup.
int ensure_kernel_attributes(const void* kernel, size_t bytes, bool non_portable_cluster);

// Largest work item of the bulk row movers: whole rows of consecutive tokens, or one column segment
// of a longer row (measured flat between 14 and 112 KB; 32 KB keeps up to seven CTAs on an SM).
constexpr int kRowsItemBytes = 32768;

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

inline size_t round_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// Device tables built from a layout (Section 3.3: R_{e,n} and N_e), one contiguous blob of
// 32-bit words that kernels copy into shared memory:
//   ent[e*N + n]   bits 0-7   |R_{e,n}|
//                  bits 8-20  offset of R_{e,n} in rlist
//                  bits 21-27 m_{e,n}: the remote-node mask of e seen from source node n (bit j = j-th
//                             node in ascending id with n skipped); 0 when n itself holds e
//                  bits 28-30 node of e's primary replica
//   primary[e]     = slot of e's primary replica
//   rlist[...]     = slots of R_{e,n}, ascending, all (e, n) groups back to back
//   cover[...]     = 128 bytes, only for N <= 4: the smallest cover b* for every set of mask values that
//                    can occur in a token (bit v-1 of the index set iff some expert of U_t has mask v)
constexpr int kEntCountBits = 8, kEntOffsetBits = 13, kEntMaskShift = 21, kEntPrimaryNodeShift = 28;
constexpr int kCoverTableWords = 32;

struct LayoutView {
    int32_t N, Q, S, E, G, D;
    int32_t n_replicas;       // entries of rlist
    int32_t words;            // total 32-bit words of the blob
    uint32_t q_inverse;       // floor(s * q_inverse / 2^20) = s / Q for every source rank s in [0, G)
    const uint32_t* blob;     // device
    __host__ __device__ int ent_off() const { return 0; }
    __host__ __device__ int primary_off() const { return E * N; }
    __host__ __device__ int rlist_off() const { return E * N + E; }
    __host__ __device__ int cover_off() const { return E * N + E + n_replicas; }
};

}  // namespace cobalt

struct cobalt_layout {
    cobalt::LayoutView view;
    int device;
};

namespace cobalt {

// ---- device side -------------------------------------------------------------------------
#ifdef __CUDACC__

// Counter hash behind Algorithm 1's RandomNode (stream 0) and UniformChoice (stream 1): a pure
// function of (seed, token, expert, stream), all arithmetic modulo 2^32, so that the draw does
// not depend on thread or launch shape.
__device__ __forceinline__ uint32_t route_hash(uint32_t seed_lo, uint32_t seed_hi, uint32_t t,
                                               uint32_t e, uint32_t stream)
{
    uint32_t x = seed_lo ^ 0x6A09E667u;
    x = (x ^ t) * 0x9E3779B9u;
    x ^= x >> 16;
    x = (x ^ seed_hi) * 0xBB67AE85u;
    x ^= x >> 15;
    x = (x ^ (2u * e + stream)) * 0x9E3779B9u;
    x ^= x >> 16;
    x *= 0xBB67AE85u;
    x ^= x >> 15;
    x *= 0x6A09E667u;
    x ^= x >> 16;
    return x;
}

// floor(x * n / 2^32): an index in [0, n)
__device__ __forceinline__ uint32_t hash_index(uint32_t x, uint32_t n) { return __umulhi(x, n); }

__device__ __forceinline__ void flag_error(uint32_t* err_word, uint32_t bits)
{
    atomicOr(err_word, bits);
}

// streaming (read-once / write-once) 16-byte accesses that stay out of L1
__device__ __forceinline__ uint4 ld_stream16(const void* p)
{
    uint4 v;
    asm("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}

__device__ __forceinline__ void st_stream16(void* p, uint4 v)
{
    asm volatile("st.global.L1::no_allocate.v4.u32 [%0], {%1,%2,%3,%4};" ::"l"(p), "r"(v.x),
                 "r"(v.y), "r"(v.z), "r"(v.w)
                 : "memory");
}

// Programmatic dependent launch: a kernel launched with launch_after_zeroing() may start while
// the zeroing kernel before it is still running; it must call wait_for_prior_kernel() before it
// first touches memory the zeroing kernel writes.
__device__ __forceinline__ void wait_for_prior_kernel() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// Clears up to four small accumulator arrays (32-bit words) in one launch.
struct ZeroList {
    uint32_t* ptr[4];
    int n[4];
};

static __global__ void zero_words_kernel(ZeroList z)
{
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // the next kernel may start right away
    const int stride = gridDim.x * blockDim.x;
#pragma unroll
    for (int k = 0; k < 4; ++k)
        for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < z.n[k]; i += stride) z.ptr[k][i] = 0;
}

// *launched tells the caller whether a zeroing kernel now precedes its own kernel in the stream:
// only then may that kernel be launched programmatically (it would otherwise overlap with a
// foreign kernel that may still be producing its inputs).
static inline int launch_zero_list(ZeroList z, cudaStream_t stream, bool* launched)
{
    *launched = false;
    int most = 0;
    for (int k = 0; k < 4; ++k) {
        if (!z.ptr[k]) z.n[k] = 0;
        if (z.n[k] > most) most = z.n[k];
    }
    if (most == 0) return COBALT_OK;
    *launched = true;
    int grid = (most + 255) / 256;
    if (grid > 296) grid = 296;
    zero_words_kernel<<<grid, 256, 0, stream>>>(z);
    COBALT_CUDA_TRY(cudaGetLastError());
    return COBALT_OK;
}

static inline int launch_zero_words(uint32_t* a, int n_a, uint32_t* b, int n_b, cudaStream_t stream, bool* launched)
{
    ZeroList z = {{a, b, nullptr, nullptr}, {n_a, n_b, 0, 0}};
    return launch_zero_list(z, stream, launched);
}

// Fills a launch attribute that lets the kernel overlap with the tail of the previous kernel
// in the stream (see wait_for_prior_kernel).
static inline void set_programmatic_launch(cudaLaunchAttribute* attr, bool allowed)
{
    attr->id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr->val.programmaticStreamSerializationAllowed = allowed ? 1 : 0;
}

#endif  // __CUDACC__

}  // namespace cobalt
