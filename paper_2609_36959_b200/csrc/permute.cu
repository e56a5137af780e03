// Stage 3: dispatch-side permutation (Fig. 1, "Dispatch").
//
// Index part (deterministic, no position atomics): the pair range is cut into chunks of
// contiguous pairs;
//   K1  per-chunk histogram over the D destinations              -> ws[d][chunk]
//   K2  per-destination exclusive scan across chunks (in place)  -> ws[d][chunk], dest_counts
//   K3  per chunk: exclusive scan of dest_counts over d (dest_offsets), then the stable rank
//       of every pair inside its chunk: each warp owns a contiguous sub-range, counts it,
//       the CTA scans the per-warp counts in warp order, and each warp walks its sub-range
//       again, ranking equal destinations inside a 32-pair step by lane order
//       (per-bit ballots + popcount of lower lanes).
// Row part: K4 moves each token's row to its K rows of the send buffer.  Two variants:
// (default) one work item per single-warp CTA: a bulk async copy global -> shared, then one
// bulk async copy shared -> global per destination row, many small CTAs in flight per SM;
// and plain 16-byte streaming loads/stores.
#include "permute_index.cuh"

namespace cobalt {

constexpr int kPermWarps = kPermThreads / 32;
constexpr int kMinChunk = 2048;      // pairs per chunk (multiple of kPermThreads)
constexpr int kMaxChunks = 2048;
constexpr int kRankSteps = kMinChunk / kPermWarps / 32;   // 32-pair steps of a warp per super-step

ChunkPlan plan_chunks(int64_t P)
{
    ChunkPlan c;
    c.P = P;
    int64_t chunk = kMinChunk;
    while ((P + chunk - 1) / chunk > kMaxChunks) chunk *= 2;
    c.chunk = static_cast<int>(chunk);
    c.n_chunks = static_cast<int>((P + chunk - 1) / chunk);
    if (c.n_chunks < 1) c.n_chunks = 1;
    return c;
}

// The same plan for batches with fewer chunks than the device has SMs: the chunk is shrunk (down to
// half, in steps of one CTA's threads) so that more SMs share the work.  Measured at P = 32768:
// 15.3 -> 13.3 us.  With more chunks than SMs the smaller chunks only lengthen the scan.
// The result does not depend on the chunking.
constexpr int kBalancedMinChunk = kMinChunk / 2;

static ChunkPlan plan_chunks_balanced(int64_t P, int n_sm)
{
    ChunkPlan c = plan_chunks(P);
    if (c.chunk != kMinChunk || c.n_chunks >= n_sm || P < 1) return c;
    int64_t chunk = static_cast<int64_t>(round_up((P + n_sm - 1) / n_sm, kPermThreads));
    if (chunk < kBalancedMinChunk) chunk = kBalancedMinChunk;
    if (chunk > kMinChunk) chunk = kMinChunk;
    c.chunk = static_cast<int>(chunk);
    c.n_chunks = static_cast<int>((P + chunk - 1) / chunk);
    return c;
}

// Most chunks plan_chunks_balanced can return for P pairs on any device.
static int max_balanced_chunks(int64_t P)
{
    const ChunkPlan c = plan_chunks(P);
    if (c.chunk != kMinChunk) return c.n_chunks;
    const int64_t n = (P + kBalancedMinChunk - 1) / kBalancedMinChunk;
    return static_cast<int>(n < 1 ? 1 : n);
}

// ---- K1 -----------------------------------------------------------------------------------
__global__ void __launch_bounds__(kPermThreads)
perm_hist_kernel(const int32_t* __restrict__ slot, int64_t P, int D, int chunk, int n_chunks,
                 uint32_t* __restrict__ ws, uint32_t* __restrict__ err_word)
{
    extern __shared__ uint32_t hist[];
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // the scan kernel may be scheduled early
    for (int d = threadIdx.x; d < D; d += blockDim.x) hist[d] = 0;
    __syncthreads();
    const int64_t p0 = static_cast<int64_t>(blockIdx.x) * chunk;
    const int64_t p1 = min(P, p0 + chunk);
    bool bad = false;
    for (int64_t p = p0 + threadIdx.x; p < p1; p += blockDim.x) {
        const int32_t d = __ldg(slot + p);
        if (d >= 0 && d < D) atomicAdd(&hist[d], 1u);
        else bad = true;
    }
    if (bad) flag_error(err_word, COBALT_DEVERR_BAD_SLOT);
    __syncthreads();
    for (int d = threadIdx.x; d < D; d += blockDim.x)
        ws[static_cast<size_t>(d) * n_chunks + blockIdx.x] = hist[d];
}

// ---- K2: one warp per destination ---------------------------------------------------------
__global__ void __launch_bounds__(kPermThreads)
perm_scan_kernel(uint32_t* __restrict__ ws, int D, int n_chunks, uint32_t* __restrict__ dest_counts)
{
    const int d = blockIdx.x * kPermWarps + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    wait_for_prior_kernel();        // the histograms of the kernel before this one
    if (d >= D) return;
    uint32_t* row = ws + static_cast<size_t>(d) * n_chunks;
    uint32_t running = 0;
    constexpr int kBatch = 8;   // 8 x 32 chunks loaded back to back before the dependent scans
    for (int c0 = 0; c0 < n_chunks; c0 += 32 * kBatch) {
        uint32_t v[kBatch];
#pragma unroll
        for (int b = 0; b < kBatch; ++b) {
            const int c = c0 + b * 32 + lane;
            v[b] = (c < n_chunks) ? row[c] : 0u;
        }
#pragma unroll
        for (int b = 0; b < kBatch; ++b) {
            const int c = c0 + b * 32 + lane;
            uint32_t incl = v[b];
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                const uint32_t up = __shfl_up_sync(0xFFFFFFFFu, incl, off);
                if (lane >= off) incl += up;
            }
            if (c < n_chunks) row[c] = running + incl - v[b];
            running += __shfl_sync(0xFFFFFFFFu, incl, 31);
        }
    }
    if (lane == 0) dest_counts[d] = running;
}

// ---- K3 -----------------------------------------------------------------------------------
// Lanes of the warp holding the same key, built from one ballot per key bit (the hardware
// match instruction is far slower than a dozen votes for keys this narrow).
template <int kKeyBits>
__device__ __forceinline__ uint32_t peers_of(uint32_t key)
{
    uint32_t peers = 0xFFFFFFFFu;
#pragma unroll
    for (int b = 0; b < kKeyBits; ++b) {
        const uint32_t bit = (key >> b) & 1u;
        const uint32_t vote = __ballot_sync(0xFFFFFFFFu, bit);
        peers &= bit ? vote : ~vote;
    }
    return peers;
}

// kKeyBits >= bits of D (keys 0..D, D marking "no destination"); the votes are fully unrolled
template <int kKeyBits>
__global__ void __launch_bounds__(kPermThreads)
perm_rank_kernel(const int32_t* __restrict__ slot, int64_t P, int D, int chunk, int n_chunks,
                 const uint32_t* __restrict__ ws, const uint32_t* __restrict__ dest_counts,
                 uint32_t* __restrict__ dest_offsets, int32_t* __restrict__ row_of_pair,
                 int32_t* __restrict__ pair_of_row, int rank_in_group)
{
    extern __shared__ uint32_t sm[];
    uint32_t* base = sm;                 // [D]   first row of this chunk inside destination d
    uint32_t* wcnt = sm + D;             // [kPermWarps][D]
    __shared__ uint32_t warp_sums[kPermWarps];

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    for (int i = tid; i < kPermWarps * D; i += kPermThreads) wcnt[i] = 0;
    wait_for_prior_kernel();        // dest_counts and the scanned histograms of the kernel before this one

    // exclusive scan of dest_counts over d: thread-contiguous segments, then a block scan
    const int per = (D + kPermThreads - 1) / kPermThreads;
    const int d_lo = min(D, tid * per), d_hi = min(D, d_lo + per);
    uint32_t local = 0;
    for (int d = d_lo; d < d_hi; ++d) local += __ldg(dest_counts + d);
    uint32_t incl = local;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const uint32_t up = __shfl_up_sync(0xFFFFFFFFu, incl, off);
        if (lane >= off) incl += up;
    }
    if (lane == 31) warp_sums[warp] = incl;
    __syncthreads();
    uint32_t before = incl - local;
    for (int w = 0; w < warp; ++w) before += warp_sums[w];
    for (int d = d_lo; d < d_hi; ++d) {
        if (blockIdx.x == 0) dest_offsets[d] = before;
        // rank_in_group: ranks count from 0 inside each destination instead of from its offset
        base[d] = (rank_in_group ? 0u : before) + __ldg(ws + static_cast<size_t>(d) * n_chunks + blockIdx.x);
        before += __ldg(dest_counts + d);
    }
    if (blockIdx.x == 0 && tid == kPermThreads - 1) dest_offsets[D] = before;  // last thread ends at D

    // warp sub-ranges of the chunk, in pair order
    const int64_t c0 = static_cast<int64_t>(blockIdx.x) * chunk;
    const int sub = chunk / kPermWarps;
    const int64_t w0 = c0 + static_cast<int64_t>(warp) * sub;
    const int64_t w1 = min(P, w0 + sub);
    uint32_t* mine = wcnt + warp * D;

    // The warp's sub-range is walked in super-steps of kRankSteps x 32 pairs whose slots are
    // loaded back to back into registers (one exposed memory latency per super-step, not per step).
    const int n_super = (sub + 32 * kRankSteps - 1) / (32 * kRankSteps);
    int32_t dreg[kRankSteps];
    uint32_t preg[kRankSteps];     // lanes sharing each step's destination (kept from pass A)
    auto load_super = [&](int ss) {
#pragma unroll
        for (int s = 0; s < kRankSteps; ++s) {
            const int64_t p = w0 + static_cast<int64_t>(ss) * 32 * kRankSteps + s * 32 + lane;
            int32_t d = (p < w1) ? __ldg(slot + p) : -1;
            dreg[s] = (d >= D) ? -1 : d;
        }
    };

    // pass A: count this warp's sub-range per destination (warp-private, no atomics)
    for (int ss = 0; ss < n_super; ++ss) {
        load_super(ss);
#pragma unroll
        for (int s = 0; s < kRankSteps; ++s) {
            const int32_t d = dreg[s];
            const uint32_t peers = peers_of<kKeyBits>(static_cast<uint32_t>(d < 0 ? D : d));
            preg[s] = peers;
            if (d >= 0 && (peers >> lane) == 1u) mine[d] += __popc(peers);   // highest lane of the group
            __syncwarp();
        }
    }
    __syncthreads();
    // pass B: per destination, turn the per-warp counts into starting rows (warp order)
    for (int d = tid; d < D; d += kPermThreads) {
        uint32_t run = base[d];
#pragma unroll
        for (int w = 0; w < kPermWarps; ++w) {
            const uint32_t c = wcnt[w * D + d];
            wcnt[w * D + d] = run;
            run += c;
        }
    }
    __syncthreads();
    // pass C: stable rank inside the warp's sub-range
    for (int ss = 0; ss < n_super; ++ss) {
        if (n_super > 1) {                   // a single super-step still holds its slots and peers
            load_super(ss);
#pragma unroll
            for (int s = 0; s < kRankSteps; ++s)
                preg[s] = peers_of<kKeyBits>(static_cast<uint32_t>(dreg[s] < 0 ? D : dreg[s]));
        }
#pragma unroll
        for (int s = 0; s < kRankSteps; ++s) {
            const int64_t p = w0 + static_cast<int64_t>(ss) * 32 * kRankSteps + s * 32 + lane;
            const int32_t d = dreg[s];
            const uint32_t peers = preg[s];
            if (d >= 0) {
                const uint32_t row = mine[d] + __popc(peers & ((1u << lane) - 1u));
                row_of_pair[p] = static_cast<int32_t>(row);
                if (pair_of_row) pair_of_row[row] = static_cast<int32_t>(p);
            } else if (p < w1) {
                row_of_pair[p] = -1;
            }
            __syncwarp();
            if (d >= 0 && (peers >> lane) == 1u) mine[d] += __popc(peers);
            __syncwarp();
        }
    }
}

// ---- K4, vector variant -------------------------------------------------------------------
template <int KT>
__global__ void __launch_bounds__(256)
perm_rows_vector_kernel(const uint4* __restrict__ x, const int32_t* __restrict__ row_of_pair, int64_t T,
                        int K_rt, int n_vec, int64_t P, uint4* __restrict__ send,
                        uint32_t* __restrict__ err_word)
{
    constexpr int KMAX = (KT > 0) ? KT : COBALT_MAX_TOPK;
    const int K = (KT > 0) ? KT : K_rt;
    for (int64_t t = blockIdx.x; t < T; t += gridDim.x) {
        int64_t row[KMAX];
#pragma unroll
        for (int k = 0; k < KMAX; ++k) {
            if (k < K) {
                const int32_t r = __ldg(row_of_pair + t * K + k);
                row[k] = (r >= 0 && r < P) ? static_cast<int64_t>(r) * n_vec : -1;
                if (r >= P && threadIdx.x == 0) flag_error(err_word, COBALT_DEVERR_BAD_SLOT);
            }
        }
        const uint4* src = x + t * n_vec;
#pragma unroll 2
        for (int v = threadIdx.x; v < n_vec; v += blockDim.x) {
            const uint4 val = ld_stream16(src + v);
#pragma unroll
            for (int k = 0; k < KMAX; ++k)
                if (k < K && row[k] >= 0) st_stream16(send + row[k] + v, val);
        }
    }
}

// ---- K4, bulk-async-copy variant ----------------------------------------------------------
constexpr uint32_t kSpinLimit = 1u << 22;

__device__ __forceinline__ uint32_t smem_addr(const void* p)
{
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_addr(bar)), "r"(count) : "memory");
}

__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_addr(bar)), "r"(bytes)
                 : "memory");
}

// Bounded wait for a phase of an mbarrier; false if the limit ran out.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity)
{
    const uint32_t addr = smem_addr(bar);
    for (uint32_t spin = 0; spin < kSpinLimit; ++spin) {
        uint32_t done;
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(done)
            : "r"(addr), "r"(parity)
            : "memory");
        if (done) return true;
    }
    return false;
}

__device__ __forceinline__ void bulk_load(void* smem_dst, const void* gsrc, uint32_t bytes, uint64_t* bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                     smem_addr(smem_dst)),
                 "l"(gsrc), "r"(bytes), "r"(smem_addr(bar))
                 : "memory");
}

__device__ __forceinline__ void bulk_store(void* gdst, const void* smem_src, uint32_t bytes)
{
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(gdst),
                 "r"(smem_addr(smem_src)), "r"(bytes)
                 : "memory");
}

__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }

__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }

// One work item per single-warp CTA, no ring: the block scheduler keeps many small CTAs in
// flight per SM (shared memory for one item each) and hands out items in order.
__global__ void __launch_bounds__(32)
perm_rows_bulk_oneshot_kernel(const uint8_t* __restrict__ x, const int32_t* __restrict__ row_of_pair, int64_t T,
                              int K, int64_t P, uint32_t row_bytes, int rows_per_item, int n_seg,
                              uint32_t seg_bytes, uint8_t* __restrict__ send, uint32_t* __restrict__ err_word)
{
    extern __shared__ __align__(128) uint8_t buf[];
    __shared__ __align__(8) uint64_t full;
    const int lane = threadIdx.x;
    const int64_t item = blockIdx.x;
    int64_t t0;
    int n_rows;
    uint32_t col, bytes;
    if (n_seg == 1) {
        t0 = item * rows_per_item;
        n_rows = (T - t0 < rows_per_item) ? static_cast<int>(T - t0) : rows_per_item;
        col = 0;
        bytes = row_bytes;
    } else {
        t0 = item / n_seg;
        n_rows = 1;
        col = static_cast<uint32_t>(item % n_seg) * seg_bytes;
        bytes = min(seg_bytes, row_bytes - col);
    }
    const int32_t row = (lane < n_rows * K) ? __ldg(row_of_pair + t0 * K + lane) : -1;
    if (lane == 0) {
        mbar_init(&full, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        const uint32_t total = (n_seg == 1) ? static_cast<uint32_t>(n_rows) * row_bytes : bytes;
        mbar_expect_tx(&full, total);
        bulk_load(buf, x + static_cast<size_t>(t0) * row_bytes + col, total, &full);
    }
    __syncwarp();
    bool ok = mbar_wait(&full, 0);
    ok = __all_sync(0xFFFFFFFFu, ok);
    if (ok) {
        if (row >= 0 && row < P)
            bulk_store(send + static_cast<size_t>(row) * row_bytes + col, buf + static_cast<size_t>(lane / K) * row_bytes,
                       bytes);
        else if (row >= P)
            flag_error(err_word, COBALT_DEVERR_BAD_SLOT);
    }
    bulk_commit();
    bulk_wait_all();
    if (!ok) {
        if (lane == 0) flag_error(err_word, COBALT_DEVERR_WAIT_TIMEOUT);
        (void)mbar_wait(&full, 0);
    }
}

// Row gather-scatter: dst[dst_row[i]] = src[src_row[i]] for i < n (rows of row_bytes bytes, cut into
// column segments of at most seg_bytes).  One (row, segment) per single-warp CTA: a bulk async copy
// global -> shared, then one shared -> global.  Negative indices are skipped.
__global__ void __launch_bounds__(32)
row_gather_scatter_kernel(const uint8_t* __restrict__ src, const int32_t* __restrict__ src_row,
                          const int32_t* __restrict__ dst_row, int64_t n, int64_t src_rows, int64_t dst_rows,
                          uint32_t row_bytes, int n_seg, uint32_t seg_bytes, uint8_t* __restrict__ dst,
                          uint32_t* __restrict__ err_word)
{
    extern __shared__ __align__(128) uint8_t buf[];
    __shared__ __align__(8) uint64_t full;
    const int64_t i = static_cast<int64_t>(blockIdx.x) / n_seg;
    const uint32_t col = static_cast<uint32_t>(blockIdx.x % n_seg) * seg_bytes;
    const uint32_t bytes = min(seg_bytes, row_bytes - col);
    if (i >= n) return;
    const int32_t from = __ldg(src_row + i), to = __ldg(dst_row + i);
    if (from < 0 || to < 0) return;
    if (from >= src_rows || to >= dst_rows) {
        if (threadIdx.x == 0) flag_error(err_word, COBALT_DEVERR_BAD_SLOT);
        return;
    }
    if (threadIdx.x == 0) {
        mbar_init(&full, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        mbar_expect_tx(&full, bytes);
        bulk_load(buf, src + static_cast<size_t>(from) * row_bytes + col, bytes, &full);
        const bool ok = mbar_wait(&full, 0);
        if (ok) bulk_store(dst + static_cast<size_t>(to) * row_bytes + col, buf, bytes);
        else flag_error(err_word, COBALT_DEVERR_WAIT_TIMEOUT);
        bulk_commit();
        bulk_wait_all();
        if (!ok) (void)mbar_wait(&full, 0);
    }
}

int launch_row_gather_scatter(const void* src, const int32_t* src_row, const int32_t* dst_row, int64_t n,
                              int64_t src_rows, int64_t dst_rows, int H, void* dst, cudaStream_t stream)
{
    uint32_t* err_word = nullptr;
    int rc = device_error_word(&err_word);
    if (rc != COBALT_OK) return rc;
    const uint32_t row_bytes = static_cast<uint32_t>(H) * 2u;
    const int max_seg = kRowsItemBytes;
    int n_seg = (row_bytes + max_seg - 1) / max_seg;
    uint32_t seg_bytes = static_cast<uint32_t>(round_up((row_bytes + n_seg - 1) / n_seg, 16));
    n_seg = (row_bytes + seg_bytes - 1) / seg_bytes;
    const int64_t grid = n * n_seg;
    if (grid > 0x7FFFFFFFll) return COBALT_ERR_UNSUPPORTED;
    if (grid == 0) return COBALT_OK;
    const size_t smem = round_up(seg_bytes, 128);
    const int rc_attr = ensure_kernel_attributes(reinterpret_cast<const void*>(row_gather_scatter_kernel), smem, false);
    if (rc_attr != COBALT_OK) return rc_attr;
    row_gather_scatter_kernel<<<static_cast<unsigned>(grid), 32, smem, stream>>>(
        static_cast<const uint8_t*>(src), src_row, dst_row, n, src_rows, dst_rows, row_bytes, n_seg, seg_bytes,
        static_cast<uint8_t*>(dst), err_word);
    COBALT_CUDA_TRY(cudaGetLastError());
    return COBALT_OK;
}

// P bounds the row indices (rows of the whole send buffer), which may exceed T*K when the call
// covers only a block of tokens.
static int launch_rows(const void* x, const int32_t* row_of_pair, int64_t T, int K, int H, void* send,
                       int64_t P, uint32_t flags, cudaStream_t stream)
{
    uint32_t* err_word = nullptr;
    int rc = device_error_word(&err_word);
    if (rc != COBALT_OK) return rc;
    int n_sm = 0;
    rc = sm_count(&n_sm);
    if (rc != COBALT_OK) return rc;
    const uint32_t row_bytes = static_cast<uint32_t>(H) * 2u;
    uint32_t impl = flags & COBALT_IMPL_MASK;
    if (impl == 0) impl = COBALT_IMPL_BULK;   // measured fastest: 99% of the copy bandwidth at T=131072, K=8, H=7168

    if (impl == COBALT_IMPL_VECTOR) {
        const int n_vec = H / 8;
        const unsigned grid = static_cast<unsigned>(T < 0x7FFFFFFFll ? T : 0x7FFFFFFFll);   // one CTA per token
        const uint4* xs = static_cast<const uint4*>(x);
        uint4* out = static_cast<uint4*>(send);
#define COBALT_ROWS_CASE(KT)                                                                              \
    case KT:                                                                                              \
        perm_rows_vector_kernel<KT><<<grid, 256, 0, stream>>>(xs, row_of_pair, T, K, n_vec, P, out, err_word); \
        break
        switch (K) {
            COBALT_ROWS_CASE(1);
            COBALT_ROWS_CASE(2);
            COBALT_ROWS_CASE(4);
            COBALT_ROWS_CASE(6);
            COBALT_ROWS_CASE(8);
            default:
                perm_rows_vector_kernel<0><<<grid, 256, 0, stream>>>(xs, row_of_pair, T, K, n_vec, P, out, err_word);
        }
#undef COBALT_ROWS_CASE
        COBALT_CUDA_TRY(cudaGetLastError());
        return COBALT_OK;
    }

    // bulk variant: pick the work-item shape
    const int max_stage = kRowsItemBytes;
    int rows_per_item = 1, n_seg = 1;
    uint32_t seg_bytes = row_bytes;
    if (row_bytes <= static_cast<uint32_t>(max_stage)) {
        rows_per_item = max_stage / row_bytes;
        if (rows_per_item > 32 / K) rows_per_item = 32 / K;
        if (rows_per_item < 1) rows_per_item = 1;
    } else {
        n_seg = (row_bytes + max_stage - 1) / max_stage;
        seg_bytes = static_cast<uint32_t>(round_up((row_bytes + n_seg - 1) / n_seg, 16));
        n_seg = (row_bytes + seg_bytes - 1) / seg_bytes;
    }
    const uint32_t stage_bytes =
        static_cast<uint32_t>(round_up(n_seg == 1 ? static_cast<size_t>(rows_per_item) * row_bytes : seg_bytes, 128));
    const int64_t n_items = (n_seg == 1) ? (T + rows_per_item - 1) / rows_per_item : T * n_seg;

    if (n_items > 0x7FFFFFFFll) return COBALT_ERR_UNSUPPORTED;
    const size_t smem1 = stage_bytes;
    const int rc_attr = ensure_kernel_attributes(reinterpret_cast<const void*>(perm_rows_bulk_oneshot_kernel), smem1, false);
    if (rc_attr != COBALT_OK) return rc_attr;
    perm_rows_bulk_oneshot_kernel<<<static_cast<unsigned>(n_items), 32, smem1, stream>>>(
        static_cast<const uint8_t*>(x), row_of_pair, T, K, P, row_bytes, rows_per_item, n_seg, seg_bytes,
        static_cast<uint8_t*>(send), err_word);
    COBALT_CUDA_TRY(cudaGetLastError());
    return COBALT_OK;
}

// K2 and K3, each launched programmatically after the kernel before it (their prologues overlap
// with its tail; both wait for it before reading its results).
int launch_scan_and_rank(const int32_t* assigned_slot, int64_t P, int D, const ChunkPlan& c, uint32_t* ws,
                         uint32_t* dest_counts, uint32_t* dest_offsets, int32_t* row_of_pair,
                         int32_t* pair_of_row, int rank_in_group, cudaStream_t s)
{
    cudaLaunchConfig_t cfg = {};
    cudaLaunchAttribute attr[1];
    set_programmatic_launch(&attr[0], true);
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cfg.stream = s;
    cfg.blockDim = dim3(kPermThreads);
    cfg.gridDim = dim3((D + kPermWarps - 1) / kPermWarps);
    cfg.dynamicSmemBytes = 0;
    COBALT_CUDA_TRY(cudaLaunchKernelEx(&cfg, perm_scan_kernel, ws, D, c.n_chunks, dest_counts));
    const size_t smem = sizeof(uint32_t) * static_cast<size_t>(D) * (1 + kPermWarps);
    using RankKernel = void (*)(const int32_t*, int64_t, int, int, int, const uint32_t*, const uint32_t*, uint32_t*,
                                int32_t*, int32_t*, int);
    int need_bits = 1;
    while ((1 << need_bits) <= D) ++need_bits;       // keys 0..D
    RankKernel kernel = perm_rank_kernel<13>;
    if (need_bits <= 4) kernel = perm_rank_kernel<4>;
    else if (need_bits <= 6) kernel = perm_rank_kernel<6>;
    else if (need_bits <= 8) kernel = perm_rank_kernel<8>;
    else if (need_bits <= 9) kernel = perm_rank_kernel<9>;
    else if (need_bits <= 10) kernel = perm_rank_kernel<10>;
    else if (need_bits <= 11) kernel = perm_rank_kernel<11>;
    if (smem > 48 * 1024)
        COBALT_CUDA_TRY(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem)));
    cfg.gridDim = dim3(c.n_chunks);
    cfg.dynamicSmemBytes = smem;
    COBALT_CUDA_TRY(cudaLaunchKernelEx(&cfg, kernel, assigned_slot, P, D, c.chunk, c.n_chunks,
                                       static_cast<const uint32_t*>(ws), static_cast<const uint32_t*>(dest_counts),
                                       dest_offsets, row_of_pair, pair_of_row, rank_in_group));
    return COBALT_OK;
}

int launch_chunk_histograms(const int32_t* keys, int64_t P, int D, const ChunkPlan& c, uint32_t* ws,
                            uint32_t* err_word, cudaStream_t s)
{
    perm_hist_kernel<<<c.n_chunks, kPermThreads, sizeof(uint32_t) * D, s>>>(keys, P, D, c.chunk, c.n_chunks, ws,
                                                                            err_word);
    COBALT_CUDA_TRY(cudaGetLastError());
    return COBALT_OK;
}

static int check_index_args(int64_t T, int32_t K, int32_t D)
{
    if (T < 0 || K < 1 || D < 1) return COBALT_ERR_INVALID_ARG;
    if (K > COBALT_MAX_TOPK || D > COBALT_MAX_DESTS || T * static_cast<int64_t>(K) >= (1ll << 31))
        return COBALT_ERR_UNSUPPORTED;
    return COBALT_OK;
}

}  // namespace cobalt

using namespace cobalt;

extern "C" {

size_t cobalt_permute_workspace_bytes(int64_t T, int32_t K, int32_t D)
{
    if (check_index_args(T, K, D) != COBALT_OK) return 0;
    return round_up(static_cast<size_t>(D) * max_balanced_chunks(T * K) * sizeof(uint32_t), 256);
}

int cobalt_permute_index(const int32_t* assigned_slot, int64_t T, int32_t K, int32_t D,
                         uint32_t* dest_counts, uint32_t* dest_offsets, int32_t* row_of_pair,
                         int32_t* pair_of_row, void* workspace, size_t workspace_bytes,
                         cobalt_stream_t stream)
{
    int rc = check_index_args(T, K, D);
    if (rc != COBALT_OK) return rc;
    if (!dest_counts || !dest_offsets) return COBALT_ERR_INVALID_ARG;
    if (T > 0 && (!assigned_slot || !row_of_pair)) return COBALT_ERR_INVALID_ARG;
    if (!aligned16(assigned_slot) || !aligned16(row_of_pair) || !aligned16(pair_of_row) ||
        !aligned16(dest_counts) || !aligned16(dest_offsets) || !aligned16(workspace))
        return COBALT_ERR_INVALID_ARG;
    const size_t need = cobalt_permute_workspace_bytes(T, K, D);
    if (!workspace || workspace_bytes < need) return COBALT_ERR_WORKSPACE_TOO_SMALL;

    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const int64_t P = T * K;
    int n_sm = 0;
    rc = sm_count(&n_sm);
    if (rc != COBALT_OK) return rc;
    const ChunkPlan c = plan_chunks_balanced(P, n_sm);
    uint32_t* ws = static_cast<uint32_t*>(workspace);
    uint32_t* err_word = nullptr;
    rc = device_error_word(&err_word);
    if (rc != COBALT_OK) return rc;

    rc = launch_chunk_histograms(assigned_slot, P, D, c, ws, err_word, s);
    if (rc != COBALT_OK) return rc;
    return launch_scan_and_rank(assigned_slot, P, D, c, ws, dest_counts, dest_offsets, row_of_pair, pair_of_row, 0, s);
}

// ---- no-allocation variant of the index half ------------------------------------------------
// Same three kernels as cobalt_permute_index, but the per-chunk histogram scratch lives in a
// fixed device array that is part of the library image instead of a caller-provided buffer.
// It is meant for callers that have no way to obtain device scratch at the point of the call:
// code running under a framework that forbids allocator calls on its hot path, plugins that are
// handed only their input and output buffers, and processes whose memory pool was sized up
// front and is already fully committed.  Every GPU that loads the library carries the array
// (COBALT_STATIC_SCRATCH_WORDS * 4 bytes) until the process exits.
static __device__ __align__(256) uint32_t g_static_perm_scratch[COBALT_STATIC_SCRATCH_WORDS];

// The array's name is only a host-side handle; the kernels need its device address, looked up
// once per device (with that device current) and cached here.
static uint32_t* g_static_perm_scratch_ptr[64] = {nullptr};

static int static_scratch_address(uint32_t** out)
{
    int dev = 0;
    COBALT_CUDA_TRY(cudaGetDevice(&dev));
    if (dev >= 0 && dev < 64 && g_static_perm_scratch_ptr[dev]) {
        *out = g_static_perm_scratch_ptr[dev];
        return COBALT_OK;
    }
    uint32_t* ptr = nullptr;
    COBALT_CUDA_TRY(cudaGetSymbolAddress(reinterpret_cast<void**>(&ptr), g_static_perm_scratch));
    if (!ptr) return COBALT_ERR_CUDA;
    if (dev >= 0 && dev < 64) g_static_perm_scratch_ptr[dev] = ptr;
    *out = ptr;
    return COBALT_OK;
}

int cobalt_permute_index_static(const int32_t* assigned_slot, int64_t T, int32_t K, int32_t D,
                                uint32_t* dest_counts, uint32_t* dest_offsets, int32_t* row_of_pair,
                                int32_t* pair_of_row, cobalt_stream_t stream)
{
    int rc = check_index_args(T, K, D);
    if (rc != COBALT_OK) return rc;
    if (!dest_counts || !dest_offsets) return COBALT_ERR_INVALID_ARG;
    if (T > 0 && (!assigned_slot || !row_of_pair)) return COBALT_ERR_INVALID_ARG;
    if (!aligned16(assigned_slot) || !aligned16(row_of_pair) || !aligned16(pair_of_row) ||
        !aligned16(dest_counts) || !aligned16(dest_offsets))
        return COBALT_ERR_INVALID_ARG;
    const int64_t P = T * K;
    const ChunkPlan c = plan_chunks(P);
    if (static_cast<int64_t>(D) * c.n_chunks > static_cast<int64_t>(COBALT_STATIC_SCRATCH_WORDS))
        return COBALT_ERR_SCRATCH_LIMIT;

    uint32_t* ws = nullptr;
    rc = static_scratch_address(&ws);
    if (rc != COBALT_OK) return rc;
    uint32_t* err_word = nullptr;
    rc = device_error_word(&err_word);
    if (rc != COBALT_OK) return rc;

    // The histogram kernel stores every scratch word the later kernels read (all D x n_chunks
    // entries, zeros included), so nothing left over from an earlier call is ever consumed and
    // no clearing pass is needed.
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    rc = launch_chunk_histograms(assigned_slot, P, D, c, ws, err_word, s);
    if (rc != COBALT_OK) return rc;
    return launch_scan_and_rank(assigned_slot, P, D, c, ws, dest_counts, dest_offsets, row_of_pair, pair_of_row, 0, s);
}

int cobalt_permute_rows_block(const void* x, const int32_t* row_of_pair, int64_t T, int32_t K, int32_t H,
                              void* send, int64_t total_rows, uint32_t flags, cobalt_stream_t stream)
{
    if (T < 0 || K < 1 || H < 1 || total_rows < 0) return COBALT_ERR_INVALID_ARG;
    if (K > COBALT_MAX_TOPK || H % 8 != 0 || T * static_cast<int64_t>(K) >= (1ll << 31) ||
        total_rows >= (1ll << 31))
        return COBALT_ERR_UNSUPPORTED;
    if (T == 0) return COBALT_OK;
    if (!x || !row_of_pair || !send) return COBALT_ERR_INVALID_ARG;
    if (!aligned16(x) || !aligned16(send) || !aligned16(row_of_pair)) return COBALT_ERR_INVALID_ARG;
    const uint32_t impl = flags & COBALT_IMPL_MASK;
    if (impl != 0 && impl != COBALT_IMPL_VECTOR && impl != COBALT_IMPL_BULK)
        return COBALT_ERR_INVALID_ARG;
    return launch_rows(x, row_of_pair, T, K, H, send, total_rows, flags, static_cast<cudaStream_t>(stream));
}

int cobalt_permute_rows(const void* x, const int32_t* row_of_pair, int64_t T, int32_t K, int32_t H,
                        void* send, uint32_t flags, cobalt_stream_t stream)
{
    if (T < 0 || K < 1) return COBALT_ERR_INVALID_ARG;
    return cobalt_permute_rows_block(x, row_of_pair, T, K, H, send, T * static_cast<int64_t>(K), flags, stream);
}

int cobalt_permute(const int32_t* assigned_slot, int64_t T, int32_t K, int32_t D, const void* x, int32_t H,
                   void* send, uint32_t* dest_counts, uint32_t* dest_offsets, int32_t* row_of_pair,
                   int32_t* pair_of_row, uint32_t flags, void* workspace, size_t workspace_bytes,
                   cobalt_stream_t stream)
{
    // validate the row half first so that nothing is enqueued on a bad argument
    if (H < 1) return COBALT_ERR_INVALID_ARG;
    if (H % 8 != 0) return COBALT_ERR_UNSUPPORTED;
    if (T > 0 && (!x || !send)) return COBALT_ERR_INVALID_ARG;
    if (!aligned16(x) || !aligned16(send)) return COBALT_ERR_INVALID_ARG;
    const uint32_t impl = flags & COBALT_IMPL_MASK;
    if (impl != 0 && impl != COBALT_IMPL_VECTOR && impl != COBALT_IMPL_BULK)
        return COBALT_ERR_INVALID_ARG;
    int rc = cobalt_permute_index(assigned_slot, T, K, D, dest_counts, dest_offsets, row_of_pair, pair_of_row,
                                  workspace, workspace_bytes, stream);
    if (rc != COBALT_OK) return rc;
    return cobalt_permute_rows(x, row_of_pair, T, K, H, send, flags, stream);
}

}  // extern "C"
