// Host-side launchers of the permutation-index kernels (chunk histograms, scan, stable rank),
// shared with the kernels that reuse the same machinery for other keys.
#pragma once

#include "common.cuh"

namespace cobalt {

constexpr int kPermThreads = 256;

struct ChunkPlan {
    int64_t P;
    int chunk;        // pairs per chunk (a multiple of kPermThreads)
    int n_chunks;
};

// Chunks of 2048 pairs, doubled until there are at most 2048 of them.
ChunkPlan plan_chunks(int64_t P);

// K1: ws[d * n_chunks + chunk] = #{p in chunk : keys[p] = d}; keys outside [0, D) are flagged and skipped.
int launch_chunk_histograms(const int32_t* keys, int64_t P, int D, const ChunkPlan& c, uint32_t* ws,
                            uint32_t* err_word, cudaStream_t s);

// K2 + K3 (both launched programmatically after the kernel before them, which must be the one that
// filled ws): per-destination scan across chunks, counts, offsets and the stable rank of every pair.
// rank_in_group != 0 writes the rank inside the pair's destination instead of the global row.
int launch_scan_and_rank(const int32_t* keys, int64_t P, int D, const ChunkPlan& c, uint32_t* ws,
                         uint32_t* dest_counts, uint32_t* dest_offsets, int32_t* row_of_pair,
                         int32_t* pair_of_row, int rank_in_group, cudaStream_t s);

// dst[dst_row[i]] = src[src_row[i]] for i < n, rows of H 16-bit elements; negative indices are skipped,
// indices beyond src_rows / dst_rows are flagged and skipped.
int launch_row_gather_scatter(const void* src, const int32_t* src_row, const int32_t* dst_row, int64_t n,
                              int64_t src_rows, int64_t dst_rows, int H, void* dst, cudaStream_t stream);

}  // namespace cobalt
