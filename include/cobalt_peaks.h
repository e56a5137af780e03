/*
 * cobalt_peaks.h -- C ABI of the measurement kernels that go with the token-routing library.
 *
 * The statistics and assignment stages of the routing path move a few megabytes; what bounds them
 * is not HBM but the rate at which an SM performs shared-memory atomic adds and issues
 * instructions.  These entry points measure those two rates on the device at hand, so that the
 * benchmark can report each stage as a fraction of the resource that binds it.  They are not part
 * of the routing path (the paper has no counterpart): libcobalt_peaks.so is a separate library that
 * only the benchmark loads.
 *
 * All pointers named *_host are host memory; `topk_ids` is a device pointer (int32 [T, K], ids in
 * [0, E), distinct within a token).  The calls launch on the default stream of the current device,
 * synchronise, and return 0 or the cudaError_t of the failed call.  Rates are per SM and per SM
 * clock, measured with the SM's cycle counter inside the kernel over the slowest CTA, one CTA of
 * 1024 threads per SM.
 */
#ifndef COBALT_PEAKS_H_
#define COBALT_PEAKS_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* Shared-memory atomic adds per clock and SM.
 * pattern 0: every lane of a warp adds to its own bank and word (no conflicts): the pipeline's peak.
 * pattern 1: the statistics kernel's own access pattern: every thread takes tokens from topk_ids and adds
 *            the token's K(K+1)/2 pairs to a lower-triangle tile of 16-bit counters, two per word
 *            (Section 3.2, Stage 1: the co-activation counts), without anything else around it.
 * adds_per_clock_host[0] receives the rate, wavefront-free of launch overhead; T tokens are spread over
 * one CTA per SM and repeated `repeats` times. */
int cobalt_peak_shared_atomics(int pattern, const int32_t* topk_ids, int64_t T, int32_t K, int32_t E,
                               int32_t repeats, double* adds_per_clock_host);

/* Warp instructions issued per clock and SM by 32 resident warps running eight independent chains of
 * integer arithmetic each, with no memory access: the rate an instruction-bound kernel can at most reach.
 * mix 0: add, shift, logic (the issue rate itself).
 * mix 1: multiply-add, shift, logic -- the mix of the counter hash behind Algorithm 1's draws
 *        (Section 3.3), where every third instruction is a 32-bit multiply.
 * The count assumes three machine instructions per step of a chain. */
int cobalt_peak_issue_rate(int32_t mix, int32_t repeats, double* warp_instructions_per_clock_host);

#ifdef __cplusplus
}
#endif
#endif /* COBALT_PEAKS_H_ */
