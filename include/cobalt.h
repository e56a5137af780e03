/*
 * cobalt.h -- C ABI of the B200 (sm_100a) token-routing library for Cobalt, the
 * co-activation-aware MoE training method.
 *
 * One training step's gating output (top-K expert ids and gate weights per token) and a given
 * expert layout (every expert's replicas placed on (node, rank) slots; the layout is a plain
 * data structure, not hardware) go through four stages:
 *
 *   cobalt_coact_stats   expert co-activation counts and per-expert loads   (Section 3.2, Stage 1)
 *   cobalt_assign        communication-aware task assignment                (Section 3.3, Algorithm 1)
 *   cobalt_permute       destination-grouped send buffer                    (Fig. 1, "Dispatch")
 *   cobalt_combine       inverse permutation + gate-weighted sum            (Fig. 1, "Weighted sum")
 *
 * Symbols (Table 1): E experts, K experts per token, G = N*Q ranks on N nodes with Q ranks
 * each, T tokens, D_t the selected experts of token t, s_t its source rank, P_r the experts
 * on rank r, r_te the rank that runs task (t, e).  Each rank has S expert slots; the global
 * slot id is d = r*S + j (rank = d / S, node = d / (S*Q)); D = G*S destinations; a (token,
 * expert) pair has index p = t*K + k; P = T*K pairs.  r_te is reported as a global slot id.
 *
 * Conventions for every call unless stated otherwise
 *  - Pointers named *_host are host memory; all others are DEVICE pointers borrowed from the
 *    caller for the duration of the enqueued work.  The library allocates nothing per call;
 *    scratch comes from the caller-provided workspace (size from the *_workspace_bytes
 *    query, 256-byte aligned).  Only the layout handle owns device memory.
 *  - Device pointers must be 16-byte aligned.
 *  - Calls enqueue kernels on `stream` (a cudaStream_t, NULL = default stream) and return
 *    without synchronising; outputs are valid once the stream reaches that point.
 *  - Return value: COBALT_OK or a negative COBALT_ERR_* code.  Nothing is enqueued when an
 *    argument check fails.  The library never throws, exits, traps or waits unboundedly.
 *  - Threads: every entry point may be called from several host threads at once.  The library
 *    keeps no mutable state besides per-device caches of device attributes (guarded), the layout
 *    handles (immutable once created; destroy one only when no call uses it) and one error word
 *    per device.  Calls that run on the GPU at the same time must not share a workspace or
 *    output buffers; cobalt_last_cuda_error is per host thread.
 *  - Data preconditions: ids in [0, E) and distinct within a token (D_t is a set); source
 *    ranks in [0, G); assigned slots in [0, D).  A violation never causes an out-of-bounds
 *    access: the kernel sets a bit in the device error word, skips the offending token or
 *    pair (its outputs are unspecified; slots are written as -1), and carries on.
 */
#ifndef COBALT_H_
#define COBALT_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define COBALT_VERSION 100

#define COBALT_OK 0
#define COBALT_ERR_INVALID_ARG (-1)          /* null / negative / misaligned argument, bad layout */
#define COBALT_ERR_WORKSPACE_TOO_SMALL (-2)
#define COBALT_ERR_UNSUPPORTED (-3)          /* outside the supported size envelope (see below) */
#define COBALT_ERR_CUDA (-4)                 /* a CUDA runtime call failed; see cobalt_last_cuda_error */
#define COBALT_ERR_SCRATCH_LIMIT (-5)        /* problem needs more than the library's built-in scratch */
#define COBALT_ERR_HOST_ALLOC (-6)           /* a host-side allocation failed (layout handle, planner scratch) */

/* Supported envelope: N <= 8 nodes, Q <= 255 ranks per node, K <= 16, E <= 1024, D <= 4096,
 * P = T*K < 2^31, H a multiple of 8 (rows are whole 16-byte vectors).
 * Every K from 1 to 16 gives the same results; the kernels of the separate stage calls are compiled with
 * the K ids of a token in registers for K = 1, 2, 4, 6, 8, 10, 12, 16 and run a generic variant (loops
 * to 16, a few microseconds slower per index stage) for the other K, while cobalt_route_index is compiled
 * for every K. */
#define COBALT_MAX_NODES 8
#define COBALT_MAX_RANKS_PER_NODE 255
#define COBALT_MAX_TOPK 16
#define COBALT_MAX_EXPERTS 1024
#define COBALT_MAX_DESTS 4096

/* bits of the device error word (cobalt_read_and_clear_device_error) */
#define COBALT_DEVERR_BAD_EXPERT_ID 0x1u     /* id outside [0, E) */
#define COBALT_DEVERR_DUPLICATE_ID 0x2u      /* an expert listed twice in one token */
#define COBALT_DEVERR_BAD_SRC_RANK 0x4u      /* source rank outside [0, G) */
#define COBALT_DEVERR_BAD_SLOT 0x8u          /* assigned slot / row index outside its range */
#define COBALT_DEVERR_WAIT_TIMEOUT 0x10u     /* a bounded wait ran out (copy pipeline, grid barrier of the fused pass) */

/* flag bits */
#define COBALT_STATS_ACCUMULATE 0x1u         /* add to coact/load instead of overwriting them */
#define COBALT_ASSIGN_NAIVE 0x1u             /* primary-replica rule instead of Algorithm 1 */
#define COBALT_ASSIGN_ROUND_ROBIN 0x2u       /* deal each (expert, node) group's tasks to its replicas in turn */
#define COBALT_SEED_ON_DEVICE 0x4u           /* cobalt_assign, cobalt_route_index: the `seed` argument is the device
                                                address (8-byte aligned) of a uint64 that the kernel reads when it
                                                runs, so that a captured CUDA graph can be replayed with a new seed */
#define COBALT_STATS_TILE16 0x10u            /* cobalt_coact_stats: 16-bit counters in the shared-memory tile wherever
                                                they cannot overflow (default: only where that is faster or the
                                                32-bit tile does not fit) */
#define COBALT_STATS_TILE32 0x20u            /* cobalt_coact_stats, cobalt_route_index: 32-bit counters wherever the tile fits */
#define COBALT_ROUTE_SEPARATE_KERNELS 0x40u  /* cobalt_route_index: run the three separate calls instead of the fused kernel */
#define COBALT_IMPL_MASK 0xF00u              /* row-kernel variant override, 0 = library default */
#define COBALT_IMPL_VECTOR 0x100u            /* row movement with plain 16-byte loads/stores */
#define COBALT_IMPL_BULK 0x200u              /* row movement with bulk async copies, one work item per CTA (default) */

typedef struct cobalt_layout cobalt_layout_t;   /* opaque, owned by the library */
typedef void* cobalt_stream_t;                  /* a cudaStream_t */

const char* cobalt_status_string(int status);
int cobalt_version(void);
/* The cudaError_t of the most recent failed runtime call on this thread (0 if none). */
int cobalt_last_cuda_error(void);

/* ---- expert layout (Section 3.1: P = {P_r}; Section 3.3: R_{e,n}, N_e) -------------------
 * slot_expert_host[r*S + j] is the expert in slot j of rank r, or -1 for an empty slot.
 * primary_slot_host[e] is the slot of e's primary replica (used by the naive rule and for
 * V_naive); NULL means "the lowest slot holding e".
 * A layout is rejected with COBALT_ERR_INVALID_ARG when an expert has no replica (Eq. 2,
 * first constraint), an expert sits twice on one rank (Section 3.2, Stage 2), an id is outside
 * [-1, E), or a given primary slot does not hold its expert; with COBALT_ERR_UNSUPPORTED
 * outside the size envelope, with COBALT_ERR_HOST_ALLOC when host memory runs out.
 * cobalt_layout_check runs only these host-side checks (no device
 * needed).  cobalt_layout_create also builds the device tables (one allocation, one copy, on
 * the current device; synchronous) and returns a handle to be released with
 * cobalt_layout_destroy (NULL is accepted). */
int cobalt_layout_check(int32_t num_nodes, int32_t ranks_per_node, int32_t slots_per_rank,
                        int32_t num_experts, const int32_t* slot_expert_host,
                        const int32_t* primary_slot_host);
int cobalt_layout_create(cobalt_layout_t** out, int32_t num_nodes, int32_t ranks_per_node,
                         int32_t slots_per_rank, int32_t num_experts,
                         const int32_t* slot_expert_host, const int32_t* primary_slot_host);
int cobalt_layout_destroy(cobalt_layout_t* layout);
/* D = G*S of a layout (0 for NULL). */
int32_t cobalt_layout_num_dests(const cobalt_layout_t* layout);

/* ---- stage 1: per-step statistics (Section 3.2, Stage 1) ---------------------------------
 * load[e]      = number of tokens selecting e (the task count whose EMA is w^_e)
 * coact[i*E+j] = number of tokens selecting both i and j (whose EMA is c^_ij); symmetric,
 *                diagonal = load.
 * topk_ids: int32 [T, K] row-major.  coact: uint32 [E*E].  load: uint32 [E].
 * Outputs are overwritten unless COBALT_STATS_ACCUMULATE is set.  T = 0 is allowed.
 * flags: COBALT_STATS_ACCUMULATE, and at most one of COBALT_STATS_TILE16 / COBALT_STATS_TILE32
 * (counter width of the privatised shared-memory tile; the results are the same). */
size_t cobalt_coact_stats_workspace_bytes(int64_t T, int32_t K, int32_t E);
int cobalt_coact_stats(const int32_t* topk_ids, int64_t T, int32_t K, int32_t E,
                       uint32_t* coact, uint32_t* load, uint32_t flags,
                       void* workspace, size_t workspace_bytes, cobalt_stream_t stream);

/* ---- stage 2: communication-aware task assignment (Section 3.3, Algorithm 1) --------------
 * Per token: experts present on the source node N(s_t) run there; for the others the
 * smallest set of remote nodes covering them is found by enumerating (N-1)-bit masks in
 * ascending order (first minimum wins), each such expert picks a node of that set and every
 * expert picks a replica inside its node, both uniformly through a counter hash of
 * (seed, t, e) so that results do not depend on launch shape.
 * The counter hash (arithmetic modulo 2^32; seed_lo / seed_hi = low / high half of seed;
 * stream 0 = node pick, 1 = replica pick):
 *     x = seed_lo ^ 0x6A09E667
 *     x = (x ^ t) * 0x9E3779B9;              x ^= x >> 16
 *     x = (x ^ seed_hi) * 0xBB67AE85;        x ^= x >> 15
 *     x = (x ^ (2*e + stream)) * 0x9E3779B9; x ^= x >> 16
 *     x = x * 0xBB67AE85;                    x ^= x >> 15
 *     x = x * 0x6A09E667;                    x ^= x >> 16
 *     index among n candidates = (x * n) >> 32
 * Node candidates are the set bits of b* & m counted from bit 0 (bit j = j-th remote node in
 * ascending node id, source node skipped); replica candidates are R_{e,n} in ascending slot id.
 * src_rank: int32 [T], or NULL to use src_rank_uniform for every token.
 * Outputs: assigned_slot int32 [T*K] (r_te as global slot id); optional (NULL to skip)
 * slot_load uint32 [D] = w_er (Section 3.1), remote_nodes uint8 [T] = the token's term of
 * Eq. 1, totals uint64 [2] = { V of this assignment, V of the naive primary-replica rule }.
 * The optional outputs are overwritten.  COBALT_ASSIGN_NAIVE assigns every task to its
 * expert's primary replica instead (the one-replica-per-expert baseline).
 * COBALT_ASSIGN_ROUND_ROBIN (not in the paper) keeps Step 1 and replaces the hashed replica
 * pick of Step 2: walking the pairs in ascending p, the j-th task of group (expert, node) goes
 * to R_{e,n}[j mod |R_{e,n}|], so replica loads inside a group differ by at most one.  The
 * running count is reproduced exactly (chunk histograms, scan, stable rank), never with racing
 * counters.  This mode needs the workspace of cobalt_assign_workspace_bytes and E*N <= 4096;
 * the other modes need none. */
size_t cobalt_assign_workspace_bytes(const cobalt_layout_t* layout, int64_t T, int32_t K);
int cobalt_assign(const cobalt_layout_t* layout, const int32_t* topk_ids,
                  const int32_t* src_rank, int32_t src_rank_uniform, int64_t T, int32_t K,
                  uint64_t seed, int32_t* assigned_slot, uint32_t* slot_load,
                  uint8_t* remote_nodes, uint64_t* totals, uint32_t flags,
                  void* workspace, size_t workspace_bytes, cobalt_stream_t stream);

/* ---- stage 3: dispatch-side permutation (Fig. 1, "Dispatch"; Section 1) --------------------
 * Groups the P pairs by destination slot, keeping ascending pair index inside a destination:
 *   dest_counts[d]  = #{p : assigned_slot[p] = d}                     uint32 [D]
 *   dest_offsets    = exclusive scan of dest_counts, last entry = P   uint32 [D+1]
 *   row_of_pair[p]  = dest_offsets[d_p] + #{q < p : d_q = d_p}        int32 [P]
 *   pair_of_row     = inverse of row_of_pair (NULL to skip)           int32 [P]
 *   send[row_of_pair[p]] = x[p / K]    bit copy of H 16-bit elements  bf16 [P, H]
 * x is bf16 [T, H].  cobalt_permute = cobalt_permute_index followed by cobalt_permute_rows;
 * the two halves are exported so that the maps can be reused (e.g. for another tensor).
 * The rows are moved as bits, so cobalt_permute_rows serves any element type whose row is a
 * multiple of 16 bytes: pass H = row bytes / 2 (an 8-bit tensor of 7168 columns is H = 3584). */
size_t cobalt_permute_workspace_bytes(int64_t T, int32_t K, int32_t D);
int cobalt_permute_index(const int32_t* assigned_slot, int64_t T, int32_t K, int32_t D,
                         uint32_t* dest_counts, uint32_t* dest_offsets, int32_t* row_of_pair,
                         int32_t* pair_of_row, void* workspace, size_t workspace_bytes,
                         cobalt_stream_t stream);
int cobalt_permute_rows(const void* x, const int32_t* row_of_pair, int64_t T, int32_t K,
                        int32_t H, void* send, uint32_t flags, cobalt_stream_t stream);
/* Token-block form: moves only T tokens whose rows x, and whose T*K entries of row_of_pair, the
 * caller passes already offset to the block; the row indices still address the whole send
 * buffer of total_rows rows.  cobalt_permute_rows is the block form with total_rows = T*K.
 * Lets a caller stream a step in token blocks (e.g. while the hidden rows are still arriving). */
int cobalt_permute_rows_block(const void* x, const int32_t* row_of_pair, int64_t T, int32_t K,
                              int32_t H, void* send, int64_t total_rows, uint32_t flags,
                              cobalt_stream_t stream);
int cobalt_permute(const int32_t* assigned_slot, int64_t T, int32_t K, int32_t D,
                   const void* x, int32_t H, void* send, uint32_t* dest_counts,
                   uint32_t* dest_offsets, int32_t* row_of_pair, int32_t* pair_of_row,
                   uint32_t flags, void* workspace, size_t workspace_bytes,
                   cobalt_stream_t stream);

/* ---- stages 1 + 2 + index half of stage 3 in one pass over the ids ---------------------------
 * Same outputs, bit for bit, as cobalt_coact_stats, cobalt_assign (Algorithm 1, hashed replica
 * pick) and cobalt_permute_index called one after the other, with dest_counts = slot_load = w_er.
 * (Section 3.2 Stage 1, Section 3.3 Algorithm 1, Fig. 1 "Dispatch".)  ONE kernel does it: a grid of
 * at most one CTA per SM, launched cooperatively, reads the top-k ids once, keeps the co-activation
 * triangle, the layout tables and the lane masks that rank the pairs in shared memory, exchanges
 * per-CTA partial results through the workspace across one grid-wide barrier (bounded wait:
 * COBALT_DEVERR_WAIT_TIMEOUT if it ever ran out) and stores every output; nothing is cleared
 * beforehand and no output is written with atomics unless COBALT_STATS_ACCUMULATE is set.
 * The kernel serves K = 1 .. 16, D <= 1024 and layouts whose triangle fits beside the other tables
 * (about 400 experts at D = 288, fewer with more destinations), on devices that support
 * cooperative launches; every other case runs the three separate calls internally, with the same
 * results.  The workspace query covers both (about 10 MB at E = 256, D = 288).  Two calls that
 * run on the GPU at the same time need a workspace each.
 * flags: COBALT_STATS_ACCUMULATE, COBALT_SEED_ON_DEVICE, COBALT_STATS_TILE32, COBALT_ROUTE_SEPARATE_KERNELS
 * (the last two select kernel variants, not results).  remote_nodes, totals, pair_of_row may be NULL.
 * Follow with cobalt_permute_rows to fill the send buffer. */
size_t cobalt_route_index_workspace_bytes(const cobalt_layout_t* layout, int64_t T, int32_t K);
int cobalt_route_index(const cobalt_layout_t* layout, const int32_t* topk_ids, const int32_t* src_rank,
                       int32_t src_rank_uniform, int64_t T, int32_t K, uint64_t seed,
                       uint32_t* coact, uint32_t* load, int32_t* assigned_slot,
                       uint8_t* remote_nodes, uint64_t* totals, uint32_t* dest_counts,
                       uint32_t* dest_offsets, int32_t* row_of_pair, int32_t* pair_of_row,
                       uint32_t flags, void* workspace, size_t workspace_bytes,
                       cobalt_stream_t stream);

/* ---- index half of stage 3 for callers that cannot provide device scratch -------------------
 * (No counterpart in the paper: this is a packaging variant of cobalt_permute_index, same
 * inputs, same outputs, bit-identical results.)
 * Some callers cannot allocate device memory where they call the library: code running inside
 * a framework that forbids allocator calls on its hot path, plugins that receive nothing but
 * their input and output buffers, and jobs whose memory pool was sized up front and is fully
 * committed.  For them the per-chunk histogram scratch is a fixed array inside the library
 * image, COBALT_STATIC_SCRATCH_WORDS uint32 (4 MiB), which every GPU that loads the library
 * holds until the process exits.  The call needs D * ceil(P / chunk) words, where chunk is
 * 2048 pairs (doubled until there are at most 2048 chunks); larger problems are refused with
 * COBALT_ERR_SCRATCH_LIMIT and nothing is enqueued.  D = 288 fits for every P; D = 4096 fits up
 * to P = 524288.  The call itself performs no device or host allocation.
 * The first call on each device looks up the array's device address (with that device
 * current) and caches it; make that first call outside any stream capture.
 * All calls share the one array and it keeps whatever the previous call left there.  Nothing
 * has to be cleared between calls, because the first kernel overwrites every word the later
 * ones read, but two calls that overlap on the GPU (different streams, or different host
 * threads without ordering) race on it: serialise them on one stream or with events. */
#define COBALT_STATIC_SCRATCH_WORDS (1u << 20)
int cobalt_permute_index_static(const int32_t* assigned_slot, int64_t T, int32_t K, int32_t D,
                                uint32_t* dest_counts, uint32_t* dest_offsets,
                                int32_t* row_of_pair, int32_t* pair_of_row,
                                cobalt_stream_t stream);

/* ---- stage 4: combine (Fig. 1, "Weighted sum"; Section 1) ----------------------------------
 * y[t][h] = bf16( sum_{k<K} gate_w[t*K+k] * float(expert_out[row_of_pair[t*K+k]][h]) ),
 * fp32 accumulation in ascending k, one round-to-nearest-even at the end.
 * expert_out: bf16 [P, H] in the row order of `send`.  gate_w: fp32 [P] (required: NULL is
 * COBALT_ERR_INVALID_ARG).  y: bf16 [T, H]. */
int cobalt_combine(const void* expert_out, const int32_t* row_of_pair, const float* gate_w,
                   int64_t T, int32_t K, int32_t H, void* y, uint32_t flags,
                   cobalt_stream_t stream);
/* Token-block form: row_of_pair, gate_w and y are passed offset to a block of T tokens;
 * expert_out is the whole buffer of total_rows rows.  cobalt_combine is total_rows = T*K. */
int cobalt_combine_block(const void* expert_out, const int32_t* row_of_pair, const float* gate_w,
                         int64_t T, int32_t K, int32_t H, void* y, int64_t total_rows,
                         uint32_t flags, cobalt_stream_t stream);

/* ---- backward of the two row stages (the method is used in training: Section 1) --------------
 * The forward maps are linear, send[r(t,k)] = x[t] and y[t] = sum_k g[t][k] * out[r(t,k)] with
 * r(t,k) = row_of_pair[t*K+k]; these are their adjoints.
 * cobalt_permute_backward: grad_x[t] = bf16( sum_k float(grad_send[r(t,k)]) ), fp32 accumulation in
 *   ascending k.  grad_send bf16 [P, H], grad_x bf16 [T, H].
 * cobalt_combine_backward: grad_expert_out[r(t,k)] = bf16( g[t][k] * float(grad_y[t]) ) and
 *   grad_gate_w[t*K+k] = sum_h float(grad_y[t][h]) * float(expert_out[r(t,k)][h]) in fp32 (a fixed
 *   reduction tree: results do not vary from run to run).  Either output may be NULL (expert_out
 *   is only read for grad_gate_w).  grad_y bf16 [T, H], grad_expert_out bf16 [P, H], grad_gate_w
 *   fp32 [P]. */
int cobalt_permute_backward(const void* grad_send, const int32_t* row_of_pair, int64_t T, int32_t K,
                            int32_t H, void* grad_x, uint32_t flags, cobalt_stream_t stream);
int cobalt_combine_backward(const void* grad_y, const void* expert_out, const int32_t* row_of_pair,
                            const float* gate_w, int64_t T, int32_t K, int32_t H,
                            void* grad_expert_out, float* grad_gate_w, uint32_t flags,
                            cobalt_stream_t stream);

/* ---- statistics epilogue and Stage 2 of the layout planner (Section 3.2) ---------------------
 * cobalt_ema_update: ema[i] = decay * ema[i] + (1 - decay) * counts[i] for n entries (device arrays;
 *   counts uint32, ema fp32), the moving averages w^_e, c^_ij and w_er the planner reads.  The paper
 *   gives no decay constant: it is the caller's.  COBALT_EMA_INITIALISE sets ema = counts instead.
 * cobalt_ochiai: ochiai[i*E+j] = coact[i*E+j] / sqrt(coact[i*E+i] * coact[j*E+j]), 0 where either
 *   expert was never selected (the similarity of Section 1's footnote).  fp32 [E*E] on the device.
 * cobalt_rebalance_intra_node (host arrays only, no device work): per node, re-partitions the
 *   replicas among the node's ranks by greedy bin packing on slot_load_host (fp32 [G*S], the EMA of
 *   w_er): longest first (ties: lower expert id, then lower old slot), each to the least-loaded
 *   rank of its node that has a free slot and does not hold that expert yet (ties: lower rank);
 *   slots of a rank fill in placement order.  A node where some replica finds no admissible rank
 *   keeps its placement.  Outputs: new_slot_expert_host [G*S]; moved_from_host [G*S] (old slot
 *   of every new slot, -1 for empty; may be NULL); *nodes_kept_host (may be NULL).  Replicas never
 *   leave their node, so no cross-node parameter movement is implied.  The load of every occupied
 *   slot must be finite and >= 0 (COBALT_ERR_INVALID_ARG otherwise). */
#define COBALT_EMA_INITIALISE 0x1u
int cobalt_ema_update(const uint32_t* counts, float* ema, int64_t n, float decay, uint32_t flags,
                      cobalt_stream_t stream);
int cobalt_ochiai(const uint32_t* coact, int32_t E, float* ochiai, cobalt_stream_t stream);
int cobalt_rebalance_intra_node(int32_t num_nodes, int32_t ranks_per_node, int32_t slots_per_rank,
                                int32_t num_experts, const int32_t* slot_expert_host,
                                const float* slot_load_host, int32_t* new_slot_expert_host,
                                int32_t* moved_from_host, int32_t* nodes_kept_host);

/* ---- node-deduplicated send layout (Section 3.1, Eq. 1; Section 1 on node-level dedup) -------
 * When ranks of one node need the same token it crosses the network once and is forwarded inside
 * the node; Eq. 1 counts exactly those crossings.  cobalt_dedup_index lays the send buffer out
 * accordingly: ONE row per (token, destination node), grouped by destination node in ascending
 * token order.
 *   node_counts[n]              rows for node n                                uint32 [N]
 *   node_offsets                exclusive scan, last = total rows              uint32 [N+1]
 *   node_row_of_token[t*N+n]    row of token t in node n's group, -1 if none   int32 [T*N]
 *   fwd_src_row[p]              row pair p is forwarded from on arrival        int32 [P]
 *   cross_node_rows[0]          rows whose node differs from the source node = V of Eq. 1
 *                               (uint64 [1]; may be NULL)
 * Fill the buffer with cobalt_permute_rows_block(x, node_row_of_token, T, N, H, dedup_send,
 * capacity_rows, ...) (N "copies" per token, absent nodes skipped; T*min(K,N) rows always
 * suffice).  cobalt_forward_rows is the receiving side's expansion,
 * recv[row_of_pair[p]] = dedup_send[fwd_src_row[p]], which reproduces the buffer of
 * cobalt_permute bit for bit.  src_rows / dst_rows bound the two index arrays. */
size_t cobalt_dedup_workspace_bytes(int64_t T, int32_t K, int32_t num_nodes);
int cobalt_dedup_index(const int32_t* assigned_slot, const int32_t* src_rank, int32_t src_rank_uniform,
                       int64_t T, int32_t K, int32_t num_nodes, int32_t ranks_per_node,
                       int32_t slots_per_rank, uint32_t* node_counts, uint32_t* node_offsets,
                       int32_t* node_row_of_token, int32_t* fwd_src_row, uint64_t* cross_node_rows,
                       void* workspace, size_t workspace_bytes, cobalt_stream_t stream);
int cobalt_forward_rows(const void* dedup_send, const int32_t* fwd_src_row, const int32_t* row_of_pair,
                        int64_t P, int32_t H, void* recv, int64_t src_rows, int64_t dst_rows,
                        cobalt_stream_t stream);

/* ---- device error word -------------------------------------------------------------------
 * Waits for `stream`, copies the COBALT_DEVERR_* bits set by kernels on the current device
 * since the last call into *out_bits_host and clears them. */
int cobalt_read_and_clear_device_error(uint32_t* out_bits_host, cobalt_stream_t stream);

#ifdef __cplusplus
}
#endif
#endif /* COBALT_H_ */
