/* pe.h — batched evaluation of candidate parallel plans (C ABI).
 *
 * Problem data follow the problem statement of Section III of "Automatic Operator-level
 * Parallelism Planning for Distributed Deep Learning — A Mixed-Integer Programming
 * Approach" (arXiv 2503.09357): an operator DAG G_m(I, B) with durations D^o_i, per-edge
 * communication durations D^c, memory adjustments A_i and weights W_i, and a cluster of
 * machines whose channels are grouped into link classes, each machine with a memory limit.
 *
 * A candidate plan is (x, pi): x[i] is the machine of operator i (Eq. 6) and pi a global
 * priority order that is a topological order of G_m; pi fixes every precedence variable
 * y of Eqs. 7-8.  For each candidate the library computes the componentwise-least start
 * and end times satisfying Eq. 3, Eqs. 7-8 and Eqs. 11-13 (communication is a delay
 * charged only between different machines), the makespan (Eqs. 1-2), each machine's busy
 * time (its bubble is makespan - busy) and each machine's peak memory level along its own
 * operator sequence (Eqs. 16-19), plus status flags.  All quantities are int32.
 *
 * Layout.  Per-candidate arrays are candidate-interleaved: element (row, c) of an [R][K]
 * array is at index row*K + c.  "By-op" arrays have one row per operator id, "by-pos"
 * arrays one row per position k of the priority order, per-machine arrays one row per
 * machine.
 *
 * Threading / ownership.  A pe_graph is immutable after creation and may be used from
 * several host threads and streams.  The library allocates device memory only in
 * pe_graph_create (the graph copy, a few KB..MB); candidates, outputs and workspace
 * belong to the caller.  No function throws; every error is a negative return code.
 */
#ifndef PE_H_
#define PE_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct pe_graph pe_graph; /* opaque; owns the device copy of the problem data */

/* Return codes. */
enum {
  PE_OK = 0,
  PE_ERR_INVALID_ARG = -1, /* NULL where data is required, sizes out of range, bad flags */
  PE_ERR_CYCLE = -2,       /* the edge list is not a DAG */
  PE_ERR_RANGE = -3,       /* negative duration / communication / weight, edge endpoint or link class out of range */
  PE_ERR_OVERFLOW = -4,    /* sum(dur) + sum_e max_l comm, or sum|A| + sum W, does not fit in int32 */
  PE_ERR_CUDA = -5,        /* a CUDA runtime call failed (no device, out of memory, launch error) */
  PE_ERR_WORKSPACE = -6,   /* workspace pointer NULL or smaller than pe_workspace_bytes() */
  PE_ERR_TIMEOUT = -7,     /* a bounded device-side wait expired (reported by pe_graph_poll_error) */
  PE_ERR_UNSUPPORTED = -8, /* the requested kernel variant cannot run this problem size */
  PE_ERR_SCRATCH_LIMIT = -9 /* pe_eval_batch_noalloc: the batch needs more than PE_NOALLOC_SCRATCH_BYTES of scratch */
};

/* Problem data (Section III).  All pointers are HOST pointers, read during the call only. */
typedef struct {
  int32_t num_ops;             /* V = |I| >= 1 */
  int32_t num_edges;           /* E = |B| >= 0 */
  const int32_t* edge_src;     /* [E] i1 of (i1, i2) in B */
  const int32_t* edge_dst;     /* [E] i2 */
  const int32_t* dur;          /* [V] D^o_i >= 0 */
  const int32_t* mem_delta;    /* [V] A_i, signed; NULL = all 0 */
  const int32_t* mem_weight;   /* [V] W_i >= 0; NULL = all 0 */
  int32_t num_devices;         /* D = |J|, 1..255 */
  int32_t num_link_classes;    /* L, 1..254 */
  const uint8_t* link_class;   /* [D*D] row-major: class of the channel (machine of i1 -> machine of i2);
                                  the diagonal is ignored; 0xFF = no channel (Eq. 10); NULL = all class 0 */
  const int32_t* comm;         /* [E*L] D^c of edge e over link class l at e*L + l, >= 0; NULL = all 0 */
  const int32_t* mem_capacity; /* [D] memory limit per machine; NULL = no limit */
  const int32_t* dur_by_machine; /* [V*D] heterogeneous machines (Section III, footnote: the model extends by giving
                                  the duration a machine index): operator i lasts dur_by_machine[i*D + j] >= 0 on
                                  machine j, D^o_i of Eq. 3 becoming D^o_{i,x_i}; NULL = homogeneous (`dur` applies).
                                  `dur` must still be given (it is ignored by the evaluation when this is set).
                                  Such graphs are evaluated by the one-thread-per-candidate kernels
                                  (PE_VARIANT_SHARED / PE_VARIANT_GLOBAL); PE_VARIANT_WARP and PE_VARIANT_TEAM return
                                  PE_ERR_UNSUPPORTED for them. */
} pe_graph_desc;

/* Host-only check of a description: ranges, acyclicity, overflow bounds.  Touches no GPU. */
int pe_graph_validate(const pe_graph_desc* desc);

/* Validate, build the by-predecessor CSR and upload it to CUDA device `cuda_device`.
 * On success *out owns the device copy until pe_destroy.  Synchronous. */
int pe_graph_create(const pe_graph_desc* desc, int cuda_device, pe_graph** out);

/* Free the device copy.  NULL is accepted.  The caller must have finished all work using it. */
int pe_destroy(pe_graph* g);

/* Flags of pe_eval_batch. */
enum {
  PE_ASSIGN_BY_POS = 1u, /* `assign` row k holds x[pi[k]] (the machine sequence) instead of row i holding x[i] */
  PE_TIMES_BY_OP = 2u,   /* `start` / `finish` row i belongs to operator i instead of row k to position k */
  PE_COMM_EXCLUSIVE = 4u, /* a channel (machine j1 -> machine j2) carries one transfer at a time (Section III;
                            Eqs. 14-15) instead of transfers being pure delays.  The transfers of a channel follow
                            each other in the order in which their receiving operators appear in pi (as pi fixes y),
                            those into one operator in the order of the edge list; the transfer of (i1, i2) starts
                            at max(e_i1, end of the channel's previous transfer) (Eqs. 13, 14), lasts D^c (Eq. 11),
                            and i2 starts no earlier than its end (Eq. 12).  Offered by the shared-state kernel (no
                            workspace) and the global-state kernel (D*D*K*4 more bytes of workspace), not by
                            PE_VARIANT_WARP; ask pe_workspace_bytes with the same flags. */
  /* Kernel variant (bits 8..11); 0 lets the library choose from (V, E, D, L) and the device. */
  PE_VARIANT_AUTO = 0u << 8,
  PE_VARIANT_GLOBAL = 1u << 8, /* one thread per candidate, finish-time state in the caller's workspace */
  PE_VARIANT_SHARED = 2u << 8, /* one thread per candidate, finish-time state in shared memory */
  PE_VARIANT_WARP = 3u << 8,   /* one warp per candidate, finish-time state in shared memory */
  PE_VARIANT_TEAM = 4u << 8,   /* one block of several warps per candidate, finish-time state in shared memory; the
                                  warps prepare windows of the order side by side and only the recurrence of
                                  Eqs. 3, 7-8, 11-13 runs window after window.  For graphs with in-degree <= 8 and
                                  16-bit orders, with start and finish both wanted or both absent; otherwise
                                  PE_ERR_UNSUPPORTED.  Uses workspace (staging copies) when K is a multiple of 4 */
  PE_VARIANT_MASK = 15u << 8
};

/* Status bits per candidate (0 = a valid topological permutation, feasible). */
enum {
  PE_STATUS_ASSIGN_RANGE = 1u,  /* a consulted machine id is >= D */
  PE_STATUS_ORDER_INVALID = 2u, /* an order entry >= V, a repeated operator, or an operator placed before a predecessor */
  PE_STATUS_MEM_EXCEEDED = 4u,  /* some machine's peak memory level is above its capacity (Section III) */
  PE_STATUS_NO_CHANNEL = 8u     /* an edge crosses a machine pair whose link class is 0xFF (Eq. 10); delay taken as 0 */
};
/* For a candidate with bit 1 or 2 set every other output (and status bits 4, 8) is unspecified. */

/* Outputs: DEVICE pointers owned by the caller; a NULL member is not computed/written. */
typedef struct {
  int32_t* start;    /* [V*K] s, by-pos (default) or by-op (PE_TIMES_BY_OP) */
  int32_t* finish;   /* [V*K] e, same layout */
  int32_t* makespan; /* [K]   max_i e_i (Eq. 2) */
  int32_t* busy;     /* [D*K] sum of D^o over the operators of machine j */
  int32_t* peak_mem; /* [D*K] max over prefixes (the empty one included) of the machine's memory level */
  uint32_t* status;  /* [K]   PE_STATUS_* bits */
} pe_outputs;

/* Bytes of device workspace pe_eval_batch needs for K candidates with these flags (may be 0). */
size_t pe_workspace_bytes(const pe_graph* g, int64_t K, uint32_t flags);

/* Which kernel variant (PE_VARIANT_*) a call with these arguments runs; negative = error code. */
int pe_eval_variant(const pe_graph* g, int64_t K, uint32_t flags);

/* Evaluate K candidates.  Asynchronous on `cuda_stream` (a cudaStream_t; NULL = default stream);
 * never synchronises.  K = 0 is a successful no-op.
 *   assign      device, u8 [V*K]: by-op x_c[i] at i*K + c, or by-pos under PE_ASSIGN_BY_POS
 *   order       device, [V*K] by-pos pi_c[k] at k*K + c; uint16_t if order_bytes == 2 (V <= 65536), uint32_t if 4
 *   out         outputs wanted (struct read during the call)
 *   workspace   device scratch of at least pe_workspace_bytes() bytes, 256-byte aligned; contents are
 *               overwritten; calls running concurrently must not share it
 * Precondition: every candidate's order is a topological permutation and every machine id < D;
 * violations are flagged per candidate in `status` and never index out of bounds. */
int pe_eval_batch(pe_graph* g, int64_t K, const uint8_t* assign, const void* order, int order_bytes, uint32_t flags,
                  const pe_outputs* out, void* workspace, size_t workspace_bytes, void* cuda_stream);

/* Host-buffer form of the same call: evaluates K candidates whose inputs and outputs live in HOST
 * memory, and synchronises the stream before returning.  The batch is processed in chunks of
 * candidates so that the upload of one chunk, the kernel of another and the download of a third
 * overlap (copies run on two streams owned by the graph, kernels on `cuda_stream`); pinned host
 * memory is needed for that overlap, pageable memory still gives correct results.
 *   host_assign / host_order   inputs, laid out as for pe_eval_batch
 *   host_out                   HOST pointers of the outputs wanted, laid out as for pe_eval_batch
 *   dev_assign [V*K] u8, dev_order [V*K*order_bytes], dev_out (DEVICE pointers for exactly the
 *   members set in host_out, each of the full size)   caller-owned staging; their contents after
 *   the call are chunk-blocked, not the [rows][K] layout, and should be treated as scratch
 *   workspace                  as for pe_eval_batch with this K
 * Calls on the same graph are serialised internally (they share the graph's copy streams). */
int pe_eval_batch_host(pe_graph* g, int64_t K, const uint8_t* host_assign, const void* host_order, int order_bytes,
                       uint32_t flags, const pe_outputs* host_out, uint8_t* dev_assign, void* dev_order,
                       const pe_outputs* dev_out, void* workspace, size_t workspace_bytes, void* cuda_stream);

/* Evaluation for callers that must not allocate device memory.  (The paper has no counterpart:
 * this is a convenience of the library, not a step of the method.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits - inside a memory pool or framework
 * that owns every byte of the device and forbids side allocations, in a latency-critical loop
 * where an allocation would synchronise the device, or in a process whose memory budget was fixed
 * at start-up.  pe_eval_batch asks such a caller for a workspace it cannot provide; this entry
 * point brings its own.
 *
 * It runs the one-thread-per-candidate kernel whose per-operator state lives in global memory
 * (the PE_VARIANT_GLOBAL kernel), with that state in a fixed array of PE_NOALLOC_SCRATCH_BYTES
 * that is part of the library image: every GPU on which the library is used holds it from the
 * first use until the process exits.  Inputs and outputs are still the caller's device buffers,
 * with the meaning and layouts of pe_eval_batch; flags may hold PE_ASSIGN_BY_POS and
 * PE_TIMES_BY_OP only (no variant bits).  Results are identical to pe_eval_batch's.
 *
 *  - Size limit: the scratch this call's kernel needs (about 4*V*K bytes, 5*V*K with PE_ASSIGN_BY_POS
 *    on graphs without a compact encoding; never more than pe_workspace_bytes(g, K, flags |
 *    PE_VARIANT_GLOBAL)) must not exceed PE_NOALLOC_SCRATCH_BYTES; a larger batch is refused with
 *    PE_ERR_SCRATCH_LIMIT and nothing is launched.  Split the batch instead.
 *  - The first call on each device looks up the array's device address (a short, synchronous
 *    set-up with that device current); make that first call before starting any stream capture.
 *  - No cudaMalloc, cudaFree or other allocating routine is called, on any call.
 *  - All calls share the one array per device.  Each call re-initialises the part it uses on
 *    `cuda_stream` before its kernel, so stale contents never leak into a result; but two calls
 *    that can overlap on the GPU (different streams, or different host threads without ordering)
 *    race on it and give wrong results.  Order them on one stream or with events.
 * Asynchronous on `cuda_stream`, like pe_eval_batch. */
#define PE_NOALLOC_SCRATCH_BYTES (64u << 20)
int pe_eval_batch_noalloc(pe_graph* g, int64_t K, const uint8_t* assign, const void* order, int order_bytes,
                          uint32_t flags, const pe_outputs* out, void* cuda_stream);

/* Priority-list decoding: the step in front of pe_eval_batch.  The paper prints no decoder from a priority
 * list to (x, pi); Section IV mentions dispatch rules only as the inspiration of its coarsening heuristic.
 * The rule below is this library's choice; what the model requires is that the resulting order be
 * consistent with B (Eq. 8).
 * A candidate ranks the operators through a list; the priority order is then built position by position:
 * among the operators not yet placed whose predecessors in B have all been placed, the one of smallest rank
 * comes next.  The result is a topological order of G_m - a valid `order` argument of pe_eval_batch - and a
 * list that already is one comes back unchanged.
 *   list        device, uint16_t [V*K]: list_c[r] = operator of rank r (0 = most urgent) at r*K + c; any
 *               permutation of the operators, it need not respect the edges
 *   order_bytes 2 (uint16_t entries); 4 is PE_ERR_UNSUPPORTED, as are V > 65536 and in-degrees above 255
 *   flags       0, or PE_VARIANT_SHARED / PE_VARIANT_GLOBAL to force where the per-candidate state lives
 *   order       device, uint16_t [V*K], out: pi_c[k] at k*K + c
 *   status      device, [K], out, may be NULL: PE_STATUS_ORDER_INVALID where the list is not a permutation
 *               (an entry >= V or an operator twice); that candidate's order is then left unwritten
 *   workspace   device scratch of at least pe_decode_workspace_bytes() bytes (may be 0), 256-byte aligned
 * Asynchronous on `cuda_stream`; never synchronises.  K = 0 is a successful no-op. */
size_t pe_decode_workspace_bytes(const pe_graph* g, int64_t K, uint32_t flags);
int pe_decode_variant(const pe_graph* g, int64_t K, uint32_t flags); /* PE_VARIANT_SHARED or _GLOBAL; negative = error */
int pe_decode_priority(pe_graph* g, int64_t K, const void* list, int order_bytes, uint32_t flags, void* order,
                       uint32_t* status, void* workspace, size_t workspace_bytes, void* cuda_stream);

/* Selection step after an evaluation (Eq. 1: the objective is the makespan; Section III: only
 * arrangements within every machine's memory limit are valid): among K evaluated candidates find the
 * one with the smallest makespan whose status has none of the bits in `reject_mask` set
 * (pass ~0u to require status == 0).  Ties go to the smallest candidate index.
 *   makespan, status   device, [K], as written by pe_eval_batch
 *   result             device, 4 x int64, 8-byte aligned: {best candidate index or -1 if none qualifies,
 *                      its makespan (INT32_MAX if none), number of qualifying candidates, internal}
 * Asynchronous on `cuda_stream`; `result` is overwritten (no initialisation needed; it also serves as
 * the reduction's running state, so concurrent calls need separate result buffers).  K = 0 writes
 * {-1, INT32_MAX, 0}.  K must be below 2^32. */
int pe_select_best(int64_t K, const int32_t* makespan, const uint32_t* status, uint32_t reject_mask, int64_t* result,
                   void* cuda_stream);

/* The k best candidates of an evaluation (Eq. 1; Section III validity as for pe_select_best): the qualifying
 * candidates (status has none of the `reject_mask` bits) with the smallest makespans, ties to the smallest
 * candidate index - what a search keeps as its elite.  The selection is a set: out_index lists it by
 * INCREASING CANDIDATE INDEX, not by makespan.
 *   makespan, status   device, [K], as written by pe_eval_batch
 *   k                  how many to keep (>= 0)
 *   out_index          device, int32 [k]: the chosen candidates; entries beyond *out_count are -1
 *   out_count          device, one int32: min(k, number of qualifying candidates)
 *   workspace          device scratch of at least pe_select_topk_workspace_bytes(K) bytes, 16-byte aligned
 * Asynchronous on `cuda_stream`; runs on the device that owns out_count.  K must be below 2^31. */
size_t pe_select_topk_workspace_bytes(int64_t K);
int pe_select_topk(int64_t K, const int32_t* makespan, const uint32_t* status, uint32_t reject_mask, int32_t k,
                   int32_t* out_index, int32_t* out_count, void* workspace, size_t workspace_bytes, void* cuda_stream);

/* Operator merging in front of candidate generation (Section IV, Algorithm 1): shrinks G_m(I, B) to at most
 * `target_ops` operators by repeatedly merging pairs, so that a search (or the paper's MIP) works on a graph
 * of manageable size.  Host-only: every pointer is a HOST pointer and no GPU is touched.
 *
 * The algorithm alternates two loops until |I| <= target_ops or a whole pass merges nothing: merges of pairs
 * joined by an edge, then merges of pairs not joined by a path.  Before candidates are looked for, the
 * topologically redundant edges {(i1, i2) in B : some i3 has (i1, i3) and (i3, i2) in B} are set aside
 * (Section IV's definition); merging works on the full edge set.
 *   - edge candidate: an edge (u, v) of the remaining graph where v has a single input and u a single output,
 *     merged duration <= max_dur_edge and merged memory requirement <= max_mem_edge.  Safe: no cycle can
 *     arise and the critical path keeps its length (Section IV).
 *   - non-edge candidate: two operators with no directed path between them in either direction (the paper says
 *     "without a direct edge"; incomparability is what rules out a cycle), within max_dur_nonedge and
 *     max_mem_nonedge - the stricter thresholds Section IV asks for are the caller's to choose.
 *   - among several candidates the one with the smallest merged duration goes first, ties to the smallest
 *     (u, v), a group being identified by its smallest operator (the paper does not say).
 *   - a merged operator's duration, A and W are the sums over its members (Section IV); it inherits every edge
 *     to or from a third operator; edges that become parallel (also duplicate input edges) are combined into
 *     one whose communication duration per link class is the larger of the two.  The memory requirement
 *     tested against the thresholds is W + max(A, 0) summed over the members (the paper gives no formula).
 * Outputs (caller-allocated): op_map [V] = merged operator of every original one, merged operators numbered in
 * the order of their smallest member; *num_ops_out, *num_edges_out; edge_src / edge_dst [E], comm [E * L]
 * (NULL allowed if the input has no comm), sorted by (source, destination); dur [V]; mem_delta, mem_weight [V]
 * (each may be NULL).  Only the first *num_ops_out / *num_edges_out entries are written.  The result is a
 * DAG and can go straight into pe_graph_create.  V above 16384 is PE_ERR_UNSUPPORTED (the adjacency is kept
 * as two V x V bit matrices), as is a description with dur_by_machine (Section IV sums one duration per
 * operator); the description is validated first (PE_ERR_CYCLE, PE_ERR_RANGE, ...). */
typedef struct {
  int32_t target_ops;      /* N >= 1: stop once |I| <= N */
  int32_t max_dur_edge;    /* thresholds of merges along an edge */
  int32_t max_mem_edge;
  int32_t max_dur_nonedge; /* thresholds of merges of unrelated operators */
  int32_t max_mem_nonedge;
} pe_coarsen_params;
int pe_coarsen(const pe_graph_desc* desc, const pe_coarsen_params* prm, int32_t* op_map, int32_t* num_ops_out,
               int32_t* num_edges_out, int32_t* edge_src, int32_t* edge_dst, int32_t* comm, int32_t* dur,
               int32_t* mem_delta, int32_t* mem_weight);

/* Synchronise `cuda_stream` and return the graph's device-side error word: PE_OK, or
 * PE_ERR_TIMEOUT if a kernel gave up a bounded wait (its outputs are then invalid).  Clears the word. */
int pe_graph_poll_error(pe_graph* g, void* cuda_stream);

/* Self-test of the library's bounded device-side wait (the only wait its kernels have is the one for the
 * bulk copy that stages the graph into shared memory): launches one small block whose barrier expects bytes
 * that no copy brings, so the wait runs out after 1024 polls, the block sets the graph's error word and
 * returns.  Nothing faults and nothing stays in flight; a following pe_graph_poll_error returns
 * PE_ERR_TIMEOUT once and the graph remains usable.  Asynchronous on `cuda_stream`. */
int pe_selftest_wait_timeout(pe_graph* g, void* cuda_stream);

/* Number of kernels this library has launched in this process so far (all graphs, all streams). */
int64_t pe_kernel_launches(void);

/* Static description of an error code. */
const char* pe_strerror(int code);

#ifdef __cplusplus
}
#endif
#endif /* PE_H_ */
