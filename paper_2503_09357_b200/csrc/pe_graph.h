// Internal: host-side graph handle and the device-side view kernels receive.
#pragma once
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include <mutex>

#include "pe.h"

// One record per operator i, 16 bytes: where its incoming edges start in the by-predecessor
// CSR, how many there are, its duration D^o_i and its memory adjustment A_i.
struct PeOpRec {
  int32_t edge_begin;
  int32_t indeg;
  int32_t dur;
  int32_t mem_delta;
};

// Byte offsets of the arrays inside the graph blob (one contiguous, 16-byte aligned block in
// device memory, copied verbatim into shared memory by the kernels that stage it).
struct PeBlobLayout {
  uint32_t ops;     // PeOpRec[V]
  uint32_t pred;    // int32[E]      predecessor id of CSR slot q
  uint32_t comm;    // int32[E*L]    D^c of CSR slot q over link class l at q*L + l
  uint32_t weight;  // int32[V]      W_i (present only if has_weight)
  uint32_t cls;     // uint8[D*D]    link class of (machine of predecessor, machine of successor)
  uint32_t cap;     // int32[D]      capacity (INT32_MAX where there is no limit)
  uint32_t durm;    // int32[V*D]    duration of operator i on machine j at i*D + j (present only if hetero)
  uint32_t bytes;   // total, multiple of 16
};

// What a kernel needs to know about the graph; `base` points at the blob (global or shared).
struct PeGraphView {
  int32_t V, E, D, L;
  int32_t has_weight;
  int32_t hetero;   // durations depend on the machine (the blob holds durm)
  PeBlobLayout lay;
};

// Compact ("narrow") encoding of the same graph, built when every value fits: V <= 65535,
// D^o and D^c below 65536, A in int8, L <= 2, in-degree <= 255, E < 2^24.  One 16-byte record
// per operator carries its first incoming edges inline, so the common operator needs a single
// load.  An edge is  lo = comm[class 0] << 16 | pred  (plus  hi = comm[class 1]  when L == 2).
//   w1 = indeg << 24 | (uint8)A << 16 | dur
//   L == 1: w2, w3 = lo of incoming edges 0 and 1;
//           w0 = lo of incoming edge 2 when indeg <= 3, else the CSR slot of the first incoming
//           edge (edges 2.. are then read from the CSR list)
//   L == 2: (w2, w3) = (lo, hi) of incoming edge 0; w0 = CSR slot of the first incoming edge
// followed by all incoming edges again in CSR order (4 bytes each for L == 1, 8 for L == 2).
// An inline slot without an edge holds pred = V with zero delay: kernels keep a sentinel state
// row V ("ended at time 0 on machine 0"), so the slot can be evaluated without a branch.
struct PeNarrowView {
  int32_t V, E, D, L;
  int32_t has_weight;
  int32_t need_cls;   // the link-class table must be consulted (L > 1 or some pair has no channel)
  int32_t max_indeg;  // largest in-degree (kernels skip the third inline slot when it is <= 2)
  uint32_t ops;       // uint4[V]
  uint32_t edges;     // uint32[E] (L == 1) or uint2[E] (L == 2)
  uint32_t weight;    // int32[V] if has_weight
  uint32_t cls;       // uint8[D*D]
  uint32_t cap;       // int32[D]
  uint32_t bytes;     // total, multiple of 16
};

// Forward view of the DAG for priority-list decoding, built when V <= 65536 and no operator has
// more than 255 incoming edges: successors of operator i are succ[ptr[i] .. ptr[i+1]).
struct PeFwdView {
  int32_t V, E;
  uint32_t ptr;    // uint32[V + 1]
  uint32_t succ;   // uint16[E]
  uint32_t indeg;  // uint8[V]
  uint32_t bytes;  // total, multiple of 16
};

struct pe_graph {
  int32_t V, E, D, L;
  int device;
  bool has_weight;
  bool hetero;         // durations depend on the machine
  int64_t time_bound;  // sum dur + sum_e max_l comm: no start/end time exceeds it
  int64_t mem_bound;   // sum |A| + sum W
  int32_t max_indeg;
  PeBlobLayout lay;
  uint8_t* d_blob;     // device copy of the blob
  bool narrow_ok;      // the compact encoding exists
  PeNarrowView nview;
  uint8_t* d_nblob;    // device copy of the compact encoding (nullptr if !narrow_ok)
  bool fwd_ok;         // the forward view exists
  PeFwdView fview;
  uint8_t* d_fwd;      // device copy of the forward view (nullptr if !fwd_ok)
  int* d_error;        // device status word (0 = ok)
  // pe_eval_batch_host pipelines copies and kernels over candidate chunks: one stream per copy
  // direction and one event per chunk and stage, created with the graph; `host_mutex` serialises
  // host-buffer calls on the same graph because they share these.
  static constexpr int kMaxChunks = 16;
  cudaStream_t copy_in, copy_out;
  cudaEvent_t ev_begin, ev_end, ev_in[kMaxChunks], ev_done[kMaxChunks];
  std::mutex host_mutex;
  // pe_eval_batch with the TEAM variant works through chunks of candidates; consecutive chunks alternate
  // between two side streams so that the staging transpositions of one overlap the evaluation of the
  // other.  `team_mutex` serialises the enqueueing of such calls on one graph (they share the events).
  cudaStream_t team_stream[2];
  cudaEvent_t team_fork, team_join[2];
  std::mutex team_mutex;
  int sm_count;
  size_t smem_optin;   // max dynamic shared memory per block
  size_t smem_per_sm;  // shared memory of an SM
};

inline PeGraphView pe_view(const pe_graph* g) {
  PeGraphView v;
  v.V = g->V; v.E = g->E; v.D = g->D; v.L = g->L;
  v.has_weight = g->has_weight ? 1 : 0;
  v.hetero = g->hetero ? 1 : 0;
  v.lay = g->lay;
  return v;
}
