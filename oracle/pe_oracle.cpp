// CPU oracle for batched plan evaluation.  TEST INFRASTRUCTURE ONLY.
//
// This file is the slow, plain statement of what the evaluation computes.  It exists so
// that tests, the smoke check and the benchmark's cpu_baseline leg can compare the CUDA
// path against it; no product code may import, link or call it, and it shares no code
// with the CUDA path.
//
// What it computes, per candidate (x, pi) of one operator DAG G_m(I, B):
//   x[i]  = machine of operation i             (the x_{i,j} of Eq. 6, given as an index)
//   pi    = a total order of I that is a topological order of G_m; it fixes the
//           precedence variables y of Eqs. 7-8: y_{i1,i2} = 1 iff i1 comes before i2 in pi
// and the result is the componentwise-least (s, e) that satisfies
//   Eq. 3      e_i - s_i = D^o_i
//   Eqs. 7-8   two operations on one machine do not overlap, in the order pi gives them
//   Eqs. 11-13 s_{i2} >= e_{i1} + D^c_{i1,i2} for (i1,i2) in B (the transfer starts when
//              i1 ends and lasts D^c); the delay is charged only when i1 and i2 run on
//              different machines, with D^c taken for the link class of the channel
//              (machine of i1 -> machine of i2); a pair with no channel (Eq. 10) sets a flag
//   s_i >= 0   (Section III: every machine is available at the beginning)
// followed by z = max_i e_i (Eqs. 1-2), the busy time of each machine, and the memory
// levels of Eqs. 16-19 along each machine's own operation sequence: the level starts at
// the sum of W_i over the operations placed on the machine (Eq. 16), each operation adds
// A_i (Eq. 19), consecutive operations on a machine hand the level on (Eqs. 17-18); the
// peak is the largest level seen, the empty prefix included.  Exceeding the capacity is
// reported as a flag, never repaired (Section III: "valid arrangement").
//
// One forward pass in pi order yields that least solution exactly, because pi is a
// topological order of B joined with the per-machine chains.  By default channel exclusivity
// (Eqs. 14-15) is not applied: communication is a pure delay.
//
// With the flag kCommExclusive the channel (j1 -> j2) carries one transfer at a time
// (Section III: "each communication channel can only handle one communication task at a
// time"; Eqs. 14-15).  The paper leaves the sequence of the transfers on a channel to the
// solver (the variables w); here pi fixes it the way it fixes y: the transfers of a channel
// follow each other in the order in which their receiving operations appear in pi, and the
// transfers into one operation in the order of the edge list.  The transfer of edge (i1, i2)
// then starts at c = max(e_i1 (Eq. 13), end of the previous transfer on its channel (Eq. 14)),
// ends at d = c + D^c (Eq. 11), and s_i2 >= d (Eq. 12).  Edges inside one machine and edges
// over a machine pair without a channel move nothing and occupy nothing.
//
// Pins (tests/test_oracle_pins.py): exhaustive enumeration on tiny DAGs against a
// constraint checker, closed forms for uniform pipelines, single-machine prefix sums,
// lower/upper bounds, a longest-path library routine on the explicit disjunctive graph,
// metamorphic relations, hand-built status cases, and hand-computed worked examples.
// The paper's own DualPipe bubble figures for PP = 4 and 8 (Section V-A) are "parity
// unpinned": the schedule behind them and its microbatch count are not printed.
//
// The second function of this file, pe_oracle_decode (at the end), states the step before
// evaluation - turning an arbitrary priority list into a priority order - and is pinned by
// tests/test_decode_pins.py: brute force over all topological orders of tiny DAGs, the
// edge-free and chain cases, idempotence, and the input generator's own random-key sort.
//
// Arrays are candidate-interleaved: element (row, c) of a [R][K] array is at row*K + c.
#include <cstdint>
#include <vector>

namespace {

constexpr uint32_t kAssignByPos = 1u;  // `assign` holds x[pi[k]] at row k instead of x[i] at row i
constexpr uint32_t kTimesByOp = 2u;    // start/finish rows are operations instead of positions
constexpr uint32_t kCommExclusive = 4u;  // channels carry one transfer at a time (Eqs. 14-15), see below

constexpr uint32_t kStatusAssignRange = 1u;
constexpr uint32_t kStatusOrderInvalid = 2u;
constexpr uint32_t kStatusMemExceeded = 4u;
constexpr uint32_t kStatusNoChannel = 8u;

}  // namespace

// Heterogeneous machines (footnote of Section III: the model extends "by including the machine
// dimension relating to the operation allocation decisions"): when `dur_by_machine` is given, operation i
// lasts dur_by_machine[i * D + j] on machine j, i.e. D^o_i of Eq. 3 becomes D^o_{i, x_i}; everything else
// is unchanged.  With a NULL table this is the homogeneous evaluation.
extern "C" int pe_oracle_eval_hetero(int32_t V, int32_t E, const int32_t* edge_src, const int32_t* edge_dst,
                                     const int32_t* dur, const int32_t* dur_by_machine, const int32_t* mem_delta,
                                     const int32_t* mem_weight, int32_t D, int32_t L, const uint8_t* link_class,
                                     const int32_t* comm, const int32_t* mem_capacity, int64_t K, int64_t c_begin,
                                     int64_t c_end, const uint8_t* assign, const void* order, int order_bytes,
                                     uint32_t flags, int32_t* start, int32_t* finish, int32_t* makespan,
                                     int32_t* busy, int32_t* peak_mem, uint32_t* status) {
  if (V <= 0 || E < 0 || D <= 0 || D > 255 || L <= 0 || K < 0 || c_begin < 0 || c_end > K) return -1;
  if (order_bytes != 2 && order_bytes != 4) return -1;
  for (int32_t b = 0; b < E; ++b)
    if (edge_src[b] < 0 || edge_src[b] >= V || edge_dst[b] < 0 || edge_dst[b] >= V) return -1;

  // incoming edges of every operation: in_ptr[i] .. in_ptr[i+1] index in_edge[], which holds edge numbers
  std::vector<int32_t> in_ptr(V + 1, 0), in_edge(E);
  for (int32_t b = 0; b < E; ++b) in_ptr[edge_dst[b] + 1]++;
  for (int32_t i = 0; i < V; ++i) in_ptr[i + 1] += in_ptr[i];
  {
    std::vector<int32_t> fill(in_ptr.begin(), in_ptr.end() - 1);
    for (int32_t b = 0; b < E; ++b) in_edge[fill[edge_dst[b]]++] = b;
  }

  std::vector<int32_t> x(V), s(V), e(V), free_at(D), busy_j(D), lvl(D), peak(D);
  std::vector<uint32_t> pi_c(V);
  std::vector<char> done(V);
  std::vector<int32_t> chan_free((flags & kCommExclusive) ? (size_t)D * D : 0);  // end of the last transfer per channel

  for (int64_t c = c_begin; c < c_end; ++c) {
    uint32_t st = 0;
    // column c of the order array: pi_c[k] is the operation at position k
    for (int32_t k = 0; k < V; ++k) {
      const size_t at = (size_t)k * (size_t)K + (size_t)c;
      pi_c[k] = order_bytes == 2 ? (uint32_t)((const uint16_t*)order)[at] : ((const uint32_t*)order)[at];
    }
    auto pi = [&](int32_t k) -> uint32_t { return pi_c[k]; };

    // the assignment x of this candidate (Eq. 6), as one machine index per operation
    for (int32_t i = 0; i < V; ++i) x[i] = 0;
    if (flags & kAssignByPos) {
      for (int32_t k = 0; k < V; ++k) {
        const uint32_t i = pi(k);
        if (i >= (uint32_t)V) continue;
        int32_t j = assign[(size_t)k * (size_t)K + (size_t)c];
        if (j >= D) { st |= kStatusAssignRange; j = D - 1; }
        x[i] = j;
      }
    } else {
      for (int32_t k = 0; k < V; ++k) {
        const uint32_t i = pi(k);
        if (i >= (uint32_t)V) continue;
        int32_t j = assign[(size_t)i * (size_t)K + (size_t)c];
        if (j >= D) { st |= kStatusAssignRange; j = D - 1; }
        x[i] = j;
      }
    }

    // Eq. 16: the weights of everything placed on machine j are resident from the start
    for (int32_t j = 0; j < D; ++j) { free_at[j] = 0; busy_j[j] = 0; lvl[j] = 0; }
    if (mem_weight)
      for (int32_t i = 0; i < V; ++i) lvl[x[i]] += mem_weight[i];
    for (int32_t j = 0; j < D; ++j) peak[j] = lvl[j];
    for (int32_t i = 0; i < V; ++i) { done[i] = 0; s[i] = 0; e[i] = 0; }
    for (int32_t& v : chan_free) v = 0;
    int32_t z = 0;

    for (int32_t k = 0; k < V; ++k) {
      const uint32_t iu = pi(k);
      if (iu >= (uint32_t)V) { st |= kStatusOrderInvalid; continue; }
      const int32_t i = (int32_t)iu;
      if (done[i]) st |= kStatusOrderInvalid;
      const int32_t j = x[i];
      int32_t r = 0;  // earliest start allowed by the incoming transfers (Eqs. 11-13)
      for (int32_t q = in_ptr[i]; q < in_ptr[i + 1]; ++q) {
        const int32_t b = in_edge[q];
        const int32_t p = edge_src[b];
        if (!done[p]) { st |= kStatusOrderInvalid; continue; }
        int32_t t = e[p];
        if (x[p] != j) {
          const uint32_t cls = link_class ? link_class[(size_t)x[p] * D + j] : 0u;
          if (cls == 0xFFu) {
            st |= kStatusNoChannel;  // Eq. 10: no channel between the two machines
          } else if (flags & kCommExclusive) {
            int32_t& chan = chan_free[(size_t)x[p] * D + j];
            const int32_t c_start = t > chan ? t : chan;           // Eq. 13 and Eq. 14
            t = c_start + (comm ? comm[(size_t)b * L + cls] : 0);  // Eq. 11
            chan = t;
          } else {
            t += comm ? comm[(size_t)b * L + cls] : 0;
          }
        }
        if (t > r) r = t;
      }
      const int32_t d_i = dur_by_machine ? dur_by_machine[(size_t)i * D + j] : dur[i];  // D^o of i on its machine
      s[i] = r > free_at[j] ? r : free_at[j];  // Eq. 7 with y from pi: after everything earlier on machine j
      e[i] = s[i] + d_i;                       // Eq. 3
      free_at[j] = e[i];
      done[i] = 1;
      busy_j[j] += d_i;
      lvl[j] += mem_delta[i];                  // Eq. 19, handed on along the machine by Eqs. 17-18
      if (lvl[j] > peak[j]) peak[j] = lvl[j];
      if (e[i] > z) z = e[i];                  // Eq. 2
    }
    if (mem_capacity)
      for (int32_t j = 0; j < D; ++j)
        if (peak[j] > mem_capacity[j]) st |= kStatusMemExceeded;

    if (start || finish) {
      for (int32_t k = 0; k < V; ++k) {
        int32_t row, i;
        if (flags & kTimesByOp) { row = k; i = k; }
        else {
          const uint32_t iu = pi(k);
          row = k; i = iu < (uint32_t)V ? (int32_t)iu : 0;
        }
        const size_t at = (size_t)row * (size_t)K + (size_t)c;
        if (start) start[at] = s[i];
        if (finish) finish[at] = e[i];
      }
    }
    if (makespan) makespan[c] = z;
    for (int32_t j = 0; j < D; ++j) {
      if (busy) busy[(size_t)j * (size_t)K + (size_t)c] = busy_j[j];
      if (peak_mem) peak_mem[(size_t)j * (size_t)K + (size_t)c] = peak[j];
    }
    if (status) status[c] = st;
  }
  return 0;
}

extern "C" int pe_oracle_eval(int32_t V, int32_t E, const int32_t* edge_src, const int32_t* edge_dst,
                              const int32_t* dur, const int32_t* mem_delta, const int32_t* mem_weight, int32_t D,
                              int32_t L, const uint8_t* link_class, const int32_t* comm,
                              const int32_t* mem_capacity, int64_t K, int64_t c_begin, int64_t c_end,
                              const uint8_t* assign, const void* order, int order_bytes, uint32_t flags,
                              int32_t* start, int32_t* finish, int32_t* makespan, int32_t* busy, int32_t* peak_mem,
                              uint32_t* status) {
  return pe_oracle_eval_hetero(V, E, edge_src, edge_dst, dur, nullptr, mem_delta, mem_weight, D, L, link_class, comm,
                               mem_capacity, K, c_begin, c_end, assign, order, order_bytes, flags, start, finish,
                               makespan, busy, peak_mem, status);
}

// ---------------------------------------------------------------------------------------------
// Priority-list decoding: the step before evaluation.  TEST INFRASTRUCTURE ONLY, like the rest.
//
// The paper prints no decoder from a priority list to an order; Section IV mentions dispatch rules
// only as the inspiration of its coarsening heuristic.  The rule written out here (a choice of
// this repository, consistent with Eq. 8): a candidate gives every operation a priority rank through a list
// (list[r] = the operation of rank r, rank 0 the most urgent; any permutation of I, it need not
// respect the precedence edges B), and the priority order pi is built one position at a time:
// among the operations not yet placed whose predecessors in B have all been placed, the one of
// smallest rank comes next.  pi is therefore a topological order of G_m, which is what the
// evaluation above asks for, and a list that already is one is returned unchanged.
//
// A list that is not a permutation (an entry >= V, an operation twice) sets kStatusOrderInvalid
// and leaves that candidate's order unspecified.
// Arrays are candidate-interleaved like everything else: element (row, c) at row*K + c.
#include <queue>

extern "C" int pe_oracle_decode(int32_t V, int32_t E, const int32_t* edge_src, const int32_t* edge_dst, int64_t K,
                                int64_t c_begin, int64_t c_end, const void* list, int order_bytes, void* order,
                                uint32_t* status) {
  if (V <= 0 || E < 0 || K < 0 || c_begin < 0 || c_end > K || !list || !order) return -1;
  if (order_bytes != 2 && order_bytes != 4) return -1;
  for (int32_t b = 0; b < E; ++b)
    if (edge_src[b] < 0 || edge_src[b] >= V || edge_dst[b] < 0 || edge_dst[b] >= V) return -1;
  auto get = [&](const void* a, size_t at) -> uint32_t {
    return order_bytes == 2 ? (uint32_t)((const uint16_t*)a)[at] : ((const uint32_t*)a)[at];
  };
  auto put = [&](size_t at, uint32_t v) {
    if (order_bytes == 2) ((uint16_t*)order)[at] = (uint16_t)v;
    else ((uint32_t*)order)[at] = v;
  };
  std::vector<std::vector<int32_t>> succ(V);
  std::vector<int32_t> indeg(V, 0);
  for (int32_t b = 0; b < E; ++b) { succ[edge_src[b]].push_back(edge_dst[b]); indeg[edge_dst[b]]++; }
  std::vector<int64_t> rank(V);
  std::vector<int32_t> waiting(V);
  for (int64_t c = c_begin; c < c_end; ++c) {
    bool ok = true;
    for (int32_t i = 0; i < V; ++i) rank[i] = -1;
    for (int32_t r = 0; r < V; ++r) {
      const uint32_t i = get(list, (size_t)r * (size_t)K + (size_t)c);
      if (i >= (uint32_t)V || rank[i] >= 0) { ok = false; continue; }
      rank[i] = r;
    }
    if (status) status[c] = ok ? 0u : kStatusOrderInvalid;
    if (!ok) continue;
    // ranks of the operations that may come next; the smallest is on top
    std::priority_queue<int64_t, std::vector<int64_t>, std::greater<int64_t>> ready;
    for (int32_t i = 0; i < V; ++i) { waiting[i] = indeg[i]; if (indeg[i] == 0) ready.push(rank[i]); }
    int32_t k = 0;
    while (!ready.empty()) {
      const int64_t r = ready.top();
      ready.pop();
      const uint32_t i = get(list, (size_t)r * (size_t)K + (size_t)c);
      put((size_t)k * (size_t)K + (size_t)c, i);
      ++k;
      for (int32_t s : succ[i])
        if (--waiting[s] == 0) ready.push(rank[s]);
    }
    if (k != V) return -2;  // the edge list has a cycle
  }
  return 0;
}
