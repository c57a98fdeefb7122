// pe_coarsen: the operator-merging heuristic of Section IV (Algorithm 1), a host-side pre-processing step
// in front of candidate generation.  No GPU work: the graph is small by the time it matters and the
// procedure is a chain of dependent merges.
//
// Representation: node ids are the smallest original operator of each group; adjacency as bit rows
// (successors and predecessors of every live node), communication durations in a hash map keyed by the
// edge.  Two-hop redundancy of an edge (a, b) is one AND of succ[a] with pred[b]; reachability is built in
// reverse topological order by OR-ing successor rows.  The rules (which pair is a candidate, which comes
// first, how attributes combine) are documented with the declaration in pe.h.
#include <algorithm>
#include <cstdint>
#include <cstring>
#include <unordered_map>
#include <vector>

#include "pe.h"

namespace {

struct Coarsener {
  int V, L, words;
  std::vector<uint64_t> succ, pred;        // [V][words]
  std::vector<char> live;
  std::vector<int64_t> dur, A, W, req;
  std::vector<int32_t> rep;                 // original operator -> node id
  std::unordered_map<uint64_t, std::vector<int32_t>> comm;
  int nlive;

  static uint64_t key(int u, int v) { return ((uint64_t)(uint32_t)u << 32) | (uint32_t)v; }
  uint64_t* srow(int u) { return succ.data() + (size_t)u * words; }
  uint64_t* prow(int u) { return pred.data() + (size_t)u * words; }
  static bool test(const uint64_t* r, int v) { return (r[v >> 6] >> (v & 63)) & 1; }
  static void set(uint64_t* r, int v) { r[v >> 6] |= (uint64_t)1 << (v & 63); }
  static void clr(uint64_t* r, int v) { r[v >> 6] &= ~((uint64_t)1 << (v & 63)); }

  void add_edge(int u, int v, const int32_t* c) {
    auto it = comm.find(key(u, v));
    if (it == comm.end()) {
      comm.emplace(key(u, v), std::vector<int32_t>(c, c + L));
      set(srow(u), v);
      set(prow(v), u);
    } else {
      for (int l = 0; l < L; ++l) it->second[l] = std::max(it->second[l], c[l]);   // parallel edges: the later arrival
    }
  }
  void drop_edge(int u, int v) {
    comm.erase(key(u, v));
    clr(srow(u), v);
    clr(prow(v), u);
  }
  bool redundant(int a, int b) {   // some c with (a, c) and (c, b)
    const uint64_t *s = srow(a), *p = prow(b);
    for (int w = 0; w < words; ++w)
      if (s[w] & p[w]) return true;
    return false;
  }
  template <typename F>
  static void for_each(const uint64_t* r, int words, F f) {
    for (int w = 0; w < words; ++w) {
      uint64_t x = r[w];
      while (x) {
        const int b = __builtin_ctzll(x);
        x &= x - 1;
        f(w * 64 + b);
      }
    }
  }

  // the only non-redundant successor / predecessor of u, or -1 if there is none or more than one
  int single(int u, bool out) {
    int found = -1, count = 0;
    for_each(out ? srow(u) : prow(u), words, [&](int v) {
      if (out ? !redundant(u, v) : !redundant(v, u)) { found = v; ++count; }
    });
    return count == 1 ? found : -1;
  }

  bool candidate_edge(const pe_coarsen_params& prm, int* cu, int* cv) {
    int64_t best = -1;
    for (int u = 0; u < V; ++u) {
      if (!live[u]) continue;
      const int v = single(u, true);
      if (v < 0 || single(v, false) != u) continue;
      const int64_t d = dur[u] + dur[v];
      if (d > prm.max_dur_edge || req[u] + req[v] > prm.max_mem_edge) continue;
      if (best < 0 || d < best) { best = d; *cu = u; *cv = v; }   // u ascending: ties keep the smallest tail
    }
    return best >= 0;
  }

  bool candidate_nonedge(const pe_coarsen_params& prm, int* cu, int* cv) {
    // reach[u] = everything below u, built from the sinks upwards
    std::vector<uint64_t> reach((size_t)V * words, 0);
    std::vector<int> outdeg(V, 0), stack;
    for (int u = 0; u < V; ++u) {
      if (!live[u]) continue;
      for_each(srow(u), words, [&](int) { ++outdeg[u]; });
      if (outdeg[u] == 0) stack.push_back(u);
    }
    while (!stack.empty()) {
      const int v = stack.back();
      stack.pop_back();
      for_each(prow(v), words, [&](int p) {
        uint64_t* rp = reach.data() + (size_t)p * words;
        const uint64_t* rv = reach.data() + (size_t)v * words;
        for (int w = 0; w < words; ++w) rp[w] |= rv[w];
        set(rp, v);
        if (--outdeg[p] == 0) stack.push_back(p);
      });
    }
    int64_t best = -1;
    for (int u = 0; u < V; ++u) {
      if (!live[u]) continue;
      const uint64_t* ru = reach.data() + (size_t)u * words;
      for (int v = u + 1; v < V; ++v) {
        if (!live[v]) continue;
        const int64_t d = dur[u] + dur[v];
        if (best >= 0 && d >= best) continue;
        if (d > prm.max_dur_nonedge || req[u] + req[v] > prm.max_mem_nonedge) continue;
        if (test(ru, v) || test(reach.data() + (size_t)v * words, u)) continue;   // a path joins them
        best = d; *cu = u; *cv = v;
      }
    }
    return best >= 0;
  }

  void merge(int a, int b) {
    const int keep = std::min(a, b), gone = std::max(a, b);
    if (comm.count(key(a, b))) drop_edge(a, b);
    if (comm.count(key(b, a))) drop_edge(b, a);
    std::vector<int> outs, ins;
    for_each(srow(gone), words, [&](int x) { outs.push_back(x); });
    for_each(prow(gone), words, [&](int p) { ins.push_back(p); });
    for (int x : outs) {
      const std::vector<int32_t> c = comm[key(gone, x)];
      drop_edge(gone, x);
      add_edge(keep, x, c.data());
    }
    for (int p : ins) {
      const std::vector<int32_t> c = comm[key(p, gone)];
      drop_edge(p, gone);
      add_edge(p, keep, c.data());
    }
    live[gone] = 0;
    --nlive;
    dur[keep] += dur[gone]; A[keep] += A[gone]; W[keep] += W[gone]; req[keep] += req[gone];
    for (int i = 0; i < V; ++i)
      if (rep[i] == gone) rep[i] = keep;
  }
};

}  // namespace

extern "C" int pe_coarsen(const pe_graph_desc* desc, const pe_coarsen_params* prm, int32_t* op_map,
                          int32_t* num_ops_out, int32_t* num_edges_out, int32_t* edge_src, int32_t* edge_dst,
                          int32_t* comm, int32_t* dur, int32_t* mem_delta, int32_t* mem_weight) {
  if (!desc || !prm || !op_map || !num_ops_out || !num_edges_out || !dur) return PE_ERR_INVALID_ARG;
  const int rc = pe_graph_validate(desc);
  if (rc != PE_OK) return rc;
  const int V = desc->num_ops, E = desc->num_edges, L = desc->num_link_classes;
  if (E > 0 && (!edge_src || !edge_dst)) return PE_ERR_INVALID_ARG;
  if (V > 16384) return PE_ERR_UNSUPPORTED;   // bit-matrix adjacency: 2 x V^2 / 8 bytes
  if (desc->dur_by_machine) return PE_ERR_UNSUPPORTED;   // Section IV sums one duration per operator
  if (prm->target_ops < 1) return PE_ERR_INVALID_ARG;
  Coarsener g;
  g.V = V; g.L = L; g.words = (V + 63) / 64; g.nlive = V;
  g.succ.assign((size_t)V * g.words, 0);
  g.pred.assign((size_t)V * g.words, 0);
  g.live.assign(V, 1);
  g.dur.resize(V); g.A.resize(V); g.W.resize(V); g.req.resize(V); g.rep.resize(V);
  for (int i = 0; i < V; ++i) {
    g.dur[i] = desc->dur[i];
    g.A[i] = desc->mem_delta ? desc->mem_delta[i] : 0;
    g.W[i] = desc->mem_weight ? desc->mem_weight[i] : 0;
    g.req[i] = g.W[i] + std::max<int64_t>(g.A[i], 0);
    g.rep[i] = i;
  }
  std::vector<int32_t> zero(L, 0);
  for (int b = 0; b < E; ++b)
    g.add_edge(desc->edge_src[b], desc->edge_dst[b], desc->comm ? desc->comm + (size_t)b * L : zero.data());

  // Algorithm 1: edge merges while there are any, then merges of unrelated pairs, until |I| <= N or a
  // whole pass finds nothing to merge
  while (g.nlive > prm->target_ops) {
    int merged = 0, u = -1, v = -1;
    while (g.nlive > prm->target_ops && g.candidate_edge(*prm, &u, &v)) { g.merge(u, v); ++merged; }
    while (g.nlive > prm->target_ops && g.candidate_nonedge(*prm, &u, &v)) { g.merge(u, v); ++merged; }
    if (!merged) break;
  }

  // number the groups by their smallest operator, list the edges sorted by (source, destination)
  std::vector<int32_t> index(V, -1);
  int n = 0;
  for (int i = 0; i < V; ++i)
    if (g.live[i]) {
      index[i] = n;
      dur[n] = (int32_t)g.dur[i];
      if (mem_delta) mem_delta[n] = (int32_t)g.A[i];
      if (mem_weight) mem_weight[n] = (int32_t)g.W[i];
      ++n;
    }
  for (int i = 0; i < V; ++i) op_map[i] = index[g.rep[i]];
  int m = 0;
  for (int u = 0; u < V; ++u) {
    if (!g.live[u]) continue;
    Coarsener::for_each(g.srow(u), g.words, [&](int v) {
      edge_src[m] = index[u];
      edge_dst[m] = index[v];
      if (comm) std::memcpy(comm + (size_t)m * L, g.comm[Coarsener::key(u, v)].data(), sizeof(int32_t) * L);
      ++m;
    });
  }
  *num_ops_out = n;
  *num_edges_out = m;
  return PE_OK;
}
