// Seeded candidate generator: device assignments and random-key topological orders.
//
// A candidate c of a workload is (x_c, pi_c): x_c[i] is the device of operator i and
// pi_c a priority order that is a topological order of the operator DAG.  pi_c comes
// from a random-key Kahn sort: every operator draws a 32-bit key and, among the ready
// operators, the one with the smallest (key, id) is emitted next.  All draws come from
// the counter-based generator of rng.py (SplitMix64 finaliser keyed by seed, stream,
// candidate, index), so candidate c does not depend on which other candidates are made.
//
// Arrays are candidate-interleaved: element (row, c) of a [V][K] array sits at row*K + c.
// This file draws inputs only; it computes no schedule.
#include <algorithm>
#include <cstdint>
#include <cstring>
#include <queue>
#include <thread>
#include <vector>

namespace {

constexpr uint64_t kGolden = 0x9E3779B97F4A7C15ull;
constexpr uint64_t kStream = 0xD1B54A32D192ED03ull;

inline uint64_t mix64(uint64_t z) {
  z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
  z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
  return z ^ (z >> 31);
}
inline uint64_t rand64(uint64_t seed, uint64_t stream, uint64_t a, uint64_t b) {
  uint64_t h = mix64(seed ^ (stream * kStream));
  h = mix64(h + (a + 1) * kGolden);
  h = mix64(h + (b + 1) * kGolden);
  return h;
}
inline uint32_t below(uint64_t h, uint32_t n) { return (uint32_t)(((h >> 32) * (uint64_t)n) >> 32); }

constexpr uint64_t kStreamKey = 101, kStreamAssign = 102, kStreamPerm = 103;
constexpr int kBlock = 64;  // candidates generated together, so rows are written 64 at a time

struct Job {
  int32_t V, E, D;
  const int32_t *succ_ptr, *succ, *indeg;
  int mode;               // 0: x[i] uniform per op; 1: x[i] = sigma(group[i]), sigma a random permutation
  const int32_t* group;   // [V] for mode 1
  int32_t num_groups;
  uint64_t seed;
  int64_t K, c_first;     // columns 0..K-1 hold candidates c_first .. c_first+K-1
  uint8_t* assign;        // [V][K] by-op, may be null
  void* order;            // [V][K] by-pos, u16 or u32
  int order_bytes;
};

void run_block(const Job& j, int64_t col0, int ncol, std::vector<uint32_t>& ord_buf, std::vector<uint8_t>& asg_buf) {
  const int V = j.V;
  std::vector<int32_t> deg(V);
  std::vector<uint32_t> key(V);
  std::vector<int32_t> perm(std::max(j.num_groups, 1));
  using Item = uint64_t;  // key << 32 | id : the smallest pops first
  std::priority_queue<Item, std::vector<Item>, std::greater<Item>> ready;
  for (int t = 0; t < ncol; ++t) {
    const uint64_t c = (uint64_t)(j.c_first + col0 + t);
    for (int i = 0; i < V; ++i) {
      deg[i] = j.indeg[i];
      key[i] = (uint32_t)(rand64(j.seed, kStreamKey, c, (uint64_t)i) >> 32);
    }
    for (int i = 0; i < V; ++i)
      if (deg[i] == 0) ready.push(((uint64_t)key[i] << 32) | (uint32_t)i);
    int k = 0;
    while (!ready.empty()) {
      const int i = (int)(uint32_t)ready.top();
      ready.pop();
      ord_buf[(size_t)k * kBlock + t] = (uint32_t)i;
      ++k;
      for (int e = j.succ_ptr[i]; e < j.succ_ptr[i + 1]; ++e) {
        const int s = j.succ[e];
        if (--deg[s] == 0) ready.push(((uint64_t)key[s] << 32) | (uint32_t)s);
      }
    }
    if (j.assign) {
      if (j.mode == 1) {
        // Fisher-Yates over the devices; group g runs on perm[g] (num_groups <= D)
        std::vector<int32_t> dev(j.D);
        for (int d = 0; d < j.D; ++d) dev[d] = d;
        for (int d = j.D - 1; d > 0; --d) {
          const uint32_t r = below(rand64(j.seed, kStreamPerm, c, (uint64_t)d), (uint32_t)(d + 1));
          std::swap(dev[d], dev[r]);
        }
        for (int g = 0; g < j.num_groups; ++g) perm[g] = dev[g % j.D];
        for (int i = 0; i < V; ++i) asg_buf[(size_t)i * kBlock + t] = (uint8_t)perm[j.group[i]];
      } else {
        for (int i = 0; i < V; ++i)
          asg_buf[(size_t)i * kBlock + t] = (uint8_t)below(rand64(j.seed, kStreamAssign, c, (uint64_t)i), (uint32_t)j.D);
      }
    }
  }
  // write the block's columns row by row
  for (int r = 0; r < V; ++r) {
    const size_t off = (size_t)r * (size_t)j.K + (size_t)col0;
    if (j.order_bytes == 2) {
      uint16_t* o = (uint16_t*)j.order + off;
      for (int t = 0; t < ncol; ++t) o[t] = (uint16_t)ord_buf[(size_t)r * kBlock + t];
    } else {
      uint32_t* o = (uint32_t*)j.order + off;
      for (int t = 0; t < ncol; ++t) o[t] = ord_buf[(size_t)r * kBlock + t];
    }
    if (j.assign) std::memcpy(j.assign + off, &asg_buf[(size_t)r * kBlock], (size_t)ncol);
  }
}

}  // namespace

extern "C" {

// Returns 0 on success, -1 on bad arguments, -2 if the edge list has a cycle.
int pegen_candidates(int32_t V, int32_t E, const int32_t* edge_src, const int32_t* edge_dst, int32_t D, int mode,
                     const int32_t* group, int32_t num_groups, uint64_t seed, int64_t K, int64_t c_first,
                     uint8_t* assign, void* order, int order_bytes, int num_threads) {
  if (V <= 0 || E < 0 || D <= 0 || D > 255 || K < 0 || !order) return -1;
  if (order_bytes != 2 && order_bytes != 4) return -1;
  if (order_bytes == 2 && V > 65536) return -1;
  if (mode == 1 && (!group || num_groups <= 0)) return -1;
  std::vector<int32_t> succ_ptr(V + 1, 0), succ(E), indeg(V, 0);
  for (int e = 0; e < E; ++e) {
    if (edge_src[e] < 0 || edge_src[e] >= V || edge_dst[e] < 0 || edge_dst[e] >= V) return -1;
    succ_ptr[edge_src[e] + 1]++;
    indeg[edge_dst[e]]++;
  }
  for (int i = 0; i < V; ++i) succ_ptr[i + 1] += succ_ptr[i];
  {
    std::vector<int32_t> fill(succ_ptr.begin(), succ_ptr.end() - 1);
    for (int e = 0; e < E; ++e) succ[fill[edge_src[e]]++] = edge_dst[e];
  }
  {  // acyclicity: a plain Kahn pass must emit every operator
    std::vector<int32_t> deg(indeg), stack;
    for (int i = 0; i < V; ++i) if (deg[i] == 0) stack.push_back(i);
    int seen = 0;
    while (!stack.empty()) {
      int i = stack.back(); stack.pop_back(); ++seen;
      for (int e = succ_ptr[i]; e < succ_ptr[i + 1]; ++e) if (--deg[succ[e]] == 0) stack.push_back(succ[e]);
    }
    if (seen != V) return -2;
  }
  if (mode == 1) for (int i = 0; i < V; ++i) if (group[i] < 0 || group[i] >= num_groups) return -1;
  Job job{V, E, D, succ_ptr.data(), succ.data(), indeg.data(), mode, group, num_groups, seed, K, c_first, assign, order, order_bytes};
  const int64_t nblocks = (K + kBlock - 1) / kBlock;
  int T = num_threads > 0 ? num_threads : (int)std::thread::hardware_concurrency();
  if (T < 1) T = 1;
  if ((int64_t)T > nblocks) T = (int)std::max<int64_t>(nblocks, 1);
  auto worker = [&](int tid) {
    std::vector<uint32_t> ord_buf((size_t)V * kBlock);
    std::vector<uint8_t> asg_buf((size_t)V * kBlock);
    for (int64_t b = tid; b < nblocks; b += T) {
      const int64_t col0 = b * kBlock;
      const int ncol = (int)std::min<int64_t>(kBlock, K - col0);
      run_block(job, col0, ncol, ord_buf, asg_buf);
    }
  };
  std::vector<std::thread> pool;
  for (int t = 1; t < T; ++t) pool.emplace_back(worker, t);
  worker(0);
  for (auto& th : pool) th.join();
  return 0;
}

// dev_seq[k][c] = assign[order[k][c]][c]: the by-position view of an assignment (pure re-indexing).
int pegen_assign_by_pos(int32_t V, int64_t K, const uint8_t* assign, const void* order, int order_bytes,
                        uint8_t* dev_seq, int num_threads) {
  if (V <= 0 || K < 0 || !assign || !order || !dev_seq) return -1;
  int T = num_threads > 0 ? num_threads : (int)std::thread::hardware_concurrency();
  if (T < 1) T = 1;
  auto worker = [&](int tid) {
    for (int64_t k = tid; k < V; k += T) {
      const size_t off = (size_t)k * (size_t)K;
      for (int64_t c = 0; c < K; ++c) {
        const uint32_t i = order_bytes == 2 ? ((const uint16_t*)order)[off + c] : ((const uint32_t*)order)[off + c];
        dev_seq[off + c] = i < (uint32_t)V ? assign[(size_t)i * (size_t)K + c] : (uint8_t)0;
      }
    }
  };
  std::vector<std::thread> pool;
  for (int t = 1; t < T; ++t) pool.emplace_back(worker, t);
  worker(0);
  for (auto& th : pool) th.join();
  return 0;
}

}  // extern "C"
