// pe_decode_priority: priority-list decoding, the step in front of pe_eval_batch.
//
// The paper prints no decoder (Section IV mentions dispatch rules only as the inspiration of its
// coarsening heuristic); the rule implemented here is this library's choice: a candidate ranks the operators through a list (list[r] =
// the operator of rank r; any permutation of I), and the priority order pi is built position by
// position: among the operators not yet placed whose predecessors in B have all been placed, the
// one of smallest rank comes next (Kahn's algorithm with the ranks as priorities).  The result is
// a topological order of G_m, i.e. a valid `order` argument of pe_eval_batch.
//
// One thread per candidate.  Because the priorities are the ranks 0..V-1, the set of available
// operators is a bitmap over ranks with two summary levels above it (one bit per 32-bit word of
// the level below; the top level is a 64-bit register, which is why V <= 65536): "take the
// smallest" is three find-first-set steps, "add" is three bit sets - no heap, no comparisons of
// keys.  Per candidate:
//   word[i]   rank of operator i (bits 0..15) | predecessors still missing (bits 16..23) |
//             seen in the list (bit 31)
//   L0, L1    the bitmap over ranks and its first summary level
//   list      (shared-state variant only) the list itself, two 16-bit entries per word; the
//             global-state variant reads list[r] back from the input when rank r is taken
// The shared-state variant keeps these as [row][thread] in shared memory (a lane's accesses stay in
// its own bank) next to the graph's successor lists, staged by bulk copy; the global-state
// variant keeps them in the caller's workspace in tiles of 32 candidates, [tile][row][32], and
// reads the successor lists through the cache.
#include <atomic>
#include <climits>

#include "pe_device.cuh"
#include "pe_graph.h"
#include "pe_launch.h"

namespace pe {

extern std::atomic<int64_t> g_decode_launches;
std::atomic<int64_t> g_decode_launches{0};

struct FwdPtrs {
  const uint32_t* ptr;
  const uint16_t* succ;
  const uint8_t* indeg;
};

__device__ __forceinline__ FwdPtrs fwd_ptrs(const uint8_t* base, const PeFwdView& f) {
  FwdPtrs p;
  p.ptr = reinterpret_cast<const uint32_t*>(base + f.ptr);
  p.succ = reinterpret_cast<const uint16_t*>(base + f.succ);
  p.indeg = base + f.indeg;
  return p;
}

constexpr uint32_t kSeen = 0x80000000u;
constexpr int kListAhead = 8;  // rows of the list requested ahead of the one being placed

template <bool STATE_SMEM>
__global__ void __launch_bounds__(256) pe_decode_kernel(PeFwdView f, const uint8_t* __restrict__ fblob, int64_t K,
                                                        const uint16_t* __restrict__ list, uint16_t* __restrict__ order,
                                                        uint32_t* __restrict__ status, uint32_t* __restrict__ gstate,
                                                        int* err) {
  extern __shared__ __align__(16) uint8_t smem_raw[];
  const int T = blockDim.x;
  const int t = threadIdx.x;
  const int V = f.V;
  const uint8_t* fbase = fblob;
  uint8_t* sm = smem_raw;
  if (STATE_SMEM) {
    uint64_t* bar = reinterpret_cast<uint64_t*>(sm + f.bytes);
    if (!stage_blob(sm, fblob, f.bytes, bar, err)) return;
    fbase = sm;
    sm += f.bytes + 16;
  }
  const FwdPtrs fp = fwd_ptrs(fbase, f);
  const int64_t c = (int64_t)blockIdx.x * T + t;
  if (c >= K) return;
  const size_t Ks = (size_t)K;
  const int n0 = (V + 31) >> 5, n1 = (n0 + 31) >> 5;
  // row r of this candidate's state is st[r * pitch]
  uint32_t* st = STATE_SMEM ? reinterpret_cast<uint32_t*>(sm) + t
                            : gstate + (size_t)(c >> 5) * (size_t)(V + n0 + n1) * 32 + (c & 31);
  const uint32_t pitch = STATE_SMEM ? (uint32_t)T : 32u;
  uint32_t* word = st;
  uint32_t* L0 = st + (size_t)V * pitch;
  uint32_t* L1 = L0 + (size_t)n0 * pitch;
  uint32_t* lst = L1 + (size_t)n1 * pitch;   // shared-state variant only: [ceil(V / 2)] pairs of entries
  uint64_t L2 = 0;

  auto add = [&](uint32_t r) {   // rank r becomes available
    uint32_t* p0 = L0 + (r >> 5) * pitch;
    const uint32_t w0 = *p0;
    *p0 = w0 | (1u << (r & 31u));
    if (w0 == 0u) {              // the word was empty: the levels above learn of it
      L1[(r >> 10) * pitch] |= 1u << ((r >> 5) & 31u);
      L2 |= 1ull << (r >> 10);
    }
  };

  for (int i = 0; i < V; ++i) word[(uint32_t)i * pitch] = (uint32_t)fp.indeg[i] << 16;
  for (int q = 0; q < n0 + n1; ++q) L0[(uint32_t)q * pitch] = 0u;

  // the list: rank and "seen" into the operators' words, operators without predecessors become available
  const uint16_t* list_col = list + c;
  bool bad = false;
  {
    uint32_t ring[kListAhead];
#pragma unroll
    for (int u = 0; u < kListAhead; ++u) ring[u] = (uint32_t)list_col[(size_t)min(u, V - 1) * Ks];
    for (int r0 = 0; r0 < V; r0 += kListAhead) {
      uint32_t cur[kListAhead];
#pragma unroll
      for (int u = 0; u < kListAhead; ++u) {
        cur[u] = ring[u];
        ring[u] = (uint32_t)list_col[(size_t)min(r0 + kListAhead + u, V - 1) * Ks];
      }
#pragma unroll
      for (int u = 0; u < kListAhead; ++u) {
        const int r = r0 + u;
        if (r < V) {
          const uint32_t i = cur[u];
          if (STATE_SMEM) reinterpret_cast<uint16_t*>(lst + (uint32_t)(r >> 1) * pitch)[r & 1] = (uint16_t)i;
          if (i >= (uint32_t)V) {
            bad = true;
          } else {
            const uint32_t w = word[i * pitch];
            if (w & kSeen) {
              bad = true;            // the operator is in the list twice
            } else {
              word[i * pitch] = w | kSeen | (uint32_t)r;
              if ((w >> 16) == 0u) add((uint32_t)r);
            }
          }
        }
      }
    }
  }
  if (status) status[c] = bad ? (uint32_t)PE_STATUS_ORDER_INVALID : 0u;
  if (bad) return;   // not a permutation: the order of this candidate stays unwritten

  // Main loop.  Every iteration hands one successor of the operator placed last its "one predecessor fewer"
  // and, once that operator's successor list is used up, places the next operator.  All candidates share the
  // graph, so every lane needs the same number of successor steps and placements in total; spreading them
  // over uniform iterations keeps the lanes of a warp busy where a loop over each operator's successors
  // would make the whole warp wait for the lane that drew the operator with the most successors.
  uint16_t* order_col = order + c;
  uint32_t e = 0, e_end = 0;
  int k = 0;
  for (int it = 0; it < 2 * V + f.E + 2; ++it) {   // (bound: at most V placements and E successor steps)
    if (e < e_end) {
      const uint32_t s = fp.succ[e++];
      const uint32_t w = word[s * pitch] - (1u << 16);
      word[s * pitch] = w;
      if (((w >> 16) & 0xFFu) == 0u) add(w & 0xFFFFu);
    }
    if (e == e_end) {
      if (k == V || L2 == 0) break;   // all placed (L2 == 0 earlier cannot happen for a permutation over a DAG)
      // the smallest available rank: first set bit of each level, top down
      const uint32_t b2 = (uint32_t)__ffsll((long long)L2) - 1u;
      uint32_t w1 = L1[b2 * pitch];
      if (w1 == 0u) break;   // (a summary bit without anything below it: cannot happen either)
      const uint32_t b1 = (uint32_t)__ffs((int)w1) - 1u;
      const uint32_t i0 = b2 * 32u + b1;
      uint32_t w0 = L0[i0 * pitch];
      if (w0 == 0u) break;
      const uint32_t b0 = (uint32_t)__ffs((int)w0) - 1u;
      const uint32_t r = i0 * 32u + b0;
      w0 &= ~(1u << b0);
      L0[i0 * pitch] = w0;
      if (w0 == 0u) {
        w1 &= ~(1u << b1);
        L1[b2 * pitch] = w1;
        if (w1 == 0u) L2 &= ~(1ull << b2);
      }
      const uint32_t i = STATE_SMEM ? (uint32_t) reinterpret_cast<const uint16_t*>(lst + (r >> 1) * pitch)[r & 1u]
                                    : (uint32_t)list_col[(size_t)r * Ks];
      order_col[(size_t)k * Ks] = (uint16_t)i;
      ++k;
      e = fp.ptr[i];
      e_end = fp.ptr[i + 1];
    }
  }
}

struct DecodePlan {
  bool shared = false;
  int threads = 0;
  size_t smem = 0;
  size_t workspace = 0;
};

static bool decode_plan(const pe_graph* g, int64_t K, uint32_t flags, DecodePlan* p) {
  if (!g->fwd_ok) return false;
  const uint32_t want = flags & PE_VARIANT_MASK;
  const size_t V = (size_t)g->V, n0 = (V + 31) / 32, n1 = (n0 + 31) / 32;
  if (want == PE_VARIANT_AUTO || want == PE_VARIANT_SHARED) {
    const size_t per = 4 * (V + n0 + n1 + (V + 1) / 2);
    const size_t fixed = (size_t)g->fview.bytes + 16;
    // with a single warp per SM the shared-state variant loses to the global-state one (measured at
    // V = 1024: 3.2e9 against ~7e9 operators/s), so it needs room for two warps unless it was asked for
    if (fixed + (want == PE_VARIANT_SHARED ? 32 : 64) * per <= g->smem_optin) {
      size_t T = (g->smem_optin - fixed) / per;
      if (T > 256) T = 256;
      T = T / 32 * 32;
      p->shared = true;
      p->threads = (int)T;
      p->smem = fixed + T * per;
      p->workspace = 0;
      return true;
    }
    if (want == PE_VARIANT_SHARED) return false;
  }
  if (want != PE_VARIANT_AUTO && want != PE_VARIANT_GLOBAL) return false;
  p->shared = false;
  p->threads = 128;
  p->smem = 0;
  p->workspace = (size_t)((K + 31) / 32) * (V + n0 + n1) * 32 * 4;
  p->workspace = (p->workspace + 255) / 256 * 256;
  return true;
}

}  // namespace pe

extern "C" size_t pe_decode_workspace_bytes(const pe_graph* g, int64_t K, uint32_t flags) {
  pe::DecodePlan p;
  if (!g || K < 0 || !pe::decode_plan(g, K, flags, &p)) return 0;
  return p.workspace;
}

extern "C" int pe_decode_variant(const pe_graph* g, int64_t K, uint32_t flags) {
  pe::DecodePlan p;
  if (!g || K < 0) return PE_ERR_INVALID_ARG;
  if (flags & ~(uint32_t)PE_VARIANT_MASK) return PE_ERR_INVALID_ARG;
  if (!pe::decode_plan(g, K, flags, &p)) return PE_ERR_UNSUPPORTED;
  return p.shared ? PE_VARIANT_SHARED : PE_VARIANT_GLOBAL;
}

extern "C" int pe_decode_priority(pe_graph* g, int64_t K, const void* list, int order_bytes, uint32_t flags, void* order,
                                  uint32_t* status, void* workspace, size_t workspace_bytes, void* cuda_stream) {
  if (!g || K < 0) return PE_ERR_INVALID_ARG;
  if (flags & ~(uint32_t)PE_VARIANT_MASK) return PE_ERR_INVALID_ARG;
  if (order_bytes != 2 && order_bytes != 4) return PE_ERR_INVALID_ARG;
  if (order_bytes != 2) return PE_ERR_UNSUPPORTED;
  pe::DecodePlan p;
  if (!pe::decode_plan(g, K, flags, &p)) return PE_ERR_UNSUPPORTED;
  if (K == 0) return PE_OK;
  if (!list || !order) return PE_ERR_INVALID_ARG;
  if ((K + p.threads - 1) / p.threads > (int64_t)INT_MAX) return PE_ERR_INVALID_ARG;
  if (p.workspace > 0 && (!workspace || workspace_bytes < p.workspace)) return PE_ERR_WORKSPACE;
  int prev = -1;
  if (cudaGetDevice(&prev) != cudaSuccess) return PE_ERR_CUDA;
  if (prev != g->device && cudaSetDevice(g->device) != cudaSuccess) return PE_ERR_CUDA;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  const unsigned grid = (unsigned)((K + p.threads - 1) / p.threads);
  int ret = PE_OK;
  if (p.shared) {
    auto kern = pe::pe_decode_kernel<true>;
    if (!pe::set_smem(kern, p.smem)) ret = PE_ERR_CUDA;
    else kern<<<grid, p.threads, p.smem, stream>>>(g->fview, g->d_fwd, K, static_cast<const uint16_t*>(list),
                                                    static_cast<uint16_t*>(order), status, nullptr, g->d_error);
  } else {
    pe::pe_decode_kernel<false><<<grid, p.threads, 0, stream>>>(g->fview, g->d_fwd, K, static_cast<const uint16_t*>(list),
                                                                static_cast<uint16_t*>(order), status,
                                                                static_cast<uint32_t*>(workspace), g->d_error);
  }
  if (ret == PE_OK) {
    pe::g_decode_launches.fetch_add(1, std::memory_order_relaxed);
    if (cudaGetLastError() != cudaSuccess) ret = PE_ERR_CUDA;
  }
  if (prev != g->device) cudaSetDevice(prev);
  return ret;
}
