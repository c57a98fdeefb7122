// Variant WARP: one warp per candidate, 32 positions of the priority order at a time.
//
// The per-operator state (end time and machine packed in one word, kNotDoneTime until the
// operator is scheduled) of a candidate lives in shared memory, so a block holds as many
// candidates as fit and a candidate with thousands of operators still runs on chip.  A warp
// takes a window of 32 consecutive positions, one per lane.  Operators in a window depend on
// each other only through (a) a predecessor edge inside the window, (b) the previous operator
// of the same machine inside the window (Eqs. 7-8).  Both kinds of producer sit at a lower
// lane, because the order is topological, so the window is resolved in rounds: in each round
// every lane whose producers are all finished computes its start and end time and publishes
// them; the number of rounds is the longest dependency chain inside the window.  A round in
// which nothing finishes means the order was not topological: the candidate is flagged and
// the window is closed without waiting.
#pragma once
#include "pe_device.cuh"

namespace pe {

template <typename OrderT, bool BY_POS, bool GRAPH_SMEM>
__global__ void __launch_bounds__(1024) pe_eval_warp_kernel(PeGraphView g, const uint8_t* __restrict__ blob, int64_t K,
                                    const uint8_t* __restrict__ assign, const OrderT* __restrict__ order,
                                    pe_outputs out, uint32_t flags, int* err, int warp_words) {
  extern __shared__ __align__(16) uint8_t smem_raw[];
  constexpr uint32_t FULL = 0xFFFFFFFFu;
  const int lane = threadIdx.x & 31;
  const int warp = threadIdx.x >> 5;
  const int nwarps = blockDim.x >> 5;
  const int D = g.D, V = g.V, L = g.L;
  uint8_t* sm = smem_raw;
  const uint8_t* gbase = blob;
  if (GRAPH_SMEM) {
    uint64_t* bar = reinterpret_cast<uint64_t*>(sm + g.lay.bytes);
    if (!stage_blob(sm, blob, g.lay.bytes, bar, err)) return;
    gbase = sm;
    sm += g.lay.bytes + 16;
  }
  const GraphPtrs gp = graph_ptrs(gbase, g);
  const size_t Ks = (size_t)K;
  const int64_t c0 = (int64_t)blockIdx.x * nwarps;

  // ---- initial state of every candidate of the block ----
  uint32_t* all_words = reinterpret_cast<uint32_t*>(sm);
  if (BY_POS) {
    for (int idx = threadIdx.x; idx < nwarps * warp_words; idx += blockDim.x) all_words[idx] = 0xFFFFFFFFu;
  } else {
    // machine of every operator from the by-op assignment: row i holds nwarps adjacent bytes
    for (int idx = threadIdx.x; idx < V * nwarps; idx += blockDim.x) {
      const int i = idx / nwarps, w = idx - i * nwarps;
      const int64_t cc = c0 + w;
      all_words[(size_t)w * warp_words + i] = 0xFFFFFF00u | (cc < K ? (uint32_t)assign[(size_t)i * Ks + cc] : 0u);
    }
  }
  __syncthreads();
  uint32_t* state = all_words + (size_t)warp * warp_words;
  int32_t* free_at = reinterpret_cast<int32_t*>(state + (V | 1));
  int32_t* lvl = free_at + D;
  int32_t* peak = lvl + D;
  int32_t* busy = peak + D;
  int32_t* wsum = busy + D;
  for (int j = lane; j < 5 * D; j += 32) free_at[j] = 0;
  __syncwarp();

  const int64_t c = c0 + warp;
  if (c >= K) return;
  const bool by_op_times = (flags & PE_TIMES_BY_OP) != 0;
  const uint32_t lt_mask = (1u << lane) - 1u;
  uint32_t st = 0;
  int32_t z = 0;

  uint32_t o_cur = lane < V ? (uint32_t)order[(size_t)lane * Ks + c] : 0xFFFFFFFFu;
  uint32_t a_cur = (BY_POS && lane < V) ? (uint32_t)assign[(size_t)lane * Ks + c] : 0u;
  for (int base = 0; base < V; base += 32) {
    const int k = base + lane;
    const bool valid = k < V;
    const uint32_t iu = o_cur;
    const uint32_t a_here = a_cur;
    {  // prefetch the next window
      const int kn = k + 32;
      o_cur = kn < V ? (uint32_t)order[(size_t)kn * Ks + c] : 0xFFFFFFFFu;
      if (BY_POS) a_cur = kn < V ? (uint32_t)assign[(size_t)kn * Ks + c] : 0u;
    }
    const bool act = valid && iu < (uint32_t)V;
    if (valid && !act) st |= PE_STATUS_ORDER_INVALID;
    const int i = act ? (int)iu : 0;
    const uint32_t wi = act ? state[i] : 0u;
    uint32_t jr = BY_POS ? a_here : state_dev(wi);
    if (act && jr >= (uint32_t)D) { st |= PE_STATUS_ASSIGN_RANGE; jr = D - 1; }
    const int j = act ? (int)jr : 0;
    if (act && state_time(wi) != kNotDoneTime) st |= PE_STATUS_ORDER_INVALID;  // scheduled in an earlier window
    const uint32_t same_op = __match_any_sync(FULL, act ? (uint32_t)i : (0x80000000u | lane));
    if (same_op & lt_mask) st |= PE_STATUS_ORDER_INVALID;                       // repeated inside this window
    const uint32_t same_dev = __match_any_sync(FULL, act ? (uint32_t)j : (0x100u | lane));
    const int prev = (same_dev & lt_mask) ? 31 - __clz(same_dev & lt_mask) : -1;
    const bool last_on_dev = (same_dev >> lane) == 1u;
    PeOpRec op;
    op.edge_begin = 0; op.indeg = 0; op.dur = 0; op.mem_delta = 0;
    if (act) op = load_op(gp.ops, i);

    bool pend = act;
    int32_t s = 0, e = 0, lv = 0;
    uint32_t pendmask = __ballot_sync(FULL, pend);
    while (pendmask) {
      const int src = prev < 0 ? lane : prev;
      const int32_t e_prev = __shfl_sync(FULL, e, src);
      const int32_t lv_prev = __shfl_sync(FULL, lv, src);
      if (pend) {
        bool ready = prev < 0 || !((pendmask >> prev) & 1u);
        int32_t r = 0;
        if (ready) {
          for (int q = op.edge_begin; q < op.edge_begin + op.indeg; ++q) {
            const uint32_t w = state[gp.pred[q]];
            if (state_time(w) == kNotDoneTime) { ready = false; break; }
            int32_t ep = (int32_t)state_time(w);
            const int xp = (int)state_dev(w);
            if (xp != j) {
              const uint32_t cl = gp.cls[xp * D + j];
              if (cl == 0xFFu) st |= PE_STATUS_NO_CHANNEL;
              else ep += gp.comm[(size_t)q * L + cl];
            }
            r = max(r, ep);
          }
        }
        if (ready) {
          s = max(r, prev < 0 ? free_at[j] : e_prev);
          e = s + op.dur;
          lv = (prev < 0 ? lvl[j] : lv_prev) + op.mem_delta;
          state[i] = pack_state((uint32_t)e, (uint32_t)j);
          pend = false;
        }
      }
      __syncwarp();
      const uint32_t now = __ballot_sync(FULL, pend);
      if (now == pendmask) {  // nothing finished: some operator waits for one that is not before it
        if (pend) {
          st |= PE_STATUS_ORDER_INVALID;
          e = op.dur;
          state[i] = pack_state((uint32_t)e, (uint32_t)j);
          pend = false;
        }
        __syncwarp();
        break;
      }
      pendmask = now;
    }

    if (act) {
      atomicAdd(&busy[j], op.dur);
      atomicMax(&peak[j], lv);
      if (gp.weight) atomicAdd(&wsum[j], gp.weight[i]);
      if (last_on_dev) { free_at[j] = e; lvl[j] = lv; }
      z = max(z, e);
      const size_t at = (size_t)(by_op_times ? i : k) * Ks + c;
      if (out.start) out.start[at] = s;
      if (out.finish) out.finish[at] = e;
    }
    __syncwarp();
  }

  for (int off = 16; off > 0; off >>= 1) {
    z = max(z, __shfl_xor_sync(FULL, z, off));
    st |= __shfl_xor_sync(FULL, st, off);
  }
  uint32_t over = 0;
  for (int j = lane; j < D; j += 32) {
    const int32_t pk = peak[j] + (gp.weight ? wsum[j] : 0);
    if (pk > gp.cap[j]) over = PE_STATUS_MEM_EXCEEDED;
    if (out.busy) out.busy[(size_t)j * Ks + c] = busy[j];
    if (out.peak_mem) out.peak_mem[(size_t)j * Ks + c] = pk;
  }
  if (__any_sync(FULL, over != 0)) st |= PE_STATUS_MEM_EXCEEDED;
  if (lane == 0) {
    if (out.makespan) out.makespan[c] = z;
    if (out.status) out.status[c] = st;
  }
}

}  // namespace pe
