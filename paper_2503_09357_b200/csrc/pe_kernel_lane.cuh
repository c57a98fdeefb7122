// One thread per candidate over the compact graph encoding: the kernel behind the SHARED
// variant (STATE_SMEM = true) and the GLOBAL variant of graphs that have a compact encoding
// (STATE_SMEM = false).
//
//  * per-operator state word: end time << 8 | machine; 0xFFFFFFxx until the operator is
//    scheduled.  With by-operator assignments the machine byte is filled in by the initial
//    pass (a coalesced read of `assign`), so the main loop never gathers from `assign`.
//      STATE_SMEM:  shared memory, [operator][thread] - a lane's gathers stay in its own bank;
//      otherwise:   the caller's workspace, in tiles of 32 candidates: [tile][operator][32].
//                   A warp then works inside its own contiguous (V+1)*128-byte region, which
//                   keeps its random accesses within one or two pages of address translation.
//    Row V is a sentinel ("ended at time 0 on machine 0"): the compact encoding points the
//    inline edge slots of operators with fewer incoming edges at it, so those slots are
//    evaluated without a branch and change nothing.
//  * per-machine state: one 16-byte record {free time, busy, level, peak} per (machine,
//    thread) in shared memory: one 128-bit load and one 128-bit store per step.
//  * graph: compact encoding (16-byte operator record with the first incoming edges inline),
//    staged into shared memory by bulk copy (STATE_SMEM) or read through the read-only cache.
//  * order entries (and by-position machine ids) are fetched kUnroll positions ahead into
//    register rings, the operator record one position ahead.
//  * validity (order entry range, repeated operator, predecessor not scheduled, machine range)
//    is accumulated with min/max and tested once at the end; an out-of-range entry is clamped
//    so that indexing stays in bounds.
// The recurrence itself (Eqs. 3, 7-8, 11-13, 16-19) is the one stated at the top of pe_eval.cu.
#pragma once
#include "pe_device.cuh"

namespace pe {

constexpr int kUnroll = 8;
constexpr uint32_t kUnscheduled = 0xFFFFFF00u;  // state words at or above this: not scheduled yet

// CLS: 0 = one link class, every pair connected (no table lookup); 1 = one class, some pair
// without a channel; 2 = two classes.  IdxT: uint32_t when (V+1)*K fits in 32 bits.
// TIMES: start and finish are both written (true) or both absent (false).
// DEPTH (one link class only): 3 = no operator has more than three incoming edges, so the three inline
// slots are all there is and the step is straight-line code; 0 = general (inline slots, then the list).
// EXCL: channels carry one transfer at a time (PE_COMM_EXCLUSIVE; Eqs. 14-15): the end of the last transfer per
// channel sits in shared memory as [machine pair][thread] behind the operator state (shared-state kernel) or in the
// workspace as tiles [tile of 32][machine pair][32] behind everything else (global-state kernel).
// StateT: uint32_t = end << 8 | machine; uint16_t (shared-state only) = end << jbits | machine when the graph's
// time bound and machine count fit 16 bits together: half the shared memory per candidate, twice the
// candidates per SM.  Two warps then share the 32-bit words of a row (one the low, one the high halves), so
// that the 32 lanes of a warp still fall into 32 different banks.
template <typename IdxT, bool BY_POS, int CLS, bool STATE_SMEM, bool TIMES, int DEPTH, bool EXCL = false,
          typename StateT = uint32_t>
__global__ void __launch_bounds__(256) pe_eval_lane_kernel(PeNarrowView g, const uint8_t* __restrict__ nblob, int64_t K,
                                                           const uint8_t* __restrict__ assign,
                                                           const uint16_t* __restrict__ order, pe_outputs out,
                                                           uint32_t flags, int* err, uint32_t* __restrict__ gstate,
                                                           int4* __restrict__ gdev, int jbits,
                                                           int32_t* __restrict__ gchan) {
  extern __shared__ __align__(16) uint8_t smem_raw[];
  constexpr bool TWO_CLASS = CLS == 2;
  constexpr bool NEED_CLS = CLS != 0;
  constexpr bool S16 = sizeof(StateT) == 2;
  static_assert(!S16 || (STATE_SMEM && !EXCL), "16-bit state words: shared-state kernel without exclusive channels");
  const uint32_t jb = S16 ? (uint32_t)jbits : 8u;                     // bits of the machine field
  const uint32_t jmask = (1u << jb) - 1u;
  const uint32_t unsched = S16 ? ((0xFFFFu >> jb) << jb) : kUnscheduled;   // time field all ones: not scheduled yet
  const int T = blockDim.x;
  const int t = threadIdx.x;
  const int D = g.D, V = g.V;
  uint8_t* sm = smem_raw;
  const uint8_t* gbase = nblob;
  if (STATE_SMEM) {
    uint64_t* bar = reinterpret_cast<uint64_t*>(smem_raw + g.bytes);
    if (!stage_blob(smem_raw, nblob, g.bytes, bar, err)) return;
    gbase = smem_raw;
    sm = smem_raw + g.bytes + 16;
  }
  const NarrowPtrs gp = narrow_ptrs(gbase, g);
  const int64_t c = (int64_t)blockIdx.x * T + t;
  // per-machine records {free, busy, level, peak}: shared memory [D][T], or (global-state kernel
  // with many machines, where shared memory would cap the number of resident candidates) the
  // workspace in tiles [tile of 32][D][32], which stays in L2.  Weight sums follow the same way.
  const bool dev_global = !STATE_SMEM && gdev != nullptr;
  const uint32_t dpitch = dev_global ? 32u : (uint32_t)T;
  int4* dev = dev_global ? gdev + (size_t)(c >> 5) * (size_t)D * 32 + (c & 31) : reinterpret_cast<int4*>(sm) + t;
  int32_t* wsum = dev_global
                      ? reinterpret_cast<int32_t*>(gdev + (size_t)((K + 31) >> 5) * (size_t)D * 32) +
                            (size_t)(c >> 5) * (size_t)D * 32 + (c & 31)
                      : reinterpret_cast<int32_t*>(sm + (size_t)D * T * 16) + t;
  const size_t wsum_bytes = g.has_weight ? (size_t)D * T * 4 : 0;
  if (c >= K) return;
  const IdxT Ki = (IdxT)K;
  // state word of operator p is state[p * pitch]
  // (16-bit words: thread t of the block sits at halfword 2 * (32 * (t / 64) + t % 32) + (t / 32) % 2 of a row)
  const uint32_t t_off = S16 ? 2u * (32u * ((uint32_t)t >> 6) + ((uint32_t)t & 31u)) + (((uint32_t)t >> 5) & 1u) : (uint32_t)t;
  StateT* state = STATE_SMEM ? reinterpret_cast<StateT*>(sm + (size_t)D * T * 16 + wsum_bytes) + t_off
                             : reinterpret_cast<StateT*>(gstate + (size_t)(c >> 5) * (size_t)(V + 1) * 32 + (c & 31));
  const uint32_t pitch = STATE_SMEM ? (uint32_t)T : 32u;
  // EXCL: end of the last transfer on channel (j1 -> j2) at chan[(j1 * D + j2) * cpitch]
  const uint32_t cpitch = STATE_SMEM ? (uint32_t)T : 32u;
  int32_t* chan = STATE_SMEM
                      ? reinterpret_cast<int32_t*>(sm + (size_t)D * T * 16 + wsum_bytes + (size_t)(V + 1) * T * 4) + t
                      : gchan + (size_t)(c >> 5) * (size_t)D * (size_t)D * 32 + (c & 31);

  const uint16_t* order_col = order + c;
  const uint8_t* assign_col = assign + c;
  uint32_t raw_max = 0;   // 16-bit words, by-operator assignments: largest machine id seen before clamping
  {  // initial state: unscheduled; by-operator assignments also deposit the machine byte.  The reads of
     // `assign` go out in batches of kInitBatch so that their latency is paid once per batch, not per row.
    constexpr int kInitBatch = 16;
    IdxT at = 0;
    int i = 0;
    if (!BY_POS) {
      for (; i + kInitBatch <= V; i += kInitBatch) {
        uint32_t x[kInitBatch];
#pragma unroll
        for (int u = 0; u < kInitBatch; ++u) { x[u] = (uint32_t)assign_col[at]; at += Ki; }
#pragma unroll
        for (int u = 0; u < kInitBatch; ++u) {
          if (S16) { raw_max = max(raw_max, x[u]); x[u] = min(x[u], (uint32_t)(D - 1)); }   // the field is only jbits wide
          state[(uint32_t)(i + u) * pitch] = (StateT)(unsched | x[u]);
        }
      }
    }
    for (; i < V; ++i) {
      uint32_t x1 = BY_POS ? 0u : (uint32_t)assign_col[at];
      if (S16) { raw_max = max(raw_max, x1); x1 = min(x1, (uint32_t)(D - 1)); }
      state[(uint32_t)i * pitch] = (StateT)(BY_POS ? 0xFFFFFFFFu : (unsched | x1));
      at += Ki;
    }
    state[(uint32_t)V * pitch] = (StateT)0;
  }
  for (int j = 0; j < D; ++j) {
    dev[j * dpitch] = make_int4(0, 0, 0, 0);
    if (gp.weight) wsum[j * dpitch] = 0;
  }
  if (EXCL)
    for (int q = 0; q < D * D; ++q) chan[(uint32_t)q * cpitch] = 0;
  const bool by_op_times = (flags & PE_TIMES_BY_OP) != 0;
  const bool deep = g.max_indeg > 2;
  const uint32_t vmax = (uint32_t)(V - 1), dmax = (uint32_t)(D - 1);
  const IdxT off_last = (IdxT)vmax * Ki;
  uint32_t st = 0;
  int32_t z = 0;
  // validity accumulators, tested after the loop
  uint32_t order_max = 0, dev_max = 0, pred_max = 0, own_min = 0xFFFFFFFFu;

  int32_t* start_col = TIMES ? out.start + c : nullptr;
  int32_t* finish_col = TIMES ? out.finish + c : nullptr;

  // register rings: o0/a0 = the block being processed, o1/a1 = the block after it
  uint32_t o0[kUnroll], o1[kUnroll], a0[kUnroll], a1[kUnroll];
  IdxT off_load = 0;  // element offset (row * K) of the next row to prefetch, clamped to the last row
  auto prefetch = [&](uint32_t (&od)[kUnroll], uint32_t (&ad)[kUnroll]) {
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
      const IdxT at = min(off_load, off_last);
      od[u] = (uint32_t)order_col[at];
      if (BY_POS) ad[u] = (uint32_t)assign_col[at];
      off_load += Ki;
    }
  };
  prefetch(o0, a0);
  prefetch(o1, a1);
  uint4 rec_next = gp.ops[min(o0[0], vmax)];
  IdxT off_k = 0;  // element offset of the current position's row

  auto step = [&](const uint32_t iu, const uint32_t a_pos, const uint32_t nxt) {
    const uint4 rec = rec_next;
    rec_next = gp.ops[min(nxt, vmax)];  // operator record of the next position, while this one is computed
    order_max = max(order_max, iu);
    const uint32_t i = min(iu, vmax);
    const uint32_t mine = state[i * pitch];
    own_min = min(own_min, mine);
    const uint32_t jr = BY_POS ? a_pos : (mine & jmask);
    dev_max = max(dev_max, jr);
    const int j = (int)min(jr, dmax);
    const int4 dv = dev[j * dpitch];
    const int indeg = (int)(rec.y >> 24);
    const int32_t dur = (int32_t)(rec.y & 0xFFFFu);
    const int32_t dA = (int32_t)(rec.y << 8) >> 24;

    // one incoming edge: lo = comm[class 0] << 16 | pred, hi = comm[class 1]
    auto edge_time = [&](uint32_t lo, uint32_t hi) -> int32_t {
      const uint32_t p = lo & 0xFFFFu;
      const uint32_t w = state[p * pitch];
      pred_max = max(pred_max, w);
      const int xp = (int)(w & jmask);
      const uint32_t xpc = min((uint32_t)xp, dmax);  // (an unscheduled source of an invalid order may still carry a raw id)
      uint32_t delay = lo >> 16;
      bool channel = true;
      if (NEED_CLS) {
        const uint32_t cl = gp.cls[xpc * D + j];
        if (TWO_CLASS) delay = cl == 1u ? hi : delay;
        if (cl == 0xFFu) {
          delay = 0;
          channel = false;
          if (p != (uint32_t)V && xp != j) st |= PE_STATUS_NO_CHANNEL;
        }
      }
      if (EXCL) {
        // the transfer starts when its source has ended (Eq. 13) and the channel is free (Eq. 14), lasts D^c (Eq. 11)
        if (xp != j && p != (uint32_t)V && channel) {
          int32_t* ch = chan + (xpc * D + j) * cpitch;
          const int32_t t_end = max((int32_t)(w >> jb), *ch) + (int32_t)delay;
          *ch = t_end;
          return t_end;
        }
        return (int32_t)(w >> jb);
      }
      return (int32_t)(w >> jb) + (xp != j ? (int32_t)delay : 0);
    };
    int32_t r = edge_time(rec.z, rec.w);
    if (TWO_CLASS) {
      if (indeg > 1) {
        const uint2* ed = reinterpret_cast<const uint2*>(gp.edges) + rec.x;
        for (int q = 1; q < indeg; ++q) r = max(r, edge_time(ed[q].x, ed[q].y));
      }
    } else if (DEPTH == 3) {
      const int32_t t1 = edge_time(rec.w, 0u);   // in edge-list order: with EXCL the order of the transfers matters
      const int32_t t2 = edge_time(rec.x, 0u);
      r = max(r, max(t1, t2));
    } else {
      r = max(r, edge_time(rec.w, 0u));
      if (deep) {  // some operator has more than two incoming edges: third inline slot, then the CSR list
        r = max(r, edge_time(indeg > 3 ? (uint32_t)V : rec.x, 0u));
        if (indeg > 3) {
          const uint32_t* ed = gp.edges + rec.x;
          for (int q = 2; q < indeg; ++q) r = max(r, edge_time(ed[q], 0u));
        }
      }
    }
    const int32_t s = max(r, dv.x);
    const int32_t e = s + dur;
    const int32_t lv = dv.z + dA;
    dev[j * dpitch] = make_int4(e, dv.y + dur, lv, max(dv.w, lv));
    state[i * pitch] = (StateT)(((uint32_t)e << jb) | (uint32_t)j);
    if (gp.weight) wsum[j * dpitch] += gp.weight[i];
    z = max(z, e);
    if (TIMES) {
      const IdxT at = by_op_times ? (IdxT)i * Ki : off_k;
      start_col[at] = s;
      finish_col[at] = e;
    }
    off_k += Ki;
  };

  int kb = 0;
  for (; kb + kUnroll <= V; kb += kUnroll) {
    uint32_t o2[kUnroll], a2[kUnroll];
    prefetch(o2, a2);
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) step(o0[u], a0[u], u + 1 < kUnroll ? o0[(u + 1) % kUnroll] : o1[0]);
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) { o0[u] = o1[u]; o1[u] = o2[u]; a0[u] = a1[u]; a1[u] = a2[u]; }
  }
#pragma unroll
  for (int u = 0; u < kUnroll; ++u)  // the last, partial block
    if (kb + u < V) step(o0[u], a0[u], o0[(u + 1) % kUnroll]);

  if (order_max > vmax) st |= PE_STATUS_ORDER_INVALID;    // an entry that is no operator
  if (own_min < unsched) st |= PE_STATUS_ORDER_INVALID;   // an operator scheduled twice
  if (pred_max >= unsched) st |= PE_STATUS_ORDER_INVALID;  // an operator ahead of one of its predecessors
  if (dev_max > dmax) st |= PE_STATUS_ASSIGN_RANGE;
  if (S16 && !BY_POS && raw_max > dmax) {
    // Some operator's machine id is out of range and was clamped when the state was set up.  The bit is due
    // only if that operator is consulted, i.e. appears in the order: certain for a permutation, otherwise
    // (a rare double fault) the order is walked once more.
    if (!(st & PE_STATUS_ORDER_INVALID)) {
      st |= PE_STATUS_ASSIGN_RANGE;
    } else {
      for (int k = 0; k < V; ++k) {
        const uint32_t iu = (uint32_t)order_col[(IdxT)k * Ki];
        if (iu <= vmax && (uint32_t)assign_col[(IdxT)iu * Ki] > dmax) st |= PE_STATUS_ASSIGN_RANGE;
      }
    }
  }
  for (int j = 0; j < D; ++j) {
    const int4 dv = dev[j * dpitch];
    const int32_t pk = dv.w + (gp.weight ? wsum[j * dpitch] : 0);  // the weights are resident from the start (Eq. 16)
    if (pk > gp.cap[j]) st |= PE_STATUS_MEM_EXCEEDED;
    if (out.busy) out.busy[(size_t)j * (size_t)K + c] = dv.y;
    if (out.peak_mem) out.peak_mem[(size_t)j * (size_t)K + c] = pk;
  }
  if (out.makespan) out.makespan[c] = z;
  if (out.status) out.status[c] = st;
}

}  // namespace pe
