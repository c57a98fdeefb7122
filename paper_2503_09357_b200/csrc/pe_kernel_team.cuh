// Variant TEAM over the compact graph encoding: one block per candidate, NW warps that take the
// windows of 32 consecutive positions of the priority order in turn, per-operator state in shared
// memory.
//
// When a candidate's state (4 bytes per operator) is so large that only a handful fit on an SM, a
// single warp per candidate leaves the SM idle: a window then costs the latency of everything it
// does, one thing after the other.  Most of that work does not depend on any start or end time:
// which operator sits at a position, its record, the machines of its predecessors and hence the
// delay of each incoming edge (Eqs. 9, 11-13), whether a predecessor sits in the same window, which
// operator precedes it on its machine inside the window (Eqs. 7-8), the memory levels (Eqs. 16-19).
// Only the recurrence itself, s_i = max(ready, free_j), e_i = s_i + D^o_i (Eqs. 3, 7-8, 11-13), has
// to follow the order.  So the block works as a pipeline:
//   * an initial pass writes every operator's position in the order and its machine into the state
//     word ("pending": position << 8 | machine), so that later nobody has to wait to learn where a
//     predecessor sits;
//   * warp w prepares windows w, w + NW, ... on its own: it reads the order entries and operator
//     records (prefetched), classifies the incoming edges into sources inside the window (lane,
//     delay) and sources before it (state address, delay), and finds the machine's previous
//     operator in the window;
//   * a baton (a named barrier between two warps) goes from window to window.  The warp that holds
//     it gathers the end times of the sources before the window (final by then) and relaxes the window
//     with shuffles: every lane takes the maximum over its in-window sources' current end times plus
//     delays, for as many rounds as the window is deep (the depth is known from the set-up, so the
//     loop needs no vote); then it publishes end << 8 | machine and passes the baton on.  Only this
//     part is serial, it touches nothing but shared memory and registers, and it never diverges;
//   * the memory levels follow each machine's sequence, not the times: they have their own, much
//     shorter, baton, and run ahead of the times.
// State word: pending = 0x80000000 | position << 8 | machine (position 0xFFFF = not in the order);
// final = end << 8 | machine, end < 2^23.  Row V is the sentinel the compact encoding's empty edge
// slots point at (final, end 0, machine 0); row V + 1 takes the writes of lanes that have nothing to
// write.
//
// Inputs and times either use the candidate-interleaved arrays of the interface directly (every lane
// then touches its own 32-byte sector) or, STAGED, candidate-major copies made by pe_transpose_kernel,
// where a window's order entries and times are 64 and 128 contiguous bytes.
//
// The kernel serves graphs in which no operator has more than eight incoming edges: three slots for the
// edges the compact record carries inline, and (WIDE) five more for edges read from the edge list.
#pragma once
#include "pe_device.cuh"

namespace pe {

constexpr uint32_t kTeamPending = 0x80000000u;
constexpr int64_t kTeamTimeLimit = (int64_t)1 << 23;   // end times must stay below this

// Named barriers between pairs of warps (64 threads: the warp that arrives does not wait).  With the barrier
// number in a register the compiler reserves all sixteen barriers of a block, and an SM has barrier resources
// for only four such blocks; with immediates it reserves what is used (two per warp plus the block's own).
template <int ID>
__device__ __forceinline__ void bar_sync_id() {
  asm volatile("bar.sync %0, 64;" ::"n"(ID) : "memory");
}
template <int ID>
__device__ __forceinline__ void bar_arrive_id() {
  asm volatile("bar.arrive %0, 64;" ::"n"(ID) : "memory");
}
// barrier number = BASE + w, w in 0 .. NW - 1 (warp-uniform).  IMM: a row of one-instruction conditionals on
// immediates (the comparisons are loop invariant: NW predicated instructions, no branch); otherwise one
// instruction with the number in a register, which is faster under the baton (measured at V = 16384 with six
// warps: 16.2 against 18.8 ms for 32768 candidates) and is used where shared memory allows no more than four
// blocks per SM anyway.
template <int BASE, int NW, bool IMM>
__device__ __forceinline__ void named_sync(int w) {
  if (!IMM) {
    asm volatile("bar.sync %0, 64;" ::"r"(BASE + w) : "memory");
    return;
  }
  if (w == 0) bar_sync_id<BASE + 0>();
  if (w == 1) bar_sync_id<BASE + 1>();
  if (NW > 2 && w == 2) bar_sync_id<BASE + 2>();
  if (NW > 3 && w == 3) bar_sync_id<BASE + 3>();
  if (NW > 4 && w == 4) bar_sync_id<BASE + 4>();
  if (NW > 5 && w == 5) bar_sync_id<BASE + 5>();
}
template <int BASE, int NW, bool IMM>
__device__ __forceinline__ void named_arrive(int w) {
  if (!IMM) {
    asm volatile("bar.arrive %0, 64;" ::"r"(BASE + w) : "memory");
    return;
  }
  if (w == 0) bar_arrive_id<BASE + 0>();
  if (w == 1) bar_arrive_id<BASE + 1>();
  if (NW > 2 && w == 2) bar_arrive_id<BASE + 2>();
  if (NW > 3 && w == 3) bar_arrive_id<BASE + 3>();
  if (NW > 4 && w == 4) bar_arrive_id<BASE + 4>();
  if (NW > 5 && w == 5) bar_arrive_id<BASE + 5>();
}

// Element (row, c) of an input or output array sits at row * row_stride + c * cand_stride: (K, 1) for
// the candidate-interleaved arrays of the interface, (1, rows) for candidate-major staging copies.
struct TeamStrides {
  size_t in_row, in_cand;     // assign, order
  size_t out_row, out_cand;   // start, finish
};

template <int NW, bool BY_POS, int CLS, bool TIMES, bool STAGED, bool WIDE>
__global__ void __launch_bounds__(NW * 32) pe_eval_team_kernel(PeNarrowView g, const uint8_t* __restrict__ nblob,
                                                               int64_t K, const uint8_t* __restrict__ assign,
                                                               const uint16_t* __restrict__ order, pe_outputs out,
                                                               uint32_t flags, TeamStrides sd) {
  extern __shared__ __align__(16) uint8_t smem_raw[];
  static_assert(NW >= 2 && NW <= 6, "two named barriers per warp (numbers 1 .. 2 NW), barrier 0 is the block's");
  constexpr uint32_t FULL = 0xFFFFFFFFu;
  constexpr bool TWO_CLASS = CLS == 2;
  constexpr bool NEED_CLS = CLS != 0;
  constexpr int NT = NW * 32;
  constexpr bool IMMBAR = NW < 6;   // six warps per block go with large states, where few blocks fit anyway
  constexpr int32_t kNever = -(1 << 29);   // delay of an empty slot: never wins the maximum
  const int tid = threadIdx.x;
  const int lane = tid & 31;
  const int warp = tid >> 5;
  const int D = g.D, V = g.V;
  const NarrowPtrs gp = narrow_ptrs(nblob, g);
  const int64_t c = blockIdx.x;
  const uint32_t vmax = (uint32_t)(V - 1), dmax = (uint32_t)(D - 1);

  uint32_t* state = reinterpret_cast<uint32_t*>(smem_raw);   // [V + 2]: row V the sentinel (always 0), row V + 1 a dump
  int32_t* free_at = reinterpret_cast<int32_t*>(state + V + 2);   // = state[V + 2 + machine]
  int32_t* lvl = free_at + D;
  int32_t* peak = lvl + D;
  int32_t* busy = peak + D;
  int32_t* wsum = busy + D;
  int32_t* red = wsum + D;   // [0] makespan, [1] status

  const uint16_t* order_col = order + (size_t)c * sd.in_cand;
  const uint8_t* assign_col = assign + (size_t)c * sd.in_cand;
  uint32_t st = 0;
  uint32_t order_max = 0, dev_max = 0;

  // ---- initial pass: machine and position of every operator ----
  for (int idx = tid; idx < 5 * D + 2; idx += NT) free_at[idx] = 0;
  if (tid == 0) state[V] = 0u;
  constexpr int kBatch = 8;   // loads in flight per thread
  if constexpr (STAGED) {
    // candidate-major staging copies: the candidate's machine ids and order entries are contiguous
    // (rows padded with zeros to a multiple of 64 entries), four entries per load
    const uint32_t* a4 = reinterpret_cast<const uint32_t*>(assign_col);
    const uint2* o4 = reinterpret_cast<const uint2*>(order_col);
    const int nq = (V + 3) >> 2;
    for (int b = tid; b < nq; b += NT * kBatch) {
      uint32_t x[kBatch];
#pragma unroll
      for (int q = 0; q < kBatch; ++q) {
        const int v4 = b + q * NT;
        x[q] = (!BY_POS && v4 < nq) ? a4[v4] : 0u;
      }
#pragma unroll
      for (int q = 0; q < kBatch; ++q) {
        const int v4 = b + q * NT;
        if (v4 < nq) {
#pragma unroll
          for (int h = 0; h < 4; ++h)
            if (4 * v4 + h < V) state[4 * v4 + h] = kTeamPending | 0xFFFF00u | ((x[q] >> (8 * h)) & 0xFFu);
        }
      }
    }
    __syncthreads();
    for (int b = tid; b < nq; b += NT * kBatch) {
      uint2 o[kBatch];
      uint32_t a[kBatch];
#pragma unroll
      for (int q = 0; q < kBatch; ++q) {
        const int v4 = b + q * NT;
        o[q] = v4 < nq ? o4[v4] : make_uint2(0xFFFFFFFFu, 0xFFFFFFFFu);
        a[q] = (BY_POS && v4 < nq) ? a4[v4] : 0u;
      }
#pragma unroll
      for (int q = 0; q < kBatch; ++q) {
        const int v4 = b + q * NT;
#pragma unroll
        for (int h = 0; h < 4; ++h) {
          const int k = 4 * v4 + h;
          const uint32_t oe = ((h < 2 ? o[q].x : o[q].y) >> (16 * (h & 1))) & 0xFFFFu;
          const uint32_t ae = (a[q] >> (8 * h)) & 0xFFu;
          if (v4 < nq && k < V && oe <= vmax) {
            if (BY_POS) {
              dev_max = max(dev_max, ae);
              state[oe] = kTeamPending | ((uint32_t)k << 8) | ae;
            } else {
              state[oe] = kTeamPending | ((uint32_t)k << 8) | (state[oe] & 0xFFu);
            }
          }
        }
      }
    }
    __syncthreads();
  } else {
  for (int b = tid; b < V; b += NT * kBatch) {
    uint32_t x[kBatch];
#pragma unroll
    for (int q = 0; q < kBatch; ++q) {
      const int i = b + q * NT;
      x[q] = (!BY_POS && i < V) ? (uint32_t)assign_col[(size_t)i * sd.in_row] : 0u;
    }
#pragma unroll
    for (int q = 0; q < kBatch; ++q) {
      const int i = b + q * NT;
      if (i < V) state[i] = kTeamPending | 0xFFFF00u | x[q];
    }
  }
  __syncthreads();
  for (int b = tid; b < V; b += NT * kBatch) {
    uint32_t o[kBatch], a[kBatch];
#pragma unroll
    for (int q = 0; q < kBatch; ++q) {
      const int k = b + q * NT;
      o[q] = k < V ? (uint32_t)order_col[(size_t)k * sd.in_row] : 0xFFFFFFFFu;
      a[q] = (BY_POS && k < V) ? (uint32_t)assign_col[(size_t)k * sd.in_row] : 0u;
    }
#pragma unroll
    for (int q = 0; q < kBatch; ++q) {
      const int k = b + q * NT;
      if (o[q] <= vmax) {
        if (BY_POS) {
          dev_max = max(dev_max, a[q]);
          state[o[q]] = kTeamPending | ((uint32_t)k << 8) | a[q];
        } else {
          state[o[q]] = kTeamPending | ((uint32_t)k << 8) | (state[o[q]] & 0xFFu);
        }
      }
    }
  }
  __syncthreads();
  }

  const bool by_op_times = (flags & PE_TIMES_BY_OP) != 0;
  const uint32_t lt_mask = (1u << lane) - 1u;
  const int nwin = (V + 31) >> 5;
  const int next_warp = (warp + 1) % NW;
  int32_t z = 0;
  int32_t* start_col = TIMES ? out.start + (size_t)c * sd.out_cand : nullptr;
  int32_t* finish_col = TIMES ? out.finish + (size_t)c * sd.out_cand : nullptr;

  // order entries two of this warp's windows ahead, operator records one ahead
  auto load_order = [&](int win) -> uint32_t {
    const int k = win * 32 + lane;
    if (k >= V) return 0u;
    return STAGED ? (uint32_t)order_col[k] : (uint32_t)order_col[(size_t)k * sd.in_row];
  };
  uint32_t o_cur = load_order(warp), o_nxt = load_order(warp + NW);
  uint4 rec_nxt = __ldg(gp.ops + min(o_cur, vmax));
  const uint32_t none = (uint32_t)V;

  for (int win = warp; win < nwin; win += NW) {
    const int base = win * 32;
    const int k = base + lane;
    const bool act = k < V;
    const uint32_t iu = o_cur;
    const uint4 rec = rec_nxt;
    o_cur = o_nxt;
    o_nxt = load_order(win + 2 * NW);
    rec_nxt = __ldg(gp.ops + min(o_cur, vmax));

    // ---- set-up: nothing here depends on a time ----
    const uint32_t i = act ? min(iu, vmax) : none;
    const uint32_t own = state[i];
    const uint32_t jr = own & 0xFFu;
    const uint32_t j = min(jr, dmax);
    if (act) {
      order_max = max(order_max, iu);
      if (!BY_POS) dev_max = max(dev_max, jr);
      if ((own >> 8) != ((kTeamPending >> 8) | (uint32_t)k)) st |= PE_STATUS_ORDER_INVALID;   // repeated operator
    }
    const int indeg = (int)(rec.y >> 24);
    const int32_t dur = act ? (int32_t)(rec.y & 0xFFFFu) : 0;
    const int32_t dA = act ? (int32_t)(rec.y << 8) >> 24 : 0;

    // previous / last operator of the same machine inside the window (Eqs. 7-8)
    const uint32_t same_dev = __match_any_sync(FULL, act ? j : (0x100u | lane));
    const uint32_t below = same_dev & lt_mask;
    const bool has_prev = below != 0;
    const bool last_on_dev = (same_dev >> lane) == 1u;

    // Incoming edges: edge q owns slot q.  A source inside the window becomes (lane, delay) for the
    // relaxation; any other becomes (state address, delay) for the gather under the baton.  The unused
    // half of a slot is neutral: lane = own lane with delay kNever, address = sentinel with delay kNever.
    // `rel` is the source's position relative to the window when its word is pending; a final word
    // (bit 31 clear) wraps to a huge value, so one unsigned compare tells "inside the window, before me".
    const uint32_t pend_base = (kTeamPending >> 8) + (uint32_t)base;
    uint32_t depmask = 0;
    uint32_t a0, a1, a2;
    int32_t g0, g1, g2, d0, d1, d2;
    int l0, l1, l2;
    auto classify = [&](uint32_t lo, uint32_t hi, uint32_t& addr, int32_t& gdel, int& lsl, int32_t& ldel) {
      const uint32_t p = lo & 0xFFFFu;
      const uint32_t w = state[p];
      const uint32_t xp = w & 0xFFu;
      uint32_t delay = lo >> 16;
      if (NEED_CLS) {
        const uint32_t cl = gp.cls[min(xp, dmax) * D + j];
        if (TWO_CLASS) delay = cl == 1u ? hi : delay;
        if (cl == 0xFFu) {
          delay = 0;
          if (p != none && xp != j) st |= PE_STATUS_NO_CHANNEL;
        }
      }
      const int32_t dly = xp != j ? (int32_t)delay : 0;
      const uint32_t rel = (w >> 8) - pend_base;
      const bool inw = rel < (uint32_t)lane;
      if (!inw && rel < 0x10000u) st |= PE_STATUS_ORDER_INVALID;   // pending, but not before this operator
      addr = inw ? none : p;
      gdel = inw ? kNever : dly;
      lsl = inw ? (int)rel : lane;
      ldel = (inw ? dly : kNever) + dur;   // D^o folded into the in-window delays (Eq. 3)
      depmask |= inw ? 1u << rel : 0u;
    };
    // (a lane beyond the end of the order goes through the same code on operator 0's record; what it
    //  classifies and flags is dropped right after)
    const uint32_t st_before = st;
    // WIDE: operators with four to eight incoming edges; edges 3.. take the extra slots
    constexpr int kExtra = WIDE ? 5 : 1;
    uint32_t xa[kExtra];
    int32_t xg[kExtra], xd[kExtra];
    int xl[kExtra];
#pragma unroll
    for (int q = 0; q < kExtra; ++q) { xa[q] = none; xg[q] = kNever; xl[q] = lane; xd[q] = kNever + dur; }
    classify(rec.z, rec.w, a0, g0, l0, d0);
    if (TWO_CLASS) {
      a1 = none; a2 = none; g1 = kNever; g2 = kNever; l1 = lane; l2 = lane; d1 = kNever + dur; d2 = kNever + dur;
      const uint2* ed = reinterpret_cast<const uint2*>(gp.edges) + rec.x;
      if (indeg > 1) { const uint2 e1 = __ldg(ed + 1); classify(e1.x, e1.y, a1, g1, l1, d1); }
      if (indeg > 2) { const uint2 e2 = __ldg(ed + 2); classify(e2.x, e2.y, a2, g2, l2, d2); }
      if constexpr (WIDE) {
#pragma unroll
        for (int q = 0; q < kExtra; ++q)
          if (indeg > 3 + q) { const uint2 eq = __ldg(ed + 3 + q); classify(eq.x, eq.y, xa[q], xg[q], xl[q], xd[q]); }
      }
    } else {
      classify(rec.w, 0u, a1, g1, l1, d1);
      if constexpr (WIDE) {
        // with more than three incoming edges the record's first word is the edge list's slot, not edge 2
        const uint32_t* ed = gp.edges + rec.x;
        const bool many = indeg > 3;
        classify(many ? __ldg(ed + 2) : rec.x, 0u, a2, g2, l2, d2);
#pragma unroll
        for (int q = 0; q < kExtra; ++q)
          if (indeg > 3 + q) classify(__ldg(ed + 3 + q), 0u, xa[q], xg[q], xl[q], xd[q]);
      } else {
        classify(rec.x, 0u, a2, g2, l2, d2);
      }
    }
    if (!act) {
      st = st_before; depmask = 0; a0 = a1 = a2 = none;
#pragma unroll
      for (int q = 0; q < kExtra; ++q) xa[q] = none;
    }
    const int prev = 31 - __clz(below);
    const int lp = has_prev ? prev : lane;
    const int32_t dp = (has_prev ? 0 : kNever) + dur;
    depmask |= has_prev ? 1u << prev : 0u;
    // Depth of the window: peel off, round by round, the lanes whose sources are all peeled.  After n
    // rounds of relaxation every lane of depth <= n holds its final value, so the number of rounds is
    // known before the baton arrives and the loop under it needs no vote.
    int nrounds = 0;
    {
      uint32_t done = __ballot_sync(FULL, depmask == 0);
      while (done != FULL) {
        done = __ballot_sync(FULL, (depmask & ~done) == 0);
        ++nrounds;
      }
    }

    // ---- memory levels (Eqs. 17-19): prefix sums of A along each machine's lanes, then the machine's
    // level before the window, under the ledger baton ----
    int32_t lv = dA;
    {
      uint32_t m = below;
      while (__any_sync(FULL, m != 0)) {
        const int top = 31 - __clz(m);   // (-1 when m == 0: the shuffle then reads lane 31 and the value is dropped)
        const int32_t a_src = __shfl_sync(FULL, dA, top);
        lv += m ? a_src : 0;
        m &= ~(1u << (top & 31));
      }
    }
    if (act) {
      atomicAdd(&busy[j], dur);
      if (gp.weight) atomicAdd(&wsum[j], gp.weight[i]);
    }
    if (win > 0) named_sync<1 + NW, NW, IMMBAR>(warp);
    if (act) {
      lv += lvl[j];
      atomicMax(&peak[j], lv);
    }
    __syncwarp();
    if (act && last_on_dev) lvl[j] = lv;
    __syncwarp();
    if (win + 1 < nwin) named_arrive<1 + NW, NW, IMMBAR>(next_warp);

    // ---- times, under the baton: every earlier window is final ----
    // (all accesses under the baton are unconditional: a lane with nothing to read reads the sentinel,
    //  a lane with nothing to write writes the dump row, so the warp never diverges here)
    const uint32_t fr_at = (act && !has_prev) ? (uint32_t)(V + 2) + j : none;            // machine free since
    const uint32_t st_at = act ? i : none + 1u;                                           // own state word
    const uint32_t fw_at = (act && last_on_dev) ? (uint32_t)(V + 2) + j : none + 1u;      // machine free from
    if (win > 0) named_sync<1, NW, IMMBAR>(warp);
    const uint32_t w0 = state[a0], w1 = state[a1], w2 = state[a2];
    const int32_t fr = (int32_t)state[fr_at];
    int32_t r_base = __vimax3_s32(__viaddmax_s32((int32_t)(w0 >> 8), g0, fr), (int32_t)(w1 >> 8) + g1,
                                  (int32_t)(w2 >> 8) + g2);
    if constexpr (WIDE) {
      uint32_t xw[kExtra];
#pragma unroll
      for (int q = 0; q < kExtra; ++q) xw[q] = state[xa[q]];
#pragma unroll
      for (int q = 0; q < kExtra; ++q) r_base = __viaddmax_s32((int32_t)(xw[q] >> 8), xg[q], r_base);
    }
    const int32_t b_end = r_base + dur;
    int32_t e = b_end;
    // every dependence points to a lower lane, so the values rise monotonically to the window's
    // longest-path solution, which they reach after `nrounds` rounds
    for (int it = 0; it < nrounds; ++it) {
      const int32_t s0 = __shfl_sync(FULL, e, l0), s1 = __shfl_sync(FULL, e, l1);
      const int32_t s2 = __shfl_sync(FULL, e, l2), s3 = __shfl_sync(FULL, e, lp);
      int32_t en = __vimax3_s32(__viaddmax_s32(s0, d0, b_end), __viaddmax_s32(s1, d1, s2 + d2), s3 + dp);
      if constexpr (WIDE) {
        int32_t xs[kExtra];
#pragma unroll
        for (int q = 0; q < kExtra; ++q) xs[q] = __shfl_sync(FULL, e, xl[q]);
#pragma unroll
        for (int q = 0; q < kExtra; ++q) en = __viaddmax_s32(xs[q], xd[q], en);
      }
      e = en;
    }
    state[st_at] = ((uint32_t)e << 8) | j;
    state[fw_at] = (uint32_t)e;
    __syncwarp();
    if (win + 1 < nwin) named_arrive<1, NW, IMMBAR>(next_warp);

    // ---- after the baton has gone: outputs ----
    z = max(z, e);
    if (TIMES && act) {
      const uint32_t row = by_op_times ? i : (uint32_t)k;
      const size_t at = STAGED ? (size_t)row : (size_t)row * sd.out_row;
      start_col[at] = e - dur;
      finish_col[at] = e;
    }
  }

  if (order_max > vmax) st |= PE_STATUS_ORDER_INVALID;
  if (dev_max > dmax) st |= PE_STATUS_ASSIGN_RANGE;
  for (int off = 16; off > 0; off >>= 1) {
    z = max(z, __shfl_xor_sync(FULL, z, off));
    st |= __shfl_xor_sync(FULL, st, off);
  }
  if (lane == 0) {
    atomicMax(&red[0], z);
    atomicOr(reinterpret_cast<uint32_t*>(&red[1]), st);
  }
  __syncthreads();
  if (warp == 0) {
    uint32_t over = 0;
    for (int j = lane; j < D; j += 32) {
      const int32_t pk = peak[j] + (gp.weight ? wsum[j] : 0);   // the weights are resident from the start (Eq. 16)
      if (pk > gp.cap[j]) over = 1;
      if (out.busy) out.busy[(size_t)j * (size_t)K + c] = busy[j];
      if (out.peak_mem) out.peak_mem[(size_t)j * (size_t)K + c] = pk;
    }
    uint32_t stf = (uint32_t)red[1];
    if (__any_sync(FULL, over != 0)) stf |= PE_STATUS_MEM_EXCEEDED;
    if (lane == 0) {
      if (out.makespan) out.makespan[c] = red[0];
      if (out.status) out.status[c] = stf;
    }
  }
}

}  // namespace pe
