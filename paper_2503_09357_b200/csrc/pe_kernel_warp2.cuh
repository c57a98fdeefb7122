// Variant WARP over the compact graph encoding: one warp per candidate, a window of 32
// consecutive positions of the priority order at a time, per-operator state in shared memory.
//
// A candidate whose state (4 bytes per operator) is too large for a thread-per-candidate
// block still fits on chip when a whole warp shares it.  Inside a window the only things an
// operator can wait for are (a) a predecessor that sits in the same window and (b) the
// previous operator of its machine in the same window (Eqs. 7-8); both sit at lower lanes
// because the order is topological.  The window is therefore resolved in two steps.
// Set-up: each lane marks its operator "in this window, lane l" in the state, then reads its
// incoming edges once; a source that is already scheduled contributes its end time plus the
// cross-machine delay (Eqs. 11-13) at once, a source at a lower lane of the window is
// remembered, as is the machine's previous operator inside the window (Eqs. 7-8).  Then
//   REG_SLOTS (no operator has more than three incoming edges): the remembered sources are
//     (lane, delay) pairs in registers and the window is relaxed with shuffles: every lane
//     repeatedly takes the maximum of what it has and its sources' current end times plus
//     delays and ends D^o later (Eq. 3); the values rise to the window's longest-path solution
//     and the loop stops when nothing changes - mostly long before the window's depth (used with
//     many warps per SM; with few, a lane instead evaluates once, when the lanes it waits for are
//     final, which keeps the loop-carried chain to a ballot and a mask test);
//   otherwise: the remembered sources are operator ids (the inline ones) or the edge list
//     itself, the lanes waited for form a mask `need`, and the window is resolved in rounds: a
//     lane whose `need` lanes have finished evaluates once, from the state in shared memory, and
//     publishes; the lowest unfinished lane is always ready, so at most 32 rounds.
// Memory levels (Eqs. 16-19) do not depend on times: they are prefix sums along each
// machine's lanes, formed once per window with shuffles.
//
// State word: end << 8 | machine when scheduled (end < 0xFFFF00); 0xFFFFC000 | lane << 8 |
// machine while in the current window; 0xFFFFFF00 | machine before that.  Row V is the
// sentinel the compact encoding's empty edge slots point at (scheduled, end 0, machine 0).
#pragma once
#include "pe_device.cuh"
#include "pe_kernel_lane.cuh"

namespace pe {

constexpr uint32_t kDoneLimit = 0xFFFF0000u;    // state words below this carry an end time
constexpr uint32_t kInWindow = 0xFFFFC000u;     // | lane << 8 | machine
constexpr uint32_t kInWindowEnd = 0xFFFFE000u;

// SLAB: the block's warps (adjacent candidates) move through the order in slabs of kSlab positions
// with a block barrier between slabs; order entries (and by-position machine ids) of a slab are read
// from global memory row by row, coalesced, into a shared tile, and start/finish times leave through
// shared tiles the same way.  Without it every lane reads and writes its own 2..4 bytes of a
// different row, which costs a memory transaction per lane.
constexpr int kSlab = 128;

// FLAT: one link class and no operator with more than three incoming edges: the three inline slots are
// all there is, so the edge-list loops (and the `more` path) drop out of the window code.
// REG_SLOTS: no operator has more than three incoming edges (whatever the link classes): in-window
// dependences are kept as (lane, delay) in registers and resolved by shuffles.
template <typename IdxT, bool BY_POS, int CLS, bool GRAPH_SMEM, bool TIMES, bool SLAB, bool FLAT, bool REG_SLOTS>
__global__ void __launch_bounds__(1024) pe_eval_warp2_kernel(PeNarrowView g, const uint8_t* __restrict__ nblob, int64_t K,
                                                             const uint8_t* __restrict__ assign,
                                                             const uint16_t* __restrict__ order, pe_outputs out,
                                                             uint32_t flags, int* err, int warp_words, int final_rounds) {
  extern __shared__ __align__(16) uint8_t smem_raw[];
  constexpr uint32_t FULL = 0xFFFFFFFFu;
  constexpr bool TWO_CLASS = CLS == 2;
  constexpr bool NEED_CLS = CLS != 0;
  const int lane = threadIdx.x & 31;
  const int warp = threadIdx.x >> 5;
  const int nwarps = blockDim.x >> 5;
  const int D = g.D, V = g.V;
  uint8_t* sm = smem_raw;
  const uint8_t* gbase = nblob;
  if (GRAPH_SMEM) {
    uint64_t* bar = reinterpret_cast<uint64_t*>(sm + g.bytes);
    if (!stage_blob(sm, nblob, g.bytes, bar, err)) return;
    gbase = sm;
    sm += g.bytes + 16;
  }
  const NarrowPtrs gp = narrow_ptrs(gbase, g);
  const IdxT Ki = (IdxT)K;
  const int64_t c0 = (int64_t)blockIdx.x * nwarps;

  // ---- initial state of every candidate of the block ----
  uint32_t* all_words = reinterpret_cast<uint32_t*>(sm);
  if (BY_POS) {
    for (int idx = threadIdx.x; idx < nwarps * warp_words; idx += blockDim.x) all_words[idx] = 0xFFFFFFFFu;
  } else {
    // machine of every operator from the by-operator assignment: row i holds nwarps adjacent bytes
    for (int idx = threadIdx.x; idx < V * nwarps; idx += blockDim.x) {
      const int i = idx / nwarps, w = idx - i * nwarps;
      const int64_t cc = c0 + w;
      all_words[(size_t)w * warp_words + i] = kUnscheduled | (cc < K ? (uint32_t)assign[(size_t)i * (size_t)K + cc] : 0u);
    }
  }
  __syncthreads();
  uint32_t* state = all_words + (size_t)warp * warp_words;  // [V + 1]
  int32_t* free_at = reinterpret_cast<int32_t*>(state + V + 1);
  int32_t* lvl = free_at + D;
  int32_t* peak = lvl + D;
  int32_t* busy = peak + D;
  int32_t* wsum = busy + D;
  for (int j = lane; j < (gp.weight ? 5 : 4) * D; j += 32) free_at[j] = 0;
  if (lane == 0) state[V] = 0u;
  __syncwarp();

  const int64_t c = c0 + warp;
  const bool cand = c < K;           // the last block may have warps without a candidate
  if (!SLAB && !cand) return;        // (with SLAB they still take part in the tile traffic and barriers)
  const bool by_op_times = (flags & PE_TIMES_BY_OP) != 0;
  const uint32_t lt_mask = (1u << lane) - 1u;
  const uint32_t vmax = (uint32_t)(V - 1), dmax = (uint32_t)(D - 1);
  uint32_t st = 0;
  int32_t z = 0;
  uint32_t order_max = 0, dev_max = 0;
  const uint16_t* order_col = order + c;
  const uint8_t* assign_col = assign + c;
  int32_t* start_col = TIMES ? out.start + c : nullptr;
  int32_t* finish_col = TIMES ? out.finish + c : nullptr;

  // One window: lane l holds position k of the order (act = it exists), operator entry iu, by-position
  // machine id a_here and the operator's record.  Returns start, end and the (clamped) operator.
  auto window = [&](const bool act, const uint32_t iu, const uint32_t a_here, const uint4 rec, int32_t& s_out,
                    int32_t& e_out, uint32_t& i_out) {
    if (act) order_max = max(order_max, iu);
    const uint32_t i = min(iu, vmax);
    const uint32_t mine = act ? state[i] : kUnscheduled;
    if (mine < kUnscheduled) st |= PE_STATUS_ORDER_INVALID;  // scheduled in an earlier window: a repeated operator
    const uint32_t jr = BY_POS ? a_here : (mine & 0xFFu);
    if (act) dev_max = max(dev_max, jr);
    const uint32_t j = min(jr, dmax);
    const int indeg = (int)(rec.y >> 24);
    const int32_t dur = (int32_t)(rec.y & 0xFFFFu);
    const int32_t dA = (int32_t)(rec.y << 8) >> 24;
    const uint32_t third = (!FLAT && indeg > 3) ? (uint32_t)V : rec.x;  // L == 1: third inline edge slot

    if (act) state[i] = kInWindow | ((uint32_t)lane << 8) | j;
    __syncwarp();
    if (act && ((state[i] >> 8) & 31u) != (uint32_t)lane) st |= PE_STATUS_ORDER_INVALID;  // repeated inside this window

    // previous / last operator of the same machine inside the window
    const uint32_t same_dev = __match_any_sync(FULL, act ? j : (0x100u | lane));
    const uint32_t below = same_dev & lt_mask;
    const int prev = below ? 31 - __clz(below) : -1;
    const bool last_on_dev = (same_dev >> lane) == 1u;
    const uint32_t i_prev = REG_SLOTS ? 0u : __shfl_sync(FULL, i, prev < 0 ? lane : prev);

    // memory level along the machine's lanes (Eqs. 17-19): level before the window + prefix sum of A
    int32_t lv = dA;
    {
      uint32_t m = below;
      while (__any_sync(FULL, m != 0)) {
        const int src = m ? __ffs(m) - 1 : lane;
        const int32_t a_src = __shfl_sync(FULL, dA, src);
        if (m) { lv += a_src; m &= m - 1; }
      }
    }
    if (act) {
      lv += lvl[j];
      atomicMax(&peak[j], lv);
      atomicAdd(&busy[j], dur);
      if (gp.weight) atomicAdd(&wsum[j], gp.weight[i]);
    }
    __syncwarp();
    if (act && last_on_dev) lvl[j] = lv;

    int32_t s = 0, e = 0;
    if constexpr (REG_SLOTS) {
      // Classify the incoming edges once.  A source that is already scheduled contributes its end
      // time (+ delay) to r_base right away.  A source that sits at a lower lane of this window becomes
      // a "slot": the lane it sits at and the delay that applies (Eqs. 11-13; the machines of both ends
      // are known by now).  With at most three incoming edges per operator three slots suffice.  The
      // previous operator of the machine inside the window (Eqs. 7-8) is a fourth slot with delay 0.
      constexpr int32_t kNever = -(1 << 29);   // delay of an empty slot: never wins the maximum
      int32_t r_base = 0;
      uint32_t depmask = 0;   // lanes of this window this operator waits for
      int l0 = lane, l1 = lane, l2 = lane;
      int32_t d0 = kNever, d1 = kNever, d2 = kNever;
      const uint32_t none = (uint32_t)V;  // the sentinel: always "ended at 0"
      auto delay_of = [&](uint32_t lo, uint32_t hi, uint32_t w) -> uint32_t {
        const uint32_t xp = w & 0xFFu;
        uint32_t delay = lo >> 16;
        if (NEED_CLS) {
          const uint32_t cl = gp.cls[min(xp, dmax) * D + j];  // (an unscheduled source of an invalid order may carry a raw id)
          if (TWO_CLASS) delay = cl == 1u ? hi : delay;
          if (cl == 0xFFu) {
            delay = 0;
            if ((lo & 0xFFFFu) != none && xp != j) st |= PE_STATUS_NO_CHANNEL;
          }
        }
        return xp != j ? delay : 0u;
      };
      // edge number q of an operator owns slot q (at most three incoming edges here)
      auto classify = [&](uint32_t lo, uint32_t hi, int& l_slot, int32_t& d_slot) {
        const uint32_t p = lo & 0xFFFFu;
        const uint32_t w = state[p];
        const uint32_t dly = delay_of(lo, hi, w);
        if (w < kDoneLimit) {
          r_base = max(r_base, (int32_t)((w >> 8) + dly));
        } else {
          const uint32_t l = (w >> 8) & 31u;
          if (w < kInWindowEnd && l < (uint32_t)lane) {
            l_slot = (int)l;
            d_slot = (int32_t)dly;
            depmask |= 1u << l;
          } else {
            st |= PE_STATUS_ORDER_INVALID;  // a predecessor that is not before this operator
          }
        }
      };
      int lp = lane;
      int32_t dp = kNever;
      if (act) {
        classify(rec.z, rec.w, l0, d0);
        if (TWO_CLASS) {
          const uint2* ed = reinterpret_cast<const uint2*>(gp.edges) + rec.x;
          if (indeg > 1) classify(ed[1].x, ed[1].y, l1, d1);
          if (indeg > 2) classify(ed[2].x, ed[2].y, l2, d2);
        } else {
          classify(rec.w, 0u, l1, d1);
          classify(rec.x, 0u, l2, d2);
        }
        if (prev < 0) r_base = max(r_base, free_at[j]);
        else { lp = prev; dp = 0; depmask |= 1u << prev; }   // Eqs. 7-8: after the machine's previous operator
      }

      // Two ways to resolve the window, both exchanging end times by shuffles only.
      // Relaxation (many warps per SM, instruction issue is what limits): every lane starts from what
      // it knows (r_base) and repeatedly takes the maximum over its slots of the slot lane's current
      // end time plus delay; all dependences point to lower lanes, so the values rise monotonically
      // to the window's longest-path solution and the loop stops when nothing changes - usually long
      // before the window's depth, because most dependences do not bind.
      // Rounds (few warps per SM, latency is what limits): a lane evaluates once, when every lane it
      // depends on is final; exactly (depth of the window) rounds, but the loop-carried chain is a
      // ballot and a mask test instead of shuffle, maximum, compare and vote.
      e = r_base + dur;
      if (!final_rounds) {
        if (__any_sync(FULL, depmask != 0)) {
          for (int it = 0; it < 34; ++it) {
            int32_t v = r_base;
            v = max(v, __shfl_sync(FULL, e, l0) + d0);
            v = max(v, __shfl_sync(FULL, e, l1) + d1);
            v = max(v, __shfl_sync(FULL, e, l2) + d2);
            v = max(v, __shfl_sync(FULL, e, lp) + dp);
            const int32_t en = v + dur;
            const bool changed = en != e;
            e = en;
            if (!__any_sync(FULL, changed)) break;
          }
        }
      } else {
        bool fin = depmask == 0;
        for (int it = 0; it < 33; ++it) {
          const uint32_t fm = __ballot_sync(FULL, fin);
          if (fm == FULL) break;
          int32_t v = r_base;
          v = max(v, __shfl_sync(FULL, e, l0) + d0);
          v = max(v, __shfl_sync(FULL, e, l1) + d1);
          v = max(v, __shfl_sync(FULL, e, l2) + d2);
          v = max(v, __shfl_sync(FULL, e, lp) + dp);
          if (!fin && (depmask & ~fm) == 0) { e = v + dur; fin = true; }
        }
      }
      s = e - dur;
      if (act) state[i] = ((uint32_t)e << 8) | j;

    } else {
      // Classify the incoming edges once.  A source that is already scheduled contributes its end
      // time (+ delay) to r_base right away; a source that sits at a lower lane of this window becomes
      // a "slot" (operator id | delay << 16) to be read when that lane has finished, and its lane joins
      // `need`.  Edges beyond the inline ones that are in-window set `more`: they are re-read from the
      // edge list at evaluation time.
      uint32_t need = 0;
      int32_t r_base = 0;
      bool more = false;
      const uint32_t none = (uint32_t)V;  // the sentinel: always "ended at 0"
      uint32_t slot0 = none, slot1 = none, slot2 = none, slot_prev = none;
      auto delay_of = [&](uint32_t lo, uint32_t hi, uint32_t w) -> uint32_t {
        const uint32_t xp = w & 0xFFu;
        uint32_t delay = lo >> 16;
        if (NEED_CLS) {
          const uint32_t cl = gp.cls[min(xp, dmax) * D + j];  // (an unscheduled source of an invalid order may carry a raw id)
          if (TWO_CLASS) delay = cl == 1u ? hi : delay;
          if (cl == 0xFFu) {
            delay = 0;
            if ((lo & 0xFFFFu) != none && xp != j) st |= PE_STATUS_NO_CHANNEL;
          }
        }
        return xp != j ? delay : 0u;
      };
      auto classify = [&](uint32_t lo, uint32_t hi, uint32_t& slot, bool inline_slot) {
        const uint32_t p = lo & 0xFFFFu;
        const uint32_t w = state[p];
        const uint32_t dly = delay_of(lo, hi, w);
        if (w < kDoneLimit) {
          r_base = max(r_base, (int32_t)((w >> 8) + dly));
        } else {
          const uint32_t l = (w >> 8) & 31u;
          if (w < kInWindowEnd && l < (uint32_t)lane) {
            need |= 1u << l;
            if (inline_slot) slot = p | (dly << 16);
            else more = true;
          } else {
            st |= PE_STATUS_ORDER_INVALID;  // a predecessor that is not before this operator
          }
        }
      };
      if (act) {
        uint32_t unused = none;
        classify(rec.z, rec.w, slot0, true);
        if (TWO_CLASS) {
          const uint2* ed = reinterpret_cast<const uint2*>(gp.edges) + rec.x;
          for (int q = 1; q < indeg; ++q) classify(ed[q].x, ed[q].y, unused, false);
        } else {
          classify(rec.w, 0u, slot1, true);
          classify(third, 0u, slot2, true);
          if (!FLAT && indeg > 3) {
            const uint32_t* ed = gp.edges + rec.x;
            for (int q = 2; q < indeg; ++q) classify(ed[q], 0u, unused, false);
          }
        }
        if (prev < 0) {
          r_base = max(r_base, free_at[j]);
        } else {
          need |= 1u << prev;  // Eqs. 7-8: after the machine's previous operator
          slot_prev = i_prev;
        }
      }

      // rounds: the lowest unfinished lane never waits, so every round finishes at least one
      auto slot_time = [&](uint32_t sl) -> int32_t { return (int32_t)((state[sl & 0xFFFFu] >> 8) + (sl >> 16)); };
      bool pend = act;
      uint32_t pendmask;
      while ((pendmask = __ballot_sync(FULL, pend)) != 0) {
        if (pend && (need & pendmask) == 0) {
          int32_t v = max(max(r_base, slot_time(slot0)), max(slot_time(slot1), max(slot_time(slot2), slot_time(slot_prev))));
          if (!FLAT && more) {  // in-window sources among the edges kept in the edge list: all finished by now
            if (TWO_CLASS) {
              const uint2* ed = reinterpret_cast<const uint2*>(gp.edges) + rec.x;
              for (int q = 1; q < indeg; ++q) {
                const uint32_t w = state[ed[q].x & 0xFFFFu];
                v = max(v, (int32_t)((w >> 8) + delay_of(ed[q].x, ed[q].y, w)));
              }
            } else {
              const uint32_t* ed = gp.edges + rec.x;
              for (int q = 2; q < indeg; ++q) {
                const uint32_t w = state[ed[q] & 0xFFFFu];
                v = max(v, (int32_t)((w >> 8) + delay_of(ed[q], 0u, w)));
              }
            }
          }
          s = v;
          e = s + dur;
          state[i] = ((uint32_t)e << 8) | j;
          pend = false;
        }
        __syncwarp();
      }

    }

    if (act && last_on_dev) free_at[j] = e;
    if (act) z = max(z, e);
    s_out = s; e_out = e; i_out = i;
    __syncwarp();
  };

  if (!SLAB) {
    // prefetch rings: order entries (and by-position machine ids) four windows ahead, operator
    // records two windows ahead, so that with a handful of warps per SM the window in hand never
    // waits for global memory
    auto load_order = [&](int k) -> uint32_t { return k < V ? (uint32_t)order_col[(IdxT)k * Ki] : 0u; };
    auto load_apos = [&](int k) -> uint32_t { return (BY_POS && k < V) ? (uint32_t)assign_col[(IdxT)k * Ki] : 0u; };
    uint32_t o_ring[4], a_ring[4];
#pragma unroll
    for (int w = 0; w < 4; ++w) { o_ring[w] = load_order(32 * w + lane); a_ring[w] = load_apos(32 * w + lane); }
    uint4 rec_ring[2];
    rec_ring[0] = gp.ops[min(o_ring[0], vmax)];
    rec_ring[1] = gp.ops[min(o_ring[1], vmax)];

    for (int base = 0; base < V; base += 32) {
      const int k = base + lane;
      const bool act = k < V;
      const uint32_t iu = o_ring[0];
      const uint32_t a_here = a_ring[0];
      const uint4 rec = rec_ring[0];
#pragma unroll
      for (int w = 0; w < 3; ++w) { o_ring[w] = o_ring[w + 1]; a_ring[w] = a_ring[w + 1]; }
      o_ring[3] = load_order(k + 128);
      a_ring[3] = load_apos(k + 128);
      rec_ring[0] = rec_ring[1];
      rec_ring[1] = gp.ops[min(o_ring[1], vmax)];
      int32_t s, e;
      uint32_t i;
      window(act, iu, a_here, rec, s, e, i);
      if (TIMES && act) {
        const IdxT at = (IdxT)(by_op_times ? i : (uint32_t)k) * Ki;
        start_col[at] = s;
        finish_col[at] = e;
      }
    }
  } else {
    // ---- slab mode: shared tiles behind the per-warp state ----
    // in_tile [2][kSlab][nwarps + 2] u16, apos_tile [2][kSlab][nwarps + 4] u8 (by-position ids),
    // s_tile / e_tile [kSlab][nwarps + 1] int32; the odd pitches keep a warp's column accesses and the
    // block's row accesses free of bank conflicts.
    const int in_pitch = nwarps + 2, ap_pitch = nwarps + 4, out_pitch = nwarps + 1;
    uint16_t* in_tile = reinterpret_cast<uint16_t*>(all_words + (size_t)nwarps * warp_words);
    uint8_t* apos_tile = reinterpret_cast<uint8_t*>(in_tile + (size_t)2 * kSlab * in_pitch);
    int32_t* s_tile = reinterpret_cast<int32_t*>(apos_tile + (BY_POS ? (((size_t)2 * kSlab * ap_pitch + 3) & ~(size_t)3) : 0));
    int32_t* e_tile = s_tile + (size_t)kSlab * out_pitch;
    const int nthreads = blockDim.x;
    constexpr int kPer = kSlab / 32;  // tile elements per thread and slab (kSlab * nwarps / (32 * nwarps))
    const int nslabs = (V + kSlab - 1) / kSlab;
    uint16_t o_reg[kPer];
    uint8_t a_reg[kPer];
    auto fetch_slab = [&](int sb) {   // rows of slab sb, coalesced: consecutive threads take consecutive candidates
#pragma unroll
      for (int q = 0; q < kPer; ++q) {
        const int el = threadIdx.x + q * nthreads;
        const int r = el / nwarps, w = el - r * nwarps;
        const int row = sb * kSlab + r;
        const bool ok = row < V && c0 + w < K;
        o_reg[q] = ok ? order[(size_t)row * (size_t)K + (size_t)(c0 + w)] : (uint16_t)0;
        if (BY_POS) a_reg[q] = ok ? assign[(size_t)row * (size_t)K + (size_t)(c0 + w)] : (uint8_t)0;
      }
    };
    auto stash_slab = [&](int buf) {
#pragma unroll
      for (int q = 0; q < kPer; ++q) {
        const int el = threadIdx.x + q * nthreads;
        const int r = el / nwarps, w = el - r * nwarps;
        in_tile[((size_t)buf * kSlab + r) * in_pitch + w] = o_reg[q];
        if (BY_POS) apos_tile[((size_t)buf * kSlab + r) * ap_pitch + w] = a_reg[q];
      }
    };
    fetch_slab(0);
    stash_slab(0);
    __syncthreads();
    for (int sb = 0; sb < nslabs; ++sb) {
      const int buf = sb & 1;
      if (sb + 1 < nslabs) fetch_slab(sb + 1);   // in flight while this slab is computed
      if (cand) {
        for (int wdw = 0; wdw < kSlab / 32; ++wdw) {
          const int r = wdw * 32 + lane;
          const int k = sb * kSlab + r;
          if (sb * kSlab + wdw * 32 >= V) break;   // warp-uniform
          const bool act = k < V;
          const uint32_t iu = in_tile[((size_t)buf * kSlab + r) * in_pitch + warp];
          const uint32_t a_here = BY_POS ? (uint32_t)apos_tile[((size_t)buf * kSlab + r) * ap_pitch + warp] : 0u;
          const uint4 rec = gp.ops[min(iu, vmax)];
          int32_t s, e;
          uint32_t i;
          window(act, iu, a_here, rec, s, e, i);
          if (TIMES) {
            if (by_op_times) {
              if (act) { start_col[(IdxT)i * Ki] = s; finish_col[(IdxT)i * Ki] = e; }
            } else {
              s_tile[(size_t)r * out_pitch + warp] = s;
              e_tile[(size_t)r * out_pitch + warp] = e;
            }
          }
        }
      }
      if (sb + 1 < nslabs) stash_slab(buf ^ 1);
      __syncthreads();   // this slab's times are complete in the tiles, the next slab's entries are in place
      if (TIMES && !by_op_times) {
#pragma unroll
        for (int q = 0; q < kPer; ++q) {
          const int el = threadIdx.x + q * nthreads;
          const int r = el / nwarps, w = el - r * nwarps;
          const int row = sb * kSlab + r;
          if (row < V && c0 + w < K) {
            const size_t at = (size_t)row * (size_t)K + (size_t)(c0 + w);
            out.start[at] = s_tile[(size_t)r * out_pitch + w];
            out.finish[at] = e_tile[(size_t)r * out_pitch + w];
          }
        }
        __syncthreads();   // tiles may be overwritten by the next slab
      }
    }
    if (!cand) return;
  }

  if (order_max > vmax) st |= PE_STATUS_ORDER_INVALID;
  if (dev_max > dmax) st |= PE_STATUS_ASSIGN_RANGE;
  for (int off = 16; off > 0; off >>= 1) {
    z = max(z, __shfl_xor_sync(FULL, z, off));
    st |= __shfl_xor_sync(FULL, st, off);
  }
  uint32_t over = 0;
  for (int j = lane; j < D; j += 32) {
    const int32_t pk = peak[j] + (gp.weight ? wsum[j] : 0);
    if (pk > gp.cap[j]) over = 1;
    if (out.busy) out.busy[(size_t)j * (size_t)K + c] = busy[j];
    if (out.peak_mem) out.peak_mem[(size_t)j * (size_t)K + c] = pk;
  }
  if (__any_sync(FULL, over != 0)) st |= PE_STATUS_MEM_EXCEEDED;
  if (lane == 0) {
    if (out.makespan) out.makespan[c] = z;
    if (out.status) out.status[c] = st;
  }
}

}  // namespace pe
