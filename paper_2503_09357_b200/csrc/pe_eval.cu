// pe_eval_batch: kernel variants and their dispatch.
//
// Every variant evaluates a candidate by one pass over its priority order (serial schedule
// generation): at position k the operator i = pi[k] on machine j = x[i] starts at
// max(ready time from its predecessors' end times plus cross-machine delays (Eqs. 11-13),
// end of the previous operator on machine j (Eqs. 7-8)), ends D^o_i later (Eq. 3), and the
// machine's memory level moves by A_i (Eqs. 16-19).  The variants differ in where the
// per-candidate state lives and how lanes map to candidates.
#include <atomic>
#include <map>
#include <mutex>
#include <utility>
#include <climits>
#include <cstdio>

#include "pe_device.cuh"
#include "pe_graph.h"
#include "pe_kernel_warp.cuh"
#include "pe_launch.h"

namespace pe {

static std::atomic<int64_t> g_launches{0};

bool raise_smem_limit(const void* func, size_t bytes) {
  static std::mutex mu;
  static std::map<std::pair<int, const void*>, size_t> limit;   // (device, kernel) -> bytes granted so far
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) return false;
  std::lock_guard<std::mutex> lock(mu);
  size_t& cur = limit[std::make_pair(dev, func)];
  if (bytes <= cur) return true;
  if (cudaFuncSetAttribute(func, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes) != cudaSuccess) return false;
  cur = bytes;
  return true;
}

// ============================================================================================
// Variant GLOBAL: one thread per candidate; end time of every operator in the caller's
// workspace, candidate-interleaved ([V][K] int32, -1 = not scheduled yet), machine of every
// operator either read back from `assign` (by-op layout) or kept in a second workspace array
// (by-position layout).  Works for any V, any time bound below 2^31, u16 or u32 orders.
// Per-machine state (free time, level, peak, busy, weight sum) sits in shared memory,
// [array][machine][thread] so that a warp's accesses fall in distinct banks.
// ============================================================================================
template <typename OrderT, bool BY_POS>
__global__ void pe_eval_global_kernel(PeGraphView g, const uint8_t* __restrict__ blob, int64_t K,
                                      const uint8_t* __restrict__ assign, const OrderT* __restrict__ order,
                                      pe_outputs out, uint32_t flags, int32_t* __restrict__ e_state,
                                      uint8_t* __restrict__ x_state, int32_t* __restrict__ chan_free) {
  extern __shared__ __align__(16) uint8_t smem_raw[];
  int32_t* dev = reinterpret_cast<int32_t*>(smem_raw);
  const int T = blockDim.x;
  const int t = threadIdx.x;
  const int64_t c = (int64_t)blockIdx.x * T + t;
  if (c >= K) return;
  const GraphPtrs gp = graph_ptrs(blob, g);
  const int D = g.D, V = g.V, L = g.L;
  const size_t Ks = (size_t)K;
  int32_t* free_at = dev + t;
  int32_t* lvl = dev + (size_t)1 * D * T + t;
  int32_t* peak = dev + (size_t)2 * D * T + t;
  int32_t* busy = dev + (size_t)3 * D * T + t;
  int32_t* wsum = dev + (size_t)4 * D * T + t;
  for (int j = 0; j < D; ++j) {
    free_at[j * T] = 0; lvl[j * T] = 0; peak[j * T] = 0; busy[j * T] = 0; wsum[j * T] = 0;
  }
  const bool by_op_times = (flags & PE_TIMES_BY_OP) != 0;
  uint32_t st = 0;
  int32_t z = 0;
  for (int k = 0; k < V; ++k) {
    const uint32_t iu = order[(size_t)k * Ks + c];
    if (iu >= (uint32_t)V) { st |= PE_STATUS_ORDER_INVALID; continue; }
    const int i = (int)iu;
    uint32_t jr = BY_POS ? assign[(size_t)k * Ks + c] : assign[(size_t)i * Ks + c];
    if (jr >= (uint32_t)D) { st |= PE_STATUS_ASSIGN_RANGE; jr = D - 1; }
    const int j = (int)jr;
    const PeOpRec op = load_op(gp.ops, i);
    if (e_state[(size_t)i * Ks + c] >= 0) st |= PE_STATUS_ORDER_INVALID;
    int32_t r = 0;
    for (int q = op.edge_begin; q < op.edge_begin + op.indeg; ++q) {
      const int p = gp.pred[q];
      int32_t ep = e_state[(size_t)p * Ks + c];
      if (ep < 0) { st |= PE_STATUS_ORDER_INVALID; continue; }
      uint32_t xp = BY_POS ? x_state[(size_t)p * Ks + c] : assign[(size_t)p * Ks + c];
      if (xp >= (uint32_t)D) xp = D - 1;
      if ((int)xp != j) {
        const uint32_t cl = gp.cls[xp * D + j];
        if (cl == 0xFFu) {
          st |= PE_STATUS_NO_CHANNEL;
        } else if (chan_free) {
          // PE_COMM_EXCLUSIVE: the channel (machine of p -> j) carries one transfer at a time; this one starts
          // when p has ended (Eq. 13) and the channel's previous transfer is through (Eq. 14), lasts D^c (Eq. 11)
          int32_t* ch = chan_free + (size_t)(xp * D + j) * Ks + c;
          ep = max(ep, *ch) + gp.comm[(size_t)q * L + cl];
          *ch = ep;
        } else {
          ep += gp.comm[(size_t)q * L + cl];
        }
      }
      r = max(r, ep);
    }
    const int32_t d_i = gp.durm ? gp.durm[(size_t)i * D + j] : op.dur;   // D^o of i on its machine (Eq. 3)
    const int32_t s = max(r, free_at[j * T]);
    const int32_t e = s + d_i;
    free_at[j * T] = e;
    e_state[(size_t)i * Ks + c] = e;
    if (BY_POS) x_state[(size_t)i * Ks + c] = (uint8_t)j;
    busy[j * T] += d_i;
    const int32_t lv = lvl[j * T] + op.mem_delta;
    lvl[j * T] = lv;
    peak[j * T] = max(peak[j * T], lv);
    if (gp.weight) wsum[j * T] += gp.weight[i];
    z = max(z, e);
    const size_t at = (size_t)(by_op_times ? i : k) * Ks + c;
    if (out.start) out.start[at] = s;
    if (out.finish) out.finish[at] = e;
  }
  for (int j = 0; j < D; ++j) {
    const int32_t pk = peak[j * T] + wsum[j * T];  // the weights are resident from the start (Eq. 16)
    if (pk > gp.cap[j]) st |= PE_STATUS_MEM_EXCEEDED;
    if (out.busy) out.busy[(size_t)j * Ks + c] = busy[j * T];
    if (out.peak_mem) out.peak_mem[(size_t)j * Ks + c] = pk;
  }
  if (out.makespan) out.makespan[c] = z;
  if (out.status) out.status[c] = st;
}

// ============================================================================================
// Variant SHARED: one thread per candidate; the per-operator state (end time and machine,
// packed in one 32-bit word) lives in shared memory as [operator][thread], so a lane's
// gathers stay in its own bank.  The graph blob is staged into shared memory by bulk copy
// when it fits next to the state, otherwise read through the read-only cache.  Needs the
// graph's time bound below 2^24 - 256.
// ============================================================================================
template <typename OrderT, bool BY_POS, bool GRAPH_SMEM>
__global__ void pe_eval_shared_kernel(PeGraphView g, const uint8_t* __restrict__ blob, int64_t K,
                                      const uint8_t* __restrict__ assign, const OrderT* __restrict__ order,
                                      pe_outputs out, uint32_t flags, int* err) {
  extern __shared__ __align__(16) uint8_t smem_raw[];
  const int T = blockDim.x;
  const int t = threadIdx.x;
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
  uint32_t* state = reinterpret_cast<uint32_t*>(sm) + t;           // [V][T]
  int32_t* dev = reinterpret_cast<int32_t*>(sm) + (size_t)V * T + t;  // [5][D][T]
  int32_t* free_at = dev;
  int32_t* lvl = dev + (size_t)1 * D * T;
  int32_t* peak = dev + (size_t)2 * D * T;
  int32_t* busy = dev + (size_t)3 * D * T;
  int32_t* wsum = dev + (size_t)4 * D * T;

  const int64_t c = (int64_t)blockIdx.x * T + t;
  if (c >= K) return;
  const size_t Ks = (size_t)K;
  for (int i = 0; i < V; ++i) state[(size_t)i * T] = 0xFFFFFFFFu;
  for (int j = 0; j < D; ++j) {
    free_at[j * T] = 0; lvl[j * T] = 0; peak[j * T] = 0; busy[j * T] = 0;
    if (gp.weight) wsum[j * T] = 0;
  }
  const bool by_op_times = (flags & PE_TIMES_BY_OP) != 0;
  uint32_t st = 0;
  int32_t z = 0;

  // software prefetch: order entry two positions ahead, machine id one position ahead
  uint32_t o_cur = order[c];
  uint32_t o_nxt = V > 1 ? (uint32_t)order[Ks + c] : 0u;
  uint32_t a_cur = BY_POS ? assign[c] : assign[(size_t)min(o_cur, (uint32_t)(V - 1)) * Ks + c];
  for (int k = 0; k < V; ++k) {
    const uint32_t iu = o_cur;
    uint32_t jr = a_cur;
    o_cur = o_nxt;
    if (k + 2 < V) o_nxt = order[(size_t)(k + 2) * Ks + c];
    if (k + 1 < V) a_cur = BY_POS ? assign[(size_t)(k + 1) * Ks + c] : assign[(size_t)min(o_cur, (uint32_t)(V - 1)) * Ks + c];
    if (iu >= (uint32_t)V) { st |= PE_STATUS_ORDER_INVALID; continue; }
    const int i = (int)iu;
    if (jr >= (uint32_t)D) { st |= PE_STATUS_ASSIGN_RANGE; jr = D - 1; }
    const int j = (int)jr;
    const PeOpRec op = load_op(gp.ops, i);
    if (state_time(state[(size_t)i * T]) != kNotDoneTime) st |= PE_STATUS_ORDER_INVALID;
    int32_t r = 0;
    for (int q = op.edge_begin; q < op.edge_begin + op.indeg; ++q) {
      const int p = gp.pred[q];
      const uint32_t w = state[(size_t)p * T];
      if (state_time(w) == kNotDoneTime) { st |= PE_STATUS_ORDER_INVALID; continue; }
      int32_t ep = (int32_t)state_time(w);
      const int xp = (int)state_dev(w);
      if (xp != j) {
        const uint32_t cl = gp.cls[xp * D + j];
        if (cl == 0xFFu) st |= PE_STATUS_NO_CHANNEL;
        else ep += gp.comm[(size_t)q * L + cl];
      }
      r = max(r, ep);
    }
    const int32_t d_i = gp.durm ? gp.durm[(size_t)i * D + j] : op.dur;   // D^o of i on its machine (Eq. 3)
    const int32_t s = max(r, free_at[j * T]);
    const int32_t e = s + d_i;
    free_at[j * T] = e;
    state[(size_t)i * T] = pack_state((uint32_t)e, (uint32_t)j);
    busy[j * T] += d_i;
    const int32_t lv = lvl[j * T] + op.mem_delta;
    lvl[j * T] = lv;
    peak[j * T] = max(peak[j * T], lv);
    if (gp.weight) wsum[j * T] += gp.weight[i];
    z = max(z, e);
    const size_t at = (size_t)(by_op_times ? i : k) * Ks + c;
    if (out.start) out.start[at] = s;
    if (out.finish) out.finish[at] = e;
  }
  for (int j = 0; j < D; ++j) {
    const int32_t pk = peak[j * T] + (gp.weight ? wsum[j * T] : 0);
    if (pk > gp.cap[j]) st |= PE_STATUS_MEM_EXCEEDED;
    if (out.busy) out.busy[(size_t)j * Ks + c] = busy[j * T];
    if (out.peak_mem) out.peak_mem[(size_t)j * Ks + c] = pk;
  }
  if (out.makespan) out.makespan[c] = z;
  if (out.status) out.status[c] = st;
}

// ============================================================================================
// Host-side planning: which variant, with what launch shape.
// ============================================================================================

static inline size_t round_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// exclusive: PE_COMM_EXCLUSIVE - the compact kernel keeps one more word per machine pair and candidate;
// the generic shared-state kernel does not offer it.
static bool plan_shared(const pe_graph* g, bool allow_compact, Plan* p, bool exclusive = false) {
  if (g->time_bound >= kPackedTimeLimit) return false;
  p->compact = false;
  p->exclusive = exclusive;
  if (g->narrow_ok && allow_compact) {  // compact graph staged in shared memory next to the state
    const size_t fixed = (size_t)g->nview.bytes + 16;
    // 16-bit state words when the machine id and every possible end time fit together (the all-ones time
    // field marks "not scheduled"): half the state, so twice the candidates per SM where the state is what
    // limits them.  Blocks are multiples of 64 threads there (two warps share the words of a row).
    int jb = 1;
    while ((1 << jb) < g->D) ++jb;
    if (!exclusive && jb < 16 && g->time_bound < ((int64_t)1 << (16 - jb)) - 1) {
      const size_t per16 = (size_t)2 * (g->V + 1) + (size_t)(g->has_weight ? 20 : 16) * g->D;
      if (fixed + 64 * per16 <= g->smem_optin) {
        size_t T = (g->smem_optin - fixed) / per16 / 64 * 64;
        if (T > 256) T = 256;
        p->variant = PE_VARIANT_SHARED;
        p->threads = (int)T;
        p->smem = fixed + T * per16;
        p->graph_smem = true;
        p->workspace = 0;
        p->ws_x_off = 0;
        p->compact = true;
        p->state16 = true;
        p->jbits = jb;
        return true;
      }
    }
    const size_t per = (size_t)4 * (g->V + 1) + (size_t)(g->has_weight ? 20 : 16) * g->D +
                       (exclusive ? (size_t)4 * g->D * g->D : 0);
    if (fixed + 32 * per <= g->smem_optin) {
      // A block size that is a multiple of 32 keeps every lane's state column in its own bank.  That is
      // given up only where rounding down would idle more than a sixth of the candidates that fit:
      // with one or two warps per SM the kernel is bound by latency, not by bank conflicts.
      size_t T = (g->smem_optin - fixed) / per;
      if (T > 256) T = 256;
      if (T / 32 * 32 * 6 >= T * 5) T = T / 32 * 32;
      p->variant = PE_VARIANT_SHARED;
      p->threads = (int)T;
      p->smem = fixed + T * per;
      p->graph_smem = true;
      p->workspace = 0;
      p->ws_x_off = 0;
      p->compact = true;
      return true;
    }
  }
  if (exclusive) return false;
  const size_t per_thread = (size_t)4 * g->V + (size_t)(g->has_weight ? 20 : 16) * g->D;
  const size_t budget = g->smem_optin;
  for (int with_graph = 1; with_graph >= 0; --with_graph) {
    const size_t fixed = with_graph ? (size_t)g->lay.bytes + 16 : 0;
    if (fixed + 32 * per_thread > budget) continue;
    size_t T = (budget - fixed) / per_thread / 32 * 32;
    if (T > 256) T = 256;
    p->variant = PE_VARIANT_SHARED;
    p->threads = (int)T;
    p->smem = fixed + T * per_thread;
    p->graph_smem = with_graph != 0;
    p->workspace = 0;
    p->ws_x_off = 0;
    return true;
  }
  return false;
}

static bool plan_warp(const pe_graph* g, int64_t K, uint32_t flags, bool allow_compact, Plan* p) {
  if (g->time_bound >= kPackedTimeLimit) return false;
  const bool compact = g->narrow_ok && allow_compact;
  p->compact = compact;
  p->slab = false;
  size_t words = (size_t)(g->V + 2) + (size_t)5 * g->D;
  words |= 1;  // odd stride between candidates: the initial fill hits distinct banks
  const size_t per_warp = words * 4;
  const size_t budget = g->smem_optin;
  const size_t blob_bytes = compact ? g->nview.bytes : g->lay.bytes;
  const bool by_pos = (flags & PE_ASSIGN_BY_POS) != 0;
  // shared tiles of the slab mode for n warps (see pe_kernel_warp2.cuh): order entries (two buffers),
  // by-position machine ids (two buffers), start and end times
  auto slab_bytes = [&](size_t n) -> size_t {
    const size_t rows = 128;
    return 2 * rows * (n + 2) * 2 + (by_pos ? ((2 * rows * (n + 4) + 3) & ~(size_t)3) : 0) + 2 * rows * (n + 1) * 4;
  };
  auto fit = [&](size_t fixed, bool slab) -> int {
    for (size_t n = 32; n >= 1; --n)
      if (fixed + n * per_warp + (slab ? slab_bytes(n) : 0) <= budget) return (int)n;
    return 0;
  };
  const int n_global = fit(0, false);
  const int n_staged = fit(blob_bytes + 16, false);
  if (n_global < 1) return false;
  bool staged = n_staged >= (n_global < 8 ? n_global : 8);
  int n = staged ? n_staged : n_global;
  // Slab mode (rows read and written contiguously through shared tiles, at the price of a block
  // barrier per 128 positions) pays off when the rows are long: with K beyond 2^19 the 32 lanes of a
  // window touch 32 different 2 MiB pages per array, and measured throughput of the per-lane path
  // drops by 40 %.  It needs a block wide enough to fill memory sectors.
  if (compact && K >= ((int64_t)1 << 19)) {
    const int ns = fit(staged ? blob_bytes + 16 : 0, true);
    if (ns >= 16) { p->slab = true; n = ns; }
  }
  p->variant = PE_VARIANT_WARP;
  p->threads = 32 * n;
  p->smem = (staged ? blob_bytes + 16 : 0) + (size_t)n * per_warp + (p->slab ? slab_bytes((size_t)n) : 0);
  p->graph_smem = staged;
  p->workspace = 0;
  p->ws_x_off = 0;
  p->warp_words = (int)words;
  return true;
}

// TEAM: one block per candidate; plan.threads / 32 warps share the candidate's windows.  With K a multiple of 4
// (the transpositions move 32-bit words) the inputs and the times go through candidate-major staging copies
// in the workspace, a chunk of candidates at a time; a chunk is sixteen times what the GPU holds at once.
static bool plan_team(const pe_graph* g, int64_t K, bool allow_compact, Plan* p) {
  if (!g->narrow_ok || !allow_compact || g->max_indeg > 8 || g->time_bound >= (int64_t)1 << 23) return false;
  const size_t smem = round_up((size_t)4 * (g->V + 2) + (size_t)4 * (5 * g->D + 2), 16);
  if (smem > g->smem_optin) return false;
  // Blocks an SM holds by shared memory decide the warps per block.  Few large blocks: six warps, so that the
  // set-up of five windows hides behind the serial part of one.  Many small blocks: two warps each - a block
  // reserves two named barriers per warp, an SM has 64 of them, and more chains beat deeper pipelines there
  // (measured at V = 4096 / D = 64: 4.46e10 with two warps, 4.36e10 with four, 3.3e10 with six; the MoE graph:
  // 2.03e10 against 1.96e10 and 1.63e10).
  size_t per_sm = (g->smem_per_sm ? g->smem_per_sm : g->smem_optin) / (smem + 1024);
  if (per_sm < 1) per_sm = 1;
  const int nw = per_sm <= 4 ? 6 : (per_sm <= 7 ? 4 : 2);
  const size_t by_barriers = (size_t)64 / (nw == 6 ? 16 : 2 * nw + 1);
  if (per_sm > by_barriers) per_sm = by_barriers;
  if (per_sm * nw * 32 > 2048) per_sm = 2048 / (nw * 32);
  p->variant = PE_VARIANT_TEAM;
  p->threads = 32 * nw;
  p->smem = smem;
  p->graph_smem = false;
  p->workspace = 0;
  p->ws_x_off = 0;
  p->compact = true;
  p->staged = K >= 64 && K % 4 == 0;
  if (p->staged) {
    // a chunk is eight times what the GPU holds at once (measured at V = 16384: 4, 8 and 16 times are
    // within 2 % of each other; two chunks are in flight)
    int64_t chunk = (int64_t)per_sm * g->sm_count * 8 / 4 * 4;
    if (chunk > K) chunk = K;
    p->team_chunk = chunk;
    p->team_vp = ((int64_t)g->V + 63) / 64 * 64;
    const size_t cells = (size_t)chunk * (size_t)p->team_vp;
    size_t at = 0;
    p->team_off_order = at;  at = round_up(at + cells * 2, 256);
    p->team_off_assign = at; at = round_up(at + cells, 256);
    p->team_off_start = at;  at = round_up(at + cells * 4, 256);
    p->team_off_finish = at; at = round_up(at + cells * 4, 256);
    p->team_half = at;
    p->workspace = chunk < K ? 2 * at : at;
  }
  return true;
}

static bool plan_global(const pe_graph* g, int64_t K, uint32_t flags, bool allow_compact, Plan* p) {
  p->compact = false;
  const bool exclusive = (flags & PE_COMM_EXCLUSIVE) != 0;
  p->exclusive = exclusive;
  if (g->narrow_ok && allow_compact && g->time_bound < kPackedTimeLimit) {
    // compact-graph kernel with the state in the workspace.  Per-machine records stay in shared
    // memory while a 128-thread block needs at most 16 KB for them; beyond that they would cap the
    // resident candidates, so they move to the workspace too (tiles that stay in L2).
    const size_t per = (size_t)(g->has_weight ? 20 : 16) * g->D;
    const size_t tiles = (size_t)((K + 31) / 32);
    const size_t state_bytes = round_up((size_t)(g->V + 1) * tiles * 32 * 4, 256);
    p->variant = PE_VARIANT_GLOBAL;
    p->threads = 128;
    p->graph_smem = false;
    p->compact = true;
    if (128 * per <= 16384) {
      p->smem = 128 * per;
      p->ws_x_off = 0;
      p->workspace = state_bytes;
    } else {
      p->smem = 0;
      p->ws_x_off = state_bytes;  // offset of the per-machine records
      p->workspace = state_bytes + round_up(tiles * 32 * per, 256);
    }
    p->ws_c_off = p->workspace;   // PE_COMM_EXCLUSIVE: end of the last transfer per channel, tiles [tile][D*D][32]
    if (exclusive) p->workspace += round_up(tiles * 32 * (size_t)g->D * g->D * 4, 256);
    return true;
  }
  const size_t per_thread = (size_t)20 * g->D;
  size_t T = g->smem_optin / per_thread / 32 * 32;
  if (T > 128) T = 128;
  if (T < 32) return false;
  p->variant = PE_VARIANT_GLOBAL;
  p->threads = (int)T;
  p->smem = T * per_thread;
  p->graph_smem = false;
  p->ws_x_off = round_up((size_t)g->V * (size_t)K * 4, 256);
  p->workspace = p->ws_x_off + ((flags & PE_ASSIGN_BY_POS) ? round_up((size_t)g->V * (size_t)K, 256) : 0);
  p->ws_c_off = p->workspace;   // PE_COMM_EXCLUSIVE: end of the last transfer per channel, [D*D][K]
  if (exclusive) p->workspace += round_up((size_t)g->D * g->D * (size_t)K * 4, 256);
  return true;
}

// allow_compact: the call can use the compact-graph kernels (u16 orders; start and finish both
// wanted or both absent).  Size queries pass true and false and take the larger workspace.
static int make_plan(const pe_graph* g, int64_t K, uint32_t flags, bool allow_compact, Plan* p) {
  if (!g || K < 0) return PE_ERR_INVALID_ARG;
  if (flags & ~(uint32_t)(PE_ASSIGN_BY_POS | PE_TIMES_BY_OP | PE_COMM_EXCLUSIVE | PE_VARIANT_MASK)) return PE_ERR_INVALID_ARG;
  *p = Plan();
  const uint32_t want = flags & PE_VARIANT_MASK;
  if (g->hetero) {   // machine-dependent durations: the generic one-thread-per-candidate kernels
    if (want == PE_VARIANT_WARP || want == PE_VARIANT_TEAM) return PE_ERR_UNSUPPORTED;
    if (!(flags & PE_COMM_EXCLUSIVE) && want != PE_VARIANT_GLOBAL && plan_shared(g, false, p) &&
        (p->threads >= 48 || want == PE_VARIANT_SHARED))
      return PE_OK;
    if (want == PE_VARIANT_SHARED) return PE_ERR_UNSUPPORTED;
    return plan_global(g, K, flags, false, p) ? PE_OK : PE_ERR_UNSUPPORTED;
  }
  if (flags & PE_COMM_EXCLUSIVE) {
    // exclusive channels: the compact shared-state kernel where a block of candidates still fits with one
    // more word per machine pair each, else the generic global-state kernel
    if (want == PE_VARIANT_AUTO || want == PE_VARIANT_SHARED) {
      if (plan_shared(g, allow_compact, p, true) && (p->threads >= 48 || want == PE_VARIANT_SHARED)) return PE_OK;
      if (want == PE_VARIANT_SHARED) return PE_ERR_UNSUPPORTED;
      *p = Plan();
    }
    if (want != PE_VARIANT_AUTO && want != PE_VARIANT_GLOBAL) return PE_ERR_UNSUPPORTED;
    return plan_global(g, K, flags, allow_compact, p) ? PE_OK : PE_ERR_UNSUPPORTED;
  }
  switch (want) {
    case PE_VARIANT_AUTO: {
      // Thread-per-candidate with everything on chip wins whenever about a warp and a half of
      // candidates fit in shared memory (measured: 55 candidates per SM at V = 1024 beat the
      // warp-per-candidate kernel by 1.35x, 44 did not).  Beyond that the state of a candidate is too
      // large: a warp per candidate (state still on chip) wins while at least four warps fit on an SM;
      // for the largest graphs the global-state kernel, which is bound by random DRAM accesses but
      // keeps thousands of candidates in flight, is faster.
      if (plan_shared(g, allow_compact, p) && p->threads >= 48) return PE_OK;
      Plan w, gl, tm;
      const bool has_w = plan_warp(g, K, flags, allow_compact, &w);
      const bool has_g = plan_global(g, K, flags, allow_compact, &gl);
      // Once fewer than about twenty single-warp candidates fit on an SM, a block of warps per candidate
      // is faster (measured at V = 4096: 3.6e10 against 2.6e10 operator-evaluations/s at D = 64, 2.7e10
      // against 2.0e10 at D = 8; at V = 16384: 3.1e10 against 1.0e10 (warp) and 2.3e10 against 1.25e10
      // (global); at V = 1024 the single-warp kernel still wins, 4.0e10 against 3.0e10).
      // Graphs with operators of more than three incoming edges take the single-warp kernel off its register
      // slots; there the block of warps wins as well (measured on the MoE graph: 1.7e10 against 0.9e10).
      if (plan_team(g, K, allow_compact, &tm) && (!has_w || w.threads < 20 * 32 || (g->max_indeg > 3 && w.threads < 24 * 32))) {
        *p = tm;
        return PE_OK;
      }
      // With three warps per SM the two are close; the global-state kernel loses once it has to keep the
      // per-machine records in the workspace as well (measured at V = 16384: 1.25e10 against 0.84e10
      // operator-evaluations/s at D = 8, 0.93e10 against 1.01e10 at D = 64).
      const bool warp_wins = w.threads >= 4 * 32 || (w.threads >= 3 * 32 && has_g && gl.smem == 0);
      if (has_w && (warp_wins || !has_g || !gl.compact)) { *p = w; return PE_OK; }
      if (has_g && gl.compact) { *p = gl; return PE_OK; }
      if (plan_shared(g, allow_compact, p)) return PE_OK;
      if (has_w) { *p = w; return PE_OK; }
      if (has_g) { *p = gl; return PE_OK; }
      return PE_ERR_UNSUPPORTED;
    }
    case PE_VARIANT_GLOBAL: return plan_global(g, K, flags, allow_compact, p) ? PE_OK : PE_ERR_UNSUPPORTED;
    case PE_VARIANT_SHARED: return plan_shared(g, allow_compact, p) ? PE_OK : PE_ERR_UNSUPPORTED;
    case PE_VARIANT_WARP: return plan_warp(g, K, flags, allow_compact, p) ? PE_OK : PE_ERR_UNSUPPORTED;
    case PE_VARIANT_TEAM: return plan_team(g, K, allow_compact, p) ? PE_OK : PE_ERR_UNSUPPORTED;
    default: return PE_ERR_UNSUPPORTED;
  }
}


template <typename OrderT, bool BY_POS>
static int launch_typed(const pe_graph* g, const Plan& p, int64_t K, const uint8_t* assign, const void* order,
                        uint32_t flags, const pe_outputs& out, void* workspace, cudaStream_t stream) {
  const PeGraphView view = pe_view(g);
  const int per_block = p.variant == PE_VARIANT_TEAM ? 1 : (p.variant == PE_VARIANT_WARP ? p.threads / 32 : p.threads);  // candidates per block
  const unsigned grid = (unsigned)((K + per_block - 1) / per_block);
  const OrderT* ord = static_cast<const OrderT*>(order);
  if (p.compact) {
    if (sizeof(OrderT) != 2) return PE_ERR_INVALID_ARG;
    const uint16_t* ord16 = static_cast<const uint16_t*>(order);
    uint32_t* gstate = static_cast<uint32_t*>(workspace);
    if (p.variant == PE_VARIANT_TEAM) {
      if (p.staged && (((uintptr_t)assign | (uintptr_t)order) & 3u)) return PE_ERR_INVALID_ARG;   // word-wise transpositions
      int64_t n = 0;
      const int rc = launch_team(g, p, BY_POS, K, assign, ord16, flags, out, workspace, stream, &n);
      if (rc != PE_OK) return rc;
      g_launches.fetch_add(n, std::memory_order_relaxed);
      return cudaGetLastError() == cudaSuccess ? PE_OK : PE_ERR_CUDA;
    }
    const int rc = p.variant == PE_VARIANT_WARP ? launch_warp2(g, p, BY_POS, K, assign, ord16, flags, out, grid, stream)
                                                : launch_lane(g, p, BY_POS, K, assign, ord16, flags, out, gstate, grid, stream);
    if (rc != PE_OK) return rc;
  } else if (p.variant == PE_VARIANT_GLOBAL) {
    int32_t* e_state = static_cast<int32_t*>(workspace);
    uint8_t* x_state = static_cast<uint8_t*>(workspace) + p.ws_x_off;
    if (cudaMemsetAsync(e_state, 0xFF, (size_t)g->V * (size_t)K * 4, stream) != cudaSuccess) return PE_ERR_CUDA;
    int32_t* chan_free = nullptr;
    if (flags & PE_COMM_EXCLUSIVE) {
      chan_free = reinterpret_cast<int32_t*>(static_cast<uint8_t*>(workspace) + p.ws_c_off);
      if (cudaMemsetAsync(chan_free, 0, (size_t)g->D * g->D * (size_t)K * 4, stream) != cudaSuccess) return PE_ERR_CUDA;
    }
    auto kern = pe_eval_global_kernel<OrderT, BY_POS>;
    if (!set_smem(kern, p.smem)) return PE_ERR_CUDA;
    kern<<<grid, p.threads, p.smem, stream>>>(view, g->d_blob, K, assign, ord, out, flags, e_state, x_state, chan_free);
  } else if (p.variant == PE_VARIANT_SHARED) {
    if (p.graph_smem) {
      auto kern = pe_eval_shared_kernel<OrderT, BY_POS, true>;
      if (!set_smem(kern, p.smem)) return PE_ERR_CUDA;
      kern<<<grid, p.threads, p.smem, stream>>>(view, g->d_blob, K, assign, ord, out, flags, g->d_error);
    } else {
      auto kern = pe_eval_shared_kernel<OrderT, BY_POS, false>;
      if (!set_smem(kern, p.smem)) return PE_ERR_CUDA;
      kern<<<grid, p.threads, p.smem, stream>>>(view, g->d_blob, K, assign, ord, out, flags, g->d_error);
    }
  } else if (p.variant == PE_VARIANT_WARP) {
    if (p.graph_smem) {
      auto kern = pe_eval_warp_kernel<OrderT, BY_POS, true>;
      if (!set_smem(kern, p.smem)) return PE_ERR_CUDA;
      kern<<<grid, p.threads, p.smem, stream>>>(view, g->d_blob, K, assign, ord, out, flags, g->d_error, p.warp_words);
    } else {
      auto kern = pe_eval_warp_kernel<OrderT, BY_POS, false>;
      if (!set_smem(kern, p.smem)) return PE_ERR_CUDA;
      kern<<<grid, p.threads, p.smem, stream>>>(view, g->d_blob, K, assign, ord, out, flags, g->d_error, p.warp_words);
    }
  } else {
    return PE_ERR_UNSUPPORTED;
  }
  g_launches.fetch_add(1, std::memory_order_relaxed);
  return cudaGetLastError() == cudaSuccess ? PE_OK : PE_ERR_CUDA;
}

}  // namespace pe

extern "C" size_t pe_workspace_bytes(const pe_graph* g, int64_t K, uint32_t flags) {
  pe::Plan a, b;
  const size_t wa = pe::make_plan(g, K, flags, true, &a) == PE_OK ? a.workspace : 0;
  const size_t wb = pe::make_plan(g, K, flags, false, &b) == PE_OK ? b.workspace : 0;
  return wa > wb ? wa : wb;
}

extern "C" int pe_eval_variant(const pe_graph* g, int64_t K, uint32_t flags) {
  pe::Plan p;
  const int rc = pe::make_plan(g, K, flags, true, &p);
  return rc != PE_OK ? rc : p.variant;
}

namespace pe { extern std::atomic<int64_t> g_decode_launches; }
extern "C" int64_t pe_kernel_launches(void) {
  return pe::g_launches.load(std::memory_order_relaxed) + pe::g_decode_launches.load(std::memory_order_relaxed);
}

extern "C" int pe_eval_batch(pe_graph* g, int64_t K, const uint8_t* assign, const void* order, int order_bytes,
                             uint32_t flags, const pe_outputs* out, void* workspace, size_t workspace_bytes,
                             void* cuda_stream) {
  if (!g || !out || K < 0) return PE_ERR_INVALID_ARG;
  if (order_bytes != 2 && order_bytes != 4) return PE_ERR_INVALID_ARG;
  if (order_bytes == 2 && g->V > 65536) return PE_ERR_INVALID_ARG;
  pe::Plan p;
  const bool allow_compact = order_bytes == 2 && ((out->start != nullptr) == (out->finish != nullptr));
  const int rc = pe::make_plan(g, K, flags, allow_compact, &p);
  if (rc != PE_OK) return rc;
  if (K == 0) return PE_OK;
  if (!assign || !order) return PE_ERR_INVALID_ARG;
  if ((K + p.threads - 1) / p.threads > (int64_t)INT_MAX) return PE_ERR_INVALID_ARG;
  if (p.workspace > 0 && (!workspace || workspace_bytes < p.workspace)) return PE_ERR_WORKSPACE;
  int prev = -1;
  if (cudaGetDevice(&prev) != cudaSuccess) return PE_ERR_CUDA;
  if (prev != g->device && cudaSetDevice(g->device) != cudaSuccess) return PE_ERR_CUDA;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  const bool by_pos = (flags & PE_ASSIGN_BY_POS) != 0;
  int ret;
  if (order_bytes == 2)
    ret = by_pos ? pe::launch_typed<uint16_t, true>(g, p, K, assign, order, flags, *out, workspace, stream)
                 : pe::launch_typed<uint16_t, false>(g, p, K, assign, order, flags, *out, workspace, stream);
  else
    ret = by_pos ? pe::launch_typed<uint32_t, true>(g, p, K, assign, order, flags, *out, workspace, stream)
                 : pe::launch_typed<uint32_t, false>(g, p, K, assign, order, flags, *out, workspace, stream);
  if (prev != g->device) cudaSetDevice(prev);
  return ret;
}

extern "C" int pe_eval_batch_host(pe_graph* g, int64_t K, const uint8_t* host_assign, const void* host_order,
                                  int order_bytes, uint32_t flags, const pe_outputs* host_out, uint8_t* dev_assign,
                                  void* dev_order, const pe_outputs* dev_out, void* workspace, size_t workspace_bytes,
                                  void* cuda_stream) {
  if (!g || !host_out || !dev_out || K < 0) return PE_ERR_INVALID_ARG;
  if (order_bytes != 2 && order_bytes != 4) return PE_ERR_INVALID_ARG;
  if (K == 0) return PE_OK;
  if (!host_assign || !host_order || !dev_assign || !dev_order) return PE_ERR_INVALID_ARG;
  // every output wanted on the host needs its device staging buffer
  if ((host_out->start && !dev_out->start) || (host_out->finish && !dev_out->finish) ||
      (host_out->makespan && !dev_out->makespan) || (host_out->busy && !dev_out->busy) ||
      (host_out->peak_mem && !dev_out->peak_mem) || (host_out->status && !dev_out->status))
    return PE_ERR_INVALID_ARG;
  int prev = -1;
  if (cudaGetDevice(&prev) != cudaSuccess) return PE_ERR_CUDA;
  if (prev != g->device && cudaSetDevice(g->device) != cudaSuccess) return PE_ERR_CUDA;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  const size_t V = (size_t)g->V, D = (size_t)g->D, Ks = (size_t)K, ob = (size_t)order_bytes;
  pe_outputs want = *dev_out;  // compute only what the host asked for
  if (!host_out->start) want.start = nullptr;
  if (!host_out->finish) want.finish = nullptr;
  if (!host_out->makespan) want.makespan = nullptr;
  if (!host_out->busy) want.busy = nullptr;
  if (!host_out->peak_mem) want.peak_mem = nullptr;
  if (!host_out->status) want.status = nullptr;

  // The batch is cut into chunks of candidates.  Chunk q's inputs go up on the graph's copy-in
  // stream, its kernel runs on the caller's stream, its outputs come down on the copy-out stream,
  // so the uploads, the kernels and the downloads of different chunks overlap (the two copy
  // directions use separate DMA engines).  A chunk of Kc candidates lives in the staging buffers
  // as a dense [rows][Kc] block at element offset rows * first; the strided host side is handled
  // by 2-D copies.
  // (measured on the default workload: 16 chunks 6.1e9, 8 chunks 5.8e9, 4 chunks 5.3e9 operator-evaluations/s
  // end to end - shorter chunks shorten the ramp before the first download and after the last upload)
  int nchunks = K >= 16 * 4096 ? 16 : (K >= 8 * 4096 ? 8 : 1);
  const int64_t per = ((K + nchunks - 1) / nchunks + 255) / 256 * 256;
  nchunks = (int)((K + per - 1) / per);
  std::lock_guard<std::mutex> lock(g->host_mutex);
  int ret = PE_OK;
  auto ok = [&](cudaError_t e) { if (e != cudaSuccess && ret == PE_OK) ret = PE_ERR_CUDA; };
  ok(cudaEventRecord(g->ev_begin, stream));           // copies start after the caller's earlier work
  ok(cudaStreamWaitEvent(g->copy_in, g->ev_begin, 0));
  ok(cudaStreamWaitEvent(g->copy_out, g->ev_begin, 0));
  for (int q = 0; q < nchunks && ret == PE_OK; ++q) {
    const size_t first = (size_t)q * (size_t)per;
    const size_t Kc = (size_t)(K - (int64_t)first < per ? K - (int64_t)first : per);
    uint8_t* d_as = dev_assign + V * first;
    uint8_t* d_or = static_cast<uint8_t*>(dev_order) + V * first * ob;
    ok(cudaMemcpy2DAsync(d_as, Kc, host_assign + first, Ks, Kc, V, cudaMemcpyHostToDevice, g->copy_in));
    ok(cudaMemcpy2DAsync(d_or, Kc * ob, static_cast<const uint8_t*>(host_order) + first * ob, Ks * ob, Kc * ob, V,
                         cudaMemcpyHostToDevice, g->copy_in));
    ok(cudaEventRecord(g->ev_in[q], g->copy_in));
    ok(cudaStreamWaitEvent(stream, g->ev_in[q], 0));
    pe_outputs run;
    run.start = want.start ? want.start + V * first : nullptr;
    run.finish = want.finish ? want.finish + V * first : nullptr;
    run.makespan = want.makespan ? want.makespan + first : nullptr;
    run.busy = want.busy ? want.busy + D * first : nullptr;
    run.peak_mem = want.peak_mem ? want.peak_mem + D * first : nullptr;
    run.status = want.status ? want.status + first : nullptr;
    if (ret == PE_OK)
      ret = pe_eval_batch(g, (int64_t)Kc, d_as, d_or, order_bytes, flags, &run, workspace, workspace_bytes, cuda_stream);
    ok(cudaEventRecord(g->ev_done[q], stream));
    ok(cudaStreamWaitEvent(g->copy_out, g->ev_done[q], 0));
    auto back = [&](void* h, const void* d, size_t rows, size_t elem) {  // [rows][Kc] block -> columns first.. of [rows][K]
      if (h && ret == PE_OK)
        ok(cudaMemcpy2DAsync(static_cast<uint8_t*>(h) + first * elem, Ks * elem, d, Kc * elem, Kc * elem, rows,
                             cudaMemcpyDeviceToHost, g->copy_out));
    };
    back(host_out->start, run.start, V, 4);
    back(host_out->finish, run.finish, V, 4);
    back(host_out->makespan, run.makespan, 1, 4);
    back(host_out->busy, run.busy, D, 4);
    back(host_out->peak_mem, run.peak_mem, D, 4);
    back(host_out->status, run.status, 1, 4);
  }
  ok(cudaEventRecord(g->ev_end, g->copy_out));
  ok(cudaStreamWaitEvent(stream, g->ev_end, 0));
  if (cudaStreamSynchronize(stream) != cudaSuccess && ret == PE_OK) ret = PE_ERR_CUDA;
  if (ret != PE_OK) {  // leave nothing of this call running on the graph's own streams
    cudaStreamSynchronize(g->copy_in);
    cudaStreamSynchronize(g->copy_out);
    cudaGetLastError();
  }
  if (prev != g->device) cudaSetDevice(prev);
  return ret;
}

// ============================================================================================
// pe_eval_batch_noalloc: the GLOBAL variant with its scratch in an array that is part of the
// library image, for callers that may not allocate device memory.
// ============================================================================================
namespace pe {

// The scratch itself.  In host code this name is only a handle for the runtime's symbol
// lookup, never a device address: the address kernels and memsets need comes from
// cudaGetSymbolAddress, looked up once per device below.
static __device__ __align__(256) uint8_t g_noalloc_scratch[PE_NOALLOC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
static std::atomic<void*> g_noalloc_addr[kMaxDevices];

// Device address of the scratch array on `device`, which must be the current device.
static int noalloc_scratch_address(int device, void** out) {
  if (device < 0 || device >= kMaxDevices) return PE_ERR_INVALID_ARG;
  void* p = g_noalloc_addr[device].load(std::memory_order_acquire);
  if (!p) {
    if (cudaGetSymbolAddress(&p, g_noalloc_scratch) != cudaSuccess || !p) {
      cudaGetLastError();
      return PE_ERR_CUDA;
    }
    g_noalloc_addr[device].store(p, std::memory_order_release);  // every thread resolves the same address
  }
  *out = p;
  return PE_OK;
}

}  // namespace pe

extern "C" int pe_eval_batch_noalloc(pe_graph* g, int64_t K, const uint8_t* assign, const void* order, int order_bytes,
                                     uint32_t flags, const pe_outputs* out, void* cuda_stream) {
  if (!g || !out || K < 0) return PE_ERR_INVALID_ARG;
  if (order_bytes != 2 && order_bytes != 4) return PE_ERR_INVALID_ARG;
  if (order_bytes == 2 && g->V > 65536) return PE_ERR_INVALID_ARG;
  if (flags & ~(uint32_t)(PE_ASSIGN_BY_POS | PE_TIMES_BY_OP)) return PE_ERR_INVALID_ARG;
  pe::Plan p;
  const bool allow_compact = order_bytes == 2 && ((out->start != nullptr) == (out->finish != nullptr));
  if (!pe::plan_global(g, K, flags, allow_compact, &p)) return PE_ERR_UNSUPPORTED;
  if (p.workspace > (size_t)PE_NOALLOC_SCRATCH_BYTES) return PE_ERR_SCRATCH_LIMIT;
  if (K == 0) return PE_OK;
  if (!assign || !order) return PE_ERR_INVALID_ARG;
  if ((K + p.threads - 1) / p.threads > (int64_t)INT_MAX) return PE_ERR_INVALID_ARG;
  int prev = -1;
  if (cudaGetDevice(&prev) != cudaSuccess) return PE_ERR_CUDA;
  if (prev != g->device && cudaSetDevice(g->device) != cudaSuccess) return PE_ERR_CUDA;
  void* scratch = nullptr;
  int ret = pe::noalloc_scratch_address(g->device, &scratch);
  if (ret == PE_OK) {
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const bool by_pos = (flags & PE_ASSIGN_BY_POS) != 0;
    // whatever the previous call left in the array never matters: the generic kernel's end times are
    // cleared by a memset that launch_typed puts on the stream before the kernel, and the compact kernel
    // writes every state word ("not scheduled") and per-machine record itself before it reads any
    if (order_bytes == 2)
      ret = by_pos ? pe::launch_typed<uint16_t, true>(g, p, K, assign, order, flags, *out, scratch, stream)
                   : pe::launch_typed<uint16_t, false>(g, p, K, assign, order, flags, *out, scratch, stream);
    else
      ret = by_pos ? pe::launch_typed<uint32_t, true>(g, p, K, assign, order, flags, *out, scratch, stream)
                   : pe::launch_typed<uint32_t, false>(g, p, K, assign, order, flags, *out, scratch, stream);
  }
  if (prev != g->device) cudaSetDevice(prev);
  return ret;
}
