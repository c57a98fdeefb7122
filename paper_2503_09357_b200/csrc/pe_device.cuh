// Device helpers shared by the evaluation kernels: graph accessors, bulk-copy staging of
// the graph blob into shared memory, packed state words.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "pe_graph.h"

namespace pe {

// ---- graph accessors over a blob base pointer (global or shared) ----
struct GraphPtrs {
  const PeOpRec* ops;
  const int32_t* pred;
  const int32_t* comm;
  const int32_t* weight;  // nullptr when the graph has no W
  const uint8_t* cls;
  const int32_t* cap;
  const int32_t* durm;    // nullptr unless durations depend on the machine
};

__device__ __forceinline__ GraphPtrs graph_ptrs(const uint8_t* base, const PeGraphView& g) {
  GraphPtrs p;
  p.ops = reinterpret_cast<const PeOpRec*>(base + g.lay.ops);
  p.pred = reinterpret_cast<const int32_t*>(base + g.lay.pred);
  p.comm = reinterpret_cast<const int32_t*>(base + g.lay.comm);
  p.weight = g.has_weight ? reinterpret_cast<const int32_t*>(base + g.lay.weight) : nullptr;
  p.cls = base + g.lay.cls;
  p.cap = reinterpret_cast<const int32_t*>(base + g.lay.cap);
  p.durm = g.hetero ? reinterpret_cast<const int32_t*>(base + g.lay.durm) : nullptr;
  return p;
}

__device__ __forceinline__ PeOpRec load_op(const PeOpRec* ops, int32_t i) {
  const int4 v = *reinterpret_cast<const int4*>(ops + i);
  PeOpRec r;
  r.edge_begin = v.x; r.indeg = v.y; r.dur = v.z; r.mem_delta = v.w;
  return r;
}

// ---- accessors over the compact encoding (PeNarrowView) ----
struct NarrowPtrs {
  const uint4* ops;
  const uint32_t* edges;
  const int32_t* weight;
  const uint8_t* cls;
  const int32_t* cap;
};

__device__ __forceinline__ NarrowPtrs narrow_ptrs(const uint8_t* base, const PeNarrowView& g) {
  NarrowPtrs p;
  p.ops = reinterpret_cast<const uint4*>(base + g.ops);
  p.edges = reinterpret_cast<const uint32_t*>(base + g.edges);
  p.weight = g.has_weight ? reinterpret_cast<const int32_t*>(base + g.weight) : nullptr;
  p.cls = base + g.cls;
  p.cap = reinterpret_cast<const int32_t*>(base + g.cap);
  return p;
}

// ---- packed per-operator state: end time in the high 24 bits, machine in the low 8 ----
// Used when the graph's time bound is below kPackedTimeLimit.  kNotDone marks an operator
// that has not been scheduled yet (its machine byte is still valid).
constexpr uint32_t kNotDoneTime = 0xFFFFFFu;
constexpr int64_t kPackedTimeLimit = 0xFFFF00;  // times must stay below the marker range
__device__ __forceinline__ uint32_t pack_state(uint32_t t, uint32_t dev) { return (t << 8) | dev; }
__device__ __forceinline__ uint32_t state_time(uint32_t w) { return w >> 8; }
__device__ __forceinline__ uint32_t state_dev(uint32_t w) { return w & 0xFFu; }

// ---- mbarrier + bulk copy (TMA, 1-D, CTA-local, never multicast) ----
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
__device__ __forceinline__ void bulk_g2s(void* dst, const void* src, uint32_t bytes, uint64_t* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                   smem_u32(dst)),
               "l"(src), "r"(bytes), "r"(smem_u32(bar))
               : "memory");
}

// Bounded wait: gives up after kWaitLimit polls (each poll may itself block for a short,
// hardware-defined time) and reports it instead of spinning for ever.
constexpr int kWaitLimit = 1 << 20;
__device__ __forceinline__ bool mbar_wait_bounded(uint64_t* bar, uint32_t parity, int limit = kWaitLimit) {
  for (int it = 0; it < limit; ++it) {
    if (mbar_try_wait(bar, parity)) return true;
    if (it > 32) __nanosleep(64);
  }
  return false;
}

// Copy `bytes` (multiple of 16, 16-byte aligned on both sides) from global to shared with
// bulk copies tracked by one mbarrier.  Every thread of the block must call this.  Returns
// the same value in all threads: true when the data has landed; false if the wait expired
// (the error word is then set and the block should return without using the data).
__device__ __forceinline__ bool stage_blob(uint8_t* dst, const uint8_t* src, uint32_t bytes, uint64_t* bar, int* err) {
  constexpr uint32_t kChunk = 32768;
  if (threadIdx.x == 0) mbar_init(bar, 1);
  __syncthreads();
  if (threadIdx.x == 0) {
    mbar_expect_tx(bar, bytes);
    for (uint32_t off = 0; off < bytes; off += kChunk)
      bulk_g2s(dst + off, src + off, (bytes - off < kChunk) ? (bytes - off) : kChunk, bar);
  }
  bool ok = mbar_wait_bounded(bar, 0);
  if (!ok) {
    atomicExch(err, PE_ERR_TIMEOUT);
    mbar_wait_bounded(bar, 0);  // give copies still in flight a second, equally bounded, chance to land
  }
  return __syncthreads_and(ok ? 1 : 0) != 0;
}

}  // namespace pe
