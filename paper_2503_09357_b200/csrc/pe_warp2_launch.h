// Internal: launch templates of pe_eval_warp2_kernel.  The instantiations are split over two translation units
// (by-operator and by-position assignments) so that they compile in parallel.
#pragma once
#include "pe_kernel_warp2.cuh"
#include "pe_launch.h"

namespace pe {


template <typename IdxT, bool BY_POS, int CLS, bool GRAPH_SMEM>
static int launch4(const pe_graph* g, const Plan& p, int64_t K, const uint8_t* assign, const uint16_t* order,
                   uint32_t flags, const pe_outputs& out, unsigned grid, cudaStream_t stream) {
  auto go = [&](auto kern) -> int {
    if (!set_smem(kern, p.smem)) return PE_ERR_CUDA;
    // few warps per SM: the window loop with the shorter loop-carried chain (see the kernel)
    const int final_rounds = p.threads / 32 < 24 ? 1 : 0;   // (measured: 1-5 % faster below about 24 warps per SM, equal above)
    kern<<<grid, p.threads, p.smem, stream>>>(g->nview, g->d_nblob, K, assign, order, out, flags, g->d_error,
                                               p.warp_words, final_rounds);
    return PE_OK;
  };
  constexpr bool kCanFlat = CLS == 0;
  const bool reg = g->max_indeg <= 3;   // in-window dependences fit the register slots
  const bool flat = kCanFlat && reg;
#define PE_W2(SLAB, FLAT, REG)                                                                       \
  return out.start ? go(pe_eval_warp2_kernel<IdxT, BY_POS, CLS, GRAPH_SMEM, true, SLAB, FLAT, REG>)  \
                   : go(pe_eval_warp2_kernel<IdxT, BY_POS, CLS, GRAPH_SMEM, false, SLAB, FLAT, REG>)
  if (flat) {
    if (p.slab) PE_W2(true, kCanFlat, true);
    PE_W2(false, kCanFlat, true);
  }
  if (reg) {
    if (p.slab) PE_W2(true, false, true);
    PE_W2(false, false, true);
  }
  if (p.slab) PE_W2(true, false, false);
  PE_W2(false, false, false);
#undef PE_W2
}

template <bool BY_POS>
static int launch1(const pe_graph* g, const Plan& p, int64_t K, const uint8_t* assign, const uint16_t* order,
                   uint32_t flags, const pe_outputs& out, unsigned grid, cudaStream_t stream) {
  const bool idx32 = (uint64_t)g->V * (uint64_t)K <= 0xFFFFFFFFull;
  const int cls = g->nview.L == 2 ? 2 : (g->nview.need_cls ? 1 : 0);
#define PE_GO(IDX, CLS, SM) return launch4<IDX, BY_POS, CLS, SM>(g, p, K, assign, order, flags, out, grid, stream)
#define PE_GO_CLS(IDX, SM)           \
  do {                               \
    if (cls == 2) PE_GO(IDX, 2, SM); \
    if (cls == 1) PE_GO(IDX, 1, SM); \
    PE_GO(IDX, 0, SM);               \
  } while (0)
  if (idx32) {
    if (p.graph_smem) PE_GO_CLS(uint32_t, true);
    PE_GO_CLS(uint32_t, false);
  }
  if (p.graph_smem) PE_GO_CLS(uint64_t, true);
  PE_GO_CLS(uint64_t, false);
#undef PE_GO_CLS
#undef PE_GO
}


int launch_warp2_by_op(const pe_graph* g, const Plan& p, int64_t K, const uint8_t* assign, const uint16_t* order,
                      uint32_t flags, const pe_outputs& out, unsigned grid, cudaStream_t stream);
int launch_warp2_by_pos(const pe_graph* g, const Plan& p, int64_t K, const uint8_t* assign, const uint16_t* order,
                      uint32_t flags, const pe_outputs& out, unsigned grid, cudaStream_t stream);

}  // namespace pe
