// Instantiations and launcher of pe_eval_warp2_kernel.
#include "pe_kernel_warp2.cuh"
#include "pe_launch.h"

namespace pe {

template <typename IdxT, bool BY_POS, int CLS, bool GRAPH_SMEM>
static int launch4(const pe_graph* g, const Plan& p, int64_t K, const uint8_t* assign, const uint16_t* order,
                   uint32_t flags, const pe_outputs& out, unsigned grid, cudaStream_t stream) {
  auto go = [&](auto kern) -> int {
    if (!set_smem(kern, p.smem)) return PE_ERR_CUDA;
    kern<<<grid, p.threads, p.smem, stream>>>(g->nview, g->d_nblob, K, assign, order, out, flags, g->d_error,
                                               p.warp_words);
    return PE_OK;
  };
  constexpr bool kCanFlat = CLS == 0;
  const bool flat = kCanFlat && g->max_indeg <= 3;
  if (flat) {
    if (p.slab)
      return out.start ? go(pe_eval_warp2_kernel<IdxT, BY_POS, CLS, GRAPH_SMEM, true, true, kCanFlat>)
                       : go(pe_eval_warp2_kernel<IdxT, BY_POS, CLS, GRAPH_SMEM, false, true, kCanFlat>);
    return out.start ? go(pe_eval_warp2_kernel<IdxT, BY_POS, CLS, GRAPH_SMEM, true, false, kCanFlat>)
                     : go(pe_eval_warp2_kernel<IdxT, BY_POS, CLS, GRAPH_SMEM, false, false, kCanFlat>);
  }
  if (p.slab)
    return out.start ? go(pe_eval_warp2_kernel<IdxT, BY_POS, CLS, GRAPH_SMEM, true, true, false>)
                     : go(pe_eval_warp2_kernel<IdxT, BY_POS, CLS, GRAPH_SMEM, false, true, false>);
  return out.start ? go(pe_eval_warp2_kernel<IdxT, BY_POS, CLS, GRAPH_SMEM, true, false, false>)
                   : go(pe_eval_warp2_kernel<IdxT, BY_POS, CLS, GRAPH_SMEM, false, false, false>);
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

int launch_warp2(const pe_graph* g, const Plan& p, bool by_pos, int64_t K, const uint8_t* assign, const uint16_t* order,
                 uint32_t flags, const pe_outputs& out, unsigned grid, cudaStream_t stream) {
  return by_pos ? launch1<true>(g, p, K, assign, order, flags, out, grid, stream)
                : launch1<false>(g, p, K, assign, order, flags, out, grid, stream);
}

}  // namespace pe
