// Internal: launch templates of pe_eval_lane_kernel.  The instantiations are split over two translation units
// (by-operator and by-position assignments) so that they compile in parallel.
#pragma once
#include "pe_kernel_lane.cuh"
#include "pe_launch.h"

namespace pe {


template <typename IdxT, bool BY_POS, int CLS, bool STATE_SMEM, int DEPTH>
static int launch4(const pe_graph* g, const Plan& p, int64_t K, const uint8_t* assign, const uint16_t* order,
                   uint32_t flags, const pe_outputs& out, uint32_t* gstate, unsigned grid, cudaStream_t stream) {
  auto go = [&](auto kern) -> int {
    if (!set_smem(kern, p.smem)) return PE_ERR_CUDA;
    // GLOBAL with the per-machine records in the workspace (plan.smem == 0): they follow the state tiles
    int4* gdev = nullptr;
    if (p.variant == PE_VARIANT_GLOBAL && p.smem == 0)
      gdev = reinterpret_cast<int4*>(reinterpret_cast<uint8_t*>(gstate) + p.ws_x_off);
    int32_t* gchan = nullptr;   // GLOBAL with exclusive channels: the per-channel words follow everything else
    if (p.variant == PE_VARIANT_GLOBAL && p.exclusive)
      gchan = reinterpret_cast<int32_t*>(reinterpret_cast<uint8_t*>(gstate) + p.ws_c_off);
    kern<<<grid, p.threads, p.smem, stream>>>(g->nview, g->d_nblob, K, assign, order, out, flags, g->d_error, gstate,
                                               gdev, p.jbits, gchan);
    return PE_OK;
  };
  if constexpr (STATE_SMEM) {
    if (p.state16)   // end time and machine fit 16 bits together: half the state per candidate
      return out.start ? go(pe_eval_lane_kernel<IdxT, BY_POS, CLS, true, true, DEPTH, false, uint16_t>)
                       : go(pe_eval_lane_kernel<IdxT, BY_POS, CLS, true, false, DEPTH, false, uint16_t>);
    if (p.exclusive)
      return out.start ? go(pe_eval_lane_kernel<IdxT, BY_POS, CLS, true, true, DEPTH, true>)
                       : go(pe_eval_lane_kernel<IdxT, BY_POS, CLS, true, false, DEPTH, true>);
  }
  if constexpr (!STATE_SMEM) {
    if (p.exclusive)
      return out.start ? go(pe_eval_lane_kernel<IdxT, BY_POS, CLS, false, true, DEPTH, true>)
                       : go(pe_eval_lane_kernel<IdxT, BY_POS, CLS, false, false, DEPTH, true>);
  }
  return out.start ? go(pe_eval_lane_kernel<IdxT, BY_POS, CLS, STATE_SMEM, true, DEPTH>)
                   : go(pe_eval_lane_kernel<IdxT, BY_POS, CLS, STATE_SMEM, false, DEPTH>);
}

template <bool BY_POS>
static int launch1(const pe_graph* g, const Plan& p, int64_t K, const uint8_t* assign, const uint16_t* order,
                   uint32_t flags, const pe_outputs& out, uint32_t* gstate, unsigned grid, cudaStream_t stream) {
  const bool smem_state = p.variant == PE_VARIANT_SHARED;
  const bool idx32 = (uint64_t)(g->V + 1) * (uint64_t)K <= 0xFFFFFFFFull;
  const int cls = g->nview.L == 2 ? 2 : (g->nview.need_cls ? 1 : 0);
  // straight-line specialisation: one fully connected link class and exactly three inline edge slots in
  // use (measured 1.25x on the random layered graphs; for graphs with at most two incoming edges the
  // general code, which skips the third slot by a uniform branch, is the faster one)
  const int depth = (cls == 0 && g->max_indeg == 3) ? 3 : 0;
#define PE_GO(IDX, CLS, SM, DEPTH) \
  return launch4<IDX, BY_POS, CLS, SM, DEPTH>(g, p, K, assign, order, flags, out, gstate, grid, stream)
#define PE_GO_CLS(IDX, SM)                             \
  do {                                                 \
    if (cls == 2) PE_GO(IDX, 2, SM, 0);                \
    if (cls == 1) PE_GO(IDX, 1, SM, 0);                \
    if (depth == 3) PE_GO(IDX, 0, SM, 3);              \
    PE_GO(IDX, 0, SM, 0);                              \
  } while (0)
  if (idx32) {
    if (smem_state) PE_GO_CLS(uint32_t, true);
    PE_GO_CLS(uint32_t, false);
  }
  if (smem_state) PE_GO_CLS(uint64_t, true);
  PE_GO_CLS(uint64_t, false);
#undef PE_GO_CLS
#undef PE_GO
}


int launch_lane_by_op(const pe_graph* g, const Plan& p, int64_t K, const uint8_t* assign, const uint16_t* order,
                     uint32_t flags, const pe_outputs& out, uint32_t* gstate, unsigned grid, cudaStream_t stream);
int launch_lane_by_pos(const pe_graph* g, const Plan& p, int64_t K, const uint8_t* assign, const uint16_t* order,
                     uint32_t flags, const pe_outputs& out, uint32_t* gstate, unsigned grid, cudaStream_t stream);

}  // namespace pe
