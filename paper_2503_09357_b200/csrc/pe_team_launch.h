// Internal: one launch of pe_eval_team_kernel.  The instantiations are spread over one translation unit per
// number of warps (pe_team_nw2.cu, pe_team_nw4.cu, pe_team_nw6.cu) so that they compile in parallel.
#pragma once
#include "pe_kernel_team.cuh"
#include "pe_launch.h"

namespace pe {

struct TeamCall {
  const pe_graph* g;
  const Plan* p;
  int64_t K;        // row pitch of the interface arrays
  int64_t kc;       // candidates of this launch
  const uint8_t* assign;
  const uint16_t* order;
  uint32_t flags;
  pe_outputs out;
  TeamStrides sd;
  cudaStream_t stream;
};

template <int NW, bool BY_POS, int CLS>
int launch3(const TeamCall& t) {
  auto go = [&](auto kern) -> int {
    if (!set_smem(kern, t.p->smem)) return PE_ERR_CUDA;
    // the state is all these blocks need from the SM's memory: ask for the largest shared-memory carve-out
    // (a hint; without it the default carve-out can hold fewer blocks than shared memory would allow)
    cudaFuncSetAttribute(kern, cudaFuncAttributePreferredSharedMemoryCarveout, (int)cudaSharedmemCarveoutMaxShared);
    kern<<<(unsigned)t.kc, NW * 32, t.p->smem, t.stream>>>(t.g->nview, t.g->d_nblob, t.K, t.assign, t.order, t.out, t.flags,
                                                            t.sd);
    return PE_OK;
  };
  const bool wide = t.g->max_indeg > 3;   // operators with four to eight incoming edges
#define PE_TEAM(TIMES, STAGED) \
  (wide ? go(pe_eval_team_kernel<NW, BY_POS, CLS, TIMES, STAGED, true>) : go(pe_eval_team_kernel<NW, BY_POS, CLS, TIMES, STAGED, false>))
  if (t.p->staged) return t.out.start ? PE_TEAM(true, true) : PE_TEAM(false, true);
  return t.out.start ? PE_TEAM(true, false) : PE_TEAM(false, false);
#undef PE_TEAM
}

template <int NW>
int launch_team_nw(const TeamCall& t, bool by_pos) {
  const int cls = t.g->nview.L == 2 ? 2 : (t.g->nview.need_cls ? 1 : 0);
  if (by_pos) {
    if (cls == 2) return launch3<NW, true, 2>(t);
    if (cls == 1) return launch3<NW, true, 1>(t);
    return launch3<NW, true, 0>(t);
  }
  if (cls == 2) return launch3<NW, false, 2>(t);
  if (cls == 1) return launch3<NW, false, 1>(t);
  return launch3<NW, false, 0>(t);
}

int launch_team_nw2(const TeamCall& t, bool by_pos);
int launch_team_nw4(const TeamCall& t, bool by_pos);
int launch_team_nw6(const TeamCall& t, bool by_pos);

}  // namespace pe
