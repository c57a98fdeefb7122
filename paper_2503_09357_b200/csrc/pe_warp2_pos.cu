// Instantiations of the warp2 kernels for by-position assignments.
#include "pe_warp2_launch.h"

namespace pe {

int launch_warp2_by_pos(const pe_graph* g, const Plan& p, int64_t K, const uint8_t* assign, const uint16_t* order,
                      uint32_t flags, const pe_outputs& out, unsigned grid, cudaStream_t stream) {
  return launch1<true>(g, p, K, assign, order, flags, out, grid, stream);
}

}  // namespace pe
