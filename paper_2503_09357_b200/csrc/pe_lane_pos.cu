// Instantiations of the lane kernels for by-position assignments.
#include "pe_lane_launch.h"

namespace pe {

int launch_lane_by_pos(const pe_graph* g, const Plan& p, int64_t K, const uint8_t* assign, const uint16_t* order,
                     uint32_t flags, const pe_outputs& out, uint32_t* gstate, unsigned grid, cudaStream_t stream) {
  return launch1<true>(g, p, K, assign, order, flags, out, gstate, grid, stream);
}

}  // namespace pe
