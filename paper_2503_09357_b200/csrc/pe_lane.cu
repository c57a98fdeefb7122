// Launcher of the lane kernels (instantiated in pe_lane_op.cu and pe_lane_pos.cu).
#include "pe_lane_launch.h"

namespace pe {

int launch_lane(const pe_graph* g, const Plan& p, bool by_pos, int64_t K, const uint8_t* assign, const uint16_t* order,
                uint32_t flags, const pe_outputs& out, uint32_t* gstate, unsigned grid, cudaStream_t stream) {
  return by_pos ? launch_lane_by_pos(g, p, K, assign, order, flags, out, gstate, grid, stream) : launch_lane_by_op(g, p, K, assign, order, flags, out, gstate, grid, stream);
}

}  // namespace pe
