// Launcher of the warp2 kernels (instantiated in pe_warp2_op.cu and pe_warp2_pos.cu).
#include "pe_warp2_launch.h"

namespace pe {

int launch_warp2(const pe_graph* g, const Plan& p, bool by_pos, int64_t K, const uint8_t* assign, const uint16_t* order,
                 uint32_t flags, const pe_outputs& out, unsigned grid, cudaStream_t stream) {
  return by_pos ? launch_warp2_by_pos(g, p, K, assign, order, flags, out, grid, stream) : launch_warp2_by_op(g, p, K, assign, order, flags, out, grid, stream);
}

}  // namespace pe
