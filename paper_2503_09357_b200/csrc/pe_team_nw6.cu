// pe_eval_team_kernel with 6 warps per block: instantiations.
#include "pe_team_launch.h"

namespace pe {

int launch_team_nw6(const TeamCall& t, bool by_pos) { return launch_team_nw<6>(t, by_pos); }

}  // namespace pe
