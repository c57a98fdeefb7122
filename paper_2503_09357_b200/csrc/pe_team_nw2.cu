// pe_eval_team_kernel with 2 warps per block: instantiations.
#include "pe_team_launch.h"

namespace pe {

int launch_team_nw2(const TeamCall& t, bool by_pos) { return launch_team_nw<2>(t, by_pos); }

}  // namespace pe
