// Kernel instantiations for GAE with observation-skip masking: the value fill and the masked GAE scan
// (see rlcs_scan.cuh for the kernel itself).
#include "rlcs_launch.cuh"

namespace rlcs {
RLCS_DEFINE_LAUNCHER(launch_fill_skip, kFillSkip, true)
RLCS_DEFINE_LAUNCHER(launch_gae_skip, kGaeSkip, true)
}  // namespace rlcs
