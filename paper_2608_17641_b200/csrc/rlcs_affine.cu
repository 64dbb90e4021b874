// Kernel instantiations for the bare (alpha, beta) scan used as a test hook.
#include "rlcs_launch.cuh"

namespace rlcs {
RLCS_DEFINE_LAUNCHER(launch_affine_bwd, kAffineBwd, false)
RLCS_DEFINE_LAUNCHER(launch_affine_fwd, kAffineFwd, false)
}  // namespace rlcs
