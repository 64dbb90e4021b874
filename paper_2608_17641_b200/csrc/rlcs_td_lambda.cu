// Kernel instantiations for one algorithm (see rlcs_scan.cuh for the kernel itself).
#include "rlcs_launch.cuh"

namespace rlcs {
RLCS_DEFINE_LAUNCHER(launch_td_lambda, kTdLambda, true)
}  // namespace rlcs
