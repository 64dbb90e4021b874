// Kernel instantiations for one algorithm (see rlcs_scan.cuh for the kernel itself).
#include "rlcs_launch.cuh"

namespace RLCS_NS {
RLCS_DEFINE_LAUNCHER(launch_td_lambda, kTdLambda, true)
}  // namespace RLCS_NS
