// Kernel instantiations for one algorithm (see rlcs_scan.cuh for the kernel itself).
#include "rlcs_launch.cuh"

namespace RLCS_NS {
RLCS_DEFINE_LAUNCHER(launch_vtrace, kVtrace, true)
}  // namespace RLCS_NS
