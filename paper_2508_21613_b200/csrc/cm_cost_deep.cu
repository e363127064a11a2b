// Explicit instantiation of the deep-pipeline kernels (see cm_cost_impl.cuh) for one cost type
// and one range of stage counts.  Compiled once per (type, range) with
//   -DCM_DEEP_T=double|"long long"  -DCM_DEEP_LO=<first stage count>  -DCM_DEEP_HI=<last>
// (the ranges are listed in cm_internal.h and in the build script).
#include "cm_cost_impl.cuh"

#if !defined(CM_DEEP_T) || !defined(CM_DEEP_LO) || !defined(CM_DEEP_HI)
#error "compile with -DCM_DEEP_T=<type> -DCM_DEEP_LO=<n> -DCM_DEEP_HI=<n>"
#endif

namespace cm {
template cudaError_t launch_deep_range<CM_DEEP_T, CM_DEEP_LO, CM_DEEP_HI>(const Tables &, const BatchDev &, const LaunchClass &, cudaStream_t);
template cudaError_t launch_tiebreak_range<CM_DEEP_T, CM_DEEP_LO, CM_DEEP_HI>(const Tables &, const BatchDev &, int, cudaStream_t);
}  // namespace cm
