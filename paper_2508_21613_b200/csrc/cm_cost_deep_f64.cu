// Explicit instantiation: deep (17..48 stages) pipelines, fp64 cost arithmetic (see cm_cost_impl.cuh).
#include "cm_cost_impl.cuh"

namespace cm {
template cudaError_t launch_deep_class<double>(const Tables &, const BatchDev &, const LaunchClass &, cudaStream_t);
template cudaError_t launch_tiebreak_deep<double>(const Tables &, const BatchDev &, int, cudaStream_t);
}  // namespace cm
