// Explicit instantiation: deep (17..48 stages) pipelines, int64-nanosecond cost arithmetic (see cm_cost_impl.cuh).
#include "cm_cost_impl.cuh"

namespace cm {
template cudaError_t launch_deep_class<long long>(const Tables &, const BatchDev &, const LaunchClass &, cudaStream_t);
template cudaError_t launch_tiebreak_deep<long long>(const Tables &, const BatchDev &, int, cudaStream_t);
}  // namespace cm
