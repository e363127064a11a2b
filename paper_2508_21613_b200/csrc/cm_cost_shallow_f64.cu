// Explicit instantiation: shallow (<= 16 stages) pipelines, fp64 cost arithmetic (see cm_cost_impl.cuh).
#include "cm_cost_impl.cuh"

namespace cm {
template cudaError_t launch_shallow_class<double>(const Tables &, const BatchDev &, const LaunchClass &, cudaStream_t);
template cudaError_t launch_shallow_any<double>(const Tables &, const BatchDev &, uint32_t, uint32_t, uint64_t, cudaStream_t);
template cudaError_t launch_shallow_pair_class<double>(const Tables &, const BatchDev &, const LaunchClass &, cudaStream_t);
template cudaError_t launch_short_class<double>(const Tables &, const BatchDev &, const LaunchClass &, cudaStream_t);
}  // namespace cm
