// Explicit instantiation: shallow (<= 16 stages) pipelines, int64-nanosecond cost arithmetic (see cm_cost_impl.cuh).
#include "cm_cost_impl.cuh"

namespace cm {
template cudaError_t launch_shallow_class<long long>(const Tables &, const BatchDev &, const LaunchClass &, cudaStream_t);
template cudaError_t launch_shallow_any<long long>(const Tables &, const BatchDev &, uint32_t, uint32_t, uint64_t, cudaStream_t);
template cudaError_t launch_shallow_pair_class<long long>(const Tables &, const BatchDev &, const LaunchClass &, cudaStream_t);
template cudaError_t launch_short_class<long long>(const Tables &, const BatchDev &, const LaunchClass &, cudaStream_t);
}  // namespace cm
