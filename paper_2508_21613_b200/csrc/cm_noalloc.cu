// cm_evaluate_argmin_noalloc: evaluate a range of candidates and reduce it to the best
// (cost, index) pair without allocating anything.
//
// Who needs this: code that reacts to a failure from a place where device allocation is
// off limits -- a recovery handler running while another framework's caching allocator
// owns every free byte of the GPU, a latency-critical path that cannot afford the
// device-wide synchronisation an allocation implies, or a process whose memory budget
// was fixed at start-up.  Such a caller prepares its candidate space ahead of time (that
// step does allocate) and later only asks "which of these candidates is cheapest?".
//
// The kernel is the per-candidate evaluation kernel of cm_evaluate with a block-level
// argmin behind it; the block partials and the arrival counter that the last block uses
// to finish the reduction live in the fixed array below instead of in allocated memory.
#include <mutex>
#include <string>

#include "cm_device.cuh"

namespace cm {

constexpr int kNoAllocThreads = 128;
constexpr int kNoAllocMaxBlocks = CM_NOALLOC_MAX_CANDIDATES / kNoAllocThreads;
// layout: [0, MaxBlocks) cost bits | [MaxBlocks, 2 MaxBlocks) candidate index | [2 MaxBlocks] arrival counter
constexpr size_t kNoAllocWords = 2 * (size_t)kNoAllocMaxBlocks + 32;

// Scratch of the entry point.  Every GPU that loads the library carries these 64.25 KB
// until the process exits.  In host code this name is only a handle for
// cudaGetSymbolAddress: it is not a device address and must never be passed to a kernel.
static __device__ __align__(256) unsigned long long cm_noalloc_scratch[kNoAllocWords];

__device__ __forceinline__ bool pair_before(uint64_t c1, uint64_t i1, uint64_t c2, uint64_t i2) {
    return c1 < c2 || (c1 == c2 && i1 < i2);
}

template <typename T>
__global__ void __launch_bounds__(kNoAllocThreads)
cm_evaluate_argmin_kernel(Tables tb, BatchDev bd, uint64_t first, uint64_t count, unsigned long long *scratch,
                          double *best_cost, int64_t *best_cost_ns, uint64_t *best_index) {
    __shared__ SProf<T> sp;
    __shared__ uint64_t wc[kNoAllocThreads / 32], wi[kNoAllocThreads / 32];
    __shared__ bool is_last;
    unsigned long long *part_cost = scratch, *part_idx = scratch + kNoAllocMaxBlocks;
    unsigned int *arrived = reinterpret_cast<unsigned int *>(scratch + 2 * kNoAllocMaxBlocks);
    stage_profile(sp, tb);
    __syncthreads();
    const uint64_t t = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    uint64_t c = inf_bits<T>(), idx = ~0ull;
    if (t < count) {
        const uint64_t e = first + t;
        const Tmpl tp = bd.tmpl[bd.scen[0].tmpl];
        uint32_t lo = 0, hi = tp.n_tseg - 1;
        while (lo < hi) {
            const uint32_t mid = (lo + hi + 1) >> 1;
            if (bd.tseg[tp.tseg_first + mid].cand_first <= e) lo = mid; else hi = mid - 1;
        }
        const uint32_t row = tp.tseg_first + lo;
        const SegView g = seg_view(bd, 0, row);
        T v;
        if (segment_candidate_cost<T>(sp, tb, g, bd.layer_mode, e - bd.tseg[row].cand_first, v)) {
            c = Num<T>::bits(v);
            idx = e;
        }
    }
    for (int o = 16; o > 0; o >>= 1) {
        const uint64_t oc = __shfl_xor_sync(0xffffffffu, c, o), oi = __shfl_xor_sync(0xffffffffu, idx, o);
        if (pair_before(oc, oi, c, idx)) { c = oc; idx = oi; }
    }
    if ((threadIdx.x & 31) == 0) { wc[threadIdx.x >> 5] = c; wi[threadIdx.x >> 5] = idx; }
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int w = 1; w < kNoAllocThreads / 32; ++w)
            if (pair_before(wc[w], wi[w], c, idx)) { c = wc[w]; idx = wi[w]; }
        part_cost[blockIdx.x] = c;
        part_idx[blockIdx.x] = idx;
        __threadfence();
        is_last = atomicAdd(arrived, 1u) == gridDim.x - 1;
    }
    __syncthreads();
    if (!is_last) return;
    // the last block to arrive sees every partial and finishes the argmin
    __threadfence();
    c = inf_bits<T>();
    idx = ~0ull;
    for (unsigned b = threadIdx.x; b < gridDim.x; b += blockDim.x) {
        const uint64_t oc = ((volatile unsigned long long *)part_cost)[b], oi = ((volatile unsigned long long *)part_idx)[b];
        if (pair_before(oc, oi, c, idx)) { c = oc; idx = oi; }
    }
    for (int o = 16; o > 0; o >>= 1) {
        const uint64_t oc = __shfl_xor_sync(0xffffffffu, c, o), oi = __shfl_xor_sync(0xffffffffu, idx, o);
        if (pair_before(oc, oi, c, idx)) { c = oc; idx = oi; }
    }
    __syncthreads();
    if ((threadIdx.x & 31) == 0) { wc[threadIdx.x >> 5] = c; wi[threadIdx.x >> 5] = idx; }
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int w = 1; w < kNoAllocThreads / 32; ++w)
            if (pair_before(wc[w], wi[w], c, idx)) { c = wc[w]; idx = wi[w]; }
        if (bd.mode == CM_COST_INT64NS) { if (best_cost_ns) *best_cost_ns = batch_cost_ns(bd, c); }
        else if (best_cost) *best_cost = __longlong_as_double((long long)c);
        if (best_index) *best_index = c < inf_bits<T>() ? idx : ~0ull;
        *arrived = 0;   // leave the counter clean for the next call
    }
}

// Device address of the scratch array, resolved once per device with that device current.
static cudaError_t noalloc_scratch_address(int device, unsigned long long **out) {
    static std::mutex mu;
    static unsigned long long *address[64] = {nullptr};
    if (device < 0 || device >= 64) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(mu);
    if (!address[device]) {
        int current = -1;
        cudaError_t e = cudaGetDevice(&current);
        if (e != cudaSuccess) return e;
        if (current != device) return cudaErrorInvalidDevice;
        void *p = nullptr;
        e = cudaGetSymbolAddress(&p, cm_noalloc_scratch);
        if (e != cudaSuccess) return e;
        address[device] = static_cast<unsigned long long *>(p);
    }
    *out = address[device];
    return cudaSuccess;
}

}  // namespace cm

using namespace cm;

extern "C" cm_status cm_evaluate_argmin_noalloc(cm_ctx *ctx, const cm_space *space, uint64_t first, uint64_t count,
                                                double *best_cost_dev, int64_t *best_cost_ns_dev,
                                                uint64_t *best_index_dev) {
    if (!ctx) return CM_EINVAL;
    try {   // the error paths below build std::string messages
    SpaceView v;
    cm_status s = cm_internal_space_view(ctx, space, &v);
    if (s != CM_OK) return s;
    if (v.policy != CM_DYNPAR) return cm_internal_fail(ctx, CM_EINVAL, "cm_evaluate_argmin_noalloc: only dynamic-parallelism spaces have a candidate range");
    if (count == 0 || count > (uint64_t)CM_NOALLOC_MAX_CANDIDATES)
        return cm_internal_fail(ctx, CM_EINVAL, "cm_evaluate_argmin_noalloc: count must be 1 .. CM_NOALLOC_MAX_CANDIDATES (" +
                                                    std::to_string(CM_NOALLOC_MAX_CANDIDATES) + "); split the range");
    if (first > v.n_cand || count > v.n_cand - first) return cm_internal_fail(ctx, CM_EINVAL, "candidate range out of bounds");
    if (cudaSetDevice(v.device) != cudaSuccess) { cudaGetLastError(); return cm_internal_fail(ctx, CM_ECUDA, "cudaSetDevice failed"); }
    unsigned long long *scratch = nullptr;
    cudaError_t e = noalloc_scratch_address(v.device, &scratch);
    if (e != cudaSuccess) { cudaGetLastError(); return cm_internal_fail(ctx, CM_ECUDA, std::string("cudaGetSymbolAddress: ") + cudaGetErrorString(e)); }
    // the arrival counter must start at zero whatever an earlier, possibly aborted, call left behind
    e = cudaMemsetAsync(scratch + 2 * kNoAllocMaxBlocks, 0, sizeof(unsigned long long), v.stream);
    if (e != cudaSuccess) { cudaGetLastError(); return cm_internal_fail(ctx, CM_ECUDA, cudaGetErrorString(e)); }
    const unsigned blocks = (unsigned)((count + kNoAllocThreads - 1) / kNoAllocThreads);
    if (native_i64(v.bd))
        cm_evaluate_argmin_kernel<long long><<<blocks, kNoAllocThreads, 0, v.stream>>>(v.tb, v.bd, first, count, scratch, best_cost_dev, best_cost_ns_dev, best_index_dev);
    else
        cm_evaluate_argmin_kernel<double><<<blocks, kNoAllocThreads, 0, v.stream>>>(v.tb, v.bd, first, count, scratch, best_cost_dev, best_cost_ns_dev, best_index_dev);
    e = cudaGetLastError();
    if (e != cudaSuccess) return cm_internal_fail(ctx, CM_ECUDA, cudaGetErrorString(e));
    return CM_OK;
    } catch (...) {
        return CM_ENOMEM;
    }
}
