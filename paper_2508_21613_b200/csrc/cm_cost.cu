// Search pass and deep tie-break pass: dispatch to the per-type launchers (kernels and the
// launchers themselves are in cm_cost_impl.cuh, instantiated in cm_cost_{shallow,deep}_{f64,i64}.cu).
#include "cm_internal.h"

namespace cm {

template <typename T> cudaError_t launch_shallow_class(const Tables &, const BatchDev &, const LaunchClass &, cudaStream_t);
template <typename T> cudaError_t launch_shallow_any(const Tables &, const BatchDev &, uint32_t, uint32_t, uint64_t, cudaStream_t);
template <typename T> cudaError_t launch_shallow_pair_class(const Tables &, const BatchDev &, const LaunchClass &, cudaStream_t);
template <typename T> cudaError_t launch_short_class(const Tables &, const BatchDev &, const LaunchClass &, cudaStream_t);
template <typename T, int LO, int HI> cudaError_t launch_deep_range(const Tables &, const BatchDev &, const LaunchClass &, cudaStream_t);
template <typename T, int LO, int HI> cudaError_t launch_tiebreak_range(const Tables &, const BatchDev &, int, cudaStream_t);
template <typename T> cudaError_t launch_solo_class(const Tables &, const BatchDev &, const LaunchClass &, cudaStream_t);
template <typename T> cudaError_t launch_warp_class(const Tables &, const BatchDev &, const LaunchClass &, cudaStream_t);

#define CM_EXTERN(T)                                                                                                   \
    extern template cudaError_t launch_shallow_class<T>(const Tables &, const BatchDev &, const LaunchClass &, cudaStream_t); \
    extern template cudaError_t launch_shallow_any<T>(const Tables &, const BatchDev &, uint32_t, uint32_t, uint64_t, cudaStream_t); \
    extern template cudaError_t launch_shallow_pair_class<T>(const Tables &, const BatchDev &, const LaunchClass &, cudaStream_t); \
    extern template cudaError_t launch_short_class<T>(const Tables &, const BatchDev &, const LaunchClass &, cudaStream_t); \
    extern template cudaError_t launch_solo_class<T>(const Tables &, const BatchDev &, const LaunchClass &, cudaStream_t); \
    extern template cudaError_t launch_warp_class<T>(const Tables &, const BatchDev &, const LaunchClass &, cudaStream_t);
CM_EXTERN(double)
CM_EXTERN(long long)
#undef CM_EXTERN

// the deep-pipeline kernels: one translation unit per cost type and range of stage counts
#define CM_DEEP_RANGE(LO, HI)                                                                                                     \
    extern template cudaError_t launch_deep_range<double, LO, HI>(const Tables &, const BatchDev &, const LaunchClass &, cudaStream_t); \
    extern template cudaError_t launch_deep_range<long long, LO, HI>(const Tables &, const BatchDev &, const LaunchClass &, cudaStream_t); \
    extern template cudaError_t launch_tiebreak_range<double, LO, HI>(const Tables &, const BatchDev &, int, cudaStream_t);         \
    extern template cudaError_t launch_tiebreak_range<long long, LO, HI>(const Tables &, const BatchDev &, int, cudaStream_t);
CM_DEEP_RANGES(CM_DEEP_RANGE)
#undef CM_DEEP_RANGE

template <typename T>
static cudaError_t launch_deep_class(const Tables &t, const BatchDev &b, const LaunchClass &c, cudaStream_t st) {
#define CM_DEEP_RANGE(LO, HI) if (c.stages >= LO && c.stages <= HI) return launch_deep_range<T, LO, HI>(t, b, c, st);
    CM_DEEP_RANGES(CM_DEEP_RANGE)
#undef CM_DEEP_RANGE
    return cudaErrorInvalidValue;
}

template <typename T>
static cudaError_t launch_tiebreak_deep(const Tables &t, const BatchDev &b, int S, cudaStream_t st) {
#define CM_DEEP_RANGE(LO, HI) if (S >= LO && S <= HI) return launch_tiebreak_range<T, LO, HI>(t, b, S, st);
    CM_DEEP_RANGES(CM_DEEP_RANGE)
#undef CM_DEEP_RANGE
    return cudaSuccess;
}

template <typename T>
static cudaError_t launch_class(const Tables &t, const BatchDev &b, const LaunchClass &c, cudaStream_t st) {
    if (c.kind == CM_CLASS_REGS) return launch_shallow_class<T>(t, b, c, st);
    if (c.kind == CM_CLASS_REGS_PAIR) return launch_shallow_pair_class<T>(t, b, c, st);
    if (c.kind == CM_CLASS_WIDE_UNI || c.kind == CM_CLASS_WIDE_LANE || c.kind == CM_CLASS_WIDE_PAIR ||
        c.kind == CM_CLASS_WIDE_LANE_PAIR) return launch_deep_class<T>(t, b, c, st);
    if (c.kind == CM_CLASS_SOLO) return launch_solo_class<T>(t, b, c, st);
    if (c.kind == CM_CLASS_WARP) return launch_warp_class<T>(t, b, c, st);
    if (c.kind == CM_CLASS_SHORT) return launch_short_class<T>(t, b, c, st);
    return cudaErrorInvalidValue;
}

// stage_mask: bit S set = some template segment of the batch has S stages (17 <= S <= 48)
cudaError_t launch_tiebreak_wide(const Tables &t, const BatchDev &b, uint64_t stage_mask, cudaStream_t st,
                                 const SideStreams *side, int *launches) {
    if (b.B <= 0 || b.max_tiles_per_seg == 0 || b.dp_max == 0) return cudaSuccess;
    int n_launch = 0;
    for (int S = kRegStagesMax + 1; S <= kWideStagesMax; ++S) n_launch += (int)((stage_mask >> S) & 1ull);
    // one kernel per depth, each over its own pipelines' slots: side by side like the search pass
    const int n_side = (side && n_launch > 1) ? (side->n < n_launch - 1 ? side->n : n_launch - 1) : 0;
    if (n_side) {
        cudaError_t e = cudaEventRecord(side->fork, st);
        for (int k = 0; k < n_side && e == cudaSuccess; ++k) e = cudaStreamWaitEvent(side->stream[k], side->fork, 0);
        if (e != cudaSuccess) return e;
    }
    cudaError_t err = cudaSuccess;
    int slot = 0;
    for (int S = kRegStagesMax + 1; S <= kWideStagesMax && err == cudaSuccess; ++S) {
        if (!((stage_mask >> S) & 1ull)) continue;
        cudaStream_t s = (n_side && slot % (n_side + 1)) ? side->stream[slot % (n_side + 1) - 1] : st;
        ++slot;
        err = native_i64(b) ? launch_tiebreak_deep<long long>(t, b, S, s) : launch_tiebreak_deep<double>(t, b, S, s);
        if (err == cudaSuccess && launches) ++*launches;
    }
    for (int k = 0; k < n_side; ++k) {
        cudaError_t e = cudaEventRecord(side->join[k], side->stream[k]);
        if (e == cudaSuccess) e = cudaStreamWaitEvent(st, side->join[k], 0);
        if (err == cudaSuccess) err = e;
    }
    return err;
}

// A 2-D grid may overshoot the class's chunk count; surplus CTAs find the last bucket,
// see indices past its plans and idle.
cudaError_t launch_cost_pass1(const Tables &t, const BatchDev &b, const LaunchClass *classes, int n_classes,
                              cudaStream_t st, const SideStreams *side, int *launches) {
    // the register-resident classes come first and share one chunk numbering
    int n_regs = 0;
    uint64_t regs_chunks = 0;
    while (n_regs < n_classes && classes[n_regs].kind == CM_CLASS_REGS) regs_chunks += classes[n_regs++].n_chunks;
    int first = 0;
    if (n_regs > 1 && regs_chunks > 0 && regs_chunks <= (uint64_t)kAnyMaxChunks) {
        const uint32_t b0 = classes[0].bucket_begin, b1 = classes[n_regs - 1].bucket_end;
        cudaError_t e = native_i64(b) ? launch_shallow_any<long long>(t, b, b0, b1, regs_chunks, st)
                                                  : launch_shallow_any<double>(t, b, b0, b1, regs_chunks, st);
        if (e != cudaSuccess) return e;
        if (launches) ++*launches;
        first = n_regs;
    }
    int n_launch = 0;
    for (int i = first; i < n_classes; ++i) n_launch += classes[i].n_chunks ? 1 : 0;
    // classes only share the per-segment minima they atomically lower: run them side by side
    const int n_side = (side && n_launch > 1) ? (side->n < n_launch - 1 ? side->n : n_launch - 1) : 0;
    if (n_side) {
        cudaError_t e = cudaEventRecord(side->fork, st);
        for (int k = 0; k < n_side && e == cudaSuccess; ++k) e = cudaStreamWaitEvent(side->stream[k], side->fork, 0);
        if (e != cudaSuccess) return e;
    }
    cudaError_t err = cudaSuccess;
    int slot = 0;
    for (int i = first; i < n_classes && err == cudaSuccess; ++i) {
        if (classes[i].n_chunks == 0) continue;
        cudaStream_t s = (n_side && slot % (n_side + 1)) ? side->stream[slot % (n_side + 1) - 1] : st;
        ++slot;
        err = native_i64(b) ? launch_class<long long>(t, b, classes[i], s) : launch_class<double>(t, b, classes[i], s);
        if (err == cudaSuccess && launches) ++*launches;
    }
    // always join, even after a failed launch, so that the side streams never run ahead unobserved
    for (int k = 0; k < n_side; ++k) {
        cudaError_t e = cudaEventRecord(side->join[k], side->stream[k]);
        if (e == cudaSuccess) e = cudaStreamWaitEvent(st, side->join[k], 0);
        if (err == cudaSuccess) err = e;
    }
    return err;
}

}  // namespace cm
