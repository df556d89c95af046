// Shared host/device helpers of the dpstep library (internal, not part of the C ABI).
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include <stddef.h>
#include "dpstep.h"

namespace dp {

// Records the text of a failed CUDA call for dp_last_cuda_error() and returns DP_ERR_CUDA.
dp_status cuda_fail(cudaError_t e, const char *where);
// Records a plain message for dp_last_cuda_error() (used where the failure is not a CUDA error code).
void note_error(const char *message);

// Number of SMs of the current device (cached per device; 148 if the query fails).
int sm_count();
// Number of SMs one tensor-core launch should spread over: dp_set_sm_target()'s value, or all of them.
int sm_target();
bool sm_target_set();   // true once dp_set_sm_target() was given a positive value: the caller runs calls side by side
// false while dp_debug_set_single_pass(0) holds: the fused clipped sum then always runs its two-pass form
bool single_pass_enabled();

// Every dp_per_example_wgrad workspace starts with this header, cleared by dp_workspace_init: the sticky status word
// at byte 0 and, from byte 256, the ticket counters with which the last block to finish a unit of work finds out
// that it is the last (each kernel leaves its counters at zero again).
constexpr size_t kWsHeaderBytes = 16384;
constexpr size_t kWsCounterOffset = 256;
constexpr int kWsCounters = (int)((kWsHeaderBytes - kWsCounterOffset) / sizeof(int));

inline bool aligned(const void *p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }
inline size_t round_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

#define DP_CUDA_TRY(expr)                                         \
    do {                                                          \
        cudaError_t e__ = (expr);                                 \
        if (e__ != cudaSuccess) return dp::cuda_fail(e__, #expr); \
    } while (0)

// Host-side count of kernel launches made by this process (read by dp_debug_launch_count).
void count_launch();

// After a kernel launch: picks up launch-configuration errors without synchronising.
#define DP_LAUNCH_CHECK(name)                                          \
    do {                                                               \
        cudaError_t e__ = cudaGetLastError();                          \
        if (e__ != cudaSuccess) return dp::cuda_fail(e__, name);       \
        dp::count_launch();                                            \
    } while (0)

__device__ __forceinline__ float to_float(float v) { return v; }
__device__ __forceinline__ float to_float(__nv_bfloat16 v) { return __bfloat162float(v); }

// Sum over the 32 lanes in a fixed butterfly order (same result on every run).
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// Block-wide sum for blockDim.x a multiple of 32 (<= 1024); every thread gets the result.
// `scratch` holds at least 32 values.  Fixed order: lanes by butterfly, then warps by butterfly.
template <typename T>
__device__ __forceinline__ T block_sum(T v, T *scratch) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarp = (blockDim.x + 31) >> 5;
    v = warp_sum(v);
    __syncthreads();                       // scratch may still be read from a previous call
    if (lane == 0) scratch[warp] = v;
    __syncthreads();
    T r = (lane < nwarp) ? scratch[lane] : T(0);
    r = warp_sum(r);
    return r;
}

// min(1, thr/sqrt(s)) written as a branch: s <= thr^2 gives exactly 1 (covers s = 0 and thr = inf).
__device__ __forceinline__ float clip_factor(double s, float thr) {
    const double t = (double)thr;
    return (s <= t * t) ? 1.0f : (float)(t / sqrt(s));
}

}  // namespace dp
