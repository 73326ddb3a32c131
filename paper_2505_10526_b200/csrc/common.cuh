// Shared device/host helpers of the verify-step library (sm_100a only).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "massv.h"

namespace massv {

constexpr int kPageSize = 16;       // tokens per KV page
constexpr int kMaxRows = 8;         // gamma + 1 <= 8
constexpr int kVocabTile = 128;     // vocabulary rows per LM-head tile
constexpr int kResidualChunk = 4096;  // vocabulary entries per residual-mass chunk
constexpr int kResidualSegments = 8;  // a chunk is eight segments of 512 entries, one per consumer warp of the draw kernel

// Record the first device-side problem without trapping.
__device__ __forceinline__ void set_status(int32_t* dev_status, int code) {
    if (dev_status) atomicCAS(dev_status, 0, code);
}

// Index checks of the debug build (-DMASSV_DEBUG): an index outside [0, limit) records MASSV_ERR_BOUNDS in the
// status word and the guarded access is skipped - no trap, no assert, the context stays usable.  In the ordinary
// build the macro is the constant true and the checks cost nothing.
#ifdef MASSV_DEBUG
__device__ __forceinline__ bool in_bounds_or_report(long long idx, long long limit, int32_t* dev_status) {
    if (idx >= 0 && idx < limit) return true;
    set_status(dev_status, MASSV_ERR_BOUNDS);
    return false;
}
#define MASSV_IN_BOUNDS(idx, limit, dev_status) (::massv::in_bounds_or_report((long long)(idx), (long long)(limit), (dev_status)))
#else
#define MASSV_IN_BOUNDS(idx, limit, dev_status) (true)
#endif

__device__ __forceinline__ float bf16_bits_to_float(uint16_t h) {
    return __uint_as_float(((uint32_t)h) << 16);
}

// Programmatic dependent launch: every kernel is launched so that it may start
// while its predecessor in the stream drains.  pdl_wait() blocks until the
// predecessor has completed and its writes are visible; it must run before the
// first access to global memory.  pdl_trigger() lets the successor begin launching.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                              Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// Same, with the grid made of thread-block clusters of cluster_x CTAs along x.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl_cluster(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                                      int cluster_x, Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = (unsigned)cluster_x;
    attr[1].val.clusterDim.y = 1;
    attr[1].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// Per-sequence result of the acceptance scan, consumed by the sampling kernels.
struct SeqState {
    int32_t n;        // index of the row the extra token is drawn from (first rejection or gamma)
    int32_t use_q;    // 1: residual max(p - q, 0); 0: p itself
    float row_max;    // max logit of row n
    float inv_sum;    // 1 / sum exp((z - max)/T) of row n
};

// Optional per-thread timing hooks (massv_set_timing_events): events recorded around the dominant kernel of a call.
struct TimingHooks {
    cudaEvent_t lm_head_start = nullptr, lm_head_stop = nullptr, attn_start = nullptr, attn_stop = nullptr;
    cudaEvent_t residual_start = nullptr, residual_stop = nullptr;
};
TimingHooks& timing_hooks();

// Host-side tally of kernel launches (see massv_launch_count).
void count_launches(int n);

// Multiprocessors of the current device (148 on B200).
inline int device_sm_count() {
    int dev = 0, n = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0)
        n = 148;
    return n;
}

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

}  // namespace massv
