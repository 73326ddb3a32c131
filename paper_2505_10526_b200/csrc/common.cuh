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

// Record the first device-side problem without trapping.
__device__ __forceinline__ void set_status(int32_t* dev_status, int code) {
    if (dev_status) atomicCAS(dev_status, 0, code);
}

__device__ __forceinline__ float bf16_bits_to_float(uint16_t h) {
    return __uint_as_float(((uint32_t)h) << 16);
}

// Per-sequence result of the acceptance scan, consumed by the sampling kernels.
struct SeqState {
    int32_t n;        // index of the row the extra token is drawn from (first rejection or gamma)
    int32_t use_q;    // 1: residual max(p - q, 0); 0: p itself
    float row_max;    // max logit of row n
    float inv_sum;    // 1 / sum exp((z - max)/T) of row n
};

// Host-side tally of kernel launches (see massv_launch_count).
void count_launches(int n);

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

}  // namespace massv
