// LM head, first correct version: z[m,v] = sum_k hidden[m,k] * lm_head[v,k] on
// CUDA cores with fp32 accumulation, followed by per-tile softmax statistics
// (max, sum of exponentials, argmax) over 128-entry vocabulary tiles.
// (Sec. 2.1: the target computes p(. | X_{1:t+i-1}) for i = 1..gamma+1.)
#include "kernels.cuh"

namespace massv {

namespace {

constexpr int kRowsPerIter = 8;

// One warp per vocabulary row, 8 token rows at a time.
__global__ void __launch_bounds__(256) lm_head_naive_kernel(LmHeadParams p) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int v = blockIdx.x * 8 + warp;
    if (v >= p.V) return;
    const uint4* w = reinterpret_cast<const uint4*>(p.lm_head + (size_t)v * p.K);
    const int chunks = p.K / 8;   // 16-byte words per row
    for (int m0 = 0; m0 < p.M; m0 += kRowsPerIter) {
        float acc[kRowsPerIter];
        for (int r = 0; r < kRowsPerIter; ++r) acc[r] = 0.f;
        for (int c = lane; c < chunks; c += 32) {
            const uint4 wv = __ldg(w + c);
            const __nv_bfloat162* wp = reinterpret_cast<const __nv_bfloat162*>(&wv);
            float wf[8];
            for (int e = 0; e < 4; ++e) { const float2 f = __bfloat1622float2(wp[e]); wf[2 * e] = f.x; wf[2 * e + 1] = f.y; }
            for (int r = 0; r < kRowsPerIter; ++r) {
                if (m0 + r >= p.M) break;
                const uint4 hv = __ldg(reinterpret_cast<const uint4*>(p.hidden + (size_t)(m0 + r) * p.K) + c);
                const __nv_bfloat162* hp = reinterpret_cast<const __nv_bfloat162*>(&hv);
                for (int e = 0; e < 4; ++e) {
                    const float2 f = __bfloat1622float2(hp[e]);
                    acc[r] += wf[2 * e] * f.x + wf[2 * e + 1] * f.y;
                }
            }
        }
        for (int r = 0; r < kRowsPerIter; ++r) {
            float s = acc[r];
            for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
            if (lane == 0 && m0 + r < p.M) p.logits[(size_t)(m0 + r) * p.V + v] = s;
        }
    }
}

// grid (n_tiles, M): statistics of one 128-entry tile of one row.
__global__ void __launch_bounds__(kVocabTile) tile_stats_kernel(LmHeadParams p) {
    const int tile = blockIdx.x, m = blockIdx.y, t = threadIdx.x;
    const int v = tile * kVocabTile + t;
    __shared__ float s_val[kVocabTile];
    __shared__ int s_idx[kVocabTile];
    const float z = v < p.V ? p.logits[(size_t)m * p.V + v] : -INFINITY;
    s_val[t] = z;
    s_idx[t] = v;
    __syncthreads();
    for (int w = kVocabTile / 2; w > 0; w >>= 1) {
        if (t < w) {
            const float a = s_val[t], b = s_val[t + w];
            if (b > a || (b == a && s_idx[t + w] < s_idx[t])) { s_val[t] = b; s_idx[t] = s_idx[t + w]; }
        }
        __syncthreads();
    }
    const float mx = s_val[0];
    const int amax = s_idx[0];
    __syncthreads();
    float e = 0.f;
    if (!p.greedy && v < p.V) e = exp2f((z - mx) * p.inv_T_log2e);
    s_val[t] = e;
    __syncthreads();
    for (int w = kVocabTile / 2; w > 0; w >>= 1) {
        if (t < w) s_val[t] += s_val[t + w];
        __syncthreads();
    }
    if (t == 0) {
        p.part_max[(size_t)tile * p.M + m] = mx;
        p.part_sum[(size_t)tile * p.M + m] = s_val[0];
        p.part_idx[(size_t)tile * p.M + m] = amax;
    }
}

}  // namespace

int lm_head_num_partials(int M, int V) { (void)M; return (V + kVocabTile - 1) / kVocabTile; }

cudaError_t launch_lm_head(const LmHeadParams& p, cudaStream_t stream) {
    if (p.logits == nullptr) return cudaErrorInvalidValue;
    lm_head_naive_kernel<<<(p.V + 7) / 8, 256, 0, stream>>>(p);
    tile_stats_kernel<<<dim3(lm_head_num_partials(p.M, p.V), p.M), kVocabTile, 0, stream>>>(p);
    count_launches(2);
    return cudaGetLastError();
}

}  // namespace massv
