// Total variation distance between the target's and the drafter's token
// distributions for every drafted position (paper Eq. 6):
//     TVD(p_j, q_j) = 1/2 * sum_v |p_j(v) - q_j(v)|,      p_j = softmax(z_j / T)
// and the acceptance probability of the rejection test, sum_v min(p_j(v), q_j(v)) = 1 - TVD.
// Three small kernels over fixed vocabulary slices, every reduction in a fixed order:
//   tvd_stats_kernel   per (row, slice): max logit and sum of exponentials (skipped when the caller hands in
//                      the statistics the acceptance call left behind: then the logits are read once);
//   tvd_sum_kernel     per (row, slice): merge the row's slice statistics, then sum |p-q| and min(p,q);
//   tvd_final_kernel   per row: add the slices in order.
#include "kernels.cuh"

namespace massv {

namespace {

constexpr int kThreadsTvd = 256;

// Sum over the block in a fixed tree; valid in thread 0.
__device__ __forceinline__ double block_sum(double x, double* sh) {
    sh[threadIdx.x] = x;
    __syncthreads();
    for (int w = kThreadsTvd / 2; w > 0; w >>= 1) {
        if (threadIdx.x < w) sh[threadIdx.x] += sh[threadIdx.x + w];
        __syncthreads();
    }
    const double r = sh[0];
    __syncthreads();
    return r;
}
__device__ __forceinline__ float block_max(float x, float* sh) {
    sh[threadIdx.x] = x;
    __syncthreads();
    for (int w = kThreadsTvd / 2; w > 0; w >>= 1) {
        if (threadIdx.x < w) sh[threadIdx.x] = fmaxf(sh[threadIdx.x], sh[threadIdx.x + w]);
        __syncthreads();
    }
    const float r = sh[0];
    __syncthreads();
    return r;
}

// Row r of the drafted positions = (sequence b, draft j): logits row b*(gamma+1)+j, q row b*gamma+j.
__device__ __forceinline__ const float* logits_row(const TvdParams& p, int row) {
    const int b = row / p.gamma, j = row % p.gamma;
    return p.logits + (size_t)(b * (p.gamma + 1) + j) * p.V;
}

__global__ void __launch_bounds__(kThreadsTvd) tvd_stats_kernel(TvdParams p) {
    __shared__ float shf[kThreadsTvd];
    __shared__ double shd[kThreadsTvd];
    pdl_wait();
    pdl_trigger();
    const int slice = blockIdx.x, row = blockIdx.y;
    const int v0 = slice * p.slice_len, v1 = min(p.V, v0 + p.slice_len);
    const float* z = logits_row(p, row);
    // one pass: every thread keeps a running (max, sum) over 16-byte loads, then the block merges
    float tm = -INFINITY, ts = 0.f;
    for (int v = v0 + 4 * threadIdx.x; v < v1; v += 4 * kThreadsTvd) {      // slices start at multiples of 4
        const float4 x = *reinterpret_cast<const float4*>(z + v);
        const float e[4] = {x.x, x.y, x.z, x.w};
        float cm = tm;
#pragma unroll
        for (int i = 0; i < 4; ++i) if (v + i < v1) cm = fmaxf(cm, e[i]);
        float cs = tm == -INFINITY ? 0.f : ts * expf((tm - cm) * p.inv_T);
#pragma unroll
        for (int i = 0; i < 4; ++i) if (v + i < v1) cs += expf((e[i] - cm) * p.inv_T);
        tm = cm; ts = cs;
    }
    const float m = block_max(tm, shf);
    double s = (tm == -INFINITY) ? 0.0 : (double)ts * (double)expf((tm - m) * p.inv_T);
    s = block_sum(s, shd);
    if (threadIdx.x == 0) {
        p.slice_max[row * kTvdSlices + slice] = m;
        p.slice_sum[row * kTvdSlices + slice] = s;
    }
}

__global__ void __launch_bounds__(kThreadsTvd) tvd_sum_kernel(TvdParams p) {
    __shared__ double shd[kThreadsTvd];
    pdl_wait();
    pdl_trigger();
    const int slice = blockIdx.x, row = blockIdx.y;
    float M = -INFINITY;
    double S = 0.0;
    if (p.row_stats) {
        // the acceptance scan's merged statistics of logits row b*(gamma+1)+j
        const int b = row / p.gamma, j = row % p.gamma;
        const float2 ms = *reinterpret_cast<const float2*>(p.row_stats + (size_t)(b * (p.gamma + 1) + j) * 2);
        M = ms.x;
        S = (double)ms.y;
    } else {
        for (int s = 0; s < kTvdSlices; ++s) M = fmaxf(M, p.slice_max[row * kTvdSlices + s]);
        for (int s = 0; s < kTvdSlices; ++s) {
            const float ms = p.slice_max[row * kTvdSlices + s];
            if (ms > -INFINITY) S += p.slice_sum[row * kTvdSlices + s] * (double)expf((ms - M) * p.inv_T);
        }
    }
    const float inv_sum = (float)(1.0 / S);
    const int v0 = slice * p.slice_len, v1 = min(p.V, v0 + p.slice_len);
    const float* z = logits_row(p, row);
    const float* q = p.draft_probs + (size_t)row * p.V;
    double a = 0.0, mn = 0.0;
    for (int v = v0 + 4 * threadIdx.x; v < v1; v += 4 * kThreadsTvd) {
        const float4 x = *reinterpret_cast<const float4*>(z + v);
        const float4 y = __ldg(reinterpret_cast<const float4*>(q + v));
        const float e[4] = {x.x, x.y, x.z, x.w}, f[4] = {y.x, y.y, y.z, y.w};
        float fa = 0.f, fm = 0.f;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            if (v + i < v1) {
                const float pv = expf((e[i] - M) * p.inv_T) * inv_sum;
                fa += fabsf(pv - f[i]);
                fm += fminf(pv, f[i]);
            }
        }
        a += (double)fa;
        mn += (double)fm;
    }
    a = block_sum(a, shd);
    mn = block_sum(mn, shd);
    if (threadIdx.x == 0) {
        p.slice_abs[row * kTvdSlices + slice] = a;
        p.slice_min[row * kTvdSlices + slice] = mn;
    }
}

__global__ void tvd_final_kernel(TvdParams p) {
    pdl_wait();
    const int row = blockIdx.x * blockDim.x + threadIdx.x;
    if (row >= p.B * p.gamma) return;
    double a = 0.0, mn = 0.0;
    for (int s = 0; s < kTvdSlices; ++s) { a += p.slice_abs[row * kTvdSlices + s]; mn += p.slice_min[row * kTvdSlices + s]; }
    p.tvd_out[row] = (float)(0.5 * a);
    if (p.accept_prob_out) p.accept_prob_out[row] = (float)mn;
}

}  // namespace

cudaError_t launch_tvd(const TvdParams& p, cudaStream_t stream) {
    const int rows = p.B * p.gamma;
    cudaError_t e = cudaSuccess;
    if (!p.row_stats) {
        e = launch_pdl(tvd_stats_kernel, dim3(kTvdSlices, rows), dim3(kThreadsTvd), 0, stream, p);
        if (e != cudaSuccess) return e;
        count_launches(1);
    }
    e = launch_pdl(tvd_sum_kernel, dim3(kTvdSlices, rows), dim3(kThreadsTvd), 0, stream, p);
    if (e != cudaSuccess) return e;
    e = launch_pdl(tvd_final_kernel, dim3((rows + 127) / 128), dim3(128), 0, stream, p);
    if (e != cudaSuccess) return e;
    count_launches(2);
    return cudaGetLastError();
}

}  // namespace massv
