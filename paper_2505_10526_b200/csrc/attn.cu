// Verify attention, first correct version: append the block's K/V, then one
// warp per (sequence, block row, query head) walks the cache with an online
// softmax in fp32.  (Sec. 2.1: the target scores the gamma+1 positions in one
// forward call.)
#include "kernels.cuh"

namespace massv {

namespace {

__device__ __forceinline__ size_t kv_offset(const AttnParams& p, int b, int pos, int g, int32_t* bad) {
    const int page = p.page_table[(size_t)b * p.max_pages + pos / kPageSize];
    if (page < 0 || page >= p.num_pages) { *bad = 1; return 0; }
    return (((size_t)page * p.Hkv + g) * kPageSize + (pos % kPageSize)) * p.d;
}

__global__ void kv_append_kernel(AttnParams p) {
    // one CTA per (sequence, row); threads copy Hkv*d elements as 16-byte words
    const int b = blockIdx.x / p.R, j = blockIdx.x % p.R;
    const int L = p.seq_lens[b];
    if (L < 0 || L + p.R > p.max_pages * kPageSize) { set_status(p.dev_status, MASSV_ERR_CAPACITY); return; }
    const int words = p.d / 8;
    for (int i = threadIdx.x; i < p.Hkv * words; i += blockDim.x) {
        const int g = i / words, w = i % words;
        int32_t bad = 0;
        const size_t dst = kv_offset(p, b, L + j, g, &bad);
        if (bad) { set_status(p.dev_status, MASSV_ERR_CAPACITY); continue; }
        const size_t src = (((size_t)b * p.R + j) * p.Hkv + g) * p.d;
        reinterpret_cast<uint4*>(p.k_pages + dst)[w] = reinterpret_cast<const uint4*>(p.k_new + src)[w];
        reinterpret_cast<uint4*>(p.v_pages + dst)[w] = reinterpret_cast<const uint4*>(p.v_new + src)[w];
    }
}

template <int D>
__global__ void __launch_bounds__(128) attn_naive_kernel(AttnParams p) {
    constexpr int E = D / 32;   // channels per lane
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int item = blockIdx.x * 4 + warp;
    if (item >= p.B * p.R * p.Hq) return;
    const int h = item % p.Hq, j = (item / p.Hq) % p.R, b = item / (p.Hq * p.R);
    const int g = h / (p.Hq / p.Hkv);
    const int L = p.seq_lens[b];
    if (L < 0 || L + p.R > p.max_pages * kPageSize) return;
    const int n_ctx = L + j + 1;
    const float scale_log2 = p.scale * 1.4426950408889634f;
    float qv[E], acc[E];
    for (int e = 0; e < E; ++e) {
        qv[e] = __bfloat162float(p.q[(size_t)item * D + lane * E + e]);
        acc[e] = 0.f;
    }
    float m = -INFINITY, l = 0.f;
    for (int i = 0; i < n_ctx; ++i) {
        int32_t bad = 0;
        const size_t off = kv_offset(p, b, i, g, &bad);
        if (bad) { set_status(p.dev_status, MASSV_ERR_CAPACITY); return; }
        float s = 0.f;
        for (int e = 0; e < E; ++e) s += qv[e] * __bfloat162float(p.k_pages[off + lane * E + e]);
        for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
        s *= scale_log2;
        const float m_new = fmaxf(m, s);
        const float corr = exp2f(m - m_new);
        const float w = exp2f(s - m_new);
        l = l * corr + w;
        // softmax weights are rounded to bf16 before multiplying V, as the tensor-core path does
        const float wb = __bfloat162float(__float2bfloat16(w));
        for (int e = 0; e < E; ++e) acc[e] = acc[e] * corr + wb * __bfloat162float(p.v_pages[off + lane * E + e]);
        m = m_new;
    }
    const float inv = 1.f / l;
    for (int e = 0; e < E; ++e) {
        const float o = acc[e] * inv;
        p.out[(size_t)item * D + lane * E + e] = __float2bfloat16(o);
        if (p.out_f32) p.out_f32[(size_t)item * D + lane * E + e] = o;
    }
    if (p.lse && lane == 0) p.lse[item] = (m + log2f(l)) * 0.6931471805599453f;
}

}  // namespace

int attn_rows_pad(int group_rows) { return (group_rows + 15) / 16 * 16; }

cudaError_t launch_verify_attn(const AttnParams& p, cudaStream_t stream) {
    kv_append_kernel<<<p.B * p.R, 128, 0, stream>>>(p);
    const int items = p.B * p.R * p.Hq;
    const int grid = (items + 3) / 4;
    switch (p.d) {
        case 64: attn_naive_kernel<64><<<grid, 128, 0, stream>>>(p); break;
        case 128: attn_naive_kernel<128><<<grid, 128, 0, stream>>>(p); break;
        case 256: attn_naive_kernel<256><<<grid, 128, 0, stream>>>(p); break;
        default: return cudaErrorInvalidValue;
    }
    count_launches(2);
    return cudaGetLastError();
}

}  // namespace massv
