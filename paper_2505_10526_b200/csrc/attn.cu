// Verify attention: the gamma+1 block rows of every sequence attend the paged
// KV cache (Sec. 2.1: the target scores positions t+1..t+gamma+1 in one forward
// call; Sec. 2.2: the cache holds image tokens, then text, then the block).
//
// The scan over the cache is bound by HBM.  All G*(gamma+1) query rows that share
// a KV head are processed by the same CTA so that every K/V byte is read once.
// Work item = (sequence, KV head, chunk of kv_chunk positions); grid =
// (max_chunks, Hkv, B) and CTAs whose chunk lies beyond the sequence retire at
// once, so the hardware scheduler balances ragged lengths.  Inside a CTA a
// producer warp streams 64-token (32-token at d = 256) K/V tiles page by page with TMA (16 x 64 boxes,
// 128-byte swizzle) into an mbarrier ring; consumer warps run
// Q K^T and P V on warp-level tensor-core MMAs (m16n8k16, bf16 -> fp32) with an
// online softmax in registers: warp (mt, ts) owns 16 query rows and a 64/TS-token
// slice of every tile.  Partial (max, sum, O) of the warps are merged through
// shared memory; sequences that span several chunks are merged by a second
// kernel.  The block's own K/V rows are appended by the CTA whose chunk holds
// their positions.  All reductions have a fixed order.
#include "kernels.cuh"
#include "ptx.cuh"

namespace massv {

namespace {

constexpr int kChunkAlign = 64;      // kv_chunk granularity (a multiple of every tile size)
constexpr int kMaxChunkPages = 256;  // kv_chunk <= 4096 tokens

__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(addr));
}
// d += a(16x16, row) * b(16x8, col), bf16 inputs, fp32 accumulate
__device__ __forceinline__ void mma_bf16(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<const uint32_t*>(&v);
}

// Byte offset of the 16-byte unit `unit` (0..7) of row `row` inside a region of
// 128-byte rows laid out with the 128-byte swizzle (what TMA writes).
__device__ __forceinline__ uint32_t swz(int row, int unit) { return (uint32_t)(row * 128 + ((unit ^ (row & 7)) << 4)); }

// TILE = tokens per pipeline stage (32 or 64).  DEEP: the CTA has an SM to itself (five
// warps), so the ring is twice as deep to keep enough bytes in flight.
template <int D, int TILE, bool DEEP>
struct AttnCfg {
    static constexpr int kChunks = D / 64;                 // 64-element column groups of a row
    static constexpr int kRegion = TILE * 128;             // bytes of one (TILE tokens x 64 elements) region
    static constexpr int kBytesK = kChunks * kRegion;
    static constexpr int kStageBytes = 2 * kBytesK;        // K then V
    static constexpr int kStages = DEEP ? 6 : ((D == 64) ? 4 : 3);
};

// Two CTAs should share an SM (one CTA's set-up and merge hide behind the other's
// streaming).  Each scheduler owns a quarter of the register file and a CTA's warps are
// dealt round-robin, so that needs at most four warps per CTA, producer included.
template <int D, int MT, int TS, int TILE>
__global__ void __launch_bounds__((MT * TS + 1) * 32, (MT * TS + 1) <= 4 ? 2 : 1)
attn_split_kernel(const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_v, const AttnParams p) {
    using Cfg = AttnCfg<D, TILE, (MT * TS + 1 > 4)>;
    constexpr int kTile = TILE;
    constexpr int NW = MT * TS;            // consumer warps
    constexpr int NT = kTile / TS;         // tokens of a tile owned by one warp
    constexpr int RP = MT * 16;            // padded query rows
    constexpr int NCH = Cfg::kChunks;
    constexpr bool kQInRegs = D <= 128;

    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t full_bar[Cfg::kStages];
    __shared__ __align__(8) uint64_t empty_bar[Cfg::kStages];
    __shared__ int s_pages[kMaxChunkPages];
    __shared__ int abort_flag;

    const int chunk = blockIdx.x, g = blockIdx.y, b = blockIdx.z;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    pdl_wait();
    const int L = p.seq_lens[b];
    if (L < 0 || L + p.R > p.max_pages * kPageSize) {            // no room for the block: skip the sequence
        if (chunk == 0 && g == 0 && threadIdx.x == 0) set_status(p.dev_status, MASSV_ERR_CAPACITY);
        return;
    }
    const int n_ctx = L + p.R;
    if (chunk * p.kv_chunk >= n_ctx) return;
    // Sliding window: block row j (position L + j) sees positions L + j - window + 1 .. L + j, so
    // nothing before row 0's lower bound is needed.  Chunks wholly before it retire, and the
    // first needed chunk starts at the tile that holds the bound.
    const int lo_min = p.window > 0 ? max(0, L - p.window + 1) : 0;
    const int first_chunk = lo_min / p.kv_chunk;
    if (chunk < first_chunk) return;
    int c_begin = chunk * p.kv_chunk;
    if (chunk == first_chunk) c_begin += ((lo_min - c_begin) / kTile) * kTile;
    const int c_end = min(n_ctx, chunk * p.kv_chunk + p.kv_chunk);
    const int n_tiles = (c_end - c_begin + kTile - 1) / kTile;
    const int n_chunks_b = (n_ctx + p.kv_chunk - 1) / p.kv_chunk - first_chunk;     // chunks that take part
    const int G = p.Hq / p.Hkv;
    const int rows = G * p.R;

    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint8_t* q_smem = smem + Cfg::kStages * Cfg::kStageBytes;    // [NCH][RP rows][128 B], swizzled

    if (threadIdx.x == 0) {
        for (int s = 0; s < Cfg::kStages; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], NW); }
        abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    {   // page ids of this chunk and the query rows (row r = block_row * G + head_in_group)
        const int n_pages = (c_end - c_begin + kPageSize - 1) / kPageSize;
        for (int i = threadIdx.x; i < n_pages; i += blockDim.x)
            s_pages[i] = p.page_table[(size_t)b * p.max_pages + c_begin / kPageSize + i];
        constexpr int UPR = D / 8;   // 16-byte units per row
        for (int i = threadIdx.x; i < RP * UPR; i += blockDim.x) {
            const int r = i / UPR, u = i % UPR;
            uint4 v = make_uint4(0u, 0u, 0u, 0u);
            if (r < rows) {
                const int j = r / G, hh = r % G;
                v = *reinterpret_cast<const uint4*>(p.q + (((size_t)b * p.R + j) * p.Hq + g * G + hh) * D + u * 8);
            }
            *reinterpret_cast<uint4*>(q_smem + (u / 8) * (RP * 128) + swz(r, u % 8)) = v;
        }
    }
    __syncthreads();
    volatile int* abort_ptr = &abort_flag;

    float o[D / 8][4];
    float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};
    const int mt = warp / TS, ts = warp % TS;

    if (warp == NW) {
        // ------------------------------------------------ TMA producer
        // A tile is 2 * (d/64) boxes per page.  One box per lane: a single thread issuing them one
        // after the other cannot keep an SM's share of HBM busy when the CTA has the SM to itself.
        uint64_t policy;
        asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(policy));
        for (int t = 0; t < n_tiles; ++t) {
            const int s = t % Cfg::kStages;
            const uint32_t ph = ((uint32_t)(t / Cfg::kStages)) & 1u;
            int freed = 0;
            if (lane == 0) freed = mbar_wait(&empty_bar[s], ph ^ 1u, abort_ptr) ? 1 : 0;
            freed = __shfl_sync(0xffffffffu, freed, 0);
            if (!freed) break;
            const int tile_start = c_begin + t * kTile;
            int n_pg = (c_end - tile_start + kPageSize - 1) / kPageSize;
            if (n_pg > kTile / kPageSize) n_pg = kTile / kPageSize;
            uint8_t* kdst = smem + (size_t)s * Cfg::kStageBytes;
            if (lane == 0) mbar_expect_tx(&full_bar[s], (uint32_t)(n_pg * NCH * 2048 * 2));
            __syncwarp();
            for (int i = lane; i < n_pg * NCH * 2; i += 32) {
                const int is_v = i & 1, dc = (i >> 1) % NCH, pg = i / (2 * NCH);
                int pid = s_pages[t * (kTile / kPageSize) + pg];
                if (pid < 0 || pid >= p.num_pages) { set_status(p.dev_status, MASSV_ERR_CAPACITY); pid = 0; }
                const int row = (pid * p.Hkv + g) * kPageSize;
                tma_load_2d(kdst + is_v * Cfg::kBytesK + dc * Cfg::kRegion + pg * 2048, is_v ? &map_v : &map_k, dc * 64, row,
                            &full_bar[s], policy);
            }
        }
        if (lane == 0 && *abort_ptr) {
            for (int i = 0; i < 64; ++i) __nanosleep(2000);   // let copies in flight land
        }
    } else {
        // ------------------------------------------------ consumers
#pragma unroll
        for (int n = 0; n < D / 8; ++n) { o[n][0] = o[n][1] = o[n][2] = o[n][3] = 0.f; }
        const float scale_log2 = p.scale * 1.4426950408889634f;
        const int r0 = mt * 16 + (lane >> 2), r1 = r0 + 8;
        // block row of each of this thread's two query rows (padding rows behave like the last block row)
        const int j0 = r0 < rows ? r0 / G : p.R - 1, j1 = r1 < rows ? r1 / G : p.R - 1;
        const uint32_t q_base = smem_u32(q_smem);
        // ldmatrix lane roles: matrix (lane >> 3), row (lane & 7) inside it
        const int lm = lane >> 3, lr = lane & 7;
        uint32_t qf[kQInRegs ? D / 16 : 1][4];
        if (kQInRegs) {
#pragma unroll
            for (int kk = 0; kk < D / 16; ++kk) {
                const int row = mt * 16 + (lm & 1) * 8 + lr, unit = (kk & 3) * 2 + (lm >> 1);
                ldmatrix_x4(qf[kk], q_base + (kk >> 2) * (RP * 128) + swz(row, unit));
            }
        }
        bool ok = true;
        for (int t = 0; t < n_tiles && ok; ++t) {
            const int s = t % Cfg::kStages;
            const uint32_t ph = ((uint32_t)(t / Cfg::kStages)) & 1u;
            if (!mbar_wait(&full_bar[s], ph, abort_ptr)) { ok = false; break; }
            const int tile_start = c_begin + t * kTile;
            const int valid = min(kTile, c_end - tile_start);
            uint8_t* kst = smem + (size_t)s * Cfg::kStageBytes;
            uint8_t* vst = kst + Cfg::kBytesK;
            if (tile_start + kTile > L) {
                constexpr int UPR = D / 8;
                // Append: the block's K/V rows (positions L .. L+gamma) are not in the cache yet.
                // The warp that owns those tokens puts them into the tile in shared memory, and
                // the mt == 0 warp also stores them to their page slots.
                const int p_first = max(L, tile_start + ts * NT), p_last = min(n_ctx, tile_start + ts * NT + NT);
                for (int i = lane; i < (p_last - p_first) * UPR; i += 32) {
                    const int pos = p_first + i / UPR, u = i % UPR, row = pos - tile_start;
                    const size_t src = (((size_t)b * p.R + (pos - L)) * p.Hkv + g) * D + u * 8;
                    const uint4 kv = *reinterpret_cast<const uint4*>(p.k_new + src);
                    const uint4 vv = *reinterpret_cast<const uint4*>(p.v_new + src);
                    *reinterpret_cast<uint4*>(kst + (u / 8) * Cfg::kRegion + swz(row, u % 8)) = kv;
                    *reinterpret_cast<uint4*>(vst + (u / 8) * Cfg::kRegion + swz(row, u % 8)) = vv;
                    if (mt == 0) {
                        const int pid = s_pages[(pos - c_begin) / kPageSize];
                        if (pid >= 0 && pid < p.num_pages) {
                            const size_t dst = (((size_t)pid * p.Hkv + g) * kPageSize + (pos % kPageSize)) * D + u * 8;
                            *reinterpret_cast<uint4*>(p.k_pages + dst) = kv;
                            *reinterpret_cast<uint4*>(p.v_pages + dst) = vv;
                        }
                    }
                }
                // Rows past the end of the context hold stale bytes; their weights are zero, but
                // 0 * NaN would still poison P V, so clear the V rows this warp will read.
                const int first = max(valid, ts * NT), last = ts * NT + NT;
                for (int i = lane; i < (last - first) * UPR; i += 32) {
                    const int row = first + i / UPR, u = i % UPR;
                    *reinterpret_cast<uint4*>(vst + (u / 8) * Cfg::kRegion + swz(row, u % 8)) = make_uint4(0u, 0u, 0u, 0u);
                }
                __syncwarp();
            }
            const uint32_t k_base = smem_u32(kst), v_base = smem_u32(vst);

            // ---- S = Q K^T for this warp's 16 rows x NT tokens
            float sacc[NT / 8][4];
#pragma unroll
            for (int n = 0; n < NT / 8; ++n) { sacc[n][0] = sacc[n][1] = sacc[n][2] = sacc[n][3] = 0.f; }
#pragma unroll
            for (int kk = 0; kk < D / 16; ++kk) {
                uint32_t a[4];
                if (kQInRegs) {
                    a[0] = qf[kk][0]; a[1] = qf[kk][1]; a[2] = qf[kk][2]; a[3] = qf[kk][3];
                } else {
                    const int row = mt * 16 + (lm & 1) * 8 + lr, unit = (kk & 3) * 2 + (lm >> 1);
                    ldmatrix_x4(a, q_base + (kk >> 2) * (RP * 128) + swz(row, unit));
                }
#pragma unroll
                for (int tg = 0; tg < NT / 16; ++tg) {
                    uint32_t bf[4];
                    const int tok = ts * NT + tg * 16 + (lm >> 1) * 8 + lr, unit = (kk & 3) * 2 + (lm & 1);
                    ldmatrix_x4(bf, k_base + (kk >> 2) * Cfg::kRegion + swz(tok, unit));
                    mma_bf16(sacc[2 * tg], a, bf[0], bf[1]);
                    mma_bf16(sacc[2 * tg + 1], a, bf[2], bf[3]);
                }
            }

            // ---- scale, causal mask, online softmax
            // some position in the tile is hidden from some block row: ahead of row 0, or (with a
            // window) older than the last row's lower bound
            const bool need_mask = tile_start + kTile > L + 1 || (p.window > 0 && tile_start < n_ctx - p.window);
            float mx0 = -INFINITY, mx1 = -INFINITY;
#pragma unroll
            for (int n = 0; n < NT / 8; ++n) {
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    float sv = sacc[n][e] * scale_log2;
                    if (need_mask) {
                        const int pos = tile_start + ts * NT + n * 8 + 2 * (lane & 3) + (e & 1);
                        const int row_pos = L + (e < 2 ? j0 : j1);
                        if (pos > row_pos || (p.window > 0 && pos < row_pos - p.window + 1)) sv = -INFINITY;
                    }
                    sacc[n][e] = sv;
                    if (e < 2) mx0 = fmaxf(mx0, sv); else mx1 = fmaxf(mx1, sv);
                }
            }
            mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 1));
            mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 2));
            mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 1));
            mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 2));
            const float mn0 = fmaxf(m_run[0], mx0), mn1 = fmaxf(m_run[1], mx1);
            const float ms0 = mn0 == -INFINITY ? 0.f : mn0, ms1 = mn1 == -INFINITY ? 0.f : mn1;
            const float corr0 = exp2f(m_run[0] - ms0), corr1 = exp2f(m_run[1] - ms1);
            m_run[0] = mn0; m_run[1] = mn1;
            float ls0 = 0.f, ls1 = 0.f;
            uint32_t pa[NT / 16][4];
#pragma unroll
            for (int n = 0; n < NT / 8; ++n) {
                const float p0 = exp2f(sacc[n][0] - ms0), p1 = exp2f(sacc[n][1] - ms0);
                const float p2 = exp2f(sacc[n][2] - ms1), p3 = exp2f(sacc[n][3] - ms1);
                ls0 += p0 + p1; ls1 += p2 + p3;
                // accumulator layout -> A-operand layout of the P V product
                pa[n >> 1][(n & 1) * 2 + 0] = pack_bf16(p0, p1);
                pa[n >> 1][(n & 1) * 2 + 1] = pack_bf16(p2, p3);
            }
            l_run[0] = l_run[0] * corr0 + ls0;
            l_run[1] = l_run[1] * corr1 + ls1;
#pragma unroll
            for (int n = 0; n < D / 8; ++n) { o[n][0] *= corr0; o[n][1] *= corr0; o[n][2] *= corr1; o[n][3] *= corr1; }

            // ---- O += P V
#pragma unroll
            for (int tk = 0; tk < NT / 16; ++tk) {
#pragma unroll
                for (int dp = 0; dp < D / 16; ++dp) {
                    uint32_t bf[4];
                    const int tok = ts * NT + tk * 16 + (lm & 1) * 8 + lr, du = dp * 2 + (lm >> 1);
                    ldmatrix_x4_trans(bf, v_base + (du >> 3) * Cfg::kRegion + swz(tok, du & 7));
                    mma_bf16(o[2 * dp], pa[tk], bf[0], bf[1]);
                    mma_bf16(o[2 * dp + 1], pa[tk], bf[2], bf[3]);
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(&empty_bar[s]);
        }
        l_run[0] += __shfl_xor_sync(0xffffffffu, l_run[0], 1);
        l_run[0] += __shfl_xor_sync(0xffffffffu, l_run[0], 2);
        l_run[1] += __shfl_xor_sync(0xffffffffu, l_run[1], 1);
        l_run[1] += __shfl_xor_sync(0xffffffffu, l_run[1], 2);
    }

    // ---------------------------------------------------- merge the warps' partial results
    __syncthreads();                         // every tile has been consumed: the ring can be reused
    pdl_trigger();
    float* st_o = reinterpret_cast<float*>(smem);            // [TS][RP][D]
    float* st_m = st_o + TS * RP * D;                        // [TS][RP]
    float* st_l = st_m + TS * RP;
    if (warp < NW) {
        const int r0 = mt * 16 + (lane >> 2), r1 = r0 + 8;
        float* base = st_o + (size_t)ts * RP * D;
#pragma unroll
        for (int n = 0; n < D / 8; ++n) {
            const int c = n * 8 + 2 * (lane & 3);
            *reinterpret_cast<float2*>(base + r0 * D + c) = make_float2(o[n][0], o[n][1]);
            *reinterpret_cast<float2*>(base + r1 * D + c) = make_float2(o[n][2], o[n][3]);
        }
        if ((lane & 3) == 0) {
            st_m[ts * RP + r0] = m_run[0]; st_l[ts * RP + r0] = l_run[0];
            st_m[ts * RP + r1] = m_run[1]; st_l[ts * RP + r1] = l_run[1];
        }
    }
    __syncthreads();
    if (abort_flag) {
        if (threadIdx.x == 0) set_status(p.dev_status, MASSV_ERR_TIMEOUT);
        return;
    }
    const bool single = n_chunks_b == 1;
    const size_t item = ((size_t)b * p.Hkv + g) * p.max_chunks + chunk;
    for (int i = threadIdx.x; i < rows * (D / 4); i += blockDim.x) {
        const int r = i / (D / 4), c = (i % (D / 4)) * 4;
        float M = -INFINITY;
#pragma unroll
        for (int w = 0; w < TS; ++w) M = fmaxf(M, st_m[w * RP + r]);
        float Lsum = 0.f;
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int w = 0; w < TS; ++w) {
            const float mw = st_m[w * RP + r];
            const float f = mw == -INFINITY ? 0.f : exp2f(mw - M);
            Lsum += st_l[w * RP + r] * f;
            const float4 v = *reinterpret_cast<const float4*>(st_o + ((size_t)w * RP + r) * D + c);
            acc.x += v.x * f; acc.y += v.y * f; acc.z += v.z * f; acc.w += v.w * f;
        }
        if (single) {
            const int j = r / G, hh = r % G;
            const size_t dst = (((size_t)b * p.R + j) * p.Hq + g * G + hh) * D + c;
            const float inv = 1.f / Lsum;
            acc.x *= inv; acc.y *= inv; acc.z *= inv; acc.w *= inv;
            uint2 packed;
            packed.x = pack_bf16(acc.x, acc.y);
            packed.y = pack_bf16(acc.z, acc.w);
            *reinterpret_cast<uint2*>(p.out + dst) = packed;
            if (p.out_f32) *reinterpret_cast<float4*>(p.out_f32 + dst) = acc;
            if (p.lse && c == 0) p.lse[((size_t)b * p.R + j) * p.Hq + g * G + hh] = (M + log2f(Lsum)) * 0.6931471805599453f;
        } else {
            *reinterpret_cast<float4*>(p.part_o + (item * RP + r) * D + c) = acc;
            if (c == 0) { p.part_ml[(item * RP + r) * 2] = M; p.part_ml[(item * RP + r) * 2 + 1] = Lsum; }
        }
    }
}

// Merge the chunks of sequences that span more than one: one CTA per
// (sequence, KV head, query row), one thread per channel.
constexpr int kCombineMaxChunks = 1024;
__global__ void __launch_bounds__(128) attn_combine_kernel(const AttnParams p, int rows_pad) {
    const int G = p.Hq / p.Hkv, rows = G * p.R;
    const int r = blockIdx.x % rows, g = (blockIdx.x / rows) % p.Hkv, b = blockIdx.x / (rows * p.Hkv);
    pdl_wait();
    pdl_trigger();
    const int L = p.seq_lens[b];
    if (L < 0 || L + p.R > p.max_pages * kPageSize) return;
    const int first_chunk = (p.window > 0 ? max(0, L - p.window + 1) : 0) / p.kv_chunk;   // as in the split kernel
    const int n_chunks = (L + p.R + p.kv_chunk - 1) / p.kv_chunk - first_chunk;
    if (n_chunks <= 1) return;
    __shared__ float s_w[kCombineMaxChunks];    // first the chunk maxima, then the merge weights
    __shared__ float s_l[kCombineMaxChunks];
    const size_t item0 = ((size_t)b * p.Hkv + g) * p.max_chunks + first_chunk;
    for (int c = threadIdx.x; c < n_chunks; c += blockDim.x) {
        const float2 ml = *reinterpret_cast<const float2*>(p.part_ml + ((item0 + c) * rows_pad + r) * 2);
        s_w[c] = ml.x;
        s_l[c] = ml.y;
    }
    __syncthreads();
    float M = -INFINITY;
    for (int c = 0; c < n_chunks; ++c) M = fmaxf(M, s_w[c]);
    __syncthreads();
    for (int c = threadIdx.x; c < n_chunks; c += blockDim.x) s_w[c] = s_w[c] == -INFINITY ? 0.f : exp2f(s_w[c] - M);
    __syncthreads();
    float Lsum = 0.f;
    for (int c = 0; c < n_chunks; ++c) Lsum += s_l[c] * s_w[c];
    const float inv = 1.f / Lsum;
    const int j = r / G, hh = r % G;
    const size_t row_out = ((size_t)b * p.R + j) * p.Hq + g * G + hh;
    const float* src = p.part_o + (item0 * rows_pad + r) * p.d;
    const size_t chunk_stride = (size_t)rows_pad * p.d;
    for (int col = threadIdx.x; col < p.d; col += blockDim.x) {
        float acc = 0.f;
        int c = 0;
        for (; c + 4 <= n_chunks; c += 4) {      // four independent loads in flight, summed in chunk order
            const float v0 = src[(size_t)c * chunk_stride + col], v1 = src[(size_t)(c + 1) * chunk_stride + col];
            const float v2 = src[(size_t)(c + 2) * chunk_stride + col], v3 = src[(size_t)(c + 3) * chunk_stride + col];
            acc += v0 * s_w[c]; acc += v1 * s_w[c + 1]; acc += v2 * s_w[c + 2]; acc += v3 * s_w[c + 3];
        }
        for (; c < n_chunks; ++c) acc += src[(size_t)c * chunk_stride + col] * s_w[c];
        acc *= inv;
        p.out[row_out * p.d + col] = __float2bfloat16(acc);
        if (p.out_f32) p.out_f32[row_out * p.d + col] = acc;
    }
    if (p.lse && threadIdx.x == 0) p.lse[row_out] = (M + log2f(Lsum)) * 0.6931471805599453f;
}

template <int D, int MT, int TS, int TILE>
cudaError_t launch_split(const AttnParams& p, const CUtensorMap& mk, const CUtensorMap& mv, cudaStream_t stream) {
    using Cfg = AttnCfg<D, TILE, (MT * TS + 1 > 4)>;
    constexpr int RP = MT * 16;
    const size_t ring = (size_t)Cfg::kStages * Cfg::kStageBytes;
    static_assert((size_t)TS * RP * D * 4 + 2 * TS * RP * 4 <= (size_t)Cfg::kStages * Cfg::kStageBytes, "merge staging fits the ring");
    const size_t smem = ring + (size_t)RP * D * 2 + 1024;
    cudaError_t e = cudaFuncSetAttribute(attn_split_kernel<D, MT, TS, TILE>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    return launch_pdl(attn_split_kernel<D, MT, TS, TILE>, dim3(p.max_chunks, p.Hkv, p.B), dim3((MT * TS + 1) * 32), smem, stream, mk, mv, p);
}

template <int D>
cudaError_t launch_split_d(const AttnParams& p, int mt, const CUtensorMap& mk, const CUtensorMap& mv, cudaStream_t stream) {
    switch (mt) {
        // d = 256 uses 32-token stages so that two CTAs (three 32 KB stages each) share an SM and
        // one CTA's set-up and merge overlap the other's streaming
        case 1: return D == 256 ? launch_split<D, 1, 2, 32>(p, mk, mv, stream) : launch_split<D, 1, 2, 64>(p, mk, mv, stream);
        case 2: return D == 256 ? launch_split<D, 2, 1, 32>(p, mk, mv, stream) : launch_split<D, 2, 1, 64>(p, mk, mv, stream);
        case 3: return D == 256 ? launch_split<D, 3, 1, 32>(p, mk, mv, stream) : launch_split<D, 3, 1, 64>(p, mk, mv, stream);
        case 4: return D == 256 ? launch_split<D, 4, 1, 32>(p, mk, mv, stream) : launch_split<D, 4, 1, 64>(p, mk, mv, stream);
        default: return cudaErrorInvalidValue;
    }
}

}  // namespace

int attn_rows_pad(int group_rows) { return (group_rows + 15) / 16 * 16; }

// Which split kernel runs.  The warp-MMA kernel re-reads every K/V tile from shared memory once
// per 16 query rows, which saturates the shared-memory pipe from about 48 rows up; the tcgen05
// kernel reads each tile once whatever the row count, and with its balanced schedule it is the
// faster one on every head_dim <= 128 shape measured.  At head_dim 256 its ring leaves room for one
// CTA per SM only, and the warp-MMA kernel (few rows per KV head on such models) stays ahead.
bool attn_use_umma(const AttnParams& p) {
    if (p.path == 1 || !attn_umma_supported(p)) return false;
    if (p.path == 2) return true;
    return p.d <= 128;
}

cudaError_t launch_verify_attn(const AttnParams& p, cudaStream_t stream) {
    if (p.kv_chunk % kChunkAlign != 0 || p.kv_chunk > kMaxChunkPages * kPageSize) return cudaErrorInvalidValue;
    CUtensorMap mk, mv;
    const uint64_t rows_total = (uint64_t)p.num_pages * p.Hkv * kPageSize;
    if (!make_tensor_map_bf16_2d(&mk, p.k_pages, rows_total, p.d, kPageSize) ||
        !make_tensor_map_bf16_2d(&mv, p.v_pages, rows_total, p.d, kPageSize))
        return cudaErrorInvalidValue;
    const int rows = (p.Hq / p.Hkv) * p.R;
    const int mt = attn_rows_pad(rows) / 16;
    cudaError_t e;
    const TimingHooks& hooks = timing_hooks();
    if (hooks.attn_start && cudaEventRecord(hooks.attn_start, stream) != cudaSuccess) return cudaGetLastError();
    if (attn_use_umma(p)) {
        const bool flat = !p.chunk_forced && attn_umma_flat_supported(p);
        int launched = 0;
        e = launch_attn_umma(p, mk, mv, stream, flat, &launched, hooks.attn_stop);
        if (e != cudaSuccess) return e;
        if (flat) {
            count_launches(launched);
            return cudaGetLastError();
        }
    } else {
        switch (p.d) {
            case 64: e = launch_split_d<64>(p, mt, mk, mv, stream); break;
            case 128: e = launch_split_d<128>(p, mt, mk, mv, stream); break;
            case 256: e = launch_split_d<256>(p, mt, mk, mv, stream); break;
            default: return cudaErrorInvalidValue;
        }
    }
    if (e != cudaSuccess) return e;
    if (hooks.attn_stop && cudaEventRecord(hooks.attn_stop, stream) != cudaSuccess) return cudaGetLastError();
    int launched = 1;
    if (p.max_chunks > 1) {
        if (p.max_chunks > kCombineMaxChunks) return cudaErrorInvalidValue;
        e = launch_pdl(attn_combine_kernel, dim3(p.B * p.Hkv * rows), dim3(p.d < 128 ? 64 : 128), 0, stream, p, attn_rows_pad(rows));
        if (e != cudaSuccess) return e;
        launched = 2;
    }
    count_launches(launched);
    return cudaGetLastError();
}

}  // namespace massv
