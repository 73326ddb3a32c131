// Verify attention on the 5th-generation tensor cores (Sec. 2.1: the gamma+1 block
// rows of a sequence attend the whole cache in one pass of the target model).
//
// Same work split as the warp-MMA kernel (CTA = sequence x KV head x chunk of the
// cache; all G*(gamma+1) query rows of the KV head share the CTA, so every K/V byte
// is read once), but both products run as tcgen05.mma with M = 64 query rows and
// the operands read straight from shared memory, so no K/V fragment ever passes
// through registers:
//
//   S[64, TILE]  = Q[64, d] K_tile^T         K tile as TMA wrote it: K-major, 128-byte swizzle
//   O[64, d]    += P[64, TILE] V_tile        V tile as TMA wrote it: [token][d] = MN-major B operand
//
// S (double buffered) and O live in tensor memory.  Warp roles: warp 0 streams K and V
// tiles page by page with TMA into a ring and patches the block's own K/V rows into
// the tiles that hold their positions (and stores them to their page slots: the
// append); one thread of warp 1 issues the MMAs; warps 2-5 own 16 query rows each:
// they read S with tcgen05.ld (16x256b: the same fragment layout as a warp-level MMA
// accumulator), apply scale, causal / window mask and the online softmax, and write P
// as bf16 into shared memory for the second product.  O is rescaled in tensor memory
// only when a row's running maximum has grown by more than 2^8 since its reference
// was set (the reference cancels in O / l, so the result is the plain softmax).
// Sequences that span several chunks are merged by attn_combine_kernel.
#include "kernels.cuh"
#include "ptx.cuh"
#include "umma.cuh"

namespace massv {

namespace {

constexpr int kUmmaRows = 64;          // MMA M: query rows per KV head, padded
constexpr int kUmmaThreads = 192;      // producer warp, MMA warp, four softmax warps
constexpr int kUmmaMaxChunkPages = 256;
constexpr float kRescaleThreshold = 8.f;   // log2 units

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
    const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<const uint32_t*>(&v);
}
__device__ __forceinline__ uint32_t swz128(int row, int unit) { return (uint32_t)(row * 128 + ((unit ^ (row & 7)) << 4)); }

// 16 TMEM lanes x 64 columns -> 32 registers per thread.  Register 4k+e holds row
// (lane/4 + 8*(e>>1)), column 8k + 2*(lane%4) + (e&1) of the 16 x 64 block.
__device__ __forceinline__ void tmem_ld_16x64(uint32_t taddr, uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.16x256b.x8.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
          "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
          "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr));
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int j = 0; j < 32; ++j) asm volatile("" : "+r"(r[j]));      // no use may move ahead of the wait
}
__device__ __forceinline__ void tmem_st_16x64(uint32_t taddr, const uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.st.sync.aligned.16x256b.x8.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
        "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};" ::"r"(taddr),
        "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]), "r"(r[10]),
        "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]), "r"(r[20]),
        "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]),
        "r"(r[31])
        : "memory");
}

template <int D, int TILE>
struct UmmaAttnCfg {
    static constexpr int kNCH = D / 64;                       // 64-element column groups of a K/V row
    static constexpr int kRegion = TILE * 128;                // bytes of one (TILE tokens x 64 elements) region
    static constexpr int kEntryBytes = kNCH * kRegion;        // one K tile or one V tile
    static constexpr int kEntries = 5;                        // ring entries, filled in the order the MMAs consume them
    static constexpr int kQRegion = kUmmaRows * 128;          // (64 rows x 64 elements)
    static constexpr int kQBytes = kNCH * kQRegion;
    static constexpr int kPBytes = (TILE / 64) * kQRegion;    // P tile: 64 rows x TILE tokens, K-major
    static constexpr int kSmem = kEntries * kEntryBytes + kQBytes + kPBytes + 1024;
    static constexpr int kColsNeeded = 2 * TILE + D;          // two S buffers and O
    static constexpr int kTmemCols = kColsNeeded <= 256 ? 256 : 512;
    static constexpr int kCtasPerSm = (kSmem <= 110 * 1024 && kTmemCols <= 256) ? 2 : 1;
};

// The MMA thread consumes tiles in the order K_0, K_1, V_0, K_2, V_1, ..., K_{n-1}, V_{n-2}, V_{n-1}
// (the score product runs two tiles ahead of the softmax).  The ring is filled in the same order,
// so an entry is never held by a tile that is not needed yet.
__device__ __forceinline__ int ring_item_of_k(int t) { return t == 0 ? 0 : 2 * t - 1; }
__device__ __forceinline__ int ring_item_of_v(int t, int n_tiles) { return t == n_tiles - 1 ? 2 * n_tiles - 1 : 2 * t + 2; }

template <int D, int TILE>
__global__ void __launch_bounds__(kUmmaThreads, UmmaAttnCfg<D, TILE>::kCtasPerSm)
attn_umma_kernel(const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_v, const AttnParams p) {
    using Cfg = UmmaAttnCfg<D, TILE>;
    constexpr int E = Cfg::kEntries;
    constexpr int NCH = Cfg::kNCH;
    constexpr int UPR = D / 8;             // 16-byte units per K/V/Q row
    constexpr int PPT = TILE / kPageSize;  // pages per tile

    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t ready_bar[E];     // tile complete (landed, and patched where needed)
    __shared__ __align__(8) uint64_t landed_bar[E];    // TMA bytes of a tile that still needs patching
    __shared__ __align__(8) uint64_t empty_bar[E];     // the MMAs that read the entry are done
    __shared__ __align__(8) uint64_t s_full_bar[2];    // S buffer written by Q K^T
    __shared__ __align__(8) uint64_t p_full_bar[2];    // P written (and the S buffer read) by the four softmax warps
    __shared__ __align__(8) uint64_t pv_done_bar[2];   // P V of a tile done: P may be overwritten, O is up to date
    __shared__ int s_pages[kUmmaMaxChunkPages];
    __shared__ uint32_t tmem_base_slot;
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
    // Sliding window: nothing before block row 0's lower bound is needed (see the warp-MMA kernel).
    const int lo_min = p.window > 0 ? max(0, L - p.window + 1) : 0;
    const int first_chunk = lo_min / p.kv_chunk;
    if (chunk < first_chunk) return;
    int c_begin = chunk * p.kv_chunk;
    if (chunk == first_chunk) c_begin += ((lo_min - c_begin) / TILE) * TILE;
    const int c_end = min(n_ctx, chunk * p.kv_chunk + p.kv_chunk);
    const int n_tiles = (c_end - c_begin + TILE - 1) / TILE;
    const int n_chunks_b = (n_ctx + p.kv_chunk - 1) / p.kv_chunk - first_chunk;
    const int G = p.Hq / p.Hkv;
    const int rows = G * p.R;

    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint8_t* q_smem = smem + E * Cfg::kEntryBytes;               // [NCH][64 rows][128 B], swizzled
    uint8_t* p_smem = q_smem + Cfg::kQBytes;                     // [TILE/64][64 rows][128 B], swizzled

    if (threadIdx.x == 0) {
        for (int e = 0; e < E; ++e) { mbar_init(&ready_bar[e], 1); mbar_init(&landed_bar[e], 1); mbar_init(&empty_bar[e], 1); }
        for (int i = 0; i < 2; ++i) { mbar_init(&s_full_bar[i], 1); mbar_init(&p_full_bar[i], 4); mbar_init(&pv_done_bar[i], 1); }
        abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        __syncwarp();
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_slot)),
                     "r"((uint32_t)Cfg::kTmemCols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    {   // page ids of this chunk and the query rows (row r = block_row * G + head_in_group; rows past the last are zero)
        const int n_pages = (c_end - c_begin + kPageSize - 1) / kPageSize;
        for (int i = threadIdx.x; i < n_pages; i += blockDim.x)
            s_pages[i] = p.page_table[(size_t)b * p.max_pages + c_begin / kPageSize + i];
        for (int i = threadIdx.x; i < kUmmaRows * UPR; i += blockDim.x) {
            const int r = i / UPR, u = i % UPR;
            uint4 v = make_uint4(0u, 0u, 0u, 0u);
            if (r < rows) {
                const int j = r / G, hh = r % G;
                v = *reinterpret_cast<const uint4*>(p.q + (((size_t)b * p.R + j) * p.Hq + g * G + hh) * D + u * 8);
            }
            *reinterpret_cast<uint4*>(q_smem + (u / 8) * Cfg::kQRegion + swz128(r, u % 8)) = v;
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");      // Q is read by the tensor core
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_slot;
    const uint32_t tmem_o = tmem_base + 2 * TILE;
    volatile int* abort_ptr = &abort_flag;

    if (warp == 0) {
        // ------------------------------------------------ TMA producer (+ append / ragged-end patch)
        uint64_t policy;
        asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(policy));
        uint32_t landed_phase = 0;       // bit e: parity of the next completion of landed_bar[e]
        for (int i = 0; i < 2 * n_tiles; ++i) {
            // item i of the consumption order: which tile, and whether its K or its V
            const int is_v = (i == 2 * n_tiles - 1) || (i > 0 && (i & 1) == 0);
            const int t = i == 0 ? 0 : (i == 2 * n_tiles - 1 ? n_tiles - 1 : (is_v ? i / 2 - 1 : (i + 1) / 2));
            const int e = i % E;
            int freed = 0;
            if (lane == 0) freed = mbar_wait(&empty_bar[e], (((uint32_t)(i / E)) & 1u) ^ 1u, abort_ptr) ? 1 : 0;
            freed = __shfl_sync(0xffffffffu, freed, 0);
            if (!freed) break;
            const int tile_start = c_begin + t * TILE;
            const int valid = min(TILE, c_end - tile_start);
            const int n_pg = (valid + kPageSize - 1) / kPageSize;
            const bool patch = tile_start + TILE > L;           // the tile holds block rows or the ragged end
            uint64_t* bar = patch ? &landed_bar[e] : &ready_bar[e];
            uint8_t* dst = smem + (size_t)e * Cfg::kEntryBytes;
            if (lane == 0) mbar_expect_tx(bar, (uint32_t)(n_pg * NCH * 2048));
            __syncwarp();
            for (int j = lane; j < n_pg * NCH; j += 32) {
                const int dc = j % NCH, pg = j / NCH;
                int pid = s_pages[t * PPT + pg];
                if (pid < 0 || pid >= p.num_pages) { set_status(p.dev_status, MASSV_ERR_CAPACITY); pid = 0; }
                tma_load_2d(dst + dc * Cfg::kRegion + pg * 2048, is_v ? &map_v : &map_k, dc * 64, (pid * p.Hkv + g) * kPageSize, bar, policy);
            }
            if (patch) {
                int ok = 0;
                if (lane == 0) ok = mbar_wait(&landed_bar[e], (landed_phase >> e) & 1u, abort_ptr) ? 1 : 0;
                ok = __shfl_sync(0xffffffffu, ok, 0);
                if (!ok) break;
                landed_phase ^= 1u << e;
                // The block's rows (positions L .. L+gamma) are not in the cache yet: put them into the
                // tile and store them to their page slots.
                const int p_first = max(L, tile_start), p_last = min(c_end, tile_start + TILE);
                const __nv_bfloat16* src_base = is_v ? p.v_new : p.k_new;
                __nv_bfloat16* pages = is_v ? p.v_pages : p.k_pages;
                for (int idx = lane; idx < (p_last - p_first) * UPR; idx += 32) {
                    const int pos = p_first + idx / UPR, u = idx % UPR, row = pos - tile_start;
                    const uint4 val = *reinterpret_cast<const uint4*>(src_base + (((size_t)b * p.R + (pos - L)) * p.Hkv + g) * D + u * 8);
                    *reinterpret_cast<uint4*>(dst + (u / 8) * Cfg::kRegion + swz128(row, u % 8)) = val;
                    const int pid = s_pages[(pos - c_begin) / kPageSize];
                    if (pid >= 0 && pid < p.num_pages)
                        *reinterpret_cast<uint4*>(pages + (((size_t)pid * p.Hkv + g) * kPageSize + (pos % kPageSize)) * D + u * 8) = val;
                }
                if (is_v) {
                    // rows past the end of the context hold stale bytes; their weights are zero, but
                    // 0 * NaN would still poison P V
                    for (int idx = lane; idx < (TILE - valid) * UPR; idx += 32) {
                        const int row = valid + idx / UPR, u = idx % UPR;
                        *reinterpret_cast<uint4*>(dst + (u / 8) * Cfg::kRegion + swz128(row, u % 8)) = make_uint4(0u, 0u, 0u, 0u);
                    }
                }
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                __syncwarp();
                if (lane == 0) mbar_arrive(&ready_bar[e]);
            }
        }
        if (lane == 0 && *abort_ptr) {
            for (int i = 0; i < 64; ++i) __nanosleep(2000);   // let copies in flight land
        }
    } else if (warp == 1) {
        // ------------------------------------------------ MMA issuer
        if (lane == 0) {
            constexpr uint32_t idesc_qk = umma_idesc_bf16(kUmmaRows, TILE, false);
            constexpr uint32_t idesc_pv = umma_idesc_bf16(kUmmaRows, D, true);
            const uint32_t q_lo = umma_desc_lo(smem_u32(q_smem));
            const uint32_t ring_addr = smem_u32(smem);
            bool ok = true;
            // S[t & 1] = Q K_t^T: d/16 steps of 16 elements (32 bytes) along the 128-byte rows
            auto issue_qk = [&](int t) {
                const int i = ring_item_of_k(t), e = i % E;
                if (!mbar_wait(&ready_bar[e], ((uint32_t)(i / E)) & 1u, abort_ptr)) { ok = false; return; }
                tc_fence_after();
                const uint32_t k_lo = umma_desc_lo(ring_addr + (uint32_t)e * Cfg::kEntryBytes);
                const uint32_t d_tmem = tmem_base + (uint32_t)((t & 1) * TILE);
#pragma unroll
                for (int kk = 0; kk < D / 16; ++kk) {
                    const uint32_t a = q_lo + (uint32_t)(((kk >> 2) * Cfg::kQRegion + (kk & 3) * 32) >> 4);
                    const uint32_t bb = k_lo + (uint32_t)(((kk >> 2) * Cfg::kRegion + (kk & 3) * 32) >> 4);
                    if (kk == 0) umma_bf16<false>(d_tmem, a, bb, idesc_qk);
                    else umma_bf16<true>(d_tmem, a, bb, idesc_qk);
                }
                umma_commit(&empty_bar[e]);
                umma_commit(&s_full_bar[t & 1]);
            };
            // O (+)= P[t & 1] V_t: TILE/16 steps of 16 tokens; V rows are tokens, so a step is 2048 bytes
            // further and the descriptor's leading offset is the distance between 64-element column groups
            auto issue_pv = [&](int t) {
                const int i = ring_item_of_v(t, n_tiles), e = i % E;
                if (!mbar_wait(&ready_bar[e], ((uint32_t)(i / E)) & 1u, abort_ptr)) { ok = false; return; }
                if (!mbar_wait(&p_full_bar[t & 1], ((uint32_t)(t >> 1)) & 1u, abort_ptr)) { ok = false; return; }
                tc_fence_after();
                const uint32_t p_lo = umma_desc_lo(smem_u32(p_smem));
                const uint32_t v_lo = (((ring_addr + (uint32_t)e * Cfg::kEntryBytes) & 0x3FFFFu) >> 4) | ((uint32_t)(Cfg::kRegion >> 4) << 16);
#pragma unroll
                for (int ks = 0; ks < TILE / 16; ++ks) {
                    const uint32_t a = p_lo + (uint32_t)(((ks >> 2) * Cfg::kQRegion + (ks & 3) * 32) >> 4);
                    const uint32_t bb = v_lo + (uint32_t)((ks * 2048) >> 4);
                    if (ks == 0 && t == 0) umma_bf16<false>(tmem_o, a, bb, idesc_pv);
                    else umma_bf16<true>(tmem_o, a, bb, idesc_pv);
                }
                umma_commit(&empty_bar[e]);
                umma_commit(&pv_done_bar[t & 1]);
            };
            issue_qk(0);
            if (ok && n_tiles > 1) issue_qk(1);
            for (int t = 0; t < n_tiles && ok; ++t) {
                issue_pv(t);
                if (ok && t + 2 < n_tiles) issue_qk(t + 2);
            }
        }
    } else {
        // ------------------------------------------------ softmax warps: 16 query rows each
        const int qd = warp & 3;                            // the TMEM lane quarter this warp may access
        const uint32_t lane_base = (uint32_t)(qd * 32) << 16;
        const int r0 = qd * 16 + (lane >> 2), r1 = r0 + 8;
        // block row of each of this thread's two query rows (padding rows behave like the last block row)
        const int j0 = r0 < rows ? r0 / G : p.R - 1, j1 = r1 < rows ? r1 / G : p.R - 1;
        const float scale_log2 = p.scale * 1.4426950408889634f;
        float m_ref[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};
        bool ok = true;
        for (int t = 0; t < n_tiles && ok; ++t) {
            const int buf = t & 1;
            if (!mbar_wait_warp(&s_full_bar[buf], ((uint32_t)(t >> 1)) & 1u, abort_ptr)) { ok = false; break; }
            tc_fence_after();
            const int tile_start = c_begin + t * TILE;
            // some position in the tile is hidden from some block row: ahead of row 0, or (with a
            // window) older than the last row's lower bound
            const bool need_mask = tile_start + TILE > L + 1 || (p.window > 0 && tile_start < n_ctx - p.window);
            float mx0 = -INFINITY, mx1 = -INFINITY;
            uint32_t s[TILE / 64][32];
#pragma unroll
            for (int h = 0; h < TILE / 64; ++h) {
                tmem_ld_16x64(tmem_base + lane_base + (uint32_t)(buf * TILE + h * 64), s[h]);
#pragma unroll
                for (int k = 0; k < 8; ++k) {
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        float sv = __uint_as_float(s[h][4 * k + e]) * scale_log2;
                        if (need_mask) {
                            const int pos = tile_start + h * 64 + k * 8 + 2 * (lane & 3) + (e & 1);
                            const int row_pos = L + (e < 2 ? j0 : j1);
                            if (pos > row_pos || (p.window > 0 && pos < row_pos - p.window + 1)) sv = -INFINITY;
                        }
                        s[h][4 * k + e] = __float_as_uint(sv);
                        if (e < 2) mx0 = fmaxf(mx0, sv); else mx1 = fmaxf(mx1, sv);
                    }
                }
            }
            mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 1));
            mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 2));
            mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 1));
            mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 2));
            // The reference maximum of a row moves only when the row's maximum has outgrown it by the
            // threshold (or when it is first set); O and l are then rescaled to the new reference.
            float f0 = 1.f, f1 = 1.f;
            bool grow = false;
            if (m_ref[0] == -INFINITY) m_ref[0] = mx0;
            else if (mx0 > m_ref[0] + kRescaleThreshold) { f0 = exp2f(m_ref[0] - mx0); m_ref[0] = mx0; grow = true; }
            if (m_ref[1] == -INFINITY) m_ref[1] = mx1;
            else if (mx1 > m_ref[1] + kRescaleThreshold) { f1 = exp2f(m_ref[1] - mx1); m_ref[1] = mx1; grow = true; }
            const float ms0 = m_ref[0] == -INFINITY ? 0.f : m_ref[0], ms1 = m_ref[1] == -INFINITY ? 0.f : m_ref[1];
            float ls0 = 0.f, ls1 = 0.f;
            uint32_t pk[TILE / 64][16];       // bf16 pairs: [2k] = row r0, [2k+1] = row r1, tokens 8k + 2*(lane%4) + {0,1}
#pragma unroll
            for (int h = 0; h < TILE / 64; ++h) {
#pragma unroll
                for (int k = 0; k < 8; ++k) {
                    const float p0 = exp2f(__uint_as_float(s[h][4 * k + 0]) - ms0), p1 = exp2f(__uint_as_float(s[h][4 * k + 1]) - ms0);
                    const float p2 = exp2f(__uint_as_float(s[h][4 * k + 2]) - ms1), p3 = exp2f(__uint_as_float(s[h][4 * k + 3]) - ms1);
                    ls0 += p0 + p1; ls1 += p2 + p3;
                    pk[h][2 * k] = pack_bf16x2(p0, p1);
                    pk[h][2 * k + 1] = pack_bf16x2(p2, p3);
                }
            }
            // P and O belong to the tensor core until P V of tile t-1 is done; P V of tile t cannot
            // start before this warp has published P below.
            if (t >= 1 && !mbar_wait_warp(&pv_done_bar[(t - 1) & 1], ((uint32_t)((t - 1) >> 1)) & 1u, abort_ptr)) { ok = false; break; }
            if (__any_sync(0xffffffffu, grow)) {
                tc_fence_after();
#pragma unroll 1
                for (int c0 = 0; c0 < D; c0 += 64) {
                    uint32_t o[32];
                    tmem_ld_16x64(tmem_o + lane_base + (uint32_t)c0, o);
#pragma unroll
                    for (int k = 0; k < 8; ++k) {
                        o[4 * k + 0] = __float_as_uint(__uint_as_float(o[4 * k + 0]) * f0);
                        o[4 * k + 1] = __float_as_uint(__uint_as_float(o[4 * k + 1]) * f0);
                        o[4 * k + 2] = __float_as_uint(__uint_as_float(o[4 * k + 2]) * f1);
                        o[4 * k + 3] = __float_as_uint(__uint_as_float(o[4 * k + 3]) * f1);
                    }
                    tmem_st_16x64(tmem_o + lane_base + (uint32_t)c0, o);
                }
                asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
                l_run[0] *= f0; l_run[1] *= f1;
            }
#pragma unroll
            for (int h = 0; h < TILE / 64; ++h) {
#pragma unroll
                for (int k = 0; k < 8; ++k) {
                    // tokens 8k .. 8k+7 of the 64-token group are 16-byte unit k of the row
                    *reinterpret_cast<uint32_t*>(p_smem + h * Cfg::kQRegion + swz128(r0, k) + 4 * (lane & 3)) = pk[h][2 * k];
                    *reinterpret_cast<uint32_t*>(p_smem + h * Cfg::kQRegion + swz128(r1, k) + 4 * (lane & 3)) = pk[h][2 * k + 1];
                }
            }
            l_run[0] += ls0; l_run[1] += ls1;
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");     // P is read by the tensor core
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&p_full_bar[buf]);
        }
        if (ok && !mbar_wait_warp(&pv_done_bar[(n_tiles - 1) & 1], ((uint32_t)((n_tiles - 1) >> 1)) & 1u, abort_ptr)) ok = false;
        tc_fence_after();
        pdl_trigger();
        if (ok) {
            l_run[0] += __shfl_xor_sync(0xffffffffu, l_run[0], 1);
            l_run[0] += __shfl_xor_sync(0xffffffffu, l_run[0], 2);
            l_run[1] += __shfl_xor_sync(0xffffffffu, l_run[1], 1);
            l_run[1] += __shfl_xor_sync(0xffffffffu, l_run[1], 2);
            const bool single = n_chunks_b == 1;
            const int rows_pad = (rows + 15) / 16 * 16;
            const size_t item = ((size_t)b * p.Hkv + g) * p.max_chunks + chunk;
            const float inv0 = 1.f / l_run[0], inv1 = 1.f / l_run[1];
            const size_t out0 = r0 < rows ? (((size_t)b * p.R + r0 / G) * p.Hq + g * G + r0 % G) : 0;
            const size_t out1 = r1 < rows ? (((size_t)b * p.R + r1 / G) * p.Hq + g * G + r1 % G) : 0;
#pragma unroll 1
            for (int c0 = 0; c0 < D; c0 += 64) {
                uint32_t o[32];
                tmem_ld_16x64(tmem_o + lane_base + (uint32_t)c0, o);
#pragma unroll
                for (int k = 0; k < 8; ++k) {
                    const int c = c0 + k * 8 + 2 * (lane & 3);
                    float a0 = __uint_as_float(o[4 * k + 0]), a1 = __uint_as_float(o[4 * k + 1]);
                    float a2 = __uint_as_float(o[4 * k + 2]), a3 = __uint_as_float(o[4 * k + 3]);
                    if (single) {
                        a0 *= inv0; a1 *= inv0; a2 *= inv1; a3 *= inv1;
                        if (r0 < rows) {
                            *reinterpret_cast<uint32_t*>(p.out + out0 * D + c) = pack_bf16x2(a0, a1);
                            if (p.out_f32) *reinterpret_cast<float2*>(p.out_f32 + out0 * D + c) = make_float2(a0, a1);
                        }
                        if (r1 < rows) {
                            *reinterpret_cast<uint32_t*>(p.out + out1 * D + c) = pack_bf16x2(a2, a3);
                            if (p.out_f32) *reinterpret_cast<float2*>(p.out_f32 + out1 * D + c) = make_float2(a2, a3);
                        }
                    } else {
                        if (r0 < rows) *reinterpret_cast<float2*>(p.part_o + (item * rows_pad + r0) * D + c) = make_float2(a0, a1);
                        if (r1 < rows) *reinterpret_cast<float2*>(p.part_o + (item * rows_pad + r1) * D + c) = make_float2(a2, a3);
                    }
                }
            }
            if ((lane & 3) == 0) {
                if (single) {
                    if (p.lse) {
                        if (r0 < rows) p.lse[out0] = (m_ref[0] + log2f(l_run[0])) * 0.6931471805599453f;
                        if (r1 < rows) p.lse[out1] = (m_ref[1] + log2f(l_run[1])) * 0.6931471805599453f;
                    }
                } else {
                    if (r0 < rows) { p.part_ml[(item * rows_pad + r0) * 2] = m_ref[0]; p.part_ml[(item * rows_pad + r0) * 2 + 1] = l_run[0]; }
                    if (r1 < rows) { p.part_ml[(item * rows_pad + r1) * 2] = m_ref[1]; p.part_ml[(item * rows_pad + r1) * 2 + 1] = l_run[1]; }
                }
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        __syncwarp();
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)Cfg::kTmemCols) : "memory");
    }
    if (threadIdx.x == 0 && abort_flag) set_status(p.dev_status, MASSV_ERR_TIMEOUT);
}

template <int D, int TILE>
cudaError_t launch_umma(const AttnParams& p, const CUtensorMap& mk, const CUtensorMap& mv, cudaStream_t stream) {
    using Cfg = UmmaAttnCfg<D, TILE>;
    static_assert(Cfg::kColsNeeded <= 512, "S buffers and O fit tensor memory");
    static_assert(Cfg::kSmem <= 227 * 1024, "ring, Q and P fit shared memory");
    cudaError_t e = cudaFuncSetAttribute(attn_umma_kernel<D, TILE>, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg::kSmem);
    if (e != cudaSuccess) return e;
    return launch_pdl(attn_umma_kernel<D, TILE>, dim3(p.max_chunks, p.Hkv, p.B), dim3(kUmmaThreads), (size_t)Cfg::kSmem, stream, mk, mv, p);
}

}  // namespace

bool attn_umma_supported(const AttnParams& p) {
    return (p.Hq / p.Hkv) * p.R <= kUmmaRows && (p.d == 64 || p.d == 128 || p.d == 256) &&
           p.kv_chunk <= kUmmaMaxChunkPages * kPageSize && p.kv_chunk % 64 == 0;
}

cudaError_t launch_attn_umma(const AttnParams& p, const CUtensorMap& mk, const CUtensorMap& mv, cudaStream_t stream) {
    switch (p.d) {
        case 64: return launch_umma<64, 64>(p, mk, mv, stream);
        case 128: return launch_umma<128, 64>(p, mk, mv, stream);
        case 256: return launch_umma<256, 64>(p, mk, mv, stream);
        default: return cudaErrorInvalidValue;
    }
}

}  // namespace massv
