// LM head on the 5th-generation tensor cores with the softmax statistics fused
// into the epilogue (Sec. 2.1: the target computes p(. | X_{1:t+i-1}) over the
// vocabulary for the gamma+1 block rows).
//
//   z[m, v] = sum_k hidden[m, k] * lm_head[v, k]        bf16 x bf16 -> fp32
//
// Operands are swapped so that the vocabulary runs along the MMA M axis: one
// tcgen05.mma computes D[128 vocab rows, N token rows] with the accumulator in
// tensor memory (lane = vocab row, column = token row).  The weight matrix is
// streamed exactly once: each persistent CTA owns a contiguous band of whole
// 128-row vocabulary tiles and walks K in 64-element blocks through a TMA ->
// shared memory ring.  Warp roles: warp 0 issues TMA loads, warp 1 issues MMAs and owns
// the TMEM allocation, warps 2-9 drain finished accumulators (double buffered)
// with tcgen05.ld, store fp32 logits when they are needed, and keep running
// (max, sum exp((z-max)/T), argmax) per token row in shared memory (warp-wide
// integer max reduction on order-preserving keys, ballot for the argmax, a
// transposed butterfly for the sums).  At the end the CTA writes one partial
// slot; the acceptance kernel merges the slots.  Every reduction has a fixed order.
#include <cuda.h>

#include "kernels.cuh"
#include "ptx.cuh"
#include "umma.cuh"

namespace massv {

namespace {

constexpr int kEpilogueWarps = 8;          // two per TMEM lane quarter
constexpr int kThreads = (2 + kEpilogueWarps) * 32;
constexpr int kBlockK = 64;                 // bf16 elements per 128-byte swizzled row
constexpr int kTileBytesW = kVocabTile * kBlockK * 2;
constexpr int kMaxStages = 12;
constexpr int kMaxCtas = 192;               // partial slots are sized for at most this many CTAs
constexpr int kRingBytes = 200 * 1024;      // shared memory given to the TMA ring
constexpr int kPrefetchBlocks = 32;         // K blocks (16 KB each) of the first tile hinted into L2 before the dependency wait
constexpr int kPairMinTile = 64;            // token rows per tile from which CTA pairs are used

struct UmmaParams {
    int M, K, V;
    int n_tile;          // token rows per MMA (multiple of 16, <= 256)
    int n_token_tiles;   // 1 or 2
    int n_groups;        // vocab bands
    int tiles_per_group; // whole 128-row tiles per band
    int stages;
    int tmem_cols;       // power of two >= 2 * n_tile
    int greedy;
    float scale_log2;    // log2(e) / T
    float* logits;       // [M, V] or nullptr
    float *part_max, *part_sum;
    int32_t* part_idx;
    int n_part = 0;      // partial slots behind part_max / part_sum / part_idx (the debug build checks the slot index)
    int32_t* dev_status;
    int idx_offset;      // added to the argmax indices that leave the kernel
    int test_skip_stage = 0;   // test builds only: withhold the second K block of the first tile
    int n_bands = 0;     // duo kernel: 256-row vocabulary bands in all
    int split_rem = 0;   // duo kernel: bands left over after tiles_per_group per pair, each cut in two half-tiles (one sub-tile each)
};

// ---- CTA pairs (cta_group::2): two CTAs of a cluster act as one 256-row MMA.  Each loads its own
// 128 weight rows and half of the hidden-state rows; the even CTA (the leader) issues the MMAs,
// which read both CTAs' shared memory and write each CTA's half of the result to its own TMEM.
__device__ __forceinline__ uint32_t cluster_cta_rank() { uint32_t r; asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r)); return r; }
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// Cluster-wide address of a shared-memory location in CTA `rank`.
__device__ __forceinline__ uint32_t cluster_addr(const void* local, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(smem_u32(local)), "r"(rank));
    return r;
}
__device__ __forceinline__ void mbar_expect_tx_at(uint32_t bar_cluster_addr, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cluster.b64 _, [%0], %1;" ::"r"(bar_cluster_addr), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive_at(uint32_t bar_cluster_addr) {
    asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(bar_cluster_addr) : "memory");
}
// TMA load into this CTA's shared memory whose completion is signalled on a barrier of the pair's leader.
__device__ __forceinline__ void tma_load_2d_pair(void* dst, const CUtensorMap* map, int x, int y, uint32_t bar_cluster_addr,
                                                 uint64_t policy) {
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint"
        " [%0], [%1, {%2, %3}], [%4], %5;" ::"r"(smem_u32(dst)),
        "l"(map), "r"(x), "r"(y), "r"(bar_cluster_addr), "l"(policy)
        : "memory");
}
template <bool ACC>
__device__ __forceinline__ void umma_bf16_pair(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t idesc) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\t"
        "setp.ne.b32 p, %5, 0;\n\t"
        "mov.b64 da, {%1, %4};\n\t"
        "mov.b64 db, {%2, %4};\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], da, db, %3, p;\n\t}" ::"r"(d_tmem),
        "r"(a_lo), "r"(b_lo), "r"(idesc), "r"(kDescHi), "r"(ACC ? 1u : 0u)
        : "memory");
}
// Arrive, in both CTAs of the pair, on the barrier at this shared-memory offset once the MMAs issued so far are done.
// This barrier arrive between the two CTAs of one pair (same GPU) is the only multicast qualifier in the sources:
// every TMA load here (tma_load_2d, tma_load_2d_pair, the 1-D bulk copies) is non-multicast and reads this GPU's
// memory only.
__device__ __forceinline__ void umma_commit_pair(uint64_t* bar) {
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;" ::"r"(smem_u32(bar)),
                 "h"((uint16_t)3)
                 : "memory");
}

template <int C>
__device__ __forceinline__ void tmem_load(uint32_t taddr, uint32_t (&r)[C]);
template <>
__device__ __forceinline__ void tmem_load<32>(uint32_t taddr, uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
          "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
          "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr));
}
template <>
__device__ __forceinline__ void tmem_load<16>(uint32_t taddr, uint32_t (&r)[16]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr));
}
// Wait for outstanding tcgen05.ld; the registers are passed through so that no
// use of them can be scheduled ahead of the wait.
template <int C>
__device__ __forceinline__ void tmem_wait_ld(uint32_t (&r)[C]) {
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int j = 0; j < C; ++j) asm volatile("" : "+r"(r[j]));
}

// ------------------------------------------------------------------ statistics
struct Stat {
    float m;   // max logit
    float s;   // sum of 2^((z - m) * scale_log2)
    int idx;   // lowest vocabulary index attaining m
};

__device__ __forceinline__ Stat stat_combine(const Stat& a, const Stat& b, float scale_log2, bool greedy) {
    Stat r;
    const bool a_wins = a.m > b.m || (a.m == b.m && a.idx < b.idx);
    r.m = a_wins ? a.m : b.m;
    r.idx = a_wins ? a.idx : b.idx;
    r.s = 0.f;
    if (!greedy) {
        // the loser's mass is rescaled to the winner's reference; -inf entries carry s == 0
        const float lo = a_wins ? b.m : a.m;
        const float s_hi = a_wins ? a.s : b.s, s_lo = a_wins ? b.s : a.s;
        const float f = (lo == -INFINITY) ? 0.f : exp2f((lo - r.m) * scale_log2);
        r.s = s_hi + s_lo * f;
    }
    return r;
}

// Order-preserving map float -> uint32, so that the integer warp reduction
// (redux.sync.max.u32) yields the float maximum.
__device__ __forceinline__ uint32_t float_key(float x) {
    const uint32_t b = __float_as_uint(x);
    return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}
__device__ __forceinline__ float key_float(uint32_t k) {
    return __uint_as_float((k & 0x80000000u) ? (k & 0x7fffffffu) : ~k);
}

// Sum C columns (one value per lane) across the 32 lanes of the warp.  Each step
// halves the number of columns a lane keeps by trading the other half with its
// partner, so the reduction costs about one exchange per column.  On return
// lane l holds the sum of column l (C == 32) or l >> 1 (C == 16) in v[0].
template <int C>
__device__ __forceinline__ void transposed_sum(float (&v)[C], int lane) {
    int n = C;
#pragma unroll
    for (int offset = 16; offset >= 1; offset >>= 1) {
        if (n > 1) {
            const int half = n / 2;
            const bool upper = (lane & offset) != 0;
#pragma unroll
            for (int i = 0; i < C / 2; ++i) {
                if (i < half) {
                    const float send = upper ? v[i] : v[i + half];
                    const float keep = upper ? v[i + half] : v[i];
                    v[i] = keep + __shfl_xor_sync(0xffffffffu, send, offset);
                }
            }
            n = half;
        } else {
            v[0] += __shfl_xor_sync(0xffffffffu, v[0], offset);
        }
    }
}

struct TileCtx {
    int v0;        // first vocabulary row of the tile
    int rows;      // valid rows (multiple of 8, <= 128)
};

// Drain one chunk of C accumulator columns of the current tile: store the
// logits if asked, and fold the chunk into `running`, the statistic of the
// column this lane owns (column `lane` of the chunk for C == 32, `lane >> 1`
// for C == 16).
template <int C>
__device__ __forceinline__ void drain_chunk(const UmmaParams& p, uint32_t taddr, int lane, int row_in_tile,
                                            const TileCtx& tile, int tok0, Stat& running) {
    uint32_t r[C];
    tmem_load<C>(taddr, r);
    tmem_wait_ld<C>(r);
    const int vrow = tile.v0 + row_in_tile;
    const bool row_ok = row_in_tile < tile.rows;
    if (p.logits != nullptr && row_ok) {
        float* dst = p.logits + (size_t)tok0 * p.V + vrow;
#pragma unroll
        for (int j = 0; j < C; ++j) {
            if (tok0 + j < p.M) dst[(size_t)j * p.V] = __uint_as_float(r[j]);
        }
    }
    const bool greedy = p.greedy != 0;
    const int warp_row0 = vrow - lane;          // vocabulary row of lane 0
    float sums[C];
    Stat mine{-INFINITY, 0.f, 0x7fffffff};
#pragma unroll
    for (int j = 0; j < C; ++j) {
        const float z = row_ok ? __uint_as_float(r[j]) + 0.f : -INFINITY;     // + 0 folds -0 into +0
        const uint32_t key = float_key(z);
        const uint32_t kmax = __reduce_max_sync(0xffffffffu, key);
        const unsigned hit = __ballot_sync(0xffffffffu, key == kmax);
        const float mx = key_float(kmax);
        sums[j] = (greedy || mx == -INFINITY) ? 0.f : exp2f((z - mx) * p.scale_log2);
        if ((C == 32 ? lane : (lane >> 1)) == j) {
            mine.m = mx;
            mine.idx = mx == -INFINITY ? 0x7fffffff : warp_row0 + (__ffs(hit) - 1);   // lowest row attaining the max
        }
    }
    if (!greedy) {
        transposed_sum<C>(sums, lane);
        mine.s = sums[0];
    }
    running = stat_combine(running, mine, p.scale_log2, greedy);
}

// PAIR: the grid is made of 2-CTA clusters; a pair works on 256-row vocabulary super-tiles (CTA rank r
// owns rows 128 r .. 128 r + 127 and half of the token rows of the hidden-state tile), which halves the
// hidden-state traffic per weight byte compared with one CTA per 128 rows.
template <bool PAIR>
__global__ void __launch_bounds__(kThreads, 1)
lm_head_umma_kernel(const __grid_constant__ CUtensorMap map_w128, const __grid_constant__ CUtensorMap map_w64,
                    const __grid_constant__ CUtensorMap map_w32, const __grid_constant__ CUtensorMap map_w16,
                    const __grid_constant__ CUtensorMap map_w8, const __grid_constant__ CUtensorMap map_h,
                    const UmmaParams p) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t full_bar[kMaxStages];
    __shared__ __align__(8) uint64_t empty_bar[kMaxStages];
    __shared__ __align__(8) uint64_t tmem_full_bar[2];
    __shared__ __align__(8) uint64_t tmem_empty_bar[2];
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag;
    __shared__ float run_m[4][256];
    __shared__ float run_s[4][256];
    __shared__ int run_i[4][256];

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const int h_rows = PAIR ? p.n_tile / 2 : p.n_tile;       // hidden-state rows this CTA loads per K block
    const int stage_bytes = kTileBytesW + h_rows * 128;
    const int num_kb = p.K / kBlockK;
    const uint32_t pair_rank = PAIR ? cluster_cta_rank() : 0u;

    // which band of vocabulary rows and which token tile this CTA (or pair) owns
    const int unit = PAIR ? blockIdx.x / 2 : blockIdx.x;
    const int group = unit / p.n_token_tiles;
    const int token_tile = unit % p.n_token_tiles;
    constexpr int tile_rows = PAIR ? 2 * kVocabTile : kVocabTile;       // rows per (super-)tile of the band
    const int row_begin = min(p.V, group * p.tiles_per_group * tile_rows);
    const int row_end = min(p.V, row_begin + p.tiles_per_group * tile_rows);
    const int n_tiles = (row_end - row_begin + tile_rows - 1) / tile_rows;
    const int tok_base = token_tile * p.n_tile;

    if (threadIdx.x == 0) {
        for (int s = 0; s < p.stages; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], 1); }
        // in a pair the leader's tmem_empty barriers collect both CTAs' epilogue warps
        for (int b = 0; b < 2; ++b) { mbar_init(&tmem_full_bar[b], 1); mbar_init(&tmem_empty_bar[b], (PAIR ? 2 : 1) * kEpilogueWarps); }
        abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {
        __syncwarp();
        if constexpr (PAIR) {
            asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_slot)),
                         "r"((uint32_t)p.tmem_cols)
                         : "memory");
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
        } else {
            asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_slot)),
                         "r"((uint32_t)p.tmem_cols)
                         : "memory");
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
        }
    }
    tc_fence_before();
    __syncthreads();
    if constexpr (PAIR) cluster_sync_all();      // the peer's barriers exist before anything signals them
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_slot;
    volatile int* abort_ptr = &abort_flag;
    // The weights do not depend on the kernel before this one: while it drains, an epilogue warp (idle
    // until the first accumulator is ready) asks L2 for the first boxes of this CTA's first tile.
    // Single-CTA tiles only: with CTA pairs the hints cost more than they bring.  Depth by measurement:
    // the step gains up to 32 boxes (-2.4 %), beyond 40 the hinted boxes are fetched twice too often.
    if constexpr (!PAIR) {
        if (warp == 2 && lane == 0 && n_tiles > 0) {
            const int n_pf = min(num_kb, kPrefetchBlocks);
            for (int kb = 0; kb < n_pf; ++kb) tma_prefetch_2d(&map_w128, kb * kBlockK, row_begin);
        }
    }
    pdl_wait();          // everything above overlapped with the tail of the previous kernel
    // The acceptance kernels behind this one are small: let them become resident now, fetch the inputs that
    // do not depend on this grid, and wait for it there.
    pdl_trigger();

    if (warp == 0) {
        // ------------------------------------------------ TMA producer
        if (lane == 0) {
            uint64_t pol_stream, pol_keep;
            asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol_stream));
            asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol_keep));
            int s = 0;
            uint32_t ph = 0;
            uint8_t* w_dst = smem;
            bool ok = true;
            for (int t = 0; t < n_tiles && ok; ++t) {
                const int v0 = row_begin + t * tile_rows + (int)pair_rank * kVocabTile;
                const int rows = PAIR ? kVocabTile : min(tile_rows, row_end - v0);
                const uint32_t tx_bytes = (uint32_t)(rows * 128 + p.n_tile * 128);
                for (int kb = 0; kb < num_kb; ++kb) {
                    if (!mbar_wait(&empty_bar[s], ph ^ 1u, abort_ptr)) { ok = false; break; }
#ifdef MASSV_TEST_HOOKS
                    if (p.test_skip_stage && t == 0 && kb == 1) {
                        // nothing is announced and nothing is copied for this stage: the MMA thread's wait for it
                        // must give up by itself
                        w_dst += stage_bytes;
                        if (++s == p.stages) { s = 0; ph ^= 1u; w_dst = smem; }
                        continue;
                    }
#endif
                    uint8_t* h_dst = w_dst + kTileBytesW;
                    if constexpr (PAIR) {
                        // Both CTAs' copies complete on the leader's barrier; the leader announces the
                        // bytes of the pair (two 128-row weight boxes, two halves of the hidden-state tile;
                        // rows past the end of either matrix are filled with zeros and still counted).
                        const uint32_t bar = cluster_addr(&full_bar[s], 0);
                        if (pair_rank == 0) mbar_expect_tx_at(bar, (uint32_t)(2 * kTileBytesW + p.n_tile * 128));
                        tma_load_2d_pair(w_dst, &map_w128, kb * kBlockK, v0, bar, pol_stream);
                        tma_load_2d_pair(h_dst, &map_h, kb * kBlockK, tok_base + (int)pair_rank * h_rows, bar, pol_keep);
                        w_dst += stage_bytes;
                        if (++s == p.stages) { s = 0; ph ^= 1u; w_dst = smem; }
                        continue;
                    }
                    mbar_expect_tx(&full_bar[s], tx_bytes);
                    if (rows == kVocabTile) {
                        tma_load_2d(w_dst, &map_w128, kb * kBlockK, v0, &full_bar[s], pol_stream);
                    } else {
                        // rows is a multiple of 8 below 128: one box per set bit
                        int r = 0;
                        if (rows & 64) { tma_load_2d(w_dst + r * 128, &map_w64, kb * kBlockK, v0 + r, &full_bar[s], pol_stream); r += 64; }
                        if (rows & 32) { tma_load_2d(w_dst + r * 128, &map_w32, kb * kBlockK, v0 + r, &full_bar[s], pol_stream); r += 32; }
                        if (rows & 16) { tma_load_2d(w_dst + r * 128, &map_w16, kb * kBlockK, v0 + r, &full_bar[s], pol_stream); r += 16; }
                        if (rows & 8) { tma_load_2d(w_dst + r * 128, &map_w8, kb * kBlockK, v0 + r, &full_bar[s], pol_stream); r += 8; }
                    }
                    tma_load_2d(h_dst, &map_h, kb * kBlockK, tok_base, &full_bar[s], pol_keep);
                    w_dst += stage_bytes;
                    if (++s == p.stages) { s = 0; ph ^= 1u; w_dst = smem; }
                }
            }
            if (!ok) {
                // let copies that are still in flight land before the CTA retires
                for (int i = 0; i < 64; ++i) __nanosleep(2000);
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------ MMA issuer
        if (lane == 0 && pair_rank == 0) {       // in a pair only the leader issues
            const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(p.n_tile >> 3) << 17) |
                                   ((uint32_t)((PAIR ? 2 * kVocabTile : kVocabTile) >> 4) << 24);
            // The issuing thread must stay far below the 64..128 cycles one MMA takes, so the
            // loop carries only 32-bit descriptor words and a stage counter.
            const uint32_t lo_step = (uint32_t)stage_bytes >> 4;
            const uint32_t a_lo0 = umma_desc_lo(smem_u32(smem));
            int s = 0;
            uint32_t ph = 0, a_lo = a_lo0;
            bool ok = true;
            for (int t = 0; t < n_tiles && ok; ++t) {
                const int buf = t & 1;
                if (!mbar_wait(&tmem_empty_bar[buf], (((uint32_t)t >> 1) & 1u) ^ 1u, abort_ptr)) { ok = false; break; }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)(buf * p.n_tile);
                for (int kb = 0; kb < num_kb; ++kb) {
                    if (!mbar_wait(&full_bar[s], ph, abort_ptr)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t b_lo = a_lo + (kTileBytesW >> 4);
                    // four K slices of 16 elements (32 bytes, i.e. 2 descriptor units) each
                    if constexpr (PAIR) {
                        if (kb == 0) umma_bf16_pair<false>(d_tmem, a_lo, b_lo, idesc);
                        else umma_bf16_pair<true>(d_tmem, a_lo, b_lo, idesc);
                        umma_bf16_pair<true>(d_tmem, a_lo + 2, b_lo + 2, idesc);
                        umma_bf16_pair<true>(d_tmem, a_lo + 4, b_lo + 4, idesc);
                        umma_bf16_pair<true>(d_tmem, a_lo + 6, b_lo + 6, idesc);
                        umma_commit_pair(&empty_bar[s]);     // frees the stage in both CTAs
                    } else {
                        if (kb == 0) umma_bf16<false>(d_tmem, a_lo, b_lo, idesc);
                        else umma_bf16<true>(d_tmem, a_lo, b_lo, idesc);
                        umma_bf16<true>(d_tmem, a_lo + 2, b_lo + 2, idesc);
                        umma_bf16<true>(d_tmem, a_lo + 4, b_lo + 4, idesc);
                        umma_bf16<true>(d_tmem, a_lo + 6, b_lo + 6, idesc);
                        umma_commit(&empty_bar[s]);      // frees the stage once these MMAs have read it
                    }
                    a_lo += lo_step;
                    if (++s == p.stages) { s = 0; ph ^= 1u; a_lo = a_lo0; }
                }
                if (ok) {
                    if constexpr (PAIR) umma_commit_pair(&tmem_full_bar[buf]);
                    else umma_commit(&tmem_full_bar[buf]);
                }
            }
        }
    } else {
        // ------------------------------------------------ epilogue (warps 2..9)
        // TMEM lanes 32*quarter .. +31 are the only ones warp (quarter = warp % 4) may read; the two
        // warps that share a quarter take alternate column chunks.
        const int quarter = warp & 3;
        const int half = (warp - 2) >> 2;
        const int row_in_tile = quarter * 32 + lane;
        const int n_chunks32 = p.n_tile / 32;
        const bool tail16 = (p.n_tile % 32) != 0;
        // running statistics per (quarter, column); each column is touched by exactly one lane of one warp
        if (half == 0)
            for (int c = lane; c < 256; c += 32) { run_m[quarter][c] = -INFINITY; run_s[quarter][c] = 0.f; run_i[quarter][c] = 0x7fffffff; }
        asm volatile("bar.sync 1, %0;" ::"r"(kEpilogueWarps * 32) : "memory");     // epilogue warps only
        bool ok = true;
        for (int t = 0; t < n_tiles && ok; ++t) {
            const int buf = t & 1;
            if (!mbar_wait(&tmem_full_bar[buf], ((uint32_t)t >> 1) & 1u, abort_ptr)) { ok = false; break; }
            tc_fence_after();
            TileCtx tile;
            tile.v0 = row_begin + t * tile_rows + (int)pair_rank * kVocabTile;     // this CTA's 128 rows
            tile.rows = max(0, min(kVocabTile, row_end - tile.v0));
            const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(buf * p.n_tile);
            for (int c = half; c < n_chunks32; c += 2) {
                const int col = c * 32 + lane;
                Stat running{run_m[quarter][col], run_s[quarter][col], run_i[quarter][col]};
                drain_chunk<32>(p, taddr + c * 32, lane, row_in_tile, tile, tok_base + c * 32, running);
                run_m[quarter][col] = running.m; run_s[quarter][col] = running.s; run_i[quarter][col] = running.idx;
            }
            if (tail16 && (n_chunks32 & 1) == half) {
                // lanes 2c and 2c+1 both end up with column c of the 16-column tail; the even lane keeps it
                const int col = n_chunks32 * 32 + (lane >> 1);
                Stat running{run_m[quarter][col], run_s[quarter][col], run_i[quarter][col]};
                drain_chunk<16>(p, taddr + n_chunks32 * 32, lane, row_in_tile, tile, tok_base + n_chunks32 * 32, running);
                __syncwarp();
                if ((lane & 1) == 0) { run_m[quarter][col] = running.m; run_s[quarter][col] = running.s; run_i[quarter][col] = running.idx; }
                __syncwarp();
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) {
                if constexpr (PAIR) mbar_arrive_at(cluster_addr(&tmem_empty_bar[buf], 0));   // the leader waits for both CTAs
                else mbar_arrive(&tmem_empty_bar[buf]);
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    // the CTA's statistics: merge the four lane quarters (ascending rows) into one partial slot
    for (int c = threadIdx.x; c < p.n_tile; c += kThreads) {
        const int tok = tok_base + c;
        if (tok < p.M) {
            Stat acc{run_m[0][c], run_s[0][c], run_i[0][c]};
#pragma unroll
            for (int qd = 1; qd < 4; ++qd)
                acc = stat_combine(acc, Stat{run_m[qd][c], run_s[qd][c], run_i[qd][c]}, p.scale_log2, p.greedy != 0);
            const size_t slot = (size_t)(PAIR ? group * 2 + (int)pair_rank : group) * p.M;
            if (MASSV_IN_BOUNDS(slot + tok, (size_t)p.n_part * p.M, p.dev_status)) {
                p.part_max[slot + tok] = acc.m;
                p.part_sum[slot + tok] = p.greedy ? 0.f : acc.s;
                p.part_idx[slot + tok] = acc.idx == 0x7fffffff ? acc.idx : acc.idx + p.idx_offset;
            }
        }
    }
    if constexpr (PAIR) cluster_sync_all();      // neither CTA frees TMEM or leaves while the other may still use it
    if (warp == 1) {
        __syncwarp();
        tc_fence_after();
        if constexpr (PAIR)
            asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)p.tmem_cols) : "memory");
        else
            asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)p.tmem_cols) : "memory");
    }
    if (threadIdx.x == 0 && abort_flag) set_status(p.dev_status, MASSV_ERR_TIMEOUT);
}

// 16 TMEM lanes x 64 columns -> 32 registers per thread.  Register 4k+e holds row (lane/4 + 8*(e>>1)) of the
// 16, column 8k + 2*(lane%4) + (e&1) of the 64.  (No wait: the caller waits once for all its loads.)
__device__ __forceinline__ void tmem_load_16x64(uint32_t taddr, uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.16x256b.x8.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
          "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
          "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr));
}

// Reduction of 16 per-thread values (one per column the thread sees) over the eight lanes that hold the same
// columns for other rows (lanes that differ in lane / 4): a transposed butterfly of 8 + 4 + 2 exchanges, after
// which a[0], a[1] belong to columns 2 * (lane / 4) and 2 * (lane / 4) + 1 of the thread's 16.
struct OpMax { __device__ __forceinline__ float operator()(float x, float y) const { return fmaxf(x, y); } };
struct OpAdd { __device__ __forceinline__ float operator()(float x, float y) const { return x + y; } };
struct OpMin { __device__ __forceinline__ float operator()(float x, float y) const { return fminf(x, y); } };
template <typename Op>
__device__ __forceinline__ void reduce_over_row_lanes(float (&a)[16], int lane, Op op) {
#pragma unroll
    for (int half = 8; half >= 2; half >>= 1) {
        const int offset = 2 * half;                      // 16, 8, 4
        const bool upper = (lane & offset) != 0;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            if (i < half) {
                const float send = upper ? a[i] : a[i + half];
                const float keep = upper ? a[i + half] : a[i];
                a[i] = op(keep, __shfl_xor_sync(0xffffffffu, send, offset));
            }
        }
    }
}
// The reverse: a[0], a[1] of every lane go back to all eight lanes, in column order (2 + 4 + 8 exchanges).
__device__ __forceinline__ void gather_over_row_lanes(float (&a)[16], int lane) {
#pragma unroll
    for (int have = 2; have <= 8; have <<= 1) {
        const int offset = 2 * have;                      // 4, 8, 16
        const bool upper = (lane & offset) != 0;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            if (i < have) {
                const float other = __shfl_xor_sync(0xffffffffu, a[i], offset);
                a[i + have] = upper ? a[i] : other;
                a[i] = upper ? other : a[i];
            }
        }
    }
}

// Statistics (and logits) of 64 accumulator columns x 32 vocabulary rows held by a warp in the 16x256b layout:
// va = rows 0-15 of the warp's lane quarter, vb = rows 16-31; this thread has rows g, g+8 (va) and g+16, g+24
// (vb), g = lane / 4, and the 16 columns 8k + 2*(lane%4) + {0,1}.  Four rows of a column are reduced inside
// the thread, the eight row groups by 14 exchanges - against 31 for 32 columns when every lane holds one row -
// and column c's running statistic lives with the thread that owns it after the reduction (columns 2*lane and
// 2*lane+1).  Rows are visited in ascending order across tiles, so an equal maximum later on never replaces
// the index; the index work runs only when some column's maximum rises.
__device__ __forceinline__ void stats_job64(const UmmaParams& p, uint32_t (&va)[32], uint32_t (&vb)[32], int lane, int quarter,
                                            const TileCtx& tile, int tok0, int n_cols, float* run_m, float* run_s, int* run_i) {
    const int g = lane >> 2, m4 = lane & 3;
    const bool greedy = p.greedy != 0;
    // rows of this thread: quarter * 32 + g + 8 h, h = 0..3
    bool row_ok[4];
#pragma unroll
    for (int h = 0; h < 4; ++h) row_ok[h] = quarter * 32 + g + 8 * h < tile.rows;
    const int vrow0 = tile.v0 + quarter * 32 + g;
    // value (local column i = 2k + parity, row slot h): va/vb[4k + 2*(h&1) + parity]
#define MASSV_VAL(i, h) ((h) < 2 ? va[4 * ((i) >> 1) + 2 * ((h) & 1) + ((i) & 1)] : vb[4 * ((i) >> 1) + 2 * ((h) & 1) + ((i) & 1)])
    if (p.logits != nullptr) {
#pragma unroll
        for (int i = 0; i < 16; ++i) {
            const int col = 8 * (i >> 1) + 2 * m4 + (i & 1);
            if (col < n_cols && tok0 + col < p.M) {
                float* dst = p.logits + (size_t)(tok0 + col) * p.V + vrow0;
#pragma unroll
                for (int h = 0; h < 4; ++h)
                    if (row_ok[h]) dst[8 * h] = __uint_as_float(MASSV_VAL(i, h));
            }
        }
    }
    // 1. column maxima over the thread's rows (rows and columns that do not exist count as -inf)
    float mx[16];
#pragma unroll
    for (int i = 0; i < 16; ++i) {
        const bool col_ok = 8 * (i >> 1) + 2 * m4 + (i & 1) < n_cols;
        float mi = -INFINITY;
#pragma unroll
        for (int h = 0; h < 4; ++h) {
            const float z = (row_ok[h] && col_ok) ? __uint_as_float(MASSV_VAL(i, h)) : -INFINITY;
            MASSV_VAL(i, h) = __float_as_uint(z);
            mi = fmaxf(mi, z);
        }
        mx[i] = mi;
    }
    // 2. over the eight row groups: this thread ends up with the maxima of columns 2*lane, 2*lane+1
    reduce_over_row_lanes(mx, lane, OpMax());
    const int c_own = 2 * lane;                                // first owned column within the 64
    float own_m[2] = {mx[0], mx[1]};
    float old_m[2] = {run_m[c_own], run_m[c_own + 1]};
    const bool raise0 = own_m[0] > old_m[0], raise1 = own_m[1] > old_m[1];
    const bool any_raise = __any_sync(0xffffffffu, raise0 || raise1);
    // 3. every thread needs the maxima of its 16 columns (for the index and for the exponentials)
    if (any_raise || !greedy) gather_over_row_lanes(mx, lane);
    int own_i[2] = {run_i[c_own], run_i[c_own + 1]};
    if (any_raise) {
        // lowest row attaining the maximum, per column: rows as floats (exact up to 2^24)
        float cand[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) {
            float c = 3.0e38f;
#pragma unroll
            for (int h = 3; h >= 0; --h)
                if (__uint_as_float(MASSV_VAL(i, h)) == mx[i]) c = (float)(g + 8 * h);
            cand[i] = c;
        }
        reduce_over_row_lanes(cand, lane, OpMin());
        if (raise0) own_i[0] = tile.v0 + quarter * 32 + (int)cand[0];
        if (raise1) own_i[1] = tile.v0 + quarter * 32 + (int)cand[1];
    }
    float own_s[2] = {0.f, 0.f};
    if (!greedy) {
        // 4. exponentials relative to the column's maximum in this tile, summed over the thread's rows, then over the row groups
        float cs[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) {
            const float bias = -mx[i] * p.scale_log2;
            float acc = 0.f;
#pragma unroll
            for (int h = 0; h < 4; ++h) acc += exp2f(fmaf(__uint_as_float(MASSV_VAL(i, h)), p.scale_log2, bias));
            cs[i] = mx[i] == -INFINITY ? 0.f : acc;            // an all -inf column would give NaN
        }
        reduce_over_row_lanes(cs, lane, OpAdd());
        own_s[0] = cs[0]; own_s[1] = cs[1];
    }
#undef MASSV_VAL
    // 5. fold into the running statistics of the two owned columns
#pragma unroll
    for (int e = 0; e < 2; ++e) {
        const int c = c_own + e;
        if (c < n_cols) {
            float rs = greedy ? 0.f : run_s[c];
            if (e == 0 ? raise0 : raise1) {
                const float f = old_m[e] == -INFINITY ? 0.f : exp2f((old_m[e] - own_m[e]) * p.scale_log2);
                rs = greedy ? 0.f : own_s[e] + rs * f;
                run_m[c] = own_m[e];
                run_i[c] = own_i[e];
            } else if (!greedy && own_m[e] != -INFINITY) {
                rs += own_s[e] * exp2f((own_m[e] - old_m[e]) * p.scale_log2);
            }
            if (!greedy) run_s[c] = rs;
        }
    }
}

// ---- One pass over the weights for 257 .. 384 token rows (CTA pairs only).
// The token rows are cut into two sub-tiles of n_tile <= 192 rows whose accumulators live in tensor memory
// at the same time (columns 0.. and 192..), so every weight block crosses from L2 into shared memory once
// and feeds two MMAs (the two-token-tile arrangement of lm_head_umma_kernel streams the weights twice and
// is bound by that traffic).  Tensor memory has no room for a second pair of accumulators; instead the
// twelve epilogue warps copy a finished sub-tile into registers (64 columns each) and hand its tensor
// memory back before they start on its statistics, which then run from registers while the next tile's
// MMAs are under way; the second sub-tile follows the same way.
constexpr int kDuoEpilogueWarps = 12;      // three per TMEM lane quarter
constexpr int kDuoThreads = (2 + kDuoEpilogueWarps) * 32;
constexpr int kDuoSubCols = 192;           // tensor-memory columns reserved per sub-tile
__global__ void __launch_bounds__(kDuoThreads, 1)
lm_head_duo_kernel(const __grid_constant__ CUtensorMap map_w128, const __grid_constant__ CUtensorMap map_h, const UmmaParams p) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t full_bar[kMaxStages];
    __shared__ __align__(8) uint64_t empty_bar[kMaxStages];
    __shared__ __align__(8) uint64_t tmem_full_bar;
    __shared__ __align__(8) uint64_t tmem_empty_bar[2];      // one per sub-tile's accumulator
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag;
    __shared__ float run_m[4][2 * kDuoSubCols];
    __shared__ float run_s[4][2 * kDuoSubCols];
    __shared__ int run_i[4][2 * kDuoSubCols];

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const int sub = p.n_tile;                                 // token rows per sub-tile
    const int h_rows = sub / 2;                               // rows of a sub-tile this CTA loads per K block
    const int h_bytes = h_rows * 128;
    const int stage_bytes = kTileBytesW + 2 * h_bytes;
    const int num_kb = p.K / kBlockK;
    const uint32_t pair_rank = cluster_cta_rank();
    const int group = blockIdx.x / 2;
    constexpr int tile_rows = 2 * kVocabTile;
    // This pair's tiles: tiles_per_group whole bands (fewer at the end of the vocabulary), then, where the bands
    // do not divide evenly, one sub-tile of a left-over band (the pair g ^ 1 takes the other sub-tile).
    const int n_full = max(0, min(p.tiles_per_group, p.n_bands - group * p.tiles_per_group));
    const int n_tiles = n_full + (group < 2 * p.split_rem ? 1 : 0);
    auto band_of = [&](int t) { return t < n_full ? group * p.tiles_per_group + t : (int)(gridDim.x / 2) * p.tiles_per_group + group / 2; };
    auto subs_of = [&](int t) { return t < n_full ? 3 : 1 << (group & 1); };      // bit q: sub-tile q is computed

    if (threadIdx.x == 0) {
        for (int s = 0; s < p.stages; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], 1); }
        mbar_init(&tmem_full_bar, 1);
        for (int q = 0; q < 2; ++q) mbar_init(&tmem_empty_bar[q], 2 * kDuoEpilogueWarps);     // the leader's collect both CTAs' epilogue warps
        abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {
        __syncwarp();
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_slot)), "r"((uint32_t)p.tmem_cols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();      // the peer's barriers exist before anything signals them
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_slot;
    volatile int* abort_ptr = &abort_flag;
    pdl_wait();
    pdl_trigger();

    if (warp == 0) {
        // ------------------------------------------------ TMA producer
        if (lane == 0) {
            uint64_t pol_stream, pol_keep;
            asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol_stream));
            asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol_keep));
            int s = 0;
            uint32_t ph = 0;
            uint8_t* w_dst = smem;
            bool ok = true;
            for (int t = 0; t < n_tiles && ok; ++t) {
                const int v0 = band_of(t) * tile_rows + (int)pair_rank * kVocabTile;
                const int subs = subs_of(t);
                // both CTAs' copies complete on the leader's barrier
                const uint32_t tx_pair = (uint32_t)(2 * (kTileBytesW + (subs == 3 ? 2 : 1) * h_bytes));
                for (int kb = 0; kb < num_kb; ++kb) {
                    if (!mbar_wait(&empty_bar[s], ph ^ 1u, abort_ptr)) { ok = false; break; }
                    const uint32_t bar = cluster_addr(&full_bar[s], 0);
                    if (pair_rank == 0) mbar_expect_tx_at(bar, tx_pair);
                    tma_load_2d_pair(w_dst, &map_w128, kb * kBlockK, v0, bar, pol_stream);
                    // rows past the end of the matrix are filled with zeros and still counted
                    if (subs & 1) tma_load_2d_pair(w_dst + kTileBytesW, &map_h, kb * kBlockK, (int)pair_rank * h_rows, bar, pol_keep);
                    if (subs & 2) tma_load_2d_pair(w_dst + kTileBytesW + h_bytes, &map_h, kb * kBlockK, sub + (int)pair_rank * h_rows, bar, pol_keep);
                    w_dst += stage_bytes;
                    if (++s == p.stages) { s = 0; ph ^= 1u; w_dst = smem; }
                }
            }
            if (!ok) {
                for (int i = 0; i < 64; ++i) __nanosleep(2000);       // let copies in flight land
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------ MMA issuer (the pair's leader)
        if (lane == 0 && pair_rank == 0) {
            const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(sub >> 3) << 17) | ((uint32_t)((2 * kVocabTile) >> 4) << 24);
            const uint32_t lo_step = (uint32_t)stage_bytes >> 4, h_step = (uint32_t)h_bytes >> 4;
            const uint32_t a_lo0 = umma_desc_lo(smem_u32(smem));
            int s = 0;
            uint32_t ph = 0, a_lo = a_lo0;
            bool ok = true;
            for (int t = 0; t < n_tiles && ok; ++t) {
                const int subs = subs_of(t);
                for (int kb = 0; kb < num_kb && ok; ++kb) {
                    if (!mbar_wait(&full_bar[s], ph, abort_ptr)) { ok = false; break; }
                    tc_fence_after();
#pragma unroll
                    for (int q = 0; q < 2; ++q) {
                        if (kb == 0) {       // the previous tile's accumulator has been copied out of tensor memory
                            if (!mbar_wait(&tmem_empty_bar[q], ((uint32_t)t & 1u) ^ 1u, abort_ptr)) { ok = false; break; }
                            tc_fence_after();
                        }
                        if (!((subs >> q) & 1)) continue;
                        const uint32_t d_tmem = tmem_base + (uint32_t)(q * kDuoSubCols);
                        const uint32_t b_lo = a_lo + (kTileBytesW >> 4) + (uint32_t)q * h_step;
                        if (kb == 0) umma_bf16_pair<false>(d_tmem, a_lo, b_lo, idesc);
                        else umma_bf16_pair<true>(d_tmem, a_lo, b_lo, idesc);
                        umma_bf16_pair<true>(d_tmem, a_lo + 2, b_lo + 2, idesc);
                        umma_bf16_pair<true>(d_tmem, a_lo + 4, b_lo + 4, idesc);
                        umma_bf16_pair<true>(d_tmem, a_lo + 6, b_lo + 6, idesc);
                    }
                    if (!ok) break;
                    umma_commit_pair(&empty_bar[s]);     // frees the stage in both CTAs
                    a_lo += lo_step;
                    if (++s == p.stages) { s = 0; ph ^= 1u; a_lo = a_lo0; }
                }
                if (ok) umma_commit_pair(&tmem_full_bar);
            }
        }
    } else {
        // ------------------------------------------------ epilogue (warps 2..13)
        // TMEM lanes 32*quarter .. +31 are the only ones warp (quarter = warp % 4) may read; the three warps
        // of a quarter take columns 64*part .. 64*part+63 of both sub-tiles.
        const int quarter = warp & 3;
        const int part = (warp - 2) >> 2;
        const int c0 = part * 64;                              // first column (token row within the sub-tile)
        for (int c = threadIdx.x - 64; c < 4 * 2 * kDuoSubCols; c += kDuoEpilogueWarps * 32) {
            (&run_m[0][0])[c] = -INFINITY; (&run_s[0][0])[c] = 0.f; (&run_i[0][0])[c] = 0x7fffffff;
        }
        asm volatile("bar.sync 1, %0;" ::"r"(kDuoEpilogueWarps * 32) : "memory");     // epilogue warps only
        bool ok = true;
        for (int t = 0; t < n_tiles && ok; ++t) {
            if (!mbar_wait_warp(&tmem_full_bar, (uint32_t)t & 1u, abort_ptr)) { ok = false; break; }
            tc_fence_after();
            TileCtx tile;
            tile.v0 = band_of(t) * tile_rows + (int)pair_rank * kVocabTile;        // this CTA's 128 rows
            tile.rows = max(0, min(kVocabTile, p.V - tile.v0));
            const int subs = subs_of(t);
            const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)c0;
#pragma unroll 1
            for (int q = 0; q < 2; ++q) {
                // the sub-tile's 64 columns of this warp: into registers, and tensor memory is free for the next tile
                uint32_t va[32], vb[32];
                const bool live = (subs >> q) & 1;             // a half-tile computes one sub-tile only
                if (live) {
                    tmem_load_16x64(taddr + q * kDuoSubCols, va);                              // rows 0-15 of the quarter
                    tmem_load_16x64(taddr + q * kDuoSubCols + (16u << 16), vb);                // rows 16-31
                    tmem_wait_ld<32>(va);
                    tmem_wait_ld<32>(vb);
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive_at(cluster_addr(&tmem_empty_bar[q], 0));
                if (!live) continue;
                const int n_cols = min(64, sub - c0);
                if (n_cols > 0) {                               // the same in every lane
                    const int col = q * kDuoSubCols + c0;
                    stats_job64(p, va, vb, lane, quarter, tile, q * sub + c0, n_cols, &run_m[quarter][col], &run_s[quarter][col], &run_i[quarter][col]);
                }
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    // the CTA's statistics: merge the four lane quarters (ascending rows) into one partial slot
    for (int i = threadIdx.x; i < 2 * sub; i += kDuoThreads) {
        const int c = (i / sub) * kDuoSubCols + i % sub, tok = i;
        if (tok < p.M) {
            Stat acc{run_m[0][c], run_s[0][c], run_i[0][c]};
#pragma unroll
            for (int qd = 1; qd < 4; ++qd)
                acc = stat_combine(acc, Stat{run_m[qd][c], run_s[qd][c], run_i[qd][c]}, p.scale_log2, p.greedy != 0);
            const size_t slot = (size_t)(group * 2 + (int)pair_rank) * p.M;
            if (MASSV_IN_BOUNDS(slot + tok, (size_t)p.n_part * p.M, p.dev_status)) {
                p.part_max[slot + tok] = acc.m;
                p.part_sum[slot + tok] = p.greedy ? 0.f : acc.s;
                p.part_idx[slot + tok] = acc.idx == 0x7fffffff ? acc.idx : acc.idx + p.idx_offset;
            }
        }
    }
    cluster_sync_all();      // neither CTA frees TMEM or leaves while the other may still use it
    if (warp == 1) {
        __syncwarp();
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)p.tmem_cols) : "memory");
    }
    if (threadIdx.x == 0 && abort_flag) set_status(p.dev_status, MASSV_ERR_TIMEOUT);
}

// ------------------------------------------------------------------ host side
int sm_count() {
    static int n = 0;
    if (n) return n;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0)
        n = 148;
    return n;
}

}  // namespace

// Upper bound of the partial slots the acceptance kernel may have to merge: one per CTA.
int lm_head_num_partials(int M, int V) {
    (void)M;
    const int slots = 2 * ((V + 2 * kVocabTile - 1) / (2 * kVocabTile));     // CTA pairs cover 256 rows at a time
    return slots < kMaxCtas ? slots : kMaxCtas;
}

// 257 .. 384 token rows: two sub-tiles, one pass over the weights (lm_head_duo_kernel).
static cudaError_t launch_lm_head_duo(const LmHeadParams& q, UmmaParams p, int ctas, cudaStream_t stream, int* n_part_used) {
    p.n_token_tiles = 1;
    p.n_tile = ((q.M + 1) / 2 + 15) / 16 * 16;        // rows per sub-tile, <= 192
    const int bands = (q.V + 2 * kVocabTile - 1) / (2 * kVocabTile);
    int groups = ctas / 2;
    if (groups > bands) groups = bands;
    // Whole bands per pair; a few left-over bands are cut into their two sub-tiles and dealt to the first pairs
    // (594 bands on 74 pairs: 8 each, and 4 pairs take half a band more - not 9 each on 66 pairs).
    p.n_bands = bands;
    p.tiles_per_group = bands / groups;
    p.split_rem = bands - p.tiles_per_group * groups;
    if (2 * p.split_rem > groups) {
        p.tiles_per_group = (bands + groups - 1) / groups;
        groups = (bands + p.tiles_per_group - 1) / p.tiles_per_group;
        p.split_rem = 0;
    }
    p.n_groups = groups;
    const int h_rows = p.n_tile / 2;
    const int stage_bytes = kTileBytesW + 2 * h_rows * 128;
    int stages = kRingBytes / stage_bytes;
    if (stages > kMaxStages) stages = kMaxStages;
    p.stages = stages;
    p.tmem_cols = 512;                                 // two accumulators at columns 0 and 192
    const int slots = groups * 2;
    if (slots > q.n_part) return cudaErrorInvalidValue;
    *n_part_used = slots;
    CUtensorMap map_w, map_h;
    if (!make_tensor_map_bf16_2d(&map_w, q.lm_head, q.V, q.K, kVocabTile)) return cudaErrorInvalidValue;
    if (!make_tensor_map_bf16_2d(&map_h, q.hidden, q.M, q.K, h_rows)) return cudaErrorInvalidValue;
    const size_t smem = (size_t)stages * stage_bytes + 1024;
    const TimingHooks& hooks = timing_hooks();
    if (hooks.lm_head_start && cudaEventRecord(hooks.lm_head_start, stream) != cudaSuccess) return cudaGetLastError();
    cudaError_t e = cudaFuncSetAttribute(lm_head_duo_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    e = launch_pdl_cluster(lm_head_duo_kernel, dim3(groups * 2), dim3(kDuoThreads), smem, stream, 2, map_w, map_h, p);
    if (e != cudaSuccess) return e;
    if (hooks.lm_head_stop && cudaEventRecord(hooks.lm_head_stop, stream) != cudaSuccess) return cudaGetLastError();
    count_launches(1);
    return cudaGetLastError();
}

cudaError_t launch_lm_head(const LmHeadParams& q, cudaStream_t stream, int* n_part_used) {
    UmmaParams p;
    p.M = q.M; p.K = q.K; p.V = q.V;
    int ctas = sm_count();
    if (ctas > kMaxCtas) ctas = kMaxCtas;
    p.greedy = q.greedy;
    p.scale_log2 = q.inv_T_log2e;
    p.logits = q.logits;
    p.part_max = q.part_max; p.part_sum = q.part_sum; p.part_idx = q.part_idx; p.n_part = q.n_part;
    p.dev_status = q.dev_status;
    p.idx_offset = q.idx_offset;
    p.test_skip_stage = q.test_skip_stage;
    if (q.M > 256 && q.M <= 2 * kDuoSubCols) return launch_lm_head_duo(q, p, ctas, stream, n_part_used);
    p.n_token_tiles = q.M > 256 ? 2 : 1;
    const int per_tile = (q.M + p.n_token_tiles - 1) / p.n_token_tiles;
    p.n_tile = (per_tile + 15) / 16 * 16;
    // From 64 token rows up, pairs of CTAs (cta_group::2) share the hidden-state tile: the traffic
    // from L2 into shared memory per weight byte drops from 1 + N/128 to 1 + N/256.
    const bool pair = p.n_tile >= kPairMinTile;
    const int band_rows = pair ? 2 * kVocabTile : kVocabTile;
    // Whole tiles per CTA (pair): a band with a short tail tile would run a full K loop with almost
    // nothing in flight.  Use the fewest CTAs that still reach the minimal tiles-per-CTA count
    // (1188 tiles on 148 SMs: 132 CTAs x 9 tiles).
    int groups = ctas / (p.n_token_tiles * (pair ? 2 : 1));
    const int bands = (q.V + band_rows - 1) / band_rows;
    if (groups > bands) groups = bands;
    p.tiles_per_group = (bands + groups - 1) / groups;
    groups = (bands + p.tiles_per_group - 1) / p.tiles_per_group;
    p.n_groups = groups;
    const int h_rows = pair ? p.n_tile / 2 : p.n_tile;
    const int stage_bytes = kTileBytesW + h_rows * 128;
    int stages = kRingBytes / stage_bytes;
    if (stages > kMaxStages) stages = kMaxStages;
    p.stages = stages;
    int cols = 32;
    while (cols < 2 * p.n_tile) cols *= 2;
    p.tmem_cols = cols;
    p.greedy = q.greedy;
    p.scale_log2 = q.inv_T_log2e;
    p.logits = q.logits;
    p.part_max = q.part_max; p.part_sum = q.part_sum; p.part_idx = q.part_idx; p.n_part = q.n_part;
    p.dev_status = q.dev_status;
    p.idx_offset = q.idx_offset;
    const int slots = groups * (pair ? 2 : 1);
    if (slots > q.n_part) return cudaErrorInvalidValue;
    *n_part_used = slots;

    CUtensorMap map_w[5], map_h;
    for (int i = 0; i < 5; ++i)
        if (!make_tensor_map_bf16_2d(&map_w[i], q.lm_head, q.V, q.K, kVocabTile >> i)) return cudaErrorInvalidValue;
    if (!make_tensor_map_bf16_2d(&map_h, q.hidden, q.M, q.K, h_rows)) return cudaErrorInvalidValue;

    const size_t smem = (size_t)stages * stage_bytes + 1024;
    cudaError_t e;
    const TimingHooks& hooks = timing_hooks();
    if (hooks.lm_head_start && cudaEventRecord(hooks.lm_head_start, stream) != cudaSuccess) return cudaGetLastError();
    if (pair) {
        e = cudaFuncSetAttribute(lm_head_umma_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        e = launch_pdl_cluster(lm_head_umma_kernel<true>, dim3(groups * p.n_token_tiles * 2), dim3(kThreads), smem, stream, 2,
                               map_w[0], map_w[1], map_w[2], map_w[3], map_w[4], map_h, p);
    } else {
        e = cudaFuncSetAttribute(lm_head_umma_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        e = launch_pdl(lm_head_umma_kernel<false>, dim3(groups * p.n_token_tiles), dim3(kThreads), smem, stream, map_w[0],
                       map_w[1], map_w[2], map_w[3], map_w[4], map_h, p);
    }
    if (e != cudaSuccess) return e;
    if (hooks.lm_head_stop && cudaEventRecord(hooks.lm_head_stop, stream) != cudaSuccess) return cudaGetLastError();
    count_launches(1);
    return cudaGetLastError();
}

}  // namespace massv
