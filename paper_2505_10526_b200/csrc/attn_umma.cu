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
// tiles page by page with TMA into a ring, and a pair's query rows (one box per block row:
// the G heads of a KV head are adjacent) into one of two Q buffers ahead of the pair's first
// tile; warp 6 (the helper) patches the block's own K/V rows into the tiles that hold their
// positions (and stores them to their page slots: the append), so the stream of copies never
// waits for a tile to land; one thread of warp 1 issues the MMAs; warps 2-5 own 16 query rows each:
// they read S with tcgen05.ld (16x256b: the same fragment layout as a warp-level MMA
// accumulator), apply scale, causal / window mask and the online softmax, and write P
// as bf16 into shared memory for the second product.  O is rescaled in tensor memory
// only when a row's running maximum has grown by more than 2^8 since its reference
// was set (the reference cancels in O / l, so the result is the plain softmax).
//
// Two schedules share the kernel.  CHUNKED: grid (chunk, KV head, sequence) as in the warp-MMA
// kernel, one piece of work per CTA, pieces of a sequence merged by attn_combine_kernel (used
// when the caller fixes kv_chunk).  FLAT: the tiles of all (sequence, KV head) pairs form one
// line, ordered by (sequence, head, position); a persistent grid of resident CTAs cuts the line
// into equal ranges, so every CTA streams the same number of bytes whatever the mix of context
// lengths, pays its set-up once, and leaves at most two partial results (a pair that began in an
// earlier CTA, a pair that continues in the next one) to attn_flat_combine_kernel.
#include "kernels.cuh"
#include "ptx.cuh"
#include "umma.cuh"

namespace massv {

namespace {

constexpr int kUmmaRows = 64;          // MMA M: query rows per KV head, padded
// Warp 0: TMA producer; warp 1: MMA issuer and owner of the tensor-memory allocation; warps 2-5: softmax (warp w
// reads TMEM lane quarter w % 4); warp 6: helper.  (Handing the softmax warps more registers with setmaxnreg -
// roles regrouped so that they form one aligned group of four warps - measured 3 % slower on long contexts.)
constexpr int kUmmaThreads = 224;
constexpr int kProducerWarp = 0, kMmaWarp = 1, kHelperWarp = 6;
constexpr int kUmmaMaxChunkPages = 256;
constexpr int kFlatMaxBatch = 1024;    // sequences the flat schedule can index in shared memory
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
    static constexpr int kEntries = 4;                        // ring entries, filled in the order the MMAs consume them
    static constexpr int kQRegion = kUmmaRows * 128;          // (64 rows x 64 elements)
    static constexpr int kQBytes = kNCH * kQRegion;
    static constexpr int kPBytes = (TILE / 64) * kQRegion;    // P tile: 64 rows x TILE tokens, K-major
    static constexpr int kSmem = kEntries * kEntryBytes + 2 * kQBytes + kPBytes + 1024;      // Q is double buffered
    static constexpr int kColsNeeded = 2 * TILE + D;          // two S buffers and O
    static constexpr int kTmemCols = kColsNeeded <= 256 ? 256 : 512;
    static constexpr int kCtasPerSm = (kSmem <= 110 * 1024 && kTmemCols <= 256) ? 2 : 1;
};

// The MMA thread consumes tiles in the order K_0, K_1, K_2, V_0, K_3, V_1, ..., K_{n-1}, V_{n-3}, V_{n-2}, V_{n-1}:
// the score product of tile t+2 is issued as soon as the softmax warps have read S of tile t (it reuses
// that buffer), the second product of tile t once they have written P.  The ring is filled in the same
// order, so an entry is never held by a tile that is not needed yet.
__device__ __forceinline__ int ring_item_of_k(int t) { return t < 2 ? t : 2 * t - 2; }
__device__ __forceinline__ int ring_item_of_v(int t, int n_tiles) { return t >= n_tiles - 2 ? 2 * n_tiles - 2 + (t - (n_tiles - 2)) : 3 + 2 * t; }
// Inverse: item i of a segment of n tiles -> tile index, and whether it is the tile's V.
__device__ __forceinline__ void ring_item_decode(int i, int n, int& t, int& is_v) {
    if (n == 1) { t = 0; is_v = i; }
    else if (i < 2) { t = i; is_v = 0; }
    else if (i >= 2 * n - 2) { t = n - 2 + (i - (2 * n - 2)); is_v = 1; }
    else { const int j = i - 2; is_v = j & 1; t = is_v ? (j - 1) / 2 : 2 + j / 2; }
}
__device__ __forceinline__ float ex2_approx(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// One piece of work: a run of tiles of one (sequence, KV head) pair.
struct Segment {
    int b, g;
    int L;               // committed length of the sequence
    int c_begin, c_end;  // token range [c_begin, c_end), c_begin a multiple of TILE
    int n_tiles;
    float* part_o;       // where the unnormalised partial result goes; nullptr: the piece is the whole pair
    float* part_ml;
};

template <int D, int TILE, bool FLAT>
__global__ void __launch_bounds__(kUmmaThreads, UmmaAttnCfg<D, TILE>::kCtasPerSm)
attn_umma_kernel(const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_v, const __grid_constant__ CUtensorMap map_q,
                 const AttnParams p) {
    using Cfg = UmmaAttnCfg<D, TILE>;
    constexpr int E = Cfg::kEntries;
    constexpr int NCH = Cfg::kNCH;
    constexpr int UPR = D / 8;             // 16-byte units per K/V/Q row
    constexpr int PPT = TILE / kPageSize;  // pages per tile
    constexpr int GROUP = 32 / PPT;        // tiles whose page ids fit one register per lane
    static_assert(PPT * NCH <= 32 && GROUP >= 3, "one TMA box per lane; V tiles trail K tiles by at most three");

    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t ready_bar[E];     // tile complete (landed, and patched where needed)
    __shared__ __align__(8) uint64_t landed_bar[E];    // TMA bytes of a tile that still needs patching
    __shared__ __align__(8) uint64_t empty_bar[E];     // the MMAs that read the entry are done
    __shared__ __align__(8) uint64_t s_full_bar[2];    // S buffer written by Q K^T
    __shared__ __align__(8) uint64_t s_read_bar[2];    // S buffer copied to registers by the four softmax warps
    __shared__ __align__(8) uint64_t p_full_bar[2];    // P written by the four softmax warps
    __shared__ __align__(8) uint64_t pv_done_bar[2];   // P V of a tile done: P may be overwritten, O is up to date
    __shared__ __align__(8) uint64_t q_ready_bar[2];   // the query rows of a segment are in shared memory (buffer = segment & 1)
    __shared__ __align__(8) uint64_t q_free_bar[2];    // every score product of the segment that used the buffer is done
    __shared__ __align__(8) uint64_t o_free_bar;       // the four softmax warps have read a finished segment's O
    __shared__ int s_cum[FLAT ? kFlatMaxBatch + 1 : 1];   // FLAT: tiles of sequences 0 .. b-1 (per KV head)
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int G = p.Hq / p.Hkv;
    const int rows = G * p.R;
    const int rows_pad = (rows + 15) / 16 * 16;
    // barriers and tensor memory do not depend on the kernel before this one
    if (threadIdx.x == 0) {
        for (int e = 0; e < E; ++e) { mbar_init(&ready_bar[e], 1); mbar_init(&landed_bar[e], 1); mbar_init(&empty_bar[e], 1); }
        for (int i = 0; i < 2; ++i) { mbar_init(&s_full_bar[i], 1); mbar_init(&s_read_bar[i], 4); mbar_init(&p_full_bar[i], 4); mbar_init(&pv_done_bar[i], 1); }
        mbar_init(&q_ready_bar[0], 1); mbar_init(&q_ready_bar[1], 1);
        mbar_init(&q_free_bar[0], 1); mbar_init(&q_free_bar[1], 1);
        mbar_init(&o_free_bar, 4);
        abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == kMmaWarp) {
        __syncwarp();
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_slot)),
                     "r"((uint32_t)Cfg::kTmemCols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    pdl_wait();

    // ---------------------------------------------------- this CTA's share of the work
    int f = 0, f_end = 0;                 // FLAT: range of the tile line; CHUNKED: one pseudo-tile
    bool has_work = true;                 // a CTA without work still has to free its tensor memory
    if constexpr (FLAT) {
        // tiles per pair of every sequence, then an exclusive prefix sum over the batch
        for (int i = threadIdx.x; i < p.B; i += blockDim.x) {
            const int L = p.seq_lens[i];
            int n = 0;
            if (L < 0 || L + p.R > p.max_pages * kPageSize) {       // no room for the block: skip the sequence
                if (blockIdx.x == 0) set_status(p.dev_status, MASSV_ERR_CAPACITY);
            } else {
                const int lo_min = p.window > 0 ? max(0, L - p.window + 1) : 0;
                n = (L + p.R + TILE - 1) / TILE - lo_min / TILE;
            }
            s_cum[i + 1] = n;
        }
        if (threadIdx.x == 0) s_cum[0] = 0;
        __syncthreads();
        if (warp == 0) {
            const int per = (p.B + 31) / 32;
            const int i0 = min(p.B, lane * per), i1 = min(p.B, i0 + per);
            int local = 0;
            for (int i = i0; i < i1; ++i) local += s_cum[i + 1];
            int incl = local;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int v = __shfl_up_sync(0xffffffffu, incl, o);
                if (lane >= o) incl += v;
            }
            int run = incl - local;
            for (int i = i0; i < i1; ++i) { run += s_cum[i + 1]; s_cum[i + 1] = run; }
        }
        __syncthreads();
        const int total = s_cum[p.B] * p.Hkv;
        const int per_cta = max(1, (total + (int)gridDim.x - 1) / (int)gridDim.x);
        if (blockIdx.x == 0) {      // what the merge kernel needs to find the pieces of a pair
            for (int i = threadIdx.x; i <= p.B; i += blockDim.x) p.flat_meta[2 + i] = s_cum[i];
            if (threadIdx.x == 0) { p.flat_meta[0] = per_cta; p.flat_meta[1] = total; }
        }
        f = min(total, (int)blockIdx.x * per_cta);
        f_end = min(total, f + per_cta);
        has_work = f < f_end;
    } else {
        const int b = blockIdx.z, chunk = blockIdx.x;
        const int L = p.seq_lens[b];
        if (L < 0 || L + p.R > p.max_pages * kPageSize) {
            if (chunk == 0 && blockIdx.y == 0 && threadIdx.x == 0) set_status(p.dev_status, MASSV_ERR_CAPACITY);
            has_work = false;
        } else {
            const int lo_min = p.window > 0 ? max(0, L - p.window + 1) : 0;
            has_work = chunk * p.kv_chunk < L + p.R && chunk >= lo_min / p.kv_chunk;
        }
        f = 0; f_end = has_work ? 1 : 0;
    }
    const int f_first = f;
    int b_hint = 0;
    // Next piece of this CTA's share; false when the share is used up.
    auto next_segment = [&](Segment& sg) -> bool {
        if (f >= f_end) return false;
        if constexpr (FLAT) {
            // the sequence whose pairs hold tile f of the line: largest b with Hkv * cum[b] <= f
            int lo = b_hint, hi = p.B - 1;
            while (lo < hi) {
                const int mid = (lo + hi + 1) >> 1;
                if (s_cum[mid] * p.Hkv <= f) lo = mid; else hi = mid - 1;
            }
            b_hint = lo;
            const int n_b = s_cum[lo + 1] - s_cum[lo];
            const int off = f - s_cum[lo] * p.Hkv;
            const int g = off / n_b, t0 = off % n_b, t1 = min(n_b, t0 + (f_end - f));
            const int L = p.seq_lens[lo];
            const int tile_lo = (p.window > 0 ? max(0, L - p.window + 1) : 0) / TILE;
            sg.b = lo; sg.g = g; sg.L = L;
            sg.c_begin = (tile_lo + t0) * TILE;
            sg.c_end = min(L + p.R, (tile_lo + t1) * TILE);
            sg.n_tiles = t1 - t0;
            if (t0 == 0 && t1 == n_b) {
                sg.part_o = nullptr; sg.part_ml = nullptr;
            } else {
                // slot 0: the piece that opens this CTA's range; slot 1: a later piece (it can only be
                // one that runs on into the next CTA)
                size_t slot = (size_t)blockIdx.x * 2 + (f == f_first ? 0 : 1);
                if (!MASSV_IN_BOUNDS(slot, 2 * kFlatMaxCtas, p.dev_status)) slot = 0;
                sg.part_o = p.flat_part_o + slot * rows_pad * D;
                sg.part_ml = p.flat_part_ml + slot * rows_pad * 2;
            }
            f += t1 - t0;
        } else {
            const int b = blockIdx.z, g = blockIdx.y, chunk = blockIdx.x;
            const int L = p.seq_lens[b];
            const int n_ctx = L + p.R;
            const int lo_min = p.window > 0 ? max(0, L - p.window + 1) : 0;
            const int first_chunk = lo_min / p.kv_chunk;
            int c_begin = chunk * p.kv_chunk;
            if (chunk == first_chunk) c_begin += ((lo_min - c_begin) / TILE) * TILE;
            sg.b = b; sg.g = g; sg.L = L;
            sg.c_begin = c_begin;
            sg.c_end = min(n_ctx, chunk * p.kv_chunk + p.kv_chunk);
            sg.n_tiles = (sg.c_end - c_begin + TILE - 1) / TILE;
            const int n_chunks_b = (n_ctx + p.kv_chunk - 1) / p.kv_chunk - first_chunk;
            if (n_chunks_b == 1) {
                sg.part_o = nullptr; sg.part_ml = nullptr;
            } else {
                const size_t item = ((size_t)b * p.Hkv + g) * p.max_chunks + chunk;
                sg.part_o = p.part_o + item * rows_pad * D;
                sg.part_ml = p.part_ml + item * rows_pad * 2;
            }
            f = f_end;
        }
        return true;
    };

    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint8_t* q_smem = smem + E * Cfg::kEntryBytes;               // two of [NCH][64 rows][128 B], swizzled
    uint8_t* p_smem = q_smem + 2 * Cfg::kQBytes;                 // [TILE/64][64 rows][128 B], swizzled
    // query rows past the last one are never copied: zero them once in both buffers
    for (int i = threadIdx.x; i < 2 * (kUmmaRows - rows) * UPR; i += blockDim.x) {
        const int buf = i / ((kUmmaRows - rows) * UPR), k = i % ((kUmmaRows - rows) * UPR), r = rows + k / UPR, u = k % UPR;
        *reinterpret_cast<uint4*>(q_smem + buf * Cfg::kQBytes + (u / 8) * Cfg::kQRegion + swz128(r, u % 8)) = make_uint4(0u, 0u, 0u, 0u);
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");

    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_slot;
    const uint32_t tmem_o = tmem_base + 2 * TILE;
    volatile int* abort_ptr = &abort_flag;
    Segment sg;
    if (!has_work) {
        // nothing to compute: fall through to the release of tensor memory
    } else if (warp == kProducerWarp) {
        // ------------------------------------------------ TMA producer
        uint64_t policy;
        asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(policy));
        int it = 0;                      // items issued so far: ring entry it % E, use it / E
        bool ok = true;
        for (int seg = 0; ok && next_segment(sg); ++seg) {
            const int n_tiles = sg.n_tiles, L = sg.L, b = sg.b, g = sg.g;
            {
                // Query rows of the pair, ahead of its tiles: row r = block_row * G + head_in_group, and the G heads of
                // a block row are adjacent in memory, so a block row is one box per 64-element column group.  The
                // buffer's last user is the segment before the previous one.
                const int qb = seg & 1;
                if (seg >= 2) {
                    int fr = 0;
                    if (lane == 0) fr = mbar_wait(&q_free_bar[qb], ((uint32_t)((seg - 2) >> 1)) & 1u, abort_ptr) ? 1 : 0;
                    if (!__shfl_sync(0xffffffffu, fr, 0)) { ok = false; break; }
                }
                if (lane == 0) mbar_expect_tx(&q_ready_bar[qb], (uint32_t)(rows * D * 2));
                __syncwarp();
                for (int i = lane; i < p.R * NCH; i += 32) {
                    const int j = i / NCH, dc = i % NCH;
                    tma_load_2d(q_smem + qb * Cfg::kQBytes + dc * Cfg::kQRegion + j * G * 128, &map_q, dc * 64, (b * p.R + j) * p.Hq + g * G,
                                &q_ready_bar[qb], policy);
                }
            }
            // Page ids travel in registers: lane l holds the id of page 32 * group + l of the segment, for
            // the group of the most advanced K tile (cur), the one before (prev: V tiles trail K tiles by up
            // to three tiles) and the one after (next: fetched a whole group ahead, so the table lookup is
            // never on the critical path).
            const int32_t* pt = p.page_table + (size_t)b * p.max_pages + sg.c_begin / kPageSize;
            const int n_pages = (sg.c_end - sg.c_begin + kPageSize - 1) / kPageSize;
            int pid_prev = 0, pid_cur = lane < n_pages ? pt[lane] : 0, pid_next = 32 + lane < n_pages ? pt[32 + lane] : 0;
            int grp_cur = 0;
            for (int i = 0; i < 2 * n_tiles; ++i, ++it) {
                // item i of the consumption order: which tile, and whether its K or its V
                int t, is_v;
                ring_item_decode(i, n_tiles, t, is_v);
                const int e = it % E;
                if (t / GROUP > grp_cur) {           // only a K tile can be the first of a new group
                    grp_cur = t / GROUP;
                    pid_prev = pid_cur; pid_cur = pid_next;
                    const int nxt = (grp_cur + 1) * 32 + lane;
                    pid_next = nxt < n_pages ? pt[nxt] : 0;
                }
                int tile_pid[PPT];                   // ids of this tile's pages
#pragma unroll
                for (int pg = 0; pg < PPT; ++pg)
                    tile_pid[pg] = __shfl_sync(0xffffffffu, t / GROUP == grp_cur ? pid_cur : pid_prev, (t % GROUP) * PPT + pg);
                int freed = 0;
                if (lane == 0) freed = mbar_wait(&empty_bar[e], (((uint32_t)(it / E)) & 1u) ^ 1u, abort_ptr) ? 1 : 0;
                freed = __shfl_sync(0xffffffffu, freed, 0);
                if (!freed) { ok = false; break; }
                const int tile_start = sg.c_begin + t * TILE;
                const int valid = min(TILE, sg.c_end - tile_start);
                const int n_pg = (valid + kPageSize - 1) / kPageSize;
                // a tile that holds block rows or the ragged end goes to the helper warp first
                const bool patch = tile_start + TILE > L;
                uint64_t* bar = patch ? &landed_bar[e] : &ready_bar[e];
                uint8_t* dst = smem + (size_t)e * Cfg::kEntryBytes;
                if (lane == 0) mbar_expect_tx(bar, (uint32_t)(n_pg * NCH * 2048));
                __syncwarp();
                if (lane < n_pg * NCH) {             // one 16-token x 64-element box per lane
                    const int dc = lane % NCH, pg = lane / NCH;
                    int pid = tile_pid[0];
#pragma unroll
                    for (int q = 1; q < PPT; ++q) pid = pg == q ? tile_pid[q] : pid;
                    if (pid < 0 || pid >= p.num_pages) { set_status(p.dev_status, MASSV_ERR_CAPACITY); pid = 0; }
                    tma_load_2d(dst + dc * Cfg::kRegion + pg * 2048, is_v ? &map_v : &map_k, dc * 64, (pid * p.Hkv + g) * kPageSize, bar, policy);
                }
            }
        }
        if (lane == 0 && *abort_ptr) {
            for (int i = 0; i < 64; ++i) __nanosleep(2000);   // let copies in flight land
        }
    } else if (warp == kHelperWarp) {
        // ------------------------------------------------ helper: append / ragged-end patch
        uint32_t landed_phase = 0;       // bit e: parity of the next completion of landed_bar[e]
        int it_base = 0;                 // ring items of earlier segments
        bool ok = true;
        for (int seg = 0; ok && next_segment(sg); ++seg) {
            const int n_tiles = sg.n_tiles, L = sg.L, b = sg.b, g = sg.g;
            // ---- tiles that hold block rows (positions L .. L+gamma, not in the cache yet) or the ragged end: the
            // rows go into the tile and to their page slots.  They are the last tiles of the segment; their items are
            // taken in ring order, the rows fetched before the tile's own bytes are waited for.
            if (sg.c_end > L) {
                const int t_first = max(0, (L - sg.c_begin) / TILE);
                const int32_t* pt = p.page_table + (size_t)b * p.max_pages;
                for (int i = ring_item_of_k(t_first); i < 2 * n_tiles && ok; ++i) {
                    int t, is_v;
                    ring_item_decode(i, n_tiles, t, is_v);
                    if (t < t_first) continue;
                    const int e = (it_base + i) % E;
                    const int tile_start = sg.c_begin + t * TILE;
                    const int valid = min(TILE, sg.c_end - tile_start);
                    uint8_t* dst = smem + (size_t)e * Cfg::kEntryBytes;
                    const int p_first = max(L, tile_start), p_last = min(sg.c_end, tile_start + TILE);
                    const __nv_bfloat16* src_base = is_v ? p.v_new : p.k_new;
                    __nv_bfloat16* pages = is_v ? p.v_pages : p.k_pages;
                    const int n_units = (p_last - p_first) * UPR;
                    constexpr int PRE = 4;                               // units per lane fetched ahead of the wait
                    uint4 val[PRE];
                    int pid[PRE];
#pragma unroll
                    for (int k = 0; k < PRE; ++k) {
                        const int idx = k * 32 + lane;
                        if (idx < n_units) {
                            const int pos = p_first + idx / UPR, u = idx % UPR;
                            val[k] = *reinterpret_cast<const uint4*>(src_base + (((size_t)b * p.R + (pos - L)) * p.Hkv + g) * D + u * 8);
                            pid[k] = pt[pos / kPageSize];
                        }
                    }
                    if (!mbar_wait_warp(&landed_bar[e], (landed_phase >> e) & 1u, abort_ptr)) { ok = false; break; }
                    landed_phase ^= 1u << e;
                    auto put = [&](int idx, const uint4& x, int page) {
                        const int pos = p_first + idx / UPR, u = idx % UPR, row = pos - tile_start;
                        *reinterpret_cast<uint4*>(dst + (u / 8) * Cfg::kRegion + swz128(row, u % 8)) = x;
                        if (page >= 0 && page < p.num_pages)
                            *reinterpret_cast<uint4*>(pages + (((size_t)page * p.Hkv + g) * kPageSize + (pos % kPageSize)) * D + u * 8) = x;
                    };
#pragma unroll
                    for (int k = 0; k < PRE; ++k)
                        if (k * 32 + lane < n_units) put(k * 32 + lane, val[k], pid[k]);
                    for (int idx = PRE * 32 + lane; idx < n_units; idx += 32) {
                        const int pos = p_first + idx / UPR, u = idx % UPR;
                        put(idx, *reinterpret_cast<const uint4*>(src_base + (((size_t)b * p.R + (pos - L)) * p.Hkv + g) * D + u * 8), pt[pos / kPageSize]);
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
            it_base += 2 * n_tiles;
        }
    } else if (warp == kMmaWarp) {
        // ------------------------------------------------ MMA issuer
        if (lane == 0) {
            constexpr uint32_t idesc_qk = umma_idesc_bf16(kUmmaRows, TILE, false);
            constexpr uint32_t idesc_pv = umma_idesc_bf16(kUmmaRows, D, true);
            uint32_t q_lo = umma_desc_lo(smem_u32(q_smem));
            const uint32_t p_lo = umma_desc_lo(smem_u32(p_smem));
            const uint32_t ring_addr = smem_u32(smem);
            bool ok = true;
            int it_base = 0, tau_base = 0, n_tiles = 0;      // ring items / tiles of earlier segments
            int cur_seg = 0;
            // S[tau & 1] = Q K_t^T: d/16 steps of 16 elements (32 bytes) along the 128-byte rows
            auto issue_qk = [&](int t) {
                const int i = it_base + ring_item_of_k(t), e = i % E, tau = tau_base + t;
                if (!mbar_wait(&ready_bar[e], ((uint32_t)(i / E)) & 1u, abort_ptr)) { ok = false; return; }
                tc_fence_after();
                const uint32_t k_lo = umma_desc_lo(ring_addr + (uint32_t)e * Cfg::kEntryBytes);
                const uint32_t d_tmem = tmem_base + (uint32_t)((tau & 1) * TILE);
#pragma unroll
                for (int kk = 0; kk < D / 16; ++kk) {
                    const uint32_t a = q_lo + (uint32_t)(((kk >> 2) * Cfg::kQRegion + (kk & 3) * 32) >> 4);
                    const uint32_t bb = k_lo + (uint32_t)(((kk >> 2) * Cfg::kRegion + (kk & 3) * 32) >> 4);
                    if (kk == 0) umma_bf16<false>(d_tmem, a, bb, idesc_qk);
                    else umma_bf16<true>(d_tmem, a, bb, idesc_qk);
                }
                umma_commit(&empty_bar[e]);
                umma_commit(&s_full_bar[tau & 1]);
                if (t == n_tiles - 1) umma_commit(&q_free_bar[cur_seg & 1]);      // the segment's last score product: its Q buffer is free
            };
            // O (+)= P V_t: TILE/16 steps of 16 tokens; V rows are tokens, so a step is 2048 bytes
            // further and the descriptor's leading offset is the distance between 64-element column groups
            auto issue_pv = [&](int t) {
                const int i = it_base + ring_item_of_v(t, n_tiles), e = i % E, tau = tau_base + t;
                if (!mbar_wait(&ready_bar[e], ((uint32_t)(i / E)) & 1u, abort_ptr)) { ok = false; return; }
                if (!mbar_wait(&p_full_bar[tau & 1], ((uint32_t)(tau >> 1)) & 1u, abort_ptr)) { ok = false; return; }
                tc_fence_after();
                const uint32_t v_lo = (((ring_addr + (uint32_t)e * Cfg::kEntryBytes) & 0x3FFFFu) >> 4) | ((uint32_t)(Cfg::kRegion >> 4) << 16);
#pragma unroll
                for (int ks = 0; ks < TILE / 16; ++ks) {
                    const uint32_t a = p_lo + (uint32_t)(((ks >> 2) * Cfg::kQRegion + (ks & 3) * 32) >> 4);
                    const uint32_t bb = v_lo + (uint32_t)((ks * 2048) >> 4);
                    if (ks == 0 && t == 0) umma_bf16<false>(tmem_o, a, bb, idesc_pv);
                    else umma_bf16<true>(tmem_o, a, bb, idesc_pv);
                }
                umma_commit(&empty_bar[e]);
                umma_commit(&pv_done_bar[tau & 1]);
            };
            for (int seg = 0; ok && next_segment(sg); ++seg) {
                n_tiles = sg.n_tiles;
                cur_seg = seg;
                // this segment's Q has landed in its buffer
                if (!mbar_wait(&q_ready_bar[seg & 1], ((uint32_t)(seg >> 1)) & 1u, abort_ptr)) { ok = false; break; }
                q_lo = umma_desc_lo(smem_u32(q_smem + (seg & 1) * Cfg::kQBytes));
                tc_fence_after();
                for (int t = 0; t < min(2, n_tiles) && ok; ++t) {
                    // the S buffers still hold the last two tiles of the segment before until the softmax warps have read them
                    const int tau = tau_base + t;
                    if (tau >= 2 && !mbar_wait(&s_read_bar[tau & 1], ((uint32_t)((tau - 2) >> 1)) & 1u, abort_ptr)) { ok = false; break; }
                    issue_qk(t);
                }
                // the first second product overwrites O: the softmax warps must have read the finished segment's
                if (ok && seg > 0 && !mbar_wait(&o_free_bar, (uint32_t)(seg - 1) & 1u, abort_ptr)) { ok = false; break; }
                for (int t = 0; t < n_tiles && ok; ++t) {
                    if (t + 2 < n_tiles) {
                        // S of tile t is in the softmax warps' registers: its buffer takes tile t+2.  Issued here,
                        // the score MMAs run while the softmax computes, and a tcgen05.ld (which queues behind
                        // the MMAs issued before it) finds only the short second product in front of it.
                        const int tau = tau_base + t;
                        if (!mbar_wait(&s_read_bar[tau & 1], ((uint32_t)(tau >> 1)) & 1u, abort_ptr)) { ok = false; break; }
                        issue_qk(t + 2);
                    }
                    if (ok) issue_pv(t);
                }
                it_base += 2 * n_tiles;
                tau_base += n_tiles;
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
        uint8_t* p_row0 = p_smem + r0 * 128 + 4 * (lane & 3);   // this thread's 4 bytes of unit 0 of row r0 (before the swizzle)
        bool ok = true;
        int tau_base = 0;
        for (int seg = 0; ok && next_segment(sg); ++seg) {
            const int L = sg.L, b = sg.b, g = sg.g, n_tiles = sg.n_tiles, n_ctx = L + p.R;
            float m_ref[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};
            for (int t = 0; t < n_tiles && ok; ++t) {
                const int tau = tau_base + t, buf = tau & 1;
                if (!mbar_wait_warp(&s_full_bar[buf], ((uint32_t)(tau >> 1)) & 1u, abort_ptr)) { ok = false; break; }
                tc_fence_after();
                const int tile_start = sg.c_begin + t * TILE;
                // some position in the tile is hidden from some block row: ahead of row 0, or (with a
                // window) older than the last row's lower bound
                const bool need_mask = tile_start + TILE > L + 1 || (p.window > 0 && tile_start < n_ctx - p.window);
                float mx0 = -INFINITY, mx1 = -INFINITY;
                uint32_t s[TILE / 64][32];         // raw scores; the scale is applied inside the exponential
#pragma unroll
                for (int h = 0; h < TILE / 64; ++h) tmem_ld_16x64(tmem_base + lane_base + (uint32_t)(buf * TILE + h * 64), s[h]);
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(&s_read_bar[buf]);        // the buffer may take the scores of tile t+2
                if (need_mask) {
                    // only the tiles at the ragged end (and, with a window, at its lower edge) come here
#pragma unroll
                    for (int h = 0; h < TILE / 64; ++h) {
#pragma unroll
                        for (int k = 0; k < 8; ++k) {
#pragma unroll
                            for (int e = 0; e < 4; ++e) {
                                const int pos = tile_start + h * 64 + k * 8 + 2 * (lane & 3) + (e & 1);
                                const int row_pos = L + (e < 2 ? j0 : j1);
                                if (pos > row_pos || (p.window > 0 && pos < row_pos - p.window + 1)) s[h][4 * k + e] = 0xff800000u;   // -inf
                            }
                        }
                    }
                }
                {
                    // row maxima with four independent chains per row
                    float ma[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY}, mb[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
                    for (int h = 0; h < TILE / 64; ++h) {
#pragma unroll
                        for (int k = 0; k < 8; ++k) {
                            ma[k & 3] = fmaxf(ma[k & 3], fmaxf(__uint_as_float(s[h][4 * k + 0]), __uint_as_float(s[h][4 * k + 1])));
                            mb[k & 3] = fmaxf(mb[k & 3], fmaxf(__uint_as_float(s[h][4 * k + 2]), __uint_as_float(s[h][4 * k + 3])));
                        }
                    }
                    mx0 = fmaxf(fmaxf(ma[0], ma[1]), fmaxf(ma[2], ma[3]));
                    mx1 = fmaxf(fmaxf(mb[0], mb[1]), fmaxf(mb[2], mb[3]));
                }
                mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 1));
                mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 2));
                mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 1));
                mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 2));
                mx0 *= scale_log2; mx1 *= scale_log2;             // log2 domain (the scale is positive)
                // The reference maximum of a row moves only when the row's maximum has outgrown it by the
                // threshold (or when it is first set); O and l are then rescaled to the new reference.
                float f0 = 1.f, f1 = 1.f;
                bool grow = false;
                if (m_ref[0] == -INFINITY) m_ref[0] = mx0;
                else if (mx0 > m_ref[0] + kRescaleThreshold) { f0 = exp2f(m_ref[0] - mx0); m_ref[0] = mx0; grow = true; }
                if (m_ref[1] == -INFINITY) m_ref[1] = mx1;
                else if (mx1 > m_ref[1] + kRescaleThreshold) { f1 = exp2f(m_ref[1] - mx1); m_ref[1] = mx1; grow = true; }
                const float ms0 = m_ref[0] == -INFINITY ? 0.f : -m_ref[0], ms1 = m_ref[1] == -INFINITY ? 0.f : -m_ref[1];
                float la[4] = {0.f, 0.f, 0.f, 0.f}, lb[4] = {0.f, 0.f, 0.f, 0.f};      // independent partial sums
                uint32_t pk[TILE / 64][16];       // bf16 pairs: [2k] = row r0, [2k+1] = row r1, tokens 8k + 2*(lane%4) + {0,1}
#pragma unroll
                for (int h = 0; h < TILE / 64; ++h) {
#pragma unroll
                    for (int k = 0; k < 8; ++k) {
                        // 2^(s * scale * log2 e - reference): one multiply-add into the exponential unit
                        const float p0 = ex2_approx(fmaf(__uint_as_float(s[h][4 * k + 0]), scale_log2, ms0));
                        const float p1 = ex2_approx(fmaf(__uint_as_float(s[h][4 * k + 1]), scale_log2, ms0));
                        const float p2 = ex2_approx(fmaf(__uint_as_float(s[h][4 * k + 2]), scale_log2, ms1));
                        const float p3 = ex2_approx(fmaf(__uint_as_float(s[h][4 * k + 3]), scale_log2, ms1));
                        la[k & 3] += p0 + p1; lb[k & 3] += p2 + p3;
                        pk[h][2 * k] = pack_bf16x2(p0, p1);
                        pk[h][2 * k + 1] = pack_bf16x2(p2, p3);
                    }
                }
                const float ls0 = (la[0] + la[1]) + (la[2] + la[3]), ls1 = (lb[0] + lb[1]) + (lb[2] + lb[3]);
                // P and O belong to the tensor core until P V of tile t-1 is done; P V of tile t cannot
                // start before this warp has published P below.
                if (t >= 1 && !mbar_wait_warp(&pv_done_bar[(tau - 1) & 1], ((uint32_t)((tau - 1) >> 1)) & 1u, abort_ptr)) { ok = false; break; }
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
                        // (r1 = r0 + 8 has the same swizzle phase: row & 7)
                        *reinterpret_cast<uint32_t*>(p_row0 + h * Cfg::kQRegion + ((k ^ (r0 & 7)) << 4)) = pk[h][2 * k];
                        *reinterpret_cast<uint32_t*>(p_row0 + h * Cfg::kQRegion + 8 * 128 + ((k ^ (r0 & 7)) << 4)) = pk[h][2 * k + 1];
                    }
                }
                l_run[0] += ls0; l_run[1] += ls1;
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");     // P is read by the tensor core
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(&p_full_bar[buf]);
            }
            const int tau_last = tau_base + n_tiles - 1;
            if (ok && !mbar_wait_warp(&pv_done_bar[tau_last & 1], ((uint32_t)(tau_last >> 1)) & 1u, abort_ptr)) ok = false;
            tc_fence_after();
            tau_base += n_tiles;
            if (!ok) break;
            // ---- this piece's result: normalised output if it is the whole pair, else (O, max, sum)
            l_run[0] += __shfl_xor_sync(0xffffffffu, l_run[0], 1);
            l_run[0] += __shfl_xor_sync(0xffffffffu, l_run[0], 2);
            l_run[1] += __shfl_xor_sync(0xffffffffu, l_run[1], 1);
            l_run[1] += __shfl_xor_sync(0xffffffffu, l_run[1], 2);
            const bool single = sg.part_o == nullptr;
            const size_t out0 = r0 < rows ? (((size_t)b * p.R + r0 / G) * p.Hq + g * G + r0 % G) : 0;
            const size_t out1 = r1 < rows ? (((size_t)b * p.R + r1 / G) * p.Hq + g * G + r1 % G) : 0;
            // (Each case has its own loop: this code runs once or twice per CTA, from a cold instruction cache,
            // so what is not executed should not be fetched either.)
            // (debug build: one decision per warp, because the tensor-memory loads below are warp-wide)
            const bool rows_in_out = __all_sync(0xffffffffu, MASSV_IN_BOUNDS(out0, (size_t)p.B * p.R * p.Hq, p.dev_status) &&
                                                                  MASSV_IN_BOUNDS(out1, (size_t)p.B * p.R * p.Hq, p.dev_status));
            if (single) {
                const float inv0 = 1.f / l_run[0], inv1 = 1.f / l_run[1];
#pragma unroll 1
                for (int c0 = 0; c0 < D && rows_in_out; c0 += 64) {
                    uint32_t o[32];
                    tmem_ld_16x64(tmem_o + lane_base + (uint32_t)c0, o);
#pragma unroll
                    for (int k = 0; k < 8; ++k) {
                        const int c = c0 + k * 8 + 2 * (lane & 3);
                        const float a0 = __uint_as_float(o[4 * k + 0]) * inv0, a1 = __uint_as_float(o[4 * k + 1]) * inv0;
                        const float a2 = __uint_as_float(o[4 * k + 2]) * inv1, a3 = __uint_as_float(o[4 * k + 3]) * inv1;
                        if (r0 < rows) {
                            *reinterpret_cast<uint32_t*>(p.out + out0 * D + c) = pack_bf16x2(a0, a1);
                            if (p.out_f32) *reinterpret_cast<float2*>(p.out_f32 + out0 * D + c) = make_float2(a0, a1);
                        }
                        if (r1 < rows) {
                            *reinterpret_cast<uint32_t*>(p.out + out1 * D + c) = pack_bf16x2(a2, a3);
                            if (p.out_f32) *reinterpret_cast<float2*>(p.out_f32 + out1 * D + c) = make_float2(a2, a3);
                        }
                    }
                }
            } else if constexpr (FLAT) {
                // A piece of a cut pair keeps the layout the accumulator has in registers: unit
                // ((qd * D/64 + c0/64) * 8 + k) * 32 + lane is one 16-byte store of (row r0: columns c, c+1; row r1:
                // the same columns), c = c0 + 8k + 2 (lane % 4).  The merge kernel reads it back the same way.
                if (qd * 16 < rows) {
                    float4* dst = reinterpret_cast<float4*>(sg.part_o) + (size_t)(qd * NCH) * 8 * 32 + lane;
#pragma unroll 1
                    for (int c0 = 0; c0 < D; c0 += 64) {
                        uint32_t o[32];
                        tmem_ld_16x64(tmem_o + lane_base + (uint32_t)c0, o);
#pragma unroll
                        for (int k = 0; k < 8; ++k)
                            dst[((c0 / 64) * 8 + k) * 32] = make_float4(__uint_as_float(o[4 * k + 0]), __uint_as_float(o[4 * k + 1]),
                                                                        __uint_as_float(o[4 * k + 2]), __uint_as_float(o[4 * k + 3]));
                    }
                }
            } else {
#pragma unroll 1
                for (int c0 = 0; c0 < D; c0 += 64) {
                    uint32_t o[32];
                    tmem_ld_16x64(tmem_o + lane_base + (uint32_t)c0, o);
#pragma unroll
                    for (int k = 0; k < 8; ++k) {
                        const int c = c0 + k * 8 + 2 * (lane & 3);
                        if (r0 < rows) *reinterpret_cast<float2*>(sg.part_o + (size_t)r0 * D + c) = make_float2(__uint_as_float(o[4 * k + 0]), __uint_as_float(o[4 * k + 1]));
                        if (r1 < rows) *reinterpret_cast<float2*>(sg.part_o + (size_t)r1 * D + c) = make_float2(__uint_as_float(o[4 * k + 2]), __uint_as_float(o[4 * k + 3]));
                    }
                }
            }
            // O is in registers or on its way to memory: the next segment's second product may overwrite it
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&o_free_bar);
            if ((lane & 3) == 0) {
                if (single) {
                    if (p.lse && rows_in_out) {
                        if (r0 < rows) p.lse[out0] = (m_ref[0] + log2f(l_run[0])) * 0.6931471805599453f;
                        if (r1 < rows) p.lse[out1] = (m_ref[1] + log2f(l_run[1])) * 0.6931471805599453f;
                    }
                } else {
                    if (r0 < rows) { sg.part_ml[r0 * 2] = m_ref[0]; sg.part_ml[r0 * 2 + 1] = l_run[0]; }
                    if (r1 < rows) { sg.part_ml[r1 * 2] = m_ref[1]; sg.part_ml[r1 * 2 + 1] = l_run[1]; }
                }
            }
        }
    }

    pdl_trigger();
    tc_fence_before();
    __syncthreads();
    if (warp == kMmaWarp) {
        __syncwarp();
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)Cfg::kTmemCols) : "memory");
    }
    if (threadIdx.x == 0 && abort_flag) set_status(p.dev_status, MASSV_ERR_TIMEOUT);
}

// Merge the pieces of every (sequence, KV head) pair that the flat schedule cut.  The pieces of a pair sit in
// consecutive CTAs of the split kernel; piece c is in slot 0 of CTA c unless the pair begins inside that CTA's
// range.  A piece has the layout of the accumulator in registers (see the split kernel): unit
// ((qd * d/64 + ch) * 8 + k) * 32 + lane holds rows qd*16 + lane/4 (.x, .y) and +8 (.z, .w), columns
// ch*64 + 8k + 2*(lane%4) + {0, 1}.  grid (pair, qd * parts + part): a CTA merges `units_per_cta` units of one
// group of 16 rows, so it needs the weights of those rows only.  Pieces are summed in a fixed order.
constexpr int kFlatCombineThreads = 256;
__global__ void __launch_bounds__(kFlatCombineThreads) attn_flat_combine_kernel(const AttnParams p, int rows_pad, int parts, int units_per_cta) {
    const int G = p.Hq / p.Hkv, rows = G * p.R;
    const int g = blockIdx.x % p.Hkv, b = blockIdx.x / p.Hkv;
    const int qd = blockIdx.y / parts, part = blockIdx.y % parts;
    pdl_wait();
    pdl_trigger();
    const int per_cta = p.flat_meta[0];
    const int cum_b = p.flat_meta[2 + b], n_b = p.flat_meta[2 + b + 1] - cum_b;
    if (n_b <= 0) return;
    const int start = cum_b * p.Hkv + g * n_b, end = start + n_b;
    const int c_first = start / per_cta, c_last = (end - 1) / per_cta;
    if (c_first == c_last) return;                 // the pair was finished by one CTA
    const int n = c_last - c_first + 1;
    auto slot_of = [&](int i) -> size_t { const int c = c_first + i; return (size_t)c * 2 + (start <= c * per_cta ? 0 : 1); };
    extern __shared__ float4 s_red[];              // [kFlatCombineThreads]: partial sums of the piece groups (below)
    float* s_w = reinterpret_cast<float*>(s_red + kFlatCombineThreads);   // [n][16]: first the piece maxima, then the merge weights
    float* s_l = s_w + (size_t)n * 16;             // [n][16]: the pieces' sums
    float* s_inv = s_l + (size_t)n * 16;           // [16]
    // every (piece, row) pair's (max, sum) with one load per thread: a pair cut into dozens of pieces
    // must not walk them one latency after the other
    for (int idx = threadIdx.x; idx < n * 16; idx += blockDim.x) {
        const int i = idx / 16, r = qd * 16 + idx % 16;
        float2 ml = make_float2(-INFINITY, 0.f);
        if (r < rows) ml = *reinterpret_cast<const float2*>(p.flat_part_ml + (slot_of(i) * rows_pad + r) * 2);
        s_w[idx] = ml.x;
        s_l[idx] = ml.y;
    }
    __syncthreads();
    if (threadIdx.x < 16) {
        const int rr = threadIdx.x, r = qd * 16 + rr;
        float M = -INFINITY;
        for (int i = 0; i < n; ++i) M = fmaxf(M, s_w[i * 16 + rr]);
        float Lsum = 0.f;
        for (int i = 0; i < n; ++i) {
            const float mi = s_w[i * 16 + rr];
            const float w = mi == -INFINITY ? 0.f : exp2f(mi - M);
            s_w[i * 16 + rr] = w;
            Lsum += s_l[i * 16 + rr] * w;
        }
        s_inv[rr] = 1.f / Lsum;
        if (p.lse && part == 0 && r < rows) p.lse[((size_t)b * p.R + r / G) * p.Hq + g * G + r % G] = (M + log2f(Lsum)) * 0.6931471805599453f;
    }
    __syncthreads();
    const int nch = p.d / 64;
    const int unit0 = qd * nch * 256 + part * units_per_cta;       // first unit of this CTA within a piece
    const float4* pieces = reinterpret_cast<const float4*>(p.flat_part_o);
    const size_t piece_units = (size_t)rows_pad * p.d / 4;
    auto store_unit = [&](int idx, float4 acc) {
        const int u = part * units_per_cta + idx;                   // unit within the row group
        const int lane = u % 32, k = (u / 32) % 8, ch = u / 256;
        const int rr = lane / 4, c = ch * 64 + k * 8 + 2 * (lane % 4);
        const float i0 = s_inv[rr], i1 = s_inv[rr + 8];
        acc.x *= i0; acc.y *= i0; acc.z *= i1; acc.w *= i1;
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int r = qd * 16 + rr + 8 * h;
            if (r < rows) {
                const size_t row_out = ((size_t)b * p.R + r / G) * p.Hq + g * G + r % G;
                const float x = h ? acc.z : acc.x, y = h ? acc.w : acc.y;
                *reinterpret_cast<uint32_t*>(p.out + row_out * p.d + c) = pack_bf16x2(x, y);
                if (p.out_f32) *reinterpret_cast<float2*>(p.out_f32 + row_out * p.d + c) = make_float2(x, y);
            }
        }
    };
    auto add_piece = [&](float4& acc, int i, int idx) {
        const float4 v = pieces[slot_of(i) * piece_units + unit0 + idx];
        const int rr = ((part * units_per_cta + idx) % 32) / 4;
        const float w0 = s_w[i * 16 + rr], w1 = s_w[i * 16 + rr + 8];
        acc.x += v.x * w0; acc.y += v.y * w0; acc.z += v.z * w1; acc.w += v.w * w1;
    };
    // Few units and many pieces (a short batch cut across the whole grid): several threads share a unit,
    // thread group k summing pieces k, k + groups, ... with all its loads in flight at once; the groups'
    // sums are then added in group order.  The order of the sums is fixed, so results repeat.
    const int groups = (int)blockDim.x / units_per_cta;
    if (groups >= 2 && n >= 4) {
        const int grp = threadIdx.x / units_per_cta, idx = threadIdx.x % units_per_cta;
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        if (grp < groups) {
#pragma unroll 4
            for (int i = grp; i < n; i += groups) add_piece(acc, i, idx);
            s_red[threadIdx.x] = acc;
        }
        __syncthreads();
        if (grp == 0) {
            for (int k = 1; k < groups; ++k) {
                const float4 v = s_red[k * units_per_cta + idx];
                acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
            }
            store_unit(idx, acc);
        }
        return;
    }
    for (int idx = threadIdx.x; idx < units_per_cta; idx += blockDim.x) {
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll 4
        for (int i = 0; i < n; ++i) add_piece(acc, i, idx);      // summed in piece order, four loads in flight
        store_unit(idx, acc);
    }
}

int flat_sm_count() {
    static int n = 0;
    if (n) return n;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0)
        n = 148;
    return n;
}

template <int D, int TILE>
cudaError_t launch_umma(const AttnParams& p, const CUtensorMap& mk, const CUtensorMap& mv, cudaStream_t stream, bool flat, int* launched,
                        cudaEvent_t split_done) {
    using Cfg = UmmaAttnCfg<D, TILE>;
    // the query rows as a [B * R * Hq, D] matrix; a box is the G adjacent heads of one block row
    CUtensorMap mq;
    if (!make_tensor_map_bf16_2d(&mq, p.q, (uint64_t)p.B * p.R * p.Hq, D, (uint32_t)(p.Hq / p.Hkv))) return cudaErrorInvalidValue;
    static_assert(Cfg::kColsNeeded <= 512, "S buffers and O fit tensor memory");
    static_assert(Cfg::kSmem <= 227 * 1024, "ring, Q and P fit shared memory");
    cudaError_t e;
    if (flat) {
        e = cudaFuncSetAttribute(attn_umma_kernel<D, TILE, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg::kSmem);
        if (e != cudaSuccess) return e;
        int ctas = flat_sm_count() * Cfg::kCtasPerSm;
        if (ctas > kFlatMaxCtas) ctas = kFlatMaxCtas;
        e = launch_pdl(attn_umma_kernel<D, TILE, true>, dim3(ctas), dim3(kUmmaThreads), (size_t)Cfg::kSmem, stream, mk, mv, mq, p);
        if (e != cudaSuccess) return e;
        if (split_done && cudaEventRecord(split_done, stream) != cudaSuccess) return cudaGetLastError();
        const int rows = (p.Hq / p.Hkv) * p.R;
        // enough CTAs to fill the machine: a pair's groups of 16 rows go to separate CTAs, and with few pairs a
        // group's units (D/64 * 256 of them) are cut further into 2, 4, 8 or 16 parts
        const int pairs = p.B * p.Hkv, rows_pad = attn_rows_pad(rows), n_qd = rows_pad / 16, units_per_qd = (D / 64) * 256;
        int parts = 1;
        while (parts < 16 && units_per_qd / (parts * 2) >= 32 && pairs * n_qd * parts < 2 * flat_sm_count()) parts *= 2;
        // (max, sum) and weight of 16 rows for at most `ctas` pieces of a pair (a pair can span every CTA)
        const size_t comb_smem = (2 * (size_t)ctas + 1) * 16 * sizeof(float) + kFlatCombineThreads * sizeof(float4);
        e = cudaFuncSetAttribute(attn_flat_combine_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)comb_smem);
        if (e != cudaSuccess) return e;
        e = launch_pdl(attn_flat_combine_kernel, dim3(pairs, n_qd * parts), dim3(kFlatCombineThreads), comb_smem, stream, p, rows_pad, parts,
                       units_per_qd / parts);
        *launched = 2;
        return e;
    }
    e = cudaFuncSetAttribute(attn_umma_kernel<D, TILE, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg::kSmem);
    if (e != cudaSuccess) return e;
    *launched = 1;
    return launch_pdl(attn_umma_kernel<D, TILE, false>, dim3(p.max_chunks, p.Hkv, p.B), dim3(kUmmaThreads), (size_t)Cfg::kSmem, stream, mk, mv, mq, p);
}

}  // namespace

bool attn_umma_supported(const AttnParams& p) {
    return (p.Hq / p.Hkv) * p.R <= kUmmaRows && (p.d == 64 || p.d == 128 || p.d == 256) &&
           p.kv_chunk <= kUmmaMaxChunkPages * kPageSize && p.kv_chunk % 64 == 0;
}

// The flat schedule needs the batch's tile counts in shared memory.
bool attn_umma_flat_supported(const AttnParams& p) { return attn_umma_supported(p) && p.B <= kFlatMaxBatch; }

// *launched: kernels launched; *needs_chunk_combine: the chunk merge kernel still has to run.
cudaError_t launch_attn_umma(const AttnParams& p, const CUtensorMap& mk, const CUtensorMap& mv, cudaStream_t stream, bool flat,
                             int* launched, cudaEvent_t split_done) {
    switch (p.d) {
        case 64: return launch_umma<64, 64>(p, mk, mv, stream, flat, launched, split_done);
        case 128: return launch_umma<128, 64>(p, mk, mv, stream, flat, launched, split_done);
        case 256: return launch_umma<256, 64>(p, mk, mv, stream, flat, launched, split_done);
        default: return cudaErrorInvalidValue;
    }
}

}  // namespace massv
