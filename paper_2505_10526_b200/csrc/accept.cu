// Speculative acceptance after the LM head (paper Sec. 2.1):
//   accept_scan_kernel      reduces the per-tile softmax statistics of every block
//                           row, runs the sequential accept/reject scan, and at
//                           T == 0 also emits the extra token (the row's argmax);
//   residual_sample_kernel  T > 0: one vocabulary pass over the single row the
//                           extra token is drawn from (residual max(p-q,0) after
//                           a rejection, p itself for the bonus token), as chunk
//                           masses followed by an inverse-CDF walk in fp64;
//   probs_kernel            optional dense p = softmax(z/T) output;
//   kv_commit_kernel        advance the committed cache lengths.
// All reductions run in a fixed order, so results are bit-identical run to run.
#include "kernels.cuh"
#include "ptx.cuh"

namespace massv {

namespace {

constexpr int kScanThreads = 256;
constexpr int kScanBatch = 6;     // partial slots a lane loads before merging (192 slots = one batch)
constexpr int kSampleThreads = 256;
constexpr int kPerThread = kResidualChunk / kSampleThreads;   // 16 contiguous entries per thread
constexpr int kResidualStages = 3; // ring entries (32 KB each: the chunk's logits and the drafter's probabilities)
constexpr int kResidualThreads = kSampleThreads + 32;   // eight consumer warps and the producer warp
constexpr int kResidualCtasPerSm = 2;
constexpr int kResidualSeqCache = 8; // sequences whose scan results a CTA keeps in shared memory
constexpr int kWalkChunks = 512;  // chunk masses staged in shared memory for the walk (vocabularies up to 2M entries)
static_assert(kPerThread == 16, "chunk layout");
static_assert(kSampleThreads / 32 == kResidualSegments, "one consumer warp per segment of a chunk");

struct Stat {
    float m;   // running max logit
    float s;   // sum of exp((z - m)/T)
    int idx;   // lowest index attaining m
};

__device__ __forceinline__ Stat combine(Stat a, Stat b, float inv_T) {
    if (b.m == -INFINITY) return a;
    if (a.m == -INFINITY) return b;
    Stat r;
    r.m = fmaxf(a.m, b.m);
    r.s = a.s * expf((a.m - r.m) * inv_T) + b.s * expf((b.m - r.m) * inv_T);
    r.idx = (a.m > b.m || (a.m == b.m && a.idx < b.idx)) ? a.idx : b.idx;
    return r;
}

// One CTA per sequence, one warp per block row.  Each lane merges a strided
// share of the partial slots (independent loads), a butterfly merges the lanes,
// and warp 0 then evaluates all gamma accept tests at once (lane j = draft j) and
// takes the first failure.
__global__ void __launch_bounds__(kScanThreads) accept_scan_kernel(AcceptParams p) {
    const int b = blockIdx.x, warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int R = p.gamma + 1, M = p.B * R;
    const bool greedy = !(p.T > 0.f);
    const float inv_T = greedy ? 1.f : 1.f / p.T;
    __shared__ Stat row_stat[kMaxRows];
    static_assert(kScanThreads / 32 >= kMaxRows, "one warp per block row");
    // The drafted tokens, their uniforms and the drafter's probabilities at them are inputs of the step, not
    // results of the kernel before this one: fetch them while that kernel drains (two dependent cold reads).
    int x_in = -1;
    float u_in = 0.f, q_in = 0.f;
    if (warp == 0 && lane < p.gamma) {
        x_in = p.draft_tokens[(size_t)b * p.gamma + lane];
        if (!greedy) {
            u_in = p.u_accept[(size_t)b * p.gamma + lane];
            if (!p.q_at_draft && x_in >= 0 && x_in < p.V) q_in = p.draft_probs[((size_t)b * p.gamma + lane) * p.V + x_in];
        }
    }
    pdl_wait();
    pdl_trigger();

    if (warp < R) {
        const int row = b * R + warp;
        Stat acc{-INFINITY, 0.f, 0x7fffffff};
        for (int i0 = 0; i0 < p.n_part; i0 += 32 * kScanBatch) {
            // issue a batch of independent loads before merging them
            Stat x[kScanBatch];
#pragma unroll
            for (int k = 0; k < kScanBatch; ++k) {
                const int i = i0 + k * 32 + lane;
                x[k] = Stat{-INFINITY, 0.f, 0x7fffffff};
                if (i < p.n_part) {
                    const size_t at = p.part_per_rank
                        ? (size_t)(i / p.part_per_rank) * p.rank_stride + (size_t)(i % p.part_per_rank) * M + row
                        : (size_t)i * M + row;
                    x[k].m = p.part_max[at];
                    x[k].s = greedy ? 0.f : p.part_sum[at];
                    x[k].idx = p.part_idx[at];
                }
            }
#pragma unroll
            for (int k = 0; k < kScanBatch; ++k) acc = combine(acc, x[k], inv_T);
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            Stat y;
            y.m = __shfl_xor_sync(0xffffffffu, acc.m, o);
            y.s = __shfl_xor_sync(0xffffffffu, acc.s, o);
            y.idx = __shfl_xor_sync(0xffffffffu, acc.idx, o);
            // both partners must form the same sum: order the operands by lane
            acc = (lane & o) ? combine(y, acc, inv_T) : combine(acc, y, inv_T);
        }
        if (lane == 0) {
            row_stat[warp] = acc;
            if (p.row_stats) { p.row_stats[(size_t)row * 2] = acc.m; p.row_stats[(size_t)row * 2 + 1] = acc.s; }
        }
    }
    __syncthreads();
    if (warp != 0) return;

    bool ok = true;
    int x = -1;
    if (lane < p.gamma) {
        x = x_in;
        if (x < 0 || x >= p.V) {
            set_status(p.dev_status, MASSV_ERR_INVALID_ARG);
            ok = false;
        } else if (greedy) {
            ok = (x == row_stat[lane].idx);
        } else {
            float zx, qx;
            if (p.z_at_draft) {                 // the owner's value is the only one that is not -inf
                zx = qx = -INFINITY;
                for (int r = 0; r < p.ranks; ++r) {
                    zx = fmaxf(zx, p.z_at_draft[r * p.rank_stride + (size_t)b * p.gamma + lane]);
                    qx = fmaxf(qx, p.q_at_draft[r * p.rank_stride + (size_t)b * p.gamma + lane]);
                }
            } else {
                zx = p.logits[(size_t)(b * R + lane) * p.V + x];
                qx = q_in;
            }
            const float px = expf((zx - row_stat[lane].m) * inv_T) / row_stat[lane].s;
            const float lhs = u_in * qx;
            ok = lhs < px;
        }
    }
    const unsigned fail = __ballot_sync(0xffffffffu, !ok);
    const int n = fail ? (__ffs(fail) - 1) : p.gamma;       // first rejected draft, or gamma if none
    int32_t* toks = p.out_tokens + (size_t)b * R;
    if (lane < R) toks[lane] = lane < n ? x : -1;
    __syncwarp();
    if (lane != 0) return;
    p.accept_len[b] = n + 1;
    if (greedy) {
        toks[n] = row_stat[n].idx;
    } else {
        SeqState st;
        st.n = n;
        st.use_q = n < p.gamma ? 1 : 0;
        st.row_max = row_stat[n].m;
        st.inv_sum = 1.f / row_stat[n].s;
        p.seq_state[b] = st;
        if (p.counters) p.counters[b] = 0u;
    }
}

// A chunk of the sampled row is 4096 vocabulary entries = 1024 groups of four.  Thread t owns groups
// t, t + 256, t + 512, t + 768 (so that a warp touches consecutive 16-byte words, in shared memory as
// in global memory); r[4 j + e] is entry e of group t + 256 j.  Vocabulary order inside the chunk is
// therefore (j, t, e).
// Barrier among warps 0-7 (the kernels' 256 arithmetic threads; a ninth warp, where there is one, stays out).
__device__ __forceinline__ void bar_sync_consumers() { asm volatile("bar.sync 1, 256;" ::: "memory"); }

// p(v) = exp((z_v - max) / T) / sum, evaluated as 2^(z_v a + bias) with a = log2(e) / T and
// bias = -max a + log2(1 / sum): one multiply-add into the exponential unit.
struct RowCtx {
    float a, bias;
    __device__ RowCtx(const SeqState& st, float inv_T) {
        a = inv_T * 1.4426950408889634f;
        bias = fmaf(-st.row_max, a, log2f(st.inv_sum));
    }
    __device__ __forceinline__ float prob(float z) const { return exp2f(fmaf(z, a, bias)); }
};
__device__ __forceinline__ void masses_of(const float4 (&zz)[4], const float4 (&qq)[4], bool use_q, int valid, const RowCtx& rc,
                                          float (&r)[kPerThread]) {
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const int e0 = 4 * ((int)threadIdx.x + kSampleThreads * j);       // first entry of the group inside the chunk
        const float z[4] = {zz[j].x, zz[j].y, zz[j].z, zz[j].w}, q[4] = {qq[j].x, qq[j].y, qq[j].z, qq[j].w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            float m = 0.f;
            if (e0 + e < valid) {
                const float pv = rc.prob(z[e]);
                m = use_q ? fmaxf(pv - q[e], 0.f) : pv;
            }
            r[4 * j + e] = m;
        }
    }
}
// The same from global memory: z and q point at the chunk's first entry; `valid` entries exist (a multiple of 4).
__device__ __forceinline__ void chunk_masses_global(const float* z, const float* q, int valid, const RowCtx& rc,
                                                    float (&r)[kPerThread]) {
    float4 zz[4], qq[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const int e0 = 4 * ((int)threadIdx.x + kSampleThreads * j);
        zz[j] = make_float4(0.f, 0.f, 0.f, 0.f);
        qq[j] = make_float4(0.f, 0.f, 0.f, 0.f);
        if (e0 < valid) {
            zz[j] = *reinterpret_cast<const float4*>(z + e0);
            if (q) qq[j] = __ldg(reinterpret_cast<const float4*>(q + e0));
        }
    }
    masses_of(zz, qq, q != nullptr, valid, rc, r);
}
// Sum of the thread's 16 masses in (j, e) order, in double.
__device__ __forceinline__ double local_mass(const float (&r)[kPerThread]) {
    double s = 0.0;
#pragma unroll
    for (int i = 0; i < kPerThread; ++i) s += (double)r[i];
    return s;
}
// Block-wide sum in a fixed order (butterfly inside a warp: both partners form the same sum; warps in
// order).  Every thread receives it.  Two barriers.
__device__ __forceinline__ double block_total(double x, double* smem_warp) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
    if ((threadIdx.x & 31) == 0) smem_warp[threadIdx.x >> 5] = x;
    bar_sync_consumers();
    double tot = 0.0;
#pragma unroll
    for (int w = 0; w < kSampleThreads / 32; ++w) tot += smem_warp[w];
    bar_sync_consumers();
    return tot;
}

// Inside the chunk that holds the target: the first entry (in vocabulary order) whose running mass
// exceeds `target`, starting from `base`, and the last entry with positive mass.  r as produced by
// masses_of.  Results through s_first / s_last (shared), valid after the call for every thread.
// The four quarters of the chunk are scanned together (one pass of shuffles, two barriers); scratch holds
// 4 doubles per warp.
constexpr int kPickScratch = 4 * (kSampleThreads / 32);
__device__ __forceinline__ void pick_in_chunk(const float (&r)[kPerThread], int chunk_first_entry, double base, double target,
                                              double* scratch, int* s_first, int* s_last) {
    const int t = threadIdx.x, lane = t & 31, warp = t >> 5;
    if (t == 0) { *s_first = 0x7fffffff; *s_last = -1; }
    double g[4], incl[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {            // quarter j of the chunk: groups 256 j .. 256 j + 255, one per thread
        g[j] = ((double)r[4 * j] + (double)r[4 * j + 1]) + ((double)r[4 * j + 2] + (double)r[4 * j + 3]);
        incl[j] = g[j];
    }
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const double y = __shfl_up_sync(0xffffffffu, incl[j], o);
            if (lane >= o) incl[j] += y;
        }
    }
    if (lane == 31) {
#pragma unroll
        for (int j = 0; j < 4; ++j) scratch[warp * 4 + j] = incl[j];
    }
    bar_sync_consumers();
    int first = 0x7fffffff, last = -1;
    double run_base = base;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        double warp_base = 0.0, quarter = 0.0;              // the warps' totals in warp order
        for (int w = 0; w < kSampleThreads / 32; ++w) {
            const double s = scratch[w * 4 + j];
            if (w < warp) warp_base += s;
            quarter += s;
        }
        double run = run_base + (warp_base + incl[j] - g[j]);
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            run += (double)r[4 * j + e];
            if (r[4 * j + e] > 0.f) {
                const int v = chunk_first_entry + 4 * (t + kSampleThreads * j) + e;
                last = v;
                if (first == 0x7fffffff && run > target) first = v;
            }
        }
        run_base += quarter;
    }
    atomicMin(s_first, first);
    atomicMax(s_last, last);
    bar_sync_consumers();
}

// The sequential part of a draw, by one warp: n chunk masses (shared memory, vocabulary order) -> the chunk that
// holds u * total, the mass before it, and whether rounding pushed the target past the last positive chunk.  Lane l
// sums a contiguous run of chunks, a shuffle scan adds the lanes up (a fixed order), and the lowest lane whose
// run crosses the target wins.  s_pick[0] = chunk (-1: no mass at all), s_pick[1] = take the last positive entry,
// s_base[0] = mass before the chunk, s_base[1] = target.
__device__ __forceinline__ void walk_chunk_masses(const double* s, int n, double u, int* s_pick, double* s_base) {
    const int lane = threadIdx.x & 31;
    const int per = (n + 31) / 32;
    const int i0 = min(n, lane * per), i1 = min(n, i0 + per);
    double local = 0.0;
    for (int i = i0; i < i1; ++i) local += s[i];
    double incl = local;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const double y = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += y;
    }
    const double tot = __shfl_sync(0xffffffffu, incl, 31);
    const double target = u * tot;
    double run = incl - local, my_base = 0.0;
    int my_pick = 0x7fffffff, my_last = -1;
    for (int i = i0; i < i1; ++i) {
        const double sm = s[i];
        if (sm > 0.0) {
            my_last = i;
            if (my_pick == 0x7fffffff && run + sm > target) { my_pick = i; my_base = run; }
        }
        run += sm;
    }
    const unsigned found = __ballot_sync(0xffffffffu, my_pick != 0x7fffffff);
    const int last_pos = __reduce_max_sync(0xffffffffu, my_last);
    const int src = found ? __ffs(found) - 1 : 0;
    const int pick = __shfl_sync(0xffffffffu, my_pick, src);
    const double base = __shfl_sync(0xffffffffu, my_base, src);
    if (lane == 0) {
        s_pick[0] = tot > 0.0 ? (found ? pick : last_pos) : -1;
        s_pick[1] = found ? 0 : 1;
        s_base[0] = found ? base : 0.0;
        s_base[1] = target;
    }
}

// (No eviction hint: the chunk that turns out to hold the drawn token is read a second time, and should then
// still be in L2.)
__device__ __forceinline__ void bulk_load_1d(void* dst, const void* src, uint32_t bytes, uint64_t* bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(smem_u32(dst)), "l"(src),
                 "r"(bytes), "r"(smem_u32(bar))
                 : "memory");
}

// The sequential part of the draw for one sequence, by the 256 threads of warps 0-7: walk the chunk masses
// (fixed summation order), then find the token inside the winning chunk.
__device__ void draw_from_chunk_masses(const AcceptParams& p, int b, const SeqState& st, float inv_T, double* warp_sums, double* s_sums,
                                       int* s_pick, double* s_base, int* s_first, int* s_last) {
    const int t = threadIdx.x, R = p.gamma + 1;
    const RowCtx rc(st, inv_T);
    double* sums = p.chunk_sums + (size_t)b * p.n_chunks;
    // The walk is sequential but its loads need not be: the masses the other CTAs wrote come from L2
    // (bypassing L1) into shared memory at once.
    const bool staged = p.n_chunks <= kWalkChunks;
    const float* z_row = p.logits + (size_t)(b * R + st.n) * p.V;
    const float* q_row = p.draft_probs ? p.draft_probs + ((size_t)b * p.gamma + st.n) * p.V : nullptr;
    int use_q = st.use_q;
    for (int attempt = 0; attempt < 2; ++attempt) {
        if (staged) {
            for (int i = t; i < p.n_chunks; i += kSampleThreads) s_sums[i] = __ldcg(sums + i);
            bar_sync_consumers();
        }
        if (staged) {
            if (t < 32) walk_chunk_masses(s_sums, p.n_chunks, (double)p.u_sample[(size_t)b * R + st.n], s_pick, s_base);
        } else if (t == 0) {
            double tot = 0.0;
            for (int i = 0; i < p.n_chunks; ++i) tot += ((volatile double*)sums)[i];
            const double target = (double)p.u_sample[(size_t)b * R + st.n] * tot;
            int pick = -1, last_pos = -1;
            double cum = 0.0, base = 0.0;
            for (int i = 0; i < p.n_chunks; ++i) {
                const double sm = ((volatile double*)sums)[i];
                if (sm > 0.0) last_pos = i;
                if (pick < 0 && sm > 0.0 && cum + sm > target) { pick = i; base = cum; }
                cum += sm;
            }
            s_pick[0] = tot > 0.0 ? (pick >= 0 ? pick : last_pos) : -1;
            s_pick[1] = (pick < 0);        // rounding pushed the target past the end: take the last positive entry
            s_base[0] = base;
            s_base[1] = target;
        }
        bar_sync_consumers();
        if (s_pick[0] >= 0 || !use_q) break;
        // The residual has no mass (p == q on this row): draw from p instead.
        use_q = 0;
        for (int cc = 0; cc < p.n_chunks; ++cc) {
            float rr[kPerThread];
            chunk_masses_global(z_row + (size_t)cc * kResidualChunk, nullptr, min(kResidualChunk, p.V - cc * kResidualChunk), rc, rr);
            const double tt = block_total(local_mass(rr), warp_sums);
            if (t == 0) sums[cc] = tt;
        }
        __threadfence();       // this CTA reads the new masses back through L2 on the second attempt
        bar_sync_consumers();
    }
    const int pick = s_pick[0];
    int32_t* tok_out = p.out_tokens + (size_t)b * R + st.n;
    if (pick < 0) {                        // no mass at all (cannot happen for a softmax row)
        if (t == 0) { *tok_out = 0; set_status(p.dev_status, MASSV_ERR_INVALID_ARG); }
    } else {
        const bool take_last = s_pick[1] != 0;
        float rr[kPerThread];
        chunk_masses_global(z_row + (size_t)pick * kResidualChunk, use_q ? q_row + (size_t)pick * kResidualChunk : nullptr,
                            min(kResidualChunk, p.V - pick * kResidualChunk), rc, rr);
        pick_in_chunk(rr, pick * kResidualChunk, s_base[0], s_base[1], warp_sums, s_first, s_last);
        if (t == 0 && MASSV_IN_BOUNDS(st.n, R, p.dev_status)) {
            const int tok = (!take_last && *s_first != 0x7fffffff) ? *s_first : *s_last;
            if (MASSV_IN_BOUNDS(tok, p.V, p.dev_status)) *tok_out = tok;
        }
    }
    bar_sync_consumers();          // the shared pick state may be reused for this CTA's next sequence
}

// The same draw by ONE warp, for callers that kept the masses of every chunk's eight 512-entry segments
// (seg_sums): chunk masses -> chunk, its eight segment masses -> segment, the segment's 512 entries (16 contiguous
// ones per lane) -> token.  Three dependent reads of a few KB instead of a 32 KB chunk and four barriers of 256
// threads, and little code: this runs once per sequence at the very end of the kernel, when nothing hides its
// latency.  Returns false (in every lane) where the residual has no mass at all: the caller then takes the
// path above, which knows the fall-back to p.
__device__ __forceinline__ bool draw_by_one_warp(const AcceptParams& p, int b, const SeqState& st, float inv_T) {
    const int lane = threadIdx.x & 31, R = p.gamma + 1;
    const double* sums = p.chunk_sums + (size_t)b * p.n_chunks;
    // 1. the chunk: lane l owns a contiguous run of chunks
    const int per = (p.n_chunks + 31) / 32;
    const int i0 = min(p.n_chunks, lane * per), i1 = min(p.n_chunks, i0 + per);
    double local = 0.0;
    for (int i = i0; i < i1; ++i) local += __ldcg(sums + i);
    double incl = local;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const double y = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += y;
    }
    const double tot = __shfl_sync(0xffffffffu, incl, 31);
    if (!(tot > 0.0)) return false;
    const double target = (double)p.u_sample[(size_t)b * R + st.n] * tot;
    double run = incl - local, my_base = 0.0;
    int my_pick = 0x7fffffff, my_last = -1;
    for (int i = i0; i < i1; ++i) {
        const double sm = __ldcg(sums + i);
        if (sm > 0.0) {
            my_last = i;
            if (my_pick == 0x7fffffff && run + sm > target) { my_pick = i; my_base = run; }
        }
        run += sm;
    }
    const unsigned found = __ballot_sync(0xffffffffu, my_pick != 0x7fffffff);
    const int last_pos = __reduce_max_sync(0xffffffffu, my_last);
    const int src = found ? __ffs(found) - 1 : 0;
    const int chunk = found ? __shfl_sync(0xffffffffu, my_pick, src) : last_pos;
    double base = found ? __shfl_sync(0xffffffffu, my_base, src) : 0.0;
    bool take_last = !found;            // rounding pushed the target past the end: the last positive entry
    // 2. the segment inside the chunk: every lane walks the same eight masses
    const double* seg = p.seg_sums + ((size_t)b * p.n_chunks + chunk) * kResidualSegments;
    double sg[kResidualSegments];
#pragma unroll
    for (int j = 0; j < kResidualSegments; ++j) sg[j] = __ldcg(seg + j);
    int seg_pick = -1, seg_last = -1;
    double seg_base = base;
    {
        double r = base;
#pragma unroll
        for (int j = 0; j < kResidualSegments; ++j) {
            if (sg[j] > 0.0) {
                seg_last = j;
                if (!take_last && seg_pick < 0 && r + sg[j] > target) { seg_pick = j; seg_base = r; }
            }
            r += sg[j];
        }
    }
    if (seg_pick < 0) { seg_pick = seg_last; take_last = true; }
    // 3. the token inside the segment: 16 contiguous entries per lane
    const RowCtx rc(st, inv_T);
    const int e0 = chunk * kResidualChunk + seg_pick * (kResidualChunk / kResidualSegments) + lane * 16;
    const float* z = p.logits + (size_t)(b * R + st.n) * p.V + e0;
    const float* q = st.use_q ? p.draft_probs + ((size_t)b * p.gamma + st.n) * p.V + e0 : nullptr;
    float m[16];
    float4 zz[4], qq[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        zz[k] = make_float4(0.f, 0.f, 0.f, 0.f);
        qq[k] = make_float4(0.f, 0.f, 0.f, 0.f);
        if (e0 + 4 * k < p.V) {                      // V is a multiple of 4: a group exists whole or not at all
            zz[k] = __ldcg(reinterpret_cast<const float4*>(z) + k);
            if (q) qq[k] = __ldg(reinterpret_cast<const float4*>(q) + k);
        }
    }
    double lane_sum = 0.0;
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        const float zs[4] = {zz[k].x, zz[k].y, zz[k].z, zz[k].w}, qs[4] = {qq[k].x, qq[k].y, qq[k].z, qq[k].w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            float v = 0.f;
            if (e0 + 4 * k < p.V) {
                const float pv = rc.prob(zs[e]);
                v = q ? fmaxf(pv - qs[e], 0.f) : pv;
            }
            m[4 * k + e] = v;
            lane_sum += (double)v;
        }
    }
    double lincl = lane_sum;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const double y = __shfl_up_sync(0xffffffffu, lincl, o);
        if (lane >= o) lincl += y;
    }
    double r = seg_base + (lincl - lane_sum);
    int first = 0x7fffffff, last = -1;
#pragma unroll
    for (int i = 0; i < 16; ++i) {
        r += (double)m[i];
        if (m[i] > 0.f) {
            last = e0 + i;
            if (first == 0x7fffffff && r > target) first = e0 + i;
        }
    }
    const int tok_first = __reduce_min_sync(0xffffffffu, first);
    const int tok_last = __reduce_max_sync(0xffffffffu, last);
    if (lane == 0 && MASSV_IN_BOUNDS(st.n, R, p.dev_status)) {
        const int tok = (!take_last && tok_first != 0x7fffffff) ? tok_first : tok_last;
        if (tok >= 0 && MASSV_IN_BOUNDS(tok, p.V, p.dev_status)) p.out_tokens[(size_t)b * R + st.n] = tok;
    }
    return true;
}

// T > 0: the extra token of every sequence, one pass over the single row it is drawn from.  Work item =
// (sequence, 4096-entry chunk); a persistent grid of one wave deals the items out in contiguous runs.
// Warp 8 is the producer: it keeps a ring of items filled with bulk copies (the chunk of the row's logits
// and, after a rejection, of the drafter's distribution: two contiguous 16 KB runs), so the bytes in flight
// do not depend on registers.  Warps 0-7 are consumers that never wait for one another: each turns its
// eighth of a landed item into masses, adds them up in double (lane sums, then a butterfly: a fixed order)
// and hands its partial sum back with the stage; the producer adds the eight partials in warp order,
// stores the chunk's mass and counts the sequence's chunks.  The CTA that completes a sequence's last
// chunk makes the sequential part of the draw once its own items are done.
__global__ void __launch_bounds__(kResidualThreads, kResidualCtasPerSm) residual_sample_kernel(AcceptParams p) {
    extern __shared__ __align__(128) uint8_t res_smem[];
    __shared__ __align__(8) uint64_t full_bar[kResidualStages];     // the item's bytes have landed
    __shared__ __align__(8) uint64_t done_bar[kResidualStages];     // the eight consumer warps are done with the stage
    __shared__ double s_part[kResidualStages][kSampleThreads / 32];
    __shared__ double warp_sums[kPickScratch];
    __shared__ double s_sums[kWalkChunks];
    __shared__ SeqState s_state[kResidualSeqCache];
    __shared__ int s_pending[kResidualSeqCache], s_n_pending;
    __shared__ int s_abort;
    __shared__ int s_pick[2];
    __shared__ double s_base[2];
    __shared__ int s_first, s_last;

    const int t = threadIdx.x, warp = t >> 5, lane = t & 31;
    const int R = p.gamma + 1;
    const float inv_T = 1.f / p.T;
    const long total_items = (long)p.B * p.n_chunks;
    const int i0 = (int)((long)blockIdx.x * total_items / gridDim.x), i1 = (int)((long)(blockIdx.x + 1) * total_items / gridDim.x);
    const int n_items = i1 - i0;
    const int b_lo = i0 / p.n_chunks;
    if (t == 0) {
        for (int s = 0; s < kResidualStages; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&done_bar[s], kSampleThreads / 32); }
        s_abort = 0;
        s_n_pending = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    pdl_wait();
    pdl_trigger();
    if (n_items <= 0) return;
    {
        const int n_seq = (i1 - 1) / p.n_chunks - b_lo + 1;
        if (t < min(n_seq, kResidualSeqCache)) {
            const SeqState st = p.seq_state[b_lo + t];
            s_state[t] = st;
            // the uniform of the draw is read at the very end, by whichever CTA completes the sequence: into L2 now
            asm volatile("prefetch.global.L2 [%0];" ::"l"(p.u_sample + (size_t)(b_lo + t) * R + st.n));
        }
    }
    __syncthreads();
    auto state_of = [&](int b) -> SeqState { return b - b_lo < kResidualSeqCache ? s_state[b - b_lo] : p.seq_state[b]; };
    volatile int* abort_ptr = &s_abort;
    constexpr int kStageBytes = 2 * kResidualChunk * 4;

    if (warp == kSampleThreads / 32) {
        // ------------------------------------------------ producer
        if (lane == 0) {
            int run_cnt = 0;               // chunks of the current sequence finished since this CTA's last arrival
            bool ok = true;
            for (int k = 0; k < n_items + kResidualStages && ok; ++k) {
                const int kd = k - kResidualStages;        // the item whose stage is about to be refilled
                if (kd >= 0) {
                    const int item = i0 + kd, b = item / p.n_chunks, c = item % p.n_chunks, s = kd % kResidualStages;
                    if (!mbar_wait(&done_bar[s], ((uint32_t)(kd / kResidualStages)) & 1u, abort_ptr)) { ok = false; break; }
                    double total = 0.0;
#pragma unroll
                    for (int w = 0; w < kSampleThreads / 32; ++w) total += s_part[s][w];
                    if (MASSV_IN_BOUNDS((size_t)b * p.n_chunks + c, (size_t)p.B * p.n_chunks, p.dev_status)) {
                        p.chunk_sums[(size_t)b * p.n_chunks + c] = total;
                        if (p.seg_sums) {       // the eight warps' shares are the chunk's eight segments, in vocabulary order
                            double2* sg = reinterpret_cast<double2*>(p.seg_sums + ((size_t)b * p.n_chunks + c) * kResidualSegments);
#pragma unroll
                            for (int w = 0; w < kSampleThreads / 32; w += 2) sg[w / 2] = make_double2(s_part[s][w], s_part[s][w + 1]);
                        }
                    }
                    ++run_cnt;
                    if (kd + 1 == n_items || (item + 1) / p.n_chunks != b) {      // this CTA's last chunk of sequence b
                        __threadfence();
                        const unsigned prev = atomicAdd(&p.counters[b], (unsigned)run_cnt);
                        if (prev + (unsigned)run_cnt == (unsigned)p.n_chunks) {
                            // every chunk of b is in: the draw is this CTA's (its slot in the list is free: a CTA
                            // completes at most one sequence per sequence it holds items of).  The fence orders the
                            // other CTAs' masses, stored before their arrivals, ahead of this CTA's reads of them
                            // (which follow the barrier below).
                            __threadfence();
                            if (s_n_pending < kResidualSeqCache) s_pending[s_n_pending++] = b;
                            else set_status(p.dev_status, MASSV_ERR_UNSUPPORTED);
                        }
                        run_cnt = 0;
                    }
                }
                if (k < n_items) {
                    const int item = i0 + k, b = item / p.n_chunks, c = item % p.n_chunks, s = k % kResidualStages;
                    const SeqState st = state_of(b);
                    const uint32_t bytes = (uint32_t)min(kResidualChunk, p.V - c * kResidualChunk) * 4u;
                    uint8_t* dst = res_smem + (size_t)s * kStageBytes;
                    mbar_expect_tx(&full_bar[s], st.use_q ? 2 * bytes : bytes);
                    bulk_load_1d(dst, p.logits + (size_t)(b * R + st.n) * p.V + (size_t)c * kResidualChunk, bytes, &full_bar[s]);
                    if (st.use_q)
                        bulk_load_1d(dst + kResidualChunk * 4, p.draft_probs + ((size_t)b * p.gamma + st.n) * p.V + (size_t)c * kResidualChunk,
                                     bytes, &full_bar[s]);
                }
            }
        }
    } else {
        // ------------------------------------------------ consumers: warp w owns groups 128 w .. 128 w + 127 of the chunk
        for (int k = 0; k < n_items; ++k) {
            const int item = i0 + k, b = item / p.n_chunks, c = item % p.n_chunks, s = k % kResidualStages;
            const SeqState st = state_of(b);
            const RowCtx rc(st, inv_T);
            const int valid = min(kResidualChunk, p.V - c * kResidualChunk);
            if (!mbar_wait_warp(&full_bar[s], ((uint32_t)(k / kResidualStages)) & 1u, abort_ptr)) break;
            const float4* zs = reinterpret_cast<const float4*>(res_smem + (size_t)s * kStageBytes);
            const float4* qs = zs + kResidualChunk / 4;
            double acc[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int g = warp * 128 + i * 32 + lane;          // group of four entries
                const float4 zv = zs[g];
                float m[4] = {rc.prob(zv.x), rc.prob(zv.y), rc.prob(zv.z), rc.prob(zv.w)};
                if (st.use_q) {
                    const float4 qv = qs[g];
                    m[0] = fmaxf(m[0] - qv.x, 0.f); m[1] = fmaxf(m[1] - qv.y, 0.f);
                    m[2] = fmaxf(m[2] - qv.z, 0.f); m[3] = fmaxf(m[3] - qv.w, 0.f);
                }
                if (4 * g >= valid) { m[0] = 0.f; m[1] = 0.f; m[2] = 0.f; m[3] = 0.f; }     // past the end of the vocabulary (V % 4 == 0)
                acc[i] = ((double)m[0] + (double)m[1]) + ((double)m[2] + (double)m[3]);
            }
            double x = (acc[0] + acc[1]) + (acc[2] + acc[3]);
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
            if (lane == 0) {
                s_part[s][warp] = x;
                mbar_arrive(&done_bar[s]);         // release: the partial sum is visible to the producer's wait
            }
            __syncwarp();
        }
    }
    __syncthreads();
    if (*abort_ptr) {
        // a copy never signalled: report it, and give copies that may still be in flight time to land
        if (t == 0) {
            set_status(p.dev_status, MASSV_ERR_TIMEOUT);
            for (int i = 0; i < 64; ++i) __nanosleep(2000);
        }
        __syncthreads();
        return;
    }
    if (warp == kSampleThreads / 32) return;
    const int n_pending = s_n_pending;
    for (int i = 0; i < n_pending; ++i) {
        const int b = s_pending[i];
        if (p.seg_sums) {
            // one warp makes the draw from the segment masses; the others join only if the residual turns out empty
            if (warp == 0) {
                const bool done = draw_by_one_warp(p, b, state_of(b), inv_T);
                if (lane == 0) s_pick[0] = done ? 1 : 0;
            }
            bar_sync_consumers();
            const bool done = s_pick[0] != 0;
            bar_sync_consumers();
            if (done) continue;
        }
        draw_from_chunk_masses(p, b, state_of(b), inv_T, warp_sums, s_sums, s_pick, s_base, &s_first, &s_last);
    }
}

// ---------------------------------------------------------------- vocabulary shards
// The same arithmetic with the vocabulary cut into contiguous shards, one per rank: a shard sees Vs
// columns of the logits and of q.  Chunks are counted inside the shard; ranks in order are vocabulary order.

// Masses of the 16 entries this thread owns in chunk c of the sampled row of a shard (same layout as above).
__device__ __forceinline__ void shard_chunk_masses(const ShardParams& p, int b, const SeqState& st, int use_q, int c,
                                                   float inv_T, float (&r)[kPerThread]) {
    const int R = p.gamma + 1;
    const float* z = p.logits + (size_t)(b * R + st.n) * p.Vs + (size_t)c * kResidualChunk;
    const float* q = use_q ? p.draft_probs + ((size_t)b * p.gamma + st.n) * p.Vs + (size_t)c * kResidualChunk : nullptr;
    chunk_masses_global(z, q, min(kResidualChunk, p.Vs - c * kResidualChunk), RowCtx(st, inv_T), r);
}

// Logit and drafter probability at each drafted token this shard owns (-inf elsewhere: a maximum
// over the ranks then yields the owner's values).
__global__ void shard_gather_draft_kernel(ShardParams p) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    pdl_wait();
    if (i >= p.B * p.gamma) return;
    const int b = i / p.gamma, j = i % p.gamma, R = p.gamma + 1;
    const int x = p.draft_tokens[i] - p.vocab_offset;
    const bool mine = x >= 0 && x < p.Vs;
    p.z_at_draft[i] = mine ? p.logits[(size_t)(b * R + j) * p.Vs + x] : -INFINITY;
    if (p.q_at_draft) p.q_at_draft[i] = mine ? p.draft_probs[((size_t)b * p.gamma + j) * p.Vs + x] : -INFINITY;
}

// grid (n_chunks, B): the shard's chunk masses of the residual max(p - q, 0) and of p on the sampled row.
__global__ void __launch_bounds__(kSampleThreads) shard_masses_kernel(ShardParams p) {
    const int c = blockIdx.x, b = blockIdx.y, t = threadIdx.x;
    const float inv_T = 1.f / p.T;
    pdl_wait();
    pdl_trigger();
    const SeqState st = p.seq_state[b];
    __shared__ double warp_sums[kSampleThreads / 32];
    float r[kPerThread];
    for (int pass = 0; pass < 2; ++pass) {
        // pass 0: the distribution the extra token is drawn from; pass 1: p itself (the fall-back when
        // the residual has no mass anywhere)
        const int use_q = pass == 0 ? st.use_q : 0;
        shard_chunk_masses(p, b, st, use_q, c, inv_T, r);
        const double total = block_total(local_mass(r), warp_sums);
        if (t == 0) (pass == 0 ? p.sums_res : p.sums_p)[(size_t)b * p.n_chunks + c] = total;
        if (pass == 0 && !st.use_q) {          // the two passes coincide
            if (t == 0) p.sums_p[(size_t)b * p.n_chunks + c] = total;
            break;
        }
    }
}

// One CTA per sequence.  Every rank walks the same chunk masses of all shards; the rank whose shard holds
// the winning chunk finds the token inside it, the others store -1.
__global__ void __launch_bounds__(kSampleThreads) shard_pick_kernel(ShardParams p) {
    const int b = blockIdx.x, t = threadIdx.x;
    const int R = p.gamma + 1, n_all = p.world * p.n_chunks;
    const float inv_T = 1.f / p.T;
    pdl_wait();
    pdl_trigger();
    const SeqState st = p.seq_state[b];
    __shared__ double warp_sums[kPickScratch];
    __shared__ double s_sums[kWalkChunks];
    __shared__ int s_pick[3];
    __shared__ double s_base[2];
    __shared__ int s_first, s_last;
    if (n_all > kWalkChunks) {
        if (t == 0) { p.token_out[b] = -1; set_status(p.dev_status, MASSV_ERR_UNSUPPORTED); }
        return;
    }
    int use_q = st.use_q;
    for (int attempt = 0; attempt < 2; ++attempt) {
        // rank r's chunks of sequence b are contiguous inside r's copy of the exchange buffer
        const double* sums = use_q ? p.all_res : p.all_p;
        for (int i = t; i < n_all; i += kSampleThreads)
            s_sums[i] = sums[(size_t)(i / p.n_chunks) * p.mass_rank_stride + (size_t)b * p.n_chunks + i % p.n_chunks];
        __syncthreads();
        if (t < 32) walk_chunk_masses(s_sums, n_all, (double)p.u_sample[(size_t)b * R + st.n], s_pick, s_base);
        __syncthreads();
        if (s_pick[0] >= 0 || !use_q) break;
        use_q = 0;                             // the residual has no mass (p == q on this row): draw from p
        __syncthreads();
    }
    const int pick = s_pick[0];
    if (pick < 0) {
        if (t == 0) { p.token_out[b] = p.rank == 0 ? 0 : -1; set_status(p.dev_status, MASSV_ERR_INVALID_ARG); }
        return;
    }
    if (pick / p.n_chunks != p.rank) {         // another shard holds the chunk
        if (t == 0) p.token_out[b] = -1;
        return;
    }
    const int c = pick % p.n_chunks;
    const bool take_last = s_pick[1] != 0;
    const double base = s_base[0], target = s_base[1];
    float r[kPerThread];
    shard_chunk_masses(p, b, st, use_q, c, inv_T, r);
    pick_in_chunk(r, c * kResidualChunk, base, target, warp_sums, &s_first, &s_last);
    if (t == 0) p.token_out[b] = p.vocab_offset + ((!take_last && s_first != 0x7fffffff) ? s_first : s_last);
}

// The extra token, once the ranks have agreed on it, goes to its place after the accepted drafts.
__global__ void shard_set_token_kernel(ShardParams p) {
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    pdl_wait();
    if (b >= p.B) return;
    int tok = -1;
    for (int r = 0; r < p.world; ++r) tok = max(tok, p.tokens_in[(size_t)r * p.B + b]);
    if (tok < 0) { set_status(p.dev_status, MASSV_ERR_INVALID_ARG); return; }
    p.out_tokens[(size_t)b * (p.gamma + 1) + p.seq_state[b].n] = tok;
}

// Histogram of TVD values: per-CTA counts in shared memory, one global atomic per non-empty bin and CTA.
constexpr int kHistMaxBins = 4096;
__global__ void __launch_bounds__(256) tvd_histogram_kernel(long long n, const float* __restrict__ tvd, int bins,
                                                            unsigned long long* counts) {
    extern __shared__ unsigned int s_hist[];
    for (int k = threadIdx.x; k < bins; k += blockDim.x) s_hist[k] = 0u;
    pdl_wait();
    __syncthreads();
    const float fb = (float)bins;
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x) {
        const float t = tvd[i];
        if (t != t) continue;
        const float scaled = __fmul_rn(t, fb);               // one rounding, never contracted
        int k = scaled <= 0.f ? 0 : (scaled >= fb ? bins - 1 : (int)scaled);
        k = min(k, bins - 1);
        atomicAdd(&s_hist[k], 1u);
    }
    __syncthreads();
    for (int k = threadIdx.x; k < bins; k += blockDim.x)
        if (s_hist[k]) atomicAdd(&counts[k], (unsigned long long)s_hist[k]);
}

// grid (blocks, world): block column w copies this rank's buffer into rank w's gathered buffer.  Plain
// stores: the destination may be another GPU's memory mapped into this one's address space.
__global__ void shard_publish_kernel(PublishParams p) {
    pdl_wait();
    char* dst = static_cast<char*>(p.dst[blockIdx.y]) + (size_t)p.rank * p.bytes;
    const char* src = static_cast<const char*>(p.src);
    const size_t stride = (size_t)gridDim.x * blockDim.x, first = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    const bool wide = p.bytes % 16 == 0 && (reinterpret_cast<uintptr_t>(src) | reinterpret_cast<uintptr_t>(p.dst[blockIdx.y])) % 16 == 0;
    if (wide) {
        for (size_t i = first; i < p.bytes / 16; i += stride)
            reinterpret_cast<uint4*>(dst)[i] = reinterpret_cast<const uint4*>(src)[i];
    } else {
        for (size_t i = first; i < p.bytes / 4; i += stride)
            reinterpret_cast<uint32_t*>(dst)[i] = reinterpret_cast<const uint32_t*>(src)[i];
    }
}

// Dense probabilities for callers that ask for them (diagnostics / tests).
__global__ void probs_kernel(AcceptParams p) {
    const int R = p.gamma + 1, M = p.B * R;
    const int row = blockIdx.y;
    pdl_wait();
    if (row >= M) return;
    const float inv_T = 1.f / p.T;
    __shared__ Stat red[256];
    __shared__ Stat rs;
    Stat acc{-INFINITY, 0.f, 0x7fffffff};
    for (int i = threadIdx.x; i < p.n_part; i += blockDim.x) {
        Stat x{p.part_max[(size_t)i * M + row], p.part_sum[(size_t)i * M + row], p.part_idx[(size_t)i * M + row]};
        acc = combine(acc, x, inv_T);
    }
    red[threadIdx.x] = acc;
    __syncthreads();
    for (int w = blockDim.x / 2; w > 0; w >>= 1) {
        if (threadIdx.x < w) red[threadIdx.x] = combine(red[threadIdx.x], red[threadIdx.x + w], inv_T);
        __syncthreads();
    }
    if (threadIdx.x == 0) rs = red[0];
    __syncthreads();
    const float inv_sum = 1.f / rs.s;
    for (int v = blockIdx.x * blockDim.x + threadIdx.x; v < p.V; v += gridDim.x * blockDim.x)
        p.probs_out[(size_t)row * p.V + v] = expf((p.logits[(size_t)row * p.V + v] - rs.m) * inv_T) * inv_sum;
}

__global__ void kv_commit_kernel(int B, int gamma, const int32_t* accept_len, int32_t* seq_lens, int32_t* dev_status) {
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    pdl_wait();
    if (b >= B) return;
    const int a = accept_len[b];
    if (a < 1 || a > gamma + 1) { set_status(dev_status, MASSV_ERR_INVALID_ARG); return; }
    seq_lens[b] += a;
}

}  // namespace

cudaError_t launch_accept(const AcceptParams& p, cudaStream_t stream) {
    if (launch_pdl(accept_scan_kernel, dim3(p.B), dim3(kScanThreads), 0, stream, p) != cudaSuccess) return cudaGetLastError();
    count_launches(1);
    if (p.T > 0.f) {
        const TimingHooks& hooks = timing_hooks();
        if (hooks.residual_start && cudaEventRecord(hooks.residual_start, stream) != cudaSuccess) return cudaGetLastError();
        const size_t ring = (size_t)kResidualStages * 2 * kResidualChunk * sizeof(float);
        if (cudaFuncSetAttribute(residual_sample_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)ring) != cudaSuccess) return cudaGetLastError();
        const long items = (long)p.B * p.n_chunks;
        const long wave = (long)kResidualCtasPerSm * device_sm_count();       // one wave of resident CTAs
        if (launch_pdl(residual_sample_kernel, dim3((unsigned)(items < wave ? items : wave)), dim3(kResidualThreads), ring, stream, p) != cudaSuccess) return cudaGetLastError();
        if (hooks.residual_stop && cudaEventRecord(hooks.residual_stop, stream) != cudaSuccess) return cudaGetLastError();
        count_launches(1);
        if (p.probs_out) {
            const int M = p.B * (p.gamma + 1);
            if (launch_pdl(probs_kernel, dim3(16, M), dim3(256), 0, stream, p) != cudaSuccess) return cudaGetLastError();
            count_launches(1);
        }
    }
    return cudaGetLastError();
}

cudaError_t launch_accept_scan_only(const AcceptParams& p, cudaStream_t stream) {
    if (launch_pdl(accept_scan_kernel, dim3(p.B), dim3(kScanThreads), 0, stream, p) != cudaSuccess) return cudaGetLastError();
    count_launches(1);
    return cudaGetLastError();
}

cudaError_t launch_shard_gather_draft(const ShardParams& p, cudaStream_t stream) {
    const int n = p.B * p.gamma;
    if (n == 0) return cudaSuccess;
    if (launch_pdl(shard_gather_draft_kernel, dim3((n + 127) / 128), dim3(128), 0, stream, p) != cudaSuccess) return cudaGetLastError();
    count_launches(1);
    return cudaGetLastError();
}
cudaError_t launch_shard_masses(const ShardParams& p, cudaStream_t stream) {
    if (launch_pdl(shard_masses_kernel, dim3(p.n_chunks, p.B), dim3(kSampleThreads), 0, stream, p) != cudaSuccess) return cudaGetLastError();
    count_launches(1);
    return cudaGetLastError();
}
cudaError_t launch_shard_pick(const ShardParams& p, cudaStream_t stream) {
    if (launch_pdl(shard_pick_kernel, dim3(p.B), dim3(kSampleThreads), 0, stream, p) != cudaSuccess) return cudaGetLastError();
    count_launches(1);
    return cudaGetLastError();
}
cudaError_t launch_shard_set_token(const ShardParams& p, cudaStream_t stream) {
    if (launch_pdl(shard_set_token_kernel, dim3((p.B + 127) / 128), dim3(128), 0, stream, p) != cudaSuccess) return cudaGetLastError();
    count_launches(1);
    return cudaGetLastError();
}

cudaError_t launch_tvd_histogram(long long n, const float* tvd, int bins, unsigned long long* counts, cudaStream_t stream) {
    if (n == 0) return cudaSuccess;
    if (bins > kHistMaxBins) return cudaErrorInvalidValue;
    long long blocks = (n + 255) / 256;
    if (blocks > 2 * 148) blocks = 2 * 148;
    // a CTA sees fewer than 2^32 values: its shared counters are 32-bit
    if (launch_pdl(tvd_histogram_kernel, dim3((unsigned)blocks), dim3(256), (size_t)bins * sizeof(unsigned int), stream, n, tvd, bins,
                   counts) != cudaSuccess)
        return cudaGetLastError();
    count_launches(1);
    return cudaGetLastError();
}

cudaError_t launch_shard_publish(const PublishParams& p, cudaStream_t stream) {
    if (p.bytes == 0) return cudaSuccess;
    size_t blocks = (p.bytes / 16 + 255) / 256;
    if (blocks < 1) blocks = 1;
    if (blocks > 64) blocks = 64;
    if (launch_pdl(shard_publish_kernel, dim3((unsigned)blocks, p.world), dim3(256), 0, stream, p) != cudaSuccess) return cudaGetLastError();
    count_launches(1);
    return cudaGetLastError();
}

cudaError_t launch_kv_commit(int B, int gamma, const int32_t* accept_len, int32_t* seq_lens, int32_t* dev_status,
                             cudaStream_t stream) {
    if (accept_len == nullptr) return cudaSuccess;   // rollback: lengths stay
    if (launch_pdl(kv_commit_kernel, dim3((B + 127) / 128), dim3(128), 0, stream, B, gamma, accept_len, seq_lens, dev_status) != cudaSuccess) return cudaGetLastError();
    count_launches(1);
    return cudaGetLastError();
}

}  // namespace massv
