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

namespace massv {

namespace {

constexpr int kScanThreads = 256;
constexpr int kScanBatch = 6;     // partial slots a lane loads before merging (192 slots = one batch)
constexpr int kSampleThreads = 256;
constexpr int kPerThread = kResidualChunk / kSampleThreads;   // 16 contiguous entries per thread
constexpr int kWalkChunks = 512;  // chunk masses staged in shared memory for the walk (vocabularies up to 2M entries)
static_assert(kPerThread == 16, "chunk layout");

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
        if (lane == 0) row_stat[warp] = acc;
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

// Masses of the 16 entries this thread owns in chunk c of the sampled row.
__device__ __forceinline__ void chunk_masses(const AcceptParams& p, int b, const SeqState& st, int use_q, int c,
                                             float inv_T, float (&r)[kPerThread]) {
    const int R = p.gamma + 1;
    const int v0 = c * kResidualChunk + threadIdx.x * kPerThread;
    const float* z = p.logits + (size_t)(b * R + st.n) * p.V;
    const float* q = use_q ? p.draft_probs + ((size_t)b * p.gamma + st.n) * p.V : nullptr;
#pragma unroll
    for (int g = 0; g < kPerThread; g += 4) {
        const int v = v0 + g;
        float zz[4] = {0.f, 0.f, 0.f, 0.f}, qq[4] = {0.f, 0.f, 0.f, 0.f};
        if (v + 3 < p.V) {
            const float4 a = *reinterpret_cast<const float4*>(z + v);
            zz[0] = a.x; zz[1] = a.y; zz[2] = a.z; zz[3] = a.w;
            if (q) {
                const float4 d = __ldg(reinterpret_cast<const float4*>(q + v));
                qq[0] = d.x; qq[1] = d.y; qq[2] = d.z; qq[3] = d.w;
            }
        } else {
            for (int e = 0; e < 4; ++e)
                if (v + e < p.V) { zz[e] = z[v + e]; if (q) qq[e] = q[v + e]; }
        }
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            float m = 0.f;
            if (v + e < p.V) {
                const float pv = expf((zz[e] - st.row_max) * inv_T) * st.inv_sum;
                m = q ? fmaxf(pv - qq[e], 0.f) : pv;
            }
            r[g + e] = m;
        }
    }
}

// Block-wide exclusive prefix of one double per thread, in thread order; *total gets the sum.
__device__ __forceinline__ double block_exclusive_scan(double x, double* smem_warp, double* total) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    double incl = x;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const double y = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += y;
    }
    if (lane == 31) smem_warp[warp] = incl;
    __syncthreads();
    double base = 0.0, tot = 0.0;
    for (int w = 0; w < kSampleThreads / 32; ++w) {
        const double s = smem_warp[w];
        if (w < warp) base += s;
        tot += s;
    }
    __syncthreads();
    *total = tot;
    return base + incl - x;
}

// grid (n_chunks, B).  Every CTA stores its chunk's mass; the CTA that arrives
// last for a sequence walks the chunk masses and then the winning chunk.
__global__ void __launch_bounds__(kSampleThreads) residual_sample_kernel(AcceptParams p) {
    const int c = blockIdx.x, b = blockIdx.y, t = threadIdx.x;
    const int R = p.gamma + 1;
    const float inv_T = 1.f / p.T;
    pdl_wait();
    pdl_trigger();
    const SeqState st = p.seq_state[b];
    __shared__ double warp_sums[kSampleThreads / 32];
    __shared__ int s_flag;
    __shared__ int s_pick[2];
    __shared__ double s_base[2];

    float r[kPerThread];
    chunk_masses(p, b, st, st.use_q, c, inv_T, r);
    double local = 0.0;
#pragma unroll
    for (int e = 0; e < kPerThread; ++e) local += (double)r[e];
    double total;
    block_exclusive_scan(local, warp_sums, &total);
    double* sums = p.chunk_sums + (size_t)b * p.n_chunks;
    if (t == 0) {
        sums[c] = total;
        __threadfence();
        const unsigned prev = atomicAdd(&p.counters[b], 1u);
        s_flag = (prev == (unsigned)p.n_chunks - 1u);
    }
    __syncthreads();
    if (!s_flag) return;
    __threadfence();

    // The walk over the chunk masses is sequential (fixed summation order) but its loads need not be:
    // the CTA fetches the masses the other CTAs wrote (L2, bypassing L1) into shared memory at once.
    __shared__ double s_sums[kWalkChunks];
    const bool staged = p.n_chunks <= kWalkChunks;
    int use_q = st.use_q;
    for (int attempt = 0; attempt < 2; ++attempt) {
        if (staged) {
            for (int i = t; i < p.n_chunks; i += kSampleThreads) s_sums[i] = __ldcg(sums + i);
            __syncthreads();
        }
        if (t == 0) {
            double tot = 0.0;
            for (int i = 0; i < p.n_chunks; ++i) tot += staged ? s_sums[i] : ((volatile double*)sums)[i];
            const double target = (double)p.u_sample[(size_t)b * R + st.n] * tot;
            int pick = -1, last_pos = -1;
            double cum = 0.0, base = 0.0;
            for (int i = 0; i < p.n_chunks; ++i) {
                const double s = staged ? s_sums[i] : ((volatile double*)sums)[i];
                if (s > 0.0) last_pos = i;
                if (pick < 0 && s > 0.0 && cum + s > target) { pick = i; base = cum; }
                cum += s;
            }
            s_pick[0] = tot > 0.0 ? (pick >= 0 ? pick : last_pos) : -1;
            s_pick[1] = (pick < 0);        // rounding pushed the target past the end: take the last positive entry
            s_base[0] = base;
            s_base[1] = target;
        }
        __syncthreads();
        if (s_pick[0] >= 0 || !use_q) break;
        // The residual has no mass (p == q on this row): draw from p instead.
        use_q = 0;
        for (int cc = 0; cc < p.n_chunks; ++cc) {
            chunk_masses(p, b, st, 0, cc, inv_T, r);
            double loc = 0.0;
#pragma unroll
            for (int e = 0; e < kPerThread; ++e) loc += (double)r[e];
            double tt;
            block_exclusive_scan(loc, warp_sums, &tt);
            if (t == 0) sums[cc] = tt;
        }
        __threadfence();       // this CTA reads the new masses back through L2 on the second attempt
        __syncthreads();
    }
    const int pick = s_pick[0];
    int32_t* tok_out = p.out_tokens + (size_t)b * R + st.n;
    if (pick < 0) {                        // no mass at all (cannot happen for a softmax row)
        if (t == 0) { *tok_out = 0; set_status(p.dev_status, MASSV_ERR_INVALID_ARG); }
        return;
    }
    const bool take_last = s_pick[1] != 0;
    const double base = s_base[0], target = s_base[1];
    chunk_masses(p, b, st, use_q, pick, inv_T, r);
    double loc = 0.0;
#pragma unroll
    for (int e = 0; e < kPerThread; ++e) loc += (double)r[e];
    double tt;
    double run = base + block_exclusive_scan(loc, warp_sums, &tt);
    int first = 0x7fffffff, last = -1;
#pragma unroll
    for (int e = 0; e < kPerThread; ++e) {
        run += (double)r[e];
        if (r[e] > 0.f) {
            const int v = pick * kResidualChunk + t * kPerThread + e;
            last = v;
            if (first == 0x7fffffff && run > target) first = v;
        }
    }
    __shared__ int s_first, s_last;
    if (t == 0) { s_first = 0x7fffffff; s_last = -1; }
    __syncthreads();
    atomicMin(&s_first, first);
    atomicMax(&s_last, last);
    __syncthreads();
    if (t == 0) *tok_out = (!take_last && s_first != 0x7fffffff) ? s_first : s_last;
}

// ---------------------------------------------------------------- vocabulary shards
// The same arithmetic with the vocabulary cut into contiguous shards, one per rank: a shard sees Vs
// columns of the logits and of q.  Chunks are counted inside the shard; ranks in order are vocabulary order.

// Masses of the 16 entries this thread owns in chunk c of the sampled row of a shard.
__device__ __forceinline__ void shard_chunk_masses(const ShardParams& p, int b, const SeqState& st, int use_q, int c,
                                                   float inv_T, float (&r)[kPerThread]) {
    const int R = p.gamma + 1;
    const int v0 = c * kResidualChunk + threadIdx.x * kPerThread;
    const float* z = p.logits + (size_t)(b * R + st.n) * p.Vs;
    const float* q = use_q ? p.draft_probs + ((size_t)b * p.gamma + st.n) * p.Vs : nullptr;
#pragma unroll
    for (int e = 0; e < kPerThread; ++e) {
        const int v = v0 + e;
        float m = 0.f;
        if (v < p.Vs) {
            const float pv = expf((z[v] - st.row_max) * inv_T) * st.inv_sum;
            m = q ? fmaxf(pv - q[v], 0.f) : pv;
        }
        r[e] = m;
    }
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
        double local = 0.0;
#pragma unroll
        for (int e = 0; e < kPerThread; ++e) local += (double)r[e];
        double total;
        block_exclusive_scan(local, warp_sums, &total);
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
    __shared__ double warp_sums[kSampleThreads / 32];
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
        if (t == 0) {
            double tot = 0.0;
            for (int i = 0; i < n_all; ++i) tot += s_sums[i];
            const double target = (double)p.u_sample[(size_t)b * R + st.n] * tot;
            int pick = -1, last_pos = -1;
            double cum = 0.0, base = 0.0;
            for (int i = 0; i < n_all; ++i) {
                const double s = s_sums[i];
                if (s > 0.0) last_pos = i;
                if (pick < 0 && s > 0.0 && cum + s > target) { pick = i; base = cum; }
                cum += s;
            }
            s_pick[0] = tot > 0.0 ? (pick >= 0 ? pick : last_pos) : -1;
            s_pick[1] = (pick < 0);
            s_base[0] = base;
            s_base[1] = target;
        }
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
    double loc = 0.0;
#pragma unroll
    for (int e = 0; e < kPerThread; ++e) loc += (double)r[e];
    double tt;
    double run = base + block_exclusive_scan(loc, warp_sums, &tt);
    int first = 0x7fffffff, last = -1;
#pragma unroll
    for (int e = 0; e < kPerThread; ++e) {
        run += (double)r[e];
        if (r[e] > 0.f) {
            const int v = c * kResidualChunk + t * kPerThread + e;
            last = v;
            if (first == 0x7fffffff && run > target) first = v;
        }
    }
    if (t == 0) { s_first = 0x7fffffff; s_last = -1; }
    __syncthreads();
    atomicMin(&s_first, first);
    atomicMax(&s_last, last);
    __syncthreads();
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
        if (launch_pdl(residual_sample_kernel, dim3(p.n_chunks, p.B), dim3(kSampleThreads), 0, stream, p) != cudaSuccess) return cudaGetLastError();
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
