// Nucleus (top-p) sampling of softmax(z / T), one row per CTA (paper Sec. 3.2: the target's responses
// for self-distillation are drawn as sample_top-p(p(. | I, X)); it is also the drafter's sampling step
// when the drafter uses top-p, and probs_out is then the q a verify step needs).
//
// Per row: w_v = exp((z_v - max z) / T) in fp32 (ex2.approx), sums in fp64 or in fixed-point integers.  The nucleus - the shortest prefix of the
// tokens ordered by weight (ties: lower index first) whose mass reaches top_p * sum - is found without
// sorting: a search over the bit pattern of w (monotone for non-negative floats) finds the largest
// threshold tau with mass{w >= tau} >= target, which is the weight of the prefix's last token; everything
// above tau is in, and of the tokens equal to tau the first ceil((target - mass{w > tau}) / tau) by index.
// The threshold search is a radix selection in four levels (9 + 9 + 9 + 4 bits of the pattern): each level
// builds a histogram of mass over the next bits of the tokens that match the prefix found so far, and a
// suffix scan over the bins finds the one in which the running mass from the top crosses the target.
// Masses are fixed-point integers there, so the shared-memory atomics add up to the same value whatever
// their order.
// The draw is the inverse CDF in vocabulary order (first index whose running mass exceeds u * total): every
// warp owns a contiguous range walked 32 entries at a time, so the running sums have a fixed order.
#include "kernels.cuh"

namespace massv {

namespace {

constexpr int kTopPThreads = 1024;
constexpr int kTopPWarps = kTopPThreads / 32;

// Integer versions (exact, so any order gives the same value).
__device__ __forceinline__ unsigned long long block_sum_u64(unsigned long long x, unsigned long long* sm) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    __syncthreads();
    if (lane == 0) sm[warp] = x;
    __syncthreads();
    unsigned long long s = 0ull;
#pragma unroll
    for (int w = 0; w < kTopPWarps; ++w) s += sm[w];
    return s;
}
// Sum of the values of all threads with a higher index.
__device__ __forceinline__ unsigned long long block_suffix_exclusive_u64(unsigned long long x, unsigned long long* sm) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    unsigned long long incl = x;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const unsigned long long y = __shfl_down_sync(0xffffffffu, incl, o);
        if (lane + o < 32) incl += y;
    }
    __syncthreads();
    if (lane == 0) sm[warp] = incl;
    __syncthreads();
    unsigned long long above = 0ull;
#pragma unroll
    for (int w = 0; w < kTopPWarps; ++w) if (w > warp) above += sm[w];
    return above + incl - x;
}

constexpr int kTopPBins = 512;      // 9 bits of the pattern per level (9 + 9 + 9 + 4)
constexpr int kTopPCopies = 8;
constexpr int kTopPMaxBlocks = kTopPBins * kTopPCopies / kTopPWarps;     // 512-entry blocks per warp: 128, i.e. V <= 2^21

__global__ void __launch_bounds__(kTopPThreads) top_p_kernel(TopPParams p) {
    const int row = blockIdx.x, t = threadIdx.x;
    const float* z = p.logits + (size_t)row * p.V;
    // 32 KB used twice: the histograms' low and high words during the threshold search, then the masses
    // of the 512-entry blocks of every warp's range
    __shared__ __align__(16) unsigned long long pool[kTopPBins * kTopPCopies];
    uint32_t* hist_lo = reinterpret_cast<uint32_t*>(pool);
    uint32_t* hist_hi = hist_lo + kTopPBins * kTopPCopies;
    double* block_mass = reinterpret_cast<double*>(pool);          // [kTopPWarps][kTopPMaxBlocks]
    __shared__ unsigned long long sm_u64[kTopPWarps];
    __shared__ int s_bin;
    __shared__ unsigned long long s_above;
    __shared__ float sm_max[kTopPWarps];
    __shared__ int s_first, s_last;
    pdl_wait();
    pdl_trigger();

    // Every pass walks the row with sixteen independent loads in flight per thread (the row comes from L2,
    // a few hundred cycles away); entries past the end read as -inf, whose weight is zero.
    constexpr int kUnroll = 16;
    auto load4 = [&](int v_first, int stride, float (&zz)[kUnroll]) {
#pragma unroll
        for (int j = 0; j < kUnroll; ++j) { const int v = v_first + j * stride; zz[j] = v < p.V ? z[v] : -INFINITY; }
    };

    // ---- row maximum
    float m = -INFINITY;
    for (int v = t; v < p.V; v += kUnroll * kTopPThreads) {
        float zz[kUnroll];
        load4(v, kTopPThreads, zz);
#pragma unroll
        for (int j = 0; j < kUnroll; ++j) m = fmaxf(m, zz[j]);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
    if ((t & 31) == 0) sm_max[t >> 5] = m;
    __syncthreads();
    m = sm_max[0];
#pragma unroll
    for (int w = 1; w < kTopPWarps; ++w) m = fmaxf(m, sm_max[w]);
    if (!(m > -INFINITY) || !(m < INFINITY)) {          // no finite logit in the row: nothing to draw from
        if (t == 0) { p.tokens[row] = 0; set_status(p.dev_status, MASSV_ERR_INVALID_ARG); }
        return;
    }
    // w = 2^((z - max) * log2(e) / T): one multiply-add into the exponential unit.  Every pass uses this
    // same function, so thresholds, ties and sums are consistent with one another.
    const float k2 = p.inv_T * 1.4426950408889634f, m2 = -m * k2;
    auto weight_of = [&](float zv) -> float {
        float y;
        asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(fmaf(zv, k2, m2)));
        return fminf(y, 1.0f);              // the approximation must not step past the pattern of 1.0f
    };

    // ---- total mass, in fixed point: w * 2^fx_bits truncated; the row's sum stays below 2^63 for V <= 2^19
    const int fx_bits = p.V <= (1 << 19) ? 44 : 30;
    // floor(w * 2^fx_bits) for 0 <= w <= 1 from the pattern of w: mantissa shifted by the exponent
    auto fixed = [&](float w) -> unsigned long long {
        const uint32_t b = __float_as_uint(w);
        const int e = (int)(b >> 23);                      // biased exponent; 0 = zero (denormals are flushed)
        if (e == 0) return 0ull;
        const unsigned long long mant = (unsigned long long)((b & 0x7FFFFFu) | 0x800000u);
        const int sh = e - 127 - 23 + fx_bits;             // w = mant * 2^(e - 127 - 23)
        return sh >= 0 ? mant << sh : (sh > -24 ? mant >> (-sh) : 0ull);
    };
    // the same number as two 32-bit words, from two float -> integer conversions (fx_bits == 44):
    // hi = floor(w * 2^12), lo = floor((w - hi * 2^-12) * 2^44); both products and the difference are exact
    auto fixed_words = [&](float w, uint32_t& hi, uint32_t& lo) {
        if (fx_bits == 44) {
            hi = __float2uint_rz(w * 4096.f);
            lo = __float2uint_rz(fmaf(-(float)hi, 1.f / 4096.f, w) * 17592186044416.f);
        } else {
            const unsigned long long f = fixed(w);
            hi = (uint32_t)(f >> 32); lo = (uint32_t)f;
        }
    };
    unsigned long long local_hi = 0ull, local_lo = 0ull;
    for (int v = t; v < p.V; v += kUnroll * kTopPThreads) {
        float zz[kUnroll];
        load4(v, kTopPThreads, zz);
#pragma unroll
        for (int j = 0; j < kUnroll; ++j) {
            uint32_t hi, lo;
            fixed_words(weight_of(zz[j]), hi, lo);
            local_hi += hi; local_lo += lo;
        }
    }
    const unsigned long long S_fx = (block_sum_u64(local_hi, sm_u64) << 32) + block_sum_u64(local_lo, sm_u64);
    unsigned long long target_fx = (unsigned long long)ceil((double)p.top_p * (double)S_fx);
    if (target_fx > S_fx) target_fx = S_fx;
    if (target_fx == 0ull) target_fx = 1ull;

    // ---- threshold: largest bit pattern tau with mass{w >= tau} >= target, by radix selection
    uint32_t prefix = 0u;                 // bits of tau found so far
    unsigned long long mass_above = 0ull; // mass of the tokens whose pattern is above every pattern with this prefix
#pragma unroll
    for (int level = 0; level < 4; ++level) {
        const int shift = level == 0 ? 22 : (level == 1 ? 13 : (level == 2 ? 4 : 0));
        const int bits = level == 3 ? 4 : 9, nbins = 1 << bits;
        const uint32_t hi_mask = level == 0 ? 0u : ~((1u << (shift + bits)) - 1u);       // bits already fixed
        for (int i = t; i < kTopPBins * kTopPCopies; i += kTopPThreads) { hist_lo[i] = 0u; hist_hi[i] = 0u; }
        __syncthreads();
        // many tokens share their leading bits: eight copies of the histogram, chosen by lane, keep
        // the atomics on a hot bin from queueing behind one another
        // (64-bit sums as two 32-bit words with an explicit carry: 32-bit shared-memory atomics are native)
        const int my_copy = (t & (kTopPCopies - 1)) * kTopPBins;
        for (int v = t; v < p.V; v += kUnroll * kTopPThreads) {
            float zz[kUnroll];
            load4(v, kTopPThreads, zz);
#pragma unroll
            for (int j = 0; j < kUnroll; ++j) {
                const float w = weight_of(zz[j]);
                const uint32_t b = __float_as_uint(w);
                if ((b & hi_mask) == prefix) {
                    uint32_t hi, lo;
                    fixed_words(w, hi, lo);
                    const int bin = my_copy + (int)((b >> shift) & (uint32_t)(nbins - 1));
                    if (lo) hi += (atomicAdd(&hist_lo[bin], lo) > ~lo) ? 1u : 0u;      // the low word wrapped
                    if (hi) atomicAdd(&hist_hi[bin], hi);
                }
            }
        }
        __syncthreads();
        // suffix sums over the bins, highest first: thread t < 512 owns bin t (all copies)
        unsigned long long own = 0ull;
        if (t < nbins) {
#pragma unroll
            for (int c = 0; c < kTopPCopies; ++c)
                own += ((unsigned long long)hist_hi[c * kTopPBins + t] << 32) + (unsigned long long)hist_lo[c * kTopPBins + t];
        }
        const unsigned long long above_me = block_suffix_exclusive_u64(own, sm_u64);        // mass in bins above t
        // the bin b with mass_above + sum(bins > b) < target <= mass_above + sum(bins >= b) exists exactly once
        const unsigned long long run = mass_above + above_me;
        if (run < target_fx && run + own >= target_fx) { s_bin = t; s_above = run; }
        __syncthreads();
        prefix |= (uint32_t)s_bin << shift;
        mass_above = s_above;
        __syncthreads();
    }
    const uint32_t tau = prefix;
    // how many of the tokens equal to tau the prefix takes (at least one: mass{w > tau} < target)
    const unsigned long long tau_fx = fixed(__uint_as_float(tau));
    unsigned long long n_ties_u = tau_fx ? (target_fx - mass_above + tau_fx - 1ull) / tau_fx : ~0ull;
    if (n_ties_u < 1ull) n_ties_u = 1ull;
    const long long n_ties = n_ties_u > (unsigned long long)4e18 ? (long long)4e18 : (long long)n_ties_u;

    // ---- ordered passes: warp w owns a contiguous range, walked 32 consecutive entries at a time
    // (lane = entry, so loads and stores are coalesced); ranks among the entries equal to tau come
    // from ballots, running masses from warp-wide sums in round order.
    const int warp = t >> 5, lane = t & 31;
    const int per_warp = ((p.V + kTopPWarps - 1) / kTopPWarps + 31) / 32 * 32;
    const int w0 = min(p.V, warp * per_warp), w1 = min(p.V, w0 + per_warp);
    const unsigned lt_mask = (1u << lane) - 1u;
    __shared__ long long warp_ties[kTopPWarps];
    __shared__ double warp_mass[kTopPWarps];
    // ties per warp
    {
        long long n = 0;
        for (int v = w0 + lane; v - lane < w1; v += kUnroll * 32) {
            float zz[kUnroll];
            load4(v, 32, zz);
#pragma unroll
            for (int j = 0; j < kUnroll; ++j) {
                const bool tie = (v + j * 32 < w1) && __float_as_uint(weight_of(zz[j])) == tau;
                n += __popc(__ballot_sync(0xffffffffu, tie));
            }
        }
        if (lane == 0) warp_ties[warp] = n;
    }
    __syncthreads();
    long long tie_base = 0;
    for (int w = 0; w < warp; ++w) tie_base += warp_ties[w];
    // mass per warp (members only): per block of 16 rounds (512 entries) every lane adds up its own
    // entries, then one warp-wide sum; the block masses are kept for the draw
    __syncthreads();                             // the histograms are not read any more: the pool changes hands
    {
        long long rank0 = tie_base;              // ties before the current round
        double acc = 0.0;
        int blk = 0;
        for (int v = w0 + lane; v - lane < w1; v += kUnroll * 32, ++blk) {
            float zz[kUnroll];
            load4(v, 32, zz);
            double x = 0.0;
#pragma unroll
            for (int j = 0; j < kUnroll; ++j) {
                const float w = (v + j * 32 < w1) ? weight_of(zz[j]) : 0.f;
                const uint32_t b = __float_as_uint(w);
                const bool tie = (v + j * 32 < w1) && b == tau;
                const unsigned ties = __ballot_sync(0xffffffffu, tie);
                const bool in = (v + j * 32 < w1) && (b > tau || (tie && rank0 + __popc(ties & lt_mask) < n_ties));
                rank0 += __popc(ties);
                if (in) x += (double)w;
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
            if (lane == 0) block_mass[warp * kTopPMaxBlocks + blk] = x;
            acc += x;
        }
        if (lane == 0) warp_mass[warp] = acc;
    }
    __syncthreads();
    double Z = 0.0, base = 0.0;
    for (int w = 0; w < kTopPWarps; ++w) { if (w < warp) base += warp_mass[w]; Z += warp_mass[w]; }
    const double target = (double)p.u[row] * Z;
    // the warp whose range holds the target walks it again with running sums; the last warp with mass
    // keeps the fall-back (rounding can push the target past the end)
    if (t == 0) { s_first = 0x7fffffff; s_last = -1; }
    __syncthreads();
    const bool holds = warp_mass[warp] > 0.0 && base <= target && target < base + warp_mass[warp];
    bool last_with_mass = warp_mass[warp] > 0.0;
    for (int w = warp + 1; w < kTopPWarps; ++w) last_with_mass = last_with_mass && !(warp_mass[w] > 0.0);
    const float inv_Z = (float)(1.0 / Z);
    {
        long long rank0 = tie_base;
        double run = base;                       // mass before the current block / round
        int first = 0x7fffffff, last = -1;
        int blk = 0;
        for (int v = w0 + lane; v - lane < w1; v += kUnroll * 32, ++blk) {
            float zz[kUnroll];
            load4(v, 32, zz);
            // only the block that holds the target is walked round by round with running sums
            const double blk_mass = block_mass[warp * kTopPMaxBlocks + blk];
            const bool scan = holds && first == 0x7fffffff && blk_mass > 0.0 && run <= target && target < run + blk_mass;
            double run_in = run;
            int blk_last = -1;
#pragma unroll
            for (int j = 0; j < kUnroll; ++j) {
                const int vv = v + j * 32;
                const float w = vv < w1 ? weight_of(zz[j]) : 0.f;
                const uint32_t b = __float_as_uint(w);
                const bool tie = vv < w1 && b == tau;
                const unsigned ties = __ballot_sync(0xffffffffu, tie);
                const bool in = vv < w1 && w > 0.f && (b > tau || (tie && rank0 + __popc(ties & lt_mask) < n_ties));
                rank0 += __popc(ties);
                if (p.probs_out && vv < w1) p.probs_out[(size_t)row * p.V + vv] = in ? w * inv_Z : 0.f;
                if (in) { last = vv; blk_last = vv; }
                if (scan) {
                    // inclusive sum over the lanes of this round, in lane order
                    double incl = in ? (double)w : 0.0;
#pragma unroll
                    for (int o = 1; o < 32; o <<= 1) {
                        const double y = __shfl_up_sync(0xffffffffu, incl, o);
                        if (lane >= o) incl += y;
                    }
                    if (in && first == 0x7fffffff && run_in + incl > target) first = vv;
                    run_in += __shfl_sync(0xffffffffu, incl, 31);
                }
            }
            if (scan) {
                // (the round sums and the block's mass add the same numbers in another order: if the last bit
                // puts the target past the running sum, the block's last member is the answer)
                first = __reduce_min_sync(0xffffffffu, first);
                if (first == 0x7fffffff) first = __reduce_max_sync(0xffffffffu, blk_last);
            }
            run += blk_mass;
        }
        first = __reduce_min_sync(0xffffffffu, first);
        last = __reduce_max_sync(0xffffffffu, last);
        if (holds && first == 0x7fffffff && last >= 0) first = last;      // no block claimed the target (rounding): the warp's last member
        if (holds && first != 0x7fffffff) atomicMin(&s_first, first);
        if (last_with_mass && last >= 0) atomicMax(&s_last, last);
    }
    __syncthreads();
    if (t == 0) p.tokens[row] = s_first != 0x7fffffff ? s_first : s_last;      // rounding past the end: last nucleus token
}

}  // namespace

cudaError_t launch_top_p(const TopPParams& p, cudaStream_t stream) {
    cudaError_t e = launch_pdl(top_p_kernel, dim3(p.rows), dim3(kTopPThreads), 0, stream, p);
    if (e != cudaSuccess) return e;
    count_launches(1);
    return cudaGetLastError();
}

}  // namespace massv
