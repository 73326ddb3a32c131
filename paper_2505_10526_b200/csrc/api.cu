// C ABI of the verify-step library: host-side validation, workspace layout and
// kernel launches.  No device memory is allocated and no stream is synchronised.
#include <math.h>

#include <atomic>

#include <nvtx3/nvToolsExt.h>

#include "kernels.cuh"

using namespace massv;

static std::atomic<uint64_t> g_launches{0};
namespace massv {
void count_launches(int n) { g_launches.fetch_add((uint64_t)n, std::memory_order_relaxed); }
TimingHooks& timing_hooks() {
    static thread_local TimingHooks hooks;
    return hooks;
}
}

namespace {

// A named range around the host side of a call, for timelines (NVTX is header-only: without a tool attached the
// push and the pop are two null-pointer checks).
struct NvtxRange {
    explicit NvtxRange(const char* name) { nvtxRangePushA(name); }
    ~NvtxRange() { nvtxRangePop(); }
};

constexpr size_t kAlign = 256;

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int auto_kv_chunk(const massv_attn_desc& d) {
    // Work is counted in token-heads over the longest context the page table can describe.
    // Large problems: about five waves of CTAs (two per SM), but chunks of at least 768 tokens
    // so that the partial results written per chunk stay a few percent of the K/V read.
    // Small problems (too few CTAs that way): split down to 64 tokens to fill the machine.
    long per_seq_tokens = (long)d.max_pages_per_seq * kPageSize;
    if (d.window > 0 && d.window + 64 < per_seq_tokens) per_seq_tokens = d.window + 64;   // only the window is read
    const double th = (double)d.batch * per_seq_tokens * d.n_kv_heads;
    long chunk = ((long)ceil(th / 1480.0) + 63) / 64 * 64;
    if (chunk < 768) chunk = 768;
    if (th / (double)chunk < 128.0) chunk = ((long)ceil(th / 128.0) + 63) / 64 * 64;
    if (chunk < 64) chunk = 64;
    if (chunk > 4096) chunk = 4096;
    return (int)chunk;
}

int check_attn_desc(const massv_attn_desc* d) {
    if (!d) return MASSV_ERR_INVALID_ARG;
    if (d->batch < 1 || d->n_q_heads < 1 || d->n_kv_heads < 1 || d->max_pages_per_seq < 1 || d->num_pages < 1 ||
        d->gamma < 0 || d->scale < 0.f || d->kv_chunk < 0 || d->window < 0)
        return MASSV_ERR_INVALID_ARG;
    if (d->gamma > kMaxRows - 1) return MASSV_ERR_UNSUPPORTED;
    if (d->page_size != kPageSize) return MASSV_ERR_UNSUPPORTED;
    if (d->head_dim != 64 && d->head_dim != 128 && d->head_dim != 256) return MASSV_ERR_UNSUPPORTED;
    if (d->n_q_heads % d->n_kv_heads != 0) return MASSV_ERR_UNSUPPORTED;
    if ((d->n_q_heads / d->n_kv_heads) * (d->gamma + 1) > 64) return MASSV_ERR_UNSUPPORTED;
    if (d->kv_chunk % 64 != 0 || d->kv_chunk > 4096) return MASSV_ERR_UNSUPPORTED;
    if (d->flags > MASSV_ATTN_KERNEL_TCGEN05) return MASSV_ERR_UNSUPPORTED;
    {
        // the chunk merge kernel indexes at most 1024 chunks per sequence: refuse here, before anything is launched
        const long chunk = d->kv_chunk > 0 ? d->kv_chunk : auto_kv_chunk(*d);
        if (((long)d->max_pages_per_seq * kPageSize + chunk - 1) / chunk > 1024) return MASSV_ERR_UNSUPPORTED;
    }
    return MASSV_OK;
}

struct AttnLayout {
    int kv_chunk, max_chunks, rows_pad;
    size_t off_o, off_ml, off_flat_o, off_flat_ml, off_flat_meta, total;
};

AttnLayout attn_layout(const massv_attn_desc& d) {
    AttnLayout l;
    l.kv_chunk = d.kv_chunk > 0 ? d.kv_chunk : auto_kv_chunk(d);
    const long max_tokens = (long)d.max_pages_per_seq * kPageSize;
    l.max_chunks = (int)((max_tokens + l.kv_chunk - 1) / l.kv_chunk);
    l.rows_pad = attn_rows_pad((d.n_q_heads / d.n_kv_heads) * (d.gamma + 1));
    const size_t items = (size_t)d.batch * d.n_kv_heads * l.max_chunks;
    l.off_o = 0;
    l.off_ml = align_up(items * l.rows_pad * d.head_dim * sizeof(float), kAlign);
    l.off_flat_o = l.off_ml + align_up(items * l.rows_pad * 2 * sizeof(float), kAlign);
    const size_t slots = (size_t)kFlatMaxCtas * 2;
    l.off_flat_ml = l.off_flat_o + align_up(slots * l.rows_pad * d.head_dim * sizeof(float), kAlign);
    l.off_flat_meta = l.off_flat_ml + align_up(slots * l.rows_pad * 2 * sizeof(float), kAlign);
    l.total = l.off_flat_meta + align_up((size_t)(kFlatMaxBatchMeta + 3) * sizeof(int32_t), kAlign);
    return l;
}

int check_accept_desc(const massv_accept_desc* d) {
    if (!d) return MASSV_ERR_INVALID_ARG;
    if (d->batch < 1 || d->gamma < 0 || d->hidden < 1 || d->vocab < 1 || !(d->temperature >= 0.f))
        return MASSV_ERR_INVALID_ARG;
    if (d->gamma > kMaxRows - 1) return MASSV_ERR_UNSUPPORTED;
    if ((long)d->batch * (d->gamma + 1) > 512) return MASSV_ERR_UNSUPPORTED;
    if (d->hidden % 64 != 0 || d->vocab % 8 != 0) return MASSV_ERR_UNSUPPORTED;
#ifdef MASSV_TEST_HOOKS
    if ((d->flags & ~MASSV_TEST_SKIP_STAGE) != 0) return MASSV_ERR_UNSUPPORTED;
#else
    if (d->flags != 0) return MASSV_ERR_UNSUPPORTED;
#endif
    return MASSV_OK;
}

struct AcceptLayout {
    int n_part, n_chunks;
    size_t off_max, off_sum, off_idx, off_state, off_chunks, off_segs, off_counters, off_rowstat, off_logits, total;
};

AcceptLayout accept_layout(const massv_accept_desc& d) {
    AcceptLayout l;
    const size_t M = (size_t)d.batch * (d.gamma + 1);
    l.n_part = lm_head_num_partials((int)M, d.vocab);
    l.n_chunks = (d.vocab + kResidualChunk - 1) / kResidualChunk;
    size_t off = 0;
    l.off_max = off; off += align_up((size_t)l.n_part * M * sizeof(float), kAlign);
    l.off_sum = off; off += align_up((size_t)l.n_part * M * sizeof(float), kAlign);
    l.off_idx = off; off += align_up((size_t)l.n_part * M * sizeof(int32_t), kAlign);
    l.off_state = off; off += align_up((size_t)d.batch * sizeof(SeqState), kAlign);
    l.off_chunks = off; off += align_up((size_t)d.batch * l.n_chunks * sizeof(double), kAlign);
    l.off_segs = off;
    if (d.temperature > 0.f) off += align_up((size_t)d.batch * l.n_chunks * kResidualSegments * sizeof(double), kAlign);
    l.off_counters = off; off += align_up((size_t)d.batch * sizeof(unsigned int), kAlign);
    l.off_rowstat = off; off += align_up(M * 2 * sizeof(float), kAlign);
    l.off_logits = off;
    if (d.temperature > 0.f) off += align_up(M * (size_t)d.vocab * sizeof(float), kAlign);
    l.total = off;
    return l;
}

}  // namespace

extern "C" {

size_t massv_verify_attn_workspace_size(const massv_attn_desc* desc) {
    if (check_attn_desc(desc) != MASSV_OK) return 0;
    return attn_layout(*desc).total;
}

int massv_verify_attn(const massv_attn_desc* desc, const void* q, const void* k_new, const void* v_new,
                      void* k_pages, void* v_pages, const int32_t* page_table, const int32_t* seq_lens,
                      void* out, float* out_f32, float* lse, void* workspace, size_t workspace_bytes,
                      int32_t* dev_status, massv_stream_t stream) {
    NvtxRange range("massv_verify_attn");
    const int rc = check_attn_desc(desc);
    if (rc != MASSV_OK) return rc;
    if (!q || !k_new || !v_new || !k_pages || !v_pages || !page_table || !seq_lens || !out) return MASSV_ERR_INVALID_ARG;
    if (!aligned16(q) || !aligned16(k_new) || !aligned16(v_new) || !aligned16(k_pages) || !aligned16(v_pages) ||
        !aligned16(out) || (out_f32 && !aligned16(out_f32)))
        return MASSV_ERR_INVALID_ARG;
    const AttnLayout l = attn_layout(*desc);
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) % kAlign) != 0 || workspace_bytes < l.total)
        return MASSV_ERR_WORKSPACE;

    AttnParams p;
    p.B = desc->batch; p.R = desc->gamma + 1; p.Hq = desc->n_q_heads; p.Hkv = desc->n_kv_heads;
    p.d = desc->head_dim; p.max_pages = desc->max_pages_per_seq; p.num_pages = desc->num_pages;
    p.scale = desc->scale > 0.f ? desc->scale : 1.f / sqrtf((float)desc->head_dim);
    p.kv_chunk = l.kv_chunk; p.max_chunks = l.max_chunks; p.window = desc->window;
    p.q = static_cast<const __nv_bfloat16*>(q);
    p.k_new = static_cast<const __nv_bfloat16*>(k_new);
    p.v_new = static_cast<const __nv_bfloat16*>(v_new);
    p.k_pages = static_cast<__nv_bfloat16*>(k_pages);
    p.v_pages = static_cast<__nv_bfloat16*>(v_pages);
    p.page_table = page_table; p.seq_lens = seq_lens;
    p.out = static_cast<__nv_bfloat16*>(out); p.out_f32 = out_f32; p.lse = lse;
    char* ws = static_cast<char*>(workspace);
    p.part_o = reinterpret_cast<float*>(ws + l.off_o);
    p.part_ml = reinterpret_cast<float*>(ws + l.off_ml);
    p.dev_status = dev_status;
    p.path = (int)desc->flags;
    p.chunk_forced = desc->kv_chunk > 0;
    p.flat_part_o = reinterpret_cast<float*>(ws + l.off_flat_o);
    p.flat_part_ml = reinterpret_cast<float*>(ws + l.off_flat_ml);
    p.flat_meta = reinterpret_cast<int32_t*>(ws + l.off_flat_meta);
    return launch_verify_attn(p, reinterpret_cast<cudaStream_t>(stream)) == cudaSuccess ? MASSV_OK : MASSV_ERR_CUDA;
}

size_t massv_accept_workspace_size(const massv_accept_desc* desc) {
    if (check_accept_desc(desc) != MASSV_OK) return 0;
    return accept_layout(*desc).total;
}

int massv_accept(const massv_accept_desc* desc, const void* hidden, const void* lm_head, const int32_t* draft_tokens,
                 const float* draft_probs, const float* u_accept, const float* u_sample, int32_t* out_tokens,
                 int32_t* accept_len, float* logits_out, float* probs_out, void* workspace, size_t workspace_bytes,
                 int32_t* dev_status, massv_stream_t stream) {
    NvtxRange range("massv_accept");
    const int rc = check_accept_desc(desc);
    if (rc != MASSV_OK) return rc;
    const bool sampling = desc->temperature > 0.f;
    if (!hidden || !lm_head || !out_tokens || !accept_len) return MASSV_ERR_INVALID_ARG;
    if (desc->gamma > 0 && !draft_tokens) return MASSV_ERR_INVALID_ARG;
    if (sampling && (!u_sample || (desc->gamma > 0 && (!draft_probs || !u_accept)))) return MASSV_ERR_INVALID_ARG;
    if (!sampling && probs_out) return MASSV_ERR_INVALID_ARG;
    if (!aligned16(hidden) || !aligned16(lm_head) || (draft_probs && !aligned16(draft_probs)) ||
        (logits_out && !aligned16(logits_out)) || (probs_out && !aligned16(probs_out)))
        return MASSV_ERR_INVALID_ARG;
    const AcceptLayout l = accept_layout(*desc);
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) % kAlign) != 0 || workspace_bytes < l.total)
        return MASSV_ERR_WORKSPACE;
    char* ws = static_cast<char*>(workspace);
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);

    LmHeadParams g;
    g.M = desc->batch * (desc->gamma + 1); g.K = desc->hidden; g.V = desc->vocab;
    g.greedy = sampling ? 0 : 1;
    g.inv_T_log2e = sampling ? 1.4426950408889634f / desc->temperature : 0.f;
    g.hidden = static_cast<const __nv_bfloat16*>(hidden);
    g.lm_head = static_cast<const __nv_bfloat16*>(lm_head);
    // fp32 logits are materialised only when the sampling pass or the caller needs them
    g.logits = logits_out ? logits_out : (sampling ? reinterpret_cast<float*>(ws + l.off_logits) : nullptr);
    g.n_part = l.n_part;
    g.part_max = reinterpret_cast<float*>(ws + l.off_max);
    g.part_sum = reinterpret_cast<float*>(ws + l.off_sum);
    g.part_idx = reinterpret_cast<int32_t*>(ws + l.off_idx);
    g.dev_status = dev_status;
#ifdef MASSV_TEST_HOOKS
    g.test_skip_stage = (desc->flags & MASSV_TEST_SKIP_STAGE) ? 1 : 0;
#endif
    int n_part_used = 0;
    if (launch_lm_head(g, s, &n_part_used) != cudaSuccess) return MASSV_ERR_CUDA;

    AcceptParams a;
    a.B = desc->batch; a.gamma = desc->gamma; a.V = desc->vocab; a.T = desc->temperature;
    a.n_part = n_part_used; a.part_max = g.part_max; a.part_sum = g.part_sum; a.part_idx = g.part_idx;
    a.logits = g.logits;
    a.draft_tokens = draft_tokens; a.draft_probs = draft_probs; a.u_accept = u_accept; a.u_sample = u_sample;
    a.out_tokens = out_tokens; a.accept_len = accept_len; a.probs_out = probs_out;
    a.seq_state = reinterpret_cast<SeqState*>(ws + l.off_state);
    a.chunk_sums = reinterpret_cast<double*>(ws + l.off_chunks);
    a.seg_sums = desc->temperature > 0.f ? reinterpret_cast<double*>(ws + l.off_segs) : nullptr;
    a.counters = reinterpret_cast<unsigned int*>(ws + l.off_counters);
    a.row_stats = reinterpret_cast<float*>(ws + l.off_rowstat);
    a.n_chunks = l.n_chunks;
    a.dev_status = dev_status;
    return launch_accept(a, s) == cudaSuccess ? MASSV_OK : MASSV_ERR_CUDA;
}

}  // extern "C"

// ---------------------------------------------------------------- vocabulary shards
namespace {
// Exchange buffer A of one rank, in 4-byte words: the three partial arrays, then z and q at the drafted tokens.
struct ShardLayoutA {
    int slots;
    size_t M, off_max, off_sum, off_idx, off_z, off_q, words;
};
ShardLayoutA shard_layout_a(const massv_accept_desc& d) {
    ShardLayoutA l;
    l.M = (size_t)d.batch * (d.gamma + 1);
    l.slots = lm_head_num_partials((int)l.M, d.vocab);
    const size_t part = (size_t)l.slots * l.M, at = (size_t)d.batch * d.gamma;
    l.off_max = 0; l.off_sum = part; l.off_idx = 2 * part; l.off_z = 3 * part; l.off_q = 3 * part + at;
    l.words = (3 * part + 2 * at + 3) & ~(size_t)3;          // every rank's copy starts 16-byte aligned
    return l;
}
int shard_chunks(const massv_accept_desc& d) { return (d.vocab + kResidualChunk - 1) / kResidualChunk; }

int check_shard(const massv_accept_desc* desc, int32_t world, int32_t rank) {
    const int rc = check_accept_desc(desc);
    if (rc != MASSV_OK) return rc;
    if (world < 1 || rank < 0 || rank >= world) return MASSV_ERR_INVALID_ARG;
    if ((long)world * desc->vocab > 0x7fffffffL) return MASSV_ERR_UNSUPPORTED;
    if ((long)world * shard_chunks(*desc) > 512) return MASSV_ERR_UNSUPPORTED;
    return MASSV_OK;
}

ShardParams shard_params(const massv_accept_desc* desc, int32_t world, int32_t rank, int32_t* dev_status) {
    ShardParams p{};
    p.B = desc->batch; p.gamma = desc->gamma; p.Vs = desc->vocab; p.vocab_offset = rank * desc->vocab;
    p.T = desc->temperature; p.world = world; p.rank = rank;
    p.n_chunks = shard_chunks(*desc);
    p.mass_rank_stride = (size_t)2 * desc->batch * p.n_chunks;
    p.dev_status = dev_status;
    return p;
}
}  // namespace

extern "C" {

size_t massv_shard_stats_words(const massv_accept_desc* desc) {
    if (check_accept_desc(desc) != MASSV_OK) return 0;
    return shard_layout_a(*desc).words;
}

size_t massv_shard_mass_count(const massv_accept_desc* desc) {
    if (check_accept_desc(desc) != MASSV_OK) return 0;
    return (size_t)2 * desc->batch * shard_chunks(*desc);
}

size_t massv_shard_state_bytes(const massv_accept_desc* desc) {
    if (check_accept_desc(desc) != MASSV_OK) return 0;
    return (size_t)desc->batch * sizeof(SeqState);
}

int massv_shard_lm_head(const massv_accept_desc* desc, int32_t world, int32_t rank, const void* hidden,
                        const void* lm_head_shard, float* logits_shard, float* stats, int32_t* n_partials,
                        int32_t* dev_status, massv_stream_t stream) {
    const int rc = check_shard(desc, world, rank);
    if (rc != MASSV_OK) return rc;
    const bool sampling = desc->temperature > 0.f;
    if (!hidden || !lm_head_shard || !stats || !n_partials) return MASSV_ERR_INVALID_ARG;
    if (sampling && !logits_shard) return MASSV_ERR_INVALID_ARG;
    if (!aligned16(hidden) || !aligned16(lm_head_shard) || !aligned16(stats) || (logits_shard && !aligned16(logits_shard)))
        return MASSV_ERR_INVALID_ARG;
    const ShardLayoutA l = shard_layout_a(*desc);
    LmHeadParams g;
    g.M = (int)l.M; g.K = desc->hidden; g.V = desc->vocab;
    g.greedy = sampling ? 0 : 1;
    g.inv_T_log2e = sampling ? 1.4426950408889634f / desc->temperature : 0.f;
    g.hidden = static_cast<const __nv_bfloat16*>(hidden);
    g.lm_head = static_cast<const __nv_bfloat16*>(lm_head_shard);
    g.logits = logits_shard;
    g.n_part = l.slots;
    g.part_max = stats + l.off_max; g.part_sum = stats + l.off_sum;
    g.part_idx = reinterpret_cast<int32_t*>(stats + l.off_idx);
    g.dev_status = dev_status;
    g.idx_offset = rank * desc->vocab;
    int used = 0;
    if (launch_lm_head(g, reinterpret_cast<cudaStream_t>(stream), &used) != cudaSuccess) return MASSV_ERR_CUDA;
    *n_partials = used;
    return MASSV_OK;
}

int massv_shard_gather_draft(const massv_accept_desc* desc, int32_t world, int32_t rank, const float* logits_shard,
                             const float* draft_probs_shard, const int32_t* draft_tokens, float* stats,
                             int32_t* dev_status, massv_stream_t stream) {
    const int rc = check_shard(desc, world, rank);
    if (rc != MASSV_OK) return rc;
    if (desc->gamma == 0 || !(desc->temperature > 0.f)) return MASSV_OK;
    if (!logits_shard || !draft_probs_shard || !draft_tokens || !stats) return MASSV_ERR_INVALID_ARG;
    const ShardLayoutA l = shard_layout_a(*desc);
    ShardParams p = shard_params(desc, world, rank, dev_status);
    p.logits = logits_shard; p.draft_probs = draft_probs_shard; p.draft_tokens = draft_tokens;
    p.z_at_draft = stats + l.off_z; p.q_at_draft = stats + l.off_q;
    return launch_shard_gather_draft(p, reinterpret_cast<cudaStream_t>(stream)) == cudaSuccess ? MASSV_OK : MASSV_ERR_CUDA;
}

int massv_shard_scan(const massv_accept_desc* desc, int32_t world, int32_t n_partials, const float* stats_all,
                     const int32_t* draft_tokens, const float* u_accept, int32_t* out_tokens, int32_t* accept_len,
                     void* state, int32_t* dev_status, massv_stream_t stream) {
    const int rc = check_shard(desc, world, 0);
    if (rc != MASSV_OK) return rc;
    const bool sampling = desc->temperature > 0.f;
    const ShardLayoutA l = shard_layout_a(*desc);
    if (n_partials < 1 || n_partials > l.slots || !stats_all || !out_tokens || !accept_len || !state)
        return MASSV_ERR_INVALID_ARG;
    if (desc->gamma > 0 && (!draft_tokens || (sampling && !u_accept))) return MASSV_ERR_INVALID_ARG;
    AcceptParams a{};
    a.B = desc->batch; a.gamma = desc->gamma; a.V = world * desc->vocab; a.T = desc->temperature;
    a.n_part = world * n_partials; a.part_per_rank = n_partials; a.ranks = world; a.rank_stride = l.words;
    a.part_max = const_cast<float*>(stats_all + l.off_max); a.part_sum = const_cast<float*>(stats_all + l.off_sum);
    a.part_idx = reinterpret_cast<int32_t*>(const_cast<float*>(stats_all + l.off_idx));
    a.draft_tokens = draft_tokens; a.u_accept = u_accept;
    if (sampling) { a.z_at_draft = stats_all + l.off_z; a.q_at_draft = stats_all + l.off_q; }
    a.out_tokens = out_tokens; a.accept_len = accept_len;
    a.seq_state = static_cast<SeqState*>(state);
    a.dev_status = dev_status;
    return launch_accept_scan_only(a, reinterpret_cast<cudaStream_t>(stream)) == cudaSuccess ? MASSV_OK : MASSV_ERR_CUDA;
}

int massv_shard_masses(const massv_accept_desc* desc, int32_t world, int32_t rank, const float* logits_shard,
                       const float* draft_probs_shard, const void* state, double* masses, int32_t* dev_status,
                       massv_stream_t stream) {
    const int rc = check_shard(desc, world, rank);
    if (rc != MASSV_OK) return rc;
    if (!(desc->temperature > 0.f)) return MASSV_ERR_INVALID_ARG;
    if (!logits_shard || !state || !masses || (desc->gamma > 0 && !draft_probs_shard)) return MASSV_ERR_INVALID_ARG;
    ShardParams p = shard_params(desc, world, rank, dev_status);
    p.logits = logits_shard; p.draft_probs = draft_probs_shard; p.seq_state = static_cast<const SeqState*>(state);
    p.sums_res = masses; p.sums_p = masses + (size_t)desc->batch * p.n_chunks;
    return launch_shard_masses(p, reinterpret_cast<cudaStream_t>(stream)) == cudaSuccess ? MASSV_OK : MASSV_ERR_CUDA;
}

int massv_shard_pick(const massv_accept_desc* desc, int32_t world, int32_t rank, const double* masses_all,
                     const float* u_sample, const void* state, const float* logits_shard,
                     const float* draft_probs_shard, int32_t* token_out, int32_t* dev_status, massv_stream_t stream) {
    const int rc = check_shard(desc, world, rank);
    if (rc != MASSV_OK) return rc;
    if (!(desc->temperature > 0.f)) return MASSV_ERR_INVALID_ARG;
    if (!masses_all || !u_sample || !state || !logits_shard || !token_out || (desc->gamma > 0 && !draft_probs_shard))
        return MASSV_ERR_INVALID_ARG;
    ShardParams p = shard_params(desc, world, rank, dev_status);
    p.logits = logits_shard; p.draft_probs = draft_probs_shard; p.seq_state = static_cast<const SeqState*>(state);
    p.all_res = masses_all; p.all_p = masses_all + (size_t)desc->batch * p.n_chunks;
    p.u_sample = u_sample; p.token_out = token_out;
    return launch_shard_pick(p, reinterpret_cast<cudaStream_t>(stream)) == cudaSuccess ? MASSV_OK : MASSV_ERR_CUDA;
}

int massv_shard_set_token(const massv_accept_desc* desc, int32_t world, const void* state, const int32_t* tokens_all,
                          int32_t* out_tokens, int32_t* dev_status, massv_stream_t stream) {
    const int rc = check_shard(desc, world, 0);
    if (rc != MASSV_OK) return rc;
    if (!state || !tokens_all || !out_tokens) return MASSV_ERR_INVALID_ARG;
    ShardParams p = shard_params(desc, world, 0, dev_status);
    p.seq_state = static_cast<const SeqState*>(state); p.tokens_in = tokens_all; p.out_tokens = out_tokens;
    return launch_shard_set_token(p, reinterpret_cast<cudaStream_t>(stream)) == cudaSuccess ? MASSV_OK : MASSV_ERR_CUDA;
}

int massv_shard_publish(const void* src, size_t bytes, void* const* gathered, int32_t world, int32_t rank,
                        massv_stream_t stream) {
    if (world < 1 || world > kMaxPeers || rank < 0 || rank >= world) return world > kMaxPeers ? MASSV_ERR_UNSUPPORTED : MASSV_ERR_INVALID_ARG;
    if (!src || !gathered || bytes % 4 != 0 || reinterpret_cast<uintptr_t>(src) % 4 != 0) return MASSV_ERR_INVALID_ARG;
    PublishParams p{};
    p.src = src; p.bytes = bytes; p.world = world; p.rank = rank;
    for (int w = 0; w < world; ++w) {
        if (!gathered[w] || reinterpret_cast<uintptr_t>(gathered[w]) % 4 != 0) return MASSV_ERR_INVALID_ARG;
        p.dst[w] = gathered[w];
    }
    return launch_shard_publish(p, reinterpret_cast<cudaStream_t>(stream)) == cudaSuccess ? MASSV_OK : MASSV_ERR_CUDA;
}

size_t massv_tvd_workspace_size(const massv_accept_desc* desc) {
    if (check_accept_desc(desc) != MASSV_OK || desc->gamma < 1 || !(desc->temperature > 0.f)) return 0;
    const size_t rows = (size_t)desc->batch * desc->gamma;
    return align_up(rows * kTvdSlices * sizeof(float), kAlign) + 3 * align_up(rows * kTvdSlices * sizeof(double), kAlign);
}

static int tvd_call(const massv_accept_desc* desc, const float* logits, const float* draft_probs, const float* row_stats, float* tvd_out,
                    float* accept_prob_out, void* workspace, size_t workspace_bytes, massv_stream_t stream) {
    const int rc = check_accept_desc(desc);
    if (rc != MASSV_OK) return rc;
    if (desc->gamma < 1 || !(desc->temperature > 0.f)) return MASSV_ERR_INVALID_ARG;
    if (!logits || !draft_probs || !tvd_out) return MASSV_ERR_INVALID_ARG;
    if (!aligned16(logits) || !aligned16(draft_probs)) return MASSV_ERR_INVALID_ARG;
    const size_t need = massv_tvd_workspace_size(desc);
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) % kAlign) != 0 || workspace_bytes < need) return MASSV_ERR_WORKSPACE;
    const size_t rows = (size_t)desc->batch * desc->gamma;
    char* ws = static_cast<char*>(workspace);
    TvdParams t;
    t.B = desc->batch; t.gamma = desc->gamma; t.V = desc->vocab; t.inv_T = 1.f / desc->temperature;
    t.slice_len = ((desc->vocab + kTvdSlices - 1) / kTvdSlices + 3) / 4 * 4;      // 16-byte aligned slices (V % 8 == 0)
    t.logits = logits; t.draft_probs = draft_probs; t.tvd_out = tvd_out; t.accept_prob_out = accept_prob_out;
    t.slice_max = reinterpret_cast<float*>(ws);
    const size_t off = align_up(rows * kTvdSlices * sizeof(float), kAlign), step = align_up(rows * kTvdSlices * sizeof(double), kAlign);
    t.slice_sum = reinterpret_cast<double*>(ws + off);
    t.slice_abs = reinterpret_cast<double*>(ws + off + step);
    t.slice_min = reinterpret_cast<double*>(ws + off + 2 * step);
    t.row_stats = row_stats;
    return launch_tvd(t, reinterpret_cast<cudaStream_t>(stream)) == cudaSuccess ? MASSV_OK : MASSV_ERR_CUDA;
}

int massv_tvd(const massv_accept_desc* desc, const float* logits, const float* draft_probs, float* tvd_out,
              float* accept_prob_out, void* workspace, size_t workspace_bytes, int32_t* dev_status, massv_stream_t stream) {
    (void)dev_status;
    return tvd_call(desc, logits, draft_probs, nullptr, tvd_out, accept_prob_out, workspace, workspace_bytes, stream);
}

int massv_tvd_after_accept(const massv_accept_desc* desc, const float* logits, const float* draft_probs,
                           const void* accept_workspace, size_t accept_workspace_bytes, float* tvd_out, float* accept_prob_out,
                           void* workspace, size_t workspace_bytes, int32_t* dev_status, massv_stream_t stream) {
    (void)dev_status;
    const int rc = check_accept_desc(desc);
    if (rc != MASSV_OK) return rc;
    const AcceptLayout l = accept_layout(*desc);
    if (!accept_workspace || (reinterpret_cast<uintptr_t>(accept_workspace) % kAlign) != 0 || accept_workspace_bytes < l.total)
        return MASSV_ERR_WORKSPACE;
    const float* row_stats = reinterpret_cast<const float*>(static_cast<const char*>(accept_workspace) + l.off_rowstat);
    return tvd_call(desc, logits, draft_probs, row_stats, tvd_out, accept_prob_out, workspace, workspace_bytes, stream);
}

int massv_tvd_histogram(int64_t n, const float* tvd, int32_t bins, int64_t* counts, massv_stream_t stream) {
    if (n < 0 || bins < 1 || !counts || (n > 0 && !tvd)) return MASSV_ERR_INVALID_ARG;
    if (bins > 4096 || n > ((int64_t)1 << 40)) return MASSV_ERR_UNSUPPORTED;
    if (reinterpret_cast<uintptr_t>(counts) % 8 != 0) return MASSV_ERR_INVALID_ARG;
    return launch_tvd_histogram((long long)n, tvd, bins, reinterpret_cast<unsigned long long*>(counts),
                                reinterpret_cast<cudaStream_t>(stream)) == cudaSuccess ? MASSV_OK : MASSV_ERR_CUDA;
}

int massv_sample_top_p(int32_t rows, int32_t vocab, float temperature, float top_p, const float* logits, const float* u,
                       int32_t* tokens, float* probs_out, int32_t* dev_status, massv_stream_t stream) {
    if (rows < 1 || vocab < 1 || !(temperature > 0.f) || !(top_p > 0.f) || !(top_p <= 1.f)) return MASSV_ERR_INVALID_ARG;
    if (!logits || !u || !tokens) return MASSV_ERR_INVALID_ARG;
    if (vocab > (1 << 21)) return MASSV_ERR_UNSUPPORTED;
    TopPParams t;
    t.rows = rows; t.V = vocab; t.inv_T = 1.f / temperature; t.top_p = top_p;
    t.logits = logits; t.u = u; t.tokens = tokens; t.probs_out = probs_out; t.dev_status = dev_status;
    return launch_top_p(t, reinterpret_cast<cudaStream_t>(stream)) == cudaSuccess ? MASSV_OK : MASSV_ERR_CUDA;
}

int massv_kv_commit(int32_t batch, int32_t gamma, const int32_t* accept_len, int32_t* seq_lens, int32_t* dev_status,
                    massv_stream_t stream) {
    NvtxRange range("massv_kv_commit");
    if (batch < 1 || gamma < 0 || !seq_lens) return MASSV_ERR_INVALID_ARG;
    if (gamma > kMaxRows - 1) return MASSV_ERR_UNSUPPORTED;
    return launch_kv_commit(batch, gamma, accept_len, seq_lens, dev_status, reinterpret_cast<cudaStream_t>(stream)) ==
                   cudaSuccess
               ? MASSV_OK
               : MASSV_ERR_CUDA;
}

const char* massv_strerror(int status) {
    switch (status) {
        case MASSV_OK: return "ok";
        case MASSV_ERR_INVALID_ARG: return "invalid argument";
        case MASSV_ERR_UNSUPPORTED: return "unsupported shape";
        case MASSV_ERR_CAPACITY: return "page table capacity exceeded or unmapped page";
        case MASSV_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
        case MASSV_ERR_CUDA: return "CUDA call failed";
        case MASSV_ERR_TIMEOUT: return "device-side wait timed out";
        case MASSV_ERR_BOUNDS: return "device-side index out of bounds (debug build)";
        default: return "unknown status";
    }
}

int massv_version(void) { return 101; }

int massv_set_timing_events(massv_event_t lm_head_start, massv_event_t lm_head_stop, massv_event_t attn_start,
                            massv_event_t attn_stop) {
    if ((lm_head_start == nullptr) != (lm_head_stop == nullptr) || (attn_start == nullptr) != (attn_stop == nullptr))
        return MASSV_ERR_INVALID_ARG;
    TimingHooks& h = timing_hooks();
    h.lm_head_start = reinterpret_cast<cudaEvent_t>(lm_head_start);
    h.lm_head_stop = reinterpret_cast<cudaEvent_t>(lm_head_stop);
    h.attn_start = reinterpret_cast<cudaEvent_t>(attn_start);
    h.attn_stop = reinterpret_cast<cudaEvent_t>(attn_stop);
    return MASSV_OK;
}

int massv_set_kernel_timing(int32_t kernel, massv_event_t start, massv_event_t stop) {
    if ((start == nullptr) != (stop == nullptr)) return MASSV_ERR_INVALID_ARG;
    TimingHooks& h = timing_hooks();
    cudaEvent_t a = reinterpret_cast<cudaEvent_t>(start), b = reinterpret_cast<cudaEvent_t>(stop);
    switch (kernel) {
        case MASSV_TIMED_LM_HEAD: h.lm_head_start = a; h.lm_head_stop = b; return MASSV_OK;
        case MASSV_TIMED_ATTN: h.attn_start = a; h.attn_stop = b; return MASSV_OK;
        case MASSV_TIMED_RESIDUAL: h.residual_start = a; h.residual_stop = b; return MASSV_OK;
        default: return MASSV_ERR_INVALID_ARG;
    }
}

uint64_t massv_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

}  // extern "C"
