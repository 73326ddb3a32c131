// Internal launch interfaces between the C ABI (api.cu) and the kernels.
#pragma once

#include <cuda.h>

#include "common.cuh"

namespace massv {

// ---------------------------------------------------------------- attention
struct AttnParams {
    int B, R, Hq, Hkv, d, max_pages;
    int64_t num_pages;
    float scale;
    int window;        // sliding window length, 0 = full attention
    int kv_chunk;      // tokens per split
    int max_chunks;    // splits launched per (sequence, kv head)
    const __nv_bfloat16 *q, *k_new, *v_new;
    __nv_bfloat16 *k_pages, *v_pages;
    const int32_t *page_table, *seq_lens;
    __nv_bfloat16* out;
    float *out_f32, *lse;
    float* part_o;     // [B, Hkv, max_chunks, rows_pad, d] unnormalised partial outputs
    float* part_ml;    // [B, Hkv, max_chunks, rows_pad, 2] running max (log2 domain) and sum
    int32_t* dev_status;
    int path;          // 0: choose by shape, 1: warp-level MMA kernel, 2: tcgen05 kernel
    bool chunk_forced; // the caller fixed kv_chunk: keep the (chunk, KV head, sequence) grid
    // flat schedule of the tcgen05 kernel: two partial slots per resident CTA, and what the merge needs
    float* flat_part_o;    // [kFlatMaxCtas * 2, rows_pad, d]
    float* flat_part_ml;   // [kFlatMaxCtas * 2, rows_pad, 2]
    int32_t* flat_meta;    // [0] tiles per CTA, [1] tiles in all, [2 + b] tiles of sequences 0 .. b-1 (per KV head)
};
constexpr int kFlatMaxCtas = 320;      // resident CTAs of the flat schedule (two per SM)
constexpr int kFlatMaxBatchMeta = 1024;
int attn_rows_pad(int group_rows);                 // query rows per KV head, padded to the MMA tile
cudaError_t launch_verify_attn(const AttnParams& p, cudaStream_t stream);
// tcgen05 variant of the split kernel (attn_umma.cu); the tensor maps are the ones the warp-MMA kernel uses
bool attn_umma_supported(const AttnParams& p);
bool attn_umma_flat_supported(const AttnParams& p);
bool attn_use_umma(const AttnParams& p);
// flat: balanced persistent schedule with its own merge kernel; otherwise the chunk grid, merged by the caller.
// *launched receives the number of kernels launched.
// split_done, when not null, is recorded right after the split kernel (before any merge kernel).
cudaError_t launch_attn_umma(const AttnParams& p, const CUtensorMap& map_k, const CUtensorMap& map_v, cudaStream_t stream, bool flat,
                             int* launched, cudaEvent_t split_done);

// ---------------------------------------------------------------- LM head
struct LmHeadParams {
    int M, K, V;
    float inv_T_log2e;              // log2(e)/T; unused at T == 0
    int greedy;                     // 1: T == 0 (no sum of exponentials, no logits needed)
    const __nv_bfloat16 *hidden, *lm_head;
    float* logits;                  // [M, V] or nullptr
    int n_part;                     // partial slots available
    float *part_max, *part_sum;     // [n_part, M]
    int32_t* part_idx;              // [n_part, M]
    int32_t* dev_status;
    int idx_offset = 0;             // added to the argmax indices (first vocabulary row of a shard)
    int test_skip_stage = 0;        // test builds only: the producer withholds one stage (see MASSV_TEST_SKIP_STAGE)
};
int lm_head_num_partials(int M, int V);            // upper bound of the partial slots, for workspace sizing
// *n_part_used receives the number of slots this launch fills (<= p.n_part).
cudaError_t launch_lm_head(const LmHeadParams& p, cudaStream_t stream, int* n_part_used);

// ---------------------------------------------------------------- acceptance
struct AcceptParams {
    int B, gamma, V;
    float T;
    int n_part;
    const float *part_max, *part_sum;
    const int32_t* part_idx;
    const float* logits;            // [B*(gamma+1), V], T > 0 only
    const int32_t* draft_tokens;
    const float *draft_probs, *u_accept, *u_sample;
    int32_t *out_tokens, *accept_len;
    float* probs_out;               // optional
    SeqState* seq_state;            // [B]
    float* row_stats = nullptr;     // optional [B*(gamma+1), 2]: the merged (max logit, sum exp((z - max)/T)) of every row
    double* chunk_sums;             // [B, n_chunks]
    double* seg_sums = nullptr;     // optional [B, n_chunks, 8]: the masses of the eight 512-entry segments of every chunk
    unsigned int* counters;         // [B]
    int n_chunks;
    int32_t* dev_status;
    // vocabulary-sharded use: the target's logit and the drafter's probability at every drafted token,
    // collected from the rank that owns the token (then `logits` / `draft_probs` are not read by the scan)
    const float* z_at_draft = nullptr;   // [B, gamma]
    const float* q_at_draft = nullptr;   // [B, gamma]
    // gathered exchange buffers: partial slot i lives in rank i / part_per_rank's copy, the copies
    // rank_stride words apart; z / q at the drafted tokens are the maximum over the ranks' copies
    int part_per_rank = 0;               // 0: one contiguous [n_part, M] array
    int ranks = 1;
    size_t rank_stride = 0;              // in 4-byte words
};
cudaError_t launch_accept(const AcceptParams& p, cudaStream_t stream);
cudaError_t launch_accept_scan_only(const AcceptParams& p, cudaStream_t stream);

// ---------------------------------------------------------------- vocabulary shards
struct ShardParams {
    int B, gamma, Vs;               // Vs: vocabulary entries of this shard
    int vocab_offset;               // first vocabulary index of this shard
    float T;
    const float* logits;            // [B*(gamma+1), Vs]
    const float* draft_probs;       // [B, gamma, Vs]
    const int32_t* draft_tokens;    // [B, gamma]
    float *z_at_draft, *q_at_draft; // [B, gamma]: -inf where another shard owns the token
    const SeqState* seq_state;      // [B]
    double *sums_res, *sums_p;      // [B, n_chunks]: chunk masses of max(p - q, 0) and of p on the sampled row
    int n_chunks;                   // chunks of this shard
    // pick
    const double *all_res, *all_p;  // rank r's [B, n_chunks] at + r * mass_rank_stride: ranks in order are vocabulary order
    size_t mass_rank_stride;        // in doubles
    int world, rank;
    const float* u_sample;          // [B, gamma+1]
    int32_t* token_out;             // [B]: the drawn token if this shard owns it, else -1
    int32_t* out_tokens;            // [B, gamma+1]
    const int32_t* tokens_in;       // [world, B]: -1 from the ranks that do not own the token
    int32_t* dev_status;
};
cudaError_t launch_shard_gather_draft(const ShardParams& p, cudaStream_t stream);
cudaError_t launch_shard_masses(const ShardParams& p, cudaStream_t stream);
cudaError_t launch_shard_pick(const ShardParams& p, cudaStream_t stream);
cudaError_t launch_shard_set_token(const ShardParams& p, cudaStream_t stream);

// counts[k] += number of tvd values in bin k of `bins` equal bins over [0, 1] (NaN not counted)
cudaError_t launch_tvd_histogram(long long n, const float* tvd, int bins, unsigned long long* counts, cudaStream_t stream);

// An all-gather by stores: this rank's buffer goes to offset rank * bytes of every rank's gathered buffer.
constexpr int kMaxPeers = 16;
struct PublishParams {
    const void* src;
    size_t bytes;                   // multiple of 4
    void* dst[kMaxPeers];           // the ranks' gathered buffers (peer-mapped device pointers)
    int world, rank;
};
cudaError_t launch_shard_publish(const PublishParams& p, cudaStream_t stream);

// ---------------------------------------------------------------- TVD diagnostic
constexpr int kTvdSlices = 16;      // vocabulary slices per row
struct TvdParams {
    int B, gamma, V;
    float inv_T;
    int slice_len;                  // entries per slice
    const float *logits, *draft_probs;
    float *tvd_out, *accept_prob_out;
    float* slice_max;               // [B*gamma, kTvdSlices]
    double *slice_sum, *slice_abs, *slice_min;
    const float* row_stats = nullptr;   // [B*(gamma+1), 2] left by the acceptance scan: then the statistics pass is skipped
};
cudaError_t launch_tvd(const TvdParams& p, cudaStream_t stream);

// ---------------------------------------------------------------- nucleus (top-p) sampling
struct TopPParams {
    int rows, V;
    float inv_T, top_p;
    const float *logits, *u;
    int32_t* tokens;
    float* probs_out;               // optional [rows, V]: the renormalised nucleus distribution
    int32_t* dev_status;
};
cudaError_t launch_top_p(const TopPParams& p, cudaStream_t stream);

cudaError_t launch_kv_commit(int B, int gamma, const int32_t* accept_len, int32_t* seq_lens, int32_t* dev_status,
                             cudaStream_t stream);

}  // namespace massv
