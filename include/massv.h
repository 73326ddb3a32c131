/*
 * massv.h - C ABI of the target-side verification step of speculative decoding
 * for vision-language models (MASSV paper, Sec. 2.1) on NVIDIA B200 (sm_100a).
 *
 * One verify step, per sequence b of a batch, takes the gamma tokens proposed
 * by a draft model plus the last emitted token (R = gamma + 1 "block rows"),
 * scores all of them with the target model in one pass, and decides how many
 * drafts survive:
 *
 *   massv_verify_attn   attention of the R block rows over a paged bf16 KV
 *                       cache (image-token prefix, then text, then the block),
 *                       appending the block's K/V to the cache;
 *   massv_accept        LM-head logits for the R rows, temperature softmax,
 *                       sequential acceptance of the drafts, the extra token
 *                       (residual draw on rejection, bonus draw otherwise),
 *                       accepted length;
 *   massv_kv_commit     advance (or, on rollback, keep) the cache lengths.
 *
 * General rules
 *   - Every pointer argument except descriptors is DEVICE memory owned by the
 *     caller and valid until the stream has run the call.  Descriptors are
 *     host structs read during the call.
 *   - Calls enqueue work on `stream` and return without synchronising it.  The
 *     library allocates no device memory; scratch comes from `workspace`
 *     (256-byte aligned, at least *_workspace_size() bytes, contents undefined
 *     on entry and exit; two calls that may overlap on the GPU need separate
 *     workspaces).
 *   - bf16 tensors are dense, row-major in the index order given, last index
 *     fastest.  Pointers must be 16-byte aligned.
 *   - The return value reports errors detectable on the host before anything is
 *     launched (nothing is enqueued then).  `dev_status`, when not NULL, is one
 *     int32 the caller zeroes; kernels store a negative massv_status there when
 *     they detect a problem on the device (an unmapped page, a wait that ran
 *     out).  It never traps or hangs the GPU.
 *   - The library draws no random numbers: uniforms are inputs.
 */
#ifndef MASSV_H
#define MASSV_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct CUstream_st *massv_stream_t;   /* a cudaStream_t */

typedef enum massv_status {
    MASSV_OK = 0,
    MASSV_ERR_INVALID_ARG = -1,   /* NULL where data is required, non-positive size, misaligned pointer */
    MASSV_ERR_UNSUPPORTED = -2,   /* shape outside the supported set (see each call) */
    MASSV_ERR_CAPACITY = -3,      /* page table cannot hold L_b + gamma + 1 positions */
    MASSV_ERR_WORKSPACE = -4,     /* workspace NULL, misaligned or too small */
    MASSV_ERR_CUDA = -5,          /* a CUDA runtime/driver call failed */
    MASSV_ERR_TIMEOUT = -6,       /* device-side wait exceeded its iteration limit (dev_status only) */
    MASSV_ERR_BOUNDS = -7         /* debug builds (-DMASSV_DEBUG) only: an index computed on the device fell outside
                                     its buffer; the access was skipped (dev_status only) */
} massv_status;

/* Geometry of the attention call. */
typedef struct massv_attn_desc {
    int32_t batch;               /* B >= 1 */
    int32_t gamma;               /* speculation length, 0..7; R = gamma + 1 query rows per sequence */
    int32_t n_q_heads;           /* Hq, a multiple of n_kv_heads; (Hq/Hkv) * R <= 64 */
    int32_t n_kv_heads;          /* Hkv */
    int32_t head_dim;            /* d: 64, 128 or 256 */
    int32_t page_size;           /* tokens per KV page: 16 */
    int32_t max_pages_per_seq;   /* row length of page_table */
    int64_t num_pages;           /* pages in the pool */
    float scale;                 /* score scale; 0 selects 1/sqrt(d) */
    int32_t kv_chunk;            /* tokens per split of the KV scan, multiple of 64, <= 4096; 0 = choose automatically */
    int32_t window;              /* sliding-window attention: a row sees only its last `window` positions; 0 = full */
    uint32_t flags;              /* kernel choice, one of MASSV_ATTN_KERNEL_*; 0 = by shape */
} massv_attn_desc;

/* massv_attn_desc.flags.  Both kernels compute the same thing to the same tolerance; the choice
 * only matters for speed (the library picks by the number of query rows per KV head) and is
 * exposed so that either kernel can be checked on any shape. */
#define MASSV_ATTN_KERNEL_AUTO 0u
#define MASSV_ATTN_KERNEL_WARP_MMA 1u   /* warp-level tensor-core MMAs, operands through registers */
#define MASSV_ATTN_KERNEL_TCGEN05 2u    /* tcgen05 MMAs with accumulators in tensor memory */

/* Geometry of the acceptance call. */
typedef struct massv_accept_desc {
    int32_t batch;               /* B >= 1; M = B * (gamma + 1) <= 512 rows */
    int32_t gamma;               /* 0..7 */
    int32_t hidden;              /* K, a multiple of 64 */
    int32_t vocab;               /* V, a multiple of 8 */
    float temperature;           /* T >= 0; 0 selects greedy verification */
    uint32_t flags;              /* reserved, 0 (see MASSV_TEST_SKIP_STAGE below) */
} massv_accept_desc;

/* Only in a library compiled with -DMASSV_TEST_HOOKS (the test suite builds one beside the product, with a
 * short MASSV_SPIN_LIMIT): massv_accept_desc.flags = MASSV_TEST_SKIP_STAGE makes the LM-head kernel's
 * producer withhold one pipeline stage - no bytes announced, no copy issued - so that the consumer's
 * bounded wait runs out and the call reports MASSV_ERR_TIMEOUT in dev_status instead of waiting for ever.
 * The product library refuses any non-zero flags. */
#define MASSV_TEST_SKIP_STAGE 0x80000000u

/* Bytes of scratch massv_verify_attn needs for this geometry (0 on a bad descriptor). */
size_t massv_verify_attn_workspace_size(const massv_attn_desc *desc);

/*
 * Target attention for the block rows (Sec. 2.1: the target scores positions
 * t+1 .. t+gamma+1 of a drafted block in a single pass; Sec. 2.2: the context
 * is m projected image features followed by text tokens).
 *
 * For sequence b with committed length L_b = seq_lens[b]:
 *   1. k_new[b,j], v_new[b,j] are stored at cache position L_b + j (j = 0..gamma)
 *      through page_table (position i lives in page page_table[b, i / 16],
 *      slot i % 16).  seq_lens is NOT modified (see massv_kv_commit).
 *   2. out[b,j,h,:] = sum_i softmax_i(scale * <q[b,j,h,:], K_i>) V_i over
 *      positions i = 0 .. L_b + j of KV head h / (Hq/Hkv): the whole committed
 *      prefix and the block rows up to and including j (causal inside the block).
 * Q and cached K are used as given (any positional encoding is already applied).
 * With desc->window = w > 0 the sum runs over positions max(0, L_b + j - w + 1) .. L_b + j only
 * (local attention layers; Sec. 4 of the paper notes Gemma3's interleaved sliding-window layers).
 *
 *   q                bf16 [B, R, Hq, d]
 *   k_new, v_new     bf16 [B, R, Hkv, d]
 *   k_pages, v_pages bf16 [num_pages, Hkv, 16, d]   (written at the block slots)
 *   page_table       int32 [B, max_pages_per_seq]; entries covering positions
 *                    0 .. L_b + gamma must be valid page ids
 *   seq_lens         int32 [B], 0 <= L_b and L_b + R <= 16 * max_pages_per_seq
 *   out              bf16 [B, R, Hq, d]
 *   out_f32          optional fp32 copy of out before rounding, same shape
 *   lse              optional fp32 [B, R, Hq]: natural-log sum of exp of the scaled scores
 * Math: bf16 operands, fp32 accumulation; softmax weights are rounded to bf16
 * before multiplying V.  A sequence whose lengths violate the capacity rule is
 * skipped and MASSV_ERR_CAPACITY is stored in dev_status.
 */
int massv_verify_attn(const massv_attn_desc *desc, const void *q, const void *k_new, const void *v_new,
                      void *k_pages, void *v_pages, const int32_t *page_table, const int32_t *seq_lens,
                      void *out, float *out_f32, float *lse,
                      void *workspace, size_t workspace_bytes, int32_t *dev_status, massv_stream_t stream);

/* Bytes of scratch massv_accept needs (0 on a bad descriptor).  Includes room
 * for the fp32 logits when T > 0, whether or not logits_out is supplied. */
size_t massv_accept_workspace_size(const massv_accept_desc *desc);

/*
 * LM head + temperature softmax + speculative acceptance (Sec. 2.1).
 *
 * Row (b,j) of `hidden` is the target's final hidden state at block position j;
 * its logits are z_j = lm_head * hidden[b,j] and, for T > 0, p_j = softmax(z_j / T)
 * is the target distribution for the token after block position j.
 *
 * T > 0: draft j (token x = draft_tokens[b,j], draft distribution
 *   q_j = draft_probs[b,j,:]) is accepted with probability min(1, p_j(x)/q_j(x)),
 *   realised with the caller's uniform as  u_accept[b,j] * q_j(x) < p_j(x)
 *   (fp32).  Drafts are examined in order; at the first rejection n the extra
 *   token is drawn from norm(max(p_n - q_n, 0)); if all gamma drafts pass
 *   (n = gamma) it is drawn from p_gamma.  The draw is an inverse-CDF walk in
 *   vocabulary order with u_sample[b,n]: the first index whose running mass
 *   exceeds u * total (fp64 running sums); zero-mass tokens are never drawn.
 *   If the residual has no mass the draw uses p_n.  draft_probs is used as
 *   given (it is the drafter's distribution at the drafter's temperature).
 * T == 0: draft j is accepted iff x equals argmax_v z_j[v] (lowest index on
 *   ties); the extra token is argmax_v z_n[v].  draft_probs, u_accept and
 *   u_sample are ignored and may be NULL.
 *
 *   hidden        bf16 [B, R, K]
 *   lm_head       bf16 [V, K]
 *   draft_tokens  int32 [B, gamma], each in [0, V)
 *   draft_probs   fp32 [B, gamma, V]           (T > 0)
 *   u_accept      fp32 [B, gamma] in [0,1)     (T > 0)
 *   u_sample      fp32 [B, R] in [0,1)         (T > 0)
 *   out_tokens    int32 [B, R]: the n accepted drafts, the extra token, then -1
 *   accept_len    int32 [B]: n + 1, the tokens gained by this target pass
 *                 (its batch mean is the paper's mean accepted length tau)
 *   logits_out    optional fp32 [B, R, V]: z
 *   probs_out     optional fp32 [B, R, V]: p (T > 0 only; must be NULL at T == 0)
 * Math: bf16 x bf16 products accumulated in fp32 on the tensor cores.
 */
int massv_accept(const massv_accept_desc *desc, const void *hidden, const void *lm_head,
                 const int32_t *draft_tokens, const float *draft_probs,
                 const float *u_accept, const float *u_sample,
                 int32_t *out_tokens, int32_t *accept_len, float *logits_out, float *probs_out,
                 void *workspace, size_t workspace_bytes, int32_t *dev_status, massv_stream_t stream);

/*
 * massv_accept for callers that have no device memory to offer as workspace and
 * may not allocate any.  (The paper has no counterpart for this call; it exists
 * for deployment reasons only.)
 *
 * Who needs it: an engine whose device pool was split up at start-up and has
 * nothing left to lend, code that runs as a guest inside another program's CUDA
 * context where allocating after initialisation is against the rules, and
 * latency-critical loops that must not call cudaMalloc because it stalls the
 * whole device.  Such callers still own the inputs and the outputs; only the
 * scratch moves into the library.
 *
 * It computes exactly what massv_accept computes, with the same kernels and the
 * same arguments, except:
 *   - there is no workspace argument.  Scratch is a fixed array of about 210 KiB
 *     of device memory that belongs to the library image: every GPU that loads
 *     the library holds it until the process exits, used or not.
 *   - the fp32 logits have no room in that array, so at T > 0 logits_out is
 *     REQUIRED (it is an ordinary output of the caller).  At T == 0 it stays
 *     optional.
 *   - limits: B * (gamma + 1) <= 64, B <= 64, vocab <= 524288.  Anything larger
 *     returns MASSV_ERR_WORKSPACE and launches nothing.
 *   - the first call on each device looks up the array's device address (the
 *     device that is current at the call).  Make that first call during start-up,
 *     outside any stream capture.  Later calls on that device reuse the address,
 *     which is remembered per device ordinal: after a cudaDeviceReset (which
 *     unloads the library image from the device) it is stale, so do not reset a
 *     device between calls.
 *   - all calls on one device share the one array, and it keeps what the last
 *     call left in it (every part is rewritten by the call's own kernels before
 *     it is read, so nothing stale is used).  Two
 *     calls that can run on the GPU at the same time (different streams without
 *     an ordering between them) would overwrite each other's scratch: keep calls
 *     on one stream or order them yourself.
 * It never calls cudaMalloc, cudaFree or any allocating routine.
 */
int massv_accept_static(const massv_accept_desc *desc, const void *hidden, const void *lm_head,
                        const int32_t *draft_tokens, const float *draft_probs,
                        const float *u_accept, const float *u_sample,
                        int32_t *out_tokens, int32_t *accept_len, float *logits_out, float *probs_out,
                        int32_t *dev_status, massv_stream_t stream);

/* Bytes of scratch massv_tvd needs (0 on a bad descriptor, gamma == 0 or T == 0). */
size_t massv_tvd_workspace_size(const massv_accept_desc *desc);

/*
 * Distribution-alignment diagnostic of the paper (Eq. 6): for every drafted
 * position (b, j), the total variation distance between the target distribution
 * p_j = softmax(z_j / T) and the draft distribution q_j,
 *     tvd_out[b,j] = 1/2 * sum_v |p_j(v) - q_j(v)|   in [0, 1],
 * and optionally accept_prob_out[b,j] = sum_v min(p_j(v), q_j(v)) = 1 - TVD, the
 * probability that the rejection test of massv_accept accepts a draft token
 * drawn from q_j.
 *   logits        fp32 [B, R, V]   (the logits_out of massv_accept; rows 0..gamma-1 are used)
 *   draft_probs   fp32 [B, gamma, V]
 *   tvd_out       fp32 [B, gamma];  accept_prob_out  optional fp32 [B, gamma]
 * Needs T > 0 and gamma >= 1.  Reads every drafted row once (B*gamma*V*8 bytes),
 * twice for the logits; sums run in fp64 in a fixed order.
 */
int massv_tvd(const massv_accept_desc *desc, const float *logits, const float *draft_probs,
              float *tvd_out, float *accept_prob_out,
              void *workspace, size_t workspace_bytes, int32_t *dev_status, massv_stream_t stream);

/*
 * The same diagnostic (Eq. 6) right after massv_accept on the same stream, with ONE read of the logits:
 * massv_accept leaves every row's merged softmax statistics (max logit, sum of exp((z - max)/T)) in its
 * workspace, and this call takes them from there instead of computing them again, so it reads each
 * drafted row of the logits and of q once (B*gamma*V*8 bytes).
 *   desc                  the descriptor massv_accept was called with (T > 0, gamma >= 1)
 *   logits                the logits_out of that massv_accept call
 *   accept_workspace      the workspace of that call, untouched since (its size is checked)
 *   tvd_out, accept_prob_out, workspace (massv_tvd_workspace_size bytes): as for massv_tvd
 * The statistics come from the LM-head kernel's fp32 arithmetic; results agree with massv_tvd's to
 * rounding (both are held to 1e-4 absolute against a double-precision evaluation).
 */
int massv_tvd_after_accept(const massv_accept_desc *desc, const float *logits, const float *draft_probs,
                           const void *accept_workspace, size_t accept_workspace_bytes,
                           float *tvd_out, float *accept_prob_out,
                           void *workspace, size_t workspace_bytes, int32_t *dev_status, massv_stream_t stream);

/*
 * Commit or roll back the speculative block (Sec. 2.1: accepted tokens are
 * added to the output and the next iteration starts from them).
 * accept_len != NULL: seq_lens[b] += accept_len[b]; cache rows of block
 * positions 0 .. n stay, rows beyond are dead and will be overwritten.
 * accept_len == NULL: rollback, seq_lens is left unchanged, which discards the
 * whole appended block.  gamma bounds accept_len (values outside [1, gamma+1]
 * store MASSV_ERR_INVALID_ARG in dev_status and leave that length unchanged).
 */
int massv_kv_commit(int32_t batch, int32_t gamma, const int32_t *accept_len, int32_t *seq_lens,
                    int32_t *dev_status, massv_stream_t stream);

/*
 * Histogram of TVD values, the form in which the paper presents Eq. 6 (Fig. 4): counts[k] += the number
 * of tvd[i] in bin k of `bins` equal-width bins over [0, 1]; bin k is [k / bins, (k + 1) / bins), the last
 * bin also takes 1.  The bin index is floor(tvd * bins) with the product rounded once in fp32, clamped to
 * [0, bins - 1]; NaN is not counted.  counts is ADDED to (int64 [bins], device memory, zeroed by the
 * caller before the first call), so one array can collect the tvd_out of many massv_tvd calls.
 *   0 <= n <= 2^40;  1 <= bins <= 4096;  tvd fp32 [n] (for instance tvd_out of massv_tvd)
 * No workspace.
 */
int massv_tvd_histogram(int64_t n, const float *tvd, int32_t bins, int64_t *counts, massv_stream_t stream);

/*
 * Nucleus (top-p) sampling of softmax(z / T), row by row (Sec. 3.2: the target's responses for the
 * drafter's self-distillation are drawn as sample_top-p(p(. | I, X)); the same call is the drafter's
 * sampling step when it samples with top-p, probs_out then being the draft distribution q that
 * massv_accept takes).  Per row: order the tokens by probability, largest first (equal probabilities:
 * lower index first); the nucleus is the shortest prefix of that order whose mass reaches top_p;
 * q = p restricted to the nucleus and renormalised; tokens[r] is the inverse CDF of q in vocabulary
 * order at u[r] (first index whose running mass exceeds u * total, never a zero-mass token).
 *
 *   rows >= 1;  1 <= vocab <= 2^21;  temperature > 0;  0 < top_p <= 1 (1 keeps every token)
 *   logits        fp32 [rows, vocab] (for instance logits_out of massv_accept)
 *   u             fp32 [rows], uniforms in [0, 1) supplied by the caller
 *   tokens        int32 [rows]
 *   probs_out     optional fp32 [rows, vocab]: q, zeros outside the nucleus
 * Math: weights exp((z - max) / T) in fp32, all sums in fp64 in a fixed order.  No workspace.  A row
 * without a finite logit stores MASSV_ERR_INVALID_ARG in dev_status and token 0.
 */
int massv_sample_top_p(int32_t rows, int32_t vocab, float temperature, float top_p, const float *logits,
                       const float *u, int32_t *tokens, float *probs_out, int32_t *dev_status,
                       massv_stream_t stream);

/*
 * Acceptance with the vocabulary cut across `world` ranks (tensor-parallel LM head).  The arithmetic is
 * that of massv_accept (Sec. 2.1: rejection test, residual norm(max(0, p - q)), bonus token; greedy
 * prefix rule at temperature 0); only where the data lives changes.  Rank r holds rows
 * [r * vocab, (r + 1) * vocab) of the LM head and the same columns of q: desc->vocab is the SHARD's size,
 * equal on every rank, so the whole vocabulary is world * vocab.  The library exchanges nothing itself:
 * each rank fills an exchange buffer, the caller all-gathers it (NCCL or any other transport; rank r's
 * copy at offset r * size of the gathered buffer), and every rank then takes the same decisions from the
 * same gathered values.  Three all-gathers per step at T > 0, one at T == 0.  On every rank:
 *
 *   1. massv_shard_lm_head      logits of the shard; per-row max / sum-exp / argmax partials (argmax
 *                               indices already global) go into `stats`; *n_partials (host) = partial
 *                               slots written, the same on every rank.
 *   2. massv_shard_gather_draft (T > 0) logit and q at each drafted token this rank owns, -inf
 *                               elsewhere, into `stats`.
 *      all-gather `stats`: fp32 words, massv_shard_stats_words per rank.
 *   3. massv_shard_scan         merges the partials of all ranks (ranks in order), takes the owner's
 *                               values at the drafted tokens, runs the rejection test (or the greedy
 *                               prefix rule), writes accept_len, the accepted drafts into out_tokens
 *                               and, at T == 0, the extra token; fills `state`
 *                               (massv_shard_state_bytes).  T == 0 ends here.
 *   4. massv_shard_masses       masses of this shard's 4096-entry chunks of the row the extra token is
 *                               drawn from: of max(p - q, 0) (of p for the bonus row) and of p.
 *      all-gather `masses`: fp64, massv_shard_mass_count per rank.
 *   5. massv_shard_pick         every rank walks the gathered masses (ranks in order = vocabulary
 *                               order) to the chunk where the running mass passes u * total; the rank
 *                               that owns it stores the token (global index), the others -1.  A
 *                               residual without mass anywhere falls back to p, as massv_accept does.
 *      all-gather token_out: int32 [batch] per rank.
 *   6. massv_shard_set_token    stores the owner's token at out_tokens[b, accept_len[b] - 1].
 *
 * logits_shard fp32 [batch * (gamma + 1), vocab] (required at T > 0, optional at T == 0);
 * draft_probs_shard fp32 [batch, gamma, vocab]; u_accept, u_sample, draft_tokens, out_tokens,
 * accept_len as for massv_accept.  world * ceil(vocab / 4096) <= 512.  `stats` 16-byte aligned.  All
 * pointers are device pointers except n_partials.  Errors as for massv_accept.
 */
size_t massv_shard_stats_words(const massv_accept_desc *desc);
size_t massv_shard_mass_count(const massv_accept_desc *desc);
size_t massv_shard_state_bytes(const massv_accept_desc *desc);
int massv_shard_lm_head(const massv_accept_desc *desc, int32_t world, int32_t rank, const void *hidden,
                        const void *lm_head_shard, float *logits_shard, float *stats, int32_t *n_partials,
                        int32_t *dev_status, massv_stream_t stream);
int massv_shard_gather_draft(const massv_accept_desc *desc, int32_t world, int32_t rank,
                             const float *logits_shard, const float *draft_probs_shard,
                             const int32_t *draft_tokens, float *stats, int32_t *dev_status,
                             massv_stream_t stream);
int massv_shard_scan(const massv_accept_desc *desc, int32_t world, int32_t n_partials, const float *stats_all,
                     const int32_t *draft_tokens, const float *u_accept, int32_t *out_tokens,
                     int32_t *accept_len, void *state, int32_t *dev_status, massv_stream_t stream);
int massv_shard_masses(const massv_accept_desc *desc, int32_t world, int32_t rank, const float *logits_shard,
                       const float *draft_probs_shard, const void *state, double *masses,
                       int32_t *dev_status, massv_stream_t stream);
int massv_shard_pick(const massv_accept_desc *desc, int32_t world, int32_t rank, const double *masses_all,
                     const float *u_sample, const void *state, const float *logits_shard,
                     const float *draft_probs_shard, int32_t *token_out, int32_t *dev_status,
                     massv_stream_t stream);
int massv_shard_set_token(const massv_accept_desc *desc, int32_t world, const void *state,
                          const int32_t *tokens_all, int32_t *out_tokens, int32_t *dev_status,
                          massv_stream_t stream);

/*
 * The all-gather of the sharded acceptance done by this library's own kernel instead of a collective
 * library: one launch stores `bytes` bytes of src at offset rank * bytes of each of the `world`
 * gathered buffers.  gathered is a HOST array of world device pointers; entry w is rank w's gathered
 * buffer as seen from this GPU (its own for w == rank, peer-mapped memory for the others: a symmetric
 * allocation or an IPC mapping), each world * bytes long.  Plain stores only.  The call orders nothing
 * between ranks: a rank may read its gathered buffer only after every rank's publish has completed
 * (the caller's barrier), and may publish into it again only after every rank has finished reading.
 * bytes % 4 == 0; pointers 4-byte aligned (16-byte aligned buffers and sizes copy 16 bytes per store);
 * world <= 16.
 */
int massv_shard_publish(const void *src, size_t bytes, void *const *gathered, int32_t world, int32_t rank,
                        massv_stream_t stream);

/* Human-readable name of a massv_status value. */
const char *massv_strerror(int status);

/* Library version: major * 10000 + minor * 100 + patch. */
int massv_version(void);

/* Number of GPU kernels this library has launched in this process so far
 * (diagnostic; lets a caller confirm that a call really ran on the device). */
uint64_t massv_launch_count(void);

/*
 * Measurement hook (no counterpart in the paper).  massv_accept and massv_verify_attn launch several
 * kernels each; a caller that wants the duration of the dominant one alone (the LM-head GEMM, the
 * attention split kernel) hands in two CUDA events per call, and the library records `start`
 * immediately before and `stop` immediately after that kernel on the call's stream.  The setting is
 * per host thread and stays until changed; NULL for both switches a hook off.  Events are
 * cudaEvent_t handles created with timing enabled and owned by the caller.  Recording them keeps
 * the timed kernel from overlapping with its neighbours in the stream, so leave the hooks off on
 * calls whose end-to-end time matters.
 */
typedef struct CUevent_st *massv_event_t;     /* a cudaEvent_t */
int massv_set_timing_events(massv_event_t lm_head_start, massv_event_t lm_head_stop,
                            massv_event_t attn_start, massv_event_t attn_stop);

/* The same hook, one kernel at a time: `kernel` is one of MASSV_TIMED_*; NULL for both events
 * switches that kernel's hook off.  MASSV_TIMED_RESIDUAL is the residual / bonus draw of
 * massv_accept at T > 0 (the one pass over the vocabulary row the extra token is drawn from). */
#define MASSV_TIMED_LM_HEAD 0
#define MASSV_TIMED_ATTN 1
#define MASSV_TIMED_RESIDUAL 2
int massv_set_kernel_timing(int32_t kernel, massv_event_t start, massv_event_t stop);

#ifdef __cplusplus
}
#endif
#endif /* MASSV_H */
