/*
 * CPU oracle for the target model's verification step of speculative decoding
 * (paper Sec. 2.1).  TEST INFRASTRUCTURE ONLY: a plain, slow restatement of the
 * definitions in fp64.  It shares no code with the CUDA library and must never
 * be on a product path; only tests, the smoke check and the benchmark's CPU
 * baseline leg call it.
 *
 * Conventions
 *   - bf16 tensors arrive as uint16_t bit patterns and are widened exactly.
 *   - All sums run in double, in index order, with a two-pass softmax.
 *   - OpenMP pragmas parallelise independent outer iterations only; the
 *     arithmetic inside one output element is sequential.
 *
 * Real-model mean accepted length (the paper's Table 1) is "parity unpinned":
 * it needs weights and datasets that are not available.  Every function below
 * is pinned by the CPU tests (closed forms, brute-force enumeration, library
 * routines).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

static double bf16_to_f64(uint16_t h)
{
    uint32_t u = ((uint32_t)h) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

/* Flat index of element (position pos, kv head g, channel c) of sequence b in a
 * page pool laid out [page][kv_head][slot][channel]. */
static size_t kv_index(const int32_t *page_table, int max_pages, int page_size, int n_kv_heads, int head_dim,
                       int b, int pos, int g, int c)
{
    int page = page_table[(size_t)b * max_pages + pos / page_size];
    int slot = pos % page_size;
    return (((size_t)page * n_kv_heads + g) * page_size + slot) * head_dim + c;
}

/*
 * The gamma+1 block positions enter the target's context (Sec. 2.1: the target
 * scores positions t+1 .. t+gamma+1 in one forward call): store their keys and
 * values at logical positions L_b .. L_b+gamma of sequence b.
 *   k_new, v_new : bf16 [B, R, Hkv, d];  pages : bf16 [P, Hkv, page, d]
 */
void oracle_kv_append(int B, int R, int n_kv_heads, int head_dim, int page_size, int max_pages,
                      const uint16_t *k_new, const uint16_t *v_new, uint16_t *k_pages, uint16_t *v_pages,
                      const int32_t *page_table, const int32_t *seq_lens)
{
    for (int b = 0; b < B; ++b)
        for (int j = 0; j < R; ++j)
            for (int g = 0; g < n_kv_heads; ++g)
                for (int c = 0; c < head_dim; ++c) {
                    size_t src = (((size_t)b * R + j) * n_kv_heads + g) * head_dim + c;
                    size_t dst = kv_index(page_table, max_pages, page_size, n_kv_heads, head_dim,
                                          b, seq_lens[b] + j, g, c);
                    k_pages[dst] = k_new[src];
                    v_pages[dst] = v_new[src];
                }
}

/*
 * Attention of the R = gamma+1 block rows over the cache (Sec. 2.1, "one
 * forward call" of the target).  Row j of sequence b sits at position L_b + j
 * and sees positions 0 .. L_b + j: the whole committed prefix (image tokens
 * first, then text: Sec. 2.2) and the block rows up to itself.  Query head h
 * reads KV head h / (Hq/Hkv).
 *   out[b,j,h,:] = sum_i softmax_i(scale * <q[b,j,h,:], K[i]>) * V[i]
 *   lse[b,j,h]   = log sum_i exp(scale * <q, K[i]>)
 * The block must already be appended.  q : bf16 [B,R,Hq,d]; out : f64 same shape.
 *
 * window > 0 selects sliding-window attention (the local layers of Gemma3-style
 * targets, which the paper's Sec. 4 notes as an architectural difference without
 * fixing a size): the row at position P sees only positions P-window+1 .. P.
 * window == 0 is full attention.
 */
void oracle_verify_attn(int B, int R, int n_q_heads, int n_kv_heads, int head_dim, int page_size, int max_pages,
                        int window, double scale, const uint16_t *q, const uint16_t *k_pages, const uint16_t *v_pages,
                        const int32_t *page_table, const int32_t *seq_lens, double *out, double *lse)
{
    int group = n_q_heads / n_kv_heads;
    long n_items = (long)B * R * n_q_heads;
#pragma omp parallel for schedule(dynamic, 1)
    for (long item = 0; item < n_items; ++item) {
        int h = (int)(item % n_q_heads);
        int j = (int)((item / n_q_heads) % R);
        int b = (int)(item / ((long)n_q_heads * R));
        int g = h / group;
        int n_ctx = seq_lens[b] + j + 1;
        int first = (window > 0 && n_ctx > window) ? n_ctx - window : 0;   /* oldest visible position */
        const uint16_t *qv = q + (size_t)item * head_dim;
        double *s = (double *)malloc(sizeof(double) * (size_t)n_ctx);
        double m = -INFINITY;
        for (int i = first; i < n_ctx; ++i) {
            double acc = 0.0;
            for (int c = 0; c < head_dim; ++c)
                acc += bf16_to_f64(qv[c]) *
                       bf16_to_f64(k_pages[kv_index(page_table, max_pages, page_size, n_kv_heads, head_dim, b, i, g, c)]);
            s[i] = scale * acc;
            if (s[i] > m) m = s[i];
        }
        double l = 0.0;
        for (int i = first; i < n_ctx; ++i) l += exp(s[i] - m);
        double *o = out + (size_t)item * head_dim;
        for (int c = 0; c < head_dim; ++c) o[c] = 0.0;
        for (int i = first; i < n_ctx; ++i) {
            double w = exp(s[i] - m) / l;
            for (int c = 0; c < head_dim; ++c)
                o[c] += w * bf16_to_f64(v_pages[kv_index(page_table, max_pages, page_size, n_kv_heads, head_dim, b, i, g, c)]);
        }
        if (lse) lse[item] = m + log(l);
        free(s);
    }
}

/*
 * Target logits over the vocabulary for every block row (Sec. 2.1: the target
 * computes p(. | X_{1:t+i-1}) for i = 1 .. gamma+1):  z[m,v] = sum_k hidden[m,k] * W[v,k].
 *   hidden : bf16 [M,K];  W : bf16 [V,K];  z : f64 [M,V]
 */
void oracle_logits(int M, int K, int V, const uint16_t *hidden, const uint16_t *W, double *z)
{
#pragma omp parallel for schedule(static)
    for (int v = 0; v < V; ++v)
        for (int m = 0; m < M; ++m) {
            double acc = 0.0;
            for (int k = 0; k < K; ++k)
                acc += bf16_to_f64(hidden[(size_t)m * K + k]) * bf16_to_f64(W[(size_t)v * K + k]);
            z[(size_t)m * V + v] = acc;
        }
}

/* p[m,:] = softmax(z[m,:] / T), T > 0 (sampling temperature, Sec. 4 "Inference Settings"). */
void oracle_softmax(int M, int V, double T, const double *z, double *p)
{
#pragma omp parallel for schedule(static)
    for (int m = 0; m < M; ++m) {
        const double *zr = z + (size_t)m * V;
        double *pr = p + (size_t)m * V;
        double mx = -INFINITY;
        for (int v = 0; v < V; ++v)
            if (zr[v] / T > mx) mx = zr[v] / T;
        double sum = 0.0;
        for (int v = 0; v < V; ++v) sum += exp(zr[v] / T - mx);
        for (int v = 0; v < V; ++v) pr[v] = exp(zr[v] / T - mx) / sum;
    }
}

/* Lowest index attaining the maximum; *gap receives (largest - second largest). */
static int argmax_lowest(const double *x, int V, double *gap)
{
    int best = 0;
    for (int v = 1; v < V; ++v)
        if (x[v] > x[best]) best = v;
    if (gap) {
        double second = -INFINITY;
        for (int v = 0; v < V; ++v)
            if (v != best && x[v] > second) second = x[v];
        *gap = x[best] - second;
    }
    return best;
}

/*
 * Inverse-CDF draw from the unnormalised non-negative masses r[0..V) with the
 * uniform u in [0,1): the first index whose running sum exceeds u * total.
 * Zero-mass entries are never returned; if rounding leaves u * total at or
 * above the full sum the last positive entry is taken.  *margin receives the
 * distance from u to the nearer normalised CDF edge of the chosen entry.
 */
static int sample_inverse_cdf(const double *r, int V, double u, double *margin)
{
    double total = 0.0;
    for (int v = 0; v < V; ++v) total += r[v];
    double target = u * total, cum = 0.0;
    int tok = -1;
    double lo = 0.0, hi = 0.0;
    for (int v = 0; v < V; ++v) {
        double prev = cum;
        cum += r[v];
        if (r[v] > 0.0 && cum > target) { tok = v; lo = prev; hi = cum; break; }
    }
    if (tok < 0)
        for (int v = V - 1; v >= 0; --v)
            if (r[v] > 0.0) { tok = v; lo = total - r[v]; hi = total; break; }
    if (margin) {
        double a = u - lo / total, b = hi / total - u;
        if (tok == V - 1 || hi >= total) b = 1.0;   /* no entry follows: only the lower edge can flip */
        if (lo <= 0.0) a = 1.0;                     /* nothing precedes: only the upper edge can flip */
        *margin = a < b ? a : b;
    }
    return tok;
}

/*
 * Sequential acceptance of the gamma drafted tokens of each sequence and the
 * extra token (Sec. 2.1).
 *
 * T > 0  (p = softmax(z/T) passed in `p`, q in `draft_probs`):
 *   draft j (token x = draft_tokens[b,j]) is accepted with probability
 *   min(1, p_j(x)/q_j(x)); with the supplied uniform this is the division-free
 *   test  u_accept[b,j] * q_j(x) < p_j(x), with the product and the comparison
 *   in double.  At the first rejection n the extra token
 *   is drawn from norm(max(p_n - q_n, 0)); if all gamma are accepted (n =
 *   gamma) it is drawn from p_gamma, the (gamma+1)-th distribution the target
 *   computed.  The draw uses u_sample[b,n].  If the residual has no mass
 *   (p == q on the row) the draw falls back to p_n.
 * T == 0 (logits passed in `z`, `p` and `draft_probs` unused):
 *   draft j is accepted iff x = argmax_v z_j[v] (lowest index on ties); the
 *   extra token is argmax_v z_n[v].
 *
 * Outputs: out_tokens[b, 0..n-1] = accepted drafts, out_tokens[b,n] = extra
 * token, rest -1; accept_len[b] = n + 1 (tokens gained by this target pass,
 * the quantity whose mean is the paper's tau).
 * Diagnostics: margin_accept[b,j] = |u - min(1,p/q)| (T>0) or top-1/top-2
 * logit gap of row j (T=0) for every examined row j <= n (else -1);
 * margin_sample[b] = CDF-edge distance of the drawn token (T>0) or the logit
 * gap of row n (T=0).
 */
void oracle_accept(int B, int gamma, int V, double T, const double *z, const double *p,
                   const int32_t *draft_tokens, const float *draft_probs,
                   const float *u_accept, const float *u_sample,
                   int32_t *out_tokens, int32_t *accept_len, double *margin_accept, double *margin_sample)
{
    int R = gamma + 1;
#pragma omp parallel for schedule(dynamic, 1)
    for (int b = 0; b < B; ++b) {
        int n = gamma;
        for (int j = 0; j < R; ++j) out_tokens[(size_t)b * R + j] = -1;
        for (int j = 0; j < gamma; ++j) margin_accept[(size_t)b * gamma + j] = -1.0;
        if (T > 0.0) {
            for (int j = 0; j < gamma; ++j) {
                int x = draft_tokens[(size_t)b * gamma + j];
                double pj = p[((size_t)b * R + j) * V + x];
                float qj = draft_probs[((size_t)b * gamma + j) * V + x];
                float u = u_accept[(size_t)b * gamma + j];
                double ratio = qj > 0.0f ? pj / (double)qj : (pj > 0.0 ? INFINITY : 0.0);
                double thr = ratio < 1.0 ? ratio : 1.0;
                margin_accept[(size_t)b * gamma + j] = fabs((double)u - thr);
                int ok = (double)u * (double)qj < pj;
                if (!ok) { n = j; break; }
                out_tokens[(size_t)b * R + j] = x;
            }
            const double *pn = p + ((size_t)b * R + n) * V;
            double *r = (double *)malloc(sizeof(double) * (size_t)V);
            double mass = 0.0;
            if (n < gamma) {
                const float *qn = draft_probs + ((size_t)b * gamma + n) * V;
                for (int v = 0; v < V; ++v) {
                    double d = pn[v] - (double)qn[v];
                    r[v] = d > 0.0 ? d : 0.0;
                    mass += r[v];
                }
            }
            if (n == gamma || !(mass > 0.0))
                for (int v = 0; v < V; ++v) r[v] = pn[v];
            out_tokens[(size_t)b * R + n] = sample_inverse_cdf(r, V, (double)u_sample[(size_t)b * R + n],
                                                              &margin_sample[b]);
            free(r);
        } else {
            double gap = 0.0;
            for (int j = 0; j < gamma; ++j) {
                int x = draft_tokens[(size_t)b * gamma + j];
                int top = argmax_lowest(z + ((size_t)b * R + j) * V, V, &gap);
                margin_accept[(size_t)b * gamma + j] = gap;
                if (x != top) { n = j; break; }
                out_tokens[(size_t)b * R + j] = x;
            }
            out_tokens[(size_t)b * R + n] = argmax_lowest(z + ((size_t)b * R + n) * V, V, &gap);
            margin_sample[b] = gap;
        }
        accept_len[b] = n + 1;
    }
}

/*
 * Commit: the n accepted drafts and the extra token join the sequence, so the
 * committed length grows by accept_len; cache rows beyond it are dead.
 * Rollback (accept_len == NULL) leaves the lengths untouched, which discards
 * the whole appended block.
 */
void oracle_kv_commit(int B, const int32_t *accept_len, int32_t *seq_lens)
{
    if (!accept_len) return;
    for (int b = 0; b < B; ++b) seq_lens[b] += accept_len[b];
}

/* Total variation distance between two distributions over V entries (Eq. 6). */
double oracle_tvd(int V, const double *p, const double *q)
{
    double s = 0.0;
    for (int v = 0; v < V; ++v) s += fabs(p[v] - q[v]);
    return 0.5 * s;
}

/*
 * Histogram of total variation distances (Fig. 4 plots the TVDs of Eq. 6 as a histogram): counts[k] +=
 * the number of values in bin k of `bins` equal-width bins over [0, 1] -- bin k is [k / bins, (k+1) / bins),
 * the last bin also takes 1.  The paper fixes neither the bin count nor the edges' arithmetic: the bin
 * index is floor(t * bins) with the product rounded once to single precision (the type the distances
 * are stored in), clamped to [0, bins - 1]; NaN values are not counted.  Returns the number counted.
 */
long long oracle_tvd_histogram(long long n, const float *tvd, int bins, long long *counts)
{
    long long counted = 0;
    for (long long i = 0; i < n; ++i) {
        const float t = tvd[i];
        if (t != t) continue;
        const float scaled = t * (float)bins;
        int k = scaled <= 0.0f ? 0 : (scaled >= (float)bins ? bins - 1 : (int)scaled);
        if (k > bins - 1) k = bins - 1;
        counts[k] += 1;
        ++counted;
    }
    return counted;
}

/*
 * Nucleus (top-p) sampling of softmax(z / T) (Sec. 3.2: the target's responses for self-distillation are
 * drawn as sample_top-p(p(. | I, X)); the same rule is the drafter's sampling step when it uses top-p).
 * Per row: order the tokens by probability, largest first (equal probabilities: lower index first); the
 * nucleus is the shortest prefix of that order whose mass reaches top_p (the whole vocabulary if rounding
 * keeps the total below top_p); q = p restricted to the nucleus and renormalised; the token is the inverse
 * CDF of q in vocabulary order at u (first index whose running mass exceeds u * total; zero-mass tokens
 * are never returned; if rounding pushes the target past the end, the last nucleus token).
 *   z [rows, V] fp32 logits, u [rows] in [0, 1)
 *   token [rows], q_out [rows, V] (may be NULL), nucleus_size [rows],
 *   margin_set [rows]   : distance of top_p from the nearer of the two prefix masses that decide where the
 *                         prefix stops (the mass before and after its last token),
 *   margin_sample [rows]: distance of u from the nearer edge of the drawn token's CDF interval.
 */
typedef struct { double p; int v; } oracle_pv;
static int oracle_pv_cmp(const void *a, const void *b)
{
    const oracle_pv *x = (const oracle_pv *)a, *y = (const oracle_pv *)b;
    if (x->p > y->p) return -1;
    if (x->p < y->p) return 1;
    return (x->v > y->v) - (x->v < y->v);
}
void oracle_sample_top_p(int rows, int V, double T, double top_p, const float *z, const float *u,
                         int32_t *token, double *q_out, int32_t *nucleus_size, double *margin_set,
                         double *margin_sample)
{
#pragma omp parallel for schedule(dynamic, 1)
    for (int r = 0; r < rows; ++r) {
        const float *zr = z + (size_t)r * V;
        oracle_pv *pv = (oracle_pv *)malloc((size_t)V * sizeof(oracle_pv));
        char *in = (char *)calloc((size_t)V, 1);
        double m = -INFINITY, s = 0.0;
        for (int v = 0; v < V; ++v) if ((double)zr[v] > m) m = (double)zr[v];
        for (int v = 0; v < V; ++v) s += exp(((double)zr[v] - m) / T);
        for (int v = 0; v < V; ++v) { pv[v].p = exp(((double)zr[v] - m) / T) / s; pv[v].v = v; }
        qsort(pv, (size_t)V, sizeof(oracle_pv), oracle_pv_cmp);
        double cum = 0.0, before = 0.0;
        int k = 0;
        while (k < V) {                       /* shortest prefix with mass >= top_p */
            before = cum;
            cum += pv[k].p;
            in[pv[k].v] = 1;
            ++k;
            if (cum >= top_p) break;
        }
        nucleus_size[r] = k;
        margin_set[r] = fmin(fabs(top_p - before), fabs(cum - top_p));
        /* restrict, renormalise (in vocabulary order), draw */
        double total = 0.0;
        for (int v = 0; v < V; ++v) if (in[v]) total += exp(((double)zr[v] - m) / T) / s;
        const double target = (double)u[r] * total;
        double run = 0.0, lo_edge = 0.0, hi_edge = 0.0;
        int tok = -1, last = -1;
        for (int v = 0; v < V; ++v) {
            const double pr = in[v] ? exp(((double)zr[v] - m) / T) / s : 0.0;
            if (q_out) q_out[(size_t)r * V + v] = pr / total;
            if (pr > 0.0) {
                last = v;
                if (tok < 0 && run + pr > target) { tok = v; lo_edge = run; hi_edge = run + pr; }
            }
            run += pr;
        }
        if (tok < 0) { tok = last; lo_edge = hi_edge = total; }
        token[r] = tok;
        margin_sample[r] = fmin(fabs((double)u[r] - lo_edge / total), fabs(hi_edge / total - (double)u[r]));
        free(pv);
        free(in);
    }
}

int oracle_num_threads(void)
{
#ifdef _OPENMP
    extern int omp_get_max_threads(void);
    return omp_get_max_threads();
#else
    return 1;
#endif
}
