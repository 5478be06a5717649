/*
 * CPU oracle for the decode-step hot path -- TEST INFRASTRUCTURE, NOT PRODUCT CODE.
 *
 * Plain, slow, fp64 definitions of what the CUDA library must compute.  Nothing
 * here is shared with the CUDA path (no common headers, helpers or tables), and
 * nothing in the product may call into this file: only the tests, the smoke
 * check and the benchmark's CPU-baseline leg do.
 *
 * What is defined (the paper names the operations but prints no formula for
 * them -- "decode phase" with an active batch, Section 2.1; verification of
 * draft tokens by the target model in the lossless formulation, Section 3.4 --
 * so each function below is the textbook definition written out):
 *
 *   ora_paged_attention  masked scaled-dot-product attention of q_len query
 *                        rows per sequence over that sequence's keys, which
 *                        live in a paged pool addressed through a block table
 *                        (Section 2.1 decode step; Section 3.4 verify step with
 *                        q_len = 1 + gamma and a causal mask inside the draft
 *                        block).  Two passes over a stored score array; no
 *                        chunking, no running rescale.
 *   ora_lse_merge        combination of attention results computed over
 *                        disjoint key subsets, through their log-sum-exp.
 *   ora_accept_greedy    temperature-0 case of lossless draft verification
 *                        (Section 3.4): per-row lowest-index argmax over the
 *                        vocabulary, then the longest draft prefix that agrees
 *                        with it, plus one token from the target.
 *   ora_accept_sample    the same verification under the paper's sampling
 *                        regime (temperature, top-k, top-p; Appendix, Table
 *                        "shared-sampling-config") with point-proposal drafts.
 *
 *   ora_rope             rotary position embedding of the step's query and key
 *                        rows ("rotate-half" pairing, the form the Qwen models
 *                        the paper evaluates use; the paper itself prints no
 *                        formula for it): the step before attention.
 *
 * All bf16 inputs are uint16 bit patterns, decoded exactly to double.
 * Pins for every function live in tests/test_oracle_*.py (brute force on
 * unpaged tensors written independently in NumPy, closed forms, invariants).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

static double bf16_to_double(uint16_t b)
{
    uint32_t u = ((uint32_t)b) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

/* Address of the D-vector of key/value token j of sequence s, kv head g. */
static const uint16_t *kv_row(const uint16_t *pool, const int32_t *block_table, int64_t max_pages,
                              int s, int64_t j, int g, int P, int64_t page_stride,
                              int64_t token_stride, int64_t head_stride)
{
    int64_t logical = j / P;
    int64_t page = block_table[(int64_t)s * max_pages + logical];
    return pool + page * page_stride + (j % P) * token_stride + (int64_t)g * head_stride;
}

/*
 * out : double [B, q_len, Hq, D]      lse : double [B, q_len, Hq] (may be NULL)
 * key_begin / key_end : optional int32 [B]; when given, only keys j with
 *   key_begin[s] <= j < key_end[s] take part (used to build split partials).
 * Query row t of sequence s sits at absolute position n_s - q_len + t and sees
 * keys 0..that position.  An empty key set yields O = 0 and LSE = -inf.
 * Returns 0, or -1 on allocation failure / bad arguments.
 */
int ora_paged_attention(const uint16_t *q, const uint16_t *k_pool, const uint16_t *v_pool,
                        const int32_t *block_table, const int32_t *kv_lens,
                        const int32_t *key_begin, const int32_t *key_end,
                        int B, int q_len, int Hq, int Hkv, int D, int P, int max_pages,
                        int64_t page_stride, int64_t token_stride, int64_t head_stride,
                        double scale, double *out, double *lse, int nthreads)
{
    if (Hkv <= 0 || Hq % Hkv != 0 || D <= 0 || P <= 0 || q_len <= 0) return -1;
    const int G = Hq / Hkv;
    int failed = 0;
#ifdef _OPENMP
    if (nthreads > 0) omp_set_num_threads(nthreads);
#else
    (void)nthreads;
#endif
#pragma omp parallel for collapse(2) schedule(dynamic, 1)
    for (int s = 0; s < B; ++s) {
        for (int h = 0; h < Hq; ++h) {
            const int g = h / G;
            const int64_t n = kv_lens[s];
            double *x = (double *)malloc(sizeof(double) * (size_t)(n > 0 ? n : 1));
            if (!x) {
#pragma omp atomic write
                failed = 1;
                continue;
            }
            for (int t = 0; t < q_len; ++t) {
                const uint16_t *qrow = q + (((int64_t)s * q_len + t) * Hq + h) * D;
                double *orow = out + (((int64_t)s * q_len + t) * Hq + h) * D;
                const int64_t pos = n - q_len + t;          /* last visible key */
                int64_t j0 = 0, j1 = pos + 1;               /* visible keys: [j0, j1) */
                if (key_begin && key_begin[s] > j0) j0 = key_begin[s];
                if (key_end && key_end[s] < j1) j1 = key_end[s];
                for (int d = 0; d < D; ++d) orow[d] = 0.0;
                if (j1 <= j0) {
                    if (lse) lse[((int64_t)s * q_len + t) * Hq + h] = -INFINITY;
                    continue;
                }
                /* pass 1: scores and their maximum */
                double m = -INFINITY;
                for (int64_t j = j0; j < j1; ++j) {
                    const uint16_t *k = kv_row(k_pool, block_table, max_pages, s, j, g, P,
                                               page_stride, token_stride, head_stride);
                    double acc = 0.0;
                    for (int d = 0; d < D; ++d) acc += bf16_to_double(qrow[d]) * bf16_to_double(k[d]);
                    x[j] = scale * acc;
                    if (x[j] > m) m = x[j];
                }
                /* pass 2: weights, normaliser, weighted sum of values */
                double l = 0.0;
                for (int64_t j = j0; j < j1; ++j) {
                    const double w = exp(x[j] - m);
                    l += w;
                    const uint16_t *v = kv_row(v_pool, block_table, max_pages, s, j, g, P,
                                               page_stride, token_stride, head_stride);
                    for (int d = 0; d < D; ++d) orow[d] += w * bf16_to_double(v[d]);
                }
                for (int d = 0; d < D; ++d) orow[d] /= l;
                if (lse) lse[((int64_t)s * q_len + t) * Hq + h] = m + log(l);
            }
            free(x);
        }
    }
    return failed ? -1 : 0;
}

/*
 * partial_o   : double [B, max_splits, R, D]   (each already normalised by its own l)
 * partial_lse : double [B, max_splits, R]      (natural log; -inf marks an empty part)
 * num_splits  : int32  [B]
 * out         : double [B, R, D]               R = q_len * Hq rows per sequence
 * O = sum_i w_i O_i / sum_i w_i with w_i = exp(LSE_i - max_i LSE_i); all parts
 * empty -> zeros.  out_lse (optional) = max + log(sum w).
 */
int ora_lse_merge(const double *partial_o, const double *partial_lse, const int32_t *num_splits,
                  int B, int max_splits, int R, int D, double *out, double *out_lse)
{
    for (int s = 0; s < B; ++s) {
        const int S = num_splits[s];
        if (S < 0 || S > max_splits) return -1;
        for (int r = 0; r < R; ++r) {
            double *o = out + ((int64_t)s * R + r) * D;
            for (int d = 0; d < D; ++d) o[d] = 0.0;
            double M = -INFINITY;
            for (int i = 0; i < S; ++i) {
                double v = partial_lse[((int64_t)s * max_splits + i) * R + r];
                if (v > M) M = v;
            }
            if (M == -INFINITY) {
                if (out_lse) out_lse[(int64_t)s * R + r] = -INFINITY;
                continue;
            }
            double W = 0.0;
            for (int i = 0; i < S; ++i) {
                double v = partial_lse[((int64_t)s * max_splits + i) * R + r];
                if (v == -INFINITY) continue;
                const double w = exp(v - M);
                W += w;
                const double *po = partial_o + (((int64_t)s * max_splits + i) * R + r) * D;
                for (int d = 0; d < D; ++d) o[d] += w * po[d];
            }
            for (int d = 0; d < D; ++d) o[d] /= W;
            if (out_lse) out_lse[(int64_t)s * R + r] = M + log(W);
        }
    }
    return 0;
}

/*
 * logits : bf16 bits, row (b, i) starts at logits + (b*(gamma+1)+i)*row_stride, V entries
 * draft  : int32 [B, gamma]
 * target_argmax : int32 [B, gamma+1]   lowest index attaining the row maximum
 *                 (numeric comparison, so +0 and -0 tie)
 * accept_len    : int32 [B]            largest a with draft[b,i]==target_argmax[b,i] for all i<a
 * out_tokens    : int32 [B, gamma+1]   draft[b,:a] ++ target_argmax[b,a], rest -1
 */
int ora_accept_greedy(const uint16_t *logits, int64_t row_stride, const int32_t *draft,
                      int B, int gamma, int V, int32_t *target_argmax, int32_t *accept_len,
                      int32_t *out_tokens, int nthreads)
{
    if (B < 0 || gamma < 0 || V <= 0) return -1;
    const int R = gamma + 1;
#ifdef _OPENMP
    if (nthreads > 0) omp_set_num_threads(nthreads);
#else
    (void)nthreads;
#endif
#pragma omp parallel for schedule(dynamic, 1)
    for (int r = 0; r < B * R; ++r) {
        const uint16_t *row = logits + (int64_t)r * row_stride;
        int best = 0;
        double bestv = bf16_to_double(row[0]);
        for (int v = 1; v < V; ++v) {
            const double x = bf16_to_double(row[v]);
            if (x > bestv) { bestv = x; best = v; }
        }
        target_argmax[r] = best;
    }
    for (int b = 0; b < B; ++b) {
        int a = 0;
        while (a < gamma && draft[(int64_t)b * gamma + a] == target_argmax[(int64_t)b * R + a]) ++a;
        accept_len[b] = a;
        for (int i = 0; i < R; ++i) {
            int32_t tok = -1;
            if (i < a) tok = draft[(int64_t)b * gamma + i];
            else if (i == a) tok = target_argmax[(int64_t)b * R + a];
            out_tokens[(int64_t)b * R + i] = tok;
        }
    }
    return 0;
}

int ora_max_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/*
 * Lossless acceptance of a draft block under temperature / top-k / top-p sampling -- the paper's
 * rollout sampling regime (Appendix, Table "shared-sampling-config": temperature 0.7, top-p 0.8,
 * top-k 20) combined with the speculative-sampling rule it adopts (Section 3.4, lossless
 * formulation).  The draft proposes ONE token per position (a point proposal, as greedy MTP-style
 * drafters do), i.e. the draft distribution is q = one-hot(draft token).
 *
 * For every row (b, i), i in [0, gamma]:
 *   1. candidates = the top_k largest logits; equal logits are ordered by ascending index
 *      (numeric comparison: +0 == -0); NaN logits are never candidates
 *   2. z_j = logit_j / temperature, p_j = exp(z_j - z_max) / sum over the candidates
 *   3. nucleus: keep the shortest prefix (in the order of step 1) whose probabilities sum to
 *      at least top_p (always at least one token); renormalise over the kept tokens
 * Acceptance for sequence b walks i = 0 .. gamma-1 with the uniforms u[b, i, 0] (accept) and
 * u[b, i, 1] (resample), all in [0, 1):
 *   - draft token x accepted iff x is kept and u_accept < p(x)
 *   - on rejection emit y drawn from norm(max(0, p - q)) = p restricted to the kept tokens other
 *     than x, by inverse CDF over the kept order: first j with cumulative weight > u_sample * total;
 *     stop
 *   - if all gamma drafts are accepted, emit one more token drawn from p_gamma the same way
 *     (nothing removed)
 * out_tokens = accepted drafts ++ that one token, padded with -1; accept_len = number accepted.
 *
 * The probabilities of every row are also returned (kept_ids / kept_p, top_k slots per row, -1 / 0
 * padded) so that tests can tell a wrong decision from one where u falls within rounding of p.
 *
 * Presence penalty (the same table lists 1.5): before step 1 the logit of every token that is
 * "present" for row (b, i) is lowered by the penalty, once, however often the token occurred:
 *   present(b, i) = tokens whose bit is set in seen[b] (bit v & 7 of byte v >> 3: what sequence b
 *                   has generated before this step; the caller keeps it)  union  draft[b, 0 .. i-1]
 *                   (row i is conditioned on those drafts having been accepted).
 * The subtraction is done in single precision on the decoded logit (the precision in which a
 * serving engine holds its logits when it applies penalties).  seen == NULL: nothing seen yet.
 *
 * Sampled drafts (draft_probs != NULL): the drafter drew draft[b, i] from a distribution q_{b,i}
 * over the vocabulary, given as float [B, gamma, q_row_stride >= V].  The general rule of the
 * lossless formulation then applies at position i with p the filtered target distribution above:
 *   - accept x iff u_accept * q(x) < p(x)              (i.e. with probability min(1, p(x) / q(x)))
 *   - on rejection emit y drawn from norm(max(0, p - q)): weights r_j = max(0, p_j - q(id_j)) over
 *     the kept tokens (p is zero elsewhere, so q is read at the kept tokens only), inverse CDF in
 *     the kept order over the slots with r_j > 0; if no slot has r_j > 0 (p <= q on all of p's
 *     support, where a rejection has probability zero) the token is drawn from p itself
 * A one-hot q reproduces the point-proposal rule.
 */
int ora_accept_sample(const uint16_t *logits, int64_t row_stride, const int32_t *draft,
                      const double *uniforms /* [B, gamma+1, 2] */, int B, int gamma, int V,
                      double temperature, int top_k, double top_p, int32_t *accept_len,
                      int32_t *out_tokens, int32_t *kept_ids /* [B, gamma+1, top_k] */,
                      double *kept_p /* [B, gamma+1, top_k] */, const uint8_t *seen,
                      int64_t seen_stride, double presence_penalty,
                      const float *draft_probs /* [B, gamma, q_row_stride] or NULL */, int64_t q_row_stride)
{
    if (B < 0 || gamma < 0 || V <= 0 || top_k < 1 || !(temperature > 0.0)) return -1;
    const int R = gamma + 1;
    const float pen = (float)presence_penalty;
    for (int r = 0; r < B * R; ++r) {
        const uint16_t *row = logits + (int64_t)r * row_stride;
        const int b = r / R, i = r % R;
        int32_t *ids = kept_ids + (int64_t)r * top_k;
        double *pp = kept_p + (int64_t)r * top_k;
        double val[top_k];
        int n = 0;
        /* step 1: insertion into a list sorted by (value descending, index ascending) */
        for (int v = 0; v < V; ++v) {
            double x = bf16_to_double(row[v]);
            if (pen != 0.0f) {
                int present = seen ? (seen[(int64_t)b * seen_stride + (v >> 3)] >> (v & 7)) & 1 : 0;
                for (int j = 0; j < i && !present; ++j) present = draft[(int64_t)b * gamma + j] == v;
                if (present) {
                    volatile float y = (float)x - pen;      /* one single-precision subtraction */
                    x = (double)y;
                }
            }
            if (x != x) continue;                       /* NaN */
            if (n == top_k && !(x > val[n - 1])) continue;   /* not better than the worst kept (ties lose: higher index) */
            int pos = n < top_k ? n : top_k - 1;
            while (pos > 0 && x > val[pos - 1]) { val[pos] = val[pos - 1]; ids[pos] = ids[pos - 1]; --pos; }
            val[pos] = x; ids[pos] = v;
            if (n < top_k) ++n;
        }
        /* steps 2 and 3 */
        double sum = 0.0;
        for (int j = 0; j < n; ++j) { pp[j] = exp(val[j] / temperature - val[0] / temperature); sum += pp[j]; }
        int keep = 0;
        double cum = 0.0;
        for (int j = 0; j < n; ++j) { pp[j] /= sum; }
        for (int j = 0; j < n; ++j) { cum += pp[j]; keep = j + 1; if (cum >= top_p) break; }
        double ksum = 0.0;
        for (int j = 0; j < keep; ++j) ksum += pp[j];
        for (int j = 0; j < keep; ++j) pp[j] /= ksum;
        for (int j = keep; j < top_k; ++j) { ids[j] = -1; pp[j] = 0.0; }
    }
    for (int b = 0; b < B; ++b) {
        int32_t *out = out_tokens + (int64_t)b * R;
        for (int i = 0; i < R; ++i) out[i] = -1;
        int a = 0;
        for (int i = 0; i <= gamma; ++i) {
            const int32_t *ids = kept_ids + ((int64_t)b * R + i) * top_k;
            const double *pp = kept_p + ((int64_t)b * R + i) * top_k;
            const double ua = uniforms[((int64_t)b * R + i) * 2], us = uniforms[((int64_t)b * R + i) * 2 + 1];
            int skip = -1;                 /* slot of the rejected draft token, if any */
            if (i < gamma) {
                const int32_t x = draft[(int64_t)b * gamma + i];
                double px = 0.0;
                for (int j = 0; j < top_k; ++j) if (ids[j] == x) { px = pp[j]; skip = j; }
                if (draft_probs) {
                    const float *q = draft_probs + ((int64_t)b * gamma + i) * q_row_stride;
                    const double qx = (x >= 0 && x < V) ? (double)q[x] : 0.0;
                    if (ua * qx < px) { out[i] = x; ++a; continue; }
                    /* rejected: residual max(0, p - q) over the kept tokens */
                    double r[top_k];
                    double total = 0.0;
                    for (int j = 0; j < top_k; ++j) {
                        r[j] = 0.0;
                        if (ids[j] < 0) continue;
                        const double d = pp[j] - (double)q[ids[j]];
                        if (d > 0.0) { r[j] = d; total += d; }
                    }
                    if (!(total > 0.0)) {            /* p <= q on the whole support: draw from p */
                        for (int j = 0; j < top_k; ++j) if (ids[j] >= 0 && pp[j] > 0.0) { r[j] = pp[j]; total += pp[j]; }
                    }
                    double cum = 0.0;
                    int32_t y = -1;
                    for (int j = 0; j < top_k; ++j) {
                        if (!(r[j] > 0.0)) continue;
                        cum += r[j];
                        y = ids[j];
                        if (cum > us * total) break;
                    }
                    out[i] = y;
                    break;
                }
                if (ua < px) { out[i] = x; ++a; continue; }
            }
            /* emit one token from the (residual) distribution and stop */
            double total = 0.0;
            for (int j = 0; j < top_k; ++j) if (ids[j] >= 0 && j != skip) total += pp[j];
            double cum = 0.0;
            int32_t y = -1;
            for (int j = 0; j < top_k; ++j) {
                if (ids[j] < 0 || j == skip) continue;
                cum += pp[j];
                y = ids[j];
                if (cum > us * total) break;
            }
            out[i] = y;
            break;
        }
        accept_len[b] = a;
    }
    return 0;
}

/*
 * Rotary position embedding, "rotate-half" pairing: dimension d < D/2 is paired with d + D/2,
 *   angle  = pos * inv_freq[d]                  (pos integer, inv_freq given as float, product in double)
 *   out[d]       = x[d] * cos(angle) - x[d + D/2] * sin(angle)
 *   out[d + D/2] = x[d + D/2] * cos(angle) + x[d] * sin(angle)
 * i.e. the complex number x[d] + i x[d + D/2] times exp(i angle).
 *   x    bf16 bits [rows, heads, D]      pos  int64 [rows]      inv_freq  float [D/2]
 *   out  double [rows, heads, D], not rounded
 */
int ora_rope(const uint16_t *x, const int64_t *pos, const float *inv_freq, int64_t rows, int heads, int D,
             double *out)
{
    if (!x || !pos || !inv_freq || !out || rows < 0 || heads < 1 || D < 2 || (D & 1)) return -1;
    const int half = D / 2;
    for (int64_t r = 0; r < rows; ++r)
        for (int h = 0; h < heads; ++h) {
            const uint16_t *xr = x + (r * heads + h) * (int64_t)D;
            double *o = out + (r * heads + h) * (int64_t)D;
            for (int d = 0; d < half; ++d) {
                const double angle = (double)pos[r] * (double)inv_freq[d];
                const double c = cos(angle), sn = sin(angle);
                const double a = bf16_to_double(xr[d]), b = bf16_to_double(xr[d + half]);
                o[d] = a * c - b * sn;
                o[d + half] = b * c + a * sn;
            }
        }
    return 0;
}
