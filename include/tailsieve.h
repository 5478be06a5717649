/*
 * tailsieve.h -- C ABI of the decode-step kernels that sit under bulk/tail rollout routing.
 *
 * The paper routes long ("tail") generations to a low-concurrency pool and the rest to a
 * high-concurrency ("bulk") pool, and turns on deeper speculative decoding on the tail pool
 * (Sections 2.1, 3.1, 3.4).  What every replica in either pool executes per step is one batched
 * decode step over its active requests (Section 2.1: per-request throughput v(b) as a function of
 * the active batch size b), or, with speculation, one verification of gamma draft tokens by the
 * target model followed by acceptance (Section 3.4).  This library is the attention and acceptance
 * part of that step for a ragged batch whose keys and values live in a paged cache.
 *
 * General rules (all entry points)
 *   - Every pointer argument except `const ts_attn_params*` is a DEVICE pointer owned by the
 *     caller.  The library allocates and frees no device memory, never synchronises the device,
 *     and only enqueues work on `stream` (a cudaStream_t passed as void*; NULL = default stream).
 *   - All device pointers must be 16-byte aligned.
 *   - bf16 tensors are IEEE bfloat16; arithmetic accumulates in fp32.
 *   - Return value: TS_OK or a negative ts_status.  Argument errors are detected on the host and
 *     returned before anything is enqueued.  Nothing traps on the device; a device-side wait that
 *     gives up records TS_ERR_TIMEOUT in the status word at the head of the workspace and the
 *     kernel returns.
 *   - One query length per call: every sequence of a batch scores the same number of positions
 *     (Section 3.4 explains why ragged query lengths are avoided: they break full-batch graph
 *     replay).
 *
 * Tensor conventions
 *   q        bf16 [num_seqs, q_len, num_q_heads, head_dim], contiguous
 *   out      bf16 [num_seqs, q_len, num_q_heads, head_dim], contiguous
 *   k_pool   bf16, element (page p, token j, kv head g, dim d) at
 *            p*kv_page_stride + j*kv_token_stride + g*kv_head_stride + d   (strides in elements,
 *            each a multiple of 8 so that every row starts on a 16-byte boundary)
 *   v_pool   same geometry as k_pool
 *   block_table int32 [num_seqs, max_pages_per_seq]; entry (s, i) is the physical page holding
 *            tokens i*page_size .. (i+1)*page_size-1 of sequence s.  Entries at or beyond
 *            ceil(kv_lens[s] / page_size) are never read.
 *   kv_lens  int32 [num_seqs]; number of keys of each sequence INCLUDING the q_len positions
 *            scored by this call (their K/V are already in the cache).  0 is allowed.
 *   Query head h reads kv head h / (num_q_heads / num_kv_heads).
 *   Query row t of sequence s stands at position kv_lens[s] - q_len + t and attends to keys
 *   0 .. that position (causal inside the block of new tokens; all keys when q_len == 1).
 *   A row with no visible key yields zeros (and -inf as its log-sum-exp).
 */
#ifndef TAILSIEVE_H_
#define TAILSIEVE_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum ts_status {
    TS_OK = 0,
    TS_ERR_INVALID_ARG = -1, /* null pointer, misaligned pointer, inconsistent sizes            */
    TS_ERR_UNSUPPORTED = -2, /* head_dim / page_size / group size outside the built set          */
    TS_ERR_WORKSPACE = -3,   /* workspace smaller than ts_attn_workspace_bytes() and friends     */
    TS_ERR_CUDA = -4,        /* a CUDA runtime/driver call or a launch failed                    */
    TS_ERR_TIMEOUT = -5      /* (device status word only) a bounded wait inside a kernel expired */
} ts_status;

typedef struct ts_attn_params {
    int32_t num_seqs;          /* B                                                              */
    int32_t q_len;             /* 1 for decode, 1 + gamma for speculative verification           */
    int32_t num_q_heads;       /* Hq, a multiple of num_kv_heads                                 */
    int32_t num_kv_heads;      /* Hkv                                                            */
    int32_t head_dim;          /* 64 or 128                                                      */
    int32_t page_size;         /* tokens per page: 16, 32, 64 or 128                             */
    int32_t num_pages;         /* pages in the pool (extent of the pool's outermost dimension)   */
    int32_t max_pages_per_seq; /* row stride of block_table                                      */
    int64_t kv_page_stride;    /* elements                                                       */
    int64_t kv_token_stride;   /* elements                                                       */
    int64_t kv_head_stride;    /* elements                                                       */
    float scale;               /* multiplies q.k in fp32, e.g. 1/sqrt(head_dim)                  */
} ts_attn_params;

/* Supported shapes: (num_q_heads / num_kv_heads) * q_len <= 128 at head_dim 128, <= 96 at head_dim 64. */

/*
 * Bytes of scratch that ts_decode_attn / ts_verify_attn need for `p` (depends on the head
 * geometry and q_len only, not on the sequence lengths).  Host-only; needs no GPU.  Returns 0 for
 * invalid parameters.
 */
size_t ts_attn_workspace_bytes(const ts_attn_params *p);

/* Scratch bytes for ts_decode_attn_splitkv (plan data only; the partials are caller arrays). */
size_t ts_splitkv_workspace_bytes(const ts_attn_params *p);

/*
 * Single-token decode attention for one batched decode step (Section 2.1: all active requests
 * advance by one token per step).  q_len must be 1.
 *   out = softmax(scale * q K^T) V per (sequence, query head) over that sequence's kv_lens keys.
 * The key range of long sequences is divided among thread blocks inside the call and recombined;
 * the result does not depend on how (up to fp32 rounding) and is bit-reproducible run to run.
 *   workspace: >= ts_attn_workspace_bytes(p) bytes, contents irrelevant on entry, clobbered.
 *              Its first 4 bytes are a device status word (TS_OK or TS_ERR_TIMEOUT).
 */
int ts_decode_attn(const ts_attn_params *p, const void *q, const void *k_pool, const void *v_pool,
                   const int32_t *block_table, const int32_t *kv_lens, void *out, void *workspace,
                   size_t workspace_bytes, void *stream);

/*
 * Attention for the speculative-verification step (Section 3.4: the target model scores the
 * 1 + gamma positions of each request in one pass).  Same contract as ts_decode_attn with
 * q_len = 1 + gamma >= 1 and the causal mask inside the block of new tokens described above.
 */
int ts_verify_attn(const ts_attn_params *p, const void *q, const void *k_pool, const void *v_pool,
                   const int32_t *block_table, const int32_t *kv_lens, void *out, void *workspace,
                   size_t workspace_bytes, void *stream);

/*
 * Split-KV form of decode attention for a few very long sequences (the tail pool's regime,
 * Section 3.4: a low-concurrency stream with a long horizon).  Each sequence's keys are cut into
 * num_splits[s] <= max_splits contiguous ranges, chosen on the device from kv_lens so that the
 * batch's total work spreads over all SMs; every range is attended to independently.
 *   partial_o   fp32 [num_seqs, max_splits, q_len, num_q_heads, head_dim]  each range's result,
 *               normalised by its own softmax denominator
 *   partial_lse fp32 [num_seqs, max_splits, q_len, num_q_heads]  natural-log sum-exp of the scaled
 *               scores of the range; -inf when no key of the range is visible to the row
 *   num_splits  int32 [num_seqs], written with the split counts (>= 1, also for empty sequences,
 *               whose single slot is written as zeros / -inf)
 *   workspace   >= ts_splitkv_workspace_bytes(p) bytes, clobbered; first 4 bytes = status word
 * Only slots i < num_splits[s] are written.  q_len may exceed 1 (same masking as ts_verify_attn).
 * max_splits in [1, 4096].
 */
int ts_decode_attn_splitkv(const ts_attn_params *p, const void *q, const void *k_pool,
                           const void *v_pool, const int32_t *block_table, const int32_t *kv_lens,
                           int32_t max_splits, float *partial_o, float *partial_lse,
                           int32_t *num_splits, void *workspace, size_t workspace_bytes,
                           void *stream);

/*
 * Log-sum-exp merge of split results:
 *   out[s,t,h,:] = sum_i w_i partial_o[s,i,t,h,:] / sum_i w_i,  w_i = exp(lse_i - max_i lse_i),
 * over i < num_splits[s]; parts with lse = -inf carry zero weight (their partial_o is not read
 * into the sum); if every part is empty the row is zero.  out is bf16 [num_seqs, q_len,
 * num_q_heads, head_dim].  Uses num_seqs, q_len, num_q_heads, head_dim of `p` only.
 */
int ts_lse_merge(const ts_attn_params *p, int32_t max_splits, const float *partial_o,
                 const float *partial_lse, const int32_t *num_splits, void *out, void *stream);

/*
 * Writes the K and V rows of the q_len tokens scored in this step into the paged cache, so that the
 * attention calls above find them there (the step before attention; the paper's decode step appends
 * one token per request, its verify step 1 + gamma -- Sections 2.1 and 3.4).
 *   new_k, new_v  bf16 [num_seqs, q_len, num_kv_heads, head_dim], contiguous
 *   Token t of sequence s goes to position kv_lens[s] - q_len + t (kv_lens already counts the new
 *   tokens, as in the attention calls), i.e. page block_table[s, pos / page_size], slot
 *   pos % page_size.  Positions below 0 are skipped.  Bit-exact copy; needs head_dim % 8 == 0.
 *   Uses q_len, num_kv_heads, head_dim, page_size, max_pages_per_seq and the three strides of `p`.
 */
int ts_kv_append(const ts_attn_params *p, const void *new_k, const void *new_v, void *k_pool, void *v_pool,
                 const int32_t *block_table, const int32_t *kv_lens, void *stream);

/*
 * ts_kv_append with the rotary position embedding of the step's query and key rows fused in: the
 * step before attention in the models the paper serves (Qwen3 family, Section 4.1); the paper itself
 * prints no formula for it, so the convention is fixed here.  "Rotate-half" pairing: with
 * angle = pos * inv_freq[d] for d < head_dim / 2 and pos = kv_lens[s] - q_len + t,
 *   y[d]              = x[d] * cos(angle) - x[d + head_dim/2] * sin(angle)
 *   y[d + head_dim/2] = x[d + head_dim/2] * cos(angle) + x[d] * sin(angle)
 * computed in fp32 from the bf16 inputs (the angle itself in double, reduced mod 2 pi before the
 * float sincos), rounded to bf16 (nearest even).
 *   q_in      bf16 [num_seqs, q_len, num_q_heads, head_dim]  -> rotated into q_out (same shape; q_out
 *             may be q_in: each element pair is read and written by one thread)
 *   new_k     bf16 [num_seqs, q_len, num_kv_heads, head_dim] -> rotated, written into k_pool
 *   new_v     same shape, copied bit for bit into v_pool
 *   inv_freq  float [head_dim / 2], device (a model constant, e.g. base^(-2d/head_dim))
 * Placement, skipping of negative positions, strides and alignment as in ts_kv_append;
 * head_dim % 16 == 0 and head_dim <= 256.  Errors are detected on the host before the launch.
 */
int ts_rope_kv_append(const ts_attn_params *p, const void *q_in, void *q_out, const void *new_k,
                      const void *new_v, void *k_pool, void *v_pool, const int32_t *block_table,
                      const int32_t *kv_lens, const float *inv_freq, void *stream);

/* Scratch bytes for ts_accept_greedy (host-only; 0 for invalid sizes). */
size_t ts_accept_workspace_bytes(int32_t num_seqs, int32_t gamma, int32_t vocab);

/*
 * Greedy (temperature-0) acceptance of a draft block -- the deterministic case of the lossless
 * verification rule the paper adopts (Section 3.4).
 *   logits        bf16; row (b, i), i in [0, gamma], starts at logits + (b*(gamma+1)+i)*row_stride
 *                 elements and holds `vocab` entries; row_stride >= vocab (rows need not be
 *                 16-byte aligned; the base pointer must be)
 *   draft         int32 [num_seqs, gamma]  (may be NULL when gamma == 0)
 *   target_argmax int32 [num_seqs, gamma+1]  lowest index attaining the row maximum (+0 and -0
 *                 compare equal; NaN entries never win; a row of -inf or NaN only gives 0)
 *   accept_len    int32 [num_seqs]  largest a with draft[b,i] == target_argmax[b,i] for all i < a
 *   out_tokens    int32 [num_seqs, gamma+1] = draft[b,:a] ++ target_argmax[b,a], padded with -1
 *   workspace     >= ts_accept_workspace_bytes(num_seqs, gamma, vocab) bytes, clobbered
 * gamma == 0 is plain greedy sampling of one token per sequence.
 */
int ts_accept_greedy(const void *logits, int64_t row_stride, const int32_t *draft, int32_t num_seqs,
                     int32_t gamma, int32_t vocab, int32_t *target_argmax, int32_t *accept_len,
                     int32_t *out_tokens, void *workspace, size_t workspace_bytes, void *stream);

/* Scratch bytes for ts_accept_sample (host-only; 0 for sizes it does not support). */
size_t ts_sample_workspace_bytes(int32_t num_seqs, int32_t gamma, int32_t vocab, int32_t top_k);

/*
 * Lossless acceptance of a draft block under the paper's rollout sampling regime -- temperature,
 * top-k and top-p (Appendix, Table "shared-sampling-config": 0.7 / 20 / 0.8) -- with the speculative
 * sampling rule of Section 3.4, for drafters that propose one token per position (point proposals,
 * draft distribution = one-hot).  Per logits row: the top_k largest logits (equal logits ordered by
 * ascending index, NaN never selected); p = softmax(logit / temperature) over them; the shortest
 * prefix whose probability reaches top_p is kept and renormalised.  Per sequence, with the uniforms
 * u[b, i, 0] (accept) and u[b, i, 1] (sample), i = 0 .. gamma, all in [0, 1):
 *   the draft token x_i is accepted iff it is kept and u_accept < p(x_i); at the first rejection
 *   one token is drawn from p with x_i removed (inverse CDF over the kept order, renormalised) and
 *   the walk stops; if all gamma drafts are accepted one more token is drawn from p_gamma.
 * The emitted tokens follow the target distribution exactly, whatever the drafts.
 *   logits      bf16, row (b, i) at logits + (b*(gamma+1)+i)*row_stride; row_stride and vocab
 *               multiples of 8 (16-byte aligned rows)
 *   draft       int32 [num_seqs, gamma] (may be NULL when gamma == 0)
 *   uniforms    fp32 [num_seqs, gamma+1, 2]
 *   accept_len  int32 [num_seqs]; out_tokens int32 [num_seqs, gamma+1], -1 padded
 *   workspace   >= ts_sample_workspace_bytes(...) bytes, clobbered
 * temperature > 0, 1 <= top_k <= 32, 0 < top_p <= 1, vocab <= 524288.  Token selection is exact;
 * probabilities are fp32, so a uniform within rounding of a probability may decide either way.
 * Penalties on already generated tokens: see ts_accept_sample_penalized below.
 */
int ts_accept_sample(const void *logits, int64_t row_stride, const int32_t *draft, const float *uniforms,
                     int32_t num_seqs, int32_t gamma, int32_t vocab, float temperature, int32_t top_k,
                     float top_p, int32_t *accept_len, int32_t *out_tokens, void *workspace,
                     size_t workspace_bytes, void *stream);

/*
 * ts_accept_sample with the presence penalty of the same sampling table (1.5 there): before the top-k
 * selection of row (b, i) the logit of every token that is present for that row is lowered by
 * presence_penalty, once however often the token occurred.  Present for row (b, i):
 *   the tokens whose bit is set in seen[b] (bit v & 7 of byte seen[b * seen_stride + (v >> 3)]): what
 *   sequence b has generated before this step, kept by the caller (device memory, may be NULL);
 *   and draft[b, 0 .. i-1], on whose acceptance row i is conditioned.
 * The subtraction is one fp32 operation on the decoded logit; selection stays exact on those values.
 * seen_stride (bytes per sequence) * 8 >= vocab.  presence_penalty = 0, or no bitmap and gamma = 0,
 * is ts_accept_sample exactly.  Everything else as ts_accept_sample.
 */
int ts_accept_sample_penalized(const void *logits, int64_t row_stride, const int32_t *draft,
                               const float *uniforms, int32_t num_seqs, int32_t gamma, int32_t vocab,
                               float temperature, int32_t top_k, float top_p, float presence_penalty,
                               const uint8_t *seen, int64_t seen_stride, int32_t *accept_len,
                               int32_t *out_tokens, void *workspace, size_t workspace_bytes, void *stream);

/*
 * ts_accept_sample_penalized for drafters that SAMPLE their tokens: draft[b, i] was drawn from a
 * proposal distribution q_{b,i} over the vocabulary, and the general rule of the lossless formulation
 * the paper adopts (Section 3.4) applies, with p the filtered target distribution of row (b, i):
 *   x_i is accepted iff u_accept * q(x_i) < p(x_i), i.e. with probability min(1, p(x_i) / q(x_i));
 *   at the first rejection one token is drawn from norm(max(0, p - q)) -- weights max(0, p_j - q(j))
 *   over the kept tokens j in their order, since p is zero elsewhere -- and the walk stops.  If that
 *   leaves no positive weight (p <= q on all of p's support: a rejection then has probability zero
 *   for a normalised q, but a caller may pass an unnormalised one) the token is drawn from p itself.
 *   draft_probs             fp32, q_{b,i} at draft_probs + (b*gamma+i)*draft_probs_row_stride, vocab
 *                           entries each; read at the draft token and at the at most top_k kept
 *                           tokens of the row only (no extra pass over the vocabulary); device memory
 *   draft_probs_row_stride  in elements, >= vocab
 * draft_probs == NULL is the point-proposal rule (q = one-hot at the draft token), i.e.
 * ts_accept_sample_penalized exactly; a one-hot draft_probs gives the same decisions.  A draft token
 * outside [0, vocab) is rejected.  Everything else as ts_accept_sample_penalized.
 */
int ts_accept_sample_proposal(const void *logits, int64_t row_stride, const int32_t *draft,
                              const float *draft_probs, int64_t draft_probs_row_stride, const float *uniforms,
                              int32_t num_seqs, int32_t gamma, int32_t vocab, float temperature, int32_t top_k,
                              float top_p, float presence_penalty, const uint8_t *seen, int64_t seen_stride,
                              int32_t *accept_len, int32_t *out_tokens, void *workspace, size_t workspace_bytes,
                              void *stream);

/*
 * ts_accept_greedy for callers that have no device memory to give and cannot get any.  (The paper
 * has no counterpart; this is a packaging variant of ts_accept_greedy.)  Who that is: a serving
 * process that handed all of HBM to its KV cache at start-up and kept no allocator for side
 * buffers; a plug-in invoked from inside another framework's step, where calling cudaMalloc is
 * off limits because it synchronises the whole device and may fail in an already full GPU; code
 * that must not touch the allocator after initialisation.  Same arguments, results and error
 * codes as ts_accept_greedy, minus the workspace: the chunk keys live in a 512 KB array that is
 * part of the library image on every GPU that loads it (held until the process exits).
 *   - Limit: num_seqs * (gamma + 1) <= 1024 rows; more returns TS_ERR_UNSUPPORTED and enqueues
 *     nothing.  (16 sequences at gamma = 16 are 272 rows; 1024 decode sequences are 1024.)
 *   - The call allocates nothing and frees nothing, on the host or the device.
 *   - The first call on each device looks up the array's device address (a host-side query that
 *     enqueues no work); make that first call before any stream capture is begun.
 *   - All calls on one device share the array, which keeps whatever the previous call left in it.
 *     Nothing in it has to be cleared between calls (each call overwrites every entry it later
 *     reads), but two calls whose kernels may run at the same time on one GPU -- different streams,
 *     or different host threads -- race on it and give wrong tokens: keep them on one stream or
 *     order them yourself.
 */
int ts_accept_greedy_noalloc(const void *logits, int64_t row_stride, const int32_t *draft,
                             int32_t num_seqs, int32_t gamma, int32_t vocab, int32_t *target_argmax,
                             int32_t *accept_len, int32_t *out_tokens, void *stream);

/*
 * Instrumentation for benchmarks (the paper has no counterpart).  While both events (cudaEvent_t
 * passed as void*) are non-NULL, every ts_decode_attn / ts_verify_attn / ts_decode_attn_splitkv
 * call records `start_event` on its stream right before its attention kernel (after the planner)
 * and `stop_event` right after it (before the merge).  Pass NULLs to switch it off.  Process-wide
 * and not thread-safe.  Always returns TS_OK.
 */
int ts_set_attn_timing_events(void *start_event, void *stop_event);

/* Static, human-readable name of a status code. */
const char *ts_status_string(int status);

#ifdef __cplusplus
}
#endif
#endif /* TAILSIEVE_H_ */
