/*
 * cfgzip.h - C ABI of the CFGzip decode-step library for NVIDIA B200 (sm_100a).
 *
 * The library implements the inference-time wrapper of CFGzip (paper Section 3.1,
 * "Inference", and Figure 1): a grammar engine that works over K equivalence-class
 * representatives hands over an allow-mask over the classes; the mask is expanded to
 * the full token vocabulary through the token->class vector c, applied to the
 * language model's logits, the next token is chosen, and the chosen token is mapped
 * to the representative r_{c_t} of its class for the engine's next step.
 *
 * Conventions shared by every call
 *   - Bit masks are packed 32-bit words, least-significant bit first: bit j of word w
 *     stands for index 32*w + j; 1 = allowed. KW = ceil(K/32), VW = ceil(V/32).
 *     Class-mask bits at index >= K are ignored. Vocab-mask bits at index >= V inside
 *     word VW-1 are written as 0; words at index >= VW of a row are never touched.
 *   - "dev" pointers are device memory of the context's GPU, "host" pointers are host
 *     memory. The caller owns every buffer it passes; the library owns only the
 *     partition tables and a small scratch area inside the context.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).
 *     Per-step calls only enqueue work on `stream`: they never synchronise, never
 *     allocate, and may be captured into a CUDA graph. Calls that share one context
 *     share its scratch area, so they must be ordered on one stream (use one context
 *     per concurrent stream).
 *   - Every function returns CFGZIP_OK (0) or a negative error code. Argument errors
 *     are detected on the host before anything is launched. Data errors that only the
 *     GPU can see (a token id outside [0, V), a row with no allowed class, a row whose
 *     partition id is not loaded) give a defined output and bump a sticky counter that
 *     cfgzip_poll_status reads; they never trap.
 */
#ifndef CFGZIP_H
#define CFGZIP_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct cfgzip_ctx cfgzip_ctx; /* opaque: device tables, scratch, sticky status */
typedef int32_t cfgzip_part_id;       /* small dense id inside one context */

enum { CFGZIP_F32 = 0, CFGZIP_BF16 = 1 };                   /* logit element type */
enum { CFGZIP_AUTO = 0, CFGZIP_DENSE = 1, CFGZIP_SPARSE = 2 }; /* expansion strategy */
enum {
    CFGZIP_OK = 0,
    CFGZIP_E_ARG = -1,       /* null pointer, negative size, stride too small, unknown enum */
    CFGZIP_E_RANGE = -2,     /* partition id not loaded, V mismatch, size beyond a limit */
    CFGZIP_E_PARTITION = -3, /* c / r do not describe a partition (see cfgzip_check_partition) */
    CFGZIP_E_ALIGN = -4,     /* reserved; unaligned logits are handled by a slower path */
    CFGZIP_E_CUDA = -5,      /* a CUDA runtime call failed (no device, launch error) */
    CFGZIP_E_NOMEM = -6      /* device allocation failed, or B exceeds the reserved rows */
};

/* Human-readable name of a status code; never NULL. */
const char* cfgzip_status_string(int status);

/*
 * Create a context on CUDA device `device`. Allocates the scratch area (a few MB)
 * and row-plan buffers for up to 16384 rows per call (see cfgzip_reserve_rows).
 * Fails with CFGZIP_E_CUDA when no usable device exists: there is no CPU fallback.
 */
int cfgzip_create(int device, cfgzip_ctx** out);
/* Free every partition and the context. Synchronises the device. */
int cfgzip_destroy(cfgzip_ctx* ctx);
/* Grow the per-call row capacity (allocates; call outside the per-step path). */
int cfgzip_reserve_rows(cfgzip_ctx* ctx, int32_t max_rows);

/*
 * Host-only check that (c, r) is a partition as Section 3.1 ("Pre-Computation")
 * defines the two vectors: c[i] in [0, K) for every token, every class non-empty,
 * r[k] in [0, V) and c[r[k]] == k. Returns CFGZIP_OK or CFGZIP_E_PARTITION /
 * CFGZIP_E_ARG. Touches no GPU.
 */
int cfgzip_check_partition(const int32_t* token_to_class /*host [V]*/, int32_t V,
                           const int32_t* class_to_rep /*host [K]*/, int32_t K);

/*
 * Host-only inverse of c: off[k]..off[k+1] delimits, inside tok, the tokens of class
 * k in ascending id (the class->token lists the sparse path scatters from).
 * `off` has K+1 entries, `tok` has V. Touches no GPU.
 */
int cfgzip_build_class_lists(const int32_t* token_to_class /*host [V]*/, int32_t V, int32_t K,
                             int32_t* off /*host [K+1]*/, int32_t* tok /*host [V]*/);

/*
 * Load one tokenizer/grammar partition (Section 3.1: vectors c and r, "cached" once per
 * tokenizer/CFG pair). Validates as cfgzip_check_partition does, builds the class->token
 * lists, copies everything to the device on `stream` and waits for the copy. Returns the
 * new id in *out_id. Not a per-step call.
 */
int cfgzip_load_partition(cfgzip_ctx* ctx, const int32_t* token_to_class /*host [V]*/, int32_t V,
                          const int32_t* class_to_rep /*host [K]*/, int32_t K, void* stream,
                          cfgzip_part_id* out_id);
/* Release a partition's device tables (synchronises the device first). */
int cfgzip_free_partition(cfgzip_ctx* ctx, cfgzip_part_id id);

/*
 * Row -> partition: `row_part` is NULL (every row uses `part0`) or a dev int32 [B] of
 * partition ids; all partitions used in one call must have the same V (K may differ;
 * class_stride_words must cover the largest KW). Rows whose id is not a loaded
 * partition of that V are skipped (outputs untouched) and counted as bad rows.
 */

/*
 * Batches whose rows keep their partitions over many decode steps (one grammar per request: Section 4 runs
 * one CFG per schema on the JSON task) need not be regrouped at every step. cfgzip_plan_rows groups the rows
 * of `row_part` (dev int32 [B]) by partition once, on `stream`; afterwards a per-step call on the same context
 * may pass CFGZIP_ROWS_AS_PLANNED in place of row_part (with the same B, and a part0 of the same V) and skips its
 * grouping launch. The caller keeps `row_part` alive and unchanged meanwhile. The kept grouping does not survive
 * a per-step call that passes an explicit row_part (assume it gone after any such call), another
 * cfgzip_plan_rows, cfgzip_reserve_rows, or loading or freeing a partition; CFGZIP_ROWS_AS_PLANNED without a
 * valid kept grouping gives CFGZIP_E_ARG. B above the reserved
 * rows gives CFGZIP_E_NOMEM (see cfgzip_reserve_rows).
 */
#define CFGZIP_ROWS_AS_PLANNED ((const int32_t*)(uintptr_t)1)
int cfgzip_plan_rows(cfgzip_ctx* ctx, cfgzip_part_id part0, const int32_t* row_part /*dev [B]*/, int32_t B,
                     void* stream);

/*
 * Expand class masks to vocab masks: vocab bit (b, i) = class bit (b, c[i])
 * (Section 3.1, "Inference": the mask entry applied to token i is m_{c_i}; Figure 1b).
 *   class_mask : dev uint32 [B, class_stride_words], class_stride_words >= KW
 *   vocab_mask : dev uint32 [B, vocab_stride_words], vocab_stride_words >= VW (written)
 *   mode       : CFGZIP_DENSE gathers through c; CFGZIP_SPARSE clears the row and
 *                scatters the members of each allowed class; CFGZIP_AUTO = dense here (the
 *                fused step below is where the automatic mode chooses).
 */
int cfgzip_expand_mask(cfgzip_ctx* ctx, cfgzip_part_id part0, const int32_t* row_part,
                       const uint32_t* class_mask, int64_t class_stride_words, uint32_t* vocab_mask,
                       int64_t vocab_stride_words, int32_t B, int mode, void* stream);

/*
 * Apply a vocab mask to logits in place: a disallowed logit becomes -inf, an allowed
 * one keeps its bits (Section 2.2 defines the masking so; Section 3.1 applies it
 * after the gather).
 *   logits : dev [B, row_stride_elems] of `dtype`, row_stride_elems >= V; elements at
 *            index >= V of a row are not touched. 16-byte aligned rows take the
 *            vectorised path, anything else a scalar one.
 */
int cfgzip_mask_logits(cfgzip_ctx* ctx, void* logits, int dtype, int64_t row_stride_elems, int32_t B,
                       int32_t V, const uint32_t* vocab_mask, int64_t vocab_stride_words, void* stream);

/*
 * The whole step in one pass over the logits (Section 3.1, "Inference"): expand the
 * class mask, mask the logits in place, take the greedy choice and the log-softmax
 * normaliser over the allowed tokens, and map the choice to its representative.
 *   argmax      : dev int32 [B]; largest allowed logit, ties to the lowest token id,
 *                 compared as values (-0.0 == +0.0); -1 when nothing is allowed
 *   rep         : nullable dev int32 [B]; r[c[argmax]] or -1
 *   lse         : nullable dev float [B]; log sum_{allowed} exp(z_i), fp32 accumulate
 *   logp_argmax : nullable dev float [B]; z_argmax - lse
 *   logp_full   : nullable dev float [B, V] (row stride V); z_i - lse, -inf where masked
 *   vocab_mask  : nullable; as in cfgzip_expand_mask
 *   mode        : CFGZIP_DENSE streams every row through the gather; CFGZIP_SPARSE builds each row's vocab
 *                 mask from the class->token lists of its allowed classes and never reads a logit that
 *                 is not allowed. CFGZIP_AUTO: the class-list kernel pays off when under 4 % (f32) or 1 %
 *                 (bf16) of the tokens are allowed, the measured break-even. Callers whose class masks are
 *                 still in host memory, where the grammar engine leaves them, get that choice for free
 *                 from cfgzip_choose_mode (cfgzip_decode_step_host with CFGZIP_AUTO uses it). On device
 *                 masks the choice needs one more launch (the class-list kernel runs first, adds up the
 *                 sizes of the classes the 8 rows of a row batch allow and finishes the batches below the
 *                 break-even; the gather kernel behind it streams the others), which costs 6 to 16 % on a
 *                 batch that turns out dense: so CFGZIP_AUTO means CFGZIP_DENSE here unless the caller
 *                 opts in (tuning knob "auto_min_mbytes"). The results do not depend on the mode.
 * A row with no allowed token, or whose allowed logits are all -inf, gets lse =
 * logp_argmax = -inf (the latter still returns the lowest allowed id). +inf and NaN
 * logits are outside the contract for the reductions (the masking itself still copies
 * them bit for bit); logits below -1.7e38 count as -inf in the normaliser.
 */
int cfgzip_masked_logsoftmax_argmax(cfgzip_ctx* ctx, cfgzip_part_id part0, const int32_t* row_part,
                                    const uint32_t* class_mask, int64_t class_stride_words, void* logits,
                                    int dtype, int64_t row_stride_elems, int32_t B, uint32_t* vocab_mask,
                                    int64_t vocab_stride_words, int32_t* argmax, int32_t* rep,
                                    float* logp_argmax, float* lse, float* logp_full, int mode,
                                    void* stream);

/*
 * The same pass with the token SAMPLED instead of taken greedily (Section 3.1, "Inference": a
 * token is drawn from the next-token distribution; Section 4: temperature 0.2 in the paper's
 * runs). The paper names no sampler; this one is the inverse CDF in token-id order:
 *   p_i   = exp(z_i / T) / sum_{allowed j} exp(z_j / T),  1/T = inv_temperature > 0 (at most 1e6)
 *   token = the lowest token id i with sum_{j <= i} p_j > u[b]
 * with ONE uniform number per row supplied by the caller (the library draws no random numbers).
 *   u          : dev float [B], values in [0, 1)
 *   token      : dev int32 [B]; -1 when nothing is allowed
 *   rep        : nullable dev int32 [B]; r[c[token]] or -1
 *   lse        : nullable dev float [B]; log sum_{allowed} exp(z_i / T)
 *   logp_token : nullable dev float [B]; z_token / T - lse
 *   logits, vocab_mask, class masks, row_part: as in cfgzip_masked_logsoftmax_argmax; the logits
 *                are masked in place and NOT scaled by 1/T
 *   mode       : CFGZIP_AUTO or CFGZIP_DENSE (CFGZIP_SPARSE gives CFGZIP_E_ARG)
 * The sums are accumulated in fp32 in a fixed order, so the result is deterministic; where u lies
 * within rounding (about 1e-6) of a boundary of the exact CDF the neighbouring token may come out.
 * A row whose allowed logits are all -inf yields the lowest allowed id with lse = logp_token = -inf.
 */
int cfgzip_masked_sample(cfgzip_ctx* ctx, cfgzip_part_id part0, const int32_t* row_part,
                         const uint32_t* class_mask, int64_t class_stride_words, void* logits, int dtype,
                         int64_t row_stride_elems, int32_t B, uint32_t* vocab_mask,
                         int64_t vocab_stride_words, const float* u, float inv_temperature, int32_t* token,
                         int32_t* rep, float* logp_token, float* lse, int mode, void* stream);

/*
 * cfgzip_masked_sample with the draw restricted to the most probable allowed tokens (the paper names no sampler,
 * Section 3.1 / Section 4; these are the two customary filters, applied to the masked, tempered distribution):
 *   order : the allowed tokens by logit, largest first; equal logits by token id, lowest first
 *   top_k : > 0 keeps the first min(top_k, allowed) tokens of that order; 0 keeps all
 *   top_p : in (0, 1) then keeps the shortest beginning of what top_k kept whose weight, sum of exp(z_i / T),
 *           reaches top_p times the weight of all that top_k kept (at least one token); >= 1 keeps all
 * The token is drawn among the kept tokens by inverse CDF in token-id order with u[b]; lse and logp_token are those
 * of the distribution renormalised over the kept tokens. top_k = 0 and top_p >= 1 give cfgzip_masked_sample.
 * Weights are summed as 40-bit fixed-point integers, so the result is deterministic; where top_p times the weight
 * lies within rounding (about 1e-6 of the weight) of a cumulative weight of the order, the kept set may end one
 * token earlier or later than in exact arithmetic. top_k < 0 or top_p <= 0 give CFGZIP_E_ARG.
 */
int cfgzip_masked_sample_filtered(cfgzip_ctx* ctx, cfgzip_part_id part0, const int32_t* row_part,
                                  const uint32_t* class_mask, int64_t class_stride_words, void* logits, int dtype,
                                  int64_t row_stride_elems, int32_t B, uint32_t* vocab_mask,
                                  int64_t vocab_stride_words, const float* u, float inv_temperature, int32_t top_k,
                                  float top_p, int32_t* token, int32_t* rep, float* logp_token, float* lse, int mode,
                                  void* stream);

/*
 * Several class masks against ONE logits row (tree or speculative decoding: the same next-token distribution is
 * needed under the grammar states of several candidate continuations). The masking of Section 3.1 ("Inference":
 * mask entry m_{c_i} per token i) is applied once per mask, the logits themselves are read once and NOT modified.
 * Row (b, j) below stands for logits row b under its j-th mask, stored at index b * masks_per_row + j:
 *   class_masks : dev uint32 [B * masks_per_row, class_stride_words]
 *   logits      : dev [B, row_stride_elems] of `dtype`, rows 16-byte aligned (CFGZIP_E_ALIGN otherwise); read only
 *   vocab_masks : nullable dev uint32 [B * masks_per_row, vocab_stride_words]
 *   argmax, rep, logp_argmax, lse : dev [B * masks_per_row] (rep, logp_argmax, lse nullable), each as in
 *                 cfgzip_masked_logsoftmax_argmax for the row masked by that one mask
 * One partition (part0) for the whole call. B * masks_per_row above the reserved rows gives CFGZIP_E_NOMEM;
 * partitions with more than 65535 classes give CFGZIP_E_RANGE.
 */
int cfgzip_multi_mask_logsoftmax_argmax(cfgzip_ctx* ctx, cfgzip_part_id part0, const uint32_t* class_masks,
                                        int64_t class_stride_words, int32_t masks_per_row, const void* logits,
                                        int dtype, int64_t row_stride_elems, int32_t B, uint32_t* vocab_masks,
                                        int64_t vocab_stride_words, int32_t* argmax, int32_t* rep,
                                        float* logp_argmax, float* lse, void* stream);

/*
 * Token -> representative of its class, reps[b] = r[c[tokens[b]]] (Section 3.1,
 * "Inference": the engine is fed r_{c_i} instead of t^(i); Figure 1a). A token id
 * outside [0, V) gives -1 and counts as a bad token.
 */
int cfgzip_map_tokens(cfgzip_ctx* ctx, cfgzip_part_id part0, const int32_t* row_part,
                      const int32_t* tokens /*dev [B]*/, int32_t* reps /*dev [B]*/, int32_t B,
                      void* stream);

/*
 * Host-only choice between CFGZIP_DENSE and CFGZIP_SPARSE for a batch whose class masks are still in host memory,
 * which is where the grammar engine leaves them (Section 3.1, "Inference": the engine produces the mask over the
 * classes; Section 4 runs it on the CPU). Adds up the sizes of the classes every row allows and returns
 * CFGZIP_SPARSE when under 4 % (f32) or 1 % (bf16) of the batch's tokens are allowed (the measured break-even of the
 * two kernels; tuning knob "auto_sparse_permille"), else CFGZIP_DENSE; a negative status on bad arguments. The count
 * stops as soon as the batch is known to be dense. Touches no GPU and launches nothing. row_part_host: NULL or host int32 [B].
 */
int cfgzip_choose_mode(cfgzip_ctx* ctx, cfgzip_part_id part0, const int32_t* row_part_host,
                       const uint32_t* class_mask_host /*host [B, class_stride_words]*/, int64_t class_stride_words,
                       int32_t B, int dtype);

/*
 * The same step for callers whose data lives on the host: copies the class masks and
 * logits (pinned or pageable host memory) to staging buffers owned by the context,
 * runs cfgzip_masked_logsoftmax_argmax, copies the requested results back and waits
 * for `stream`. Staging buffers grow on first use (that call allocates).
 *   logits_host     : host [B, V] of `dtype`, dense rows; left unmodified
 *   masked_logits   : nullable host [B, V]; receives the masked logits
 *   vocab_mask_host : nullable host uint32 [B, VW]
 *   argmax/rep/lse/logp_argmax : nullable host [B]
 *   mode            : CFGZIP_AUTO chooses with cfgzip_choose_mode from the host masks (no extra launch)
 */
int cfgzip_decode_step_host(cfgzip_ctx* ctx, cfgzip_part_id part0, const int32_t* row_part_host,
                            const uint32_t* class_mask_host, int64_t class_stride_words,
                            const void* logits_host, int dtype, int32_t B, void* masked_logits,
                            uint32_t* vocab_mask_host, int32_t* argmax, int32_t* rep, float* logp_argmax,
                            float* lse, int mode, void* stream);

/*
 * Synchronise `stream`, then return and clear the sticky counters: rows that had no
 * allowed token, token ids out of range in cfgzip_map_tokens, rows skipped for a bad
 * partition id. Any output pointer may be NULL. Returns CFGZIP_E_CUDA if a kernel reported
 * that one of its asynchronous copies never completed (its bounded wait ran out); the
 * results of that call are then undefined.
 */
int cfgzip_poll_status(cfgzip_ctx* ctx, void* stream, int32_t* n_empty_rows, int32_t* n_bad_tokens,
                       int32_t* n_bad_rows);

/*
 * The fused step for callers that are not allowed to allocate device memory. (The paper has
 * no counterpart for this call; it exists for integration reasons only.)
 *
 * Everything above needs a context, and creating one or loading a partition calls
 * cudaMalloc. Some hosts of this library cannot do that at the point where they need the
 * step: a plugin that runs inside another runtime's memory pool and must not grow the
 * process's device footprint behind its back, code running inside a region where the CUDA
 * allocator is off limits, or a job whose memory budget was fixed at start-up. This entry
 * point takes no context and calls no allocating routine. The token->class and
 * class->representative vectors are DEVICE arrays the caller already holds, and the only
 * memory the call uses beyond its arguments is a fixed scratch array compiled into the
 * library (about 1 MiB; every GPU that loads the library carries a copy until the process
 * exits).
 *
 *   token_to_class : dev int32 [V]; an id outside [0, K) makes that token disallowed
 *   class_to_rep   : dev int32 [K]
 *   other arguments and all results as in cfgzip_masked_logsoftmax_argmax (no logp_full, no
 *   row partitions, no sticky counters; rows may have any alignment)
 *
 * Limits and rules
 *   - B <= 1024 rows per call; more gives CFGZIP_E_RANGE and nothing is launched.
 *   - It runs on the CURRENT device of the calling thread. The first call on each device asks
 *     the runtime for the address of that device's copy of the scratch array; make that first
 *     call outside any stream capture.
 *   - All calls on one GPU share the scratch array, whatever their stream. It is not cleared
 *     between calls except for the per-row tickets, which every call zeroes on `stream` before
 *     its kernel. Two calls that can overlap on the GPU (different streams, no dependency)
 *     race on it and give wrong results: order them.
 *   - It is slower than the context-based call (one token per thread, no shared-memory
 *     tables); use it where allocation is impossible, not as the default.
 */
int cfgzip_step_noalloc(const int32_t* token_to_class /*dev [V]*/, int32_t V,
                        const int32_t* class_to_rep /*dev [K]*/, int32_t K, const uint32_t* class_mask,
                        int64_t class_stride_words, void* logits, int dtype, int64_t row_stride_elems,
                        int32_t B, uint32_t* vocab_mask, int64_t vocab_stride_words, int32_t* argmax,
                        int32_t* rep, float* logp_argmax, float* lse, void* stream);

/*
 * Measurement aid (the paper has no counterpart): one launch that reads every whole 16-byte vector of
 * logits [B, row_stride_elems] (first V elements of each row), flips the sign bit of each element and
 * writes it back in place. It is the cheapest pass over the bytes a fused step must read and write;
 * timing it in the same launch protocol as the step gives the floor the step's time is compared with.
 * Calling it twice restores the buffer. Rows must be 16-byte aligned (CFGZIP_E_ALIGN otherwise).
 */
int cfgzip_rmw_floor(cfgzip_ctx* ctx, void* logits, int dtype, int64_t row_stride_elems, int32_t B, int32_t V,
                     void* stream);

/*
 * ---- Offline step (Section 3.1 "Pre-Computation", Section 3.2, Appendix C): from a grammar and a vocabulary to
 * the vectors c and r that cfgzip_load_partition takes. Done once per tokenizer / grammar pair.
 *
 * A grammar in Greibach normal form (Section 2.1): production i is  prod_head[i] -> prod_terminal[i] beta_i  with
 * beta_i = prod_rhs[prod_rhs_off[i] .. prod_rhs_off[i+1]) a possibly empty sequence of non-terminals 0 ..
 * n_nonterminals-1 (host arrays, copied). The production S -> epsilon, if the grammar has one, is left out: it
 * consumes no character and plays no part below. cfgzip_grammar_create also computes the stack-adjacency relation
 * of Appendix C (graph over the non-terminals, breadth-first search from the non-terminal in front of each
 * non-terminal Z of a right-hand side to the non-terminals that have a production pushing nothing).
 * CFGZIP_E_RANGE: a symbol outside [0, n_nonterminals).
 */
typedef struct cfgzip_grammar cfgzip_grammar;
int cfgzip_grammar_create(int32_t n_nonterminals, int32_t start, const int32_t* prod_head, const uint8_t* prod_terminal,
                          const int32_t* prod_rhs_off /*host [n_prod + 1]*/, const int32_t* prod_rhs, int32_t n_prod,
                          cfgzip_grammar** out);
int cfgzip_grammar_destroy(cfgzip_grammar* g);
/* adjacency[y * n_nonterminals + z] = 1 when z may be popped right after y was popped by a production that pushes
 * nothing (Appendix C); host uint8 [n_nonterminals^2]. */
int cfgzip_grammar_adjacency(const cfgzip_grammar* g, uint8_t* adjacency);

/*
 * Displacement of every token (Algorithm 1 with the stack backtrack restricted by the adjacency relation: the
 * symbol guessed for the input stack must be adjacent to the symbol popped last; no restriction for the first
 * symbol), written as one signature row per token: row[0] = n, then n integers: the (input stack, output stack)
 * pairs in lexicographic order, each as  len(sigma_i), sigma_i.., len(sigma_o), sigma_o..  (stacks top first), then
 * zeros up to row_words. Two tokens have equal displacement exactly when their rows are equal.
 *   token_bytes / token_off : host; token i is bytes [token_off[i], token_off[i+1])
 *   signatures              : host int32 [V, row_words] (written)
 *   signature_words         : nullable host int32 [V]; the n of each token (-1: more than max_pairs pairs)
 * Returns CFGZIP_E_RANGE when some token needs more than row_words - 1 integers or more than max_pairs pairs (the
 * rows of the other tokens are still written; the offending rows are zero). Host only, touches no GPU.
 */
int cfgzip_displacement_signatures(const cfgzip_grammar* g, const uint8_t* token_bytes, const int64_t* token_off,
                                   int32_t V, int32_t row_words, int32_t* signatures, int32_t* signature_words,
                                   int64_t max_pairs);

/*
 * Grouping on the GPU (Section 3.1, "Pre-Computation": tokens with equal displacement form a class, the byte-wise
 * shortest member represents it, c maps tokens to classes and r classes to representatives). Rows are compared
 * word for word (a hash only picks where to look first), so the grouping is exact.
 *   signatures     : dev int32 [V, row_words]          token_len : dev int32 [V], byte length of each token
 *   token_to_class : dev int32 [V] (written): classes numbered in the order of their lowest token id
 *   class_to_rep   : dev int32 [V] (first *n_classes entries written): shortest member, lowest id among the shortest
 *   n_classes      : dev int32 [1]
 *   class_off / class_tok : both NULL, or dev int32 [V + 1] / [V]: the class -> token lists in ascending token id
 *                    (entries of class_off past n_classes read V)
 * Runs on the current device; allocates its scratch (about 50 bytes per token), synchronises `stream` before it
 * returns and frees the scratch: an offline call, not a per-step one. No context is needed.
 */
int cfgzip_group_tokens(const int32_t* signatures, int32_t row_words, const int32_t* token_len, int32_t V,
                        int32_t* token_to_class, int32_t* class_to_rep, int32_t* n_classes, int32_t* class_off,
                        int32_t* class_tok, void* stream);

/* Kernels this context has launched so far (monotonic; for launch accounting). */
int cfgzip_launch_count(cfgzip_ctx* ctx, int64_t* out);

/*
 * Tuning knobs for benchmarking; defaults are chosen from the device at create time.
 *   "ctas_per_sm"  target resident thread blocks per SM for the fused kernel (1..16)
 *   "token_warps"  0 = automatic, else warps side by side along the vocabulary (1..16)
 *   "row_warps"    0 = automatic, else 1, 2 or 4 row batches handled by separate warps
 *   "pdl"          1 = programmatic dependent launch where it pays (steps under 192 MB of logits;
 *                  default), 0 = never, 2 = always
 *   "pipeline"     1 = aligned logits stream through per-warp rings of bulk asynchronous copies
 *                  in shared memory (default), 0 = plain 16-byte loads into registers
 *   "tensor_map"   1 = a batch of 8 consecutive rows arrives as one tiled 2-D copy through a
 *                  tensor map (default), 0 = one bulk copy per row
 *   "pipe_warps"   warps per thread block of the pipelined kernel (1..16)
 *   "waves"        thread blocks launched per resident block slot of the pipelined kernel (1..16)
 *   "pipe_depth"   stages per warp of the pipelined kernel (2..8; lowered to fit shared memory); unset, long
 *                  steps take a third stage where it fits
 *   "stage_alias"  1 = always lay the class-mask staging area over the first warps' rings (default 0: only where
 *                  that keeps warps or buys the third stage)
 *   "auto_sparse_permille"  CFGZIP_AUTO: a row batch stays with the class-list kernel when under this many
 *                  thousandths of its tokens are allowed (0..1000; 0 = always dense; -1 = by element type, the default: 40 for
 *                  f32, 10 for bf16)
 *   "auto_min_mbytes"  CFGZIP_AUTO on device-resident masks: steps of at least this many megabytes of logits let the GPU
 *                  choose per batch of 8 rows, at the price of one more launch (-1 = never, the default)
 *   "fold"         0 = every warp of the streaming kernel publishes its row states and a second launch (one block or
 *                  warp per row) folds them and writes the results (default: the fastest at every size measured);
 *                  1 = the streaming kernel's last block of every row group does that itself, one launch per step;
 *                  2 = the warps of a block merge their states in shared memory before publishing, second launch kept
 *   "lane_octets"  bf16 streaming kernel: octets (8 tokens) a lane handles per row of a work item: 1 = 16 bytes,
 *                  2 = 32 bytes (chunks of 512 tokens, at most 12 warps per block), 0 = automatic (default; currently
 *                  always 1: two octets measured 2 % faster at 256 rows with 8 warps x 3 stages and slower elsewhere)
 *   "prefetch_items"  work items per warp of the streaming kernel whose logits are asked into the L2 (a hint, nothing is
 *                  read) while the kernel in front is still finishing, on programmatic launches of steps of at least
 *                  "prefetch_min_mbytes" megabytes of logits (0..64, default 4; 0 = none)
 *   "prefetch_min_mbytes"  see above (default 48: shorter steps were measured slower with the hint)
 *   "rotate"       1 (default) = the round-robin deal of a row batch's chunks to the warps of the streaming kernel
 *                  starts at another warp for every row batch, so that the warps that get one chunk more differ from
 *                  row batch to row batch; 0 = always at the first warp
 *   "test_expire_waits"  test hook, default 0: 1 makes every warp of the streaming kernel report its first wait
 *                  for an asynchronous copy as run out AFTER the wait has completed, so that the error path
 *                  (flag, bounded drain of the copies in flight, cfgzip_poll_status -> CFGZIP_E_CUDA) can be
 *                  exercised with nothing left in flight; the results of such a call are undefined
 *   "spread"       1 = launches of at most one block per SM (the streaming kernel of a small batch, the per-row
 *                  kernels of 32 to 148 rows) ask for more than half of an SM's shared memory, so that two of
 *                  their blocks never share an SM (default), 0 = only what the block needs
 * Unknown names give CFGZIP_E_ARG.
 */
int cfgzip_set_tuning(cfgzip_ctx* ctx, const char* name, int32_t value);

/*
 * Host-only: the launch shape the library would choose for a fused dense step on a device with
 * `sm_count` SMs and `smem_optin` bytes of opt-in shared memory per block (default tuning). For
 * tests of the planner; touches no GPU. out[0] kernel kind (2 pipelined, 1 register, 0 per-row),
 * [1] row groups (upper bound), [2] blocks per group S, [3] octets per block (register kernel),
 * [4] warps along tokens, [5] threads per block, [6] stages per warp, [7] dynamic shared memory
 * bytes, [8] class-table words, [9] staging stride, [10] class masks by bulk copy, [11] published
 * states per row, [12] sparse path: blocks per row (0 = per-row kernel), [13] sparse path: mask
 * words per block, [14] capacity of the state scratch, [15] blocks per SM the launch is sized for.
 */
int cfgzip_plan_query(int32_t sm_count, int32_t smem_optin, int32_t V, int32_t K, int32_t B, int dtype,
                      int32_t n_partitions, int32_t aligned_class_masks, int32_t out[16]);

#ifdef __cplusplus
}
#endif
#endif /* CFGZIP_H */
