/*
 * CPU oracle for the CFGzip per-decode-step wrapper path.
 *
 * TEST INFRASTRUCTURE ONLY. This file is the slow, element-by-element
 * statement of what the path computes, written from the paper's Section 3.1
 * ("Pre-Computation" and "Inference" paragraphs) and Section 2.2. It shares
 * no code, header, table or helper with the CUDA library and is never called
 * from the product path. Floating-point reductions are carried in double.
 *
 * Conventions (where the paper is silent, the reading taken is stated):
 *   - c[i]  : class id of token i, 0 <= c[i] < K      (Section 3.1, vector c)
 *   - r[k]  : token id representing class k            (Section 3.1, vector r)
 *   - masks are packed 32-bit words, bit j of word w <-> index 32*w + j,
 *     1 = allowed. Class-mask bits >= K are ignored; vocab-mask bits >= V
 *     inside the last word are written 0.
 *   - the paper's "z_i <- z_i * m_{c_i}" with m in {-inf, 1} is read as a
 *     select: a disallowed logit becomes -inf (Section 2.2 says exactly
 *     that), an allowed logit keeps its bits.
 *   - the token choice is greedy: largest allowed value, ties to the lowest
 *     token id, comparison on values (so -0.0 == +0.0).
 *   - a row with nothing allowed yields argmax = rep = -1 and -inf log
 *     quantities; a row whose allowed logits are all -inf yields the lowest
 *     allowed token id and -inf log quantities.
 *   - sampling (Section 3.1 draws the token from the next-token
 *     distribution, Section 4 fixes the temperature, neither names the
 *     sampler): p_i = exp(z_i/T) / sum_{allowed j} exp(z_j/T); the uniform
 *     number u in [0,1) is an input; the chosen token is the lowest id whose
 *     cumulative probability, taken in token-id order, exceeds u.
 *
 * Parity pins: every function here is pinned by tests/test_oracle_pins.py
 * (closed forms, invariants, a library log-softmax, brute force, hand-worked
 * examples); nothing in this file is "parity unpinned".
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

enum { ORACLE_F32 = 0, ORACLE_BF16 = 1 };

/* bfloat16 -> float is exact: the 16 bits are the top half of the float. */
static float bf16_to_float(uint16_t h) {
    uint32_t u = (uint32_t)h << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return f;
}

static float load_logit(const void* z, int dtype, int64_t idx) {
    if (dtype == ORACLE_BF16) return bf16_to_float(((const uint16_t*)z)[idx]);
    return ((const float*)z)[idx];
}

static void store_neg_inf(void* z, int dtype, int64_t idx) {
    if (dtype == ORACLE_BF16) {
        ((uint16_t*)z)[idx] = 0xFF80u;
    } else {
        uint32_t u = 0xFF800000u;
        memcpy((float*)z + idx, &u, sizeof u);
    }
}

static int get_bit(const uint32_t* words, int64_t i) { return (int)((words[i >> 5] >> (i & 31)) & 1u); }

/*
 * Gather-expansion of the class mask into a token mask (Section 3.1,
 * "Inference": the mask entry used for token i is m_{c_i}).
 * vocab_mask row b receives ceil(V/32) words.
 */
void oracle_expand_mask(const int32_t* c, int32_t V, int32_t K, const uint32_t* class_mask,
                        int64_t class_stride_words, uint32_t* vocab_mask, int64_t vocab_stride_words,
                        int32_t B) {
    (void)K;
    int32_t VW = (V + 31) / 32;
    for (int32_t b = 0; b < B; ++b) {
        const uint32_t* m = class_mask + (int64_t)b * class_stride_words;
        uint32_t* v = vocab_mask + (int64_t)b * vocab_stride_words;
        for (int32_t w = 0; w < VW; ++w) v[w] = 0u;
        for (int32_t i = 0; i < V; ++i) {
            int allowed = get_bit(m, c[i]);
            v[i >> 5] |= (uint32_t)allowed << (i & 31);
        }
    }
}

/*
 * Inverse of c: for class k, tok[off[k] .. off[k+1]) lists its tokens in
 * ascending token id. Follows from the definition of c (Section 3.1).
 */
void oracle_build_csr(const int32_t* c, int32_t V, int32_t K, int32_t* off, int32_t* tok) {
    for (int32_t k = 0; k <= K; ++k) off[k] = 0;
    for (int32_t i = 0; i < V; ++i) off[c[i] + 1] += 1;
    for (int32_t k = 0; k < K; ++k) off[k + 1] += off[k];
    /* visiting tokens in ascending id keeps every class list ascending */
    int32_t* next = (int32_t*)malloc((size_t)K * sizeof(int32_t));
    for (int32_t k = 0; k < K; ++k) next[k] = off[k];
    for (int32_t i = 0; i < V; ++i) tok[next[c[i]]++] = i;
    free(next);
}

/*
 * The same token mask reached from the class side: clear the row, then for
 * every allowed class set the bit of each of its members.
 */
void oracle_expand_mask_csr(const int32_t* off, const int32_t* tok, int32_t V, int32_t K,
                            const uint32_t* class_mask, int64_t class_stride_words, uint32_t* vocab_mask,
                            int64_t vocab_stride_words, int32_t B) {
    int32_t VW = (V + 31) / 32;
    for (int32_t b = 0; b < B; ++b) {
        const uint32_t* m = class_mask + (int64_t)b * class_stride_words;
        uint32_t* v = vocab_mask + (int64_t)b * vocab_stride_words;
        for (int32_t w = 0; w < VW; ++w) v[w] = 0u;
        for (int32_t k = 0; k < K; ++k) {
            if (!get_bit(m, k)) continue;
            for (int32_t j = off[k]; j < off[k + 1]; ++j) v[tok[j] >> 5] |= 1u << (tok[j] & 31);
        }
    }
}

/*
 * Logit masking (Section 2.2: the logit of a disallowed token is set to
 * -inf; Section 3.1 applies it through the token mask). In place; elements
 * at index >= V of a row are not touched.
 */
void oracle_mask_logits(void* logits, int dtype, int64_t row_stride_elems, int32_t B, int32_t V,
                        const uint32_t* vocab_mask, int64_t vocab_stride_words) {
    for (int32_t b = 0; b < B; ++b) {
        const uint32_t* v = vocab_mask + (int64_t)b * vocab_stride_words;
        for (int32_t i = 0; i < V; ++i)
            if (!get_bit(v, i)) store_neg_inf(logits, dtype, (int64_t)b * row_stride_elems + i);
    }
}

/*
 * Greedy choice and log-softmax renormalised over the allowed set, from
 * logits that are already masked. lse = log sum_{allowed} exp(z_i);
 * logp_i = z_i - lse; logp_argmax = z_best - lse = -log sum exp(z_i - z_best).
 * logp_full (nullable) is [B, V] doubles with row stride V.
 */
void oracle_logsoftmax_argmax(const void* logits, int dtype, int64_t row_stride_elems, int32_t B, int32_t V,
                              const uint32_t* vocab_mask, int64_t vocab_stride_words, int32_t* argmax,
                              double* lse, double* logp_argmax, double* logp_full) {
    for (int32_t b = 0; b < B; ++b) {
        const uint32_t* v = vocab_mask + (int64_t)b * vocab_stride_words;
        int64_t base = (int64_t)b * row_stride_elems;
        int32_t best = -1;
        for (int32_t i = 0; i < V; ++i) {
            if (!get_bit(v, i)) continue;
            if (best < 0 || load_logit(logits, dtype, base + i) > load_logit(logits, dtype, base + best)) best = i;
        }
        argmax[b] = best;
        double M = best < 0 ? -INFINITY : (double)load_logit(logits, dtype, base + best);
        double S = 0.0;
        if (best >= 0 && M > -INFINITY)
            for (int32_t i = 0; i < V; ++i)
                if (get_bit(v, i)) S += exp((double)load_logit(logits, dtype, base + i) - M);
        int finite = best >= 0 && M > -INFINITY;
        lse[b] = finite ? M + log(S) : -INFINITY;
        logp_argmax[b] = finite ? -log(S) : -INFINITY;
        if (logp_full) {
            for (int32_t i = 0; i < V; ++i) {
                double lp = -INFINITY;
                if (finite && get_bit(v, i)) lp = (double)load_logit(logits, dtype, base + i) - lse[b];
                logp_full[(int64_t)b * V + i] = lp;
            }
        }
    }
}

/*
 * Token -> representative of its class, r_{c_t} (Section 3.1, "Inference";
 * Figure 1a). A token id outside [0, V) maps to -1.
 */
void oracle_map_tokens(const int32_t* c, const int32_t* r, int32_t V, int32_t K, const int32_t* tokens,
                       int32_t* reps, int32_t B) {
    (void)K;
    for (int32_t b = 0; b < B; ++b) {
        int32_t t = tokens[b];
        reps[b] = (t >= 0 && t < V) ? r[c[t]] : -1;
    }
}

/*
 * One whole decode step for rows that share one partition: the four steps
 * above in the order the paper gives them (expand, mask, choose/normalise,
 * map to representative). vocab_mask must hold B rows of ceil(V/32) words.
 */
void oracle_decode_step(const int32_t* c, const int32_t* r, int32_t V, int32_t K, const uint32_t* class_mask,
                        int64_t class_stride_words, void* logits, int dtype, int64_t row_stride_elems,
                        int32_t B, uint32_t* vocab_mask, int64_t vocab_stride_words, int32_t* argmax,
                        int32_t* rep, double* lse, double* logp_argmax, double* logp_full) {
    oracle_expand_mask(c, V, K, class_mask, class_stride_words, vocab_mask, vocab_stride_words, B);
    oracle_mask_logits(logits, dtype, row_stride_elems, B, V, vocab_mask, vocab_stride_words);
    oracle_logsoftmax_argmax(logits, dtype, row_stride_elems, B, V, vocab_mask, vocab_stride_words, argmax, lse,
                             logp_argmax, logp_full);
    oracle_map_tokens(c, r, V, K, argmax, rep, B);
}

/*
 * Sampling from the tempered distribution over the allowed tokens (Section 3.1,
 * "Inference": the next token is a draw from the model's distribution; Section 4:
 * temperature T, 0.2 in the paper's runs), from logits that are already masked.
 *   p_i      = exp(z_i / T) / sum_{allowed j} exp(z_j / T)          (0 where masked)
 *   token    = min { i : sum_{j <= i} p_j > u },  u in [0,1) given per row
 *              (if rounding leaves no such i, the last token with p_i > 0)
 *   lse      = log sum_{allowed} exp(z_i / T)
 *   logp_tok = z_token / T - lse
 * cdf (nullable, [B, V] doubles, row stride V) receives sum_{j <= i} p_j so that a test can
 * see how close u lies to a boundary. Degenerate rows as for the greedy choice: nothing
 * allowed -> token -1; all allowed logits -inf -> lowest allowed id; both with -inf logs.
 */
void oracle_sample(const void* logits, int dtype, int64_t row_stride_elems, int32_t B, int32_t V,
                   const uint32_t* vocab_mask, int64_t vocab_stride_words, double inv_temperature,
                   const double* u, int32_t* token, double* lse, double* logp_token, double* cdf) {
    for (int32_t b = 0; b < B; ++b) {
        const uint32_t* v = vocab_mask + (int64_t)b * vocab_stride_words;
        int64_t base = (int64_t)b * row_stride_elems;
        int32_t first = -1;
        double M = -INFINITY;
        for (int32_t i = 0; i < V; ++i) {
            if (!get_bit(v, i)) continue;
            if (first < 0) first = i;
            double z = (double)load_logit(logits, dtype, base + i);
            if (z > M) M = z;
        }
        int finite = first >= 0 && M > -INFINITY;
        double S = 0.0;
        if (finite)
            for (int32_t i = 0; i < V; ++i)
                if (get_bit(v, i)) S += exp(((double)load_logit(logits, dtype, base + i) - M) * inv_temperature);
        int32_t pick = finite ? -1 : first, last_pos = -1;
        double run = 0.0;
        for (int32_t i = 0; i < V; ++i) {
            double w = 0.0;
            if (finite && get_bit(v, i)) w = exp(((double)load_logit(logits, dtype, base + i) - M) * inv_temperature);
            run += w;
            if (w > 0.0) last_pos = i;
            if (finite && pick < 0 && run > u[b] * S) pick = i;
            if (cdf) cdf[(int64_t)b * V + i] = finite ? run / S : 0.0;
        }
        if (finite && pick < 0) pick = last_pos;
        token[b] = pick;
        lse[b] = finite ? M * inv_temperature + log(S) : -INFINITY;
        logp_token[b] = finite ? ((double)load_logit(logits, dtype, base + pick) - M) * inv_temperature - log(S) : -INFINITY;
    }
}

/*
 * One whole sampling step for rows that share one partition: expand, mask, sample, map the
 * sampled token to its representative (the order of Section 3.1, "Inference").
 */
void oracle_sample_step(const int32_t* c, const int32_t* r, int32_t V, int32_t K, const uint32_t* class_mask,
                        int64_t class_stride_words, void* logits, int dtype, int64_t row_stride_elems, int32_t B,
                        uint32_t* vocab_mask, int64_t vocab_stride_words, double inv_temperature, const double* u,
                        int32_t* token, int32_t* rep, double* lse, double* logp_token, double* cdf) {
    oracle_expand_mask(c, V, K, class_mask, class_stride_words, vocab_mask, vocab_stride_words, B);
    oracle_mask_logits(logits, dtype, row_stride_elems, B, V, vocab_mask, vocab_stride_words);
    oracle_sample(logits, dtype, row_stride_elems, B, V, vocab_mask, vocab_stride_words, inv_temperature, u, token, lse,
                  logp_token, cdf);
    oracle_map_tokens(c, r, V, K, token, rep, B);
}

/*
 * Several class masks against one logits row (tree or speculative decoding: one next-token
 * distribution, several grammar states). Not in the paper as such: it is the decode step of
 * Section 3.1 ("Inference") taken once per mask on a private copy of the row, so the caller's
 * logits stay as they are. Entry (b, j) of every output sits at index b * masks_per_row + j;
 * class_masks and vocab_masks hold one row per (b, j) in that order.
 */
void oracle_multi_mask_step(const int32_t* c, const int32_t* r, int32_t V, int32_t K, const uint32_t* class_masks,
                            int64_t class_stride_words, int32_t masks_per_row, const void* logits, int dtype,
                            int64_t row_stride_elems, int32_t B, uint32_t* vocab_masks, int64_t vocab_stride_words,
                            int32_t* argmax, int32_t* rep, double* lse, double* logp_argmax) {
    size_t elem = dtype == ORACLE_BF16 ? 2 : 4;
    void* row = malloc((size_t)V * elem);
    for (int32_t b = 0; b < B; ++b) {
        for (int32_t j = 0; j < masks_per_row; ++j) {
            int64_t e = (int64_t)b * masks_per_row + j;
            memcpy(row, (const char*)logits + (size_t)b * (size_t)row_stride_elems * elem, (size_t)V * elem);
            oracle_decode_step(c, r, V, K, class_masks + e * class_stride_words, class_stride_words, row, dtype, V, 1,
                               vocab_masks + e * vocab_stride_words, vocab_stride_words, argmax + e, rep + e, lse + e,
                               logp_argmax + e, NULL);
        }
    }
    free(row);
}

/*
 * Sampling restricted to the most probable tokens (top-k, top-p) of the tempered distribution over the allowed
 * tokens. The paper only says that the token is sampled (Section 3.1, "Inference") at a temperature (Section 4);
 * the two filters are the customary ones, read as follows on logits that are already masked:
 *   order    : the allowed tokens by value, largest first, equal values by token id, lowest first;
 *   top_k    : > 0 keeps the first min(top_k, allowed) tokens of that order, 0 keeps all;
 *   top_p    : < 1 then keeps the shortest beginning of what top_k kept whose weight sum_{kept} exp((z_i - M) / T)
 *              reaches top_p times the weight of all that top_k kept (at least one token); >= 1 keeps all;
 *   sampling : among the kept tokens F as in oracle_sample, inverse CDF in token-id order with u:
 *              p_i = exp(z_i / T) / sum_{F} exp(z_j / T), token = min { i in F : sum_{j in F, j <= i} p_j > u };
 *   lse      = log sum_{F} exp(z_i / T),   logp_tok = z_token / T - lse.
 * n_kept receives |F|; kept (nullable, [B, V] bytes) the membership of F; p_margin (nullable) how far, as a
 * fraction of the weight top_k kept, the top_p target lies from the nearer of the two cumulative weights around
 * the cut, leaving out a side on which the cut cannot move (+inf when top_p keeps all): a test can tell from it
 * whether rounding may move the cut.
 * Degenerate rows as in oracle_sample (nothing allowed: -1; allowed logits all -inf: the lowest allowed id).
 */
typedef struct { float z; int32_t id; } oracle_entry;

static int oracle_entry_before(const void* a, const void* b) {
    const oracle_entry* x = (const oracle_entry*)a;
    const oracle_entry* y = (const oracle_entry*)b;
    if (x->z > y->z) return -1;
    if (x->z < y->z) return 1;
    return (x->id > y->id) - (x->id < y->id);
}

void oracle_sample_filtered(const void* logits, int dtype, int64_t row_stride_elems, int32_t B, int32_t V,
                            const uint32_t* vocab_mask, int64_t vocab_stride_words, double inv_temperature,
                            int32_t top_k, double top_p, const double* u, int32_t* token, double* lse,
                            double* logp_token, int32_t* n_kept, double* p_margin, uint8_t* kept) {
    oracle_entry* order = (oracle_entry*)malloc((size_t)(V > 0 ? V : 1) * sizeof(oracle_entry));
    uint8_t* in_f = (uint8_t*)malloc((size_t)(V > 0 ? V : 1));
    for (int32_t b = 0; b < B; ++b) {
        const uint32_t* v = vocab_mask + (int64_t)b * vocab_stride_words;
        int64_t base = (int64_t)b * row_stride_elems;
        int32_t n = 0;
        for (int32_t i = 0; i < V; ++i) {
            in_f[i] = 0;
            if (get_bit(v, i)) {
                order[n].z = load_logit(logits, dtype, base + i);
                order[n].id = i;
                ++n;
            }
        }
        qsort(order, (size_t)n, sizeof(oracle_entry), oracle_entry_before);
        double M = n > 0 ? (double)order[0].z : -INFINITY;
        int finite = n > 0 && M > -INFINITY;
        int32_t keep = n;
        if (top_k > 0 && top_k < keep) keep = top_k;
        double margin = INFINITY;
        if (finite && top_p < 1.0) {
            double Sk = 0.0;
            for (int32_t j = 0; j < keep; ++j) Sk += exp(((double)order[j].z - M) * inv_temperature);
            double target = top_p * Sk, run = 0.0;
            int32_t cut = keep;
            for (int32_t j = 0; j < keep; ++j) {
                double before = run;
                run += exp(((double)order[j].z - M) * inv_temperature);
                if (run >= target) {
                    cut = j + 1;
                    /* the cut cannot move before the first token nor behind the last one top_k kept */
                    margin = INFINITY;
                    if (j > 0) margin = fmin(margin, (target - before) / Sk);
                    if (j + 1 < keep) margin = fmin(margin, (run - target) / Sk);
                    break;
                }
            }
            keep = cut;
        }
        for (int32_t j = 0; j < keep; ++j) in_f[order[j].id] = 1;
        double S = 0.0;
        if (finite)
            for (int32_t i = 0; i < V; ++i)
                if (in_f[i]) S += exp(((double)load_logit(logits, dtype, base + i) - M) * inv_temperature);
        int32_t pick = -1, last_pos = -1, first = n > 0 ? V : -1;
        for (int32_t j = 0; j < n; ++j)
            if (order[j].id < first) first = order[j].id;
        if (!finite) pick = first;
        double run = 0.0;
        for (int32_t i = 0; i < V && finite; ++i) {
            if (!in_f[i]) continue;
            double w = exp(((double)load_logit(logits, dtype, base + i) - M) * inv_temperature);
            run += w;
            if (w > 0.0) last_pos = i;
            if (pick < 0 && run > u[b] * S) pick = i;
        }
        if (finite && pick < 0) pick = last_pos;
        token[b] = pick;
        lse[b] = finite ? M * inv_temperature + log(S) : -INFINITY;
        logp_token[b] = finite ? ((double)load_logit(logits, dtype, base + pick) - M) * inv_temperature - log(S) : -INFINITY;
        if (n_kept) n_kept[b] = keep;
        if (p_margin) p_margin[b] = margin;
        if (kept) memcpy(kept + (size_t)b * (size_t)V, in_f, (size_t)V);
    }
    free(order);
    free(in_f);
}
