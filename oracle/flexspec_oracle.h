/*
 * flexspec_oracle.h -- TEST INFRASTRUCTURE, NOT PRODUCT CODE.
 *
 * A plain, slow, fp64 CPU statement of the cloud-side verification step of
 * edge-cloud speculative decoding (Algorithm 2, "Step 2: cloud-side parallel
 * verification"; Section IV-C on the per-user KV session).  It exists so that
 * the CUDA path can be compared against something written directly from the
 * paper.  It shares no code with the CUDA path and must never be called by it:
 * only tests, the smoke check and the benchmark's CPU-baseline leg use it.
 *
 * Symbols:  p = TARGET distribution, q = DRAFT distribution (the convention of
 * the speculative-sampling rule the paper builds on; Algorithm 2 itself writes
 * the target's output as q -- that letter is not carried over).
 *
 * Row convention.  Sequence b with draft length k_b owns k_b+1 consecutive
 * query rows: row 0 is the position of the last committed token, row j>=1 the
 * position of draft token x_{j-1}.  The distribution read from row j judges
 * draft token x_j; row k_b gives the bonus distribution.
 */
#ifndef FLEXSPEC_ORACLE_H
#define FLEXSPEC_ORACLE_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* bf16 <-> fp64.  Decoding is exact; encoding rounds to nearest, ties to even,
 * in one step from the fp64 value (no intermediate fp32 rounding). */
double   fso_bf16_to_f64(uint16_t h);
uint16_t fso_f64_to_bf16(double x);

/* Philox4x32-10 (Salmon et al., SC'11): counter-based generator.  out[4]. */
void   fso_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4]);
/* Uniform in [0,1) with 24 bits: key = (lo32(seed), hi32(seed)),
 * counter = (index, stream, 0, 0), take word 0, u = (word >> 8) * 2^-24.
 * stream 0 = acceptance test of draft position `index`; stream 1 = the draw of
 * the emitted token after `index` accepted drafts. */
double fso_uniform(uint64_t seed, uint32_t index, uint32_t stream);

/* Attention over a paged KV cache (Section IV-C: the cloud keeps each user's
 * KV session and scores only the new positions; Algorithm 2 Step 2).
 *   hidden     bf16 [M][n_q_heads*head_dim]; row r, head h is the query vector.
 *   kv_pages   bf16 [num_pages][2][n_kv_heads][page_size][head_dim] (0=K, 1=V)
 *   page_table int32 [batch][max_pages_per_seq]; token t of sequence b lives in
 *              page page_table[b][t / page_size], slot t % page_size.
 *   kv_len[b]  = context + draft_len[b] + 1 (the window's K/V are already there)
 *   Row j of sequence b sees tokens t < kv_len[b] - (draft_len[b]+1) + j + 1.
 *   query head h reads kv head h / (n_q_heads / n_kv_heads).
 *   o = softmax(Q K^T / sqrt(head_dim)) V, fp64 throughout.
 * seq_sel/n_sel: evaluate only these sequences (NULL -> all); rows of other
 * sequences are left untouched.  attn_f64 (may be NULL) receives the unrounded
 * result, attn_bf16 (may be NULL) the result rounded to bf16: the one
 * deliberate rounding point, because the LM head consumes bf16. */
void fso_attention(const uint16_t* hidden, const uint16_t* kv_pages,
                   const int32_t* page_table, int32_t max_pages_per_seq,
                   const int32_t* kv_len, const int32_t* draft_len, int32_t batch,
                   int32_t n_q_heads, int32_t n_kv_heads, int32_t head_dim, int32_t page_size,
                   const int32_t* seq_sel, int32_t n_sel,
                   double* attn_f64, uint16_t* attn_bf16);

/* LM head: logits[r][v] = sum_i x[r][i] * w[v][i], fp64, i ascending.
 * row_sel/n_rows: only these rows (NULL -> all m rows). */
void fso_lm_head(const uint16_t* x, const uint16_t* w, int32_t m, int32_t d, int32_t vocab,
                 const int32_t* row_sel, int32_t n_rows, double* logits);

/* softmax(z / temperature) over v in [0,vocab); entries whose mask bit is 0
 * (mask word v/32, bit v%32; mask may be NULL) or whose logit is -inf get
 * probability exactly 0. */
void fso_softmax(const double* z, int32_t vocab, double temperature,
                 const uint32_t* mask, double* prob);

/* Nucleus (top-p) filter of a distribution, the sampling rule of the paper's stochastic regime
 * (Section V: T = 1, top-p 0.9): with the tokens ordered by decreasing probability (ties: lower
 * index first), m is the smallest prefix length whose mass reaches top_p; every token whose
 * probability is at least that of the m-th token is kept (so ties with the m-th token are all
 * kept), the rest get probability 0 and the kept ones are renormalised.  top_p >= 1 leaves prob
 * untouched.  margin (may be NULL) receives the distance of top_p from the nearer of the two
 * cumulative sums around the cut, i.e. how close the cut was to falling one token earlier/later. */
void fso_nucleus(double* prob, int32_t vocab, double top_p, double* margin);

/* Top-k filter of a distribution (the usual companion of top-p in sampling stacks; the paper's
 * stochastic regime names top-p only): every token whose probability is at least that of the k-th
 * most probable one is kept (ties with it are all kept, so the set is defined by a threshold and not
 * by a sort's tie order), the rest get probability 0, the kept ones are renormalised.
 * top_k <= 0 or >= vocab leaves prob untouched.  Applied BEFORE the nucleus filter. */
void fso_topk(double* prob, int32_t vocab, int32_t top_k);

/* The weights the emitted token is drawn from, for one target row (Algorithm 2: "sample correction
 * token"): r[v] = max(0, p(v) - q(v)) when zd_row is given (first rejection; p, q the softmaxes of
 * the two rows at `temperature`, p filtered by top-k and then to its nucleus), or r = p when zd_row is
 * NULL (bonus row) or the residual has no mass.  Returns Z = sum_v r[v]; r is not normalised. */
double fso_emission(const double* zt_row, const float* zd_row, int32_t vocab, double temperature,
                    int32_t top_k, double top_p, const uint32_t* mask, double* r, double* topp_margin);

/* Acceptance + emitted token for a batch of sequences.  The TARGET distribution of every row is
 * softmax(z / T) filtered by top-k (if 0 < top_k < vocab) and then to its nucleus (if top_p < 1),
 * SAMPLE mode only.  T is `temperature`, or temperatures[b] per sequence when that array is given
 * (both logit sets of the sequence are divided by it).
 * mode 0 = SAMPLE: accept x_j iff u_j * q_j(x_j) < p_j(x_j); after n accepted
 *   drafts emit a token from max(0, p_n - q_n)/Z (n < k) or from p_k (n == k)
 *   by inverse CDF in vocabulary order: min{v : sum_{w<=v} r_w > u' * Z}.
 * mode 1 = GREEDY (Algorithm 2 literally): accept while x_j == argmax of the
 *   target row (lowest index wins ties); emit the argmax of row n.
 *   target_logits fp64 [M][vocab] (rows packed by sequence, k_b+1 each)
 *   draft_logits  fp32 [S][vocab] (k_b rows each; unused in GREEDY, may be NULL)
 *   draft_tokens  int32 [S]
 *   vocab_mask    uint32 [batch][ceil(vocab/32)] or NULL; applies to the target.
 * Outputs (any debug pointer may be NULL):
 *   accepted_len[b], next_token[b];
 *   p_tok[S], q_tok[S], u_acc[S]: p_j(x_j), q_j(x_j), u_j (positions that were
 *     never reached still get their values: the test is evaluated for every j);
 *   acc_margin[S] = |u_j - min(1, p/q)|;
 *   cdf_margin[b] = distance from u'*Z to the nearer edge of the chosen CDF
 *     interval, divided by Z;  resid_mass[b] = Z. */
void fso_accept(int32_t mode, const double* target_logits, const float* draft_logits,
                const int32_t* draft_tokens, const int32_t* draft_len, const uint64_t* seeds,
                int32_t batch, int32_t vocab, double temperature, const double* temperatures /* [batch] or NULL */,
                int32_t top_k, double top_p, const uint32_t* vocab_mask,
                const int32_t* seq_sel, int32_t n_sel,
                int32_t* accepted_len, int32_t* next_token,
                double* p_tok, double* q_tok, double* u_acc, double* acc_margin,
                double* cdf_margin, double* resid_mass, double* topp_margin /* [M] or NULL */);

/* KV session around the step (Section IV-C).
 * fso_kv_append: the K/V rows of the k_b + 1 window positions (new_k / new_v, bf16 bit patterns,
 *   [M][n_kv_heads][head_dim], rows packed by sequence) are written into the pages: row j of
 *   sequence b is token kv_len[b] - (draft_len[b] + 1) + j.  Bytes are copied, nothing is computed.
 * fso_kv_rollback: after tau = accepted_len[b] accepted drafts the K/V of the later window
 *   positions are invalid; the sequence keeps its committed context, the accepted drafts' positions
 *   and position 0 of the window: kv_len_next = (kv_len - (k+1)) + tau + 1. */
void fso_kv_append(uint16_t* kv_pages, const int32_t* page_table, int32_t max_pages_per_seq,
                   const int32_t* kv_len, const int32_t* draft_len, int32_t batch,
                   int32_t n_kv_heads, int32_t head_dim, int32_t page_size,
                   const uint16_t* new_k, const uint16_t* new_v);
void fso_kv_rollback(const int32_t* kv_len, const int32_t* draft_len, const int32_t* accepted_len,
                     int32_t batch, int32_t* kv_len_next);

/* fso_kv_release: after the rollback the pages that hold no valid token any more are given back
 *   (Section IV-C: the invalid KV pairs are discarded): for every sequence the page-table entries
 *   ceil(kv_len_next / page_size) .. ceil(kv_len_prev / page_size) - 1 are appended to free_list
 *   (sequence by sequence, ascending entry index), *free_count is advanced and the entries become -1. */
void fso_kv_release(int32_t* page_table, int32_t max_pages_per_seq, const int32_t* kv_len_prev,
                    const int32_t* kv_len_next, int32_t batch, int32_t page_size,
                    int32_t* free_list, int32_t* free_count);

int32_t fso_num_threads(void);

#ifdef __cplusplus
}
#endif
#endif
