/*
 * flexspec.h -- C ABI of the B200 (sm_100a) cloud-side verification step of
 * edge-cloud speculative decoding.
 *
 * One verification step (Algorithm 2, "Step 2: cloud-side parallel
 * verification"; Section III-A system model; Section IV-C KV session): for a
 * batch of user sequences the cloud receives a block of k_b draft tokens per
 * sequence, scores the k_b+1 positions in parallel against the user's cached KV
 * session, decides how many draft tokens to accept (tau) and emits one further
 * token, so that the verified output is draft[0:tau] followed by that token.
 *
 * Three GPU stages, each a hand-written CUDA kernel:
 *   attention : paged-KV grouped-query attention of the k_b+1 query rows,
 *               causal inside the draft window (split over the KV range).
 *   lm_head   : logits[M][V] = attn_out[M][d] . W[V][d]^T on tcgen05 / TMEM.
 *   sample    : softmax of target and draft logits, acceptance test
 *               u * q(x) < p(x) with counter-based uniforms, first rejection,
 *               residual / bonus draw -- or the greedy arg-max rule that
 *               Algorithm 2 prints.
 *
 * Symbols: p = TARGET distribution, q = DRAFT distribution.  (Algorithm 2
 * writes the target's output as q; that letter is not used here.)
 *
 * Conventions
 *   - Every function returns 0 (FLEXSPEC_OK) or a negative FLEXSPEC_ERR_* code;
 *     nothing throws, aborts or exits.  Argument errors are detected on the
 *     host before any launch.
 *   - "DEVICE" pointers are CUDA global-memory addresses on the handle's
 *     device, "HOST" pointers ordinary host memory.  The caller owns every
 *     input and output buffer; the handle owns its workspace, which includes
 *     its own re-tiled copy of the LM-head weights (made by flexspec_create).
 *   - Calls that take a stream are asynchronous on it; outputs are valid once
 *     the stream has been synchronised.  A handle is not thread-safe and must
 *     be used on one stream at a time.
 *   - Row layout.  Sequence b owns k_b+1 consecutive query rows, starting at
 *     row sum_{b'<b}(k_b'+1): row 0 is the position of the last committed
 *     token, row j>=1 the position of draft token x_{j-1}.  The distribution
 *     read from row j judges draft token x_j; row k_b is the bonus row.  Draft
 *     rows (tokens, draft logits) are packed the same way with k_b per sequence.
 *   - M = sum_b (k_b+1) query rows, S = sum_b k_b draft positions.
 *   - flexspec_verify and the stage calls never write to the KV pages; the session
 *     calls around the step do (Section IV-C): flexspec_kv_append writes the window's
 *     K/V rows before it, flexspec_kv_rollback computes the truncated kv_len after a
 *     rejection and flexspec_kv_release hands the pages past it back.
 */
#ifndef FLEXSPEC_H
#define FLEXSPEC_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define FLEXSPEC_OK                0
#define FLEXSPEC_ERR_INVALID_ARG  -1   /* NULL pointer, size out of range, inconsistent lengths */
#define FLEXSPEC_ERR_UNSUPPORTED  -2   /* shape outside what the kernels are built for          */
#define FLEXSPEC_ERR_OOM          -3   /* workspace allocation failed                           */
#define FLEXSPEC_ERR_CUDA         -4   /* a CUDA runtime / driver call failed                   */
#define FLEXSPEC_ERR_TIMEOUT      -5   /* a bounded device-side wait gave up (status word)      */
#define FLEXSPEC_ERR_BAD_PAGE     -6   /* page table entry outside [0, num_pages)               */
#define FLEXSPEC_ERR_BAD_TOKEN    -7   /* draft token outside [0, vocab)                        */
#define FLEXSPEC_ERR_NO_DEVICE    -8   /* no usable CUDA device / driver                        */

#define FLEXSPEC_MODE_SAMPLE 0   /* speculative sampling: accept w.p. min(1, p/q), residual / bonus draw */
#define FLEXSPEC_MODE_GREEDY 1   /* Algorithm 2 as printed: accept while x_j == argmax of the target row */

#define FLEXSPEC_FLAG_DEBUG 1u   /* keep p(x_j), q(x_j), u_j per draft position (see flexspec_get_debug) */

typedef struct flexspec_handle flexspec_handle;   /* opaque */

typedef struct {
    int32_t  n_q_heads;     /* H; d_model = H * head_dim, must be a multiple of 64           */
    int32_t  n_kv_heads;    /* Hkv, divides H                                                 */
    int32_t  head_dim;      /* 64 or 128                                                      */
    int32_t  vocab;         /* 1 <= V <= 1048576                                              */
    int32_t  page_size;     /* tokens per KV page: must be 16                                 */
    int32_t  max_batch;     /* 1..1024 sequences per call                                     */
    int32_t  k_max;         /* largest draft length k_b, 0..63                                */
    int32_t  max_kv_len;    /* largest kv_len[b] (context + k_b + 1)                          */
    int32_t  mode;          /* FLEXSPEC_MODE_*                                                */
    int32_t  device;        /* CUDA device ordinal                                            */
    uint32_t flags;         /* FLEXSPEC_FLAG_*                                                */
} flexspec_config;

/* The per-user KV sessions (Section IV-C), as one paged pool. */
typedef struct {
    const void*    kv_pages;          /* DEVICE bf16 [num_pages][2][n_kv_heads][page_size][head_dim];
                                         index 0 of the second axis is K, 1 is V; 16-byte aligned   */
    int32_t        num_pages;
    const int32_t* page_table;        /* DEVICE int32 [batch][max_pages_per_seq]: token t of sequence b
                                         lives in page page_table[b][t/16], slot t%16; entries past
                                         ceil(kv_len[b]/16) are never read                          */
    int32_t        max_pages_per_seq;
    const int32_t* kv_len;            /* DEVICE int32 [batch] = committed context + k_b + 1: the K/V
                                         of the k_b+1 window positions are already in the pages     */
    const int32_t* kv_len_host;       /* HOST copy of kv_len (launch geometry only)                 */
} flexspec_kv;

typedef struct {            /* DEVICE pointers into the handle's workspace, valid until destroy */
    const void*    attn_out;   /* bf16 [M][d_model], last verify / attention call                 */
    const float*   logits;     /* fp32 [M][vocab], last verify / lm_head call into the workspace  */
    const double*  p_tok;      /* fp64 [S]  p_j(x_j)   (FLEXSPEC_FLAG_DEBUG, SAMPLE mode)          */
    const double*  q_tok;      /* fp64 [S]  q_j(x_j)                                              */
    const float*   u_acc;      /* fp32 [S]  u_j                                                   */
    const int32_t* status;     /* int32 [4] device status word: [0] first error code, [1] detail  */
    const double*  topp;       /* fp64 [M][2] per target row, written when top-k / top-p is on: the lowest kept
                                  logit and the kept mass in units of the row's largest term          */
} flexspec_debug;

/* Create a handle for one target model's verification step (the frozen head and the KV-session
 * layout of Sections IV-A and IV-C): validates the shape, allocates the workspace on cfg->device
 * (logits [max_batch*(k_max+1)][vocab] fp32, the re-tiled copy of the LM-head weights, attention
 * partials, small tables) and builds the TMA descriptors of that copy.
 *   lm_head_w : DEVICE bf16 [vocab][d_model] (row v is the output embedding of
 *               token v), 16-byte aligned.  It is read during this call only: the handle keeps
 *               its own copy (vocab * d_model * 2 bytes, rounded up to whole tiles) in the order
 *               the LM head streams it, one contiguous block per pipeline stage; the caller may
 *               free or overwrite its buffer afterwards (later changes are not seen).
 * Errors: INVALID_ARG, UNSUPPORTED, OOM, CUDA, NO_DEVICE. */
int flexspec_create(const flexspec_config* cfg, const void* lm_head_w, flexspec_handle** out);

/* The whole verification step (Algorithm 2, Step 2) on `stream`:
 * attention -> LM head -> acceptance + emitted token.
 *   hidden        DEVICE bf16 [M][d_model]; row r viewed as [H][head_dim] is the query of
 *                 every head (the attention output feeds the LM head directly)
 *   draft_tokens  DEVICE int32 [S]
 *   draft_logits  DEVICE fp32 [S][vocab]; may be NULL in GREEDY mode.  When vocab is a multiple
 *                 of 4 the rows are read with 16-byte loads and the array must start on a
 *                 16-byte boundary (else INVALID_ARG); otherwise 4-byte alignment is enough.
 *   draft_len     DEVICE int32 [batch], draft_len_host its HOST copy (launch geometry)
 *   seeds         DEVICE uint64 [batch]; uniforms are Philox4x32-10 with key =
 *                 (lo32, hi32) of the seed, counter = (j, stream, 0, 0), word 0,
 *                 u = (word >> 8) * 2^-24; stream 0 = acceptance test of draft j,
 *                 stream 1 = draw of the emitted token after j accepted drafts.
 *                 May be NULL in GREEDY mode.
 *   temperature   both logit sets are divided by it; 0 selects the greedy rule
 *   vocab_mask    DEVICE uint32 [batch][ceil(vocab/32)] or NULL: a 0 bit forbids
 *                 that token for the target (p = 0 exactly)
 *   accepted_len  DEVICE int32 [batch] out: tau_b in [0, k_b]
 *   next_token    DEVICE int32 [batch] out: the token emitted after the accepted prefix
 * Errors: INVALID_ARG (NULLs, batch > max_batch, k_b > k_max, kv_len out of range or
 * smaller than k_b+1, too few pages per sequence), CUDA. Device-side problems
 * (bad page id, bad token id, a wait that gave up, a DEVICE draft_len that disagrees
 * with draft_len_host: INVALID_ARG, and the sampling stage then treats every k_b as 0)
 * are recorded in the status word, see flexspec_status.  Outputs of a call whose status
 * word is non-zero are undefined. */
int flexspec_verify(flexspec_handle* h, const flexspec_kv* kv, const void* hidden,
                    const int32_t* draft_tokens, const float* draft_logits,
                    const int32_t* draft_len, const int32_t* draft_len_host,
                    const uint64_t* seeds, int32_t batch, float temperature,
                    const uint32_t* vocab_mask,
                    int32_t* accepted_len, int32_t* next_token, void* stream);

/* The same step (Algorithm 2, Step 2: the cloud receives the draft block over the uplink and
 * returns the verified tokens) for callers whose per-step inputs live in HOST memory: copies
 * hidden, draft tokens, draft logits, lengths, seeds and the optional vocabulary mask to the
 * device, runs flexspec_verify, copies accepted_len / next_token back and synchronises.
 * The KV pool and page table stay on the device (they are the persistent session state of
 * Section IV-C); kv->kv_len may be NULL here (taken from kv->kv_len_host).
 * Every other pointer argument is a HOST pointer (vocab_mask may be NULL). */
int flexspec_verify_host(flexspec_handle* h, const flexspec_kv* kv, const void* hidden,
                         const int32_t* draft_tokens, const float* draft_logits,
                         const int32_t* draft_len, const uint64_t* seeds, int32_t batch,
                         float temperature, const uint32_t* vocab_mask,
                         int32_t* accepted_len, int32_t* next_token, void* stream);

/* Stage 1 alone (Section IV-C; Algorithm 2 "restore KV cache" + target forward over the block):
 * attn_out DEVICE bf16 [M][d_model] out, or NULL to write the handle's workspace. */
int flexspec_attention(flexspec_handle* h, const flexspec_kv* kv, const void* hidden,
                       const int32_t* draft_len, const int32_t* draft_len_host, int32_t batch,
                       void* attn_out, void* stream);

/* Stage 2 alone: logits[m_rows][vocab] = x[m_rows][d_model] . W^T (the frozen LM head of
 * the target, Section IV-A).  x DEVICE bf16 (NULL = workspace attn_out), logits DEVICE fp32
 * (NULL = workspace).  m_rows <= max_batch*(k_max+1). */
int flexspec_lm_head(flexspec_handle* h, const void* x, int32_t m_rows, float* logits, void* stream);

/* Stage 3 alone (Algorithm 2 acceptance loop and correction token; the stochastic rule of
 * the speculative-sampling papers it cites).  logits DEVICE fp32 [M][vocab] (NULL = workspace),
 * aligned like draft_logits; other arguments as in flexspec_verify. */
int flexspec_sample(flexspec_handle* h, const float* logits,
                    const int32_t* draft_tokens, const float* draft_logits,
                    const int32_t* draft_len, const int32_t* draft_len_host,
                    const uint64_t* seeds, int32_t batch, float temperature,
                    const uint32_t* vocab_mask,
                    int32_t* accepted_len, int32_t* next_token, void* stream);

/* KV session, before the step (Section IV-C: the cloud computes the K/V pairs of the newly received
 * tokens only).  Writes the K/V rows of the k_b + 1 window positions of every sequence into its
 * pages: row j of sequence b goes to token position kv_len[b] - (k_b + 1) + j.
 *   kv_pages    DEVICE bf16 pool as in flexspec_kv (written here, and only here)
 *   new_k/new_v DEVICE bf16 [M][n_kv_heads][head_dim], rows packed like the query rows, 16-byte aligned
 *   kv_len      DEVICE int32 [batch] = committed context + k_b + 1 (the length verification will see)
 * The pages of the window positions must already be in the page table.  Asynchronous on `stream`.
 * Errors: INVALID_ARG, CUDA; a page id outside the pool is recorded in the status word. */
int flexspec_kv_append(flexspec_handle* h, void* kv_pages, int32_t num_pages, const int32_t* page_table,
                       int32_t max_pages_per_seq, const int32_t* kv_len, const int32_t* kv_len_host,
                       const void* new_k, const void* new_v, const int32_t* draft_len,
                       const int32_t* draft_len_host, int32_t batch, void* stream);

/* KV session, after the step (Section IV-C: on a rejection the invalid K/V pairs are discarded).
 * With paged storage the rollback is a new length, computed on the device so that a serving loop
 * needs no host round trip: kv_len_next[b] = kv_len[b] - (k_b + 1) + accepted_len[b] + 1, i.e. the
 * committed context plus the accepted drafts plus the position whose K/V the next step appends
 * first.  All pointers DEVICE int32 [batch]; kv_len_next may alias kv_len. */
int flexspec_kv_rollback(flexspec_handle* h, const int32_t* kv_len, const int32_t* draft_len,
                         const int32_t* accepted_len, int32_t batch, int32_t* kv_len_next, void* stream);

/* KV session, after the rollback: the pages that hold no valid token any more are handed back
 * (Section IV-C: "discarding" the invalid K/V pairs -- with paged storage that is a free list).
 * For every sequence the page-table entries ceil(kv_len_next[b] / 16) .. ceil(kv_len_prev[b] / 16) - 1
 * are appended to free_list (one reservation per sequence: its pages stay together, in ascending
 * entry order; the order of the sequences in the list is not defined) and set to -1.
 *   page_table   DEVICE int32 [batch][max_pages_per_seq], modified in place
 *   kv_len_prev  DEVICE int32 [batch]: the length the pages were allocated for (before the rollback)
 *   kv_len_next  DEVICE int32 [batch]: e.g. the output of flexspec_kv_rollback
 *   free_list    DEVICE int32 [free_capacity]; free_count DEVICE int32 [1], advanced atomically (the
 *                caller sets it, usually to the list's current fill)
 * Note that the next step's window positions then need pages again: release only what the serving
 * loop will not re-use at once.  Asynchronous on `stream`.  Errors: INVALID_ARG, CUDA; an entry
 * outside [0, num_pages) or a list that is too short is recorded in the status word. */
int flexspec_kv_release(flexspec_handle* h, int32_t* page_table, int32_t max_pages_per_seq, int32_t num_pages,
                        const int32_t* kv_len_prev, const int32_t* kv_len_next, int32_t batch, int32_t* free_list,
                        int32_t free_capacity, int32_t* free_count, void* stream);

/* The acceptance / emitted-token stage (flexspec_sample) without a handle and without any
 * allocation.  (No counterpart in the paper: it exists for how some hosts have to run.)
 * Meant for callers that cannot obtain device memory at call time: a serving process whose
 * memory pool took the whole device at start-up, so that a cudaMalloc inside the library would
 * fail or eat into the pool's reserve; or a step loop that must never stall on the implicit
 * device synchronisation of an allocation or a free.  Such callers cannot use flexspec_create,
 * which allocates the workspace.
 *   - The working memory is one fixed array inside the loaded library (276 224 bytes, held on
 *     every GPU that loads the library until the process exits).  Limits that follow from it:
 *     batch <= 64, sum_b (k_b + 1) <= 1024, vocab <= 131072; larger calls return
 *     FLEXSPEC_ERR_UNSUPPORTED and launch nothing.
 *   - Runs on the CURRENT device of the calling thread.  The first call on a device looks up
 *     the device address of the array (a cheap runtime query, no allocation); make that first
 *     call outside any stream capture, and from one thread: the look-up is not synchronised,
 *     so two threads must not make the first call on a device at the same time.
 *   - All calls on a device share the array, and it keeps the previous call's contents; each
 *     call clears the part that has to start at zero (the status word) on `stream` before its
 *     kernels, which rewrite everything else before reading it.  Two calls
 *     whose GPU work may overlap (different streams, no ordering) race on the array: serialise
 *     them.
 *   - Arguments as flexspec_sample (the same alignment of the two logit arrays included), all
 *     DEVICE pointers except draft_len_host; `mode` is a FLEXSPEC_MODE_* value.  A draft token outside [0, vocab) is clamped, not reported.
 * Errors: INVALID_ARG, UNSUPPORTED (limits above), NO_DEVICE, CUDA. */
int flexspec_sample_static(const float* logits, const int32_t* draft_tokens, const float* draft_logits,
                           const int32_t* draft_len, const int32_t* draft_len_host, const uint64_t* seeds,
                           int32_t batch, int32_t vocab, int32_t mode, float temperature,
                           const uint32_t* vocab_mask, int32_t* accepted_len, int32_t* next_token,
                           void* stream);

/* Nucleus (top-p) sampling of the target, the paper's stochastic regime (Section V: T = 1,
 * top-p 0.9).  From the next verify / sample call on, the target distribution of every row is its
 * nucleus: the tokens whose probability is at least that of the last token of the smallest
 * top-probability prefix holding mass >= top_p (ties with that token are all kept), renormalised;
 * acceptance tests, the residual and the bonus draw use it.  top_p = 1 (the default) switches the
 * filter off.  SAMPLE mode only; 0 < top_p <= 1, else INVALID_ARG. */
int flexspec_set_top_p(flexspec_handle* h, float top_p);

/* All sampling controls of the target distribution at once (Section V, Regime B: T = 1, top-p 0.9;
 * top-k is the usual companion of top-p and is applied first).  From the next verify / sample call on:
 *   top_p         as flexspec_set_top_p (1 = off);
 *   top_k         keep the top_k most probable tokens of every target row (ties with the k-th are all
 *                 kept) and renormalise, before the nucleus is taken; 0 = off;
 *   temperatures  DEVICE fp32 [batch] or NULL: when given, sequence b uses temperatures[b] instead
 *                 of the call's scalar temperature for both of its logit sets.  The array is read by
 *                 every following call (it is borrowed, not copied) and must hold positive finite
 *                 values: anything else is reported as INVALID_ARG in the status word and the scalar
 *                 is used for that sequence.  The scalar still selects the greedy rule when it is 0.
 * SAMPLE mode only.  Errors: INVALID_ARG. */
int flexspec_set_sampling(flexspec_handle* h, float top_p, int32_t top_k, const float* temperatures);

/* Workspace pointers for stage-wise comparison with an independent implementation of Algorithm 2,
 * Step 2 (attention output, logits, p_j(x_j), q_j(x_j), u_j of the last call). */
int flexspec_get_debug(flexspec_handle* h, flexspec_debug* out);

/* Device-side error reporting (no counterpart in the paper).  Synchronises the device, copies the status word to status_host[4] (may be NULL), clears it
 * and returns its first entry (0 or a FLEXSPEC_ERR_* code recorded by a kernel). */
int flexspec_status(flexspec_handle* h, int32_t* status_host);

/* Diagnostic for the bounded waits (no counterpart in the paper).  Every device-side wait of the
 * library (TMA arrivals, tensor-core completions, hand-overs between warps) gives up after a fixed
 * wall time, records FLEXSPEC_ERR_TIMEOUT in the status word and lets its kernel return, so a stalled
 * pipeline never turns into a hung GPU.  This call launches a one-thread kernel that waits, with that
 * same routine, on a barrier nobody ever signals: after limit_ns (1 us .. 50 ms, else INVALID_ARG)
 * the wait runs out and flexspec_status returns FLEXSPEC_ERR_TIMEOUT; the handle stays usable. */
int flexspec_selftest_wait_timeout(flexspec_handle* h, int64_t limit_ns, void* stream);

/* Per-kernel timing.  With profiling on, verify brackets the kernels of the caller's stream with
 * CUDA events; flexspec_get_stage_ms synchronises those events and writes the last call's
 * durations in milliseconds: [0] fork of the second stream, [1] attention, [2] unused,
 * [3] LM head (with the softmax statistics of the target rows), [4] nucleus thresholds (top-p
 * only), [5] acceptance kernel (tests, first rejection, emitted token).  The row-offset kernel
 * and the draft-logit statistics run on a second stream beside attention and are not timed.
 * Unused stages read 0. */
int flexspec_set_profiling(flexspec_handle* h, int32_t on);
int flexspec_get_stage_ms(flexspec_handle* h, float ms[6]);

/* Number of kernels the last verify / stage call launched. */
int flexspec_last_launches(flexspec_handle* h);

/* Releases the workspace (the KV sessions and the LM-head weights are the caller's and are not
 * touched).  NULL is accepted. */
int flexspec_destroy(flexspec_handle* h);

const char* flexspec_strerror(int code);
const char* flexspec_version(void);

#ifdef __cplusplus
}
#endif
#endif
