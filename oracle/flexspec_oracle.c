/*
 * flexspec_oracle.c -- TEST INFRASTRUCTURE, NOT PRODUCT CODE.
 *
 * fp64 CPU statement of the cloud-side verification step (Algorithm 2, Step 2;
 * Section IV-C).  Scalar loops in the order the definitions are written;
 * OpenMP only across independent rows / sequences.  No code is shared with the
 * CUDA path.  See flexspec_oracle.h for conventions.
 *
 * Pin status.  Attention, LM head, softmax, Philox, the acceptance rule, the
 * residual draw and the greedy rule are each pinned by CPU tests against
 * something other than this file (dense brute force, library fp64 routines,
 * published known-answer vectors, closed forms, chi-square on the emitted
 * token).  Parity unpinned: which particular (accepted_len, next_token) a
 * given seed produces -- that is fixed only by the counter/key convention
 * stated in the header, which the paper does not define.
 */
#include "flexspec_oracle.h"

#include <math.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* ------------------------------------------------------------------ bf16 */

double fso_bf16_to_f64(uint16_t h)
{
    uint32_t u = (uint32_t)h << 16;
    float f;
    memcpy(&f, &u, 4);
    return (double)f;
}

uint16_t fso_f64_to_bf16(double x)
{
    if (isnan(x)) return 0x7fc0;
    uint16_t sign = signbit(x) ? 0x8000 : 0;
    double a = fabs(x);
    if (a == 0.0) return sign;
    if (isinf(a)) return sign | 0x7f80;
    int e;
    (void)frexp(a, &e);               /* a = m * 2^e, m in [0.5, 1) */
    int q = e - 8;                    /* quantum 2^q keeps 8 significant bits */
    if (q < -133) q = -133;           /* bf16 subnormal spacing */
    double r = nearbyint(ldexp(a, -q)); /* ties to even (default rounding mode) */
    double y = ldexp(r, q);
    if (y >= ldexp(1.0, 128)) return sign | 0x7f80;
    float f = (float)y;               /* exact: y has at most 8 significant bits */
    uint32_t u;
    memcpy(&u, &f, 4);
    return sign | (uint16_t)(u >> 16);
}

/* ---------------------------------------------------------------- Philox */

static void mulhilo32(uint32_t a, uint32_t b, uint32_t* hi, uint32_t* lo)
{
    uint64_t p = (uint64_t)a * (uint64_t)b;
    *hi = (uint32_t)(p >> 32);
    *lo = (uint32_t)p;
}

void fso_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4])
{
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
    uint32_t k0 = key[0], k1 = key[1];
    for (int round = 0; round < 10; ++round) {
        if (round > 0) { k0 += 0x9E3779B9u; k1 += 0xBB67AE85u; }
        uint32_t hi0, lo0, hi1, lo1;
        mulhilo32(0xD2511F53u, c0, &hi0, &lo0);
        mulhilo32(0xCD9E8D57u, c2, &hi1, &lo1);
        uint32_t n0 = hi1 ^ c1 ^ k0;
        uint32_t n1 = lo1;
        uint32_t n2 = hi0 ^ c3 ^ k1;
        uint32_t n3 = lo0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

double fso_uniform(uint64_t seed, uint32_t index, uint32_t stream)
{
    uint32_t ctr[4] = { index, stream, 0u, 0u };
    uint32_t key[2] = { (uint32_t)(seed & 0xffffffffu), (uint32_t)(seed >> 32) };
    uint32_t out[4];
    fso_philox4x32_10(ctr, key, out);
    return (double)(out[0] >> 8) * (1.0 / 16777216.0);
}

/* ------------------------------------------------------------- attention */

void fso_attention(const uint16_t* hidden, const uint16_t* kv_pages,
                   const int32_t* page_table, int32_t max_pages_per_seq,
                   const int32_t* kv_len, const int32_t* draft_len, int32_t batch,
                   int32_t n_q_heads, int32_t n_kv_heads, int32_t head_dim, int32_t page_size,
                   const int32_t* seq_sel, int32_t n_sel,
                   double* attn_f64, uint16_t* attn_bf16)
{
    const int64_t d_model = (int64_t)n_q_heads * head_dim;
    const int32_t group = n_q_heads / n_kv_heads;
    const double scale = 1.0 / sqrt((double)head_dim);

    /* first query row of every sequence */
    int64_t* row0 = (int64_t*)malloc(sizeof(int64_t) * (size_t)(batch + 1));
    row0[0] = 0;
    for (int32_t b = 0; b < batch; ++b) row0[b + 1] = row0[b] + draft_len[b] + 1;

    const int32_t n_eval = seq_sel ? n_sel : batch;
    for (int32_t s = 0; s < n_eval; ++s) {
        const int32_t b = seq_sel ? seq_sel[s] : s;
        const int32_t k = draft_len[b];
        const int32_t ctx = kv_len[b] - (k + 1);
        const int64_t n_rows = (int64_t)(k + 1) * n_q_heads;
#pragma omp parallel
        {
            double* score = (double*)malloc(sizeof(double) * (size_t)(kv_len[b] > 0 ? kv_len[b] : 1));
            double* out = (double*)malloc(sizeof(double) * (size_t)head_dim);
#pragma omp for schedule(dynamic, 1)
            for (int64_t rh = 0; rh < n_rows; ++rh) {
                const int32_t j = (int32_t)(rh / n_q_heads);
                const int32_t h = (int32_t)(rh % n_q_heads);
                const int32_t kvh = h / group;
                const int64_t r = row0[b] + j;
                const int32_t n_vis = ctx + j + 1;
                const uint16_t* qv = hidden + r * d_model + (int64_t)h * head_dim;

                double smax = -INFINITY;
                for (int32_t t = 0; t < n_vis; ++t) {
                    const int64_t page = page_table[(int64_t)b * max_pages_per_seq + t / page_size];
                    const int32_t slot = t % page_size;
                    const uint16_t* kt = kv_pages +
                        ((((page * 2 + 0) * n_kv_heads + kvh) * page_size + slot) * (int64_t)head_dim);
                    double dot = 0.0;
                    for (int32_t e = 0; e < head_dim; ++e)
                        dot += fso_bf16_to_f64(qv[e]) * fso_bf16_to_f64(kt[e]);
                    score[t] = scale * dot;
                    if (score[t] > smax) smax = score[t];
                }
                double denom = 0.0;
                for (int32_t t = 0; t < n_vis; ++t) {
                    score[t] = exp(score[t] - smax);
                    denom += score[t];
                }
                for (int32_t e = 0; e < head_dim; ++e) out[e] = 0.0;
                for (int32_t t = 0; t < n_vis; ++t) {
                    const int64_t page = page_table[(int64_t)b * max_pages_per_seq + t / page_size];
                    const int32_t slot = t % page_size;
                    const uint16_t* vt = kv_pages +
                        ((((page * 2 + 1) * n_kv_heads + kvh) * page_size + slot) * (int64_t)head_dim);
                    const double a = score[t] / denom;
                    for (int32_t e = 0; e < head_dim; ++e)
                        out[e] += a * fso_bf16_to_f64(vt[e]);
                }
                for (int32_t e = 0; e < head_dim; ++e) {
                    const int64_t o = r * d_model + (int64_t)h * head_dim + e;
                    if (attn_f64) attn_f64[o] = out[e];
                    if (attn_bf16) attn_bf16[o] = fso_f64_to_bf16(out[e]);
                }
            }
            free(score);
            free(out);
        }
    }
    free(row0);
}

/* --------------------------------------------------------------- LM head */

void fso_lm_head(const uint16_t* x, const uint16_t* w, int32_t m, int32_t d, int32_t vocab,
                 const int32_t* row_sel, int32_t n_rows, double* logits)
{
    const int32_t n_eval = row_sel ? n_rows : m;
    /* decode the selected activation rows once */
    double* xd = (double*)malloc(sizeof(double) * (size_t)n_eval * (size_t)d);
    for (int32_t s = 0; s < n_eval; ++s) {
        const int32_t r = row_sel ? row_sel[s] : s;
        for (int32_t i = 0; i < d; ++i)
            xd[(int64_t)s * d + i] = fso_bf16_to_f64(x[(int64_t)r * d + i]);
    }
#pragma omp parallel
    {
        double* wd = (double*)malloc(sizeof(double) * (size_t)d);
#pragma omp for schedule(static)
        for (int32_t v = 0; v < vocab; ++v) {
            for (int32_t i = 0; i < d; ++i) wd[i] = fso_bf16_to_f64(w[(int64_t)v * d + i]);
            for (int32_t s = 0; s < n_eval; ++s) {
                const int32_t r = row_sel ? row_sel[s] : s;
                const double* xr = xd + (int64_t)s * d;
                double acc = 0.0;
                for (int32_t i = 0; i < d; ++i) acc += xr[i] * wd[i];
                logits[(int64_t)r * vocab + v] = acc;
            }
        }
        free(wd);
    }
    free(xd);
}

/* --------------------------------------------------------------- softmax */

static int mask_allows(const uint32_t* mask, int32_t v)
{
    return mask == NULL || ((mask[v >> 5] >> (v & 31)) & 1u);
}

void fso_softmax(const double* z, int32_t vocab, double temperature,
                 const uint32_t* mask, double* prob)
{
    double zmax = -INFINITY;
    for (int32_t v = 0; v < vocab; ++v)
        if (mask_allows(mask, v) && z[v] / temperature > zmax) zmax = z[v] / temperature;
    double denom = 0.0;
    for (int32_t v = 0; v < vocab; ++v) {
        if (mask_allows(mask, v) && z[v] != -INFINITY) {
            prob[v] = exp(z[v] / temperature - zmax);
            denom += prob[v];
        } else {
            prob[v] = 0.0;
        }
    }
    for (int32_t v = 0; v < vocab; ++v) prob[v] = prob[v] / denom;
}

/* --------------------------------------------------------------- nucleus */

typedef struct { double p; int32_t v; } fso_pv;
static int cmp_pv_desc(const void* a, const void* b)
{
    const fso_pv* x = (const fso_pv*)a;
    const fso_pv* y = (const fso_pv*)b;
    if (x->p > y->p) return -1;
    if (x->p < y->p) return 1;
    return (x->v > y->v) - (x->v < y->v);
}

void fso_nucleus(double* prob, int32_t vocab, double top_p, double* margin)
{
    if (margin) *margin = INFINITY;
    if (!(top_p < 1.0)) return;
    fso_pv* s = (fso_pv*)malloc(sizeof(fso_pv) * (size_t)vocab);
    for (int32_t v = 0; v < vocab; ++v) { s[v].p = prob[v]; s[v].v = v; }
    qsort(s, (size_t)vocab, sizeof(fso_pv), cmp_pv_desc);
    double c = 0.0, c_prev = 0.0;
    int32_t m = 0;
    for (; m < vocab; ++m) {
        c_prev = c;
        c += s[m].p;
        if (c >= top_p) break;
    }
    if (m == vocab) m = vocab - 1;
    const double thr = s[m].p;
    if (margin) {
        const double a = fabs(c - top_p), b = fabs(top_p - c_prev);
        *margin = a < b ? a : b;
    }
    double z = 0.0;
    for (int32_t v = 0; v < vocab; ++v) z += (prob[v] >= thr && prob[v] > 0.0) ? prob[v] : 0.0;
    for (int32_t v = 0; v < vocab; ++v) prob[v] = (prob[v] >= thr && prob[v] > 0.0) ? prob[v] / z : 0.0;
    free(s);
}

/* ------------------------------------------------------------------ top-k */

void fso_topk(double* prob, int32_t vocab, int32_t top_k)
{
    if (top_k <= 0 || top_k >= vocab) return;
    fso_pv* s = (fso_pv*)malloc(sizeof(fso_pv) * (size_t)vocab);
    for (int32_t v = 0; v < vocab; ++v) { s[v].p = prob[v]; s[v].v = v; }
    qsort(s, (size_t)vocab, sizeof(fso_pv), cmp_pv_desc);
    const double thr = s[top_k - 1].p;                    /* probability of the k-th largest */
    double z = 0.0;
    for (int32_t v = 0; v < vocab; ++v) z += (prob[v] >= thr && prob[v] > 0.0) ? prob[v] : 0.0;
    for (int32_t v = 0; v < vocab; ++v) prob[v] = (prob[v] >= thr && prob[v] > 0.0) ? prob[v] / z : 0.0;
    free(s);
}

/* the target distribution of one row: softmax at the temperature, then top-k, then top-p */
static void target_dist(const double* zt_row, int32_t vocab, double temperature, int32_t top_k, double top_p,
                        const uint32_t* mask, double* p, double* topp_margin)
{
    fso_softmax(zt_row, vocab, temperature, mask, p);
    fso_topk(p, vocab, top_k);
    fso_nucleus(p, vocab, top_p, topp_margin);
}

/* ------------------------------------------------- acceptance + emission */

static int32_t argmax_lowest(const double* z, int32_t vocab, const uint32_t* mask)
{
    int32_t best = -1;
    double zb = -INFINITY;
    for (int32_t v = 0; v < vocab; ++v) {
        if (!mask_allows(mask, v)) continue;
        if (best < 0 || z[v] > zb) { best = v; zb = z[v]; }
    }
    return best;
}

/* inverse CDF in vocabulary order: min{v : sum_{w<=v} r_w > thr}; if rounding
 * leaves none, the last index with r_v > 0.  Reports the chosen interval. */
static int32_t inverse_cdf(const double* r, int32_t vocab, double thr,
                           double* c_below, double* c_at)
{
    double c = 0.0;
    int32_t last_pos = -1;
    double last_below = 0.0, last_at = 0.0;
    for (int32_t v = 0; v < vocab; ++v) {
        const double below = c;
        c += r[v];
        if (r[v] > 0.0) { last_pos = v; last_below = below; last_at = c; }
        if (c > thr) { *c_below = below; *c_at = c; return v; }
    }
    *c_below = last_below; *c_at = last_at;
    return last_pos;
}

/* Unnormalised weights of the emitted token and their sum Z: max(0, p - q) when a draft row is
 * given (the first rejection) and that residual has positive mass, else p (the bonus row, or a
 * residual that rounding emptied). */
double fso_emission(const double* zt_row, const float* zd_row, int32_t vocab, double temperature,
                    int32_t top_k, double top_p, const uint32_t* mask, double* r, double* topp_margin)
{
    double* p = (double*)malloc(sizeof(double) * (size_t)vocab);
    target_dist(zt_row, vocab, temperature, top_k, top_p, mask, p, topp_margin);
    double z_mass = 0.0;
    if (zd_row != NULL) {
        double* q = (double*)malloc(sizeof(double) * (size_t)vocab);
        double* zq = (double*)malloc(sizeof(double) * (size_t)vocab);
        for (int32_t v = 0; v < vocab; ++v) zq[v] = (double)zd_row[v];
        fso_softmax(zq, vocab, temperature, NULL, q);
        for (int32_t v = 0; v < vocab; ++v) {
            r[v] = p[v] - q[v] > 0.0 ? p[v] - q[v] : 0.0;
            z_mass += r[v];
        }
        free(q); free(zq);
    }
    if (zd_row == NULL || !(z_mass > 0.0)) {
        z_mass = 0.0;
        for (int32_t v = 0; v < vocab; ++v) { r[v] = p[v]; z_mass += r[v]; }
    }
    free(p);
    return z_mass;
}

static void verify_one(int32_t mode, const double* zt, const float* zd, const int32_t* x,
                       int32_t k, int32_t vocab, double temperature, int32_t top_k, double top_p, uint64_t seed,
                       const uint32_t* mask, double* topp_margin,
                       int32_t* accepted_len, int32_t* next_token,
                       double* p_tok, double* q_tok, double* u_acc, double* acc_margin,
                       double* cdf_margin, double* resid_mass)
{
    if (mode == 1) { /* GREEDY: Algorithm 2, the acceptance loop as printed */
        int32_t n = 0;
        while (n < k && x[n] == argmax_lowest(zt + (int64_t)n * vocab, vocab, mask)) ++n;
        *accepted_len = n;
        *next_token = argmax_lowest(zt + (int64_t)n * vocab, vocab, mask);
        if (cdf_margin) *cdf_margin = INFINITY;
        if (resid_mass) *resid_mass = 1.0;
        return;
    }

    double* p = (double*)malloc(sizeof(double) * (size_t)vocab);
    double* q = (double*)malloc(sizeof(double) * (size_t)vocab);
    double* zq = (double*)malloc(sizeof(double) * (size_t)vocab);
    double* r = (double*)malloc(sizeof(double) * (size_t)vocab);

    /* the acceptance test at every draft position; n = first failure */
    int32_t n = k;
    for (int32_t j = 0; j < k; ++j) {
        target_dist(zt + (int64_t)j * vocab, vocab, temperature, top_k, top_p, mask, p, topp_margin ? topp_margin + j : NULL);
        for (int32_t v = 0; v < vocab; ++v) zq[v] = (double)zd[(int64_t)j * vocab + v];
        fso_softmax(zq, vocab, temperature, NULL, q);
        const double u = fso_uniform(seed, (uint32_t)j, 0u);
        const double pj = p[x[j]], qj = q[x[j]];
        const int accept = (u * qj < pj);
        if (!accept && j < n) n = j;
        if (p_tok) p_tok[j] = pj;
        if (q_tok) q_tok[j] = qj;
        if (u_acc) u_acc[j] = u;
        if (acc_margin) {
            double ratio = (pj >= qj) ? (pj > 0.0 ? 1.0 : 0.0) : pj / qj;
            acc_margin[j] = fabs(u - ratio);
        }
    }

    /* emitted token: residual at the first rejection, else the bonus row */
    double z_mass = fso_emission(zt + (int64_t)n * vocab, n < k ? zd + (int64_t)n * vocab : NULL, vocab,
                                 temperature, top_k, top_p, mask, r, topp_margin ? topp_margin + n : NULL);
    const double u2 = fso_uniform(seed, (uint32_t)n, 1u);
    double c_below, c_at;
    const double thr = u2 * z_mass;
    *next_token = inverse_cdf(r, vocab, thr, &c_below, &c_at);
    *accepted_len = n;
    if (cdf_margin) {
        double m1 = fabs(thr - c_below), m2 = fabs(c_at - thr);
        *cdf_margin = (m1 < m2 ? m1 : m2) / z_mass;
    }
    if (resid_mass) *resid_mass = z_mass;

    free(p); free(q); free(zq); free(r);
}

void fso_accept(int32_t mode, const double* target_logits, const float* draft_logits,
                const int32_t* draft_tokens, const int32_t* draft_len, const uint64_t* seeds,
                int32_t batch, int32_t vocab, double temperature, const double* temperatures, int32_t top_k,
                double top_p, const uint32_t* vocab_mask,
                const int32_t* seq_sel, int32_t n_sel,
                int32_t* accepted_len, int32_t* next_token,
                double* p_tok, double* q_tok, double* u_acc, double* acc_margin,
                double* cdf_margin, double* resid_mass, double* topp_margin)
{
    int64_t* row0 = (int64_t*)malloc(sizeof(int64_t) * (size_t)(batch + 1));
    int64_t* tok0 = (int64_t*)malloc(sizeof(int64_t) * (size_t)(batch + 1));
    row0[0] = 0; tok0[0] = 0;
    for (int32_t b = 0; b < batch; ++b) {
        row0[b + 1] = row0[b] + draft_len[b] + 1;
        tok0[b + 1] = tok0[b] + draft_len[b];
    }
    const int32_t mask_words = (vocab + 31) / 32;
    const int32_t n_eval = seq_sel ? n_sel : batch;
#pragma omp parallel for schedule(dynamic, 1)
    for (int32_t s = 0; s < n_eval; ++s) {
        const int32_t b = seq_sel ? seq_sel[s] : s;
        const int64_t t0 = tok0[b];
        verify_one(mode,
                   target_logits + row0[b] * vocab,
                   draft_logits ? draft_logits + t0 * vocab : NULL,
                   draft_tokens + t0, draft_len[b], vocab, temperatures ? temperatures[b] : temperature, top_k, top_p,
                   seeds ? seeds[b] : 0,
                   vocab_mask ? vocab_mask + (int64_t)b * mask_words : NULL,
                   topp_margin ? topp_margin + row0[b] : NULL,
                   accepted_len + b, next_token + b,
                   p_tok ? p_tok + t0 : NULL, q_tok ? q_tok + t0 : NULL,
                   u_acc ? u_acc + t0 : NULL, acc_margin ? acc_margin + t0 : NULL,
                   cdf_margin ? cdf_margin + b : NULL, resid_mass ? resid_mass + b : NULL);
    }
    free(row0); free(tok0);
}

/* ------------------------------------------------------------ KV session */

void fso_kv_append(uint16_t* kv_pages, const int32_t* page_table, int32_t max_pages_per_seq,
                   const int32_t* kv_len, const int32_t* draft_len, int32_t batch,
                   int32_t n_kv_heads, int32_t head_dim, int32_t page_size,
                   const uint16_t* new_k, const uint16_t* new_v)
{
    int64_t row = 0;
    for (int32_t b = 0; b < batch; ++b) {
        const int32_t k = draft_len[b];
        const int32_t ctx = kv_len[b] - (k + 1);
        for (int32_t j = 0; j <= k; ++j, ++row) {
            const int32_t t = ctx + j;
            const int64_t page = page_table[(int64_t)b * max_pages_per_seq + t / page_size];
            const int32_t slot = t % page_size;
            for (int32_t h = 0; h < n_kv_heads; ++h)
                for (int32_t e = 0; e < head_dim; ++e) {
                    const int64_t src = (row * n_kv_heads + h) * head_dim + e;
                    kv_pages[(((page * 2 + 0) * n_kv_heads + h) * page_size + slot) * (int64_t)head_dim + e] = new_k[src];
                    kv_pages[(((page * 2 + 1) * n_kv_heads + h) * page_size + slot) * (int64_t)head_dim + e] = new_v[src];
                }
        }
    }
}

void fso_kv_rollback(const int32_t* kv_len, const int32_t* draft_len, const int32_t* accepted_len,
                     int32_t batch, int32_t* kv_len_next)
{
    for (int32_t b = 0; b < batch; ++b) {
        const int32_t ctx = kv_len[b] - (draft_len[b] + 1);
        kv_len_next[b] = ctx + accepted_len[b] + 1;
    }
}

void fso_kv_release(int32_t* page_table, int32_t max_pages_per_seq, const int32_t* kv_len_prev,
                    const int32_t* kv_len_next, int32_t batch, int32_t page_size,
                    int32_t* free_list, int32_t* free_count)
{
    for (int32_t b = 0; b < batch; ++b) {
        const int32_t keep = (kv_len_next[b] + page_size - 1) / page_size;   /* pages that still hold valid tokens */
        const int32_t had = (kv_len_prev[b] + page_size - 1) / page_size;
        for (int32_t i = keep; i < had; ++i) {
            int32_t* e = page_table + (int64_t)b * max_pages_per_seq + i;
            free_list[(*free_count)++] = *e;
            *e = -1;
        }
    }
}

int32_t fso_num_threads(void)
{
#ifdef _OPENMP
    return (int32_t)omp_get_max_threads();
#else
    return 1;
#endif
}
