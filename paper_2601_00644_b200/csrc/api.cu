// Host layer of the C ABI declared in include/flexspec.h: argument validation, workspace,
// TMA descriptors, launch sequencing.  No step of the verification runs on the host.
#include <math.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <new>

#include <nvtx3/nvToolsExt.h>

#include "internal.h"

using namespace fs;

struct flexspec_handle {
    Handle h;
};

namespace {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// The driver entry point is looked up at run time so that the library loads (and its symbols
// can be inspected) on a machine without a GPU driver.
EncodeTiledFn encode_tiled_fn()
{
    static EncodeTiledFn fn = nullptr;
    if (fn == nullptr) {
        void* ptr = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(ptr);
    }
    return fn;
}

// 2-D bf16 row-major tensor [rows][cols], box [box_rows][64 cols], 128-byte swizzle, zero fill.
int make_map_2d(CUtensorMap* map, const void* base, uint64_t rows, uint64_t cols, uint32_t box_rows)
{
    EncodeTiledFn fn = encode_tiled_fn();
    if (fn == nullptr) return FLEXSPEC_ERR_NO_DEVICE;
    cuuint64_t dims[2] = {cols, rows};
    cuuint64_t strides[1] = {cols * 2};
    cuuint32_t box[2] = {64, box_rows};
    cuuint32_t elem[2] = {1, 1};
    CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, elem,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? FLEXSPEC_OK : FLEXSPEC_ERR_CUDA;
}

template <typename T>
int dev_alloc(T** p, size_t count)
{
    *p = nullptr;
    if (count == 0) count = 1;
    cudaError_t e = cudaMalloc(reinterpret_cast<void**>(p), count * sizeof(T));
    if (e != cudaSuccess) { cudaGetLastError(); return FLEXSPEC_ERR_OOM; }
    return FLEXSPEC_OK;
}

// Named range on the host timeline (header-only NVTX: a no-op unless a profiler is attached).
struct NvtxRange {
    explicit NvtxRange(const char* name) { nvtxRangePushA(name); }
    ~NvtxRange() { nvtxRangePop(); }
};

struct DeviceGuard {
    int prev = -1;
    bool ok = false;
    explicit DeviceGuard(int dev)
    {
        if (cudaGetDevice(&prev) != cudaSuccess) { cudaGetLastError(); prev = -1; }
        ok = (cudaSetDevice(dev) == cudaSuccess);
        if (!ok) cudaGetLastError();
    }
    ~DeviceGuard() { if (prev >= 0) cudaSetDevice(prev); }
};

void free_workspace(Handle& h)
{
    cudaFree(h.attn_out); cudaFree(h.logits); cudaFree(h.part_o); cudaFree(h.part_ml); cudaFree(h.att_tickets);
    cudaFree(h.plan.cu_q); cudaFree(h.plan.cu_d); cudaFree(h.plan.row_seq); cudaFree(h.plan.k_eff); cudaFree(h.plan.row_c);
    cudaFree(h.stats); cudaFree(h.tstats); cudaFree(h.topp); cudaFree(h.w_tiled);
    cudaFree(h.dbg_p); cudaFree(h.dbg_q); cudaFree(h.dbg_u); cudaFree(h.status);
    cudaFree(h.stage_dev); cudaFree(h.out_dev);
    if (h.out_host) cudaFreeHost(h.out_host);
    for (int i = 0; i < kNumStageEvents; ++i)
        if (h.ev[i]) cudaEventDestroy(h.ev[i]);
    if (h.ev_fork) cudaEventDestroy(h.ev_fork);
    if (h.ev_join) cudaEventDestroy(h.ev_join);
    if (h.ev_plan) cudaEventDestroy(h.ev_plan);
    if (h.side) cudaStreamDestroy(h.side);
    free(h.att_seq);
    h.att_seq = nullptr;
}

// geometry of one call, derived from the host copies of the lengths
struct Geometry {
    int32_t m_rows = 0, s_rows = 0, k_batch_max = 0, kv_max = 0;
    int64_t att_blocks = 0;      // attention work blocks (128 tokens of one (sequence, kv head, row block) pair)
};

int check_lengths(const Handle& h, const int32_t* draft_len_host, const int32_t* kv_len_host, int32_t batch,
                  int32_t max_pages_per_seq, Geometry* g)
{
    if (batch < 1 || batch > h.cfg.max_batch || draft_len_host == nullptr) return FLEXSPEC_ERR_INVALID_ARG;
    for (int b = 0; b < batch; ++b) {
        const int k = draft_len_host[b];
        if (k < 0 || k > h.cfg.k_max) return FLEXSPEC_ERR_INVALID_ARG;
        g->m_rows += k + 1;
        g->s_rows += k;
        if (k > g->k_batch_max) g->k_batch_max = k;
        if (kv_len_host != nullptr) {
            const int l = kv_len_host[b];
            if (l < k + 1 || l > h.cfg.max_kv_len) return FLEXSPEC_ERR_INVALID_ARG;
            if ((l + h.cfg.page_size - 1) / h.cfg.page_size > max_pages_per_seq) return FLEXSPEC_ERR_INVALID_ARG;
            if (l > g->kv_max) g->kv_max = l;
            const int group = h.cfg.n_q_heads / h.cfg.n_kv_heads;
            const int64_t pairs = static_cast<int64_t>(h.cfg.n_kv_heads) *
                                  ((group * (k + 1) + kAttRowsPerPair - 1) / kAttRowsPerPair);
            g->att_blocks += pairs * ((l + kAttBlockTokens - 1) / kAttBlockTokens);
        }
    }
    if (g->att_blocks > 0x7fffffffLL) return FLEXSPEC_ERR_UNSUPPORTED;
    return FLEXSPEC_OK;
}

// ---------------------------------------------------------------------------------------------
// Attention work list.  All 128-token blocks of all (sequence, kv head, row block) pairs, numbered
// sequence by sequence and pair by pair, are cut into one contiguous range per CTA.  Two cuts are
// built and the cheaper one is taken:
//   balanced  : equal ranges (a pair may straddle CTAs; its parts are merged in the kernel);
//   pair-wise : every CTA takes whole pairs, under the smallest capacity that needs no more CTAs than
//               there are SMs (no pair is split, so nothing is merged).
// Cost of a CTA, in microseconds from per-CTA timelines of the kernel: its blocks x the block period
// for the tile width, a pipeline drain / refill per further segment, and the park-and-merge tail
// if one of its segments is part of a split pair.
int32_t pairwise_ctas(const SeqBlocks* sq, int32_t batch, int64_t cap, int32_t* begins, int32_t max_ctas)
{
    // greedy: walk the pairs in order, open a new CTA when the next pair does not fit; returns the CTAs used
    int32_t used = 0;
    int64_t load = 0, pos = 0;
    for (int b = 0; b < batch; ++b) {
        for (int pr = 0; pr < sq[b].pairs; ++pr) {
            if (used == 0 || load + sq[b].nb > cap) {
                if (used == max_ctas) return max_ctas + 1;
                if (begins != nullptr) begins[used] = static_cast<int32_t>(pos);
                ++used;
                load = 0;
            }
            load += sq[b].nb;
            pos += sq[b].nb;
        }
    }
    return used;
}

double cut_cost(const SeqBlocks* sq, int32_t batch, const int32_t* begins, int32_t n_ctas, int64_t total, double t_blk)
{
    const double t_seg = 4.0, t_split = 7.5;
    double worst = 0.0;
    int b = 0;
    int64_t seq0 = 0;                                    // first block of sequence b
    for (int c = 0; c < n_ctas; ++c) {
        const int64_t lo = begins[c], hi = (c + 1 < n_ctas) ? begins[c + 1] : total;
        while (seq0 + static_cast<int64_t>(sq[b].pairs) * sq[b].nb <= lo) { seq0 += static_cast<int64_t>(sq[b].pairs) * sq[b].nb; ++b; }
        // segments of [lo, hi): walk the pairs it touches
        int segs = 0;
        bool split = false;
        int bb = b;
        int64_t s0 = seq0, x = lo;
        while (x < hi) {
            const int64_t in_seq = x - s0;
            const int64_t pair_lo = s0 + in_seq / sq[bb].nb * sq[bb].nb, pair_hi = pair_lo + sq[bb].nb;
            ++segs;
            if (pair_lo < lo || pair_hi > hi) split = true;
            x = pair_hi < hi ? pair_hi : hi;
            if (x >= s0 + static_cast<int64_t>(sq[bb].pairs) * sq[bb].nb) { s0 += static_cast<int64_t>(sq[bb].pairs) * sq[bb].nb; ++bb; }
        }
        const double cost = static_cast<double>(hi - lo) * t_blk + (segs > 1 ? (segs - 1) * t_seg : 0.0) + (split ? t_split : 0.0);
        if (cost > worst) worst = cost;
    }
    return worst;
}

int plan_attention(const Handle& h, const int32_t* draft_len_host, const int32_t* kv_len_host, int32_t batch,
                   const Geometry& g, int32_t n_pad, AttTable* tab, int32_t* n_ctas_out)
{
    const flexspec_config& c = h.cfg;
    const int group = c.n_q_heads / c.n_kv_heads;
    SeqBlocks* sq = h.att_seq;                           // host scratch of the handle, max_batch entries
    int32_t max_nb = 0;
    for (int b = 0; b < batch; ++b) {
        const int k = draft_len_host[b];
        sq[b].pairs = c.n_kv_heads * ((group * (k + 1) + kAttRowsPerPair - 1) / kAttRowsPerPair);
        sq[b].nb = (kv_len_host[b] + kAttBlockTokens - 1) / kAttBlockTokens;
        sq[b].rows = k + 1;
        if (sq[b].nb > max_nb) max_nb = sq[b].nb;
    }
    const int64_t total = g.att_blocks;
    int32_t max_ctas = h.sm_count < kAttMaxCtas ? h.sm_count : kAttMaxCtas;
    if (total < max_ctas) max_ctas = static_cast<int32_t>(total);
    const double t_blk = n_pad <= 32 ? 1.7 : (n_pad <= 64 ? 2.4 : (n_pad <= 96 ? 3.5 : 4.5));

    int32_t begins_a[kAttMaxCtas], begins_b[kAttMaxCtas];
    // balanced
    const int32_t n_a = max_ctas;
    for (int cta = 0; cta < n_a; ++cta) begins_a[cta] = static_cast<int32_t>(cta * total / n_a);
    const double cost_a = cut_cost(sq, batch, begins_a, n_a, total, t_blk);
    // pair-wise: smallest capacity (bisection) that fits into max_ctas CTAs
    int64_t lo = max_nb, hi = total;
    while (lo < hi) {
        const int64_t mid = (lo + hi) / 2;
        if (pairwise_ctas(sq, batch, mid, nullptr, max_ctas) <= max_ctas) hi = mid; else lo = mid + 1;
    }
    const int32_t n_b = pairwise_ctas(sq, batch, lo, begins_b, max_ctas);
    const double cost_b = (n_b <= max_ctas) ? cut_cost(sq, batch, begins_b, n_b, total, t_blk) : 1e300;
    const bool use_b = cost_b < cost_a;
    const int32_t* begins = use_b ? begins_b : begins_a;
    const int32_t n_ctas = use_b ? n_b : n_a;

    // fill the table: one pass over the sequences
    int b = 0;
    int64_t seq0 = 0;
    int32_t row0 = 0, pair0 = 0;
    for (int cta = 0; cta < n_ctas; ++cta) {
        const int64_t x = begins[cta];
        while (seq0 + static_cast<int64_t>(sq[b].pairs) * sq[b].nb <= x) {
            seq0 += static_cast<int64_t>(sq[b].pairs) * sq[b].nb;
            row0 += sq[b].rows; pair0 += sq[b].pairs;
            ++b;
        }
        AttCta& e = tab->cta[cta];
        e.blk_begin = static_cast<int32_t>(x);
        e.n_my = static_cast<int32_t>(((cta + 1 < n_ctas) ? begins[cta + 1] : total) - x);
        e.b = b; e.blk_off = static_cast<int32_t>(x - seq0);
        e.q_row0 = row0; e.pair0 = pair0; e.blk0 = static_cast<int32_t>(seq0);
        e.k = draft_len_host[b]; e.kvl = kv_len_host[b]; e.pad = 0;
    }
    *n_ctas_out = n_ctas;
    return FLEXSPEC_OK;
}

void mark(Handle& h, int idx, cudaStream_t s)
{
    if (h.profiling) { cudaEventRecord(h.ev[idx], s); h.ev_used[idx] = 1; }
}

int run_plan(Handle& h, const int32_t* draft_len, const int32_t* draft_tokens, int32_t batch, const Geometry& g,
             const SampleParams& sp, cudaStream_t s)
{
    if (launch_plan(draft_len, draft_tokens, batch, h.cfg.vocab, g.m_rows, g.s_rows, g.k_batch_max, sp.temps,
                    sp.inv_temp_log2, h.plan, h.status, s) != cudaSuccess)
        return FLEXSPEC_ERR_CUDA;
    h.launches++;
    return FLEXSPEC_OK;
}

int run_attention(Handle& h, const flexspec_kv* kv, const void* hidden, const int32_t* draft_len,
                  const int32_t* draft_len_host, const Geometry& g, int32_t batch, void* attn_out, cudaStream_t s)
{
    const flexspec_config& c = h.cfg;
    const int group = c.n_q_heads / c.n_kv_heads;
    // one tensor map over the whole pool: rows of head_dim bf16
    CUtensorMap kv_map;
    const uint64_t pool_rows = static_cast<uint64_t>(kv->num_pages) * 2 * c.n_kv_heads * c.page_size;
    int rc = make_map_2d(&kv_map, kv->kv_pages, pool_rows, static_cast<uint64_t>(c.head_dim), 16);
    if (rc != FLEXSPEC_OK) return rc;

    AttnParams p;
    p.m_rows = g.m_rows; p.k_cap = g.k_batch_max; p.kv_cap = g.kv_max;
    p.hidden = static_cast<const __nv_bfloat16*>(hidden);
    p.page_table = kv->page_table;
    p.kv_len = kv->kv_len;
    p.draft_len = draft_len;
    p.batch = batch;
    p.n_q_heads = c.n_q_heads; p.n_kv_heads = c.n_kv_heads; p.group = group;
    p.max_pages_per_seq = kv->max_pages_per_seq; p.num_pages = kv->num_pages;
    const int rows_max = group * (g.k_batch_max + 1) < kAttRowsPerPair ? group * (g.k_batch_max + 1) : kAttRowsPerPair;
    p.n_pad = (rows_max + 15) / 16 * 16;
    p.p_bufs = attention_p_bufs(p.n_pad);
    attention_stages(c.head_dim, p.n_pad, &p.k_stages, &p.v_stages);
    if (p.k_stages < 1 || p.v_stages < 2) return FLEXSPEC_ERR_UNSUPPORTED;
    p.scale_log2 = static_cast<float>(1.4426950408889634 / sqrt(static_cast<double>(c.head_dim)));
    p.part_o = h.part_o; p.part_ml = h.part_ml; p.tickets = h.att_tickets;
    p.attn_out = static_cast<__nv_bfloat16*>(attn_out);
    p.status = h.status;
    AttTable tab;
    int32_t n_ctas = 0;
    rc = plan_attention(h, draft_len_host, kv->kv_len_host, batch, g, p.n_pad, &tab, &n_ctas);
    if (rc != FLEXSPEC_OK) return rc;
    if (launch_attention(h, kv_map, p, tab, n_ctas, s) != cudaSuccess) return FLEXSPEC_ERR_CUDA;
    h.launches++;
    return FLEXSPEC_OK;
}

int run_lm_head(Handle& h, const void* x, int32_t m_rows, float* logits, const SampleParams* sp, cudaStream_t s)
{
    const flexspec_config& c = h.cfg;
    LmHeadParams p;
    p.logits = logits;
    p.m_rows = m_rows; p.vocab = c.vocab; p.d_model = h.d_model;
    const int m16 = (m_rows + 15) / 16 * 16;
    if (m16 <= 256) { p.n_tile = m16; p.n_blocks = 1; }
    else if (m16 <= 512) { p.n_blocks = 2; p.n_tile = ((m_rows + 1) / 2 + 15) / 16 * 16; }   // two blocks that just cover the rows
    else { p.n_tile = 256; p.n_blocks = 2; }
    const int rows_per_pass = p.n_tile * p.n_blocks;
    p.n_pass = (m_rows + rows_per_pass - 1) / rows_per_pass;
    p.n_full_tiles = h.lm_full_tiles; p.last_rows = h.lm_last_rows; p.n_vtiles = h.lm_full_tiles + h.lm_last_tiles;
    p.num_stages = lm_head_pick_stages(p.n_tile, p.n_blocks);
    p.n_bufs = 512 / p.n_tile < 4 ? 512 / p.n_tile : 4;       // what fits into the 512 TMEM columns, four at most
    p.tstats = nullptr; p.n_tparts = 0; p.inv_temp_log2 = 1.f; p.greedy = 0;
    p.row_seq = nullptr; p.vocab_mask = nullptr; p.mask_words = 0; p.row_c = nullptr;
    if (sp != nullptr) {
        p.tstats = h.tstats; p.n_tparts = 4 * p.n_vtiles; p.inv_temp_log2 = sp->inv_temp_log2; p.greedy = sp->greedy;
        p.row_seq = sp->row_seq; p.vocab_mask = sp->vocab_mask; p.mask_words = sp->mask_words;
        p.row_c = sp->temps != nullptr ? sp->row_c : nullptr;
    }
    p.status = h.status;
    CUtensorMap x_map;
    int rc = make_map_2d(&x_map, x, static_cast<uint64_t>(m_rows), static_cast<uint64_t>(h.d_model),
                         static_cast<uint32_t>(p.n_tile));
    if (rc != FLEXSPEC_OK) return rc;
    if (launch_lm_head(h, x_map, p, s) != cudaSuccess) return FLEXSPEC_ERR_CUDA;
    h.launches++;
    return FLEXSPEC_OK;
}

void fill_sample_params(Handle& h, SampleParams& p, const float* logits, const int32_t* draft_tokens,
                        const float* draft_logits, const int32_t* draft_len, const uint64_t* seeds, const Geometry& g,
                        int32_t batch, float temperature, const uint32_t* vocab_mask, int32_t* accepted_len,
                        int32_t* next_token)
{
    const flexspec_config& c = h.cfg;
    memset(&p, 0, sizeof(p));
    p.greedy = (c.mode == FLEXSPEC_MODE_GREEDY || temperature == 0.f) ? 1 : 0;
    p.logits = logits; p.draft_logits = draft_logits; p.draft_tokens = draft_tokens;
    p.draft_len = draft_len; p.seeds = seeds; p.vocab_mask = vocab_mask;
    p.cu_q = h.plan.cu_q; p.cu_d = h.plan.cu_d; p.row_seq = h.plan.row_seq; p.k_eff = h.plan.k_eff;
    p.row_c = h.plan.row_c; p.temps = p.greedy ? nullptr : h.temps;
    p.batch = batch; p.vocab = c.vocab; p.m_rows = g.m_rows; p.s_rows = g.s_rows;
    p.n_chunks = (c.vocab + kSampleChunk - 1) / kSampleChunk;
    p.mask_words = (c.vocab + 31) / 32;
    p.inv_temp_log2 = p.greedy ? 1.f : static_cast<float>(1.4426950408889634 / static_cast<double>(temperature));
    p.stats = h.stats;
    p.tstats = h.stats; p.n_tparts = p.n_chunks;          // target parts from the statistics kernel unless the LM head wrote them
    p.top_p = p.greedy ? 1.f : h.top_p; p.top_k = p.greedy ? 0 : h.top_k; p.topp = h.topp;
    p.filtered = (p.top_p < 1.f || (p.top_k > 0 && p.top_k < c.vocab)) ? 1 : 0;
    p.accepted_len = accepted_len; p.next_token = next_token;
    if (c.flags & FLEXSPEC_FLAG_DEBUG) { p.dbg_p = h.dbg_p; p.dbg_q = h.dbg_q; p.dbg_u = h.dbg_u; }
    p.status = h.status;
}

// the whole stage on one stream: statistics of every row, decision, draw
int run_sample(Handle& h, const float* logits, const int32_t* draft_tokens, const float* draft_logits,
               const int32_t* draft_len, const uint64_t* seeds, const Geometry& g, int32_t batch,
               float temperature, const uint32_t* vocab_mask, int32_t* accepted_len, int32_t* next_token,
               cudaStream_t s)
{
    SampleParams p;
    fill_sample_params(h, p, logits, draft_tokens, draft_logits, draft_len, seeds, g, batch, temperature, vocab_mask,
                       accepted_len, next_token);
    if (launch_sample_stats(p, 0, p.greedy ? p.m_rows : p.m_rows + p.s_rows, s) != cudaSuccess) return FLEXSPEC_ERR_CUDA;
    h.launches++;
    if (p.filtered) {
        if (launch_sample_filter(p, false, s) != cudaSuccess) return FLEXSPEC_ERR_CUDA;
        h.launches++;
    }
    if (launch_sample_accept(p, false, s) != cudaSuccess) return FLEXSPEC_ERR_CUDA;
    h.launches++;
    return FLEXSPEC_OK;
}

// The sampling kernels read the logit rows with 16-byte loads when the vocabulary is a multiple of
// four (every row then starts on a 16-byte boundary if the array does); otherwise with 4-byte loads.
bool logits_aligned(const void* ptr, int32_t vocab)
{
    return (reinterpret_cast<uintptr_t>(ptr) & ((vocab & 3) == 0 ? 15u : 3u)) == 0;
}

bool sample_args_ok(const Handle& h, const int32_t* draft_tokens, const float* draft_logits,
                    const uint64_t* seeds, float temperature, const Geometry& g)
{
    const bool greedy = (h.cfg.mode == FLEXSPEC_MODE_GREEDY || temperature == 0.f);
    if (!(temperature >= 0.f) || isinf(temperature)) return false;
    if (g.s_rows > 0 && draft_tokens == nullptr) return false;
    if (!greedy && (seeds == nullptr || (g.s_rows > 0 && draft_logits == nullptr))) return false;
    return true;
}

}  // namespace

extern "C" {

int flexspec_create(const flexspec_config* cfg, const void* lm_head_w, flexspec_handle** out)
{
    if (out == nullptr) return FLEXSPEC_ERR_INVALID_ARG;
    *out = nullptr;
    if (cfg == nullptr || lm_head_w == nullptr) return FLEXSPEC_ERR_INVALID_ARG;
    const flexspec_config& c = *cfg;
    if (c.n_q_heads < 1 || c.n_kv_heads < 1 || c.vocab < 1 || c.max_batch < 1 || c.k_max < 0 ||
        c.max_kv_len < 1 || c.device < 0)
        return FLEXSPEC_ERR_INVALID_ARG;
    if (c.mode != FLEXSPEC_MODE_SAMPLE && c.mode != FLEXSPEC_MODE_GREEDY) return FLEXSPEC_ERR_INVALID_ARG;
    if (c.n_q_heads % c.n_kv_heads != 0) return FLEXSPEC_ERR_INVALID_ARG;
    if (c.max_kv_len < c.k_max + 1) return FLEXSPEC_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(lm_head_w) & 15u) != 0) return FLEXSPEC_ERR_INVALID_ARG;
    if (c.head_dim != 64 && c.head_dim != 128) return FLEXSPEC_ERR_UNSUPPORTED;
    if (c.page_size != 16) return FLEXSPEC_ERR_UNSUPPORTED;
    if (c.max_batch > kMaxBatch || c.k_max > kMaxK) return FLEXSPEC_ERR_UNSUPPORTED;
    const int64_t d_model = static_cast<int64_t>(c.n_q_heads) * c.head_dim;
    if (d_model % 64 != 0 || d_model > 65536) return FLEXSPEC_ERR_UNSUPPORTED;
    const int64_t max_m = static_cast<int64_t>(c.max_batch) * (c.k_max + 1);
    if (max_m * c.vocab > (1LL << 40) || c.vocab > kMaxVocab) return FLEXSPEC_ERR_UNSUPPORTED;

    int n_dev = 0;
    if (cudaGetDeviceCount(&n_dev) != cudaSuccess || c.device >= n_dev) { cudaGetLastError(); return FLEXSPEC_ERR_NO_DEVICE; }
    DeviceGuard guard(c.device);
    if (!guard.ok) return FLEXSPEC_ERR_NO_DEVICE;
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, c.device) != cudaSuccess) return FLEXSPEC_ERR_CUDA;
    if (prop.major != 10) return FLEXSPEC_ERR_UNSUPPORTED;       // kernels are built for sm_100a only

    flexspec_handle* fh = new (std::nothrow) flexspec_handle();
    if (fh == nullptr) return FLEXSPEC_ERR_OOM;
    Handle& h = fh->h;
    memset(&h, 0, sizeof(h));
    h.cfg = c;
    h.d_model = static_cast<int32_t>(d_model);
    h.max_m = static_cast<int32_t>(max_m);
    h.max_s = c.max_batch * c.k_max;
    h.sm_count = prop.multiProcessorCount;
    h.top_p = 1.f;
    h.att_seq = static_cast<SeqBlocks*>(malloc(sizeof(SeqBlocks) * static_cast<size_t>(c.max_batch)));
    if (h.att_seq == nullptr) { delete fh; return FLEXSPEC_ERR_OOM; }

    const int n_chunks = (c.vocab + kSampleChunk - 1) / kSampleChunk;
    // LM-head tiling: full waves of 128-row tiles, then one wave of shorter tiles, one per SM, so that
    // the last wave ends everywhere at the same time
    {
        const int tiles128 = (c.vocab + 127) / 128;
        h.lm_full_tiles = tiles128; h.lm_last_rows = 128; h.lm_last_tiles = 0;
        if (tiles128 > h.sm_count && tiles128 % h.sm_count != 0) {
            h.lm_full_tiles = tiles128 / h.sm_count * h.sm_count;
            const int rows_rem = c.vocab - h.lm_full_tiles * 128;
            int lr = (rows_rem + h.sm_count - 1) / h.sm_count;
            if (lr > 128) lr = 128;
            h.lm_last_rows = lr;
            h.lm_last_tiles = (rows_rem + lr - 1) / lr;
        }
    }
    int rc = FLEXSPEC_OK;
    auto A = [&](int r) { if (rc == FLEXSPEC_OK) rc = r; };
    A(dev_alloc(&h.attn_out, static_cast<size_t>(max_m) * d_model));
    A(dev_alloc(&h.logits, static_cast<size_t>(max_m) * c.vocab));
    // attention partial slots: one per (pair, CTA) segment, index pair + CTA
    const int group = c.n_q_heads / c.n_kv_heads;
    h.att_pairs_max = c.max_batch * c.n_kv_heads * ((group * (c.k_max + 1) + kAttRowsPerPair - 1) / kAttRowsPerPair);
    // split-merge scratch: every CTA parks at most its first and its last segment
    const size_t att_slots = static_cast<size_t>(2) * h.sm_count;
    A(dev_alloc(&h.part_o, att_slots * kAttRowsPerPair * c.head_dim));
    A(dev_alloc(&h.part_ml, att_slots * 4 * kAttRowsPerPair * 2));
    A(dev_alloc(&h.att_tickets, static_cast<size_t>(h.att_pairs_max) * 12));
    A(dev_alloc(&h.plan.cu_q, static_cast<size_t>(c.max_batch) + 1));
    A(dev_alloc(&h.plan.cu_d, static_cast<size_t>(c.max_batch) + 1));
    A(dev_alloc(&h.plan.row_seq, static_cast<size_t>(max_m)));
    A(dev_alloc(&h.plan.k_eff, static_cast<size_t>(c.max_batch)));
    A(dev_alloc(&h.plan.row_c, static_cast<size_t>(max_m) + h.max_s));
    A(dev_alloc(&h.stats, static_cast<size_t>(max_m + h.max_s) * n_chunks));
    A(dev_alloc(&h.tstats, static_cast<size_t>(max_m) * 4 * ((c.vocab + 127) / 128 + h.sm_count)));
    A(dev_alloc(&h.topp, static_cast<size_t>(max_m) * 2));
    A(dev_alloc(&h.dbg_p, static_cast<size_t>(h.max_s)));
    A(dev_alloc(&h.dbg_q, static_cast<size_t>(h.max_s)));
    A(dev_alloc(&h.dbg_u, static_cast<size_t>(h.max_s)));
    A(dev_alloc(&h.status, 4));
    A(dev_alloc(&h.out_dev, static_cast<size_t>(2) * c.max_batch));
    if (rc == FLEXSPEC_OK && cudaMallocHost(reinterpret_cast<void**>(&h.out_host), static_cast<size_t>(2) * c.max_batch * sizeof(int32_t)) != cudaSuccess) {
        cudaGetLastError();
        h.out_host = nullptr;
        rc = FLEXSPEC_ERR_OOM;
    }
    if (rc == FLEXSPEC_OK) {
        // staging for flexspec_verify_host: hidden | draft logits | tokens | lengths (2) | seeds
        h.stage_bytes = static_cast<size_t>(max_m) * d_model * 2 + static_cast<size_t>(h.max_s) * c.vocab * 4 +
                        static_cast<size_t>(h.max_s) * 4 + static_cast<size_t>(c.max_batch) * (4 + 4 + 8) +
                        static_cast<size_t>(c.max_batch) * ((c.vocab + 31) / 32) * 4 + 4096;
        if (cudaMalloc(&h.stage_dev, h.stage_bytes) != cudaSuccess) { cudaGetLastError(); rc = FLEXSPEC_ERR_OOM; }
    }
    if (rc == FLEXSPEC_OK) {
        if (cudaMemset(h.att_tickets, 0, sizeof(int32_t) * static_cast<size_t>(h.att_pairs_max) * 12) != cudaSuccess ||
            cudaMemset(h.status, 0, sizeof(int32_t) * 4) != cudaSuccess)
            rc = FLEXSPEC_ERR_CUDA;
    }
    for (int i = 0; i < kNumStageEvents && rc == FLEXSPEC_OK; ++i)
        if (cudaEventCreate(&h.ev[i]) != cudaSuccess) rc = FLEXSPEC_ERR_CUDA;
    if (rc == FLEXSPEC_OK &&
        (cudaStreamCreateWithFlags(&h.side, cudaStreamNonBlocking) != cudaSuccess ||
         cudaEventCreateWithFlags(&h.ev_fork, cudaEventDisableTiming) != cudaSuccess ||
         cudaEventCreateWithFlags(&h.ev_join, cudaEventDisableTiming) != cudaSuccess ||
         cudaEventCreateWithFlags(&h.ev_plan, cudaEventDisableTiming) != cudaSuccess))
        rc = FLEXSPEC_ERR_CUDA;
    // W is copied once into the order the LM head streams it (a stage of its pipeline = one contiguous block);
    // the caller's buffer is not needed afterwards
    const uint64_t w_rows = static_cast<uint64_t>(h.lm_full_tiles) * 128 + static_cast<uint64_t>(h.lm_last_tiles) * h.lm_last_rows;
    A(dev_alloc(&h.w_tiled, static_cast<size_t>(w_rows) * d_model));
    if (rc == FLEXSPEC_OK &&
        (launch_retile_w(lm_head_w, h.w_tiled, c.vocab, d_model, h.lm_full_tiles, h.lm_last_tiles, h.lm_last_rows, nullptr) != cudaSuccess ||
         cudaStreamSynchronize(nullptr) != cudaSuccess))
        rc = FLEXSPEC_ERR_CUDA;
    if (rc == FLEXSPEC_OK) rc = make_map_2d(&h.w_map, h.w_tiled, w_rows * (d_model / 64), 64, 128);
    if (rc == FLEXSPEC_OK) rc = make_map_2d(&h.w_map_last, h.w_tiled, w_rows * (d_model / 64), 64, static_cast<uint32_t>(h.lm_last_rows));
    if (rc == FLEXSPEC_OK && (attention_init(c.head_dim) != cudaSuccess || lm_head_init() != cudaSuccess || sample_init() != cudaSuccess))
        rc = FLEXSPEC_ERR_CUDA;
    if (rc != FLEXSPEC_OK) {
        cudaGetLastError();
        free_workspace(h);
        delete fh;
        return rc;
    }
    *out = fh;
    return FLEXSPEC_OK;
}

int flexspec_destroy(flexspec_handle* fh)
{
    if (fh == nullptr) return FLEXSPEC_OK;
    DeviceGuard guard(fh->h.cfg.device);
    cudaDeviceSynchronize();
    free_workspace(fh->h);
    delete fh;
    return FLEXSPEC_OK;
}

static int kv_args_ok(const Handle& h, const flexspec_kv* kv, bool need_dev_len)
{
    if (kv == nullptr || kv->kv_pages == nullptr || kv->page_table == nullptr || kv->kv_len_host == nullptr)
        return 0;
    if (need_dev_len && kv->kv_len == nullptr) return 0;
    if (kv->num_pages < 1 || kv->max_pages_per_seq < 1) return 0;
    if ((reinterpret_cast<uintptr_t>(kv->kv_pages) & 15u) != 0) return 0;
    if (static_cast<int64_t>(kv->num_pages) * 2 * h.cfg.n_kv_heads * h.cfg.page_size > 0x7fffffffLL) return 0;
    return 1;
}

int flexspec_attention(flexspec_handle* fh, const flexspec_kv* kv, const void* hidden,
                       const int32_t* draft_len, const int32_t* draft_len_host, int32_t batch,
                       void* attn_out, void* stream)
{
    NvtxRange nvtx_range("flexspec_attention");
    if (fh == nullptr || hidden == nullptr || draft_len == nullptr) return FLEXSPEC_ERR_INVALID_ARG;
    Handle& h = fh->h;
    if (!kv_args_ok(h, kv, true)) return FLEXSPEC_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(hidden) & 15u) != 0) return FLEXSPEC_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(attn_out) & 15u) != 0) return FLEXSPEC_ERR_INVALID_ARG;
    Geometry g;
    int rc = check_lengths(h, draft_len_host, kv->kv_len_host, batch, kv->max_pages_per_seq, &g);
    if (rc != FLEXSPEC_OK) return rc;
    DeviceGuard guard(h.cfg.device);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    h.launches = 0;
    return run_attention(h, kv, hidden, draft_len, draft_len_host, g, batch, attn_out ? attn_out : h.attn_out, s);
}

int flexspec_lm_head(flexspec_handle* fh, const void* x, int32_t m_rows, float* logits, void* stream)
{
    NvtxRange nvtx_range("flexspec_lm_head");
    if (fh == nullptr) return FLEXSPEC_ERR_INVALID_ARG;
    Handle& h = fh->h;
    if (m_rows < 1 || m_rows > h.max_m) return FLEXSPEC_ERR_INVALID_ARG;
    if (x != nullptr && (reinterpret_cast<uintptr_t>(x) & 15u) != 0) return FLEXSPEC_ERR_INVALID_ARG;
    DeviceGuard guard(h.cfg.device);
    h.launches = 0;
    return run_lm_head(h, x ? x : h.attn_out, m_rows, logits ? logits : h.logits, nullptr, static_cast<cudaStream_t>(stream));
}

int flexspec_sample(flexspec_handle* fh, const float* logits, const int32_t* draft_tokens,
                    const float* draft_logits, const int32_t* draft_len, const int32_t* draft_len_host,
                    const uint64_t* seeds, int32_t batch, float temperature, const uint32_t* vocab_mask,
                    int32_t* accepted_len, int32_t* next_token, void* stream)
{
    NvtxRange nvtx_range("flexspec_sample");
    if (fh == nullptr || draft_len == nullptr || accepted_len == nullptr || next_token == nullptr)
        return FLEXSPEC_ERR_INVALID_ARG;
    Handle& h = fh->h;
    Geometry g;
    int rc = check_lengths(h, draft_len_host, nullptr, batch, 0, &g);
    if (rc != FLEXSPEC_OK) return rc;
    if (!sample_args_ok(h, draft_tokens, draft_logits, seeds, temperature, g)) return FLEXSPEC_ERR_INVALID_ARG;
    if (!logits_aligned(logits, h.cfg.vocab) || !logits_aligned(draft_logits, h.cfg.vocab)) return FLEXSPEC_ERR_INVALID_ARG;
    DeviceGuard guard(h.cfg.device);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    h.launches = 0;
    {
        SampleParams sp0;
        fill_sample_params(h, sp0, logits ? logits : h.logits, draft_tokens, draft_logits, draft_len, seeds, g, batch, temperature,
                           vocab_mask, accepted_len, next_token);
        rc = run_plan(h, draft_len, draft_tokens, batch, g, sp0, s);
    }
    if (rc != FLEXSPEC_OK) return rc;
    return run_sample(h, logits ? logits : h.logits, draft_tokens, draft_logits, draft_len, seeds, g, batch,
                      temperature, vocab_mask, accepted_len, next_token, s);
}

// The step on device buffers.  dlog_in_flight: the draft logits are still being copied from the host on the
// second stream (queued there by the caller before anything else).  Then the plan runs on the main stream,
// the statistics of the draft logits wait for it behind the copy, and the main stream joins the second one
// only before the decision, so that attention and the LM head run beside the copy.
static int verify_impl(flexspec_handle* fh, const flexspec_kv* kv, const void* hidden,
                       const int32_t* draft_tokens, const float* draft_logits, bool dlog_in_flight,
                       const int32_t* draft_len, const int32_t* draft_len_host,
                       const uint64_t* seeds, int32_t batch, float temperature, const uint32_t* vocab_mask,
                       int32_t* accepted_len, int32_t* next_token, void* stream)
{
    if (fh == nullptr || hidden == nullptr || draft_len == nullptr || accepted_len == nullptr ||
        next_token == nullptr)
        return FLEXSPEC_ERR_INVALID_ARG;
    Handle& h = fh->h;
    if (!kv_args_ok(h, kv, true)) return FLEXSPEC_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(hidden) & 15u) != 0) return FLEXSPEC_ERR_INVALID_ARG;
    Geometry g;
    int rc = check_lengths(h, draft_len_host, kv->kv_len_host, batch, kv->max_pages_per_seq, &g);
    if (rc != FLEXSPEC_OK) return rc;
    if (!sample_args_ok(h, draft_tokens, draft_logits, seeds, temperature, g)) return FLEXSPEC_ERR_INVALID_ARG;
    if (!logits_aligned(draft_logits, h.cfg.vocab)) return FLEXSPEC_ERR_INVALID_ARG;
    DeviceGuard guard(h.cfg.device);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    h.launches = 0;
    memset(h.ev_used, 0, sizeof(h.ev_used));
    SampleParams sp;
    fill_sample_params(h, sp, h.logits, draft_tokens, draft_logits, draft_len, seeds, g, batch, temperature, vocab_mask,
                       accepted_len, next_token);
    mark(h, 0, s);
    // ---- second stream: row offsets of the ragged batch and the statistics of the draft logits need
    // nothing from the target model, so they run beside attention and the LM head
    const bool host_copy = dlog_in_flight && draft_logits != nullptr && g.s_rows > 0;
    if (host_copy) {
        rc = run_plan(h, draft_len, draft_tokens, batch, g, sp, s);
        if (rc != FLEXSPEC_OK) return rc;
        if (cudaEventRecord(h.ev_plan, s) != cudaSuccess || cudaStreamWaitEvent(h.side, h.ev_plan, 0) != cudaSuccess)
            return FLEXSPEC_ERR_CUDA;
    } else {
        if (cudaEventRecord(h.ev_fork, s) != cudaSuccess || cudaStreamWaitEvent(h.side, h.ev_fork, 0) != cudaSuccess)
            return FLEXSPEC_ERR_CUDA;
        rc = run_plan(h, draft_len, draft_tokens, batch, g, sp, h.side);
        if (rc != FLEXSPEC_OK) return rc;
    }
    if (!sp.greedy && sp.s_rows > 0) {
        if (launch_sample_stats(sp, sp.m_rows, sp.s_rows, h.side) != cudaSuccess) return FLEXSPEC_ERR_CUDA;
        h.launches++;
    }
    if (cudaEventRecord(h.ev_join, h.side) != cudaSuccess) return FLEXSPEC_ERR_CUDA;
    // ---- main stream
    mark(h, 1, s);
    rc = run_attention(h, kv, hidden, draft_len, draft_len_host, g, batch, h.attn_out, s);
    if (rc != FLEXSPEC_OK) return rc;
    mark(h, 2, s);
    mark(h, 3, s);
    // With device inputs the second stream's work is long done by now; joining here keeps LM head -> decision
    // -> draw back to back on this stream, so that the last two can be launched programmatically.  With the
    // draft logits still on their way from the host the join waits until just before the decision.
    if (!host_copy && cudaStreamWaitEvent(s, h.ev_join, 0) != cudaSuccess) return FLEXSPEC_ERR_CUDA;
    sp.tstats = h.tstats;                                                     // the LM head leaves the target rows' parts
    sp.n_tparts = 4 * (h.lm_full_tiles + h.lm_last_tiles);
    rc = run_lm_head(h, h.attn_out, g.m_rows, h.logits, &sp, s);
    if (rc != FLEXSPEC_OK) return rc;
    mark(h, 4, s);
    if (sp.filtered) {
        if (launch_sample_filter(sp, true, s) != cudaSuccess) return FLEXSPEC_ERR_CUDA;   // the plan's tables are there: joined above
        h.launches++;
    }
    if (host_copy && cudaStreamWaitEvent(s, h.ev_join, 0) != cudaSuccess) return FLEXSPEC_ERR_CUDA;
    mark(h, 5, s);
    if (launch_sample_accept(sp, !host_copy, s) != cudaSuccess) return FLEXSPEC_ERR_CUDA;
    h.launches++;
    mark(h, 6, s);
    return FLEXSPEC_OK;
}

int flexspec_verify(flexspec_handle* fh, const flexspec_kv* kv, const void* hidden,
                    const int32_t* draft_tokens, const float* draft_logits,
                    const int32_t* draft_len, const int32_t* draft_len_host,
                    const uint64_t* seeds, int32_t batch, float temperature, const uint32_t* vocab_mask,
                    int32_t* accepted_len, int32_t* next_token, void* stream)
{
    NvtxRange nvtx_range("flexspec_verify");
    return verify_impl(fh, kv, hidden, draft_tokens, draft_logits, false, draft_len, draft_len_host, seeds, batch,
                       temperature, vocab_mask, accepted_len, next_token, stream);
}

int flexspec_verify_host(flexspec_handle* fh, const flexspec_kv* kv, const void* hidden,
                         const int32_t* draft_tokens, const float* draft_logits, const int32_t* draft_len,
                         const uint64_t* seeds, int32_t batch, float temperature, const uint32_t* vocab_mask,
                         int32_t* accepted_len, int32_t* next_token, void* stream)
{
    NvtxRange nvtx_range("flexspec_verify_host");
    if (fh == nullptr || hidden == nullptr || draft_len == nullptr || accepted_len == nullptr ||
        next_token == nullptr)
        return FLEXSPEC_ERR_INVALID_ARG;
    Handle& h = fh->h;
    if (!kv_args_ok(h, kv, false)) return FLEXSPEC_ERR_INVALID_ARG;
    Geometry g;
    int rc = check_lengths(h, draft_len, kv->kv_len_host, batch, kv->max_pages_per_seq, &g);
    if (rc != FLEXSPEC_OK) return rc;
    if (!sample_args_ok(h, draft_tokens, draft_logits, seeds, temperature, g)) return FLEXSPEC_ERR_INVALID_ARG;
    DeviceGuard guard(h.cfg.device);
    cudaStream_t s = static_cast<cudaStream_t>(stream);

    // carve the staging buffer (256-byte aligned pieces)
    uint8_t* base = static_cast<uint8_t*>(h.stage_dev);
    size_t off = 0;
    auto carve = [&](size_t bytes) { uint8_t* p = base + off; off = (off + bytes + 255) & ~size_t(255); return p; };
    void* d_hidden = carve(static_cast<size_t>(g.m_rows) * h.d_model * 2);
    float* d_dlog = reinterpret_cast<float*>(carve(static_cast<size_t>(g.s_rows) * h.cfg.vocab * 4));
    int32_t* d_tok = reinterpret_cast<int32_t*>(carve(static_cast<size_t>(g.s_rows) * 4));
    int32_t* d_len = reinterpret_cast<int32_t*>(carve(static_cast<size_t>(batch) * 4));
    int32_t* d_kvl = reinterpret_cast<int32_t*>(carve(static_cast<size_t>(batch) * 4));
    uint64_t* d_seed = reinterpret_cast<uint64_t*>(carve(static_cast<size_t>(batch) * 8));
    const size_t mask_bytes = vocab_mask != nullptr ? static_cast<size_t>(batch) * ((h.cfg.vocab + 31) / 32) * 4 : 0;
    uint32_t* d_mask = reinterpret_cast<uint32_t*>(carve(mask_bytes));
    if (off > h.stage_bytes) return FLEXSPEC_ERR_INVALID_ARG;

    bool ok = true;
    auto H2D = [&](void* dst, const void* src, size_t bytes) {
        if (bytes > 0 && src != nullptr) ok = ok && cudaMemcpyAsync(dst, src, bytes, cudaMemcpyHostToDevice, s) == cudaSuccess;
    };
    // The small inputs go first: host-to-device copies are served in the order they were issued, whatever their
    // stream, and attention needs these.  The draft logits, by far the largest input, follow on the second
    // stream (idle: the previous call ended with a synchronisation); nothing on the main stream needs them
    // before the decision, so attention and the LM head run beside their copy.
    H2D(d_hidden, hidden, static_cast<size_t>(g.m_rows) * h.d_model * 2);
    H2D(d_tok, draft_tokens, static_cast<size_t>(g.s_rows) * 4);
    H2D(d_len, draft_len, static_cast<size_t>(batch) * 4);
    H2D(d_kvl, kv->kv_len_host, static_cast<size_t>(batch) * 4);
    H2D(d_seed, seeds, static_cast<size_t>(batch) * 8);
    H2D(d_mask, vocab_mask, mask_bytes);
    if (!ok) { cudaGetLastError(); return FLEXSPEC_ERR_CUDA; }
    const bool big = draft_logits != nullptr && g.s_rows > 0;
    if (big && cudaMemcpyAsync(d_dlog, draft_logits, static_cast<size_t>(g.s_rows) * h.cfg.vocab * 4, cudaMemcpyHostToDevice,
                               h.side) != cudaSuccess) {
        cudaGetLastError();
        return FLEXSPEC_ERR_CUDA;
    }

    flexspec_kv kv_dev = *kv;
    kv_dev.kv_len = d_kvl;
    rc = verify_impl(fh, &kv_dev, d_hidden, d_tok, draft_logits ? d_dlog : nullptr, big, d_len, draft_len,
                     seeds ? d_seed : nullptr, batch, temperature, vocab_mask ? d_mask : nullptr, h.out_dev,
                     h.out_dev + batch, s);
    if (rc != FLEXSPEC_OK) return rc;
    // both result arrays lie side by side on the device: one copy into the handle's pinned buffer, then two
    // 4 * batch byte copies on the host
    ok = cudaMemcpyAsync(h.out_host, h.out_dev, static_cast<size_t>(batch) * 8, cudaMemcpyDeviceToHost, s) == cudaSuccess;
    ok = ok && cudaStreamSynchronize(s) == cudaSuccess;
    if (!ok) { cudaGetLastError(); return FLEXSPEC_ERR_CUDA; }
    memcpy(accepted_len, h.out_host, static_cast<size_t>(batch) * 4);
    memcpy(next_token, h.out_host + batch, static_cast<size_t>(batch) * 4);
    return FLEXSPEC_OK;
}

int flexspec_kv_append(flexspec_handle* fh, void* kv_pages, int32_t num_pages, const int32_t* page_table,
                       int32_t max_pages_per_seq, const int32_t* kv_len, const int32_t* kv_len_host,
                       const void* new_k, const void* new_v, const int32_t* draft_len, const int32_t* draft_len_host,
                       int32_t batch, void* stream)
{
    if (fh == nullptr || kv_pages == nullptr || page_table == nullptr || kv_len == nullptr || kv_len_host == nullptr ||
        new_k == nullptr || new_v == nullptr || draft_len == nullptr)
        return FLEXSPEC_ERR_INVALID_ARG;
    Handle& h = fh->h;
    if (num_pages < 1 || max_pages_per_seq < 1) return FLEXSPEC_ERR_INVALID_ARG;
    if (((reinterpret_cast<uintptr_t>(kv_pages) | reinterpret_cast<uintptr_t>(new_k) | reinterpret_cast<uintptr_t>(new_v)) & 15u) != 0)
        return FLEXSPEC_ERR_INVALID_ARG;
    Geometry g;
    int rc = check_lengths(h, draft_len_host, kv_len_host, batch, max_pages_per_seq, &g);
    if (rc != FLEXSPEC_OK) return rc;
    DeviceGuard guard(h.cfg.device);
    KvAppendParams p;
    p.kv_pages = kv_pages; p.page_table = page_table; p.kv_len = kv_len; p.draft_len = draft_len;
    p.new_k = new_k; p.new_v = new_v;
    p.batch = batch; p.n_kv_heads = h.cfg.n_kv_heads; p.head_dim = h.cfg.head_dim;
    p.max_pages_per_seq = max_pages_per_seq; p.num_pages = num_pages;
    p.status = h.status;
    h.launches = 0;
    if (launch_kv_append(p, g.m_rows, static_cast<cudaStream_t>(stream)) != cudaSuccess) return FLEXSPEC_ERR_CUDA;
    h.launches++;
    return FLEXSPEC_OK;
}

int flexspec_kv_rollback(flexspec_handle* fh, const int32_t* kv_len, const int32_t* draft_len,
                         const int32_t* accepted_len, int32_t batch, int32_t* kv_len_next, void* stream)
{
    if (fh == nullptr || kv_len == nullptr || draft_len == nullptr || accepted_len == nullptr || kv_len_next == nullptr)
        return FLEXSPEC_ERR_INVALID_ARG;
    Handle& h = fh->h;
    if (batch < 1 || batch > h.cfg.max_batch) return FLEXSPEC_ERR_INVALID_ARG;
    DeviceGuard guard(h.cfg.device);
    if (launch_kv_rollback(kv_len, draft_len, accepted_len, batch, kv_len_next, static_cast<cudaStream_t>(stream)) != cudaSuccess)
        return FLEXSPEC_ERR_CUDA;
    h.launches = 1;
    return FLEXSPEC_OK;
}

int flexspec_kv_release(flexspec_handle* fh, int32_t* page_table, int32_t max_pages_per_seq, int32_t num_pages,
                        const int32_t* kv_len_prev, const int32_t* kv_len_next, int32_t batch, int32_t* free_list,
                        int32_t free_capacity, int32_t* free_count, void* stream)
{
    if (fh == nullptr || page_table == nullptr || kv_len_prev == nullptr || kv_len_next == nullptr || free_list == nullptr ||
        free_count == nullptr)
        return FLEXSPEC_ERR_INVALID_ARG;
    Handle& h = fh->h;
    if (batch < 1 || batch > h.cfg.max_batch || max_pages_per_seq < 1 || num_pages < 1 || free_capacity < 0)
        return FLEXSPEC_ERR_INVALID_ARG;
    DeviceGuard guard(h.cfg.device);
    if (launch_kv_release(page_table, max_pages_per_seq, kv_len_prev, kv_len_next, batch, num_pages, free_list, free_capacity,
                          free_count, h.status, static_cast<cudaStream_t>(stream)) != cudaSuccess)
        return FLEXSPEC_ERR_CUDA;
    h.launches = 1;
    return FLEXSPEC_OK;
}

int flexspec_set_top_p(flexspec_handle* fh, float top_p)
{
    if (fh == nullptr || !(top_p > 0.f) || top_p > 1.f) return FLEXSPEC_ERR_INVALID_ARG;
    fh->h.top_p = top_p;
    return FLEXSPEC_OK;
}

int flexspec_set_sampling(flexspec_handle* fh, float top_p, int32_t top_k, const float* temperatures)
{
    if (fh == nullptr || !(top_p > 0.f) || top_p > 1.f || top_k < 0) return FLEXSPEC_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(temperatures) & 3u) != 0) return FLEXSPEC_ERR_INVALID_ARG;
    fh->h.top_p = top_p;
    fh->h.top_k = top_k;
    fh->h.temps = temperatures;
    return FLEXSPEC_OK;
}

int flexspec_get_debug(flexspec_handle* fh, flexspec_debug* out)
{
    if (fh == nullptr || out == nullptr) return FLEXSPEC_ERR_INVALID_ARG;
    const Handle& h = fh->h;
    out->attn_out = h.attn_out;
    out->logits = h.logits;
    out->p_tok = h.dbg_p;
    out->q_tok = h.dbg_q;
    out->u_acc = h.dbg_u;
    out->status = h.status;
    out->topp = h.topp;
    return FLEXSPEC_OK;
}

int flexspec_status(flexspec_handle* fh, int32_t* status_host)
{
    if (fh == nullptr) return FLEXSPEC_ERR_INVALID_ARG;
    Handle& h = fh->h;
    DeviceGuard guard(h.cfg.device);
    int32_t st[4] = {0, 0, 0, 0};
    if (cudaDeviceSynchronize() != cudaSuccess) { cudaGetLastError(); return FLEXSPEC_ERR_CUDA; }
    if (cudaMemcpy(st, h.status, sizeof(st), cudaMemcpyDeviceToHost) != cudaSuccess) return FLEXSPEC_ERR_CUDA;
    if (st[0] != 0) {
        // a kernel that gave up may have left its arrival tickets half counted: start the next call clean
        if (cudaMemset(h.status, 0, sizeof(st)) != cudaSuccess ||
            cudaMemset(h.att_tickets, 0, sizeof(int32_t) * static_cast<size_t>(h.att_pairs_max) * 12) != cudaSuccess)
            return FLEXSPEC_ERR_CUDA;
    }
    if (status_host != nullptr) memcpy(status_host, st, sizeof(st));
    return st[0];
}

int flexspec_selftest_wait_timeout(flexspec_handle* fh, int64_t limit_ns, void* stream)
{
    if (fh == nullptr || limit_ns < 1000 || limit_ns > 50ll * 1000 * 1000) return FLEXSPEC_ERR_INVALID_ARG;
    Handle& h = fh->h;
    DeviceGuard guard(h.cfg.device);
    if (launch_wait_timeout(h.status, static_cast<uint64_t>(limit_ns), static_cast<cudaStream_t>(stream)) != cudaSuccess)
        return FLEXSPEC_ERR_CUDA;
    h.launches = 1;
    return FLEXSPEC_OK;
}

int flexspec_set_profiling(flexspec_handle* fh, int32_t on)
{
    if (fh == nullptr) return FLEXSPEC_ERR_INVALID_ARG;
    fh->h.profiling = on ? 1 : 0;
    memset(fh->h.ev_used, 0, sizeof(fh->h.ev_used));
    return FLEXSPEC_OK;
}

int flexspec_get_stage_ms(flexspec_handle* fh, float ms[6])
{
    if (fh == nullptr || ms == nullptr) return FLEXSPEC_ERR_INVALID_ARG;
    Handle& h = fh->h;
    for (int i = 0; i < 6; ++i) ms[i] = 0.f;
    if (!h.profiling || !h.ev_used[0] || !h.ev_used[6]) return FLEXSPEC_ERR_INVALID_ARG;
    DeviceGuard guard(h.cfg.device);
    if (cudaEventSynchronize(h.ev[6]) != cudaSuccess) { cudaGetLastError(); return FLEXSPEC_ERR_CUDA; }
    // events: 0 call start, 1 after the fork of the second stream, 2 = 3 after attention, 4 after the LM head,
    // 5 after the nucleus kernel (top-p only; else = 4), 6 after the acceptance kernel
    for (int i = 0; i < 6; ++i) {
        if (!h.ev_used[i] || !h.ev_used[i + 1]) continue;
        if (cudaEventElapsedTime(&ms[i], h.ev[i], h.ev[i + 1]) != cudaSuccess) { cudaGetLastError(); return FLEXSPEC_ERR_CUDA; }
    }
    return FLEXSPEC_OK;
}

int flexspec_last_launches(flexspec_handle* fh)
{
    if (fh == nullptr) return FLEXSPEC_ERR_INVALID_ARG;
    return fh->h.launches;
}

const char* flexspec_strerror(int code)
{
    switch (code) {
        case FLEXSPEC_OK: return "ok";
        case FLEXSPEC_ERR_INVALID_ARG: return "invalid argument";
        case FLEXSPEC_ERR_UNSUPPORTED: return "unsupported shape or device";
        case FLEXSPEC_ERR_OOM: return "out of device memory";
        case FLEXSPEC_ERR_CUDA: return "CUDA call failed";
        case FLEXSPEC_ERR_TIMEOUT: return "device-side wait timed out";
        case FLEXSPEC_ERR_BAD_PAGE: return "page table entry out of range";
        case FLEXSPEC_ERR_BAD_TOKEN: return "draft token out of range";
        case FLEXSPEC_ERR_NO_DEVICE: return "no usable CUDA device";
        default: return "unknown error";
    }
}

const char* flexspec_version(void) { return "flexspec-b200 0.1 (sm_100a)"; }

}  // extern "C"
