// Host-side internals shared by the .cu files of the library: the handle, launch wrappers.
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/flexspec.h"

namespace fs {

constexpr int kMaxBatch = 1024;
constexpr int kMaxK = 63;
constexpr int kSampleChunk = 8192;        // vocabulary entries per CTA of the statistics kernel
constexpr int kAcceptCluster = 8;         // CTAs (one thread-block cluster) per sequence in the acceptance kernel
constexpr int kWarpChunk = 1024;          // vocabulary entries whose mass one warp adds up at a time there
constexpr int kMaxWarpChunksPerCta = 128; // per-CTA list of warp-chunk masses in shared memory
constexpr int kMaxVocab = kAcceptCluster * kMaxWarpChunksPerCta * kWarpChunk;   // 1 048 576
constexpr int kAttBlockTokens = 128;      // KV tokens per attention work block / pipeline stage
constexpr int kAttRowsPerPair = 128;      // query rows per (sequence, kv head) row block (MMA M)
constexpr int kAttProducerWarps = 2;      // issuing a TMA request costs ~55 cycles of its warp: two warps share a block's 32
constexpr int kAttThreads = (kAttProducerWarps + 1 + 4 + 1) * 32;   // TMA warps, QK^T issuer, 4 softmax warps, PV issuer
constexpr int kAttMaxStages = 8;          // K / V ring depth (what fits in shared memory is used)
constexpr int kNumStageEvents = 7;

struct Plan {                 // device tables written by the plan kernel, read by the sampling stage
    int32_t* cu_q;            // [max_batch+1] first query row of each sequence
    int32_t* cu_d;            // [max_batch+1] first draft row of each sequence
    int32_t* row_seq;         // [max_m] sequence of each query row
    float* row_c;             // [max_m + max_s] log2(e) / T of the sequence of every target row, then of every draft row
    int32_t* k_eff;           // [max_batch] draft length the sampling kernels use: draft_len[b] once it has been
                              // checked against the geometry the host sized the launches for (0 if it disagrees)
};

struct AttnParams {
    const __nv_bfloat16* hidden;
    const int32_t* page_table;
    const int32_t* kv_len;
    const int32_t* draft_len;
    int32_t batch, n_q_heads, n_kv_heads, group;
    int32_t max_pages_per_seq, num_pages;
    int32_t m_rows, k_cap, kv_cap;   // geometry the host sized the call for: device lengths are clamped to it
    int32_t n_pad;            // MMA N: the largest pair's query rows rounded up to 16 (<= 128)
    int32_t k_stages;         // depth of the K ring (128-token tiles)
    int32_t v_stages;         // depth of the V ring
    int32_t p_bufs;           // P^T buffers (2, or 1 when shared memory is short)
    float scale_log2;         // log2(e) / sqrt(head_dim)
    float* part_o;            // [2 * CTAs][Dh][128] unnormalised partial outputs (a CTA's first / last segment)
    float* part_ml;           // [2 * CTAs][4 warps][128][2]  (running max in log2 units, sum)
    int32_t* tickets;         // [pairs][4 quarters][3 column parts] self-resetting arrival counters of the split merge
    __nv_bfloat16* attn_out;  // [M][d_model]
    int32_t* status;
};

// Where every CTA of the attention kernel starts in the batch-wide list of 128-token blocks, computed
// on the host from the host copies of the lengths and passed with the launch as a kernel parameter
// (nothing has to be read or scanned on the device before the first K/V request).
constexpr int kAttMaxCtas = 160;
struct AttCta {
    int32_t blk_begin;        // first block of this CTA in the batch-wide list
    int32_t n_my;             // blocks of this CTA (> 0)
    int32_t b;                // sequence of the first block ...
    int32_t blk_off;          // ... and the block's offset inside that sequence's blocks
    int32_t q_row0, pair0, blk0;   // first query row / first pair / first block of sequence b
    int32_t k, kvl;           // draft length and kv length of sequence b (host copy)
    int32_t pad;
};
struct AttTable {
    AttCta cta[kAttMaxCtas];
};

struct KvAppendParams {
    void* kv_pages;               // bf16 [num_pages][2][n_kv_heads][16][head_dim]
    const int32_t* page_table;
    const int32_t* kv_len;
    const int32_t* draft_len;
    const void* new_k;            // bf16 [M][n_kv_heads][head_dim]
    const void* new_v;
    int32_t batch, n_kv_heads, head_dim, max_pages_per_seq, num_pages;
    int32_t* status;
};

struct LmHeadParams {
    float* logits;            // [m_rows][vocab]
    int32_t m_rows, vocab, d_model;
    int32_t n_tile;           // token columns per accumulator block (multiple of 16, <= 256)
    int32_t n_blocks;         // accumulator blocks per pass (1 or 2)
    int32_t n_pass;           // passes over W when m_rows > n_tile * n_blocks
    int32_t n_vtiles;         // vocabulary tiles: n_full_tiles of 128 rows, then tiles of last_rows rows
    int32_t n_full_tiles;
    int32_t last_rows;        // height of the tiles of the last wave (<= 128)
    int32_t num_stages;       // shared-memory pipeline depth
    int32_t n_bufs;           // accumulator ring: buffers of n_tile TMEM columns (n_blocks <= n_bufs <= 8)
    // optional: softmax statistics of the rows, one part per (row, 32 vocabulary rows), for the
    // sampling stage (null = not wanted)
    float2* tstats;           // [m_rows][n_tparts], n_tparts = 4 * n_vtiles
    int32_t n_tparts;
    float inv_temp_log2;      // log2(e) / T
    const float* row_c;       // [m_rows] per-row log2(e) / T (per-sequence temperatures); null: inv_temp_log2 for all
    int32_t greedy;           // parts are (max, arg-max index) instead of (max, sum exp)
    const int32_t* row_seq;   // [m_rows] sequence of each row (for the vocabulary mask)
    const uint32_t* vocab_mask;
    int32_t mask_words;
    int32_t* status;
};

struct SampleParams {
    const float* logits;          // [M][V] target
    const float* draft_logits;    // [S][V]
    const int32_t* draft_tokens;  // [S]
    const int32_t* draft_len;     // [B]
    const uint64_t* seeds;        // [B]
    const uint32_t* vocab_mask;   // [B][mask_words] or null
    const int32_t* cu_q;
    const int32_t* cu_d;
    const int32_t* row_seq;
    int32_t batch, vocab, m_rows, s_rows, n_chunks, mask_words;
    int32_t row_begin;            // first row of this launch of the statistics kernel
    float inv_temp_log2;          // log2(e) / T of the call (scalar temperature)
    const float* temps;           // [B] per-sequence temperatures (device) or null
    const float* row_c;           // [M + S] log2(e) / T per row, written by the plan kernel
    int32_t greedy;
    float2* stats;                // [(M+S)][n_chunks] parts written by the statistics kernel: (chunk max in logit
                                  // units, sum exp), or (max, arg-max index as int bits) in greedy mode
    const float2* tstats;         // parts of the target rows: [M][n_tparts] (from the LM head), or = stats
    int32_t n_tparts;
    const int32_t* k_eff;         // [B] checked draft lengths (plan kernel)
    float top_p;                  // nucleus mass of the target distribution; >= 1: no filtering
    int32_t top_k;                // keep the top_k most probable tokens first; <= 0: no filtering
    int32_t filtered;             // top-k or top-p is on: the filter kernel ran and p.topp holds its thresholds
    double* topp;                 // [M][2]: lowest kept logit of the row's nucleus, mass of the nucleus (in units of
                                  // 2^((z - max) * c)); written by the nucleus kernel when top_p < 1
    int32_t* accepted_len;
    int32_t* next_token;
    double* dbg_p; double* dbg_q; float* dbg_u;   // [S] or null
    int32_t* status;
};

struct SeqBlocks { int32_t pairs, nb, rows; };   // attention planner, per sequence: pairs, blocks per pair, query rows

struct Handle {
    flexspec_config cfg;
    SeqBlocks* att_seq;       // HOST [max_batch]
    int32_t d_model, max_m, max_s;
    int32_t sm_count;
    __nv_bfloat16* w_tiled;   // the handle's copy of W in streaming order: [tile][k block][tile rows][64]
    CUtensorMap w_map;        // over w_tiled viewed as rows of 64 elements, box of 128 rows (one k block of a full tile)
    CUtensorMap w_map_last;   // same tensor, box of lm_last_rows rows (tiles of the last wave)
    int32_t lm_full_tiles, lm_last_rows, lm_last_tiles;
    // workspace
    __nv_bfloat16* attn_out;
    float* logits;
    float* part_o; float* part_ml; int32_t* att_tickets; int32_t att_pairs_max;
    Plan plan;
    float2* stats; float2* tstats; double* topp; float top_p; int32_t top_k; const float* temps;
    double* dbg_p; double* dbg_q; float* dbg_u;
    int32_t* status;
    // host staging for flexspec_verify_host
    void* stage_dev; size_t stage_bytes;
    int32_t* out_dev;
    int32_t* out_host;        // pinned: both result arrays of the host-buffer entry point come back in one copy
    // second stream: the plan and the draft-logit statistics run beside attention and the LM head
    cudaStream_t side; cudaEvent_t ev_fork, ev_join, ev_plan;
    // profiling
    int32_t profiling, launches;
    cudaEvent_t ev[kNumStageEvents];
    int32_t ev_used[kNumStageEvents];
};

// launch wrappers (each returns a cudaError_t from the launch)
// m_rows / s_rows / k_cap: the geometry derived from the HOST copy of the lengths; the kernel checks the
// device copy against it
// temps / scalar_c: per-sequence temperatures (device, may be null) and log2(e) / T of the call
cudaError_t launch_plan(const int32_t* draft_len, const int32_t* draft_tokens, int32_t batch, int32_t vocab,
                        int32_t m_rows, int32_t s_rows, int32_t k_cap, const float* temps, float scalar_c, Plan plan,
                        int32_t* status, cudaStream_t stream);
cudaError_t launch_attention(const Handle& h, const CUtensorMap& kv_map, const AttnParams& p, const AttTable& table,
                             int32_t n_ctas, cudaStream_t stream);
cudaError_t launch_lm_head(const Handle& h, const CUtensorMap& x_map, const LmHeadParams& p, cudaStream_t stream);
cudaError_t launch_retile_w(const void* w, void* out, int vocab, int d_model, int n_full, int n_last, int last_rows,
                            cudaStream_t stream);
cudaError_t launch_sample_stats(const SampleParams& p, int32_t row_begin, int32_t row_count, cudaStream_t stream);
// pdl: launch with programmatic stream serialization (the kernel may start while its predecessor in
// the stream drains; it waits on the device before touching the predecessor's results)
cudaError_t launch_sample_filter(const SampleParams& p, bool pdl, cudaStream_t stream);
cudaError_t launch_sample_accept(const SampleParams& p, bool pdl, cudaStream_t stream);

template <typename... KArgs, typename... Args>
inline cudaError_t launch_kernel_ex(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                                    bool pdl, Args... args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = pdl ? 1 : 0;
    cfg.attrs = attr; cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, args...);
}

cudaError_t launch_kv_append(const KvAppendParams& p, int32_t m_rows, cudaStream_t stream);
cudaError_t launch_kv_rollback(const int32_t* kv_len, const int32_t* draft_len, const int32_t* accepted_len, int32_t batch,
                               int32_t* kv_len_next, cudaStream_t stream);
cudaError_t launch_kv_release(int32_t* page_table, int32_t max_pages_per_seq, const int32_t* kv_len_prev,
                              const int32_t* kv_len_next, int32_t batch, int32_t num_pages, int32_t* free_list,
                              int32_t free_capacity, int32_t* free_count, int32_t* status, cudaStream_t stream);
cudaError_t launch_wait_timeout(int32_t* status, uint64_t limit_ns, cudaStream_t stream);
cudaError_t attention_init(int head_dim);   // opt-in shared memory sizes
int attention_p_bufs(int n_pad);
void attention_stages(int head_dim, int n_pad, int* k_stages, int* v_stages);
cudaError_t lm_head_init();
cudaError_t sample_init();                  // opt-in shared memory size of the acceptance kernel (per device)
size_t lm_head_smem_bytes(int n_tile, int n_blocks, int num_stages);
int lm_head_pick_stages(int n_tile, int n_blocks);

}  // namespace fs
