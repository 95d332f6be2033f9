// Stage 3: the acceptance loop and the emitted token of Algorithm 2, Step 2, for a ragged batch
// in one launch sequence.
//
// SAMPLE mode is the speculative-sampling rule the paper builds on (Section II-A: a draft is
// verified so that outputs are distributed exactly as the target's): with p = softmax(target/T),
// q = softmax(draft/T), accept x_j iff u_j * q_j(x_j) < p_j(x_j); at the first rejection n draw
// from max(0, p_n - q_n)/Z, and from p_k if all k drafts were accepted.  GREEDY mode is the loop
// as Algorithm 2 prints it: accept while x_j equals the arg-max of the target row, emit the
// arg-max of the first row that disagrees (or of the bonus row).
//
//   stats  : grid (vocabulary chunk of 8192, row): one streaming read of the logits; per chunk the
//            max and the sum of 2^((z-max)*c), c = log2(e)/T, in fp32 (online per thread, merged
//            by shuffles, one block barrier).  Serves the draft rows (ahead of time, on a second
//            stream) and, for the stand-alone stage, the target rows; inside flexspec_verify the
//            LM-head kernel writes the target rows' parts from its epilogue.
//   decide : one CTA per sequence merges the parts of its rows, evaluates the acceptance tests
//            with Philox uniforms, finds the first rejection by warp vote, stores accepted_len.
//   draw   : grid (chunk of 2048, sequence) over row n of each sequence only: probability mass of
//            the residual (and of p) per chunk, fp32 exponentials accumulated in fp64; the last
//            CTA of a sequence picks the chunk that holds u' * Z and scans it in vocabulary order
//            (inverse CDF).
#include "common.cuh"
#include "internal.h"

namespace fs {

constexpr int kSampleThreads = 256;
constexpr int kSampleWarps = kSampleThreads / 32;
constexpr int kElemsPerThread = kSampleChunk / kSampleThreads;   // 32
constexpr int kDrawElems = kDrawChunk / kSampleThreads;          // 8

__device__ __forceinline__ bool mask_allows(const uint32_t* mask_row, int v)
{
    return mask_row == nullptr || ((mask_row[v >> 5] >> (v & 31)) & 1u);
}

// (max, sum of 2^((z - max) * c)) pairs: merge of two partial softmax statistics
__device__ __forceinline__ void merge_ms(float& m, float& s, float m2, float s2, float c)
{
    const float mm = fmaxf(m, m2);
    const float base = (mm == -INFINITY) ? 0.f : mm;
    s = s * fast_exp2((m - base) * c) + s2 * fast_exp2((m2 - base) * c);
    m = mm;
}

// ------------------------------------------------------------------------------------ statistics
// One part per (row, vocabulary chunk): SAMPLE (max, sum of 2^((z - max) * c)); GREEDY (max, lowest
// index holding it, as int bits).  Rows [0, M) are target rows, rows [M, M+S) draft rows.  The
// LM-head kernel can write the target rows' parts itself (one part per 32 vocabulary rows); this
// kernel serves the draft rows and, for the stand-alone sampling stage, the target rows too.
__global__ void __launch_bounds__(kSampleThreads)
sample_stats_kernel(const SampleParams p)
{
    __shared__ float red_m[kSampleWarps];
    __shared__ float red_s[kSampleWarps];
    __shared__ int red_i[kSampleWarps];

    const int chunk = blockIdx.x;
    const int row = blockIdx.y + p.row_begin;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const bool is_target = row < p.m_rows;
    const float* src;
    const uint32_t* mask_row = nullptr;
    if (is_target) {
        src = p.logits + static_cast<int64_t>(row) * p.vocab;
        if (p.vocab_mask != nullptr) mask_row = p.vocab_mask + static_cast<int64_t>(p.row_seq[row]) * p.mask_words;
    } else {
        src = p.draft_logits + static_cast<int64_t>(row - p.m_rows) * p.vocab;
    }

    const int v0 = chunk * kSampleChunk;
    const int v_end = min(p.vocab, v0 + kSampleChunk);
    float z[kElemsPerThread];
    // thread t handles float4 groups t, t+256, ... of the chunk (coalesced)
    const bool vec_ok = ((p.vocab & 3) == 0);
#pragma unroll
    for (int i = 0; i < kElemsPerThread / 4; ++i) {
        const int v = v0 + (i * kSampleThreads + threadIdx.x) * 4;
        float4 x = make_float4(-INFINITY, -INFINITY, -INFINITY, -INFINITY);
        if (vec_ok && v + 3 < v_end) {
            x = __ldg(reinterpret_cast<const float4*>(src + v));
        } else {
            if (v + 0 < v_end) x.x = __ldg(src + v + 0);
            if (v + 1 < v_end) x.y = __ldg(src + v + 1);
            if (v + 2 < v_end) x.z = __ldg(src + v + 2);
            if (v + 3 < v_end) x.w = __ldg(src + v + 3);
        }
        if (mask_row != nullptr) {
            if (v + 0 < v_end && !mask_allows(mask_row, v + 0)) x.x = -INFINITY;
            if (v + 1 < v_end && !mask_allows(mask_row, v + 1)) x.y = -INFINITY;
            if (v + 2 < v_end && !mask_allows(mask_row, v + 2)) x.z = -INFINITY;
            if (v + 3 < v_end && !mask_allows(mask_row, v + 3)) x.w = -INFINITY;
        }
        z[4 * i + 0] = x.x; z[4 * i + 1] = x.y; z[4 * i + 2] = x.z; z[4 * i + 3] = x.w;
    }

    float mx = -INFINITY;
#pragma unroll
    for (int i = 0; i < kElemsPerThread; ++i) mx = fmaxf(mx, z[i]);
    const float c = p.inv_temp_log2;
    float2* out = p.stats + static_cast<int64_t>(row) * p.n_chunks + chunk;

    if (p.greedy) {
        // (max, lowest index holding it)
        int best = 0x7fffffff;
#pragma unroll
        for (int i = 0; i < kElemsPerThread; ++i) {
            const int v = v0 + ((i >> 2) * kSampleThreads + threadIdx.x) * 4 + (i & 3);
            if (z[i] == mx && v < v_end) best = min(best, v);
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            const float m2 = __shfl_xor_sync(0xffffffffu, mx, o);
            const int i2 = __shfl_xor_sync(0xffffffffu, best, o);
            if (m2 > mx || (m2 == mx && i2 < best)) { mx = m2; best = i2; }
        }
        if (lane == 0) { red_m[warp] = mx; red_i[warp] = best; }
        __syncthreads();
        if (warp != 0) return;
        float m = (lane < kSampleWarps) ? red_m[lane] : -INFINITY;
        int bi = (lane < kSampleWarps) ? red_i[lane] : 0x7fffffff;
#pragma unroll
        for (int o = kSampleWarps / 2; o > 0; o >>= 1) {
            const float m2 = __shfl_xor_sync(0xffffffffu, m, o);
            const int i2 = __shfl_xor_sync(0xffffffffu, bi, o);
            if (m2 > m || (m2 == m && i2 < bi)) { m = m2; bi = i2; }
        }
        if (lane == 0) *out = make_float2(m, __int_as_float(bi));
    } else {
        const float base = (mx == -INFINITY) ? 0.f : mx;
        float se = 0.f;
#pragma unroll
        for (int i = 0; i < kElemsPerThread; ++i) se += fast_exp2((z[i] - base) * c);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            const float m2 = __shfl_xor_sync(0xffffffffu, mx, o);
            const float s2 = __shfl_xor_sync(0xffffffffu, se, o);
            merge_ms(mx, se, m2, s2, c);
        }
        if (lane == 0) { red_m[warp] = mx; red_s[warp] = se; }
        __syncthreads();
        if (warp != 0) return;
        float m = (lane < kSampleWarps) ? red_m[lane] : -INFINITY;
        float sm = (lane < kSampleWarps) ? red_s[lane] : 0.f;
#pragma unroll
        for (int o = kSampleWarps / 2; o > 0; o >>= 1) {
            const float m2 = __shfl_xor_sync(0xffffffffu, m, o);
            const float s2 = __shfl_xor_sync(0xffffffffu, sm, o);
            merge_ms(m, sm, m2, s2, c);
        }
        if (lane == 0) *out = make_float2(m, sm);
    }
}

// Rows [row_begin, row_begin + row_count) of the (target rows, then draft rows) list.
cudaError_t launch_sample_stats(const SampleParams& p, int32_t row_begin, int32_t row_count, cudaStream_t stream)
{
    if (row_count <= 0) return cudaSuccess;
    SampleParams q = p;
    q.row_begin = row_begin;
    dim3 grid(p.n_chunks, row_count);
    sample_stats_kernel<<<grid, kSampleThreads, 0, stream>>>(q);
    return cudaGetLastError();
}

// ------------------------------------------------------------------------------------ nucleus (top-p)
// The paper's stochastic regime samples the target with top-p 0.9.  The nucleus of a row is the set
// of tokens whose logit is at least tau, where tau is the largest logit value such that the tokens
// with logit >= tau hold at least top_p of the row's mass (ties with tau are all kept).  One CTA
// per target row finds tau exactly by a 4-round radix selection over the order-preserving 32-bit
// keys of the logits, 8 bits per round: a 256-bin histogram of probability MASS over the keys that
// match the prefix found so far (one private fp32 histogram per warp, filled with the native
// shared-memory float add -- with flat logits every key of a round falls into one or two bins, and
// a single shared fp64 histogram serialised to a millisecond --, then summed in fp64), and a walk
// from the top bin down to the bin in which the cumulative mass reaches the target.
constexpr int kNucThreads = 1024;

__device__ __forceinline__ uint32_t order_key(float z)       // larger float <-> larger key
{
    const uint32_t u = __float_as_uint(z);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float key_to_float(uint32_t k)
{
    return __uint_as_float((k & 0x80000000u) ? (k & 0x7fffffffu) : ~k);
}

__global__ void __launch_bounds__(kNucThreads)
sample_nucleus_kernel(const SampleParams p)
{
    __shared__ double s_hist[256];
    __shared__ float s_whist[kNucThreads / 32][256];
    __shared__ float s_redf[kNucThreads / 32];
    __shared__ double s_redd[kNucThreads / 32];
    __shared__ double s_above, s_target, s_binmass;
    __shared__ uint32_t s_prefix;
    const int row = blockIdx.x;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const float cf = p.inv_temp_log2;
    const uint32_t* mask_row = (p.vocab_mask != nullptr) ? p.vocab_mask + static_cast<int64_t>(p.row_seq[row]) * p.mask_words : nullptr;

    // ---- (max, mass) of the row from its parts
    const float2* tp = p.tstats + static_cast<int64_t>(row) * p.n_tparts;
    float m = -INFINITY, sf = 0.f;
    for (int i = tid; i < p.n_tparts; i += kNucThreads) {
        const float2 pt = __ldcg(&tp[i]);
        merge_ms(m, sf, pt.x, pt.y, cf);
    }
    const float mt = m;
    m = warp_max(m);
    if (lane == 0) s_redf[warp] = m;
    __syncthreads();
    for (int w = 0; w < kNucThreads / 32; ++w) m = fmaxf(m, s_redf[w]);
    double sm = (mt == -INFINITY) ? 0.0 : static_cast<double>(sf) * static_cast<double>(fast_exp2((mt - m) * cf));
    sm = warp_sum(sm);
    if (lane == 0) s_redd[warp] = sm;
    __syncthreads();
    sm = 0.0;
    for (int w = 0; w < kNucThreads / 32; ++w) sm += s_redd[w];
    if (tid == 0) { s_above = 0.0; s_target = static_cast<double>(p.top_p) * sm; s_prefix = 0u; }

    const float* src = p.logits + static_cast<int64_t>(row) * p.vocab;
    for (int round = 0; round < 4; ++round) {
        const int shift = 24 - 8 * round;
        for (int i = tid; i < (kNucThreads / 32) * 256; i += kNucThreads) (&s_whist[0][0])[i] = 0.f;
        __syncthreads();
        const uint32_t prefix = s_prefix;
        const uint32_t hi_mask = (round == 0) ? 0u : (0xffffffffu << (shift + 8));
        // eight loads in flight per thread (the row comes out of L2: a dependent load per element would
        // cost its full latency 125 times per round)
        for (int v0 = 0; v0 < p.vocab; v0 += kNucThreads * 8) {
            float zz[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const int v = v0 + i * kNucThreads + tid;
                zz[i] = (v < p.vocab) ? __ldg(src + v) : -INFINITY;
            }
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const int v = v0 + i * kNucThreads + tid;
                float z = zz[i];
                if (mask_row != nullptr && v < p.vocab && !mask_allows(mask_row, v)) z = -INFINITY;
                const uint32_t key = order_key(z);
                if (z != -INFINITY && (key & hi_mask) == (prefix & hi_mask))
                    atomicAdd(&s_whist[warp][(key >> shift) & 255u], fast_exp2((z - m) * cf));
            }
        }
        __syncthreads();
        if (tid < 256) {
            double acc = 0.0;
#pragma unroll 8
            for (int w = 0; w < kNucThreads / 32; ++w) acc += static_cast<double>(s_whist[w][tid]);
            s_hist[tid] = acc;
        }
        __syncthreads();
        if (tid == 0) {
            double cum = s_above;
            int bin = 255;
            for (; bin > 0; --bin) {
                if (cum + s_hist[bin] >= s_target) break;
                cum += s_hist[bin];
            }
            s_above = cum;
            s_binmass = s_hist[bin];
            s_prefix = prefix | (static_cast<uint32_t>(bin) << shift);
        }
        __syncthreads();
    }
    if (tid == 0) {
        p.topp[static_cast<int64_t>(row) * 2] = static_cast<double>(key_to_float(s_prefix));
        p.topp[static_cast<int64_t>(row) * 2 + 1] = s_above + s_binmass;
    }
}

cudaError_t launch_sample_nucleus(const SampleParams& p, cudaStream_t stream)
{
    sample_nucleus_kernel<<<p.m_rows, kNucThreads, 0, stream>>>(p);
    return cudaGetLastError();
}

// ------------------------------------------------------------------------------------ decision
// grid (row j, sequence b): the CTA merges the parts of target row j (and draft row j) of the
// sequence -- maximum first, then the sum with fp32 weights accumulated in fp64 -- and leaves
// (max, sum) per row together with the outcome of the row's own acceptance test (Philox uniform,
// u * q(x) < p(x)).  The CTA that arrives last for the sequence (atomic ticket, nobody waits) finds
// the first rejection by warp vote and stores accepted_len; GREEDY compares the draft with the
// rows' arg-max.
__device__ __forceinline__ float block_max(float v, float* red, int lane, int warp)
{
    v = warp_max(v);
    __syncthreads();                                   // red may still be read from a previous use
    if (lane == 0) red[warp] = v;
    __syncthreads();
    float r = red[0];
#pragma unroll
    for (int w = 1; w < kSampleWarps; ++w) r = fmaxf(r, red[w]);
    return r;
}
__device__ __forceinline__ double block_sum(double v, double* red, int lane, int warp)
{
    v = warp_sum(v);
    __syncthreads();
    if (lane == 0) red[warp] = v;
    __syncthreads();
    double r = 0.0;
#pragma unroll
    for (int w = 0; w < kSampleWarps; ++w) r += red[w];
    return r;
}

constexpr int kRowStat = 8;       // doubles per (sequence, row): max_p, sum_p, max_q, sum_q, rejected

__global__ void __launch_bounds__(kSampleThreads)
sample_decide_kernel(const SampleParams p)
{
    __shared__ float red_f[kSampleWarps];
    __shared__ double red_d[kSampleWarps];
    __shared__ int red_i[kSampleWarps];
    __shared__ int s_last;
    const int j = blockIdx.x;
    const int b = blockIdx.y;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    pdl_launch_dependents();
    const int k_b = p.draft_len[b];                      // inputs of the step: not written by the preceding kernel
    if (j > k_b) return;
    const int q0 = p.cu_q[b], d0 = p.cu_d[b];
    const double scale = static_cast<double>(p.inv_temp_log2);
    const float cf = p.inv_temp_log2;
    double* rs = p.row_stats + (static_cast<int64_t>(b) * (kMaxK + 1) + j) * kRowStat;
    const bool test_row = !p.greedy && j < k_b;

    // ---- everything that depends only on the step's inputs and on the draft-logit statistics (second
    // stream, joined before the preceding kernel started) is done before that kernel's results are
    // awaited: the draft token, q_j(x_j) and the uniform of this row's acceptance test
    int x = 0;
    double mq = 0.0, sq = 1.0, qt = 0.0, u = 0.0;
    if (test_row && warp == 0) {
        const float2* dp = p.stats + static_cast<int64_t>(p.m_rows + d0 + j) * p.n_chunks;
        float mqf = -INFINITY;
        for (int i = lane; i < p.n_chunks; i += 32) mqf = fmaxf(mqf, __ldcg(&dp[i].x));
        mqf = warp_max(mqf);
        double acc = 0.0;
        for (int i = lane; i < p.n_chunks; i += 32) {
            const float2 pt = __ldcg(&dp[i]);
            if (pt.x != -INFINITY) acc += static_cast<double>(pt.y) * static_cast<double>(fast_exp2((pt.x - mqf) * cf));
        }
        sq = warp_sum(acc);
        mq = static_cast<double>(mqf);
        if (lane == 0) {
            x = p.draft_tokens[d0 + j];
            x = min(max(x, 0), p.vocab - 1);
            const double zq = static_cast<double>(p.draft_logits[static_cast<int64_t>(d0 + j) * p.vocab + x]);
            qt = (zq == -INFINITY) ? 0.0 : exp2((zq - mq) * scale) / sq;
            u = philox_uniform(p.seeds[b], static_cast<uint32_t>(j), 0u);
        }
    }
    pdl_wait();

    // ---- target row j: merge the parts (one pass, running (max, sum) per thread in fp32, fp64 sums across the block)
    double zp = 0.0;
    if (test_row && threadIdx.x == 0) {
        zp = static_cast<double>(p.logits[static_cast<int64_t>(q0 + j) * p.vocab + x]);
        if (p.vocab_mask != nullptr && !mask_allows(p.vocab_mask + static_cast<int64_t>(b) * p.mask_words, x)) zp = -INFINITY;
    }
    {
        const float2* tp = p.tstats + static_cast<int64_t>(q0 + j) * p.n_tparts;
        const int n = p.n_tparts;
        if (p.greedy) {
            float m = -INFINITY;
            int best = 0x7fffffff;
#pragma unroll 8
            for (int i = threadIdx.x; i < n; i += kSampleThreads) {
                const float2 pt = __ldcg(&tp[i]);
                const int idx = __float_as_int(pt.y);
                if (pt.x > m || (pt.x == m && idx < best)) { m = pt.x; best = idx; }
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                const float m2 = __shfl_xor_sync(0xffffffffu, m, o);
                const int i2 = __shfl_xor_sync(0xffffffffu, best, o);
                if (m2 > m || (m2 == m && i2 < best)) { m = m2; best = i2; }
            }
            if (lane == 0) { red_f[warp] = m; red_i[warp] = best; }
            __syncthreads();
            if (threadIdx.x == 0) {
                for (int w = 1; w < kSampleWarps; ++w)
                    if (red_f[w] > m || (red_f[w] == m && red_i[w] < best)) { m = red_f[w]; best = red_i[w]; }
                rs[0] = static_cast<double>(best);
            }
        } else {
            float m = -INFINITY, sf = 0.f;
#pragma unroll 8
            for (int i = threadIdx.x; i < n; i += kSampleThreads) {
                const float2 pt = __ldcg(&tp[i]);
                merge_ms(m, sf, pt.x, pt.y, cf);
            }
            const float mt = m;
            m = block_max(m, red_f, lane, warp);
            double sm = (mt == -INFINITY) ? 0.0 : static_cast<double>(sf) * static_cast<double>(fast_exp2((mt - m) * cf));
            sm = block_sum(sm, red_d, lane, warp);
            if (threadIdx.x == 0) {
                double tau = -INFINITY;                   // nucleus of the target row: its lowest kept logit and its mass
                if (p.top_p < 1.f) { tau = p.topp[static_cast<int64_t>(q0 + j) * 2]; sm = p.topp[static_cast<int64_t>(q0 + j) * 2 + 1]; }
                rs[0] = static_cast<double>(m); rs[1] = sm; rs[2] = mq; rs[3] = sq; rs[5] = tau;
                double rej = 0.0;
                if (test_row) {
                    const double pt = (zp == -INFINITY || zp < tau) ? 0.0 : exp2((zp - static_cast<double>(m)) * scale) / sm;
                    rej = (u * qt < pt) ? 0.0 : 1.0;
                    if (p.dbg_p != nullptr) {
                        p.dbg_p[d0 + j] = pt;
                        p.dbg_q[d0 + j] = qt;
                        p.dbg_u[d0 + j] = static_cast<float>(u);
                    }
                }
                rs[4] = rej;
            }
        }
    }
    // ---- ticket: the last row of the sequence finds the first rejection
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) {
        const int tk = atomicAdd(&p.counters[b], 1);
        s_last = (tk == k_b);
        if (s_last) { p.counters[b] = 0; __threadfence(); }          // ready for the next call
    }
    __syncthreads();
    if (!s_last || warp != 0) return;
    __threadfence();

    const double* rs0 = p.row_stats + static_cast<int64_t>(b) * (kMaxK + 1) * kRowStat;
    int n = k_b;
    for (int base = 0; base < k_b; base += 32) {
        const int jj = base + lane;
        bool rej = false;
        if (jj < k_b)
            rej = p.greedy ? (p.draft_tokens[d0 + jj] != static_cast<int>(__ldcg(rs0 + jj * kRowStat)))
                           : (__ldcg(rs0 + jj * kRowStat + 4) != 0.0);
        const unsigned vote = __ballot_sync(0xffffffffu, rej);
        if (vote != 0u && n == k_b) n = base + __ffs(vote) - 1;
    }
    if (lane == 0) {
        p.accepted_len[b] = n;
        const double* rn = rs0 + n * kRowStat;
        if (p.greedy) {
            p.next_token[b] = static_cast<int>(__ldcg(rn));
        } else {
            double* ri = p.row_info + static_cast<int64_t>(b) * 8;
            ri[0] = __ldcg(rn); ri[1] = 1.0 / __ldcg(rn + 1);
            ri[2] = (n < k_b) ? __ldcg(rn + 2) : 0.0; ri[3] = (n < k_b) ? 1.0 / __ldcg(rn + 3) : 1.0;
            ri[4] = __ldcg(rn + 5);
        }
    }
}

cudaError_t launch_sample_decide(const SampleParams& p, int32_t k_batch_max, bool pdl, cudaStream_t stream)
{
    return launch_kernel_ex(sample_decide_kernel, dim3(k_batch_max + 1, p.batch), dim3(kSampleThreads), 0, stream, pdl, p);
}

// ------------------------------------------------------------------------------------ draw
// Row n of one sequence: p_v and the residual max(0, p_v - q_v).  The exponentials are the same
// fp32 2^x as in the statistics pass, so numerator and normaliser share their rounding; products
// and all sums are fp64.
struct DrawRow {
    const float* zt; const float* zd; const uint32_t* mask;
    float mp, mq, c, tau;         // tau: lowest logit of the target row's nucleus (-inf: no top-p filter)
    double inv_sp, inv_sq;
    bool residual;
    __device__ __forceinline__ double prob_p(float z, int v) const
    {
        if (z == -INFINITY || z < tau || !mask_allows(mask, v)) return 0.0;
        return static_cast<double>(fast_exp2((z - mp) * c)) * inv_sp;
    }
    __device__ __forceinline__ double prob_q(float z) const
    {
        if (z == -INFINITY) return 0.0;
        return static_cast<double>(fast_exp2((z - mq) * c)) * inv_sq;
    }
    // loads the 8 consecutive entries starting at v (v % 8 == 0) of the target / draft row
    __device__ __forceinline__ void load8(const float* row, int v, int v_end, bool vec_ok, float (&out)[8]) const
    {
        if (vec_ok && v + 7 < v_end) {
            const float4 a = __ldg(reinterpret_cast<const float4*>(row + v));
            const float4 b = __ldg(reinterpret_cast<const float4*>(row + v + 4));
            out[0] = a.x; out[1] = a.y; out[2] = a.z; out[3] = a.w;
            out[4] = b.x; out[5] = b.y; out[6] = b.z; out[7] = b.w;
        } else {
#pragma unroll
            for (int i = 0; i < 8; ++i) out[i] = (v + i < v_end) ? __ldg(row + v + i) : -INFINITY;
        }
    }
};

__device__ __forceinline__ double warp_inclusive_scan(double v, int lane)
{
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const double t = __shfl_up_sync(0xffffffffu, v, o);
        if (lane >= o) v += t;
    }
    return v;
}

__global__ void __launch_bounds__(kSampleThreads)
sample_draw_kernel(const SampleParams p)
{
    __shared__ double red_r[kSampleWarps];
    __shared__ double red_p[kSampleWarps];
    __shared__ int s_is_last, s_chunk, s_use_p, s_found, s_last;
    __shared__ double s_before, s_thr;

    const int chunk = blockIdx.x;
    const int b = blockIdx.y;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int k_b = p.draft_len[b];
    pdl_wait();                                          // accepted_len and the row statistics come from the decision kernel
    const int n = p.accepted_len[b];
    DrawRow row;
    row.zt = p.logits + static_cast<int64_t>(p.cu_q[b] + n) * p.vocab;
    row.residual = (n < k_b);
    row.zd = row.residual ? p.draft_logits + static_cast<int64_t>(p.cu_d[b] + n) * p.vocab : nullptr;
    row.mask = (p.vocab_mask != nullptr) ? p.vocab_mask + static_cast<int64_t>(b) * p.mask_words : nullptr;
    const double* ri = p.row_info + static_cast<int64_t>(b) * 8;
    row.mp = static_cast<float>(ri[0]); row.inv_sp = ri[1];
    row.mq = static_cast<float>(ri[2]); row.inv_sq = ri[3];
    row.tau = static_cast<float>(ri[4]);
    row.c = p.inv_temp_log2;
    const bool vec_ok = ((p.vocab & 3) == 0);

    // thread t owns the contiguous entries [v0 + 8t, v0 + 8t + 8): vocabulary order is kept
    {
        const int v0 = chunk * kDrawChunk;
        const int v_end = min(p.vocab, v0 + kDrawChunk);
        const int my0 = v0 + threadIdx.x * kDrawElems;
        double mass_r = 0.0, mass_p = 0.0;
        if (my0 < v_end) {
            float zt[8], zd[8];
            row.load8(row.zt, my0, v_end, vec_ok, zt);
            if (row.residual) row.load8(row.zd, my0, v_end, vec_ok, zd);
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const double pv = row.prob_p(zt[i], my0 + i);
                mass_p += pv;
                if (row.residual) { const double d = pv - row.prob_q(zd[i]); mass_r += d > 0.0 ? d : 0.0; }
            }
        }
        mass_r = warp_sum(mass_r);
        mass_p = warp_sum(mass_p);
        if (lane == 0) { red_r[warp] = mass_r; red_p[warp] = mass_p; }
        __syncthreads();
        if (threadIdx.x == 0) {
            double tr = 0.0, tp = 0.0;
#pragma unroll
            for (int w = 0; w < kSampleWarps; ++w) { tr += red_r[w]; tp += red_p[w]; }
            double* cm = p.chunk_mass + (static_cast<int64_t>(b) * p.n_dchunks + chunk) * 2;
            cm[0] = tr; cm[1] = tp;
            __threadfence();
            const int t = atomicAdd(&p.counters[kMaxBatch + b], 1);
            s_is_last = (t == p.n_dchunks - 1);
            if (s_is_last) { p.counters[kMaxBatch + b] = 0; __threadfence(); }
        }
        __syncthreads();
        if (!s_is_last) return;
        __threadfence();
    }

    // ---- the last CTA of the sequence: pick the chunk that holds u' * Z ...
    const double* cm = p.chunk_mass + static_cast<int64_t>(b) * p.n_dchunks * 2;
    if (warp == 0) {
        double z_r = 0.0, z_p = 0.0;
        for (int c0 = 0; c0 < p.n_dchunks; c0 += 32) {
            const int cc = c0 + lane;
            z_r += (cc < p.n_dchunks) ? cm[cc * 2] : 0.0;
            z_p += (cc < p.n_dchunks) ? cm[cc * 2 + 1] : 0.0;
        }
        z_r = warp_sum(z_r);
        z_p = warp_sum(z_p);
        const int use_p = !(row.residual && z_r > 0.0);       // bonus row, or a residual lost to rounding
        const double z_mass = use_p ? z_p : z_r;
        const double thr = philox_uniform(p.seeds[b], static_cast<uint32_t>(n), 1u) * z_mass;
        double carry = 0.0, last_before = 0.0;
        int pick = -1, last_pos = 0;
        double before = 0.0;
        for (int c0 = 0; c0 < p.n_dchunks && pick < 0; c0 += 32) {
            const int cc = c0 + lane;
            const double m = (cc < p.n_dchunks) ? cm[cc * 2 + use_p] : 0.0;
            const double incl = warp_inclusive_scan(m, lane) + carry;
            const unsigned hit = __ballot_sync(0xffffffffu, cc < p.n_dchunks && incl > thr);
            const unsigned pos = __ballot_sync(0xffffffffu, m > 0.0);
            if (hit != 0u) {
                const int l = __ffs(hit) - 1;
                pick = c0 + l;
                before = __shfl_sync(0xffffffffu, incl - m, l);
            } else if (pos != 0u) {
                const int l = 31 - __clz(pos);
                last_pos = c0 + l;
                last_before = __shfl_sync(0xffffffffu, incl - m, l);
            }
            carry = __shfl_sync(0xffffffffu, incl, 31);
        }
        if (pick < 0) { pick = last_pos; before = last_before; }
        if (lane == 0) {
            s_chunk = pick; s_use_p = use_p; s_before = before; s_thr = thr;
            s_found = 0x7fffffff; s_last = -1;
        }
    }
    __syncthreads();

    // ... and scan it in vocabulary order
    const bool use_p = s_use_p != 0;
    const int w0 = s_chunk * kDrawChunk + threadIdx.x * kDrawElems;
    const int w_end = min(p.vocab, (s_chunk + 1) * kDrawChunk);
    double r[8];
    double mine = 0.0;
    {
        float zt[8], zd[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) { zt[i] = -INFINITY; zd[i] = -INFINITY; }
        if (w0 < w_end) {
            row.load8(row.zt, w0, w_end, vec_ok, zt);
            if (!use_p) row.load8(row.zd, w0, w_end, vec_ok, zd);
        }
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            double v = 0.0;
            if (w0 + i < w_end) {
                const double pv = row.prob_p(zt[i], w0 + i);
                if (use_p) v = pv;
                else { const double d = pv - row.prob_q(zd[i]); v = d > 0.0 ? d : 0.0; }
            }
            r[i] = v;
            mine += v;
        }
    }
    const double incl = warp_inclusive_scan(mine, lane);
    if (lane == 31) red_r[warp] = incl;
    __syncthreads();
    double run = s_before + (incl - mine);
    for (int w = 0; w < warp; ++w) run += red_r[w];
    int found = 0x7fffffff, last_pos = -1;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        run += r[i];
        if (r[i] > 0.0) last_pos = w0 + i;
        if (run > s_thr && found == 0x7fffffff && r[i] > 0.0) found = w0 + i;
    }
    if (found != 0x7fffffff) atomicMin(&s_found, found);
    if (last_pos >= 0) atomicMax(&s_last, last_pos);
    __syncthreads();
    if (threadIdx.x == 0) {
        // if rounding left no entry above the threshold: the last entry with positive mass
        p.next_token[b] = (s_found != 0x7fffffff) ? s_found : (s_last >= 0 ? s_last : 0);
    }
}

cudaError_t launch_sample_draw(const SampleParams& p, bool pdl, cudaStream_t stream)
{
    return launch_kernel_ex(sample_draw_kernel, dim3(p.n_dchunks, p.batch), dim3(kSampleThreads), 0, stream, pdl, p);
}

}  // namespace fs
