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
//   plan   : prefix sums of the draft lengths, row -> sequence table, token range check.
//   stats  : grid (vocabulary chunk, row) over all M target rows and S draft rows: chunk max
//            and sum of exp in fp32 (one streaming read of both logit sets).  The last CTA to
//            finish for a sequence (atomic ticket, no waiting) merges the chunk statistics in
//            fp64, evaluates the acceptance tests with Philox uniforms, finds the first
//            rejection by warp vote and stores accepted_len.
//   draw   : grid (chunk, sequence): probability mass of the residual (or of p) per chunk in
//            fp64; the last CTA of a sequence picks the chunk that holds u' * Z and scans it in
//            vocabulary order (inverse CDF).
#include "common.cuh"
#include "internal.h"

namespace fs {

constexpr int kSampleThreads = 256;
constexpr int kElemsPerThread = kSampleChunk / kSampleThreads;   // 32

// ------------------------------------------------------------------------------------ plan
__global__ void __launch_bounds__(kMaxBatch)
plan_kernel(const int32_t* __restrict__ draft_len, const int32_t* __restrict__ draft_tokens, int32_t batch,
            int32_t vocab, Plan plan, int32_t* status)
{
    __shared__ int32_t scan_q[kMaxBatch];
    __shared__ int32_t scan_d[kMaxBatch];
    const int t = threadIdx.x;
    const int k = (t < batch) ? draft_len[t] : 0;
    scan_q[t] = (t < batch) ? k + 1 : 0;
    scan_d[t] = k;
    __syncthreads();
    for (int off = 1; off < kMaxBatch; off <<= 1) {          // inclusive Hillis-Steele scan
        const int aq = (t >= off) ? scan_q[t - off] : 0;
        const int ad = (t >= off) ? scan_d[t - off] : 0;
        __syncthreads();
        scan_q[t] += aq;
        scan_d[t] += ad;
        __syncthreads();
    }
    if (t < batch) {
        const int q0 = scan_q[t] - (k + 1);
        const int d0 = scan_d[t] - k;
        plan.cu_q[t] = q0;
        plan.cu_d[t] = d0;
        for (int j = 0; j <= k; ++j) plan.row_seq[q0 + j] = t;
        if (draft_tokens != nullptr)
            for (int j = 0; j < k; ++j) {
                const int x = draft_tokens[d0 + j];
                if (x < 0 || x >= vocab) report_error(status, kErrBadToken, x, 7);
            }
        if (t == batch - 1) {
            plan.cu_q[batch] = scan_q[t];
            plan.cu_d[batch] = scan_d[t];
        }
    }
}

cudaError_t launch_plan(const int32_t* draft_len, const int32_t* draft_tokens, int32_t batch, int32_t vocab,
                        Plan plan, int32_t* status, cudaStream_t stream)
{
    plan_kernel<<<1, kMaxBatch, 0, stream>>>(draft_len, draft_tokens, batch, vocab, plan, status);
    return cudaGetLastError();
}

// ------------------------------------------------------------------------------------ helpers
__device__ __forceinline__ bool mask_allows(const uint32_t* mask_row, int v)
{
    return mask_row == nullptr || ((mask_row[v >> 5] >> (v & 31)) & 1u);
}

// block-wide reductions over kSampleThreads threads (8 warps)
__device__ __forceinline__ float block_max(float v, float* red)
{
    v = warp_max(v);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
    __syncthreads();
    float r = red[0];
#pragma unroll
    for (int w = 1; w < kSampleThreads / 32; ++w) r = fmaxf(r, red[w]);
    __syncthreads();
    return r;
}
__device__ __forceinline__ float block_sum(float v, float* red)
{
    v = warp_sum(v);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
    __syncthreads();
    float r = 0.f;
#pragma unroll
    for (int w = 0; w < kSampleThreads / 32; ++w) r += red[w];      // fixed order: deterministic
    __syncthreads();
    return r;
}
__device__ __forceinline__ double block_sum(double v, double* red)
{
    v = warp_sum(v);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
    __syncthreads();
    double r = 0.0;
#pragma unroll
    for (int w = 0; w < kSampleThreads / 32; ++w) r += red[w];
    __syncthreads();
    return r;
}

// Merge of per-chunk (max, sum exp2((z - max) * scale)) in chunk order, fp64.
__device__ __forceinline__ void merge_row_stats(const float2* st, int n_chunks, double scale, double& mx, double& sum)
{
    double m = -INFINITY;
    for (int c = 0; c < n_chunks; ++c) m = fmax(m, static_cast<double>(st[c].x));
    double s = 0.0;
    for (int c = 0; c < n_chunks; ++c) {
        const double mc = static_cast<double>(st[c].x);
        if (mc != -INFINITY) s += static_cast<double>(st[c].y) * exp2((mc - m) * scale);
    }
    mx = m;
    sum = s;
}

// ------------------------------------------------------------------------------------ stats + decision
// Rows [0, M) are target rows, rows [M, M+S) draft rows.
__global__ void __launch_bounds__(kSampleThreads)
sample_stats_kernel(const SampleParams p)
{
    __shared__ float red[kSampleThreads / 32];
    __shared__ int red_idx[kSampleThreads / 32];
    __shared__ int s_is_last;

    const int chunk = blockIdx.x;
    const int row = blockIdx.y;
    const bool is_target = row < p.m_rows;
    int b;
    const float* src;
    const uint32_t* mask_row = nullptr;
    if (is_target) {
        b = p.row_seq[row];
        src = p.logits + static_cast<int64_t>(row) * p.vocab;
        if (p.vocab_mask != nullptr) mask_row = p.vocab_mask + static_cast<int64_t>(b) * p.mask_words;
    } else {
        const int dr = row - p.m_rows;
        // sequence of a draft row: the target row with the same (b, j) is row dr + b, so search
        int lo = 0, hi = p.batch - 1;                     // largest b with cu_d[b] <= dr and k_b > 0
        while (lo < hi) {
            const int mid = (lo + hi + 1) >> 1;
            if (p.cu_d[mid] <= dr) lo = mid; else hi = mid - 1;
        }
        b = lo;
        src = p.draft_logits + static_cast<int64_t>(dr) * p.vocab;
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

    if (p.greedy) {
        if (is_target) {
            // lowest index holding the chunk maximum
            int best = 0x7fffffff;
            const float bm = block_max(mx, red);
#pragma unroll
            for (int i = 0; i < kElemsPerThread; ++i) {
                const int v = v0 + ((i >> 2) * kSampleThreads + threadIdx.x) * 4 + (i & 3);
                if (z[i] == bm && v < v_end) best = min(best, v);
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) best = min(best, __shfl_xor_sync(0xffffffffu, best, o));
            if ((threadIdx.x & 31) == 0) red_idx[threadIdx.x >> 5] = best;
            __syncthreads();
            if (threadIdx.x == 0) {
                for (int w = 1; w < kSampleThreads / 32; ++w) best = min(best, red_idx[w]);
                p.stats[static_cast<int64_t>(row) * p.n_chunks + chunk] = make_float2(bm, 0.f);
                p.arg_idx[static_cast<int64_t>(row) * p.n_chunks + chunk] = best;
            }
        }
    } else {
        const float bm = block_max(mx, red);
        const float base = (bm == -INFINITY) ? 0.f : bm;
        float se = 0.f;
#pragma unroll
        for (int i = 0; i < kElemsPerThread; ++i) se += fast_exp2((z[i] - base) * p.inv_temp_log2);
        const float bs = block_sum(se, red);
        if (threadIdx.x == 0) p.stats[static_cast<int64_t>(row) * p.n_chunks + chunk] = make_float2(bm, bs);
    }

    // ---- ticket: the last CTA of sequence b takes the decision
    const int k_b = p.draft_len[b];
    const int expected = (p.greedy ? (k_b + 1) : (2 * k_b + 1)) * p.n_chunks;
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) {
        const int t = atomicAdd(&p.counters[b], 1);
        s_is_last = (t == expected - 1);
        if (s_is_last) p.counters[b] = 0;                 // ready for the next call
    }
    __syncthreads();
    if (!s_is_last) return;
    __threadfence();
    if (threadIdx.x >= 32) return;

    const int q0 = p.cu_q[b], d0 = p.cu_d[b];
    const int lane = threadIdx.x;
    const double scale = static_cast<double>(p.inv_temp_log2);
    int n = k_b;
    if (p.greedy) {
        __shared__ int s_argmax[kMaxK + 1];
        for (int j = lane; j <= k_b; j += 32) {
            const float2* st = p.stats + static_cast<int64_t>(q0 + j) * p.n_chunks;
            const int32_t* ai = p.arg_idx + static_cast<int64_t>(q0 + j) * p.n_chunks;
            float bm = -INFINITY;
            int best = 0;
            for (int c = 0; c < p.n_chunks; ++c)
                if (c == 0 || st[c].x > bm) { bm = st[c].x; best = ai[c]; }     // strict: lowest index wins
            s_argmax[j] = best;
        }
        __syncwarp();
        for (int base = 0; base < k_b; base += 32) {
            const int j = base + lane;
            const bool rej = (j < k_b) && (p.draft_tokens[d0 + j] != s_argmax[j]);
            const unsigned vote = __ballot_sync(0xffffffffu, rej);
            if (vote != 0u && n == k_b) n = base + __ffs(vote) - 1;
        }
        if (lane == 0) {
            p.accepted_len[b] = n;
            p.next_token[b] = s_argmax[n];
        }
        return;
    }

    const uint64_t seed = p.seeds[b];
    for (int base = 0; base < k_b; base += 32) {
        const int j = base + lane;
        bool rej = false;
        if (j < k_b) {
            double mp, sp, mq, sq;
            merge_row_stats(p.stats + static_cast<int64_t>(q0 + j) * p.n_chunks, p.n_chunks, scale, mp, sp);
            merge_row_stats(p.stats + static_cast<int64_t>(p.m_rows + d0 + j) * p.n_chunks, p.n_chunks, scale, mq, sq);
            int x = p.draft_tokens[d0 + j];
            x = min(max(x, 0), p.vocab - 1);
            double zp = static_cast<double>(p.logits[static_cast<int64_t>(q0 + j) * p.vocab + x]);
            if (p.vocab_mask != nullptr &&
                !mask_allows(p.vocab_mask + static_cast<int64_t>(b) * p.mask_words, x)) zp = -INFINITY;
            const double zq = static_cast<double>(p.draft_logits[static_cast<int64_t>(d0 + j) * p.vocab + x]);
            const double pt = (zp == -INFINITY) ? 0.0 : exp2((zp - mp) * scale) / sp;
            const double qt = (zq == -INFINITY) ? 0.0 : exp2((zq - mq) * scale) / sq;
            const double u = philox_uniform(seed, static_cast<uint32_t>(j), 0u);
            rej = !(u * qt < pt);
            if (p.dbg_p != nullptr) {
                p.dbg_p[d0 + j] = pt;
                p.dbg_q[d0 + j] = qt;
                p.dbg_u[d0 + j] = static_cast<float>(u);
            }
        }
        const unsigned vote = __ballot_sync(0xffffffffu, rej);
        if (vote != 0u && n == k_b) n = base + __ffs(vote) - 1;
    }
    if (lane == 0) {
        p.accepted_len[b] = n;
        double mp, sp, mq = 0.0, sq = 0.0;
        merge_row_stats(p.stats + static_cast<int64_t>(q0 + n) * p.n_chunks, p.n_chunks, scale, mp, sp);
        if (n < k_b)
            merge_row_stats(p.stats + static_cast<int64_t>(p.m_rows + d0 + n) * p.n_chunks, p.n_chunks, scale, mq, sq);
        double* ri = p.row_info + static_cast<int64_t>(b) * 4;
        ri[0] = mp; ri[1] = sp; ri[2] = mq; ri[3] = sq;
    }
}

cudaError_t launch_sample_stats(const SampleParams& p, cudaStream_t stream)
{
    const int rows = p.greedy ? p.m_rows : p.m_rows + p.s_rows;
    dim3 grid(p.n_chunks, rows);
    sample_stats_kernel<<<grid, kSampleThreads, 0, stream>>>(p);
    return cudaGetLastError();
}

// ------------------------------------------------------------------------------------ draw
// Residual (or bonus) probability of vocabulary entry v of sequence b, fp64.
struct DrawRow {
    const float* zt; const float* zd; const uint32_t* mask;
    double mp, sp, mq, sq, scale;
    bool residual;
    __device__ __forceinline__ double prob_p(int v) const
    {
        const float z = zt[v];
        if (z == -INFINITY || !mask_allows(mask, v)) return 0.0;
        return exp2((static_cast<double>(z) - mp) * scale) / sp;
    }
    __device__ __forceinline__ double prob_q(int v) const
    {
        const float z = zd[v];
        if (z == -INFINITY) return 0.0;
        return exp2((static_cast<double>(z) - mq) * scale) / sq;
    }
    __device__ __forceinline__ double resid(int v) const
    {
        const double d = prob_p(v) - prob_q(v);
        return d > 0.0 ? d : 0.0;
    }
};

__global__ void __launch_bounds__(kSampleThreads)
sample_draw_kernel(const SampleParams p)
{
    __shared__ double red[kSampleThreads / 32];
    __shared__ double scan[kSampleThreads];
    __shared__ int s_is_last, s_chunk, s_use_p, s_found;
    __shared__ double s_before, s_thr;

    const int chunk = blockIdx.x;
    const int b = blockIdx.y;
    const int k_b = p.draft_len[b];
    const int n = p.accepted_len[b];
    DrawRow row;
    row.zt = p.logits + static_cast<int64_t>(p.cu_q[b] + n) * p.vocab;
    row.residual = (n < k_b);
    row.zd = row.residual ? p.draft_logits + static_cast<int64_t>(p.cu_d[b] + n) * p.vocab : nullptr;
    row.mask = (p.vocab_mask != nullptr) ? p.vocab_mask + static_cast<int64_t>(b) * p.mask_words : nullptr;
    const double* ri = p.row_info + static_cast<int64_t>(b) * 4;
    row.mp = ri[0]; row.sp = ri[1]; row.mq = ri[2]; row.sq = ri[3];
    row.scale = static_cast<double>(p.inv_temp_log2);

    // thread t owns the contiguous elements [v0 + t*32, v0 + t*32 + 32): vocabulary order is kept
    const int v0 = chunk * kSampleChunk;
    const int v_end = min(p.vocab, v0 + kSampleChunk);
    const int my0 = v0 + threadIdx.x * kElemsPerThread;
    double mass_r = 0.0, mass_p = 0.0;
    for (int i = 0; i < kElemsPerThread; ++i) {
        const int v = my0 + i;
        if (v < v_end) {
            const double pv = row.prob_p(v);
            mass_p += pv;
            if (row.residual) { const double d = pv - row.prob_q(v); mass_r += d > 0.0 ? d : 0.0; }
        }
    }
    const double tot_r = block_sum(mass_r, red);
    const double tot_p = block_sum(mass_p, red);
    double* cm = p.chunk_mass + (static_cast<int64_t>(b) * p.n_chunks) * 2;
    if (threadIdx.x == 0) { cm[chunk * 2 + 0] = tot_r; cm[chunk * 2 + 1] = tot_p; }

    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) {
        const int t = atomicAdd(&p.counters[kMaxBatch + b], 1);
        s_is_last = (t == p.n_chunks - 1);
        if (s_is_last) p.counters[kMaxBatch + b] = 0;
    }
    __syncthreads();
    if (!s_is_last) return;
    __threadfence();

    // ---- the last CTA of the sequence: pick the chunk, then scan it in vocabulary order
    if (threadIdx.x == 0) {
        double z_r = 0.0, z_p = 0.0;
        for (int c = 0; c < p.n_chunks; ++c) { z_r += cm[c * 2]; z_p += cm[c * 2 + 1]; }
        const int use_p = !(row.residual && z_r > 0.0);       // bonus row, or a residual lost to rounding
        const double z_mass = use_p ? z_p : z_r;
        const double u2 = philox_uniform(p.seeds[b], static_cast<uint32_t>(n), 1u);
        const double thr = u2 * z_mass;
        double c_run = 0.0, before = 0.0;
        int pick = -1, last_pos = 0;
        double last_before = 0.0;
        for (int c = 0; c < p.n_chunks; ++c) {
            const double m = cm[c * 2 + use_p];
            if (m > 0.0) { last_pos = c; last_before = c_run; }
            if (c_run + m > thr) { pick = c; before = c_run; break; }
            c_run += m;
        }
        if (pick < 0) { pick = last_pos; before = last_before; }
        s_chunk = pick; s_use_p = use_p; s_before = before; s_thr = thr;
        s_found = 0x7fffffff;
    }
    __syncthreads();
    const int pc = s_chunk;
    const bool use_p = s_use_p != 0;
    const int w0 = pc * kSampleChunk + threadIdx.x * kElemsPerThread;
    const int w_end = min(p.vocab, (pc + 1) * kSampleChunk);
    double r[kElemsPerThread];
    double mine = 0.0;
    for (int i = 0; i < kElemsPerThread; ++i) {
        const int v = w0 + i;
        r[i] = (v < w_end) ? (use_p ? row.prob_p(v) : row.resid(v)) : 0.0;
        mine += r[i];
    }
    scan[threadIdx.x] = mine;
    __syncthreads();
    if (threadIdx.x == 0) {                                   // exclusive scan, sequential: exact order
        double run = s_before;
        for (int t = 0; t < kSampleThreads; ++t) { const double m = scan[t]; scan[t] = run; run += m; }
    }
    __syncthreads();
    double run = scan[threadIdx.x];
    int found = 0x7fffffff, last_pos = -1;
    for (int i = 0; i < kElemsPerThread; ++i) {
        run += r[i];
        if (r[i] > 0.0) last_pos = w0 + i;
        if (run > s_thr && found == 0x7fffffff && w0 + i < w_end) found = w0 + i;
    }
    if (found != 0x7fffffff) atomicMin(&s_found, found);
    __syncthreads();
    if (s_found == 0x7fffffff) {
        // rounding left no entry above the threshold: take the last entry with positive mass
        __shared__ int s_last;
        if (threadIdx.x == 0) s_last = -1;
        __syncthreads();
        if (last_pos >= 0) atomicMax(&s_last, last_pos);
        __syncthreads();
        if (threadIdx.x == 0) p.next_token[b] = s_last >= 0 ? s_last : 0;
    } else if (threadIdx.x == 0) {
        p.next_token[b] = s_found;
    }
}

cudaError_t launch_sample_draw(const SampleParams& p, cudaStream_t stream)
{
    dim3 grid(p.n_chunks, p.batch);
    sample_draw_kernel<<<grid, kSampleThreads, 0, stream>>>(p);
    return cudaGetLastError();
}

}  // namespace fs
