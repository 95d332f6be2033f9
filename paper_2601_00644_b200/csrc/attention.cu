// Stage 1: paged-KV grouped-query attention of the k_b+1 query rows of every sequence, causal
// inside the draft window (Section IV-C: the cloud keeps each user's KV session and scores only
// the newly received block; Algorithm 2, Step 2).
//
// Work decomposition.  A "pair" is (sequence b, kv head, block of up to 128 query rows): the
// query rows of all `group` heads that share the kv head, group*(k_b+1) of them, so every K/V
// page is read from HBM once per kv head.  A pair's KV range is cut into blocks of 128 tokens
// (8 pages of 16).  All blocks of the batch, numbered sequence by sequence and pair by pair, are
// divided into equal contiguous ranges, one per CTA, with one CTA per SM: a single balanced wave
// whatever the mix of context lengths and draft lengths.  A CTA therefore works on a few
// "segments" (runs of blocks of one pair).
//
// Inside a CTA: warp 0 is the TMA producer (one 4 KB K and V page per lane, 128-byte swizzle,
// 3 stages of 128 tokens, full/empty mbarriers, every wait bounded); the other warps consume.
// Each consumer warp owns one 16-row tile of the pair and a subset of the pages of every stage:
// QK^T and PV on mma.sync m16n8k16 (bf16 in, fp32 accumulate), fp32 online softmax in registers
// with the row max / sum reduced over the 4 lanes of a quad by shuffles.  At the end of a segment
// every consumer warp writes its unnormalised partial (running max, sum, output tile); a second
// small kernel merges the partials of a pair by log-sum-exp and rounds to bf16.
#include "common.cuh"
#include "internal.h"

namespace fs {

constexpr int kAttPagesPerStage = 8;     // 8 pages = 128 tokens = kAttBlockTokens
constexpr int kAttStages = 3;
constexpr int kPageTokens = 16;
constexpr int kAttMaxThreads = (kAttMaxConsumerWarps + 1) * 32;

template <int DH>
struct AttCfg {
    static constexpr int kHalves = DH / 64;                    // 128-byte column slabs per row
    static constexpr int kSlabBytes = kPageTokens * 128;       // 16 tokens x 64 bf16
    static constexpr int kPageBytes = kHalves * kSlabBytes;    // K (or V) of one page, one kv head
    static constexpr int kStageBytes = kAttPagesPerStage * 2 * kPageBytes;
    static constexpr int kBarOffset = kAttStages * kStageBytes;
    static constexpr int kSmemBytes = kBarOffset + 128 + 1024;  // + barriers + alignment slack
};

// byte offset of 16-byte chunk `c` of row `r` inside a 128-byte-swizzled slab
__device__ __forceinline__ uint32_t swz(uint32_t r, uint32_t c)
{
    return r * 128u + ((c ^ (r & 7u)) << 4);
}

// Position in the batch-wide block list; producer and consumers walk it in lock step.
struct AttCursor {
    int b, pair, blk;             // sequence, pair inside it, block inside the pair
    int k, kvl, nb, rbc, pairs;   // of sequence b: draft length, kv length, blocks per pair,
                                  // row blocks per kv head, pairs
    __device__ __forceinline__ void load_seq(const AttnParams& p)
    {
        k = p.draft_len[b];
        kvl = p.kv_len[b];
        nb = (kvl + kAttBlockTokens - 1) / kAttBlockTokens;
        rbc = (p.group * (k + 1) + kAttRowsPerPair - 1) / kAttRowsPerPair;
        pairs = p.n_kv_heads * rbc;
    }
    __device__ __forceinline__ void start(const AttnParams& p, int2 where)
    {
        b = where.x;
        load_seq(p);
        pair = where.y / nb;
        blk = where.y % nb;
    }
    // returns true when the step left the current pair
    __device__ __forceinline__ bool advance(const AttnParams& p, bool more)
    {
        if (++blk < nb) return false;
        blk = 0;
        if (++pair == pairs) {
            pair = 0;
            ++b;
            if (more && b < p.batch) load_seq(p);
        }
        return true;
    }
};

template <int DH>
__global__ void __launch_bounds__(kAttMaxThreads, 1)
attention_kernel(const __grid_constant__ CUtensorMap kv_map, const AttnParams p)
{
    using Cfg = AttCfg<DH>;
    const int64_t total_blocks = p.seq_blk0[p.batch];
    const int cta = blockIdx.x;
    const int blk_begin = static_cast<int>(cta * total_blocks / gridDim.x);
    const int blk_end = static_cast<int>((cta + 1) * total_blocks / gridDim.x);
    const int n_my = blk_end - blk_begin;
    if (n_my <= 0) return;

    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint64_t* full_bar = reinterpret_cast<uint64_t*>(smem + Cfg::kBarOffset);
    uint64_t* empty_bar = full_bar + kAttStages;

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const int n_cw = (blockDim.x >> 5) - 1;             // consumer warps

    if (threadIdx.x == 0) {
        for (int s = 0; s < kAttStages; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], n_cw); }
        fence_barrier_init();
        tma_prefetch_desc(&kv_map);
    }
    __syncthreads();

    AttCursor cur;
    cur.start(p, p.cta_start[cta]);

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        const uint64_t pol = l2_policy_evict_first();
        for (int q = 0; q < n_my; ++q) {
            const int s = q % kAttStages;
            const int use = q / kAttStages;
            if (use > 0) mbar_wait(&empty_bar[s], (use - 1) & 1, p.status, 1);
            const int kvh = cur.pair / cur.rbc;
            const int t_begin = cur.blk * kAttBlockTokens;
            const int t_end = min(cur.kvl, t_begin + kAttBlockTokens);
            const int npg = (t_end - t_begin + kPageTokens - 1) / kPageTokens;
            if (lane == 0) mbar_arrive_expect_tx(&full_bar[s], static_cast<uint32_t>(npg * 2 * Cfg::kPageBytes));
            __syncwarp();
            if (lane < npg) {
                const int page_idx = cur.blk * kAttPagesPerStage + lane;
                int phys = p.page_table[static_cast<int64_t>(cur.b) * p.max_pages_per_seq + page_idx];
                if (phys < 0 || phys >= p.num_pages) {
                    report_error(p.status, kErrBadPage, phys, 1);
                    phys = 0;                               // stay inside the pool
                }
                uint8_t* dst = smem + s * Cfg::kStageBytes + lane * 2 * Cfg::kPageBytes;
                const int row_k = ((phys * 2 + 0) * p.n_kv_heads + kvh) * kPageTokens;
                const int row_v = ((phys * 2 + 1) * p.n_kv_heads + kvh) * kPageTokens;
#pragma unroll
                for (int hf = 0; hf < Cfg::kHalves; ++hf) {
                    tma_load_2d(dst + hf * Cfg::kSlabBytes, &kv_map, &full_bar[s], hf * 64, row_k, pol);
                    tma_load_2d(dst + Cfg::kPageBytes + hf * Cfg::kSlabBytes, &kv_map, &full_bar[s], hf * 64, row_v, pol);
                }
            }
            __syncwarp();
            cur.advance(p, q + 1 < n_my);
        }
        return;     // consumers wait on every full barrier, so no copy is in flight when the CTA ends
    }

    // ---------------------------------------------------------------------- consumers
    const int cw = warp - 1;
    const int g = lane >> 2, tq = lane & 3;

    uint32_t qa[DH / 16][4];
    float o[DH / 8][4];
    float m_run[2], l_run[2];
    int limit[2];
    int rt = 0, slice = 0, n_slices = 1, n_rt = 1, ctx = 0;
    bool new_segment = true;

    for (int q = 0; q < n_my; ++q) {
        if (new_segment) {
            // ---- set up the pair: row tile of this warp, query fragments, causal limits
            const int kvh = cur.pair / cur.rbc;
            const int row_lo = (cur.pair % cur.rbc) * kAttRowsPerPair;
            const int n_rows = p.group * (cur.k + 1);
            const int rows_here = min(kAttRowsPerPair, n_rows - row_lo);
            n_rt = (rows_here + 15) >> 4;
            rt = cw % n_rt;
            slice = cw / n_rt;
            n_slices = (n_cw - rt + n_rt - 1) / n_rt;
            ctx = cur.kvl - (cur.k + 1);
            const int q_row0 = p.cu_q[cur.b];
#pragma unroll
            for (int i = 0; i < 2; ++i) {
                const int rho = row_lo + rt * 16 + g + i * 8;
                const bool real = rho < n_rows;
                limit[i] = real ? ctx + rho / p.group + 1 : cur.kvl;     // padded rows see everything
                const uint32_t* src = nullptr;
                if (real) {
                    const int j = rho / p.group, hh = rho % p.group;
                    src = reinterpret_cast<const uint32_t*>(
                        p.hidden + (static_cast<int64_t>(q_row0 + j) * p.n_q_heads + kvh * p.group + hh) * DH);
                }
#pragma unroll
                for (int kk = 0; kk < DH / 16; ++kk) {
                    // A fragment of m16n8k16: regs 0/1 = rows g / g+8, cols 2tq..; regs 2/3 = cols 8+2tq..
                    qa[kk][i] = real ? __ldg(src + kk * 8 + tq) : 0u;
                    qa[kk][i + 2] = real ? __ldg(src + kk * 8 + 4 + tq) : 0u;
                }
            }
#pragma unroll
            for (int nt = 0; nt < DH / 8; ++nt) { o[nt][0] = o[nt][1] = o[nt][2] = o[nt][3] = 0.f; }
            m_run[0] = m_run[1] = -INFINITY;
            l_run[0] = l_run[1] = 0.f;
            new_segment = false;
        }

        const int s = q % kAttStages;
        mbar_wait(&full_bar[s], (q / kAttStages) & 1, p.status, 2);
        const int t_begin = cur.blk * kAttBlockTokens;
        const int t_end = min(cur.kvl, t_begin + kAttBlockTokens);
        const int npg = (t_end - t_begin + kPageTokens - 1) / kPageTokens;
        const uint8_t* stage = smem + s * Cfg::kStageBytes;

        for (int pi = slice; pi < npg; pi += n_slices) {
            const uint8_t* kp = stage + pi * 2 * Cfg::kPageBytes;
            const uint8_t* vp = kp + Cfg::kPageBytes;
            const int tok0 = t_begin + pi * kPageTokens;

            // S = Q K^T for 16 rows x 16 tokens
            float sc[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
            {
                const int mi = lane >> 3;
                const uint32_t tok = (mi >> 1) * 8 + (lane & 7);
#pragma unroll
                for (int kk = 0; kk < DH / 16; ++kk) {
                    const int ch = 2 * kk + (mi & 1);
                    uint32_t kb[4];
                    ldmatrix_x4(kb, smem_u32(kp + (ch >> 3) * Cfg::kSlabBytes + swz(tok, ch & 7)));
                    mma_bf16_16816(sc[0], qa[kk], kb[0], kb[1]);
                    mma_bf16_16816(sc[1], qa[kk], kb[2], kb[3]);
                }
            }
            // scale to log2 units, causal mask inside the draft window
            const bool need_mask = (tok0 + kPageTokens > ctx + 1);
#pragma unroll
            for (int nt = 0; nt < 2; ++nt)
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    float v = sc[nt][e] * p.scale_log2;
                    if (need_mask) {
                        const int t = tok0 + nt * 8 + tq * 2 + (e & 1);
                        if (t >= limit[e >> 1]) v = -INFINITY;
                    }
                    sc[nt][e] = v;
                }
            // online softmax: row max over the quad, rescale, exponentiate
            float alpha[2];
#pragma unroll
            for (int i = 0; i < 2; ++i) {
                float mx = fmaxf(fmaxf(sc[0][2 * i], sc[0][2 * i + 1]), fmaxf(sc[1][2 * i], sc[1][2 * i + 1]));
                mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
                mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
                const float m_new = fmaxf(m_run[i], mx);
                const float m_safe = (m_new == -INFINITY) ? 0.f : m_new;
                alpha[i] = fast_exp2(m_run[i] - m_safe);
                m_run[i] = m_new;
                float rs = 0.f;
#pragma unroll
                for (int nt = 0; nt < 2; ++nt) {
                    sc[nt][2 * i] = fast_exp2(sc[nt][2 * i] - m_safe);
                    sc[nt][2 * i + 1] = fast_exp2(sc[nt][2 * i + 1] - m_safe);
                    rs += sc[nt][2 * i] + sc[nt][2 * i + 1];
                }
                l_run[i] = l_run[i] * alpha[i] + rs;
            }
            uint32_t pa[4];
            pa[0] = pack_bf16(sc[0][0], sc[0][1]);
            pa[1] = pack_bf16(sc[0][2], sc[0][3]);
            pa[2] = pack_bf16(sc[1][0], sc[1][1]);
            pa[3] = pack_bf16(sc[1][2], sc[1][3]);
            // O = alpha * O + P V
            {
                const int mi = lane >> 3;
                const uint32_t tok = (mi & 1) * 8 + (lane & 7);
#pragma unroll
                for (int dp = 0; dp < DH / 16; ++dp) {
                    const int ch = 2 * dp + (mi >> 1);
                    uint32_t vb[4];
                    ldmatrix_x4_trans(vb, smem_u32(vp + (ch >> 3) * Cfg::kSlabBytes + swz(tok, ch & 7)));
#pragma unroll
                    for (int h2 = 0; h2 < 2; ++h2) {
                        float (&acc)[4] = o[2 * dp + h2];
                        acc[0] *= alpha[0]; acc[1] *= alpha[0];
                        acc[2] *= alpha[1]; acc[3] *= alpha[1];
                        mma_bf16_16816(acc, pa, vb[2 * h2], vb[2 * h2 + 1]);
                    }
                }
            }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&empty_bar[s]);           // this warp is done with stage s

        const int pair_global = p.seq_pair0[cur.b] + cur.pair;
        const bool left_pair = cur.advance(p, q + 1 < n_my);
        if (left_pair || q + 1 == n_my) {
            // ---- end of the segment: this warp's partial -> slot (pair + CTA), unique per segment
#pragma unroll
            for (int i = 0; i < 2; ++i) {
                l_run[i] += __shfl_xor_sync(0xffffffffu, l_run[i], 1);
                l_run[i] += __shfl_xor_sync(0xffffffffu, l_run[i], 2);
            }
            const int64_t slot = static_cast<int64_t>(pair_global + cta) * kAttMaxConsumerWarps + cw;
            float* po = p.part_o + slot * 16 * DH;
            float* pml = p.part_ml + slot * 16 * 2;
            const bool has = (m_run[0] != -INFINITY) || (m_run[1] != -INFINITY);
            if (has) {
#pragma unroll
                for (int nt = 0; nt < DH / 8; ++nt) {
                    *reinterpret_cast<float2*>(po + g * DH + nt * 8 + tq * 2) = make_float2(o[nt][0], o[nt][1]);
                    *reinterpret_cast<float2*>(po + (g + 8) * DH + nt * 8 + tq * 2) = make_float2(o[nt][2], o[nt][3]);
                }
            }
            if (tq == 0) {
                *reinterpret_cast<float2*>(pml + g * 2) = make_float2(m_run[0], l_run[0]);
                *reinterpret_cast<float2*>(pml + (g + 8) * 2) = make_float2(m_run[1], l_run[1]);
            }
            new_segment = true;
        }
    }
}

// Merge of a pair's partials: out = sum_i 2^(m_i - M) o_i / sum_i 2^(m_i - M) l_i, rounded to bf16.
// The partials of pair P were written by the CTAs whose block ranges intersect the pair's blocks,
// by every consumer warp that shares the row tile.
__global__ void __launch_bounds__(256)
attention_combine_kernel(const CombineParams p)
{
    const int b = blockIdx.y;
    const int k_b = p.draft_len[b];
    const int kvl = p.kv_len[b];
    const int nb = (kvl + kAttBlockTokens - 1) / kAttBlockTokens;
    const int n_rows = p.group * (k_b + 1);
    const int rbc = (n_rows + kAttRowsPerPair - 1) / kAttRowsPerPair;
    const int pair = blockIdx.x;
    if (pair >= p.n_kv_heads * rbc) return;
    const int kvh = pair / rbc;
    const int row_lo = (pair % rbc) * kAttRowsPerPair;
    const int rows_here = min(kAttRowsPerPair, n_rows - row_lo);
    const int n_rt = (rows_here + 15) >> 4;

    const int64_t total_blocks = p.seq_blk0[p.batch];
    const int64_t blk_first = p.seq_blk0[b] + static_cast<int64_t>(pair) * nb;
    const int64_t blk_last = blk_first + nb - 1;
    // CTA c owns blocks [c*T/G, (c+1)*T/G): the owner of block x is ceil((x+1)*G/T) - 1
    const int c0 = static_cast<int>(((blk_first + 1) * p.n_ctas - 1) / total_blocks);
    const int c1 = static_cast<int>(((blk_last + 1) * p.n_ctas - 1) / total_blocks);
    const int pair_global = p.seq_pair0[b] + pair;
    const int q_row0 = p.cu_q[b];
    const int dh = p.head_dim;
    const int cols4 = dh / 4;

    for (int idx = threadIdx.x; idx < rows_here * cols4; idx += blockDim.x) {
        const int r = idx / cols4;
        const int c4 = (idx % cols4) * 4;
        const int tile = r >> 4, rr = r & 15;
        const int slices = (p.n_cw - tile + n_rt - 1) / n_rt;
        float m_all = -INFINITY;
        for (int c = c0; c <= c1; ++c)
            for (int sl = 0; sl < slices; ++sl) {
                const int64_t slot = static_cast<int64_t>(pair_global + c) * kAttMaxConsumerWarps + tile + sl * n_rt;
                m_all = fmaxf(m_all, p.part_ml[(slot * 16 + rr) * 2]);
            }
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        float l_all = 0.f;
        for (int c = c0; c <= c1; ++c)
            for (int sl = 0; sl < slices; ++sl) {
                const int64_t slot = static_cast<int64_t>(pair_global + c) * kAttMaxConsumerWarps + tile + sl * n_rt;
                const float2 ml = *reinterpret_cast<const float2*>(p.part_ml + (slot * 16 + rr) * 2);
                if (ml.x == -INFINITY) continue;             // that warp saw no visible token
                const float wgt = fast_exp2(ml.x - m_all);
                l_all += wgt * ml.y;
                const float4 v = *reinterpret_cast<const float4*>(p.part_o + (slot * 16 + rr) * dh + c4);
                acc.x += wgt * v.x; acc.y += wgt * v.y; acc.z += wgt * v.z; acc.w += wgt * v.w;
            }
        const int rho = row_lo + r;
        const int j = rho / p.group, hh = rho % p.group;
        const int64_t out_row = static_cast<int64_t>(q_row0 + j) * p.n_q_heads + kvh * p.group + hh;
        const float inv = 1.f / l_all;
        __nv_bfloat162 lo = __floats2bfloat162_rn(acc.x * inv, acc.y * inv);
        __nv_bfloat162 hi = __floats2bfloat162_rn(acc.z * inv, acc.w * inv);
        uint2 pk;
        pk.x = *reinterpret_cast<uint32_t*>(&lo);
        pk.y = *reinterpret_cast<uint32_t*>(&hi);
        *reinterpret_cast<uint2*>(p.attn_out + out_row * dh + c4) = pk;
    }
}

cudaError_t attention_init(int head_dim)
{
    if (head_dim == 128)
        return cudaFuncSetAttribute(attention_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                    AttCfg<128>::kSmemBytes);
    return cudaFuncSetAttribute(attention_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                AttCfg<64>::kSmemBytes);
}

// consumer warps per CTA for a batch whose largest pair has `max_tile_rows` query rows
int attention_consumer_warps(int max_tile_rows)
{
    const int rows = max_tile_rows > kAttRowsPerPair ? kAttRowsPerPair : max_tile_rows;
    const int rt = rows > 0 ? (rows + 15) / 16 : 1;
    int slices = (8 + rt / 2) / rt;                  // round(8 / rt) ...
    if (slices < 1) slices = 1;                      // ... at least 1
    int w = rt * slices;
    if (w > kAttMaxConsumerWarps) w = rt;
    return w;
}

cudaError_t launch_attention(const Handle& h, const CUtensorMap& kv_map, const AttnParams& p, int32_t n_ctas,
                             int32_t n_cw, cudaStream_t stream)
{
    dim3 grid(n_ctas);
    dim3 block((n_cw + 1) * 32);
    if (h.cfg.head_dim == 128)
        attention_kernel<128><<<grid, block, AttCfg<128>::kSmemBytes, stream>>>(kv_map, p);
    else
        attention_kernel<64><<<grid, block, AttCfg<64>::kSmemBytes, stream>>>(kv_map, p);
    return cudaGetLastError();
}

cudaError_t launch_attention_combine(const CombineParams& p, cudaStream_t stream)
{
    dim3 grid(p.pairs_per_seq_max, p.batch);
    attention_combine_kernel<<<grid, 256, 0, stream>>>(p);
    return cudaGetLastError();
}

}  // namespace fs
