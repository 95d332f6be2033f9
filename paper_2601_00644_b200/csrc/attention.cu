// Stage 1: paged-KV grouped-query attention of the k_b+1 query rows of every sequence, causal
// inside the draft window (Section IV-C: the cloud keeps each user's KV session and scores only
// the newly received block; Algorithm 2, Step 2).
//
// One CTA handles (sequence b, kv head, KV split).  The query rows of all `group` heads that
// share the kv head form one tile of group*(k_b+1) rows, so every K/V page is read from HBM once
// per kv head.  K/V pages (16 tokens) are brought in by TMA with the 128-byte swizzle, 8 pages
// per pipeline stage; QK^T and PV run on mma.sync m16n8k16 (bf16 in, fp32 accumulate) with an
// fp32 online softmax in registers (row max / sum over the 4 lanes of a quad by shuffles).
// Each warp owns one 16-row tile and a subset of the pages of every stage; warps that share a
// row tile are merged through shared memory at the end.  With more than one split the CTA writes
// an unnormalised partial (running max, sum, output); a second kernel merges splits.
#include "common.cuh"
#include "internal.h"

namespace fs {

constexpr int kAttPagesPerStage = 8;     // 8 pages = 128 tokens = kAttSplitQuantum
constexpr int kAttStages = 3;
constexpr int kAttMaxWarps = 10;
constexpr int kAttRowsPerCta = 128;
constexpr int kPageTokens = 16;

template <int DH>
struct AttCfg {
    static constexpr int kHalves = DH / 64;                    // 128-byte column slabs per row
    static constexpr int kSlabBytes = kPageTokens * 128;       // 16 tokens x 64 bf16
    static constexpr int kPageBytes = kHalves * kSlabBytes;    // K (or V) of one page, one kv head
    static constexpr int kStageBytes = kAttPagesPerStage * 2 * kPageBytes;
    static constexpr int kQSlabBytes = kAttRowsPerCta * 128;
    static constexpr int kQBytes = kHalves * kQSlabBytes;
    static constexpr int kBarOffset = kAttStages * kStageBytes + kQBytes;
    static constexpr int kSmemBytes = kBarOffset + 64 + 1024;  // + barriers/misc + alignment slack
    static constexpr int kMergeRowFloats = DH + 4;             // padded row of the merge buffer
};

// byte offset of 16-byte chunk `c` of row `r` inside a 128-byte-swizzled slab
__device__ __forceinline__ uint32_t swz(uint32_t r, uint32_t c)
{
    return r * 128u + ((c ^ (r & 7u)) << 4);
}

template <int DH>
__global__ void __launch_bounds__(kAttMaxWarps * 32, 1)
attention_split_kernel(const __grid_constant__ CUtensorMap kv_map, const AttnParams p)
{
    using Cfg = AttCfg<DH>;
    const int split = blockIdx.x;
    const int kvh = blockIdx.y / p.row_blocks;
    const int rb = blockIdx.y % p.row_blocks;
    const int b = blockIdx.z;

    const int k_b = p.draft_len[b];
    const int kvl = p.kv_len[b];
    const int ctx = kvl - (k_b + 1);
    const int n_rows = p.group * (k_b + 1);           // query rows of this (sequence, kv head)
    const int row_lo = rb * kAttRowsPerCta;
    if (row_lo >= n_rows) return;
    const int n_split = (kvl + p.split_len - 1) / p.split_len;
    if (split >= n_split) return;
    const int rows_here = min(kAttRowsPerCta, n_rows - row_lo);
    const int n_rt = (rows_here + 15) >> 4;           // 16-row tiles in this CTA
    const int t_begin = split * p.split_len;
    const int t_end = min(kvl, t_begin + p.split_len);
    const int n_pages = (t_end - t_begin + kPageTokens - 1) / kPageTokens;
    const int n_iter = (n_pages + kAttPagesPerStage - 1) / kAttPagesPerStage;
    const int q_row0 = p.cu_q[b];

    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t* q_smem = smem + kAttStages * Cfg::kStageBytes;
    uint64_t* full_bar = reinterpret_cast<uint64_t*>(smem + Cfg::kBarOffset);

    const int tid = threadIdx.x;
    const int warp = tid >> 5;
    const int lane = tid & 31;
    const int n_warps = blockDim.x >> 5;

    if (tid == 0) {
        for (int s = 0; s < kAttStages; ++s) mbar_init(&full_bar[s], 1);
        fence_barrier_init();
        tma_prefetch_desc(&kv_map);
    }
    __syncthreads();

    // ---- producer: lanes 0..7 of warp 0 each fetch one page (K and V) of the stage
    const uint64_t pol = l2_policy_evict_first();
    auto issue_stage = [&](int it) {
        const int s = it % kAttStages;
        const int pg0 = it * kAttPagesPerStage;
        const int npg = min(kAttPagesPerStage, n_pages - pg0);
        if (lane == 0) mbar_arrive_expect_tx(&full_bar[s], static_cast<uint32_t>(npg * 2 * Cfg::kPageBytes));
        __syncwarp();
        if (lane < npg) {
            const int page_idx = t_begin / kPageTokens + pg0 + lane;
            int phys = p.page_table[static_cast<int64_t>(b) * p.max_pages_per_seq + page_idx];
            if (phys < 0 || phys >= p.num_pages) {
                report_error(p.status, kErrBadPage, phys, 1);
                phys = 0;                                   // stay inside the pool
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
    };
    if (warp == 0) {
        for (int it = 0; it < min(kAttStages, n_iter); ++it) issue_stage(it);
    }

    // ---- query tile -> shared memory (swizzled like the K/V slabs), then per-warp fragments
    {
        const int chunks_per_row = DH / 8;
        const int total = n_rt * 16 * chunks_per_row;
        for (int idx = tid; idx < total; idx += blockDim.x) {
            const int r = idx / chunks_per_row;
            const int ch = idx % chunks_per_row;
            uint4 v = make_uint4(0u, 0u, 0u, 0u);
            const int rho = row_lo + r;
            if (rho < n_rows) {
                const int j = rho / p.group, hh = rho % p.group;
                const __nv_bfloat16* src = p.hidden +
                    (static_cast<int64_t>(q_row0 + j) * p.n_q_heads + kvh * p.group + hh) * DH + ch * 8;
                v = *reinterpret_cast<const uint4*>(src);
            }
            *reinterpret_cast<uint4*>(q_smem + (ch >> 3) * Cfg::kQSlabBytes + swz(r, ch & 7)) = v;
        }
    }
    __syncthreads();

    // warp -> (row tile, slice of the pages of each stage)
    const int rt = warp % n_rt;
    const int slice = warp / n_rt;
    const int n_slices = (n_warps - rt + n_rt - 1) / n_rt;       // warps sharing this row tile

    uint32_t qa[DH / 16][4];
    {
        const int mi = lane >> 3;
        const int r = rt * 16 + (mi & 1) * 8 + (lane & 7);
#pragma unroll
        for (int kk = 0; kk < DH / 16; ++kk) {
            const int ch = 2 * kk + (mi >> 1);
            ldmatrix_x4(qa[kk], smem_u32(q_smem + (ch >> 3) * Cfg::kQSlabBytes + swz(r, ch & 7)));
        }
    }

    // rows of this thread inside the tile: g and g+8; their causal limits
    const int g = lane >> 2, tq = lane & 3;
    int limit[2];
#pragma unroll
    for (int i = 0; i < 2; ++i) {
        const int rho = row_lo + rt * 16 + g + i * 8;
        limit[i] = (rho < n_rows) ? ctx + rho / p.group + 1 : kvl;    // padded rows see everything
    }

    float o[DH / 8][4];
#pragma unroll
    for (int nt = 0; nt < DH / 8; ++nt) { o[nt][0] = o[nt][1] = o[nt][2] = o[nt][3] = 0.f; }
    float m_run[2] = {-INFINITY, -INFINITY};
    float l_run[2] = {0.f, 0.f};

    for (int it = 0; it < n_iter; ++it) {
        const int s = it % kAttStages;
        mbar_wait(&full_bar[s], (it / kAttStages) & 1, p.status, 1);
        const int pg0 = it * kAttPagesPerStage;
        const int npg = min(kAttPagesPerStage, n_pages - pg0);
        const uint8_t* stage = smem + s * Cfg::kStageBytes;

        for (int pi = slice; pi < npg; pi += n_slices) {
            const uint8_t* kp = stage + pi * 2 * Cfg::kPageBytes;
            const uint8_t* vp = kp + Cfg::kPageBytes;
            const int tok0 = t_begin + (pg0 + pi) * kPageTokens;

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
                    for (int q = 0; q < 2; ++q) {
                        float (&acc)[4] = o[2 * dp + q];
                        acc[0] *= alpha[0]; acc[1] *= alpha[0];
                        acc[2] *= alpha[1]; acc[3] *= alpha[1];
                        mma_bf16_16816(acc, pa, vb[2 * q], vb[2 * q + 1]);
                    }
                }
            }
        }
        __syncthreads();                               // every warp is done with stage s
        if (warp == 0 && it + kAttStages < n_iter) issue_stage(it + kAttStages);
    }

    // ---- merge the warps that share a row tile, then write the result / the split partial
#pragma unroll
    for (int i = 0; i < 2; ++i) {
        l_run[i] += __shfl_xor_sync(0xffffffffu, l_run[i], 1);
        l_run[i] += __shfl_xor_sync(0xffffffffu, l_run[i], 2);
    }
    float* mo = reinterpret_cast<float*>(smem);                                   // [warp][16][DH+4]
    float* mml = mo + kAttMaxWarps * 16 * Cfg::kMergeRowFloats;                   // [warp][16][2]
    {
        float* my = mo + warp * 16 * Cfg::kMergeRowFloats;
#pragma unroll
        for (int nt = 0; nt < DH / 8; ++nt) {
            *reinterpret_cast<float2*>(my + g * Cfg::kMergeRowFloats + nt * 8 + tq * 2) = make_float2(o[nt][0], o[nt][1]);
            *reinterpret_cast<float2*>(my + (g + 8) * Cfg::kMergeRowFloats + nt * 8 + tq * 2) = make_float2(o[nt][2], o[nt][3]);
        }
        if (tq == 0) {
            mml[(warp * 16 + g) * 2 + 0] = m_run[0];
            mml[(warp * 16 + g) * 2 + 1] = l_run[0];
            mml[(warp * 16 + g + 8) * 2 + 0] = m_run[1];
            mml[(warp * 16 + g + 8) * 2 + 1] = l_run[1];
        }
    }
    __syncthreads();

    const int cols4 = DH / 4;
    for (int idx = tid; idx < rows_here * cols4; idx += blockDim.x) {
        const int r = idx / cols4;
        const int c4 = (idx % cols4) * 4;
        const int tile = r >> 4, rr = r & 15;
        const int slices = (n_warps - tile + n_rt - 1) / n_rt;
        float m_all = -INFINITY;
        for (int sl = 0; sl < slices; ++sl) m_all = fmaxf(m_all, mml[((tile + sl * n_rt) * 16 + rr) * 2]);
        const float m_safe = (m_all == -INFINITY) ? 0.f : m_all;
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        float l_all = 0.f;
        for (int sl = 0; sl < slices; ++sl) {
            const int w = tile + sl * n_rt;
            const float wgt = fast_exp2(mml[(w * 16 + rr) * 2] - m_safe);
            l_all += wgt * mml[(w * 16 + rr) * 2 + 1];
            const float4 v = *reinterpret_cast<const float4*>(mo + (w * 16 + rr) * Cfg::kMergeRowFloats + c4);
            acc.x += wgt * v.x; acc.y += wgt * v.y; acc.z += wgt * v.z; acc.w += wgt * v.w;
        }
        const int rho = row_lo + r;
        const int j = rho / p.group, hh = rho % p.group;
        const int64_t out_row = static_cast<int64_t>(q_row0 + j) * p.n_q_heads + kvh * p.group + hh;
        if (n_split == 1) {
            const float inv = 1.f / l_all;
            __nv_bfloat162 lo = __floats2bfloat162_rn(acc.x * inv, acc.y * inv);
            __nv_bfloat162 hi = __floats2bfloat162_rn(acc.z * inv, acc.w * inv);
            uint2 pk;
            pk.x = *reinterpret_cast<uint32_t*>(&lo);
            pk.y = *reinterpret_cast<uint32_t*>(&hi);
            *reinterpret_cast<uint2*>(p.attn_out + out_row * DH + c4) = pk;
        } else {
            const int64_t prow = static_cast<int64_t>(split) * p.part_stride + out_row;
            *reinterpret_cast<float4*>(p.part_o + prow * DH + c4) = acc;
            if (c4 == 0) {
                p.part_ml[prow * 2 + 0] = m_all;
                p.part_ml[prow * 2 + 1] = l_all;
            }
        }
    }
}

// Merge of the KV splits: out = sum_s 2^(m_s - M) o_s / sum_s 2^(m_s - M) l_s, rounded to bf16.
__global__ void __launch_bounds__(256)
attention_combine_kernel(const CombineParams p)
{
    const int b = blockIdx.y;
    const int j = blockIdx.x;
    const int k_b = p.draft_len[b];
    if (j > k_b) return;
    const int kvl = p.kv_len[b];
    const int n_split = (kvl + p.split_len - 1) / p.split_len;
    if (n_split <= 1) return;                       // the attention kernel wrote the result itself
    const int64_t row = p.cu_q[b] + j;
    const int dh4 = p.head_dim / 4;
    const int total = p.n_q_heads * dh4;
    for (int idx = threadIdx.x; idx < total; idx += blockDim.x) {
        const int h = idx / dh4;
        const int c4 = (idx % dh4) * 4;
        const int64_t rh = row * p.n_q_heads + h;
        float m_all = -INFINITY;
        for (int s = 0; s < n_split; ++s) m_all = fmaxf(m_all, p.part_ml[(s * p.part_stride + rh) * 2]);
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        float l_all = 0.f;
        for (int s = 0; s < n_split; ++s) {
            const int64_t pr = s * p.part_stride + rh;
            const float wgt = fast_exp2(p.part_ml[pr * 2] - m_all);
            l_all += wgt * p.part_ml[pr * 2 + 1];
            const float4 v = *reinterpret_cast<const float4*>(p.part_o + pr * p.head_dim + c4);
            acc.x += wgt * v.x; acc.y += wgt * v.y; acc.z += wgt * v.z; acc.w += wgt * v.w;
        }
        const float inv = 1.f / l_all;
        __nv_bfloat162 lo = __floats2bfloat162_rn(acc.x * inv, acc.y * inv);
        __nv_bfloat162 hi = __floats2bfloat162_rn(acc.z * inv, acc.w * inv);
        uint2 pk;
        pk.x = *reinterpret_cast<uint32_t*>(&lo);
        pk.y = *reinterpret_cast<uint32_t*>(&hi);
        *reinterpret_cast<uint2*>(p.attn_out + rh * p.head_dim + c4) = pk;
    }
}

cudaError_t attention_init(int head_dim)
{
    if (head_dim == 128)
        return cudaFuncSetAttribute(attention_split_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                    AttCfg<128>::kSmemBytes);
    return cudaFuncSetAttribute(attention_split_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                AttCfg<64>::kSmemBytes);
}

// warps per CTA for a batch whose largest (sequence, kv head) tile has `max_rows` query rows
static int attention_warps(int max_rows)
{
    const int rows = max_rows > kAttRowsPerCta ? kAttRowsPerCta : max_rows;
    const int rt = rows > 0 ? (rows + 15) / 16 : 1;
    int slices = (8 + rt / 2) / rt;                  // round(8 / rt) ...
    if (slices < 1) slices = 1;                      // ... at least 1
    int w = rt * slices;
    if (w > kAttMaxWarps) w = rt;
    return w;
}

cudaError_t launch_attention(const Handle& h, const CUtensorMap& kv_map, const AttnParams& p, int32_t batch,
                             int32_t max_rows_per_seq, int32_t max_splits, cudaStream_t stream)
{
    const int max_tile_rows = p.group * max_rows_per_seq;
    dim3 grid(max_splits, p.n_kv_heads * p.row_blocks, batch);
    dim3 block(attention_warps(max_tile_rows) * 32);
    if (h.cfg.head_dim == 128)
        attention_split_kernel<128><<<grid, block, AttCfg<128>::kSmemBytes, stream>>>(kv_map, p);
    else
        attention_split_kernel<64><<<grid, block, AttCfg<64>::kSmemBytes, stream>>>(kv_map, p);
    return cudaGetLastError();
}

cudaError_t launch_attention_combine(const CombineParams& p, int32_t batch, cudaStream_t stream)
{
    dim3 grid(p.rows_per_seq_max, batch);
    attention_combine_kernel<<<grid, 256, 0, stream>>>(p);
    return cudaGetLastError();
}

}  // namespace fs
