// Stage 2: LM-head projection logits[M][V] = X[M][d] . W[V][d]^T (the frozen head of the target,
// Section IV-A; the scores of Algorithm 2, Step 2) on the 5th-generation tensor cores.
//
// The vocabulary is the large dimension and M (a few to a few hundred token rows) the small one,
// so the operands are swapped: a 128-row tile of W is the MMA's A operand (M = 128) and the token
// rows are its B operand (N = n_tile <= 256), both K-major bf16 staged by TMA with the 128-byte
// swizzle.  The fp32 accumulator D[128 vocab rows][token columns] lives in TMEM; with lanes =
// vocabulary rows, a warp's store of one token column is 32 consecutive floats of a logits row.
//
// Persistent CTAs (one per SM) walk over the vocabulary tiles.  Warp 0 is the TMA producer, warp 1
// issues tcgen05.mma from one thread and owns the TMEM allocation, warps 2..17 drain the
// accumulators.  Shared-memory stages and the (double-buffered, when it fits) accumulators are
// handed over through mbarriers; every wait is bounded.
//
// W is streamed from HBM exactly once per pass; X (M x d bf16, L2 resident) is re-read per tile.
// On request the epilogue also leaves the softmax statistics of every row (maximum and sum of
// exponentials, or maximum and arg-max) per 32 vocabulary rows, so that the sampling stage does
// not have to read the logits again to normalise them.
#include "common.cuh"
#include "internal.h"

namespace fs {

constexpr int kLmBlockV = 128;          // vocabulary rows per tile (MMA M)
constexpr int kLmBlockK = 64;           // bf16 elements per 128-byte swizzle row
constexpr int kLmUmmaK = 16;
constexpr int kLmEpilogueWarps = 16;
constexpr int kLmThreads = (2 + kLmEpilogueWarps) * 32;   // TMA warp, MMA warp, epilogue warps
constexpr int kLmMaxStages = 12;
constexpr int kLmATileBytes = kLmBlockV * kLmBlockK * 2;     // 16 KB
constexpr int kLmTmemCols = 512;
constexpr int kLmMaxAccBufs = 8;        // accumulator ring (buffers of n_tile TMEM columns)
constexpr int kLmSmemLimit = 232448;    // 227 KB opt-in maximum per CTA
constexpr int kLmBarBytes = 512;

static inline int lm_stage_bytes(int n_tile, int n_blocks) { return kLmATileBytes + n_blocks * n_tile * 128; }

int lm_head_pick_stages(int n_tile, int n_blocks)
{
    int s = (kLmSmemLimit - 1024 - kLmBarBytes) / lm_stage_bytes(n_tile, n_blocks);
    if (s > kLmMaxStages) s = kLmMaxStages;
    return s;
}
size_t lm_head_smem_bytes(int n_tile, int n_blocks, int num_stages)
{
    return static_cast<size_t>(num_stages) * lm_stage_bytes(n_tile, n_blocks) + 1024 + kLmBarBytes;
}

__global__ void __launch_bounds__(kLmThreads, 1)
lm_head_kernel(const __grid_constant__ CUtensorMap w_map, const __grid_constant__ CUtensorMap w_map_last,
               const __grid_constant__ CUtensorMap x_map, const LmHeadParams p)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const int b_bytes = p.n_blocks * p.n_tile * 128;
    const int stage_bytes = kLmATileBytes + b_bytes;
    uint64_t* full_bar = reinterpret_cast<uint64_t*>(smem + p.num_stages * stage_bytes);
    uint64_t* empty_bar = full_bar + kLmMaxStages;
    uint64_t* tmem_full = empty_bar + kLmMaxStages;
    uint64_t* tmem_empty = tmem_full + kLmMaxAccBufs;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(tmem_empty + kLmMaxAccBufs);

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    pdl_launch_dependents();                             // let the next kernel of the stream be set up while this one runs

    if (threadIdx.x == 0) {
        for (int s = 0; s < p.num_stages; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], 1); }
        for (int a = 0; a < p.n_bufs; ++a) { mbar_init(&tmem_full[a], 1); mbar_init(&tmem_empty[a], kLmEpilogueWarps); }
        fence_barrier_init();
        tma_prefetch_desc(&w_map);
        tma_prefetch_desc(&w_map_last);
        tma_prefetch_desc(&x_map);
    }
    if (warp == 1) {
        tmem_alloc(tmem_slot, kLmTmemCols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    const int num_kb = p.d_model / kLmBlockK;
    const int total_tiles = p.n_vtiles * p.n_pass;
    // Vocabulary tile vt: the first n_full_tiles are 128 rows high; the tiles of the last wave are
    // last_rows high (one per CTA, so that the wave ends everywhere at the same time).
    auto tile_row0 = [&](int vt) {
        return vt < p.n_full_tiles ? vt * kLmBlockV : p.n_full_tiles * kLmBlockV + (vt - p.n_full_tiles) * p.last_rows;
    };
    // Accumulators: a ring of n_bufs buffers of n_tile TMEM columns; a tile takes n_blocks consecutive
    // buffers, one per block of token columns.  With a buffer to spare the MMAs of the next tile start
    // (and, where two blocks share the ring with one spare, continue as soon as the epilogue has
    // drained the first block) while the epilogue still drains this tile.
    const int rows_per_pass = p.n_blocks * p.n_tile;

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            const uint64_t pol_w = l2_policy_evict_first();
            const uint64_t pol_x = l2_policy_evict_last();
            int s = 0;
            uint32_t ph = 0;
            int last_s = -1;
            uint32_t last_ph = 0;
            bool ok = true;
            uint8_t* st = smem;
            for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x) {
                const int vt = tile / p.n_pass, pass = tile % p.n_pass;
                // the tile's k blocks lie one after the other in the re-tiled copy of W, w_rows rows of 64 elements each
                const int w_rows = vt < p.n_full_tiles ? kLmBlockV : p.last_rows;
                const int w_row0 = vt < p.n_full_tiles ? vt * num_kb * kLmBlockV
                                                       : (p.n_full_tiles * kLmBlockV + (vt - p.n_full_tiles) * p.last_rows) * num_kb;
                const bool full_tile = vt < p.n_full_tiles;
                const CUtensorMap* wm = full_tile ? &w_map : &w_map_last;
                const uint32_t tx = static_cast<uint32_t>(full_tile ? stage_bytes : p.last_rows * 128 + b_bytes);
                const int x_row0 = pass * rows_per_pass;
                int w_row = w_row0;
                for (int kb = 0; kb < num_kb; ++kb, w_row += w_rows) {
                    if (!mbar_wait(&empty_bar[s], ph ^ 1u, p.status, 2)) { ok = false; break; }
                    mbar_arrive_expect_tx(&full_bar[s], tx);
                    tma_load_2d(st, wm, &full_bar[s], 0, w_row, pol_w);
                    tma_load_2d(st + kLmATileBytes, &x_map, &full_bar[s], kb * kLmBlockK, x_row0, pol_x);
                    if (p.n_blocks > 1)
                        tma_load_2d(st + kLmATileBytes + p.n_tile * 128, &x_map, &full_bar[s], kb * kLmBlockK, x_row0 + p.n_tile, pol_x);
                    last_s = s; last_ph = ph;
                    st += stage_bytes;
                    if (++s == p.num_stages) { s = 0; ph ^= 1u; st = smem; }
                }
            }
            // do not leave while a copy of ours may still be landing in shared memory
            if (last_s >= 0) mbar_wait(&full_bar[last_s], last_ph, p.status, 3);
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            const uint32_t idesc = umma_idesc_bf16(kLmBlockV, static_cast<uint32_t>(p.n_tile));
            int s = 0;
            uint32_t ph = 0;
            int seq = 0;                                 // accumulator buffers handed out so far
            bool ok = true;
            uint32_t a_addr = smem_u32(smem);
            for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x) {
                // the tile's accumulator buffers: their previous contents must have been drained (use u of a
                // buffer waits for the epilogue of use u - 1; a fresh barrier lets use 0 through)
                const int slot0 = seq % p.n_bufs, slot1 = (seq + 1) % p.n_bufs;
                if (!mbar_wait(&tmem_empty[slot0], (static_cast<uint32_t>(seq / p.n_bufs) & 1u) ^ 1u, p.status, 4)) { ok = false; break; }
                if (p.n_blocks > 1 &&
                    !mbar_wait(&tmem_empty[slot1], (static_cast<uint32_t>((seq + 1) / p.n_bufs) & 1u) ^ 1u, p.status, 4)) { ok = false; break; }
                tc_fence_after();
                const uint32_t acc0 = tmem_base + static_cast<uint32_t>(slot0 * p.n_tile);
                const uint32_t acc1 = tmem_base + static_cast<uint32_t>(slot1 * p.n_tile);
                for (int kb = 0; kb < num_kb; ++kb) {
                    if (!mbar_wait(&full_bar[s], ph, p.status, 5)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t b_addr = a_addr + kLmATileBytes;
                    if (p.n_blocks == 1) {
#pragma unroll
                        for (int k = 0; k < kLmBlockK / kLmUmmaK; ++k) {
                            const uint64_t da = umma_desc_k_sw128(a_addr + k * kLmUmmaK * 2);
                            const uint64_t db = umma_desc_k_sw128(b_addr + k * kLmUmmaK * 2);
                            umma_bf16(acc0, da, db, idesc, (kb > 0 || k > 0) ? 1u : 0u);
                        }
                    } else {
                        // two blocks of token columns share the W tile: the two MMAs of a 16-wide slice follow one
                        // another, the first keeps its A operand in the collector and the second takes it from
                        // there, so the slice of W is read from shared memory once, not twice
#pragma unroll
                        for (int k = 0; k < kLmBlockK / kLmUmmaK; ++k) {
                            const uint64_t da = umma_desc_k_sw128(a_addr + k * kLmUmmaK * 2);
                            const uint64_t db0 = umma_desc_k_sw128(b_addr + k * kLmUmmaK * 2);
                            const uint64_t db1 = umma_desc_k_sw128(b_addr + p.n_tile * 128 + k * kLmUmmaK * 2);
                            const uint32_t accum = (kb > 0 || k > 0) ? 1u : 0u;
                            umma_bf16_a_fill(acc0, da, db0, idesc, accum);
                            umma_bf16_a_lastuse(acc1, da, db1, idesc, accum);
                        }
                    }
                    umma_commit(&empty_bar[s]);          // stage is free once these MMAs have read it
                    a_addr += static_cast<uint32_t>(stage_bytes);
                    if (++s == p.num_stages) { s = 0; ph ^= 1u; a_addr = smem_u32(smem); }
                }
                if (ok) {                                // accumulators complete
                    umma_commit(&tmem_full[slot0]);
                    if (p.n_blocks > 1) umma_commit(&tmem_full[slot1]);
                }
                seq += p.n_blocks;
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue (16 warps)
        // four warps per quarter of the TMEM lanes (a warp reaches the lanes 32 * (warp % 4) ...), each taking
        // every fourth group of 16 token columns
        const int quarter = warp & 3;                    // TMEM lanes 32*quarter .. +31
        const int half = (warp - 2) >> 2;
        int seq = 0;
        bool ok = true;
        for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x) {
          const int vt = tile / p.n_pass, pass = tile % p.n_pass;
          const int tile_rows = vt < p.n_full_tiles ? kLmBlockV : p.last_rows;
          const int v = (quarter * 32 + lane < tile_rows) ? tile_row0(vt) + quarter * 32 + lane : p.vocab;   // past the tile: not a row
          for (int nb = 0; nb < p.n_blocks && ok; ++nb, ++seq) {
            const int slot = seq % p.n_bufs;
            if (!mbar_wait(&tmem_full[slot], static_cast<uint32_t>(seq / p.n_bufs) & 1u, p.status, 6)) { ok = false; break; }
            tc_fence_after();
            const int row_base = pass * rows_per_pass + nb * p.n_tile;
            const uint32_t taddr0 = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) +
                                    static_cast<uint32_t>(slot * p.n_tile);
            for (int c0 = half * 16; c0 < p.n_tile; c0 += (kLmEpilogueWarps / 4) * 16) {
                if (row_base + c0 >= p.m_rows) break;    // warp-uniform
                uint32_t r[16];
                tmem_ld_x16(taddr0 + static_cast<uint32_t>(c0), r);
                tmem_ld_wait();
                if (v < p.vocab) {
#pragma unroll
                    for (int i = 0; i < 16; ++i) {
                        const int row = row_base + c0 + i;
                        if (row < p.m_rows)
                            p.logits[static_cast<int64_t>(row) * p.vocab + v] = __uint_as_float(r[i]);
                    }
                }
                if (p.tstats != nullptr) {
                    // softmax statistics of this warp's 32 vocabulary rows for each of the 16 token
                    // columns; the 16 reductions are interleaved so that their shuffle chains overlap.
                    // Columns past m_rows hold zeros (out-of-range rows of X) and are not stored.
                    float zv[16], mx[16], sc[16];
                    uint32_t allow = 0xffffu;
                    if (p.vocab_mask != nullptr && v < p.vocab) {
#pragma unroll
                        for (int i = 0; i < 16; ++i) {
                            const int row = min(row_base + c0 + i, p.m_rows - 1);
                            const uint32_t w = __ldg(p.vocab_mask + static_cast<int64_t>(__ldg(p.row_seq + row)) * p.mask_words + (v >> 5));
                            if (((w >> (v & 31)) & 1u) == 0u) allow &= ~(1u << i);
                        }
                    }
#pragma unroll
                    for (int i = 0; i < 16; ++i) zv[i] = (v < p.vocab && ((allow >> i) & 1u)) ? __uint_as_float(r[i]) : -INFINITY;
#pragma unroll
                    for (int i = 0; i < 16; ++i) mx[i] = redux_max(zv[i]);
                    if (p.greedy) {
#pragma unroll
                        for (int i = 0; i < 16; ++i) {
                            const unsigned eq = __ballot_sync(0xffffffffu, zv[i] == mx[i]);
                            sc[i] = __int_as_float(tile_row0(vt) + quarter * 32 + __ffs(eq) - 1);
                        }
                    } else {
                        // log2(e) / T of every column's sequence (lane i < 16 fetches column i's)
                        float c_lane = p.inv_temp_log2;
                        if (p.row_c != nullptr && lane < 16) c_lane = __ldg(p.row_c + min(row_base + c0 + lane, p.m_rows - 1));
#pragma unroll
                        for (int i = 0; i < 16; ++i)
                            sc[i] = fast_exp2((zv[i] - ((mx[i] == -INFINITY) ? 0.f : mx[i])) *
                                              (p.row_c != nullptr ? __shfl_sync(0xffffffffu, c_lane, i) : p.inv_temp_log2));
                        // 16 sums over the 32 lanes by halving exchanges (8 + 4 + 2 + 1 + 1 shuffles instead of 80):
                        // a lane keeps the half of the columns its lane bit selects and adds its partner's share,
                        // so that lanes 2 c and 2 c + 1 end up with the sum of column c
#pragma unroll
                        for (int o = 16, w = 8; o > 1; o >>= 1, w >>= 1) {
                            const bool up = (lane & o) != 0;
#pragma unroll
                            for (int i = 0; i < 8; ++i) {
                                if (i < w) {
                                    const float give = up ? sc[i] : sc[i + w];
                                    const float keep = up ? sc[i + w] : sc[i];
                                    sc[i] = keep + __shfl_xor_sync(0xffffffffu, give, o);
                                }
                            }
                        }
                        sc[0] += __shfl_xor_sync(0xffffffffu, sc[0], 1);
                    }
                    // lane l now holds column l >> 1 (GREEDY: every lane holds all 16 arg-max indices)
                    const int col = lane >> 1;
                    float part_m = -INFINITY, part_s = p.greedy ? 0.f : sc[0];
#pragma unroll
                    for (int i = 0; i < 16; ++i)
                        if (col == i) { part_m = mx[i]; if (p.greedy) part_s = sc[i]; }
                    if ((lane & 1) == 0 && row_base + c0 + col < p.m_rows)
                        p.tstats[static_cast<int64_t>(row_base + c0 + col) * p.n_tparts + vt * 4 + quarter] =
                            make_float2(part_m, part_s);
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&tmem_empty[slot]);
          }
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, kLmTmemCols);
    }
}

cudaError_t lm_head_init()
{
    return cudaFuncSetAttribute(lm_head_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kLmSmemLimit);
}

// W in the order the kernel streams it: for every vocabulary tile (n_full tiles of 128 rows, then n_last tiles of
// last_rows rows) its d / 64 k blocks one after the other, each a [tile rows][64] bf16 block (16 KB for a full
// tile), so that a stage of the pipeline is one contiguous piece of memory instead of 128 pieces of 128 bytes a
// whole row of W apart.  Rows past the vocabulary are zero.  One thread moves 16 bytes.
__global__ void retile_w_kernel(const __nv_bfloat16* __restrict__ w, __nv_bfloat16* __restrict__ out, int vocab, int d_model,
                                int n_full, int n_last, int last_rows)
{
    const int num_kb = d_model / kLmBlockK;
    const int64_t rows_total = static_cast<int64_t>(n_full) * kLmBlockV + static_cast<int64_t>(n_last) * last_rows;
    const int64_t n_chunks = rows_total * num_kb * 8;                 // 16-byte chunks of the copy
    const int64_t full_rows = static_cast<int64_t>(n_full) * num_kb * kLmBlockV;
    for (int64_t q = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x; q < n_chunks; q += static_cast<int64_t>(gridDim.x) * blockDim.x) {
        const int64_t R = q >> 3;                                     // row of 64 elements in the copy
        const int c = static_cast<int>(q & 7);
        int64_t src_row;
        int kb;
        if (R < full_rows) {
            const int64_t t = R / kLmBlockV;
            src_row = (t / num_kb) * kLmBlockV + R % kLmBlockV;
            kb = static_cast<int>(t % num_kb);
        } else {
            const int64_t t = (R - full_rows) / last_rows;
            src_row = static_cast<int64_t>(n_full) * kLmBlockV + (t / num_kb) * last_rows + (R - full_rows) % last_rows;
            kb = static_cast<int>(t % num_kb);
        }
        uint4 v = make_uint4(0u, 0u, 0u, 0u);
        if (src_row < vocab) v = *reinterpret_cast<const uint4*>(w + src_row * d_model + kb * kLmBlockK + c * 8);
        *reinterpret_cast<uint4*>(out + q * 8) = v;
    }
}

cudaError_t launch_retile_w(const void* w, void* out, int vocab, int d_model, int n_full, int n_last, int last_rows,
                            cudaStream_t stream)
{
    retile_w_kernel<<<2048, 256, 0, stream>>>(static_cast<const __nv_bfloat16*>(w), static_cast<__nv_bfloat16*>(out), vocab, d_model,
                                              n_full, n_last, last_rows);
    return cudaGetLastError();
}

cudaError_t launch_lm_head(const Handle& h, const CUtensorMap& x_map, const LmHeadParams& p, cudaStream_t stream)
{
    const int total_tiles = p.n_vtiles * p.n_pass;
    const int grid = total_tiles < h.sm_count ? total_tiles : h.sm_count;
    const size_t smem = lm_head_smem_bytes(p.n_tile, p.n_blocks, p.num_stages);
    lm_head_kernel<<<grid, kLmThreads, smem, stream>>>(h.w_map, h.w_map_last, x_map, p);
    return cudaGetLastError();
}

}  // namespace fs
