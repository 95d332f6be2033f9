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
// "segments" (runs of blocks of one pair).  Every CTA derives its own range from draft_len[] and
// kv_len[] (a block-wide prefix sum over the sequences), so no planning kernel runs first.
//
// Both contractions run on the 5th-generation tensor cores with accumulators in tensor memory
// (the legacy warp-level MMA path cannot keep up with the KV stream):
//   S[128 query rows][128 tokens] = Q K^T     A = Q tile, B = K tile, both K-major in shared memory
//   O[128 query rows][Dh]        += P V       A = P (bf16, written by the softmax threads),
//                                             B = V tile as TMA delivers it ([token][Dh]: MN-major)
// The query rows of the pair occupy the first rows of the M = 128 tile; the remaining rows are
// padding whose results are never read.
//
// Warp roles.  Warp 0: TMA producer (one 16-token K and V page per lane, 128-byte swizzle, a ring
// of 128-token stages).  Warp 1: one thread issues every tcgen05.mma; the warp owns the TMEM
// allocation.  Warps 2..5: softmax, one thread per TMEM lane (= tile row, so a row's maximum and
// sum need no shuffles): two passes over the scores of the block with tcgen05.ld -- maximum, then
// p = 2^(s - m) written to shared memory as bf16 -- with S double buffered so that the next
// block's QK^T overlaps.  A pair with at most 32 (64) rows is replicated 4 (2) times over the
// tile rows and each copy takes a quarter (half) of the block's tokens, so all four warps work
// on small pairs.  The running maximum is only raised when it grew by more than 2^8 (O in TMEM
// is then rescaled); the final division by the row sum makes the stale maximum cancel.  At the end of a segment the softmax threads read O from TMEM; if the
// pair spans several CTAs they park (m, l, O) in global scratch and the CTA that completes the
// pair last (atomic ticket, nobody waits) merges the parts by log-sum-exp in CTA order.
// Every mbarrier wait is bounded.
#include "common.cuh"
#include "internal.h"

namespace fs {

constexpr int kPageTokens = 16;
constexpr int kAttPagesPerStage = kAttBlockTokens / kPageTokens;    // 8
constexpr int kAttSoftmaxThreads = 128;
constexpr int kAttTmemCols = 512;
constexpr uint32_t kTmemS0 = 0, kTmemS1 = 128, kTmemO = 256;        // column offsets
constexpr float kRescaleThreshold = 8.f;                             // log2 units

template <int DH>
struct AttCfg {
    static constexpr int kSlabs = DH / 64;                     // 128-byte column slabs per row
    static constexpr int kSlabBytes = 128 * 128;               // 128 rows x 64 bf16
    static constexpr int kStageBytes = 2 * kSlabs * kSlabBytes;      // K slabs, then V slabs
    static constexpr int kStages = (DH == 128) ? 2 : 4;
    static constexpr int kQOffset = kStages * kStageBytes;
    static constexpr int kQBytes = kSlabs * kSlabBytes;
    static constexpr int kPOffset = kQOffset + kQBytes;
    static constexpr int kPBytes = 2 * kSlabBytes;             // 128 rows x 128 tokens bf16
    static constexpr int kBarOffset = kPOffset + 2 * kPBytes;
    static constexpr int kSmemBytes = kBarOffset + 256 + 1024; // + barriers + alignment slack
};

struct AttBars {
    uint64_t kv_full[4], kv_empty[4];
    uint64_t s_full[2], s_empty[2];
    uint64_t p_full[2], p_empty[2];
    uint64_t q_full, o_full, group;
    uint32_t tmem_slot;
};
static_assert(sizeof(AttBars) <= 256, "barrier block");

__device__ __forceinline__ void prefetch_l2(const void* p)
{
    asm volatile("prefetch.global.L2 [%0];" ::"l"(p));
}

// 32 lanes x 32 consecutive fp32 columns: thread i of the warp reads TMEM lane (base lane + i).
__device__ __forceinline__ void tmem_ld_x32(uint32_t taddr, uint32_t (&r)[32])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tmem_st_x32(uint32_t taddr, const uint32_t (&r)[32])
{
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
        "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
        ::"r"(taddr),
          "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
          "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]),
          "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]),
          "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
        : "memory");
}
__device__ __forceinline__ void tmem_st_wait()
{
    asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
}

// Shared-memory matrix descriptor of an MN-major bf16 operand laid out by TMA with the 128-byte
// swizzle: rows of 64 MN-elements (128 B) indexed by k, groups of 8 k-rows `sbo` bytes apart,
// the next 64 MN-elements `lbo` bytes away.
__device__ __forceinline__ uint64_t umma_desc_mn_sw128(uint32_t smem_addr, uint32_t lbo, uint32_t sbo)
{
    uint64_t d = 0;
    d |= static_cast<uint64_t>((smem_addr & 0x3FFFFu) >> 4);
    d |= static_cast<uint64_t>((lbo >> 4) & 0x3FFFu) << 16;
    d |= static_cast<uint64_t>((sbo >> 4) & 0x3FFFu) << 32;
    d |= static_cast<uint64_t>(1) << 46;                       // descriptor version of this architecture
    d |= static_cast<uint64_t>(2) << 61;                       // 128-byte swizzle
    return d;
}
constexpr uint32_t kIdescBMajorMN = 1u << 16;

// Exclusive prefix sum over the block of one int per thread; returns the block total in `total`.
__device__ __forceinline__ int block_exclusive_scan(int v, int* warp_tot, int& total)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int n_warps = (blockDim.x + 31) >> 5;
    int incl = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int t = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += t;
    }
    if (lane == 31) warp_tot[warp] = incl;
    __syncthreads();
    int before = 0, sum = 0;
    for (int w = 0; w < n_warps; ++w) {
        const int t = warp_tot[w];
        if (w < warp) before += t;
        sum += t;
    }
    __syncthreads();
    total = sum;
    return before + incl - v;
}

// Position in the batch-wide block list; every role walks it in lock step.
struct AttCursor {
    int b, pair, blk;             // sequence, pair inside it, block inside the pair
    int k, kvl, nb, rbc, pairs;   // of sequence b: draft length, kv length, blocks per pair,
                                  // row blocks per kv head, pairs
    int q_row0, pair0, blk0;      // first query row / first pair / first block of sequence b
    __device__ __forceinline__ void load_seq(const AttnParams& p)
    {
        k = p.draft_len[b];
        kvl = p.kv_len[b];
        nb = (kvl + kAttBlockTokens - 1) / kAttBlockTokens;
        rbc = (p.group * (k + 1) + kAttRowsPerPair - 1) / kAttRowsPerPair;
        pairs = p.n_kv_heads * rbc;
    }
    // returns true when the step left the current pair
    __device__ __forceinline__ bool advance(const AttnParams& p, bool more)
    {
        if (++blk < nb) return false;
        blk = 0;
        if (++pair == pairs) {
            pair = 0;
            q_row0 += k + 1;
            pair0 += pairs;
            blk0 += pairs * nb;
            ++b;
            if (more && b < p.batch) load_seq(p);
        }
        return true;
    }
};

struct AttStart { int b, blk_off, q_row0, pair0, blk0, total; };

template <int DH>
__global__ void __launch_bounds__(kAttThreads, 1)
attention_kernel(const __grid_constant__ CUtensorMap kv_map, const AttnParams p)
{
    using Cfg = AttCfg<DH>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    AttBars* bars = reinterpret_cast<AttBars*>(smem + Cfg::kBarOffset);
    __shared__ int s_warp_tot[32];
    __shared__ AttStart s_start;
    __shared__ int s_flag;
    __shared__ float s_xch[3][kAttSoftmaxThreads];          // [0..1] row maxima (by block parity), [2] row sums, exchanged between the copies of a row

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const int cta = blockIdx.x;

    if (threadIdx.x == 0) {
        for (int s = 0; s < 4; ++s) { mbar_init(&bars->kv_full[s], 1); mbar_init(&bars->kv_empty[s], 1); }
        for (int a = 0; a < 2; ++a) {
            mbar_init(&bars->s_full[a], 1); mbar_init(&bars->s_empty[a], kAttSoftmaxThreads);
            mbar_init(&bars->p_full[a], kAttSoftmaxThreads); mbar_init(&bars->p_empty[a], 1);
        }
        mbar_init(&bars->q_full, kAttSoftmaxThreads);
        mbar_init(&bars->o_full, 1);
        mbar_init(&bars->group, kAttSoftmaxThreads);
        fence_barrier_init();
        tma_prefetch_desc(&kv_map);
    }
    if (warp == 1) {
        tmem_alloc(&bars->tmem_slot, kAttTmemCols);
        tmem_relinquish();
    }

    // ---- where this CTA starts: prefix sums of blocks / pairs / rows over the sequences
    int blk_begin, n_my;
    {
        const int per = (p.batch + blockDim.x - 1) / blockDim.x;
        const int b_lo = min(p.batch, static_cast<int>(threadIdx.x) * per);
        const int b_hi = min(p.batch, b_lo + per);
        int my_blocks = 0, my_pairs = 0, my_rows = 0;
        for (int b = b_lo; b < b_hi; ++b) {
            const int k = p.draft_len[b];
            const int nb = (p.kv_len[b] + kAttBlockTokens - 1) / kAttBlockTokens;
            const int pairs = p.n_kv_heads * ((p.group * (k + 1) + kAttRowsPerPair - 1) / kAttRowsPerPair);
            my_blocks += pairs * nb;
            my_pairs += pairs;
            my_rows += k + 1;
        }
        int total, unused;
        const int ex_blocks = block_exclusive_scan(my_blocks, s_warp_tot, total);
        const int ex_pairs = block_exclusive_scan(my_pairs, s_warp_tot, unused);
        const int ex_rows = block_exclusive_scan(my_rows, s_warp_tot, unused);
        const int64_t t64 = total;
        blk_begin = static_cast<int>(cta * t64 / gridDim.x);
        n_my = static_cast<int>((cta + 1) * t64 / gridDim.x) - blk_begin;
        if (n_my > 0 && blk_begin >= ex_blocks && blk_begin < ex_blocks + my_blocks) {
            int blk0 = ex_blocks, pair0 = ex_pairs, row0 = ex_rows;
            for (int b = b_lo; b < b_hi; ++b) {
                const int k = p.draft_len[b];
                const int nb = (p.kv_len[b] + kAttBlockTokens - 1) / kAttBlockTokens;
                const int pairs = p.n_kv_heads * ((p.group * (k + 1) + kAttRowsPerPair - 1) / kAttRowsPerPair);
                if (blk_begin < blk0 + pairs * nb) {
                    s_start.b = b; s_start.blk_off = blk_begin - blk0;
                    s_start.q_row0 = row0; s_start.pair0 = pair0; s_start.blk0 = blk0;
                    break;
                }
                blk0 += pairs * nb; pair0 += pairs; row0 += k + 1;
            }
        }
        if (threadIdx.x == 0) s_start.total = total;
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = bars->tmem_slot;
    const int64_t total_blocks = s_start.total;

    AttCursor cur;
    if (n_my > 0) {
        cur.b = s_start.b;
        cur.q_row0 = s_start.q_row0; cur.pair0 = s_start.pair0; cur.blk0 = s_start.blk0;
        cur.load_seq(p);
        cur.pair = s_start.blk_off / cur.nb;
        cur.blk = s_start.blk_off % cur.nb;
    }

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        const uint64_t pol = l2_policy_evict_first();
        bool new_pair = true;
        bool ok = true;
        int last_st = -1;
        uint32_t last_ph = 0;
        for (int q = 0; q < n_my && ok; ++q) {
            const int kvh = cur.pair / cur.rbc;
            if (new_pair) {
                // bring the pair's query rows into L2 ahead of the softmax threads that copy them
                const int row_lo = (cur.pair % cur.rbc) * kAttRowsPerPair;
                const int rows_here = min(kAttRowsPerPair, p.group * (cur.k + 1) - row_lo);
                const int j_lo = row_lo / p.group, j_hi = (row_lo + rows_here - 1) / p.group;
                const int lines_per_j = (p.group * DH * 2 + 127) / 128;
                for (int i = lane; i < (j_hi - j_lo + 1) * lines_per_j; i += 32) {
                    const int j = j_lo + i / lines_per_j;
                    const uint8_t* base = reinterpret_cast<const uint8_t*>(
                        p.hidden + (static_cast<int64_t>(cur.q_row0 + j) * p.n_q_heads + kvh * p.group) * DH);
                    prefetch_l2(base + (i % lines_per_j) * 128);
                }
            }
            const int st = q % Cfg::kStages;
            const int use = q / Cfg::kStages;
            if (use > 0 && !mbar_wait(&bars->kv_empty[st], (use - 1) & 1, p.status, 1)) { ok = false; break; }
            const int t_begin = cur.blk * kAttBlockTokens;
            const int t_end = min(cur.kvl, t_begin + kAttBlockTokens);
            const int npg = (t_end - t_begin + kPageTokens - 1) / kPageTokens;
            if (lane == 0)
                mbar_arrive_expect_tx(&bars->kv_full[st], static_cast<uint32_t>(npg * 2 * Cfg::kSlabs * kPageTokens * 128));
            __syncwarp();
            if (lane < npg) {
                const int page_idx = cur.blk * kAttPagesPerStage + lane;
                int phys = p.page_table[static_cast<int64_t>(cur.b) * p.max_pages_per_seq + page_idx];
                if (phys < 0 || phys >= p.num_pages) {
                    report_error(p.status, kErrBadPage, phys, 1);
                    phys = 0;                               // stay inside the pool
                }
                uint8_t* dst = smem + st * Cfg::kStageBytes + lane * (kPageTokens * 128);
                const int row_k = ((phys * 2 + 0) * p.n_kv_heads + kvh) * kPageTokens;
                const int row_v = ((phys * 2 + 1) * p.n_kv_heads + kvh) * kPageTokens;
#pragma unroll
                for (int hf = 0; hf < Cfg::kSlabs; ++hf) {
                    tma_load_2d(dst + hf * Cfg::kSlabBytes, &kv_map, &bars->kv_full[st], hf * 64, row_k, pol);
                    tma_load_2d(dst + (Cfg::kSlabs + hf) * Cfg::kSlabBytes, &kv_map, &bars->kv_full[st], hf * 64, row_v, pol);
                }
            }
            __syncwarp();
            last_st = st; last_ph = use & 1;
            new_pair = cur.advance(p, q + 1 < n_my);
        }
        // do not leave while a copy of ours may still be landing in shared memory
        if (last_st >= 0) mbar_wait(&bars->kv_full[last_st], last_ph, p.status, 9);
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0 && n_my > 0) {
            const uint32_t idesc_s = umma_idesc_bf16(128, 128);
            const uint32_t idesc_o = umma_idesc_bf16(128, DH) | kIdescBMajorMN;
            const uint32_t q_addr = smem_u32(smem + Cfg::kQOffset);
            bool ok = true;
            int seg = 0;
            // S[q & 1] = Q K^T of block q (waits: the pair's Q tile, the K/V stage, the S buffer)
            auto issue_s = [&](int q, bool seg_first, int seg_idx) -> bool {
                const int st = q % Cfg::kStages, buf = q & 1, u = q >> 1;
                if (seg_first && !mbar_wait(&bars->q_full, seg_idx & 1, p.status, 2)) return false;
                if (!mbar_wait(&bars->kv_full[st], (q / Cfg::kStages) & 1, p.status, 3)) return false;
                if (u > 0 && !mbar_wait(&bars->s_empty[buf], (u - 1) & 1, p.status, 4)) return false;
                tc_fence_after();
                const uint32_t k_addr = smem_u32(smem + st * Cfg::kStageBytes);
                const uint32_t acc = tmem_base + (buf ? kTmemS1 : kTmemS0);
#pragma unroll
                for (int kk = 0; kk < DH / 16; ++kk) {
                    const uint32_t off = (kk >> 2) * Cfg::kSlabBytes + (kk & 3) * 32;
                    umma_bf16(acc, umma_desc_k_sw128(q_addr + off), umma_desc_k_sw128(k_addr + off), idesc_s, kk > 0 ? 1u : 0u);
                }
                umma_commit(&bars->s_full[buf]);
                return true;
            };
            bool seg_first = true;
            ok = issue_s(0, true, 0);
            for (int q = 0; q < n_my && ok; ++q) {
                const bool seg_last = (cur.blk == cur.nb - 1) || (q + 1 == n_my);
                const int st = q % Cfg::kStages, buf = q & 1, u = q >> 1;
                if (!seg_last && q + 1 < n_my) { if (!issue_s(q + 1, false, seg)) { ok = false; break; } }   // overlap with softmax of q
                if (!mbar_wait(&bars->p_full[buf], u & 1, p.status, 5)) { ok = false; break; }
                tc_fence_after();
                {
                    const uint32_t p_addr = smem_u32(smem + Cfg::kPOffset + buf * Cfg::kPBytes);
                    const uint32_t v_addr = smem_u32(smem + st * Cfg::kStageBytes + Cfg::kSlabs * Cfg::kSlabBytes);
#pragma unroll
                    for (int ks = 0; ks < kAttBlockTokens / 16; ++ks) {
                        const uint64_t da = umma_desc_k_sw128(p_addr + (ks >> 2) * Cfg::kSlabBytes + (ks & 3) * 32);
                        const uint64_t db = umma_desc_mn_sw128(v_addr + ks * 2048, Cfg::kSlabBytes, 1024);
                        umma_bf16(tmem_base + kTmemO, da, db, idesc_o, (seg_first && ks == 0) ? 0u : 1u);
                    }
                }
                umma_commit(&bars->kv_empty[st]);
                umma_commit(&bars->p_empty[buf]);
                umma_commit(&bars->o_full);
                cur.advance(p, q + 1 < n_my);
                seg_first = seg_last;
                if (seg_last) {
                    ++seg;
                    if (q + 1 < n_my && !issue_s(q + 1, true, seg)) { ok = false; break; }
                }
            }
        }
    } else {
        // ------------------------------------------------------------------ softmax
        // Thread t owns TMEM lane t.  When the pair has at most 32 (64) query rows the Q tile holds
        // 4 (2) copies of them, copy c in tile rows [c*span, (c+1)*span), span = 128 / copies, and
        // the thread of tile row c*span + r handles tokens [c*span, (c+1)*span) of row r in every
        // block: all four warps share the work of a small pair.  The copies agree on the row
        // maximum through shared memory and write their part of P into row r of ONE P tile, so O is
        // complete in tile rows [0, span) and needs no merge.
        const int quarter = warp & 3;                       // TMEM lanes 32*quarter .. +31
        const int t = quarter * 32 + lane;                  // tile row
        const uint32_t t_lane = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16);
        uint8_t* q_smem = smem + Cfg::kQOffset;
        bool ok = true;
        bool seg_first = true;
        int seg = 0;
        uint32_t group_phase = 0;
        float m_used = -INFINITY, l_run = 0.f;
        int rows_here = 0, row_lo = 0, limit = 0, ctx = 0;
        int copies = 1, span = 128, c = 0, r = t;

        // all softmax threads meet; bounded like every other wait
        auto group_sync = [&](int where) -> bool {
            mbar_arrive(&bars->group);
            const bool done = mbar_wait(&bars->group, group_phase, p.status, where);
            group_phase ^= 1u;
            return done;
        };

        for (int q = 0; q < n_my && ok; ++q) {
            const int kvh = cur.pair / cur.rbc;
            if (seg_first) {
                // ---- the pair's query rows -> shared memory in the K-major swizzled layout of operand A
                row_lo = (cur.pair % cur.rbc) * kAttRowsPerPair;
                const int n_rows = p.group * (cur.k + 1);
                rows_here = min(kAttRowsPerPair, n_rows - row_lo);
                ctx = cur.kvl - (cur.k + 1);
                copies = rows_here <= 32 ? 4 : (rows_here <= 64 ? 2 : 1);
                span = kAttRowsPerPair / copies;
                c = t / span;
                r = t % span;
                if (r < rows_here) {
                    const int rho = row_lo + r;
                    const int j = rho / p.group, hh = rho % p.group;
                    limit = ctx + j + 1;
                    const uint4* src = reinterpret_cast<const uint4*>(
                        p.hidden + (static_cast<int64_t>(cur.q_row0 + j) * p.n_q_heads + kvh * p.group + hh) * DH);
                    uint4 v[DH / 8];
#pragma unroll
                    for (int ch = 0; ch < DH / 8; ++ch) v[ch] = __ldg(src + ch);
#pragma unroll
                    for (int ch = 0; ch < DH / 8; ++ch)
                        *reinterpret_cast<uint4*>(q_smem + (ch >> 3) * Cfg::kSlabBytes + t * 128 + (((ch & 7) ^ (t & 7)) << 4)) = v[ch];
                }
                m_used = -INFINITY;
                l_run = 0.f;
                fence_proxy_async();
                tc_fence_before();
                mbar_arrive(&bars->q_full);
            }
            const bool seg_last = (cur.blk == cur.nb - 1) || (q + 1 == n_my);
            const int st = q % Cfg::kStages, buf = q & 1, u = q >> 1;
            const int t_begin = cur.blk * kAttBlockTokens;
            const bool real = r < rows_here;
            const bool warp_real = (quarter * 32) % span < rows_here;    // warp-uniform: a real row among this warp's lanes
            const bool o_owner = (quarter * 32 < span) && warp_real;      // warp-uniform: this warp's lanes hold real rows of O
            const uint32_t t_s = t_lane + (buf ? kTmemS1 : kTmemS0) + static_cast<uint32_t>(c * span);
            const int lim_local = (real ? limit : 0) - t_begin - c * span;   // my tokens [0, lim_local) are visible
            const bool need_mask = (t_begin + kAttBlockTokens > ctx + 1);

            if (!mbar_wait(&bars->s_full[buf], u & 1, p.status, 6)) { ok = false; break; }
            tc_fence_after();

            // ---- pass 1: maximum over my tokens of the block, then over the copies of the row
            float mx = -INFINITY;
            if (warp_real) {
                float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
                for (int c0 = 0; c0 < span; c0 += 32) {
                    uint32_t sv[32];
                    tmem_ld_x32(t_s + c0, sv);
                    tmem_ld_wait();
#pragma unroll
                    for (int i = 0; i < 32; ++i) {
                        float v = __uint_as_float(sv[i]);
                        if (need_mask && c0 + i >= lim_local) v = -INFINITY;
                        mx4[i & 3] = fmaxf(mx4[i & 3], v);
                    }
                }
                mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3])) * p.scale_log2;   // scale > 0: the maximum commutes
                if (!real) mx = -INFINITY;                                 // padding rows stay inert
            }
            if (copies > 1) {
                float* xch = s_xch[q & 1];
                xch[t] = mx;
                if (!group_sync(13)) { ok = false; break; }
                mx = xch[r];
                for (int cc = 1; cc < copies; ++cc) mx = fmaxf(mx, xch[cc * span + r]);
            }
            // ---- raise the running maximum only if it grew by more than the threshold
            float alpha = 1.f;
            if (seg_first) {
                m_used = mx;
            } else if (mx > m_used + kRescaleThreshold) {
                alpha = fast_exp2(m_used - mx);                            // m_used == -inf gives 0
                m_used = mx;
                l_run *= alpha;
            }
            if (o_owner && !seg_first && __any_sync(0xffffffffu, alpha != 1.f)) {
                // O += P V of the previous block must have landed before O is rescaled
                if (!mbar_wait(&bars->o_full, (q - 1) & 1, p.status, 7)) { ok = false; break; }
                tc_fence_after();
#pragma unroll
                for (int c0 = 0; c0 < DH; c0 += 32) {
                    uint32_t o[32];
                    tmem_ld_x32(t_lane + kTmemO + c0, o);
                    tmem_ld_wait();
#pragma unroll
                    for (int i = 0; i < 32; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * alpha);
                    tmem_st_x32(t_lane + kTmemO + c0, o);
                }
                tmem_st_wait();
            }
            // the P buffer is free once the P V product of two blocks ago has read it
            if (u > 0 && !mbar_wait(&bars->p_empty[buf], (u - 1) & 1, p.status, 8)) { ok = false; break; }
            if (warp_real) {
                // ---- pass 2: p = 2^(s * scale - m), bf16, into row r of operand A of the P V product
                const float m_safe = (m_used == -INFINITY) ? 0.f : m_used;
                uint8_t* p_row = smem + Cfg::kPOffset + buf * Cfg::kPBytes + r * 128;
                float rs0 = 0.f, rs1 = 0.f;
                for (int c0 = 0; c0 < span; c0 += 32) {
                    uint32_t sv[32];
                    tmem_ld_x32(t_s + c0, sv);
                    tmem_ld_wait();
                    uint32_t pk[16];
#pragma unroll
                    for (int i = 0; i < 32; i += 2) {
                        float e0 = fast_exp2(fmaf(__uint_as_float(sv[i]), p.scale_log2, -m_safe));
                        float e1 = fast_exp2(fmaf(__uint_as_float(sv[i + 1]), p.scale_log2, -m_safe));
                        if (need_mask) {
                            if (c0 + i >= lim_local) e0 = 0.f;
                            if (c0 + i + 1 >= lim_local) e1 = 0.f;
                        }
                        rs0 += e0;
                        rs1 += e1;
                        pk[i >> 1] = pack_bf16(e0, e1);
                    }
                    if (real) {
#pragma unroll
                        for (int ch = 0; ch < 4; ++ch) {
                            const int chunk = ((c * span + c0) >> 3) + ch;  // 16-byte chunk (8 tokens) of the row
                            *reinterpret_cast<uint4*>(p_row + (chunk >> 3) * Cfg::kSlabBytes + (((chunk & 7) ^ (r & 7)) << 4)) =
                                make_uint4(pk[4 * ch], pk[4 * ch + 1], pk[4 * ch + 2], pk[4 * ch + 3]);
                        }
                    }
                }
                l_run += rs0 + rs1;
            }
            // rows of V past the end of the sequence may hold anything (the pool is the caller's, or
            // the page was never loaded): their weight is exactly 0, but 0 * NaN is NaN, so clear them
            if (t_begin + kAttBlockTokens > cur.kvl && t >= cur.kvl - t_begin) {
                uint8_t* v_row = smem + st * Cfg::kStageBytes + Cfg::kSlabs * Cfg::kSlabBytes + t * 128;
#pragma unroll
                for (int hf = 0; hf < Cfg::kSlabs; ++hf)
#pragma unroll
                    for (int ch = 0; ch < 8; ++ch)
                        *reinterpret_cast<uint4*>(v_row + hf * Cfg::kSlabBytes + ch * 16) = make_uint4(0u, 0u, 0u, 0u);
            }
            fence_proxy_async();
            tc_fence_before();
            mbar_arrive(&bars->p_full[buf]);
            mbar_arrive(&bars->s_empty[buf]);

            const int pair_global = cur.pair0 + cur.pair;
            const int64_t pair_blk_first = static_cast<int64_t>(cur.blk0) + static_cast<int64_t>(cur.pair) * cur.nb;
            const int pair_nb = cur.nb, pair_q_row0 = cur.q_row0;
            cur.advance(p, q + 1 < n_my);
            seg_first = seg_last;
            if (!seg_last) continue;

            // ------------------------------------------------------------ end of the segment
            ++seg;
            if (copies > 1) {
                // the copies of a row hold the sums over their own tokens (same maximum): add them up
                float* xch = s_xch[2];
                xch[t] = l_run;
                if (!group_sync(14)) { ok = false; break; }
                l_run = xch[r];
                for (int cc = 1; cc < copies; ++cc) l_run += xch[cc * span + r];
            }
            if (!mbar_wait(&bars->o_full, q & 1, p.status, 10)) { ok = false; break; }
            tc_fence_after();
            // which CTAs hold blocks of this pair: CTA c owns blocks [c*T/G, (c+1)*T/G), so the owner of
            // block x is ceil((x+1)*G/T) - 1
            const int64_t pair_blk_last = pair_blk_first + pair_nb - 1;
            const int c_first = static_cast<int>(((pair_blk_first + 1) * gridDim.x - 1) / total_blocks);
            const int c_last = static_cast<int>(((pair_blk_last + 1) * gridDim.x - 1) / total_blocks);
            const int rho = row_lo + r;
            const int64_t out_row = static_cast<int64_t>(pair_q_row0 + rho / p.group) * p.n_q_heads + kvh * p.group + rho % p.group;
            __nv_bfloat16* out = p.attn_out + out_row * DH;
            const bool writer = o_owner && real;                           // c == 0 and a real row

            if (c_first == c_last) {
                // the whole pair was ours: normalise and store
                if (o_owner) {
                    const float inv = 1.f / l_run;
#pragma unroll
                    for (int cc = 0; cc < DH; cc += 32) {
                        uint32_t o[32];
                        tmem_ld_x32(t_lane + kTmemO + cc, o);
                        tmem_ld_wait();
                        if (writer) {
#pragma unroll
                            for (int i = 0; i < 32; i += 8) {
                                uint4 w;
                                w.x = pack_bf16(__uint_as_float(o[i]) * inv, __uint_as_float(o[i + 1]) * inv);
                                w.y = pack_bf16(__uint_as_float(o[i + 2]) * inv, __uint_as_float(o[i + 3]) * inv);
                                w.z = pack_bf16(__uint_as_float(o[i + 4]) * inv, __uint_as_float(o[i + 5]) * inv);
                                w.w = pack_bf16(__uint_as_float(o[i + 6]) * inv, __uint_as_float(o[i + 7]) * inv);
                                *reinterpret_cast<uint4*>(out + cc + i) = w;
                            }
                        }
                    }
                }
                tc_fence_before();
                continue;
            }

            // ---- the pair spans CTAs c_first..c_last: park (m, l, O); a CTA's parts are its first and its last segment
            const int my_slot = cta * 2 + ((seg == 1) ? 0 : 1);
            if (o_owner) {
                float* po = p.part_o + (static_cast<int64_t>(my_slot) * kAttRowsPerPair + r) * DH;
#pragma unroll
                for (int cc = 0; cc < DH; cc += 32) {
                    uint32_t o[32];
                    tmem_ld_x32(t_lane + kTmemO + cc, o);
                    tmem_ld_wait();
                    if (writer) {
#pragma unroll
                        for (int i = 0; i < 32; i += 4)
                            __stcg(reinterpret_cast<float4*>(po + cc + i),
                                   make_float4(__uint_as_float(o[i]), __uint_as_float(o[i + 1]),
                                               __uint_as_float(o[i + 2]), __uint_as_float(o[i + 3])));
                    }
                }
                if (writer)
                    __stcg(reinterpret_cast<float2*>(p.part_ml + (static_cast<int64_t>(my_slot) * kAttRowsPerPair + r) * 2),
                           make_float2(m_used, l_run));
            }
            tc_fence_before();
            __threadfence();
            if (!group_sync(11)) { ok = false; break; }                    // every softmax thread has published
            if (t == 0) {
                const int tk = atomicAdd(&p.tickets[pair_global], 1);
                const int last = (tk == c_last - c_first);
                if (last) p.tickets[pair_global] = 0;                      // ready for the next call
                s_flag = last;
            }
            if (!group_sync(12)) { ok = false; break; }
            if (s_flag && writer) {
                // ---- this CTA completed the pair: out = sum_c 2^(m_c - M) O_c / sum_c 2^(m_c - M) l_c,
                // parts taken in CTA order.  The first CTA holds the head of the pair in its last segment unless
                // its range starts exactly there; every later CTA holds its part in its first segment.
                __threadfence();
                const int blk_begin_c0 = static_cast<int>(static_cast<int64_t>(c_first) * total_blocks / gridDim.x);
                const int slot_c0 = c_first * 2 + ((blk_begin_c0 == pair_blk_first) ? 0 : 1);
                float m_all = -INFINITY;
                for (int cc = c_first; cc <= c_last; ++cc) {
                    const int slot = (cc == c_first) ? slot_c0 : cc * 2;
                    m_all = fmaxf(m_all, __ldcg(p.part_ml + (static_cast<int64_t>(slot) * kAttRowsPerPair + r) * 2));
                }
                float l_all = 0.f;
                for (int cc = c_first; cc <= c_last; ++cc) {
                    const int slot = (cc == c_first) ? slot_c0 : cc * 2;
                    const float2 ml = __ldcg(reinterpret_cast<const float2*>(p.part_ml + (static_cast<int64_t>(slot) * kAttRowsPerPair + r) * 2));
                    if (ml.x != -INFINITY) l_all += fast_exp2(ml.x - m_all) * ml.y;
                }
                const float inv = 1.f / l_all;
#pragma unroll 1
                for (int col = 0; col < DH; col += 32) {
                    float acc[32];
#pragma unroll
                    for (int i = 0; i < 32; ++i) acc[i] = 0.f;
                    for (int cc = c_first; cc <= c_last; ++cc) {
                        const int slot = (cc == c_first) ? slot_c0 : cc * 2;
                        const float mc = __ldcg(p.part_ml + (static_cast<int64_t>(slot) * kAttRowsPerPair + r) * 2);
                        if (mc == -INFINITY) continue;                     // that part saw no visible token
                        const float wgt = fast_exp2(mc - m_all);
                        const float4* po = reinterpret_cast<const float4*>(
                            p.part_o + (static_cast<int64_t>(slot) * kAttRowsPerPair + r) * DH + col);
#pragma unroll
                        for (int i = 0; i < 8; ++i) {
                            const float4 v = __ldcg(po + i);
                            acc[4 * i] += wgt * v.x; acc[4 * i + 1] += wgt * v.y;
                            acc[4 * i + 2] += wgt * v.z; acc[4 * i + 3] += wgt * v.w;
                        }
                    }
#pragma unroll
                    for (int i = 0; i < 32; i += 8) {
                        uint4 w;
                        w.x = pack_bf16(acc[i] * inv, acc[i + 1] * inv);
                        w.y = pack_bf16(acc[i + 2] * inv, acc[i + 3] * inv);
                        w.z = pack_bf16(acc[i + 4] * inv, acc[i + 5] * inv);
                        w.w = pack_bf16(acc[i + 6] * inv, acc[i + 7] * inv);
                        *reinterpret_cast<uint4*>(out + col + i) = w;
                    }
                }
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, kAttTmemCols);
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

cudaError_t launch_attention(const Handle& h, const CUtensorMap& kv_map, const AttnParams& p, int32_t n_ctas,
                             cudaStream_t stream)
{
    dim3 grid(n_ctas);
    dim3 block(kAttThreads);
    if (h.cfg.head_dim == 128)
        attention_kernel<128><<<grid, block, AttCfg<128>::kSmemBytes, stream>>>(kv_map, p);
    else
        attention_kernel<64><<<grid, block, AttCfg<64>::kSmemBytes, stream>>>(kv_map, p);
    return cudaGetLastError();
}

}  // namespace fs
