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
// "segments" (runs of blocks of one pair).  The host, which has a copy of the lengths, cuts the list
// -- equal ranges, or whole pairs per CTA when that balances well enough to save every split --
// and passes each CTA's starting point as a kernel parameter, so a CTA requests its first K/V tile
// without reading or scanning anything first.
//
// Both contractions run on the 5th-generation tensor cores with accumulators in tensor memory
// (the legacy warp-level MMA path cannot keep up with the KV stream).  A verification step has
// few query rows per kv head (8..72 in the paper-shaped workloads), so the operands are swapped:
// the 128 tokens of a block are the MMA's M dimension and the query rows its N dimension
// (n_pad = rows rounded up to 16), which makes tensor work, the Q tile and the P tile scale with
// the real row count:
//   S^T[128 tokens][n_pad] = K Q^T      A = K tile, B = Q tile, both K-major, 128-byte swizzle
//   O^T[Dh][n_pad]        += V^T P^T    A = V tile as TMA delivers it ([token][Dh]: MN-major),
//                                       B = P^T written by the softmax threads ([token][row]:
//                                       MN-major, unswizzled 8x8 core matrices)
//
// Warp roles (8 warps).  Warps 0-1: TMA producers, each owning half of every block's pages (a TMA request
// costs about 55 cycles of the issuing warp, and a block needs 32 of them); separate rings of
// 128-token K and V tiles; the page ids of the next block are looked up one block ahead.
// Warp 2: one thread issues the QK^T products; the warp owns the TMEM allocation.  Warp 7: one thread
// issues the PV products (one thread issuing both bounded the kernel).  Warps 3-6: softmax,
// thread t = token t of the block (TMEM lane t of S^T).  The maximum of a query row over the
// block is a column maximum: redux.sync.max over each warp, then over the four warps through
// shared memory.  The running maximum is only raised when it grew by more than 2^8 (O^T in TMEM
// is then rescaled); the final division by the row sum makes the stale maximum cancel.  Row sums
// are kept per thread and added up across lanes once per segment.  At the end of a segment
// thread t owns row Dh-index t of O^T; if the pair spans several CTAs every warp parks its 32
// rows of (m, l, O^T) in global scratch and the warp that arrives last for those rows (atomic
// ticket, nobody waits) merges the parts by log-sum-exp in CTA order.  Every mbarrier wait is
// bounded.
#include "common.cuh"
#include "internal.h"

namespace fs {

constexpr int kPageTokens = 16;
constexpr int kAttPagesPerStage = kAttBlockTokens / kPageTokens;    // 8
// warp order: 2 TMA producers, the S^T issuer, 4, 8 or 12 softmax warps (HALVES = 1, 2 or 3), the PV issuer;
// named barrier 1 joins everyone who touches tensor memory: 64 + 128 * HALVES threads
constexpr int kAttTmemCols = 512;
constexpr uint32_t kTmemS0 = 0, kTmemS1 = 128, kTmemO = 256;        // column offsets
constexpr float kRescaleThreshold = 8.f;                             // log2 units
constexpr int kAttSmemLimit = 232448;                                // 227 KB opt-in maximum per CTA
constexpr int kAttStaticReserve = 1024;                              // __shared__ variables of the kernel

struct AttBars {
    uint64_t k_full[kAttMaxStages], k_empty[kAttMaxStages];
    uint64_t v_full[kAttMaxStages], v_empty[kAttMaxStages];
    uint64_t s_full[2], s_empty[2];
    uint64_t p_full[2], p_empty[2];
    uint64_t q_full, o_full[2], group[3];       // o_full alternates with the block parity (see the PV issuer)
    uint32_t tmem_slot;
};
static_assert(sizeof(AttBars) <= 512, "barrier block");

// Dynamic shared memory, all offsets from a 1024-byte aligned base:
//   [k_stages x K slabs] [v_stages x V slabs] [Q: slabs x n_pad x 128 B] [P^T: p_bufs x n_pad x 256 B]
//   [barriers] [exchange of column maxima / row sums between the warps: 3 x 4 x n_pad floats]
//   [running maxima: n_pad floats] [overflow flags]
// K and V travel in separate rings: a K tile is free again after the QK^T product, a V tile only
// after the softmax and the second product, so V gets the deeper ring.
template <int DH>
struct AttCfg {
    static constexpr int kSlabs = DH / 64;                     // 128-byte column slabs per row
    static constexpr int kSlabBytes = 128 * 128;               // 128 tokens x 64 bf16
    static constexpr int kTileBytes = kSlabs * kSlabBytes;     // K (or V) of one 128-token block
    __host__ __device__ static constexpr int q_bytes(int n_pad) { return kSlabs * n_pad * 128; }
    __host__ __device__ static constexpr int p_bytes(int n_pad) { return n_pad * 256; }
    __host__ __device__ static constexpr int col_bytes(int n_pad) { return (3 * 4 + 1) * n_pad * 4 + 128; }
    __host__ __device__ static constexpr int fixed_bytes(int n_pad, int p_bufs)
    {
        return q_bytes(n_pad) + p_bufs * p_bytes(n_pad) + 512 + col_bytes(n_pad) + 1024;
    }
};

// the widest tile leaves room for enough K/V tiles only with a single P^T buffer
int attention_p_bufs(int n_pad) { return n_pad > 112 ? 1 : 2; }

// ring depths that fit: K gets two tiles of four or five, three of six or more; V gets the rest
void attention_stages(int head_dim, int n_pad, int* k_stages, int* v_stages)
{
    const int pb = attention_p_bufs(n_pad);
    const int tile = head_dim == 128 ? AttCfg<128>::kTileBytes : AttCfg<64>::kTileBytes;
    const int fixed = head_dim == 128 ? AttCfg<128>::fixed_bytes(n_pad, pb) : AttCfg<64>::fixed_bytes(n_pad, pb);
    const int tiles = (kAttSmemLimit - kAttStaticReserve - fixed) / tile;
    int ks = tiles >= 4 ? 2 : 1;
    if (tiles >= 6) ks = 3;                       // measured: 3 + 3 beats 2 + 4 by ~0.5 us at the 8B shape
    int vs = tiles - ks;
    if (vs > kAttMaxStages) vs = kAttMaxStages;
    *k_stages = ks;
    *v_stages = vs;
}

// The attention kernel waits in dozens of places and its code has to stay small enough for the
// instruction caches (its cold paths run once per CTA): one shared copy of the wait loop.
static __device__ __noinline__ bool att_wait_slow(uint64_t* bar, uint32_t parity, int32_t* status, int32_t where)
{
    return mbar_wait(bar, parity, status, where);
}
// a barrier that has already completed costs one non-blocking test
__device__ __forceinline__ bool att_wait(uint64_t* bar, uint32_t parity, int32_t* status, int32_t where)
{
    if (mbar_test_wait(bar, parity)) return true;
    return att_wait_slow(bar, parity, status, where);
}
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
// swizzle: rows of 64 MN-elements (128 B) indexed by k, groups of 8 k-rows `k_stride` bytes apart,
// the next 64 MN-elements `mn_stride` bytes away.
__device__ __forceinline__ uint64_t umma_desc_mn_sw128(uint32_t smem_addr, uint32_t mn_stride, uint32_t k_stride)
{
    uint64_t d = 0;
    d |= static_cast<uint64_t>((smem_addr & 0x3FFFFu) >> 4);
    d |= static_cast<uint64_t>((mn_stride >> 4) & 0x3FFFu) << 16;   // leading byte offset
    d |= static_cast<uint64_t>((k_stride >> 4) & 0x3FFFu) << 32;    // stride byte offset
    d |= static_cast<uint64_t>(1) << 46;                             // descriptor version of this architecture
    d |= static_cast<uint64_t>(2) << 61;                             // 128-byte swizzle
    return d;
}
// MN-major bf16 operand without swizzle: 8 (k) x 8 (mn) core matrices of 128 contiguous bytes
// (a k-row is 16 B), the next 8 k-rows `k_stride` bytes away, the next 8 MN-elements `mn_stride`.
__device__ __forceinline__ uint64_t umma_desc_mn_plain(uint32_t smem_addr, uint32_t mn_stride, uint32_t k_stride)
{
    uint64_t d = 0;
    d |= static_cast<uint64_t>((smem_addr & 0x3FFFFu) >> 4);
    d |= static_cast<uint64_t>((k_stride >> 4) & 0x3FFFu) << 16;    // leading byte offset
    d |= static_cast<uint64_t>((mn_stride >> 4) & 0x3FFFu) << 32;   // stride byte offset
    d |= static_cast<uint64_t>(1) << 46;
    return d;
}
constexpr uint32_t kIdescAMajorMN = 1u << 15;
constexpr uint32_t kIdescBMajorMN = 1u << 16;

// Position in the batch-wide block list; every role walks it in lock step.
struct AttCursor {
    int b, pair, blk;             // sequence, pair inside it, block inside the pair
    int k, kvl, nb, rbc, pairs;   // of sequence b: draft length, kv length, blocks per pair,
                                  // row blocks per kv head, pairs
    int q_row0, pair0, blk0;      // first query row / first pair / first block of sequence b
    // the device copies of the lengths are clamped to what the host sized the call for, so that a
    // device array that disagrees with its host copy cannot send an index outside its buffer
    __device__ __forceinline__ void load_seq(const AttnParams& p)
    {
        set_seq(p, p.draft_len[b], p.kv_len[b]);
    }
    __device__ __forceinline__ void set_seq(const AttnParams& p, int k_in, int kvl_in)
    {
        k = min(max(k_in, 0), p.k_cap);
        kvl = min(max(kvl_in, k + 1), p.kv_cap);
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

// Sums 32 per-lane values across the warp so that lane i ends up with the total of v[i]:
// 31 shuffles (halving exchange) instead of 32 full reductions.  v is destroyed.
__device__ __forceinline__ float warp_transpose_sum(float (&v)[32], int lane)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const bool up = (lane & o) != 0;
#pragma unroll
        for (int i = 0; i < o; ++i) {
            const float give = up ? v[i] : v[i + o];
            const float keep = up ? v[i + o] : v[i];
            v[i] = keep + __shfl_xor_sync(0xffffffffu, give, o);
        }
    }
    return v[0];
}

struct AttSmem {                  // pointers into dynamic shared memory
    uint8_t* k_ring;
    uint8_t* v_ring;
    uint8_t* q;
    uint8_t* pt;                  // P^T buffers
    AttBars* bars;
    float* xch;                   // [3][4][n_pad]: column maxima (by block parity) and row sums, one row per warp
    float* m_col;                 // [n_pad] running maximum of every column (query row), log2 units
    int* flags;                   // [parts][2][4] "a score exceeded its maximum by more than the threshold", by block parity and warp
};

// CTA that holds block x of the batch-wide list: the last one whose range starts at or before x.
static __device__ __noinline__ int att_owner(const AttTable& tab, int n_ctas, int x)
{
    int lo = 0, hi = n_ctas - 1;
    while (lo < hi) {
        const int mid = (lo + hi + 1) >> 1;
        if (tab.cta[mid].blk_begin <= x) lo = mid; else hi = mid - 1;
    }
    return lo;
}

// ------------------------------------------------------------------------------------ softmax role
// NCH = chunks of 32 columns (query rows) of S^T: n_pad <= 32 * NCH.  Per-column state (running
// maximum, row sum, output row) lives in lane i of every warp for column 32*ci + i and is
// broadcast by shuffles, so the four warps only meet once per block (column maxima) and once
// per segment (row sums).
template <int DH, int NCHT, int HALVES>
__device__ __forceinline__ void att_softmax(const AttnParams& p, const AttTable& tab, const AttSmem& sm, AttCursor cur, int n_my)
{
    using Cfg = AttCfg<DH>;
    constexpr int NCH = (NCHT + HALVES - 1) / HALVES;   // chunks of 32 columns this thread may own
    constexpr int kSoftmaxThreads = 128 * HALVES;
    AttBars* bars = sm.bars;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int quarter = warp & 3;                       // TMEM lanes 32*quarter .. +31
    // HALVES == 2 or 3: that many warps share every quarter (the same 32 tokens) and split the columns (query
    // rows) chunk-wise: the warp of part h owns chunks h, h + HALVES.  Column state, exchanges and barriers of the two halves
    // are separate; they only meet in the hand-overs to the MMA warps.
    const int half = HALVES > 1 ? ((warp - (kAttProducerWarps + 1)) >> 2) : 0;
    const int t = quarter * 32 + lane;                  // token of the block (S^T), Dh index (O^T)
    const int cta = blockIdx.x;
    const int n_pad = p.n_pad;
    uint32_t t_lane = 0;                                // set once the TMEM allocation is known (after the first Q tile is staged)
    const int q_slab = n_pad * 128;
    const bool o_lane = quarter * 32 < DH;              // warp-uniform: this warp's lanes hold rows of O^T

    if (n_my <= 0) {                                    // not produced by the host planner; keep the rendezvous whole
        asm volatile("bar.sync 1, %0;" ::"n"(64 + 128 * HALVES) : "memory");
        return;
    }
    bool ok = true, seg_first = true;
    int seg = 0;
    uint32_t group_phase = 0;
    // the four softmax warps meet on an mbarrier, one arrival per warp (128 arrivals on one shared-memory
    // word serialise: measured ~0.2 us per barrier and block)
    auto group_sync = [&](int where) -> bool {
        __syncwarp();
        if (lane == 0) mbar_arrive(&bars->group[half]);
        const bool done = att_wait(&bars->group[half], group_phase, p.status, where);
        group_phase ^= 1u;
        return done;
    };

    float lsum[NCH * 32];                               // my token's share of the row sums, per column
    float m_used[NCH];                                  // lane i: running maximum of column 32*ci + i (log2 units)
    int row_c[NCH];                                     // lane i: output row index (row * n_q_heads + head) of that column
    int rows_here = 0, row_lo = 0, ctx = 0;

    for (int q = 0; q < n_my && ok; ++q) {
        if (seg_first) {
            const int kvh = cur.pair / cur.rbc;
            // ---- the pair's query rows -> shared memory, K-major swizzled rows of operand B
            row_lo = (cur.pair % cur.rbc) * kAttRowsPerPair;
            rows_here = min(kAttRowsPerPair, p.group * (cur.k + 1) - row_lo);
            ctx = cur.kvl - (cur.k + 1);
            for (int idx = half * 128 + t; idx < rows_here * (DH / 8); idx += kSoftmaxThreads) {
                const int row = idx / (DH / 8), ch = idx % (DH / 8);
                const int rho = row_lo + row;
                const int tok_row = min(cur.q_row0 + rho / p.group, p.m_rows - 1);
                const int64_t src_row = static_cast<int64_t>(tok_row) * p.n_q_heads + kvh * p.group + rho % p.group;
                const uint4 v = __ldg(reinterpret_cast<const uint4*>(p.hidden + src_row * DH) + ch);
                *reinterpret_cast<uint4*>(sm.q + (ch >> 3) * q_slab + row * 128 + (((ch & 7) ^ (row & 7)) << 4)) = v;
            }
#pragma unroll
            for (int i = 0; i < NCH * 32; ++i) lsum[i] = 0.f;
#pragma unroll
            for (int cs = 0; cs < NCH; ++cs) { const int ci = half + cs * HALVES;
                m_used[cs] = -INFINITY;
                const int rho = row_lo + ci * 32 + lane;
                row_c[cs] = min(cur.q_row0 + rho / p.group, p.m_rows - 1) * p.n_q_heads + kvh * p.group + rho % p.group;
            }
            fence_proxy_async();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&bars->q_full);
            if (q == 0) {
                // the MMA warp allocated tensor memory meanwhile: meet it (warps 2..6) and read the base
                asm volatile("bar.sync 1, %0;" ::"n"(64 + 128 * HALVES) : "memory");
                tc_fence_after();
                t_lane = bars->tmem_slot + (static_cast<uint32_t>(quarter * 32) << 16);
            }
        }
        const bool seg_last = (cur.blk == cur.nb - 1) || (q + 1 == n_my);
        const int buf = q & 1, u = q >> 1;
        const int t_begin = cur.blk * kAttBlockTokens;
        // token t of the block sees query row (column) c iff col_min <= c < rows_here: it is at
        // distance d = t_abs - ctx into the draft window and row c belongs to window position c / group
        const int d = t_begin + t - ctx;
        const int col_min = d > 0 ? d * p.group - row_lo : 0;
        const uint32_t col_span = static_cast<uint32_t>(max(0, rows_here - col_min));
        const uint32_t t_s = t_lane + (buf ? kTmemS1 : kTmemS0);

        if (!att_wait(&bars->s_full[buf], u & 1, p.status, 6)) { ok = false; break; }
        tc_fence_after();

        // the P^T buffer is free once the product that last read it has completed
        const int pbuf = q % p.p_bufs, pu = q / p.p_bufs;
        if (pu > 0 && !att_wait(&bars->p_empty[pbuf], (pu - 1) & 1, p.status, 8)) { ok = false; break; }

        // ---- One pass per block in the common case: p = 2^(s * scale - m) against the running maxima kept
        // in shared memory, written as bf16 into row t of operand B of the second product, while noting
        // whether any score exceeded its row's maximum by more than the threshold.  The four warps then
        // agree; only if one of them saw such a score (or at the start of a segment, where there is no
        // maximum yet) are the exact column maxima taken, O^T and the row sums rescaled -- this block's
        // contribution to the row sums included -- and the block's P^T written again against the new maxima.
        bool fresh = seg_first;                          // the maxima are (re)computed before the pass
        bool add = true;                                 // the pass adds to the row sums
#pragma unroll 1
        for (int pass = 0; pass < 2 && ok; ++pass) {
            if (fresh) {
                // ---- exact column maxima over my warp's 32 tokens, then over the four warps
                float* xch = sm.xch + (q & 1) * 4 * n_pad;
#pragma unroll
                for (int cs = 0; cs < NCH; ++cs) { const int ci = half + cs * HALVES;
                    if (ci * 32 < n_pad) {
                        uint32_t sv[32];
                        tmem_ld_x32(t_s + ci * 32, sv);
                        tmem_ld_wait();
                        float mine = -INFINITY;
#pragma unroll
                        for (int i = 0; i < 32; ++i) {
                            const bool masked = static_cast<uint32_t>(ci * 32 + i - col_min) >= col_span;
                            const float w = redux_max(masked ? -INFINITY : __uint_as_float(sv[i]));
                            if (lane == i) mine = w;
                        }
                        if (ci * 32 + lane < n_pad) xch[quarter * n_pad + ci * 32 + lane] = mine;
                    }
                }
                if (!group_sync(17)) { ok = false; break; }
                float alpha[NCH];
                bool rescale = false;
#pragma unroll
                for (int cs = 0; cs < NCH; ++cs) { const int ci = half + cs * HALVES;
                    alpha[cs] = 1.f;
                    const int col = ci * 32 + lane;
                    if (col < n_pad) {
                        const float mx = fmaxf(fmaxf(xch[col], xch[n_pad + col]), fmaxf(xch[2 * n_pad + col], xch[3 * n_pad + col])) *
                                         p.scale_log2;       // scale > 0: the maximum commutes
                        // ---- raise the running maximum only if it grew by more than the threshold
                        if (seg_first) {
                            m_used[cs] = mx;
                        } else if (mx > m_used[cs] + kRescaleThreshold) {
                            alpha[cs] = fast_exp2(m_used[cs] - mx);            // m_used == -inf gives 0
                            m_used[cs] = mx;
                            rescale = true;
                        }
                        if (quarter == 0) sm.m_col[col] = m_used[cs];
                    }
                }
                if (!seg_first && __any_sync(0xffffffffu, rescale)) {
                    // O^T += V^T P^T of the previous block must have landed before O^T is rescaled
                    if (!att_wait(&bars->o_full[(q - 1) & 1], ((q - 1) >> 1) & 1, p.status, 7)) { ok = false; break; }
                    tc_fence_after();
#pragma unroll
                    for (int cs = 0; cs < NCH; ++cs) { const int ci = half + cs * HALVES;
                        if (ci * 32 < n_pad) {
                            uint32_t o[32];
                            if (o_lane) {
                                tmem_ld_x32(t_lane + kTmemO + ci * 32, o);
                                tmem_ld_wait();
                            }
#pragma unroll
                            for (int i = 0; i < 32; ++i) {
                                const float a = __shfl_sync(0xffffffffu, alpha[cs], i);
                                lsum[cs * 32 + i] *= a;
                                if (o_lane) o[i] = __float_as_uint(__uint_as_float(o[i]) * a);
                            }
                            if (o_lane) tmem_st_x32(t_lane + kTmemO + ci * 32, o);
                        }
                    }
                    if (o_lane) tmem_st_wait();
                }
                if (!group_sync(18)) { ok = false; break; }                // the new maxima are in shared memory
            }
            // ---- p = 2^(s * scale - m)
            float ex = -INFINITY;
            {
                uint8_t* p_row = sm.pt + pbuf * Cfg::p_bytes(n_pad) + t * 16;
#pragma unroll
                for (int cs = 0; cs < NCH; ++cs) { const int ci = half + cs * HALVES;
                    if (ci * 32 < n_pad) {
                        uint32_t sv[32];
                        tmem_ld_x32(t_s + ci * 32, sv);
                        tmem_ld_wait();
                        uint32_t pk[16];
#pragma unroll
                        for (int i4 = 0; i4 < 8; ++i4) {
                            const float4 mv = *reinterpret_cast<const float4*>(sm.m_col + ci * 32 + 4 * i4);
                            const float mm[4] = {mv.x, mv.y, mv.z, mv.w};
                            float e[4];
#pragma unroll
                            for (int j = 0; j < 4; ++j) {
                                const int i = 4 * i4 + j;
                                const float x = fmaf(__uint_as_float(sv[i]), p.scale_log2, -mm[j]);
                                const bool masked = static_cast<uint32_t>(ci * 32 + i - col_min) >= col_span;   // also rows without a maximum yet
                                e[j] = masked ? 0.f : fast_exp2(x);
                                ex = fmaxf(ex, masked ? -INFINITY : x);
                                if (add) lsum[cs * 32 + i] += e[j];
                            }
                            pk[2 * i4] = pack_bf16(e[0], e[1]);
                            pk[2 * i4 + 1] = pack_bf16(e[2], e[3]);
                        }
#pragma unroll
                        for (int g8 = 0; g8 < 4; ++g8)
                            if (ci * 32 + g8 * 8 < n_pad)
                                *reinterpret_cast<uint4*>(p_row + (ci * 4 + g8) * 2048) =
                                    make_uint4(pk[4 * g8], pk[4 * g8 + 1], pk[4 * g8 + 2], pk[4 * g8 + 3]);
                    }
                }
            }
            if (fresh) break;                            // written against maxima taken from this very block
            const bool hot = __any_sync(0xffffffffu, ex > kRescaleThreshold);
            if (lane == 0) sm.flags[half * 8 + (q & 1) * 4 + quarter] = hot ? 1 : 0;
            if (!group_sync(14)) { ok = false; break; }
            const int* fl = sm.flags + half * 8 + (q & 1) * 4;
            if ((fl[0] | fl[1] | fl[2] | fl[3]) == 0) break;
            fresh = true;                                // second round: new maxima, then P^T again, the row sums
            add = false;                                 // already hold this block (they are rescaled with the rest)
        }
        if (!ok) break;
        // rows of V past the end of the sequence may hold anything (the pool is the caller's, or
        // the page was never loaded): their weight is exactly 0, but 0 * NaN is NaN, so clear them
        if (t_begin + kAttBlockTokens > cur.kvl) {
            // (the tile must have landed first, or the copy would overwrite the zeros)
            if (!att_wait(&bars->v_full[q % p.v_stages], (q / p.v_stages) & 1, p.status, 22)) { ok = false; break; }
        }
        if (half == 0 && t_begin + kAttBlockTokens > cur.kvl && t >= cur.kvl - t_begin) {
            uint8_t* v_row = sm.v_ring + (q % p.v_stages) * Cfg::kTileBytes + t * 128;
#pragma unroll
            for (int hf = 0; hf < Cfg::kSlabs; ++hf)
#pragma unroll
                for (int ch = 0; ch < 8; ++ch)
                    *reinterpret_cast<uint4*>(v_row + hf * Cfg::kSlabBytes + ch * 16) = make_uint4(0u, 0u, 0u, 0u);
        }
        fence_proxy_async();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) {
            mbar_arrive(&bars->p_full[pbuf]);
            mbar_arrive(&bars->s_empty[buf]);
        }

        const int pair_global = cur.pair0 + cur.pair;
        const int pair_blk_first = cur.blk0 + cur.pair * cur.nb;
        const int pair_nb = cur.nb;
        cur.advance(p, q + 1 < n_my);
        seg_first = seg_last;
        if (!seg_last) continue;

        // ---------------------------------------------------------------- end of the segment
        ++seg;
        // ---- row sums: add my warp's tokens, then the four warps; lane i ends up with column 32*ci + i
        float* xl = sm.xch + 2 * 4 * n_pad;
        float l_c[NCH];
#pragma unroll
        for (int cs = 0; cs < NCH; ++cs) { const int ci = half + cs * HALVES;
            l_c[cs] = 0.f;
            if (ci * 32 < n_pad) {
                float tmp[32];
#pragma unroll
                for (int i = 0; i < 32; ++i) tmp[i] = lsum[cs * 32 + i];
                const float mine = warp_transpose_sum(tmp, lane);
                if (ci * 32 + lane < n_pad) xl[quarter * n_pad + ci * 32 + lane] = mine;
            }
        }
        if (!group_sync(15)) { ok = false; break; }
#pragma unroll
        for (int cs = 0; cs < NCH; ++cs) { const int ci = half + cs * HALVES;
            const int col = ci * 32 + lane;
            if (col < n_pad) l_c[cs] = (xl[col] + xl[n_pad + col]) + (xl[2 * n_pad + col] + xl[3 * n_pad + col]);
        }
        if (!att_wait(&bars->o_full[q & 1], (q >> 1) & 1, p.status, 10)) { ok = false; break; }
        tc_fence_after();
        if (!o_lane) continue;                                         // nothing of O^T in this warp's lanes
        // does the pair reach into another CTA's range?  (this CTA holds blocks [blk_begin, blk_begin + n_my))
        const int pair_blk_last = pair_blk_first + pair_nb - 1;
        const bool whole = pair_blk_first >= tab.cta[cta].blk_begin && pair_blk_last < tab.cta[cta].blk_begin + n_my;

        if (whole) {
            // the whole pair was ours: normalise and store; thread t holds element t of every row
            __nv_bfloat16* out_t = p.attn_out + t;
#pragma unroll
            for (int cs = 0; cs < NCH; ++cs) { const int ci = half + cs * HALVES;
                if (ci * 32 < n_pad) {
                    uint32_t o[32];
                    tmem_ld_x32(t_lane + kTmemO + ci * 32, o);
                    tmem_ld_wait();
                    const float inv_l = 1.f / l_c[cs];
#pragma unroll
                    for (int i = 0; i < 32; ++i) {
                        const float il = __shfl_sync(0xffffffffu, inv_l, i);
                        const int row = __shfl_sync(0xffffffffu, row_c[cs], i);
                        if (ci * 32 + i < rows_here) out_t[static_cast<int64_t>(row) * DH] = __float2bfloat16_rn(__uint_as_float(o[i]) * il);
                    }
                }
            }
            tc_fence_before();
            continue;
        }

        const int c_first = att_owner(tab, gridDim.x, pair_blk_first);
        const int c_last = att_owner(tab, gridDim.x, pair_blk_last);
        // ---- the pair spans CTAs c_first..c_last: every warp parks its 32 rows of O^T with its own copy
        // of (m, l) and takes its own ticket; the warp that arrives last for (pair, warp) merges those
        // rows.  A CTA's parts are its first and its last segment.
        const int my_slot = cta * 2 + ((seg == 1) ? 0 : 1);
        {
            float* po = p.part_o + (static_cast<int64_t>(my_slot) * DH + t) * kAttRowsPerPair;
            float* pml = p.part_ml + (static_cast<int64_t>(my_slot) * 4 + quarter) * kAttRowsPerPair * 2;
#pragma unroll
            for (int cs = 0; cs < NCH; ++cs) { const int ci = half + cs * HALVES;
                if (ci * 32 < n_pad) {
                    uint32_t o[32];
                    tmem_ld_x32(t_lane + kTmemO + ci * 32, o);
                    tmem_ld_wait();
#pragma unroll
                    for (int i = 0; i < 32; i += 4)
                        if (ci * 32 + i < n_pad)
                            __stcg(reinterpret_cast<float4*>(po + ci * 32 + i),
                                   make_float4(__uint_as_float(o[i]), __uint_as_float(o[i + 1]),
                                               __uint_as_float(o[i + 2]), __uint_as_float(o[i + 3])));
                    if (ci * 32 + lane < n_pad)
                        __stcg(reinterpret_cast<float2*>(pml + (ci * 32 + lane) * 2), make_float2(m_used[cs], l_c[cs]));
                }
            }
        }
        tc_fence_before();
        __threadfence();
        __syncwarp();
        int last = 0;
        if (lane == 0) {
            int32_t* tk = p.tickets + (static_cast<int64_t>(pair_global) * 4 + quarter) * 3 + half;
            last = (atomicAdd(tk, 1) == c_last - c_first);
            if (last) *tk = 0;                                         // ready for the next call
        }
        last = __shfl_sync(0xffffffffu, last, 0);
        if (!last) continue;

        // ---- this warp completed its rows of the pair: out = sum_c 2^(m_c - M) O_c / sum_c 2^(m_c - M) l_c,
        // parts taken in CTA order.  The first CTA holds the head of the pair in its last segment unless its
        // range starts exactly there; every later CTA holds its part in its first segment.  (This path runs
        // once or twice per CTA and is always cold in the instruction cache: it is kept compact.)
        __threadfence();
        const int slot_c0 = c_first * 2 + ((tab.cta[c_first].blk_begin == pair_blk_first) ? 0 : 1);
        // one pass over the parts: the (m, l) of my column and my row of O^T are requested together, and
        // the accumulator is rescaled whenever a part raises a column's maximum
        float m_all[NCH], l_all[NCH];
#pragma unroll
        for (int cs = 0; cs < NCH; ++cs) { m_all[cs] = -INFINITY; l_all[cs] = 0.f; }
#pragma unroll
        for (int i = 0; i < NCH * 32; ++i) lsum[i] = 0.f;              // reused as the accumulator of my O^T row
#pragma unroll 1
        for (int cc = c_first; cc <= c_last; ++cc) {
            const int slot = (cc == c_first) ? slot_c0 : cc * 2;
            const float4* po = reinterpret_cast<const float4*>(p.part_o + (static_cast<int64_t>(slot) * DH + t) * kAttRowsPerPair);
            const float2* pml = reinterpret_cast<const float2*>(p.part_ml) + (static_cast<int64_t>(slot) * 4 + quarter) * kAttRowsPerPair;
#pragma unroll
            for (int cs = 0; cs < NCH; ++cs) { const int ci = half + cs * HALVES;
                if (ci * 32 < n_pad) {
                    float4 v[8];
#pragma unroll
                    for (int i = 0; i < 8; ++i) v[i] = __ldcg(po + ci * 8 + i);
                    float2 ml = make_float2(-INFINITY, 0.f);
                    if (ci * 32 + lane < n_pad) ml = __ldcg(pml + ci * 32 + lane);
                    // my column: weight of what is accumulated so far, weight of this part (a part that saw no
                    // visible token has m = -inf, weight 0 and O^T = 0)
                    const float mn = fmaxf(m_all[cs], ml.x);
                    const float base = (mn == -INFINITY) ? 0.f : mn;
                    const float w_old = fast_exp2(m_all[cs] - base);
                    const float w_new = fast_exp2(ml.x - base);
                    l_all[cs] = l_all[cs] * w_old + ml.y * w_new;
                    m_all[cs] = mn;
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        const float vv[4] = {v[i].x, v[i].y, v[i].z, v[i].w};
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            const float wo = __shfl_sync(0xffffffffu, w_old, 4 * i + j);
                            const float wn = __shfl_sync(0xffffffffu, w_new, 4 * i + j);
                            lsum[cs * 32 + 4 * i + j] = lsum[cs * 32 + 4 * i + j] * wo + wn * vv[j];
                        }
                    }
                }
            }
        }
        __nv_bfloat16* out_t = p.attn_out + t;
#pragma unroll
        for (int cs = 0; cs < NCH; ++cs) { const int ci = half + cs * HALVES;
            const float inv_l = 1.f / l_all[cs];
#pragma unroll
            for (int i = 0; i < 32; ++i) {
                const float il = __shfl_sync(0xffffffffu, inv_l, i);
                const int row = __shfl_sync(0xffffffffu, row_c[cs], i);
                if (ci * 32 + i < rows_here) out_t[static_cast<int64_t>(row) * DH] = __float2bfloat16_rn(lsum[cs * 32 + i] * il);
            }
        }
    }
}

template <int DH, int NCHT, int HALVES>
__global__ void __launch_bounds__((4 + 4 * HALVES) * 32, 1)
attention_kernel(const __grid_constant__ CUtensorMap kv_map, const __grid_constant__ AttnParams p,
                 const __grid_constant__ AttTable tab)
{
    using Cfg = AttCfg<DH>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const int n_pad = p.n_pad;
    AttSmem sm;
    sm.k_ring = smem;
    sm.v_ring = smem + p.k_stages * Cfg::kTileBytes;
    sm.q = sm.v_ring + p.v_stages * Cfg::kTileBytes;
    sm.pt = sm.q + Cfg::q_bytes(n_pad);
    sm.bars = reinterpret_cast<AttBars*>(sm.pt + p.p_bufs * Cfg::p_bytes(n_pad));
    sm.xch = reinterpret_cast<float*>(reinterpret_cast<uint8_t*>(sm.bars) + 512);
    sm.m_col = sm.xch + 12 * n_pad;
    sm.flags = reinterpret_cast<int*>(sm.m_col + n_pad);
    AttBars* bars = sm.bars;
    __shared__ int s_phys[kAttProducerWarps][8][2 * kAttPagesPerStage / kAttProducerWarps];   // per producer warp: page ids
                                                        // of the blocks between its prefetch cursor and its copies, by lane

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const int cta = blockIdx.x;

    if (threadIdx.x == 0) {
        for (int s = 0; s < p.k_stages; ++s) { mbar_init(&bars->k_full[s], 1); mbar_init(&bars->k_empty[s], 1); }
        for (int s = 0; s < p.v_stages; ++s) { mbar_init(&bars->v_full[s], 1); mbar_init(&bars->v_empty[s], 1); }
        for (int a = 0; a < 2; ++a) {
            mbar_init(&bars->s_full[a], 1); mbar_init(&bars->s_empty[a], 4 * HALVES);   // one arrival per softmax warp
            mbar_init(&bars->p_full[a], 4 * HALVES); mbar_init(&bars->p_empty[a], 1);
        }
        for (int a = 0; a < 3; ++a) mbar_init(&bars->group[a], 4);                      // the four warps of one column part
        mbar_init(&bars->q_full, 4 * HALVES);
        mbar_init(&bars->o_full[0], 1);
        mbar_init(&bars->o_full[1], 1);
        fence_barrier_init();
        tma_prefetch_desc(&kv_map);
    }
    __syncthreads();                                    // barriers are initialised: the producers may start

    // ---- where this CTA starts (host-computed)
    const int n_my = tab.cta[cta].n_my;
    AttCursor cur;
    cur.b = tab.cta[cta].b;
    cur.q_row0 = tab.cta[cta].q_row0; cur.pair0 = tab.cta[cta].pair0; cur.blk0 = tab.cta[cta].blk0;
    cur.set_seq(p, tab.cta[cta].k, tab.cta[cta].kvl);
    cur.pair = tab.cta[cta].blk_off / cur.nb;
    cur.blk = tab.cta[cta].blk_off % cur.nb;
    uint32_t tmem_base = 0;

    if (warp < kAttProducerWarps) {
        // ------------------------------------------------------------------ TMA producers
        // Producer warp w owns pages [w*PW, (w+1)*PW) of every block; lane l < 2*PW issues the K and the
        // V copy of (page l / 2, 64-column half l % 2).
        constexpr int PW = kAttPagesPerStage / kAttProducerWarps;          // pages per producer warp
        const uint64_t pol = l2_policy_evict_first();
        const int my_page = warp * PW + (lane >> 1);                       // page of the block this lane copies
        const int my_half = lane & 1;
        const bool copy_lane = lane < 2 * PW && my_half < Cfg::kSlabs;
        int (*ring)[2 * PW] = s_phys[warp];
        bool new_pair = true;
        bool ok = true;
        // A second cursor runs one block ahead of the copies and looks the page ids up (one page-table
        // read per block, kept in a small shared-memory ring until the copy needs them; the read for
        // the next block is in flight while this block is handled).  (Asking for the pages to be
        // brought into L2 further ahead was measured and did not pay: 4 blocks ahead cost 1.7 us per
        // step at the 8B shape, 8 blocks 3 us.)
        AttCursor pf = cur;
        int pf_q = 0;
        auto pf_load = [&](const AttCursor& c) -> int {
            const int pt_begin = c.blk * kAttBlockTokens;
            const int pnpg = (min(c.kvl, pt_begin + kAttBlockTokens) - pt_begin + kPageTokens - 1) / kPageTokens;
            return (lane < 2 * PW && my_page < pnpg)
                       ? p.page_table[static_cast<int64_t>(c.b) * p.max_pages_per_seq + c.blk * kAttPagesPerStage + my_page] : -1;
        };
        auto pf_issue = [&](int ph) {
            if (lane < 2 * PW) ring[pf_q & 7][lane] = ph;
            ++pf_q;
            pf.advance(p, pf_q < n_my);
        };
        int pf_ph = pf_load(pf);
        pf_issue(pf_ph);
        pf_ph = (pf_q < n_my) ? pf_load(pf) : -1;
        for (int q = 0; q < n_my && ok; ++q) {
            const int kvh = cur.pair / cur.rbc;
            if (new_pair && warp == 0) {
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
            const int ks = q % p.k_stages, k_use = q / p.k_stages;
            const int vs = q % p.v_stages, v_use = q / p.v_stages;
            const int t_begin = cur.blk * kAttBlockTokens;
            const int t_end = min(cur.kvl, t_begin + kAttBlockTokens);
            const int npg = (t_end - t_begin + kPageTokens - 1) / kPageTokens;
            const bool active = copy_lane && my_page < npg;
            int phys = (lane < 2 * PW) ? ring[q & 7][lane] : -1;
            if (active && (phys < 0 || phys >= p.num_pages)) {
                report_error(p.status, kErrBadPage, phys, 1);
                phys = 0;                                   // stay inside the pool
            }
            const uint32_t tile_tx = static_cast<uint32_t>(npg * Cfg::kSlabs * kPageTokens * 128);
            const int smem_off = my_half * Cfg::kSlabBytes + my_page * (kPageTokens * 128);
            // K tile
            if (k_use > 0 && !att_wait(&bars->k_empty[ks], (k_use - 1) & 1, p.status, 1)) { ok = false; break; }
            if (warp == 0 && lane == 0) mbar_arrive_expect_tx(&bars->k_full[ks], tile_tx);
            if (active)
                tma_load_2d(sm.k_ring + ks * Cfg::kTileBytes + smem_off, &kv_map, &bars->k_full[ks], my_half * 64,
                            ((phys * 2 + 0) * p.n_kv_heads + kvh) * kPageTokens, pol);
            // V tile
            if (v_use > 0 && !att_wait(&bars->v_empty[vs], (v_use - 1) & 1, p.status, 20)) { ok = false; break; }
            if (warp == 0 && lane == 0) mbar_arrive_expect_tx(&bars->v_full[vs], tile_tx);
            if (active)
                tma_load_2d(sm.v_ring + vs * Cfg::kTileBytes + smem_off, &kv_map, &bars->v_full[vs], my_half * 64,
                            ((phys * 2 + 1) * p.n_kv_heads + kvh) * kPageTokens, pol);
            __syncwarp();
#pragma unroll 1
            for (int step = 0; step < 2 && pf_q < n_my && pf_q <= q + 1; ++step) {
                pf_issue(pf_ph);
                pf_ph = (pf_q < n_my) ? pf_load(pf) : -1;
            }
            new_pair = cur.advance(p, q + 1 < n_my);
        }
        // do not leave while a copy of ours may still be landing in shared memory
        if (ok && n_my > 0) {
            const int ql = n_my - 1;
            att_wait(&bars->k_full[ql % p.k_stages], (ql / p.k_stages) & 1, p.status, 9);
            att_wait(&bars->v_full[ql % p.v_stages], (ql / p.v_stages) & 1, p.status, 9);
        }
    } else if (warp == kAttProducerWarps) {
        // ------------------------------------------------------------------ MMA issuer of S^T = K Q^T
        // The two products are issued by two threads in two warps: one thread issuing both, with its
        // barrier waits and commits, took 1.7 us per block and was what bounded the kernel.
        // This warp also owns the tensor memory: it allocates while the producers already request K/V
        // and the softmax warps stage the first Q tile, then meets the other consumers (named barrier 1).
        tmem_alloc(&bars->tmem_slot, kAttTmemCols);
        tmem_relinquish();
        tc_fence_before();
        asm volatile("bar.sync 1, %0;" ::"n"(64 + 128 * HALVES) : "memory");
        tc_fence_after();
        tmem_base = bars->tmem_slot;
        if (lane == 0 && n_my > 0) {
            // descriptors are built once and only advanced by adding (byte offset >> 4) to their address
            // field, ring positions are carried, not divided
            const uint32_t idesc_s = umma_idesc_bf16(128, static_cast<uint32_t>(n_pad));
            const uint64_t dq0 = umma_desc_k_sw128(smem_u32(sm.q));
            const uint64_t dk0 = umma_desc_k_sw128(smem_u32(sm.k_ring));
            const uint32_t q_slab16 = (static_cast<uint32_t>(n_pad) * 128u) >> 4;
            int ks = 0; uint32_t kpar = 0;                 // K ring slot / parity of its full barrier
            int buf = 0; uint32_t spar = 1;                // S^T buffer; parity to wait for on s_empty (previous use)
            int seg = 0;
            bool seg_first = true;
            for (int q = 0; q < n_my; ++q) {
                // waits: the pair's Q tile (new segment), the K tile, the S^T buffer (two blocks back)
                if (seg_first && !att_wait(&bars->q_full, seg & 1, p.status, 2)) break;
                if (!att_wait(&bars->k_full[ks], kpar, p.status, 3)) break;
                if (q >= 2 && !att_wait(&bars->s_empty[buf], spar, p.status, 4)) break;
                tc_fence_after();
                const uint64_t dk = dk0 + static_cast<uint32_t>((ks * Cfg::kTileBytes) >> 4);
                const uint32_t acc = tmem_base + (buf ? kTmemS1 : kTmemS0);
#pragma unroll
                for (int kk = 0; kk < DH / 16; ++kk)
                    umma_bf16(acc, dk + static_cast<uint32_t>(((kk >> 2) * Cfg::kSlabBytes + (kk & 3) * 32) >> 4),
                              dq0 + ((kk >> 2) * q_slab16 + (kk & 3) * 2), idesc_s, kk > 0 ? 1u : 0u);
                umma_commit(&bars->s_full[buf]);
                umma_commit(&bars->k_empty[ks]);
                if (++ks == p.k_stages) { ks = 0; kpar ^= 1u; }
                if (buf == 1) spar ^= 1u;                  // both buffers used once more: next round waits the other parity
                buf ^= 1;
                seg_first = (cur.blk == cur.nb - 1);       // the next block opens a segment
                if (seg_first) ++seg;
                cur.advance(p, q + 1 < n_my);
            }
        }
    } else if (warp == kAttProducerWarps + 1 + 4 * HALVES) {
        // ------------------------------------------------------------------ MMA issuer of O^T += V^T P^T
        asm volatile("bar.sync 1, %0;" ::"n"(64 + 128 * HALVES) : "memory");
        tc_fence_after();
        tmem_base = bars->tmem_slot;
        if (lane == 0 && n_my > 0) {
            const uint32_t idesc_o = umma_idesc_bf16(128, static_cast<uint32_t>(n_pad)) | kIdescAMajorMN | kIdescBMajorMN;
            const uint64_t dv0 = umma_desc_mn_sw128(smem_u32(sm.v_ring), Cfg::kSlabBytes, 1024);
            const uint64_t dp0 = umma_desc_mn_plain(smem_u32(sm.pt), 2048, 128);
            const uint32_t p_buf16 = static_cast<uint32_t>(Cfg::p_bytes(n_pad)) >> 4;
            int vs = 0; uint32_t vpar = 0;                 // V ring slot / parity
            int pb = 0; uint32_t ppar = 0;                 // P^T buffer / parity of p_full
            bool seg_first = true;
            for (int q = 0; q < n_my; ++q) {
                if (!att_wait(&bars->v_full[vs], vpar, p.status, 21)) break;
                if (!att_wait(&bars->p_full[pb], ppar, p.status, 5)) break;
                tc_fence_after();
                const uint64_t dv = dv0 + static_cast<uint32_t>((vs * Cfg::kTileBytes) >> 4);
                const uint64_t dp = dp0 + static_cast<uint32_t>(pb) * p_buf16;
#pragma unroll
                for (int ks = 0; ks < kAttBlockTokens / 16; ++ks)      // 16 tokens: two groups of 8 k-rows in both operands
                    umma_bf16(tmem_base + kTmemO, dv + static_cast<uint32_t>((ks * 2048) >> 4), dp + static_cast<uint32_t>((ks * 256) >> 4),
                              idesc_o, (seg_first && ks == 0) ? 0u : 1u);
                umma_commit(&bars->v_empty[vs]);
                umma_commit(&bars->p_empty[pb]);
                // "O^T holds block q": two barriers, alternating with q.  A softmax warp that waits for block q
                // only knows that the product of block q - 2 has completed (it waited for that P^T buffer); with
                // one barrier its parity could not tell block q - 1 still pending from block q done, with two
                // each barrier is exactly one phase ahead of what the waiter has seen.
                umma_commit(&bars->o_full[q & 1]);
                if (++vs == p.v_stages) { vs = 0; vpar ^= 1u; }
                if (++pb == p.p_bufs) { pb = 0; ppar ^= 1u; }
                seg_first = (cur.blk == cur.nb - 1);       // the next block opens a segment
                cur.advance(p, q + 1 < n_my);
            }
        }
    } else {
        att_softmax<DH, NCHT, HALVES>(p, tab, sm, cur, n_my);
    }

    tc_fence_before();
    __syncthreads();
    if (warp == kAttProducerWarps) {
        tc_fence_after();
        tmem_dealloc(tmem_base, kAttTmemCols);
    }
}

// one kernel per (head dim, chunks of 32 query rows): each instance keeps only the registers and the
// code of its own softmax width
template <int DH, int NCHT, int HALVES>
static cudaError_t att_set_smem()
{
    return cudaFuncSetAttribute(attention_kernel<DH, NCHT, HALVES>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                kAttSmemLimit - kAttStaticReserve);
}
template <int DH>
static cudaError_t att_init_dh()
{
    cudaError_t e = att_set_smem<DH, 1, 1>();
    if (e == cudaSuccess) e = att_set_smem<DH, 2, 2>();
    if (e == cudaSuccess) e = att_set_smem<DH, 3, 3>();
    if (e == cudaSuccess) e = att_set_smem<DH, 4, 2>();
    return e;
}
cudaError_t attention_init(int head_dim)
{
    return head_dim == 128 ? att_init_dh<128>() : att_init_dh<64>();
}

template <int DH>
static void att_launch_dh(const CUtensorMap& kv_map, const AttnParams& p, const AttTable& tab, int32_t n_ctas, cudaStream_t stream)
{
    const size_t smem = static_cast<size_t>(p.k_stages + p.v_stages) * AttCfg<DH>::kTileBytes +
                        AttCfg<DH>::fixed_bytes(p.n_pad, p.p_bufs);
    // up to 32 query rows per kv head: four softmax warps, one thread per token; beyond: eight, two threads
    // per token that split the rows (one warp per scheduler could not hide the latencies of a wide tile)
    dim3 grid(n_ctas);
    if (p.n_pad <= 32) attention_kernel<DH, 1, 1><<<grid, 256, smem, stream>>>(kv_map, p, tab);
    else if (p.n_pad <= 64) attention_kernel<DH, 2, 2><<<grid, 384, smem, stream>>>(kv_map, p, tab);
    else if (p.n_pad <= 96) attention_kernel<DH, 3, 3><<<grid, 512, smem, stream>>>(kv_map, p, tab);   // three threads per token
    else attention_kernel<DH, 4, 2><<<grid, 384, smem, stream>>>(kv_map, p, tab);
}

cudaError_t launch_attention(const Handle& h, const CUtensorMap& kv_map, const AttnParams& p, const AttTable& tab,
                             int32_t n_ctas, cudaStream_t stream)
{
    if (h.cfg.head_dim == 128) att_launch_dh<128>(kv_map, p, tab, n_ctas, stream);
    else att_launch_dh<64>(kv_map, p, tab, n_ctas, stream);
    return cudaGetLastError();
}

}  // namespace fs
