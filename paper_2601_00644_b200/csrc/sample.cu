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
//   accept : one cluster of eight CTAs per sequence: merges the parts of the sequence's rows,
//            evaluates the acceptance tests with Philox uniforms, finds the first rejection by warp
//            vote, and draws the emitted token from row n by inverse CDF in vocabulary order
//            (fp32 exponentials accumulated in fp64) -- results travel between the CTAs through
//            distributed shared memory, so the whole decision is one launch.
#include <cooperative_groups.h>

#include "common.cuh"
#include "internal.h"

namespace fs {

constexpr int kSampleThreads = 256;
constexpr int kSampleWarps = kSampleThreads / 32;
constexpr int kElemsPerThread = kSampleChunk / kSampleThreads;   // 32

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
    const float c = p.row_c[row];                         // log2(e) / T of the row's sequence
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

namespace cg = cooperative_groups;

// asynchronous copies global -> shared memory
__device__ __forceinline__ void cp_async_16(float* smem_dst, const float* src)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_u32(smem_dst)), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_4(float* smem_dst, const float* src)
{
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(smem_u32(smem_dst)), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_wait_all()
{
    asm volatile("cp.async.wait_all;" ::: "memory");
}

// ------------------------------------------------------------------------------------ top-k / top-p filter
// The paper's stochastic regime samples the target with top-p 0.9; top-k is its usual companion and
// is applied first.  Both filters are thresholds on the logit: the kept set of a row is
// {v : z_v >= tau}, tau being the k-th largest logit (top-k; ties with it are kept), respectively the
// largest logit such that the tokens with logit >= tau hold at least top_p of the (top-k filtered)
// mass.  tau is found exactly by a selection over an order-preserving integer code of the logits:
// round after round the interval of codes that can still hold tau is cut into up to 128 bins, every
// live entry adds its weight (1 for top-k, its probability mass for top-p) to the bin of its code,
// and a walk over the bins from the largest logits down finds the bin in which the running weight
// reaches the target.  As soon as that bin holds at most kFilterCand entries they are collected and
// ranked directly by their logits, which ends the selection.
//
// The code of an entry is a 23-bit fixed-point image of d = m - z over [0, d_max]: the mantissa of
// 1 + d / d_max (one fused multiply-add; values past d_max share the last code).  m is the row
// maximum and d_max a multiple of the spread of the part maxima, both taken from the softmax
// statistics of the row, so no pass over the row is spent on them.  The code grows with d but is not
// one-to-one; that is harmless: entries that share a code are told apart when they are ranked by
// their logits, and should a single code ever hold more than kFilterCand entries, the selection
// carries on over the bit pattern of z itself inside that group (second phase).  The result is exact
// whatever d_max was; a poor d_max only costs rounds.
//
// One cluster of four CTAs per target row, a contiguous slice of the vocabulary per CTA.  The first
// round reads the slice from global memory (the one read of the logits that comes from DRAM), leaves
// every entry's first-round bin in shared memory (one byte per entry) and accumulates into a
// histogram with one column per lane (bank = lane: an atomic instruction of a warp is one wavefront,
// where 32 lanes falling into a few dozen bins of a plain histogram were measured at 3.8 wavefronts
// per instruction and bound the whole kernel); the columns are added up before the hand-over.  The
// later rounds scan the stored bytes, list the entries whose byte lies in the live range (a few
// percent), fetch those logits out of L2 all at once and from then on work on the list.  A round
// ends with one cluster barrier, after which every CTA adds up the four histograms (read from its
// peers' shared memory; histograms alternate between two buffers, so one barrier per round is
// enough) and walks them; all CTAs reach the same result, so nothing is broadcast.
// Masses are accumulated as fixed-point integers (2^(-d c) rounded to units of 2^-31, added as two
// 16-bit limbs with the native 32-bit shared-memory atomics; 64-bit shared-memory atomics were
// measured 15x slower): integer addition is exact and order-independent, so the histograms, the
// totals and the comparison with the target are the same whatever the order of the atomic adds, and
// a row's result does not depend on scheduling.  The rounding of one entry is at most 2^-32 and
// unbiased: over a 128 K row its sum stays near 1e-8 of the mass.
constexpr int kFilterCluster = 4;
constexpr int kFilterThreads = 512;
constexpr int kFilterWarps = kFilterThreads / 32;
constexpr int kFilterBins = 128;
constexpr int kFilterCodeBits = 23;
constexpr int kFilterShift0 = kFilterCodeBits - 7;        // first round: the leading seven bits of the code
constexpr int kFilterCodesMax = 32768;                    // entries of a slice whose first-round bin is kept in shared memory
constexpr int kFilterList = 2048;                         // live entries of a slice listed after the first round
constexpr int kFilterCand = 128;                          // a bin with at most this many entries is ranked directly
constexpr int kFilterMaxRounds = 32;                      // (a selection needs far fewer: every round shrinks the interval)
constexpr double kMassUnit = 2147483648.0;                // 2^31
constexpr float kMassUnitF = 2147483648.0f;

__device__ __forceinline__ uint32_t order_key(float z)       // larger float <-> larger key
{
    const uint32_t u = __float_as_uint(z);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float key_to_float(uint32_t k)
{
    return __uint_as_float((k & 0x80000000u) ? (k & 0x7fffffffu) : ~k);
}

// what a round of the selection looks at (identical in the four CTAs of a row)
struct FilterRound {
    uint32_t lo, hi;                                    // live codes: lo <= code <= hi
    uint32_t base;                                      // bin = clamp((code >> shift) - base, 0, kFilterBins - 1)
    int shift;
    int phase;                                          // 0: code of d;  1: code = ~key(z) among the entries whose code of d is dsel
    uint32_t dsel;
    int next;                                           // after the walk: 0 another round, 1 collect and rank, 2 tau is known
    uint32_t n_sel;                                     // entries in the chosen bin (when the round counted them)
    unsigned long long above;                           // weight of the codes below lo (the logits above the live interval)
    unsigned long long target;
    float tau;
    unsigned long long kept;
};

struct FilterShared {
    uint32_t hist[2][3][kFilterBins];                   // [buffer][mass bits 16..31 | mass bits 0..15 | entries][bin]
    unsigned long long tot[kFilterBins];                // cluster-wide weight per bin
    uint32_t totc[kFilterBins];                         // cluster-wide entries per bin
    float cand_z[kFilterCand];
    uint32_t cand_w[kFilterCand];
    float red_hi[kFilterWarps], red_lo[kFilterWarps];
    unsigned long long red64[kFilterWarps];
    unsigned long long slice_mass[kFilterCluster];
    uint32_t n_cand;
    uint32_t list_n;
    FilterRound r;
};

// 2^(-d c) in fixed point (units of 2^-31, round to nearest), d = m - z >= 0
__device__ __forceinline__ uint32_t mass_of(float d, float cf)
{
    return __float2uint_rn(fast_exp2(d * -cf) * kMassUnitF);   // <= 2^31
}
// 23-bit code of d >= 0: the mantissa of min(1 + d * inv_dmax, 2 - 2^-23)
__device__ __forceinline__ uint32_t code_of(float d, float inv_dmax)
{
    return __float_as_uint(fminf(fmaf(d, inv_dmax, 1.f), 1.99999988f)) - 0x3f800000u;
}
__device__ __forceinline__ int bin_of(uint32_t code, int shift, uint32_t base)
{
    const uint32_t t = code >> shift;
    return t <= base ? 0 : static_cast<int>(min(t - base, static_cast<uint32_t>(kFilterBins - 1)));
}

__global__ void __cluster_dims__(kFilterCluster, 1, 1) __launch_bounds__(kFilterThreads, 3)
sample_filter_kernel(const SampleParams p)
{
    // first-round bin of every entry of this CTA's slice (when it fits), then the first round's histogram with one
    // column per lane: [limb][bin][lane].  Once its columns are added up the histogram is dead and its room holds
    // the list of live entries (indices, then logits).
    extern __shared__ __align__(16) uint8_t s_bin0[];
    __shared__ FilterShared sh;
    cg::cluster_group cluster = cg::this_cluster();
    const int rank = static_cast<int>(cluster.block_rank());
    const int row = blockIdx.y;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    cluster_arrive();                                   // "this CTA runs" (awaited before the first peer access)

    // ---- this CTA's slice: [v0, v1), a multiple of four entries long so that 16-byte loads stay aligned
    const int per = ((p.vocab + kFilterCluster - 1) / kFilterCluster + 3) & ~3;
    const int v0 = min(p.vocab, rank * per), v1 = min(p.vocab, v0 + per);
    const int n = v1 - v0;
    const bool coded = per <= kFilterCodesMax;
    const bool vec_ok = ((p.vocab & 3) == 0);
    uint32_t* s_big = reinterpret_cast<uint32_t*>(s_bin0 + (coded ? per : 0));
    uint16_t* s_idx = reinterpret_cast<uint16_t*>(s_big);
    float* s_list = reinterpret_cast<float*>(s_big + kFilterList * sizeof(uint16_t) / sizeof(uint32_t));
    for (int i = tid; i < 3 * kFilterBins; i += kFilterThreads) (&sh.hist[0][0][0])[i] = 0u;
    for (int i = tid; i < 2 * kFilterBins * 32; i += kFilterThreads) s_big[i] = 0u;
    if (tid == 0) sh.n_cand = 0u;
    pdl_wait();                                         // the logits and their statistics come from the preceding kernel
    pdl_launch_dependents();
    const float cf = p.row_c[row];
    const uint32_t* mask_row = (p.vocab_mask != nullptr) ? p.vocab_mask + static_cast<int64_t>(p.row_seq[row]) * p.mask_words : nullptr;
    const float* src = p.logits + static_cast<int64_t>(row) * p.vocab + v0;

    // ---- row maximum m and the spread of the part maxima, from the row's softmax statistics (every CTA reads all
    // the parts, a few loads per thread all in flight at once: cheaper than an exchange between the CTAs)
    float m, part_lo;
    {
        const float2* tp = p.tstats + static_cast<int64_t>(row) * p.n_tparts;
        float hi = -INFINITY, lo = INFINITY;
#pragma unroll 4
        for (int t = tid; t < p.n_tparts; t += kFilterThreads) {
            const float x = __ldcg(&tp[t].x);
            hi = fmaxf(hi, x);
            if (x > -INFINITY) lo = fminf(lo, x);
        }
        hi = warp_max(hi);
        lo = -warp_max(-lo);
        if (lane == 0) { sh.red_hi[warp] = hi; sh.red_lo[warp] = lo; }
        __syncthreads();
        m = sh.red_hi[0]; part_lo = sh.red_lo[0];
#pragma unroll
        for (int w = 1; w < kFilterWarps; ++w) { m = fmaxf(m, sh.red_hi[w]); part_lo = fminf(part_lo, sh.red_lo[w]); }
        cluster_wait();                                 // all four CTAs have started
    }
    if (m == -INFINITY) {                               // nothing can be selected in this row
        if (rank == 0 && tid == 0) {
            p.topp[static_cast<int64_t>(row) * 2] = -static_cast<double>(INFINITY);
            p.topp[static_cast<int64_t>(row) * 2 + 1] = 0.0;
        }
        cluster_sync();
        return;
    }
    // d_max: a multiple of the spread of the part maxima (the maxima of 32-entry parts spread almost like the
    // row's bulk, those of large parts much less), and no more than where the mass vanishes (2^-40 of the
    // largest).  A d_max that misses only costs rounds: the last code takes what lies beyond it.
    float inv_dmax;
    {
        const float spread = m - part_lo;
        float dmax = 40.f / cf;
        if (spread > 0.f && spread < INFINITY) dmax = fminf(dmax, spread * ((p.vocab / max(p.n_tparts, 1) >= 1024) ? 8.f : 2.25f));
        inv_dmax = 1.f / dmax;
    }

    const bool do_k = p.top_k > 0 && p.top_k < p.vocab;
    const bool do_p = p.top_p < 1.f;
    float floor_z = -3.402823466e38f;                   // logits below it are out: first "finite", later the top-k cut
    bool bytes_valid = false;
    int round_no = 0;                                   // alternates the histogram buffers

    // one logit that may be live: test it, add it to the histogram or hand it over as a candidate
    auto consider = [&](float z, int sel, const FilterRound& r, uint32_t* hist, bool collect) {
        if (!(z >= floor_z)) return;
        const float d = m - z;
        if (!(d >= 0.f)) return;
        const uint32_t dcode = code_of(d, inv_dmax);
        uint32_t code = dcode;
        if (r.phase != 0) {
            if (dcode != r.dsel) return;
            code = ~order_key(z);
        }
        if (code - r.lo > r.hi - r.lo) return;
        const uint32_t w = sel == 0 ? 1u : mass_of(d, cf);
        if (collect) {
            const uint32_t idx = atomicAdd(cluster.map_shared_rank(&sh.n_cand, 0), 1u);
            if (idx < static_cast<uint32_t>(kFilterCand)) {
#pragma unroll 1
                for (int c = 0; c < kFilterCluster; ++c) {
                    cluster.map_shared_rank(&sh.cand_z[0], c)[idx] = z;
                    cluster.map_shared_rank(&sh.cand_w[0], c)[idx] = w;
                }
            }
        } else {
            const int bin = bin_of(code, r.shift, r.base);
            if (sel != 0) {
                atomicAdd(&hist[bin], w >> 16);
                atomicAdd(&hist[kFilterBins + bin], w & 0xffffu);
            }
            atomicAdd(&hist[2 * kFilterBins + bin], 1u);
        }
    };
    auto fetch = [&](int i) -> float {                  // entry i of the slice, -inf when it is masked out
        const float z = __ldg(src + i);
        return (mask_row != nullptr && !mask_allows(mask_row, v0 + i)) ? -INFINITY : z;
    };
    // A pass over the slice for the round r.  The stored first-round bins tell which entries can be live; the
    // first such pass of a selection lists them (index, then value: the fetches of a round are all in flight
    // together instead of one after the other in a thread), and the later passes, whose live sets lie inside
    // that one, walk the list.  A list that does not fit sends the selection back to scanning.
    int list_state = 0;                                 // 0 none yet, 1 valid, 2 did not fit
    auto scan = [&](int sel, const FilterRound& r, uint32_t* hist, bool collect) {
        if (list_state == 1) {
            const int nl = static_cast<int>(sh.list_n);
            for (int j = tid; j < nl; j += kFilterThreads) consider(s_list[j], sel, r, hist, collect);
            return;
        }
        if (!bytes_valid) {
#pragma unroll 1
            for (int i = tid; i < n; i += kFilterThreads) consider(fetch(i), sel, r, hist, collect);
            return;
        }
        // live range of the stored bytes: the first-round bins of the interval's ends (of the group's code in phase 1)
        const uint32_t b_lo = (r.phase == 0 ? r.lo : r.dsel) >> kFilterShift0;
        const uint32_t b_span = ((r.phase == 0 ? r.hi : r.dsel) >> kFilterShift0) - b_lo;
        const uint32_t lo4 = b_lo * 0x01010101u, span4 = b_span * 0x01010101u;
        // the bytes of a word that lie in the live range, as four flag bits
        auto hits_of = [&](int i0) -> uint32_t {
            const uint32_t b4 = *reinterpret_cast<const uint32_t*>(s_bin0 + i0);
            uint32_t flags;                             // bit 7 of every byte that hits
            if (b_span == 0u) {
                const uint32_t x = b4 ^ lo4;            // zero bytes hit
                flags = ~(((x & 0x7f7f7f7fu) + 0x7f7f7f7fu) | x) & 0x80808080u;
            } else {
                flags = __vcmpleu4(__vsub4(b4, lo4), span4) & 0x80808080u;
            }
            uint32_t nib = ((flags >> 7) * 0x00204081u >> 21) & 15u;
            if (!vec_ok && i0 + 4 > n) nib &= (1u << (n - i0)) - 1u;   // (a slice is a multiple of four entries otherwise)
            return nib;
        };
        if (list_state == 0) {
            // one look at this thread's (at most 16) words: the hits as a 64-bit mask; room for the warp's hits is
            // reserved with one atomic, then the indices are written
            unsigned long long mask = 0ull;
            int word = 0;
#pragma unroll 1
            for (int i0 = tid * 4; i0 < n; i0 += kFilterThreads * 4, ++word)
                mask |= static_cast<unsigned long long>(hits_of(i0)) << (4 * word);
            const uint32_t mine = static_cast<uint32_t>(__popcll(mask));
            uint32_t incl = mine;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const uint32_t t0 = __shfl_up_sync(0xffffffffu, incl, o);
                if (lane >= o) incl += t0;
            }
            uint32_t at = 0u;
            if (lane == 31) at = atomicAdd(&sh.list_n, incl);
            at = __shfl_sync(0xffffffffu, at, 31) + incl - mine;
            while (mask != 0ull) {
                const int pos = __ffsll(static_cast<long long>(mask)) - 1;
                mask &= mask - 1ull;
                if (at < static_cast<uint32_t>(kFilterList))
                    s_idx[at] = static_cast<uint16_t>(tid * 4 + (pos >> 2) * (kFilterThreads * 4) + (pos & 3));
                ++at;
            }
            __syncthreads();
            const uint32_t total = sh.list_n;
            if (total <= static_cast<uint32_t>(kFilterList)) {
                list_state = 1;
                for (int j = tid; j < static_cast<int>(total); j += kFilterThreads) {
                    const float z = fetch(s_idx[j]);
                    s_list[j] = z;
                    consider(z, sel, r, hist, collect);
                }
                return;
            }
            list_state = 2;
        }
#pragma unroll 1
        for (int i0 = tid * 4; i0 < n; i0 += kFilterThreads * 4) {
            uint32_t nib = hits_of(i0);
            while (nib != 0u) {
                const int u = __ffs(nib) - 1;
                nib &= nib - 1u;
                consider(fetch(i0 + u), sel, r, hist, collect);
            }
        }
    };

    // ---- selections: top-k on counts (if on), then top-p on mass among the logits that survived
    for (int sel = do_k ? 0 : 1; sel < (do_p ? 2 : 1); ++sel) {
        // sel 0: weight 1, target k.   sel 1: weight mass, target top_p * (mass of the logits >= floor_z)
        if (tid == 0) {
            FilterRound r0;
            r0.lo = 0u; r0.hi = code_of(m - floor_z, inv_dmax);   // every code down to the floor's
            r0.base = 0u; r0.shift = kFilterShift0; r0.phase = 0; r0.dsel = 0u; r0.next = 0; r0.n_sel = 0u;
            r0.above = 0ull; r0.target = 0ull; r0.tau = floor_z; r0.kept = 0ull;
            sh.r = r0;
            sh.list_n = 0u;
        }
        __syncthreads();
        bool first = true;                              // first round of the selection: its total fixes the target
        list_state = 0;
        for (int it = 0; it < kFilterMaxRounds; ++it, ++round_no) {
            const FilterRound r = sh.r;
            uint32_t* hist = &sh.hist[round_no & 1][0][0];
            bool counted = true;                        // the round records how many entries each bin holds
            if (!bytes_valid && first) {
                // The first pass of the kernel: every entry of the slice, straight from global memory; leaves the
                // bins in shared memory.  Lane l adds into column l of the histogram, so the 32 atomics of a warp
                // instruction go to 32 banks.  For top-p the entry count is left out (two atomics per entry).
                counted = sel == 0;
                if (round_no != 0) {                    // (cleared in the prologue for the kernel's first round)
                    for (int i = tid; i < 2 * kFilterBins * 32; i += kFilterThreads) s_big[i] = 0u;
                    __syncthreads();
                }
                uint32_t* col = s_big + lane;
                // (the first selection of the kernel has no floor yet, and an entry that cannot be selected is -inf: its
                // distance clamps into the last bin, where its mass is 0 and a count too many only matters to a
                // top-k that reaches down there -- the next round counts that bin's live entries exactly, and a k
                // beyond them keeps every logit, as it should)
                const bool plain = round_no == 0;
                auto entries4 = [&](const float* zin, int i0) {
                    float z[4] = {zin[0], zin[1], zin[2], zin[3]};
                    if (mask_row != nullptr) {
#pragma unroll
                        for (int u = 0; u < 4; ++u)
                            if (i0 + u < n && !mask_allows(mask_row, v0 + i0 + u)) z[u] = -INFINITY;
                    }
                    uint32_t tb[4];                     // bits of min(1 + d / d_max, 2 - 2^-23): byte 2 = 0x80 | bin
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        const float d = m - z[u];
                        tb[u] = __float_as_uint(fminf(fmaf(d, inv_dmax, 1.f), 1.99999988f));
                        if (plain) {
                            uint32_t* at = col + ((tb[u] >> 11) & 0xfe0u);         // bin * 32 words
                            if (sel == 0) {
                                atomicAdd(at, 1u);
                            } else {
                                const uint32_t w = mass_of(d, cf);
                                atomicAdd(at, w >> 16);
                                atomicAdd(at + kFilterBins * 32, w & 0xffffu);
                            }
                        } else {
                            const bool live = z[u] >= floor_z && d >= 0.f;
                            if (!live) tb[u] = 0x3fff0000u;                         // the last bin
                            const uint32_t bin = (tb[u] >> 16) & 0x7fu;
                            if (live) {
                                if (sel == 0) {
                                    atomicAdd(col + bin * 32u, 1u);
                                } else {
                                    const uint32_t w = mass_of(d, cf);
                                    atomicAdd(col + bin * 32u, w >> 16);
                                    atomicAdd(col + (kFilterBins + bin) * 32u, w & 0xffffu);
                                }
                            }
                        }
                    }
                    if (coded)
                        *reinterpret_cast<uint32_t*>(s_bin0 + i0) =
                            __byte_perm(__byte_perm(tb[0], tb[1], 0x0062), __byte_perm(tb[2], tb[3], 0x0062), 0x5410) ^ 0x80808080u;
                };
                // four loads of a thread are in flight before the first of them is used
                constexpr int kStep = kFilterThreads * 4;
#pragma unroll 1
                for (int base = tid * 4; base < n; base += 4 * kStep) {
                    float z[4][4];
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        const int i0 = base + q * kStep;
                        if (vec_ok && i0 < n) {
                            const float4 x = __ldg(reinterpret_cast<const float4*>(src + i0));
                            z[q][0] = x.x; z[q][1] = x.y; z[q][2] = x.z; z[q][3] = x.w;
                        } else {
#pragma unroll
                            for (int u = 0; u < 4; ++u) z[q][u] = (i0 + u < n) ? __ldg(src + i0 + u) : -INFINITY;
                        }
                    }
#pragma unroll
                    for (int q = 0; q < 4; ++q)
                        if (base + q * kStep < n) entries4(z[q], base + q * kStep);
                }
                __syncthreads();
                // add up the columns: thread (limb, bin) reads its 32 columns, rotated so that a warp's reads fall
                // into 32 banks
                if (tid < 2 * kFilterBins) {
                    uint32_t sum = 0u;
#pragma unroll 8
                    for (int k = 0; k < 32; ++k) sum += s_big[tid * 32 + ((k + tid) & 31)];
                    if (sel != 0) hist[tid] = sum;
                    else if (tid < kFilterBins) hist[2 * kFilterBins + tid] = sum;
                }
                bytes_valid = coded;
            } else {
                scan(sel, r, hist, false);
            }
            cluster_sync();                             // all four histograms of this round are complete
            // cluster-wide histogram: thread t adds bin t of the four CTAs; the other buffer is cleared for the
            // next round (its last readers arrived at the barrier above after they were done with it)
            if (tid < kFilterBins) {
                unsigned long long acc = 0ull;
                uint32_t cnt = 0u;
#pragma unroll
                for (int c = 0; c < kFilterCluster; ++c) {
                    const uint32_t* peer = cluster.map_shared_rank(hist, c);
                    if (sel != 0) acc += (static_cast<unsigned long long>(peer[tid]) << 16) + peer[kFilterBins + tid];
                    if (counted) cnt += peer[2 * kFilterBins + tid];
                }
                sh.tot[tid] = sel == 0 ? static_cast<unsigned long long>(cnt) : acc;
                sh.totc[tid] = cnt;
                uint32_t* other = &sh.hist[(round_no & 1) ^ 1][0][0];
                other[tid] = 0u; other[kFilterBins + tid] = 0u; other[2 * kFilterBins + tid] = 0u;
            }
            __syncthreads();
            if (warp == 0) {
                // walk from the largest logits (bin 0) down: lane l owns bins 4 l ... 4 l + 3
                constexpr int kPerLane = kFilterBins / 32;
                unsigned long long mine = 0ull;
#pragma unroll
                for (int j = 0; j < kPerLane; ++j) mine += sh.tot[lane * kPerLane + j];
                unsigned long long incl = mine;          // inclusive scan over lanes
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const unsigned long long t0 = __shfl_up_sync(0xffffffffu, incl, o);
                    if (lane >= o) incl += t0;
                }
                unsigned long long target = r.target;
                if (first) {
                    // total weight of the live entries = the base of the target
                    const unsigned long long total = __shfl_sync(0xffffffffu, incl, 31);
                    target = (sel == 0) ? static_cast<unsigned long long>(p.top_k)
                                        : static_cast<unsigned long long>(static_cast<double>(p.top_p) * static_cast<double>(total));
                    if (target < 1ull) target = 1ull;
                }
                unsigned long long run = r.above + incl - mine;
                const unsigned hit = __ballot_sync(0xffffffffu, run + mine >= target);
                // (with exact sums the last lane always reaches the target; the guard keeps the walk defined)
                const int l = hit != 0u ? __ffs(hit) - 1 : 31;
                if (lane == l) {
                    int bin = lane * kPerLane;
                    for (int j = 0; j < kPerLane - 1; ++j, ++bin) {
                        if (run + sh.tot[bin] >= target) break;
                        run += sh.tot[bin];
                    }
                    // the codes of the chosen bin; the end bins of a window also hold what lies outside it
                    const unsigned long long v = static_cast<unsigned long long>(r.base) + static_cast<unsigned long long>(bin);
                    uint32_t lo = r.lo, hi = r.hi;
                    if (bin > 0) lo = static_cast<uint32_t>(max(static_cast<unsigned long long>(lo), v << r.shift));
                    if (bin < kFilterBins - 1) hi = static_cast<uint32_t>(min(static_cast<unsigned long long>(hi), ((v + 1ull) << r.shift) - 1ull));
                    FilterRound q = r;
                    q.target = target; q.above = run; q.lo = lo; q.hi = hi;
                    q.n_sel = counted ? sh.totc[bin] : 0xffffffffu;
                    if (q.n_sel <= static_cast<uint32_t>(kFilterCand)) {
                        q.next = 1;                     // few enough: collect them and rank them directly
                    } else if (lo == hi) {
                        if (r.phase == 0) {
                            // one code of d, many entries: go on over the bits of z itself inside this group
                            q.phase = 1; q.dsel = lo; q.lo = 0u; q.hi = 0xffffffffu; q.shift = 25; q.base = 0u;
                        } else {
                            q.next = 2;                 // one logit value: it is tau, and all its entries are kept
                            q.tau = key_to_float(~lo);
                            q.kept = run + sh.tot[bin];
                        }
                    } else {
                        // cut the interval into (at most 129, the last two sharing a bin) equal parts
                        const int width = 32 - __clz(hi - lo);
                        q.shift = max(0, width - 7);
                        q.base = lo >> q.shift;
                    }
                    sh.r = q;
                }
            }
            __syncthreads();
            first = false;
            if (sh.r.next != 0) { ++round_no; break; }
        }
        const FilterRound r = sh.r;
        if (r.next == 1) {
            // every CTA hands its entries of the chosen bin to all four CTAs; each ranks them on its own
            scan(sel, r, nullptr, true);
            cluster_sync();
            const int nc = static_cast<int>(min(r.n_sel, static_cast<uint32_t>(kFilterCand)));
            if (tid < nc) {
                const float zt = sh.cand_z[tid];
                unsigned long long gt = 0ull, ge = 0ull;   // weight of the candidates above zt / not below zt
#pragma unroll 4
                for (int j = 0; j < nc; ++j) {
                    const float zj = sh.cand_z[j];
                    const unsigned long long wj = sh.cand_w[j];
                    gt += zj > zt ? wj : 0ull;
                    ge += zj >= zt ? wj : 0ull;
                }
                if (r.above + gt < r.target && r.above + ge >= r.target) { sh.r.tau = zt; sh.r.kept = r.above + ge; }
            }
            __syncthreads();
            if (tid == 0) sh.n_cand = 0u;               // (rank 0's counter; the next hand-over is two barriers away)
        } else if (r.next == 0 && rank == 0 && tid == 0) {
            report_error(p.status, kErrTimeout, row, 7);   // cannot happen: every round shrinks the interval
        }
        floor_z = sh.r.tau;                             // every logit >= it is kept
        __syncthreads();
    }
    double kept_mass = static_cast<double>(sh.r.kept) / kMassUnit;
    if (!do_p) {
        // top-k alone: the mass of the kept logits is one more pass (a plain reduction, no histogram)
        unsigned long long acc = 0ull;
        const uint32_t b_hi = code_of(m - floor_z, inv_dmax) >> kFilterShift0;
        for (int i = tid; i < n; i += kFilterThreads) {
            if (bytes_valid && s_bin0[i] > b_hi) continue;
            const float z = fetch(i);
            if (z >= floor_z) acc += mass_of(m - z, cf);
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
        if (lane == 0) sh.red64[warp] = acc;
        __syncthreads();
        if (tid < kFilterCluster) {
            unsigned long long t = 0ull;
#pragma unroll
            for (int w = 0; w < kFilterWarps; ++w) t += sh.red64[w];
            cluster.map_shared_rank(&sh.slice_mass[0], tid)[rank] = t;
        }
        cluster_sync();
        unsigned long long t = 0ull;
#pragma unroll
        for (int c = 0; c < kFilterCluster; ++c) t += sh.slice_mass[c];
        kept_mass = static_cast<double>(t) / kMassUnit;
    }
    if (rank == 0 && tid == 0) {
        p.topp[static_cast<int64_t>(row) * 2] = static_cast<double>(floor_z);
        p.topp[static_cast<int64_t>(row) * 2 + 1] = kept_mass;
    }
    cluster_sync();                                     // no CTA leaves while a peer may still read its shared memory
}

static size_t filter_smem_bytes(int vocab)
{
    const int per = ((vocab + kFilterCluster - 1) / kFilterCluster + 3) & ~3;
    return (per <= kFilterCodesMax ? static_cast<size_t>(per) : 0) + static_cast<size_t>(2 * kFilterBins * 32) * sizeof(uint32_t);
}

cudaError_t launch_sample_filter(const SampleParams& p, bool pdl, cudaStream_t stream)
{
    return launch_kernel_ex(sample_filter_kernel, dim3(kFilterCluster, p.m_rows), dim3(kFilterThreads), filter_smem_bytes(p.vocab),
                            stream, pdl, p);
}

// ------------------------------------------------------------------------------------ acceptance
// One thread-block cluster of eight CTAs per sequence does the whole decision in one launch; the
// CTAs hand their results to one another through distributed shared memory, so there are no
// global-memory tickets, fences or second launch on the path from the logits to the outputs.
//
//   before the dependency wait (the kernel is launched programmatically behind the LM head): what
//     needs only the step's inputs and the draft-logit statistics -- the draft token, q_j(x_j) and
//     the Philox uniform of every acceptance test of this CTA's rows (rows are dealt round-robin).
//   A  each CTA merges the parts of its target rows (maximum first, then the sum with fp32 weights
//     accumulated in fp64), evaluates u * q(x) < p(x) (GREEDY: compares x with the arg-max) and
//     writes the row's result into the shared memory of all eight CTAs.        -- cluster barrier --
//   B  every CTA finds the first rejection n by warp vote over the row results (GREEDY ends here).
//   C  row n only: the vocabulary is cut into eight contiguous slices, one per CTA, and a slice into
//     chunks of 1024 entries, one warp each, streamed through shared memory in halves; the mass of
//     the emission weights of every group of 16 entries and of every chunk is recorded, slice
//     totals go to all CTAs.                                                    -- cluster barrier --
//   D  the CTA whose slice holds u' * Z picks the chunk, then the group of 16, from its lists and
//     scans those 16 entries in vocabulary order (inverse CDF).  If rounding leaves no entry above
//     the threshold, the last entry with positive mass is taken, at every level.
//
// The kernel runs once per step and is short, and the step streams gigabytes through L2 in between,
// so its instructions are fetched cold (from DRAM) every time: straight-line code was measured at
// about a microsecond per few KB on this path.  The loops of C and D are therefore kept rolled and
// the logits travel to shared memory asynchronously (all copies of a chunk in flight at once) instead
// of into a long unrolled register tile; D then scans the picked chunk where C left it.
//
// Arithmetic of C and D.  The weights are kept in units of 1 / s_p (s = sum of 2^((z - max) c) of a
// row): w_v = max(0, e_p(v) - rho e_q(v)) at a rejection, rho = s_p / s_q, and w_v = e_p(v) for the
// bonus row, with e = the same fp32 2^x as in the statistics.  A common factor does not move the
// inverse CDF, so no entry is ever normalised.  Entries are fp32 (one fused multiply-add); a lane
// adds the 16 of a group in fp32 and everything above that -- groups, chunks, slices, the running
// sums of the final scan -- is fp64.  (Double-precision arithmetic per entry was measured at 12 us for this
// phase alone: the vector fp64 rate of this GPU is a small fraction of its fp32 rate.)
constexpr int kAcceptThreads = 256;        // two CTAs per SM: every cluster of a 16-sequence batch finds room at once
constexpr int kAcceptWarps = kAcceptThreads / 32;
constexpr int kAcceptRowsPerCta = (kMaxK + 1 + kAcceptCluster - 1) / kAcceptCluster;   // 8

struct RowResult {
    double s_p, s_q, tau;             // sum of 2^((z - max) * c) of the target / draft row; lowest kept logit of the nucleus
    float m_p, m_q;                   // maxima (logit units)
    float rho;                        // s_p / s_q of a row that has a draft row (the residual's scale), else 0
    int32_t rej;                      // 1: this row's draft token is rejected
    int32_t argmax;                   // GREEDY: lowest index holding the row's maximum
};

// Row n of one sequence: the unnormalised weights the emitted token is drawn from.
struct DrawRow {
    const float* zt; const float* zd; const uint32_t* mask;
    float mp, mq, c, tau;             // tau: lowest logit of the target row's nucleus (-inf: no top-p filter)
    float rho;                        // s_p / s_q
    bool residual;
    bool plain;                       // no vocabulary mask and no nucleus: e_p needs no per-entry checks
    // 2^((z - max) c); a logit of -inf gives 2^-inf = 0 by itself
    __device__ __forceinline__ float e_p(float z, int v) const
    {
        if (!plain && (z < tau || !mask_allows(mask, v))) return 0.f;
        return fast_exp2((z - mp) * c);
    }
    __device__ __forceinline__ float e_q(float z) const { return fast_exp2((z - mq) * c); }
    // weight of entry v; use_p: draw from p itself (bonus row, or a residual without mass)
    __device__ __forceinline__ float weight(float zt_v, float zd_v, int v, bool use_p) const
    {
        const float ep = e_p(zt_v, v);
        return use_p ? ep : fmaxf(fmaf(-rho, e_q(zd_v), ep), 0.f);
    }
};
// Streaming of row n through shared memory.  A chunk (kWarpChunk = 1024 entries) is two sub-chunks of
// 512; a sub-chunk is 32 groups of 16 consecutive entries, group g being added up by lane g.  Inside a
// group the four 16-byte pieces are permuted by (g >> 1) & 3, so that the lanes' 16-byte reads of
// their own groups (64 bytes apart) fall into different banks.
constexpr int kSubChunk = 512;
constexpr int kGroup = 16;
constexpr int kGroupsPerChunk = kWarpChunk / kGroup;                    // 64
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
__device__ __forceinline__ void cp_async_wait_group_1() { asm volatile("cp.async.wait_group 1;" ::: "memory"); }
// One warp requests the entries [base, base + kSubChunk) of a row (those below vocab); nothing is
// awaited.  vec_ok: the row starts on a 16-byte boundary and vocab is a multiple of four.
__device__ __forceinline__ void stage_sub(float* dst, const float* row, int base, int vocab, bool vec_ok, int lane)
{
    if (vec_ok) {
#pragma unroll
        for (int it = 0; it < kSubChunk / 128; ++it) {
            const int q = it * 32 + lane;                               // 16-byte piece of the sub-chunk
            const int g = q >> 2, j = q & 3;
            if (base + 4 * q < vocab) cp_async_16(dst + g * kGroup + ((j ^ ((g >> 1) & 3)) << 2), row + base + 4 * q);
        }
    } else {
#pragma unroll 4
        for (int e = lane; e < kSubChunk; e += 32) {
            const int g = e >> 4, j = (e >> 2) & 3;
            if (base + e < vocab) cp_async_4(dst + g * kGroup + ((j ^ ((g >> 1) & 3)) << 2) + (e & 3), row + base + e);
        }
    }
}

__device__ __forceinline__ double warp_inclusive_scan(double v, int lane)
{
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const double t = __shfl_up_sync(0xffffffffu, v, o);
        if (lane >= o) v += t;
    }
    return v;
}

// In a list of n masses (vocabulary order) finds the first entry at which the running sum, started
// at `carry`, exceeds thr; if none does, the last entry with positive mass (-1 if there is none).
// Called by one full warp; `mass(i)` returns the i-th mass.  Returns the index and the running sum
// before it.
template <typename MassFn>
__device__ __forceinline__ int warp_pick(int n, double carry, double thr, int lane, MassFn mass, double& before)
{
    int pick = -1, last_pos = -1;
    double last_before = 0.0;
    before = carry;
    for (int c0 = 0; c0 < n && pick < 0; c0 += 32) {
        const int cc = c0 + lane;
        const double m = (cc < n) ? mass(cc) : 0.0;
        const double incl = warp_inclusive_scan(m, lane) + carry;
        const unsigned hit = __ballot_sync(0xffffffffu, cc < n && m > 0.0 && incl > thr);
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
    return pick;
}

__global__ void __cluster_dims__(kAcceptCluster, 1, 1) __launch_bounds__(kAcceptThreads)
sample_accept_kernel(const SampleParams p)
{
    __shared__ RowResult s_row[kMaxK + 1];               // results of all rows of the sequence (every CTA holds a copy)
    __shared__ RowResult s_tmp;
    __shared__ double2 s_wc[kMaxWarpChunksPerCta];       // (residual mass, p mass) of this CTA's chunks
    __shared__ double s_slice[kAcceptCluster][2];        // slice totals of all CTAs
    __shared__ float red_f[kAcceptWarps];
    __shared__ double red_d[kAcceptWarps];
    __shared__ int red_i[kAcceptWarps];
    __shared__ int s_x[kAcceptRowsPerCta];
    __shared__ double s_qt[kAcceptRowsPerCta], s_u[kAcceptRowsPerCta], s_mq[kAcceptRowsPerCta], s_sq[kAcceptRowsPerCta];
    __shared__ double s_u2[kMaxK + 1];                   // uniform of the emitted token after n accepted drafts, every n
    __shared__ int s_n;

    cg::cluster_group cluster = cg::this_cluster();
    const int rank = static_cast<int>(cluster.block_rank());
    const int b = blockIdx.y;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int k_b = p.k_eff[b];                            // tables of the plan kernel: complete before the preceding kernel started
    const int q0 = p.cu_q[b], d0 = p.cu_d[b];
    const float cf = p.row_c[q0];                          // log2(e) / T of this sequence
    const double scale = static_cast<double>(cf);
    const int my_rows = (k_b >= rank) ? (k_b - rank) / kAcceptCluster + 1 : 0;      // rows rank, rank + 8, ... <= k_b
    cluster_arrive();                                      // "this CTA runs": awaited before the first write into a peer's shared memory

    // ---- what needs no target logits.  The uniforms of the emitted token, one per possible n:
    if (!p.greedy && threadIdx.x <= k_b) s_u2[threadIdx.x] = philox_uniform(p.seeds[b], static_cast<uint32_t>(threadIdx.x), 1u);
    // ---- draft side of this CTA's acceptance tests: warp i handles row rank + 8 i
    if (warp < my_rows) {
        const int j = rank + warp * kAcceptCluster;
        if (j < k_b) {
            int x = p.draft_tokens[d0 + j];
            x = min(max(x, 0), p.vocab - 1);
            if (!p.greedy) {
                // the row's parts (at most a few per lane: kept in registers, so they are read once)
                const float2* dp = p.stats + static_cast<int64_t>(p.m_rows + d0 + j) * p.n_chunks;
                float2 part[4];
                float mqf = -INFINITY;
#pragma unroll
                for (int t = 0; t < 4; ++t) {
                    const int i = lane + 32 * t;
                    part[t] = (i < p.n_chunks) ? __ldcg(&dp[i]) : make_float2(-INFINITY, 0.f);
                    mqf = fmaxf(mqf, part[t].x);
                }
                for (int i = lane + 128; i < p.n_chunks; i += 32) mqf = fmaxf(mqf, __ldcg(&dp[i].x));   // vocabularies beyond 1M / 8: none today
                mqf = warp_max(mqf);
                double acc = 0.0;
#pragma unroll
                for (int t = 0; t < 4; ++t)
                    if (part[t].x != -INFINITY) acc += static_cast<double>(part[t].y) * static_cast<double>(fast_exp2((part[t].x - mqf) * cf));
                for (int i = lane + 128; i < p.n_chunks; i += 32) {
                    const float2 pt = __ldcg(&dp[i]);
                    if (pt.x != -INFINITY) acc += static_cast<double>(pt.y) * static_cast<double>(fast_exp2((pt.x - mqf) * cf));
                }
                const double sq = warp_sum(acc);
                if (lane == 0) {
                    const double mq = static_cast<double>(mqf);
                    const double zq = static_cast<double>(p.draft_logits[static_cast<int64_t>(d0 + j) * p.vocab + x]);
                    s_mq[warp] = mq; s_sq[warp] = sq;
                    s_qt[warp] = (zq == -INFINITY) ? 0.0 : static_cast<double>(fast_exp2(static_cast<float>((zq - mq) * scale))) / sq;
                    s_u[warp] = philox_uniform(p.seeds[b], static_cast<uint32_t>(j), 0u);
                }
            }
            if (lane == 0) s_x[warp] = x;
        } else if (lane == 0) {
            s_x[warp] = 0; s_mq[warp] = 0.0; s_sq[warp] = 1.0; s_qt[warp] = 0.0; s_u[warp] = 0.0;
        }
    }
    __syncthreads();
    pdl_wait();                                            // the target logits and their parts come from the preceding kernel
    cluster_wait();                                        // all eight CTAs of the cluster have started

    // ---- A: this CTA's target rows
    for (int i = 0; i < my_rows; ++i) {
        const int j = rank + i * kAcceptCluster;
        const bool test_row = j < k_b;
        const int x = s_x[i];
        double zp = 0.0;
        if (test_row && !p.greedy && threadIdx.x == 0) {
            zp = static_cast<double>(p.logits[static_cast<int64_t>(q0 + j) * p.vocab + x]);
            if (p.vocab_mask != nullptr && !mask_allows(p.vocab_mask + static_cast<int64_t>(b) * p.mask_words, x)) zp = -INFINITY;
        }
        const float2* tp = p.tstats + static_cast<int64_t>(q0 + j) * p.n_tparts;
        const int n = p.n_tparts;
        if (p.greedy) {
            float m = -INFINITY;
            int best = 0x7fffffff;
#pragma unroll 8
            for (int t = threadIdx.x; t < n; t += kAcceptThreads) {
                const float2 pt = __ldcg(&tp[t]);
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
                for (int w = 1; w < kAcceptWarps; ++w)
                    if (red_f[w] > m || (red_f[w] == m && red_i[w] < best)) { m = red_f[w]; best = red_i[w]; }
                s_tmp.argmax = best;
                s_tmp.rej = (test_row && x != best) ? 1 : 0;
                s_tmp.m_p = m; s_tmp.m_q = 0.f; s_tmp.s_p = 1.0; s_tmp.s_q = 1.0; s_tmp.tau = -INFINITY; s_tmp.rho = 0.f;
            }
        } else {
            float m = -INFINITY, sf = 0.f;
#pragma unroll 16
            for (int t = threadIdx.x; t < n; t += kAcceptThreads) {
                const float2 pt = __ldcg(&tp[t]);
                merge_ms(m, sf, pt.x, pt.y, cf);
            }
            // block-wide (max, sum): maxima through shared memory, then the sums rescaled to the common maximum
            const float mt = m;
            m = warp_max(m);
            if (lane == 0) red_f[warp] = m;
            __syncthreads();
#pragma unroll
            for (int w = 0; w < kAcceptWarps; ++w) m = fmaxf(m, red_f[w]);
            double sm = (mt == -INFINITY) ? 0.0 : static_cast<double>(sf) * static_cast<double>(fast_exp2((mt - m) * cf));
            sm = warp_sum(sm);
            if (lane == 0) red_d[warp] = sm;
            __syncthreads();
            if (threadIdx.x == 0) {
                sm = 0.0;
#pragma unroll
                for (int w = 0; w < kAcceptWarps; ++w) sm += red_d[w];
                double tau = -INFINITY;                   // nucleus of the target row: its lowest kept logit and its mass
                if (p.filtered) { tau = p.topp[static_cast<int64_t>(q0 + j) * 2]; sm = p.topp[static_cast<int64_t>(q0 + j) * 2 + 1]; }
                int rej = 0;
                if (test_row) {
                    const double u = s_u[i], qt = s_qt[i];
                    // the same fp32 2^x as in the statistics (the exponent itself is formed in fp64)
                    const double pt = (zp == -INFINITY || zp < tau) ? 0.0
                        : static_cast<double>(fast_exp2(static_cast<float>((zp - static_cast<double>(m)) * scale))) / sm;
                    rej = (u * qt < pt) ? 0 : 1;
                    if (p.dbg_p != nullptr) {
                        p.dbg_p[d0 + j] = pt;
                        p.dbg_q[d0 + j] = qt;
                        p.dbg_u[d0 + j] = static_cast<float>(u);
                    }
                }
                s_tmp.m_p = m; s_tmp.s_p = sm; s_tmp.tau = tau;
                s_tmp.m_q = static_cast<float>(s_mq[i]); s_tmp.s_q = s_sq[i];
                s_tmp.rho = test_row ? static_cast<float>(sm / s_sq[i]) : 0.f;
                s_tmp.rej = rej; s_tmp.argmax = 0;
            }
        }
        __syncthreads();
        if (threadIdx.x < kAcceptCluster) *cluster.map_shared_rank(&s_row[j], threadIdx.x) = s_tmp;
        __syncthreads();                                   // s_tmp and the reduction arrays are reused by the next row
    }
    cluster_sync();                                        // every row result is in every CTA's shared memory

    // ---- B: first rejection
    if (warp == 0) {
        int n = k_b;
        for (int base = 0; base < k_b; base += 32) {
            const int jj = base + lane;
            const bool rej = jj < k_b && s_row[jj].rej != 0;
            const unsigned vote = __ballot_sync(0xffffffffu, rej);
            if (vote != 0u && n == k_b) n = base + __ffs(vote) - 1;
        }
        if (lane == 0) {
            s_n = n;
            if (rank == 0) {
                p.accepted_len[b] = n;
                if (p.greedy) p.next_token[b] = s_row[n].argmax;
            }
        }
    }
    __syncthreads();
    if (p.greedy) return;                                  // uniform over the cluster; no barrier follows
    const int n = s_n;

    // ---- C: masses of row n over this CTA's slice of the vocabulary
    extern __shared__ float s_dyn[];                       // [warps][2 buffers][target | draft][kSubChunk], then the group masses
    DrawRow row;
    row.zt = p.logits + static_cast<int64_t>(q0 + n) * p.vocab;
    row.residual = (n < k_b);
    row.zd = row.residual ? p.draft_logits + static_cast<int64_t>(d0 + n) * p.vocab : nullptr;
    row.mask = (p.vocab_mask != nullptr) ? p.vocab_mask + static_cast<int64_t>(b) * p.mask_words : nullptr;
    row.mp = s_row[n].m_p;
    row.mq = row.residual ? s_row[n].m_q : 0.f;
    row.rho = row.residual ? s_row[n].rho : 0.f;
    row.tau = static_cast<float>(s_row[n].tau);
    row.plain = (row.mask == nullptr && row.tau == -INFINITY);
    row.c = cf;
    const bool vec_ok = ((p.vocab & 3) == 0);
    const int wc_total = (p.vocab + kWarpChunk - 1) / kWarpChunk;
    const int wc_per_cta = (wc_total + kAcceptCluster - 1) / kAcceptCluster;     // <= kMaxWarpChunksPerCta (vocab <= kMaxVocab)
    const int wc_begin = min(wc_total, rank * wc_per_cta);
    const int n_wc = min(wc_total, wc_begin + wc_per_cta) - wc_begin;
    float* my_buf = s_dyn + warp * (4 * kSubChunk);        // two buffers of (target, draft) sub-chunks
    float2* s_grp = reinterpret_cast<float2*>(s_dyn + kAcceptWarps * 4 * kSubChunk);   // [n_wc][kGroupsPerChunk] (residual, p) masses
    {
        // A warp streams its chunks (warp, warp + 8, ...) as sub-chunks of 512 entries through two small
        // buffers: the copy of sub-chunk s + 2 is requested as soon as s has been added up, so transfer
        // and arithmetic overlap.  Lane l adds the 16 consecutive entries [16 l, 16 l + 16) of a sub-chunk
        // (a "group"): its sum is the group's mass, the warp's sum the chunk's.
        const int n_sub = 2 * ((n_wc - warp + kAcceptWarps - 1) / kAcceptWarps);      // of this warp (0 if it has no chunk)
        auto sub_base = [&](int sidx) { return (wc_begin + warp + kAcceptWarps * (sidx >> 1)) * kWarpChunk + (sidx & 1) * kSubChunk; };
        auto issue = [&](int sidx) {
            float* dst = my_buf + (sidx & 1) * (2 * kSubChunk);
            stage_sub(dst, row.zt, sub_base(sidx), p.vocab, vec_ok, lane);
            if (row.residual) stage_sub(dst + kSubChunk, row.zd, sub_base(sidx), p.vocab, vec_ok, lane);
            cp_async_commit();
        };
        if (n_sub > 0) { issue(0); issue(1); }
        double cr = 0.0, cp = 0.0;
#pragma unroll 1
        for (int sidx = 0; sidx < n_sub; ++sidx) {
            if (sidx + 1 < n_sub) cp_async_wait_group_1(); else cp_async_wait_all();
            __syncwarp();
            const float* zt_s = my_buf + (sidx & 1) * (2 * kSubChunk);
            const float* zd_s = zt_s + kSubChunk;
            const int v0 = sub_base(sidx) + lane * kGroup;
            float mr = 0.f, mp = 0.f;
            if (row.plain && sub_base(sidx) + kSubChunk <= p.vocab) {
                // no mask, no nucleus, no ragged end: nothing depends on the entry's index, so the 16 exponentials
                // of a lane (32 with the draft's) are independent instructions the scheduler can overlap; the
                // sums are then taken in the entries' order, exactly as in the general loop below
                float ze[kGroup], zq[kGroup];
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const int pos = lane * kGroup + ((j ^ ((lane >> 1) & 3)) << 2);
                    const float4 a = *reinterpret_cast<const float4*>(zt_s + pos);
                    ze[4 * j + 0] = a.x; ze[4 * j + 1] = a.y; ze[4 * j + 2] = a.z; ze[4 * j + 3] = a.w;
                    if (row.residual) {
                        const float4 d = *reinterpret_cast<const float4*>(zd_s + pos);
                        zq[4 * j + 0] = d.x; zq[4 * j + 1] = d.y; zq[4 * j + 2] = d.z; zq[4 * j + 3] = d.w;
                    }
                }
#pragma unroll
                for (int i = 0; i < kGroup; ++i) ze[i] = fast_exp2((ze[i] - row.mp) * row.c);
                if (row.residual) {
#pragma unroll
                    for (int i = 0; i < kGroup; ++i) zq[i] = fmaxf(fmaf(-row.rho, fast_exp2((zq[i] - row.mq) * row.c), ze[i]), 0.f);
#pragma unroll
                    for (int i = 0; i < kGroup; ++i) mr += zq[i];
                }
#pragma unroll
                for (int i = 0; i < kGroup; ++i) mp += ze[i];
            } else {
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const int pos = lane * kGroup + ((j ^ ((lane >> 1) & 3)) << 2);
                    const float4 a = *reinterpret_cast<const float4*>(zt_s + pos);
                    float4 d = make_float4(0.f, 0.f, 0.f, 0.f);
                    if (row.residual) d = *reinterpret_cast<const float4*>(zd_s + pos);
                    const float za[4] = {a.x, a.y, a.z, a.w}, zq[4] = {d.x, d.y, d.z, d.w};
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const int v = v0 + 4 * j + e;
                        if (v < p.vocab) {
                            const float ep = row.e_p(za[e], v);
                            mp += ep;
                            if (row.residual) mr += fmaxf(fmaf(-row.rho, row.e_q(zq[e]), ep), 0.f);
                        }
                    }
                }
            }
            const int chunk = warp + kAcceptWarps * (sidx >> 1);
            s_grp[chunk * kGroupsPerChunk + (sidx & 1) * 32 + lane] = make_float2(mr, mp);
            cr += static_cast<double>(mr);
            cp += static_cast<double>(mp);
            __syncwarp();                                  // everyone has read the buffer
            if (sidx + 2 < n_sub) issue(sidx + 2);
            if (sidx & 1) {                                // the chunk is complete
                const double dr = warp_sum(cr), dp = warp_sum(cp);
                if (lane == 0) s_wc[chunk] = make_double2(dr, dp);
                cr = 0.0; cp = 0.0;
            }
        }
    }
    __syncthreads();
    if (warp == 0) {
        double tr = 0.0, tp = 0.0;
        for (int i = lane; i < n_wc; i += 32) { tr += s_wc[i].x; tp += s_wc[i].y; }
        tr = warp_sum(tr);
        tp = warp_sum(tp);
        if (lane < kAcceptCluster) {
            double* dst = cluster.map_shared_rank(&s_slice[0][0], lane);
            dst[rank * 2 + 0] = tr;
            dst[rank * 2 + 1] = tp;
        }
    }
    cluster_sync();                                        // slice totals are everywhere; no remote access after this
    if (warp != 0) return;

    // ---- D: which slice holds u' * Z, which chunk of it, which group of 16, which entry
    double z_r = 0.0, z_p = 0.0;
#pragma unroll
    for (int c = 0; c < kAcceptCluster; ++c) { z_r += s_slice[c][0]; z_p += s_slice[c][1]; }
    const bool use_p = !(row.residual && z_r > 0.0);      // bonus row, or a residual lost to rounding
    const double thr = s_u2[n] * (use_p ? z_p : z_r);
    // the slice that holds thr (every lane walks the eight totals itself: shorter than a shuffle scan)
    double before = 0.0;
    int slice = -1;
    {
        double run = 0.0, last_before = 0.0;
        int last_pos = -1;
#pragma unroll
        for (int c = 0; c < kAcceptCluster; ++c) {
            const double m = s_slice[c][use_p ? 1 : 0];
            if (slice < 0 && m > 0.0) {
                if (run + m > thr) { slice = c; before = run; }
                else { last_pos = c; last_before = run; }
            }
            run += m;
        }
        if (slice < 0) { slice = last_pos; before = last_before; }
    }
    if (slice < 0) {                                       // no mass anywhere (every token masked): token 0
        if (rank == 0 && lane == 0) p.next_token[b] = 0;
        return;
    }
    if (slice != rank) return;
    const int wc = max(0, warp_pick(n_wc, before, thr, lane, [&](int i) { return use_p ? s_wc[i].y : s_wc[i].x; }, before));
    const float2* grp_mass = s_grp + wc * kGroupsPerChunk;
    const int grp = max(0, warp_pick(kGroupsPerChunk, before, thr, lane, [&](int g) {
        return static_cast<double>(use_p ? grp_mass[g].y : grp_mass[g].x); }, before));
    // the group's 16 entries come from L2 once more (lane e takes entry e); same fp32 weights as above
    const int v = (wc_begin + wc) * kWarpChunk + grp * kGroup + lane;
    float w = 0.f;
    if (lane < kGroup && v < p.vocab) w = row.weight(__ldg(row.zt + v), use_p ? 0.f : __ldg(row.zd + v), v, use_p);
    const double run = before + warp_inclusive_scan(static_cast<double>(w), lane);
    const unsigned hit = __ballot_sync(0xffffffffu, w > 0.f && run > thr);
    const unsigned pos = __ballot_sync(0xffffffffu, w > 0.f);
    // if rounding left no entry above the threshold: the last entry with positive mass
    const int pick = hit != 0u ? __ffs(hit) - 1 : (pos != 0u ? 31 - __clz(pos) : 0);
    if (lane == 0) p.next_token[b] = min((wc_begin + wc) * kWarpChunk + grp * kGroup + pick, p.vocab - 1);
}

// dynamic shared memory of the acceptance kernel: the streaming buffers plus the group masses of the slice
static size_t accept_smem_bytes(int vocab)
{
    const int wc_total = (vocab + kWarpChunk - 1) / kWarpChunk;
    const int wc_per_cta = (wc_total + kAcceptCluster - 1) / kAcceptCluster;
    return static_cast<size_t>(kAcceptWarps) * 4 * kSubChunk * sizeof(float) + static_cast<size_t>(wc_per_cta) * kGroupsPerChunk * sizeof(float2);
}
constexpr size_t kAcceptSmemMax = static_cast<size_t>(kAcceptWarps) * 4 * kSubChunk * sizeof(float) +
                                  static_cast<size_t>(kMaxWarpChunksPerCta) * kGroupsPerChunk * sizeof(float2);   // 131 072

cudaError_t sample_init()
{
    cudaError_t e = cudaFuncSetAttribute(sample_accept_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         static_cast<int>(kAcceptSmemMax));
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(sample_filter_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 static_cast<int>(filter_smem_bytes(kFilterCluster * kFilterCodesMax)));
    return e;
}

cudaError_t launch_sample_accept(const SampleParams& p, bool pdl, cudaStream_t stream)
{
    return launch_kernel_ex(sample_accept_kernel, dim3(kAcceptCluster, p.batch), dim3(kAcceptThreads), accept_smem_bytes(p.vocab),
                            stream, pdl, p);
}

}  // namespace fs
