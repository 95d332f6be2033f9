// Plan kernel: the small per-call tables the sampling stage reads.  One CTA; thread b handles
// sequence b.  Prefix sums of (k_b + 1) and k_b give the packed row offsets of the ragged batch
// (FlexSpec's channel-aware stride makes k_b differ per sequence, Section IV-B).  Draft tokens
// are range-checked here, and the device copy of the lengths is checked against the host's.
#include "common.cuh"
#include "internal.h"

namespace fs {

// inclusive scan over the block (blockDim.x <= 1024), one value per thread
__device__ __forceinline__ int block_inclusive_scan(int v, int* warp_tot)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int t = __shfl_up_sync(0xffffffffu, v, o);
        if (lane >= o) v += t;
    }
    if (lane == 31) warp_tot[warp] = v;
    __syncthreads();
    if (warp == 0) {
        int w = warp_tot[lane];
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int t = __shfl_up_sync(0xffffffffu, w, o);
            if (lane >= o) w += t;
        }
        warp_tot[lane] = w;
    }
    __syncthreads();
    const int before = (warp > 0) ? warp_tot[warp - 1] : 0;
    __syncthreads();
    return v + before;
}

// The launches of a call are sized on the host from the HOST copy of the draft lengths (m_rows,
// s_rows, k_cap = the largest k_b), while the kernels index with the DEVICE copy.  If the two
// disagree -- a length outside [0, k_cap], or totals that differ -- every later index could leave
// its array, so the call is neutralised instead: an error goes to the status word, every
// sequence is treated as k_b = 0 on row min(b, m_rows - 1), and all tables stay inside [0, m_rows).
__global__ void __launch_bounds__(kMaxBatch)
plan_kernel(const int32_t* __restrict__ draft_len, const int32_t* __restrict__ draft_tokens, int32_t batch,
            int32_t vocab, int32_t m_rows, int32_t s_rows, int32_t k_cap, const float* __restrict__ temps, float scalar_c,
            Plan plan, int32_t* status)
{
    __shared__ int warp_tot[32];
    const int t = threadIdx.x;
    const bool live = t < batch;
    const int k_raw = live ? draft_len[t] : 0;
    const int k = min(max(k_raw, 0), k_cap);
    if (t < 32) warp_tot[t] = 0;
    __syncthreads();
    const int q_end = block_inclusive_scan(live ? k + 1 : 0, warp_tot);
    const int d_end = block_inclusive_scan(k, warp_tot);
    int bad = (live && k_raw != k) ? 1 : 0;
    if (t == batch - 1 && (q_end != m_rows || d_end != s_rows)) bad = 1;
    bad = __syncthreads_or(bad);
    if (bad) {
        if (t == 0) report_error(status, kErrInvalidArg, k_raw, 7);
        if (live) {
            plan.k_eff[t] = 0;
            plan.cu_q[t] = min(t, m_rows - 1);
            plan.cu_d[t] = 0;
        }
        if (t == 0) { plan.cu_q[batch] = m_rows; plan.cu_d[batch] = 0; }
        for (int r = t; r < m_rows; r += blockDim.x) plan.row_seq[r] = 0;
        for (int r = t; r < m_rows + s_rows; r += blockDim.x) plan.row_c[r] = scalar_c;
        return;
    }
    if (live) {
        const int q0 = q_end - (k + 1), d0 = d_end - k;
        plan.k_eff[t] = k;
        plan.cu_q[t] = q0;
        plan.cu_d[t] = d0;
        // log2(e) / T of the sequence: its own temperature if given (it must be a positive finite number)
        float c = scalar_c;
        if (temps != nullptr) {
            const float tb = temps[t];
            if (tb > 0.f && tb < 3.0e38f) c = 1.4426950408889634f / tb;
            else report_error(status, kErrInvalidArg, t, 8);
        }
        for (int j = 0; j <= k; ++j) { plan.row_seq[q0 + j] = t; plan.row_c[q0 + j] = c; }
        for (int j = 0; j < k; ++j) plan.row_c[m_rows + d0 + j] = c;
        if (draft_tokens != nullptr)
            for (int j = 0; j < k; ++j) {
                const int x = draft_tokens[d0 + j];
                if (x < 0 || x >= vocab) report_error(status, kErrBadToken, x, 7);
            }
        if (t == batch - 1) {
            plan.cu_q[batch] = q_end;
            plan.cu_d[batch] = d_end;
        }
    }
}

cudaError_t launch_plan(const int32_t* draft_len, const int32_t* draft_tokens, int32_t batch, int32_t vocab,
                        int32_t m_rows, int32_t s_rows, int32_t k_cap, const float* temps, float scalar_c, Plan plan,
                        int32_t* status, cudaStream_t stream)
{
    const int threads = (batch + 31) / 32 * 32;
    plan_kernel<<<1, threads, 0, stream>>>(draft_len, draft_tokens, batch, vocab, m_rows, s_rows, k_cap, temps, scalar_c,
                                           plan, status);
    return cudaGetLastError();
}

}  // namespace fs
