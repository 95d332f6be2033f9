// The steps on either side of verification that touch the per-user KV session (Section IV-C):
//   append   : "the Cloud computes the KV pairs only for these newly received tokens" -- the K/V
//              rows of the k_b + 1 window positions are written into the sequence's pages at
//              positions kv_len[b] - (k_b + 1) + j, before the verification step reads them;
//   rollback : "if a rejection occurs at index j < K, the Cloud performs a KV cache rollback,
//              discarding all invalid KV pairs from index j onward" -- with paged storage that is
//              a new length: the committed context grows by the accepted drafts plus the emitted
//              token's predecessor, kv_len_next[b] = kv_len[b] - (k_b + 1) + accepted_len[b] + 1.
#include "common.cuh"
#include "internal.h"

namespace fs {

// grid (row, K|V); block = threads over the n_kv_heads * head_dim / 8 16-byte chunks of a row
__global__ void __launch_bounds__(256)
kv_append_kernel(const KvAppendParams p)
{
    const int row = blockIdx.x;                         // packed query row: sequence b, window position j
    const int which = blockIdx.y;                       // 0 = K, 1 = V
    // sequence of the row: largest b with cu_q[b] <= row (cu_q is computed here from draft_len)
    __shared__ int s_b, s_j;
    if (threadIdx.x == 0) {
        int acc = 0, b = 0;
        for (; b < p.batch; ++b) {
            const int n = p.draft_len[b] + 1;
            if (row < acc + n) break;
            acc += n;
        }
        s_b = b; s_j = row - acc;
    }
    __syncthreads();
    const int b = s_b, j = s_j;
    if (b >= p.batch) return;
    const int k_b = p.draft_len[b];
    const int t = p.kv_len[b] - (k_b + 1) + j;          // token position in the sequence
    if (t < 0) { report_error(p.status, kErrBadPage, t, 8); return; }
    int phys = p.page_table[static_cast<int64_t>(b) * p.max_pages_per_seq + t / 16];
    if (phys < 0 || phys >= p.num_pages) { report_error(p.status, kErrBadPage, phys, 8); return; }
    const int slot = t % 16;
    const int chunks_per_head = p.head_dim / 8;
    const uint4* src = reinterpret_cast<const uint4*>(which == 0 ? p.new_k : p.new_v) +
                       static_cast<int64_t>(row) * p.n_kv_heads * chunks_per_head;
    for (int c = threadIdx.x; c < p.n_kv_heads * chunks_per_head; c += blockDim.x) {
        const int hd = c / chunks_per_head, ch = c % chunks_per_head;
        uint4* dst = reinterpret_cast<uint4*>(p.kv_pages) +
                     ((((static_cast<int64_t>(phys) * 2 + which) * p.n_kv_heads + hd) * 16 + slot) * chunks_per_head + ch);
        *dst = __ldg(src + c);
    }
}

__global__ void kv_rollback_kernel(const int32_t* __restrict__ kv_len, const int32_t* __restrict__ draft_len,
                                   const int32_t* __restrict__ accepted_len, int32_t batch, int32_t* __restrict__ kv_len_next)
{
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b < batch) kv_len_next[b] = kv_len[b] - (draft_len[b] + 1) + accepted_len[b] + 1;
}

// Page release after a rollback (Section IV-C: the invalid KV pairs are discarded).  One warp per
// sequence: the page-table entries that hold no valid token any more -- indices
// ceil(kv_len_next / 16) .. ceil(kv_len_prev / 16) - 1 -- are pushed onto a free list (one atomic
// reservation per sequence, so a sequence's pages stay together and in order) and set to -1.
__global__ void kv_release_kernel(int32_t* __restrict__ page_table, int32_t max_pages_per_seq,
                                  const int32_t* __restrict__ kv_len_prev, const int32_t* __restrict__ kv_len_next,
                                  int32_t batch, int32_t num_pages, int32_t* __restrict__ free_list, int32_t free_capacity,
                                  int32_t* __restrict__ free_count, int32_t* status)
{
    const int b = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (b >= batch) return;
    const int had = min((max(kv_len_prev[b], 0) + 15) / 16, max_pages_per_seq);
    const int keep = min((max(kv_len_next[b], 0) + 15) / 16, had);
    const int n = had - keep;
    if (n <= 0) return;
    int base = 0;
    if (lane == 0) base = atomicAdd(free_count, n);
    base = __shfl_sync(0xffffffffu, base, 0);
    for (int i = lane; i < n; i += 32) {
        int32_t* e = page_table + static_cast<int64_t>(b) * max_pages_per_seq + keep + i;
        const int phys = *e;
        if (phys < 0 || phys >= num_pages) report_error(status, kErrBadPage, phys, 9);
        if (base + i < free_capacity) free_list[base + i] = phys;
        else report_error(status, kErrInvalidArg, base + i, 9);          // the caller's list is too short
        *e = -1;
    }
}
cudaError_t launch_kv_release(int32_t* page_table, int32_t max_pages_per_seq, const int32_t* kv_len_prev,
                              const int32_t* kv_len_next, int32_t batch, int32_t num_pages, int32_t* free_list,
                              int32_t free_capacity, int32_t* free_count, int32_t* status, cudaStream_t stream)
{
    const int threads = 128;
    kv_release_kernel<<<(batch * 32 + threads - 1) / threads, threads, 0, stream>>>(
        page_table, max_pages_per_seq, kv_len_prev, kv_len_next, batch, num_pages, free_list, free_capacity, free_count, status);
    return cudaGetLastError();
}

// Diagnostic: one thread waits on a barrier on which nobody ever arrives, with the bounded wait every
// pipeline of the library uses; the wait runs out after limit_ns, the timeout lands in the status
// word and the kernel returns normally.
__global__ void wait_timeout_kernel(int32_t* status, uint64_t limit_ns)
{
    __shared__ uint64_t bar;
    if (threadIdx.x == 0) {
        mbar_init(&bar, 1);
        fence_barrier_init();
        mbar_wait_ns(&bar, 0u, status, 99, limit_ns);
    }
}
cudaError_t launch_wait_timeout(int32_t* status, uint64_t limit_ns, cudaStream_t stream)
{
    wait_timeout_kernel<<<1, 32, 0, stream>>>(status, limit_ns);
    return cudaGetLastError();
}

cudaError_t launch_kv_append(const KvAppendParams& p, int32_t m_rows, cudaStream_t stream)
{
    if (m_rows <= 0) return cudaSuccess;
    kv_append_kernel<<<dim3(m_rows, 2), 256, 0, stream>>>(p);
    return cudaGetLastError();
}

cudaError_t launch_kv_rollback(const int32_t* kv_len, const int32_t* draft_len, const int32_t* accepted_len, int32_t batch,
                               int32_t* kv_len_next, cudaStream_t stream)
{
    kv_rollback_kernel<<<(batch + 127) / 128, 128, 0, stream>>>(kv_len, draft_len, accepted_len, batch, kv_len_next);
    return cudaGetLastError();
}

}  // namespace fs
