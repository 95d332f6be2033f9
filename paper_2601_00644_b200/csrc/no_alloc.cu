// flexspec_sample_static: the acceptance / emitted-token stage for callers that must not allocate.
// Its working memory is one fixed array that is part of the loaded library image on every GPU,
// so the call needs neither a handle nor any allocation; see include/flexspec.h.
#include <string.h>

#include "internal.h"

using namespace fs;

namespace {

constexpr int kStaticMaxBatch = 64;
constexpr int kStaticMaxRows = 1024;                 // M = sum_b (k_b + 1)
constexpr int kStaticMaxVocab = 131072;
constexpr int kStaticChunks = (kStaticMaxVocab + kSampleChunk - 1) / kSampleChunk;       // 16

constexpr size_t align256(size_t x) { return (x + 255) & ~static_cast<size_t>(255); }

// layout of the scratch array (every piece 256-byte aligned): 276 224 bytes in all
constexpr size_t kOffStatus = 0;                                                          // int32[4]
constexpr size_t kOffCuQ = kOffStatus + 256;                                              // int32[batch + 1]
constexpr size_t kOffCuD = kOffCuQ + align256(sizeof(int32_t) * (kStaticMaxBatch + 1));
constexpr size_t kOffKEff = kOffCuD + align256(sizeof(int32_t) * (kStaticMaxBatch + 1));   // int32[batch]
constexpr size_t kOffRowSeq = kOffKEff + align256(sizeof(int32_t) * kStaticMaxBatch);      // int32[rows]
constexpr size_t kOffRowC = kOffRowSeq + align256(sizeof(int32_t) * kStaticMaxRows);       // float[2 * rows]
constexpr size_t kOffStats = kOffRowC + align256(sizeof(float) * 2 * kStaticMaxRows);      // float2[2 * rows][chunks]
constexpr size_t kScratchBytes = kOffStats + align256(sizeof(float2) * 2 * kStaticMaxRows * kStaticChunks);

// In host code this name is only a handle for the runtime: the device address comes from
// cudaGetSymbolAddress (below), once per device.
static __device__ __align__(256) unsigned char g_sample_scratch[kScratchBytes];

constexpr int kMaxDevices = 64;
unsigned char* g_scratch_ptr[kMaxDevices];           // device address of the array, per device ordinal

}  // namespace

extern "C" int flexspec_sample_static(const float* logits, const int32_t* draft_tokens, const float* draft_logits,
                                      const int32_t* draft_len, const int32_t* draft_len_host, const uint64_t* seeds,
                                      int32_t batch, int32_t vocab, int32_t mode, float temperature,
                                      const uint32_t* vocab_mask, int32_t* accepted_len, int32_t* next_token,
                                      void* stream)
{
    if (logits == nullptr || draft_len == nullptr || draft_len_host == nullptr || accepted_len == nullptr ||
        next_token == nullptr)
        return FLEXSPEC_ERR_INVALID_ARG;
    if (mode != FLEXSPEC_MODE_SAMPLE && mode != FLEXSPEC_MODE_GREEDY) return FLEXSPEC_ERR_INVALID_ARG;
    if (!(temperature >= 0.f) || temperature > 3.0e38f) return FLEXSPEC_ERR_INVALID_ARG;
    if (batch < 1 || vocab < 1) return FLEXSPEC_ERR_INVALID_ARG;
    // sizes beyond what the fixed array was laid out for
    if (batch > kStaticMaxBatch || vocab > kStaticMaxVocab) return FLEXSPEC_ERR_UNSUPPORTED;
    int32_t m_rows = 0, s_rows = 0, k_batch_max = 0;
    for (int b = 0; b < batch; ++b) {
        const int k = draft_len_host[b];
        if (k < 0 || k > kMaxK) return FLEXSPEC_ERR_INVALID_ARG;
        if (k > k_batch_max) k_batch_max = k;
        m_rows += k + 1;
        s_rows += k;
    }
    if (m_rows > kStaticMaxRows) return FLEXSPEC_ERR_UNSUPPORTED;
    const bool greedy = (mode == FLEXSPEC_MODE_GREEDY || temperature == 0.f);
    if (s_rows > 0 && draft_tokens == nullptr) return FLEXSPEC_ERR_INVALID_ARG;
    if (!greedy && (seeds == nullptr || (s_rows > 0 && draft_logits == nullptr))) return FLEXSPEC_ERR_INVALID_ARG;
    // the kernels read logit rows with 16-byte loads when vocab is a multiple of four
    const uintptr_t align_mask = (vocab & 3) == 0 ? 15u : 3u;
    if (((reinterpret_cast<uintptr_t>(logits) | reinterpret_cast<uintptr_t>(draft_logits)) & align_mask) != 0)
        return FLEXSPEC_ERR_INVALID_ARG;

    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return FLEXSPEC_ERR_NO_DEVICE; }
    if (dev < 0 || dev >= kMaxDevices) return FLEXSPEC_ERR_UNSUPPORTED;
    if (g_scratch_ptr[dev] == nullptr) {
        // first call on this device: look the array's device address up
        void* ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_sample_scratch) != cudaSuccess || ptr == nullptr) {
            cudaGetLastError();
            return FLEXSPEC_ERR_CUDA;
        }
        if (sample_init() != cudaSuccess) { cudaGetLastError(); return FLEXSPEC_ERR_CUDA; }   // a function attribute, no allocation
        g_scratch_ptr[dev] = static_cast<unsigned char*>(ptr);
    }
    unsigned char* base = g_scratch_ptr[dev];
    cudaStream_t s = static_cast<cudaStream_t>(stream);

    // the array keeps whatever the previous call left: the status word must start at zero (the
    // tables and statistics behind it are fully rewritten by this call's kernels before they are read)
    if (cudaMemsetAsync(base + kOffStatus, 0, kOffCuQ - kOffStatus, s) != cudaSuccess) {
        cudaGetLastError();
        return FLEXSPEC_ERR_CUDA;
    }

    int32_t* status = reinterpret_cast<int32_t*>(base + kOffStatus);
    Plan plan;
    plan.cu_q = reinterpret_cast<int32_t*>(base + kOffCuQ);
    plan.cu_d = reinterpret_cast<int32_t*>(base + kOffCuD);
    plan.k_eff = reinterpret_cast<int32_t*>(base + kOffKEff);
    plan.row_seq = reinterpret_cast<int32_t*>(base + kOffRowSeq);
    plan.row_c = reinterpret_cast<float*>(base + kOffRowC);
    const float scalar_c = greedy ? 1.f : static_cast<float>(1.4426950408889634 / static_cast<double>(temperature));
    if (launch_plan(draft_len, draft_tokens, batch, vocab, m_rows, s_rows, k_batch_max, nullptr, scalar_c, plan, status,
                    s) != cudaSuccess)
        return FLEXSPEC_ERR_CUDA;

    SampleParams p;
    memset(&p, 0, sizeof(p));
    p.greedy = greedy ? 1 : 0;
    p.logits = logits; p.draft_logits = draft_logits; p.draft_tokens = draft_tokens;
    p.draft_len = draft_len; p.seeds = seeds; p.vocab_mask = vocab_mask;
    p.cu_q = plan.cu_q; p.cu_d = plan.cu_d; p.row_seq = plan.row_seq; p.k_eff = plan.k_eff;
    p.batch = batch; p.vocab = vocab; p.m_rows = m_rows; p.s_rows = s_rows;
    p.n_chunks = (vocab + kSampleChunk - 1) / kSampleChunk;
    p.mask_words = (vocab + 31) / 32;
    p.inv_temp_log2 = scalar_c;
    p.row_c = plan.row_c; p.temps = nullptr; p.top_k = 0; p.filtered = 0;
    p.stats = reinterpret_cast<float2*>(base + kOffStats);
    p.tstats = p.stats; p.n_tparts = p.n_chunks;
    p.top_p = 1.f; p.topp = nullptr;
    p.accepted_len = accepted_len; p.next_token = next_token;
    p.status = status;
    if (launch_sample_stats(p, 0, greedy ? m_rows : m_rows + s_rows, s) != cudaSuccess) return FLEXSPEC_ERR_CUDA;
    if (launch_sample_accept(p, false, s) != cudaSuccess) return FLEXSPEC_ERR_CUDA;
    return FLEXSPEC_OK;
}
