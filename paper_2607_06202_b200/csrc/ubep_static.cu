// ubep_get_dispatch_layout_static: the counts-only step for callers that cannot give the
// library any device memory of their own beyond inputs and outputs -- no arena, no buffer
// handle.  The per-chunk histograms and the completion ticket of the counting kernel live
// in a fixed array inside this library's device image instead.
#include <cstdint>

#include "../../include/ubep.h"
#include "ubep_kernels.h"

namespace {

// Scratch held by every GPU that loads the library, until the process exits:
// kStaticChunks * kStaticBins histogram words, one ticket word, one status word (~257 KB).
constexpr int kStaticChunks = 64;
constexpr int kStaticBins = UBEP_STATIC_MAX_BINS;
constexpr int kStaticWords = kStaticChunks * kStaticBins + 64;
static __device__ __align__(256) int32_t g_static_scratch[kStaticWords];

// Device address of g_static_scratch per device ordinal.  In host code the array's name is
// only a stand-in for the symbol, so the address the kernel gets comes from
// cudaGetSymbolAddress, asked once per device with that device current.
constexpr int kMaxDevices = 64;
int32_t* g_scratch_addr[kMaxDevices] = {};

int scratch_for_current_device(int32_t** out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return UBEP_ERR_CUDA;
    if (g_scratch_addr[dev] == nullptr) {
        void* ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess || ptr == nullptr) return UBEP_ERR_CUDA;
        g_scratch_addr[dev] = static_cast<int32_t*>(ptr);
    }
    *out = g_scratch_addr[dev];
    return UBEP_OK;
}

}  // namespace

extern "C" int ubep_get_dispatch_layout_static(const int32_t* topk_idx, int32_t T, int32_t topk, int32_t num_experts,
                                               int32_t num_ranks, int32_t* num_tokens_per_rank,
                                               int32_t* num_tokens_per_expert, uint8_t* is_token_in_rank,
                                               void* cuda_stream) {
    if (T < 0 || topk < 1 || topk > ubep::kMaxTopk || num_ranks < 1 || num_experts < 1) return UBEP_ERR_ARG;
    if (num_experts % num_ranks != 0 || num_experts > 65535) return UBEP_ERR_ARG;
    if (num_experts + num_ranks > kStaticBins) return UBEP_ERR_ARG;   // beyond the fixed scratch
    if ((int64_t)T * topk > INT32_MAX || (T > 0 && topk_idx == nullptr)) return UBEP_ERR_ARG;
    if ((reinterpret_cast<uintptr_t>(topk_idx) & 15u) != 0) return UBEP_ERR_ARG;
    int32_t* scratch = nullptr;
    const int rc = scratch_for_current_device(&scratch);
    if (rc != UBEP_OK) return rc;
    ubep::Params p{};
    p.T = T; p.k = topk; p.E = num_experts; p.R = num_ranks; p.L = num_experts / num_ranks;
    p.B = num_experts + num_ranks;
    p.nchunks = kStaticChunks;
    p.topk_idx = topk_idx;
    p.status = scratch + kStaticChunks * kStaticBins + 32;   // ids out of range are skipped; code kept here
    unsigned* ticket = reinterpret_cast<unsigned*>(scratch + kStaticChunks * kStaticBins);
    // The kernel writes every histogram word it later reads and re-arms the ticket (back to
    // zero) when its last CTA finishes, so nothing has to be cleared between calls.
    const cudaError_t e = ubep::launch_layout(p, num_tokens_per_rank, num_tokens_per_expert, is_token_in_rank, scratch,
                                              ticket, static_cast<cudaStream_t>(cuda_stream));
    return e == cudaSuccess ? UBEP_OK : UBEP_ERR_CUDA;
}
