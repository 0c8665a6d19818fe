// bs_softmax_verify_noalloc: bs_softmax_verify for callers that cannot hand the library a
// workspace because they cannot allocate device memory at the point of the call -- code running
// inside a serving loop whose memory pool is fixed up front, plugins that are only given their
// input and output buffers, or call sites where cudaMalloc is forbidden because it synchronises
// the device.  The scratch memory is a fixed array inside the library image instead.
//
// The array lives on every GPU that loads the library, for the life of the process, and is shared
// by all calls: two calls that run at the same time on one GPU would trample each other's row
// partials and arrival counters.
#include <atomic>
#include "bs_common.cuh"

namespace bs {

// Scratch of the statistics kernel: arrival counters, status words, row statistics and
// per-segment partials, laid out by workspace_layout().
static __device__ __align__(256) unsigned char g_noalloc_scratch[BS_NOALLOC_SCRATCH_BYTES];

// Device address of the array, per device.  In host code `g_noalloc_scratch` is only a handle of
// the symbol: the address a kernel can use has to be asked for, with the device current.
static std::atomic<void*> g_scratch_ptr[64];

static bs_status scratch_address(void** out) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return cuda_status(e);
    if (dev < 0 || dev >= 64) return BS_ERR_UNSUPPORTED;
    if (!g_scratch_ptr[dev]) {
        void* ptr = nullptr;
        e = cudaGetSymbolAddress(&ptr, g_noalloc_scratch);
        if (e != cudaSuccess) return cuda_status(e);
        g_scratch_ptr[dev] = ptr;
    }
    *out = g_scratch_ptr[dev];
    return BS_OK;
}

}  // namespace bs

using namespace bs;

extern "C" bs_status bs_softmax_verify_noalloc(const void* target_logits, const void* draft_logits, bs_dtype dtype,
                                               const int32_t* draft_tokens, const int32_t* gamma,
                                               const float* u_accept, float temperature, int B, int Gmax, int V,
                                               int32_t* accept_len, float* p_tok, float* q_tok, void* stream) {
    if (B < 1 || Gmax < 0 || V < 1) return BS_ERR_INVALID_ARG;
    if (B > BS_MAX_BATCH || Gmax > BS_MAX_GAMMA || V > BS_MAX_VOCAB) return BS_ERR_UNSUPPORTED;
    const Workspace w = workspace_layout(B, Gmax, V);
    if (w.total > (size_t)BS_NOALLOC_SCRATCH_BYTES) return BS_ERR_WORKSPACE;   // beyond the built-in scratch
    void* scratch = nullptr;
    const bs_status s = scratch_address(&scratch);
    if (s != BS_OK) return s;
    // The array keeps whatever the last call left.  Everything the kernels read before writing
    // (arrival counters, status and abort words) sits in front of the row statistics: clear it.
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const cudaError_t e = cudaMemsetAsync(scratch, 0, w.off_row_stats, st);
    if (e != cudaSuccess) return cuda_status(e);
    return bs_softmax_verify(target_logits, draft_logits, dtype, draft_tokens, gamma, u_accept, temperature,
                             B, Gmax, V, accept_len, p_tok, q_tok, scratch, w.total, stream);
}
