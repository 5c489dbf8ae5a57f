// gdn_prefill_static: the chunked prefill for callers that are not allowed to allocate
// device memory.  Its scratch (the chunk table and the per-chunk T', W, P and scalar blocks)
// lives in a fixed array inside the library image instead of a caller-provided workspace.
#include "gdn_common.cuh"
#include "gdn_validate.h"

namespace gdn {
size_t prefill_chunked_workspace_bytes(int total_tokens, int num_seqs, int Hqk, int Hv, bool allow_split);
cudaError_t prefill_chunked_dispatch(const void* q, const void* k, const void* v, const float* g,
                                     const float* beta, const float* A_log, const float* dt_bias,
                                     const int32_t* cu_seqlens, const float* initial_state,
                                     void* out, float* final_state, int total_tokens, int num_seqs,
                                     int max_seqlen, int Hqk, int Hv, void* workspace, size_t workspace_bytes,
                                     bool allow_split, QkFront fr, cudaStream_t st);
}  // namespace gdn

// The scratch itself.  Every device that loads the library carries these bytes until the
// process exits.  In host code this name is only a stand-in for the symbol: the device
// address has to be looked up (once per device) before a kernel can be given it.
// The kernels are handed a 1024-byte aligned workspace like the one every other prefill entry
// point insists on, so the array carries 768 spare bytes and the looked-up address is rounded up.
constexpr size_t kStaticAlign = 1024;
static __device__ __align__(256) unsigned char g_static_scratch[GDN_PREFILL_STATIC_SCRATCH_BYTES + kStaticAlign - 256];

static void* g_static_scratch_addr[64];  // per device ordinal, rounded up to 1024 bytes; NULL until looked up

namespace gdn {
// The scratch of the current device if gdn_prefill_static has run on it, else NULL (no look-up here).
void* static_scratch_if_ready() {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    return g_static_scratch_addr[dev];
}
}  // namespace gdn

extern "C" int gdn_prefill_static(const void* q, const void* k, const void* v, const float* g, const float* beta,
                                  const int32_t* cu_seqlens, const float* initial_state, void* out,
                                  float* final_state, int total_tokens, int num_seqs, int max_seqlen, int Hqk,
                                  int Hv, int dk, int dv, void* stream) {
    using namespace gdn;
    bool nothing = false;
    if (int rc = check_prefill(q, k, v, g, beta, cu_seqlens, initial_state, out, final_state, total_tokens, num_seqs,
                               max_seqlen, Hqk, Hv, dk, dv, &nothing))
        return rc;
    if (nothing) return GDN_OK;
    // sizes beyond the fixed scratch are refused, never truncated
    if (prefill_chunked_workspace_bytes(total_tokens, num_seqs, Hqk, Hv, false) > (size_t)GDN_PREFILL_STATIC_SCRATCH_BYTES)
        return GDN_ERR_WORKSPACE;

    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return GDN_ERR_CUDA;
    if (dev < 0 || dev >= 64) return GDN_ERR_UNSUPPORTED;
    if (!g_static_scratch_addr[dev]) {
        // set-up, once per device, with that device current: translate the symbol into the address
        // the kernels can use
        void* ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess || !ptr) return GDN_ERR_CUDA;
        const uintptr_t a = (reinterpret_cast<uintptr_t>(ptr) + kStaticAlign - 1) & ~(uintptr_t)(kStaticAlign - 1);
        g_static_scratch_addr[dev] = reinterpret_cast<void*>(a);
    }
    cudaError_t e = prefill_chunked_dispatch(q, k, v, g, beta, nullptr, nullptr, cu_seqlens, initial_state, out, final_state,
                                             total_tokens, num_seqs, max_seqlen, Hqk, Hv, g_static_scratch_addr[dev],
                                             (size_t)GDN_PREFILL_STATIC_SCRATCH_BYTES, false, QkFront{1.f, 0},
                                             (cudaStream_t)stream);
    return e == cudaSuccess ? GDN_OK : GDN_ERR_CUDA;
}
