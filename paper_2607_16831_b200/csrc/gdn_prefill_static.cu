// gdn_prefill_static: the chunked prefill for callers that are not allowed to allocate
// device memory.  Its scratch (the chunk table and the per-chunk T', W, P and scalar blocks)
// lives in a fixed array inside the library image instead of a caller-provided workspace.
#include "gdn_common.cuh"

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
static __device__ __align__(256) unsigned char g_static_scratch[GDN_PREFILL_STATIC_SCRATCH_BYTES];

static void* g_static_scratch_addr[64];  // per device ordinal; NULL until looked up

extern "C" int gdn_prefill_static(const void* q, const void* k, const void* v, const float* g, const float* beta,
                                  const int32_t* cu_seqlens, const float* initial_state, void* out,
                                  float* final_state, int total_tokens, int num_seqs, int max_seqlen, int Hqk,
                                  int Hv, int dk, int dv, void* stream) {
    using namespace gdn;
    if (total_tokens < 0 || num_seqs < 0 || max_seqlen < 0) return GDN_ERR_SHAPE;
    if (Hqk <= 0 || Hv <= 0 || dk <= 0 || dv <= 0 || Hv % Hqk != 0) return GDN_ERR_SHAPE;
    if (dk != kD || dv != kD) return GDN_ERR_UNSUPPORTED;
    if (max_seqlen > total_tokens) return GDN_ERR_SHAPE;
    if (total_tokens > 0 && (num_seqs == 0 || max_seqlen == 0)) return GDN_ERR_SHAPE;
    if ((long long)max_seqlen * num_seqs < total_tokens) return GDN_ERR_SHAPE;
    if (num_seqs == 0) return GDN_OK;
    if (!cu_seqlens) return GDN_ERR_NULL;
    if (total_tokens > 0 && (!q || !k || !v || !g || !beta || !out)) return GDN_ERR_NULL;
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(g) || !aligned16(beta) || !aligned16(out) ||
        !aligned16(initial_state) || !aligned16(final_state) || (reinterpret_cast<uintptr_t>(cu_seqlens) & 3u))
        return GDN_ERR_ALIGN;
    if ((long long)num_seqs * Hv * 16 > 0x7fffffffLL) return GDN_ERR_SHAPE;
    // sizes beyond the fixed scratch are refused, never truncated
    if (prefill_chunked_workspace_bytes(total_tokens, num_seqs, Hqk, Hv, false) > (size_t)GDN_PREFILL_STATIC_SCRATCH_BYTES)
        return GDN_ERR_WORKSPACE;

    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return GDN_ERR_CUDA;
    if (dev < 0 || dev >= 64) return GDN_ERR_UNSUPPORTED;
    int major = 0;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return GDN_ERR_CUDA;
    if (major != 10) return GDN_ERR_UNSUPPORTED;
    if (!g_static_scratch_addr[dev]) {
        // set-up, once per device, with that device current: translate the symbol into the address
        // the kernels can use
        void* ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess || !ptr) return GDN_ERR_CUDA;
        g_static_scratch_addr[dev] = ptr;
    }
    cudaError_t e = prefill_chunked_dispatch(q, k, v, g, beta, nullptr, nullptr, cu_seqlens, initial_state, out, final_state,
                                             total_tokens, num_seqs, max_seqlen, Hqk, Hv, g_static_scratch_addr[dev],
                                             (size_t)GDN_PREFILL_STATIC_SCRATCH_BYTES, false, QkFront{1.f, 0},
                                             (cudaStream_t)stream);
    return e == cudaSuccess ? GDN_OK : GDN_ERR_CUDA;
}
