// Host-side argument validation shared by the entry points of libgdn (internal).
#pragma once
#include "gdn_common.cuh"

namespace gdn {

// Is the current device of the sm_100 family?  The answer is looked up once per device ordinal.
inline bool device_supported() {
    static int ok[64];  // 0 = not looked up yet, 1 = sm_100 family, 2 = something else
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return false;
    if (dev < 0 || dev >= 64) return false;
    if (ok[dev] == 0) {
        int major = 0;
        if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return false;
        ok[dev] = (major == 10) ? 1 : 2;
    }
    return ok[dev] == 1;
}

inline int check_heads(int Hqk, int Hv, int dk, int dv) {
    if (Hqk <= 0 || Hv <= 0 || dk <= 0 || dv <= 0) return GDN_ERR_SHAPE;
    if (Hv % Hqk != 0) return GDN_ERR_SHAPE;
    if (dk != kD || dv != kD) return GDN_ERR_UNSUPPORTED;
    return GDN_OK;
}

// Everything gdn_prefill and its variants check before they look at the workspace.
// *nothing_to_do: valid arguments that describe no work (no sequences).
inline int check_prefill(const void* q, const void* k, const void* v, const float* g, const float* beta,
                         const int32_t* cu_seqlens, const float* initial_state, void* out, float* final_state,
                         int total_tokens, int num_seqs, int max_seqlen, int Hqk, int Hv, int dk, int dv,
                         bool* nothing_to_do) {
    *nothing_to_do = false;
    if (total_tokens < 0 || num_seqs < 0 || max_seqlen < 0) return GDN_ERR_SHAPE;
    if (int rc = check_heads(Hqk, Hv, dk, dv)) return rc;
    if (max_seqlen > total_tokens) return GDN_ERR_SHAPE;
    if (total_tokens > 0 && (num_seqs == 0 || max_seqlen == 0)) return GDN_ERR_SHAPE;
    if ((long long)max_seqlen * num_seqs < total_tokens) return GDN_ERR_SHAPE;
    if (num_seqs == 0) { *nothing_to_do = true; return GDN_OK; }
    if (!cu_seqlens) return GDN_ERR_NULL;
    if (total_tokens > 0 && (!q || !k || !v || !g || !beta || !out)) return GDN_ERR_NULL;
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(g) || !aligned16(beta) ||
        !aligned16(out) || !aligned16(initial_state) || !aligned16(final_state) ||
        (reinterpret_cast<uintptr_t>(cu_seqlens) & 3u))
        return GDN_ERR_ALIGN;
    if ((long long)num_seqs * Hv * 16 > 0x7fffffffLL) return GDN_ERR_SHAPE;
    if (!device_supported()) return GDN_ERR_UNSUPPORTED;
    return GDN_OK;
}

}  // namespace gdn
