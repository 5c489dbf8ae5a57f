// C-ABI entry points of libgdn: argument validation and launch dispatch only.
#include <cstdlib>
#include <stdio.h>
#include <stdlib.h>

#include "gdn_common.cuh"
#include "gdn_validate.h"

namespace gdn {
cudaError_t decode_dispatch(const void* q, const void* k, const void* v, const float* g, const float* beta,
                            const float* A_log, const float* dt_bias, const float* s_in, float* s_out, void* out,
                            int B, int Hqk, int Hv, int variant, QkFront fr, cudaStream_t st);
cudaError_t decode_multi_dispatch(const void* q, const void* k, const void* v, const float* g, const float* beta,
                                  const float* A_log, const float* dt_bias, const float* s_in, float* s_out, void* out,
                                  int B, int T, int Hqk, int Hv, QkFront fr, cudaStream_t st);
cudaError_t prefill_recurrent_dispatch(const void* q, const void* k, const void* v, const float* g,
                                       const float* beta, const float* A_log, const float* dt_bias,
                                       const int32_t* cu_seqlens, const float* initial_state, void* out,
                                       float* final_state, int total_tokens, int num_seqs, int Hqk, int Hv,
                                       int* status_word, QkFront fr, cudaStream_t st);
size_t prefill_chunked_workspace_bytes(int total_tokens, int num_seqs, int Hqk, int Hv, bool allow_split);
cudaError_t prefill_partial_dispatch(const void* q, const void* k, const void* v, const float* g, const float* beta,
                                     const int32_t* cu_seqlens, void* out0, void* qt, float* H, float* P,
                                     int total_tokens, int num_seqs, int Hqk, int Hv, void* workspace,
                                     cudaStream_t st);
cudaError_t prefill_apply_dispatch(const float* S_in, const void* qt, void* out, const int32_t* cu_seqlens,
                                   int total_tokens, int num_seqs, int max_seqlen, int Hv, void* workspace,
                                   cudaStream_t st);
cudaError_t launch_state_scan(const float* S0, const float* P, const float* H, int steps, float* S_out, int num_seqs,
                              int Hv, cudaStream_t st);
void* static_scratch_if_ready();
cudaError_t prefill_chunked_dispatch(const void* q, const void* k, const void* v, const float* g,
                                     const float* beta, const float* A_log, const float* dt_bias,
                                     const int32_t* cu_seqlens, const float* initial_state,
                                     void* out, float* final_state, int total_tokens, int num_seqs,
                                     int max_seqlen, int Hqk, int Hv, void* workspace, size_t workspace_bytes,
                                     bool allow_split, QkFront fr, cudaStream_t st);

// Maps a CUDA runtime error to a status; with GDN_DEBUG set in the environment the runtime's
// message goes to stderr (the only case in which the library prints).
static int cuda_status(cudaError_t e, const char* where) {
    if (e == cudaSuccess) return GDN_OK;
    if (getenv("GDN_DEBUG")) fprintf(stderr, "libgdn: %s: %s\n", where, cudaGetErrorString(e));
    return GDN_ERR_CUDA;
}

static int decode_impl(const void* q, const void* k, const void* v, const float* g, const float* beta,
                       const float* A_log, const float* dt_bias, bool gated, const float* state_in, float* state_out,
                       void* out, int B, int Hqk, int Hv, int dk, int dv, int variant, QkFront fr, void* stream) {
    if (B < 0) return GDN_ERR_SHAPE;
    if (int rc = check_heads(Hqk, Hv, dk, dv)) return rc;
    if (B == 0) return GDN_OK;
    if (!q || !k || !v || !g || !beta || !state_in || !state_out || !out) return GDN_ERR_NULL;
    if (gated && (!A_log || !dt_bias)) return GDN_ERR_NULL;
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(g) || !aligned16(beta) ||
        !aligned16(state_in) || !aligned16(state_out) || !aligned16(out) ||
        (reinterpret_cast<uintptr_t>(A_log) & 3u) || (reinterpret_cast<uintptr_t>(dt_bias) & 3u))
        return GDN_ERR_ALIGN;
    if ((long long)B * Hv * 32 > 0x7fffffffLL) return GDN_ERR_SHAPE;
    if (!device_supported()) return GDN_ERR_UNSUPPORTED;
    return cuda_status(decode_dispatch(q, k, v, g, beta, gated ? A_log : nullptr, gated ? dt_bias : nullptr, state_in,
                                       state_out, out, B, Hqk, Hv, variant, fr, (cudaStream_t)stream), "gdn_decode");
}

// Short-sequence dispatch of gdn_prefill.  When no sequence is longer than one chunk the chunked
// path pays for whole 64-token chunks and three dependent launches (about 22 us even for a few
// tokens, 12 us + 0.09 us per (sequence, head) chain beyond that), while the token-serial kernel
// costs about 0.45 us per token of the longest sequence, or 0.0052 us per token and chain once the
// chains fill the GPU.  Both models are fits to measurements on B200 over 1..64 sequences of 4..128
// tokens at 8 and 32 value heads; the faster one by the model is used.
// GDN_PREFILL_SHORT_FALLBACK=0 (environment) keeps the chunked path.
static bool prefer_token_serial(int num_seqs, int Hv, int max_seqlen) {
    if (max_seqlen > kChunk) return false;
    if (const char* env = getenv("GDN_PREFILL_SHORT_FALLBACK"))
        if (env[0] == '0') return false;
    const double chains = (double)num_seqs * Hv;
    const double per_token = 0.0052 * chains > 0.45 ? 0.0052 * chains : 0.45;
    const double t_serial = 1.3 + 0.012 * chains + per_token * max_seqlen;
    const double t_chunked = 12.0 + 0.09 * chains > 22.5 ? 12.0 + 0.09 * chains : 22.5;
    return t_serial < t_chunked;
}

}  // namespace gdn

using namespace gdn;

extern "C" {

const char* gdn_status_string(int status) {
    switch (status) {
        case GDN_OK: return "GDN_OK";
        case GDN_ERR_NULL: return "GDN_ERR_NULL: a required pointer is NULL";
        case GDN_ERR_SHAPE: return "GDN_ERR_SHAPE: inconsistent or negative sizes";
        case GDN_ERR_UNSUPPORTED: return "GDN_ERR_UNSUPPORTED: head size other than 128 or device is not sm_100";
        case GDN_ERR_WORKSPACE: return "GDN_ERR_WORKSPACE: workspace missing, too small or misaligned";
        case GDN_ERR_ALIGN: return "GDN_ERR_ALIGN: a tensor pointer is not 16-byte aligned";
        case GDN_ERR_CUDA: return "GDN_ERR_CUDA: the CUDA runtime reported an error";
        default: return "GDN_ERR_UNKNOWN";
    }
}

int gdn_decode(const void* q, const void* k, const void* v, const float* g, const float* beta,
               const float* state_in, float* state_out, void* out, int B, int Hqk, int Hv, int dk, int dv,
               void* stream) {
    return decode_impl(q, k, v, g, beta, nullptr, nullptr, false, state_in, state_out, out, B, Hqk, Hv, dk, dv, -1,
                       QkFront{1.f, 0}, stream);
}

int gdn_decode_variant(const void* q, const void* k, const void* v, const float* g, const float* beta,
                       const float* state_in, float* state_out, void* out, int B, int Hqk, int Hv, int dk, int dv,
                       int variant, void* stream) {
    if (variant < 0 || variant >= gdn_decode_num_variants()) return GDN_ERR_SHAPE;
    return decode_impl(q, k, v, g, beta, nullptr, nullptr, false, state_in, state_out, out, B, Hqk, Hv, dk, dv, variant,
                       QkFront{1.f, 0}, stream);
}

int gdn_decode_num_variants(void) { return 12; }

static int decode_multi_impl(const void* q, const void* k, const void* v, const float* g, const float* beta,
                             const float* A_log, const float* dt_bias, const float* state_in, float* state_out,
                             void* out, int B, int T, int Hqk, int Hv, int dk, int dv, QkFront fr, void* stream,
                             const char* name) {
    if (B < 0 || T < 0) return GDN_ERR_SHAPE;
    if (int rc = check_heads(Hqk, Hv, dk, dv)) return rc;
    if (B == 0) return GDN_OK;
    if (!state_in || !state_out) return GDN_ERR_NULL;
    if (T > 0 && (!q || !k || !v || !g || !beta || !out)) return GDN_ERR_NULL;
    if ((A_log == nullptr) != (dt_bias == nullptr)) return GDN_ERR_NULL;
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(g) || !aligned16(beta) ||
        !aligned16(state_in) || !aligned16(state_out) || !aligned16(out) ||
        (reinterpret_cast<uintptr_t>(A_log) & 3u) || (reinterpret_cast<uintptr_t>(dt_bias) & 3u))
        return GDN_ERR_ALIGN;
    if ((long long)B * Hv * 32 > 0x7fffffffLL || (long long)B * T > 0x7fffffffLL) return GDN_ERR_SHAPE;
    if (!device_supported()) return GDN_ERR_UNSUPPORTED;
    return cuda_status(decode_multi_dispatch(q, k, v, g, beta, A_log, dt_bias, state_in, state_out, out, B, T, Hqk, Hv,
                                             fr, (cudaStream_t)stream), name);
}

int gdn_decode_multi(const void* q, const void* k, const void* v, const float* g, const float* beta,
                     const float* state_in, float* state_out, void* out, int B, int T, int Hqk, int Hv, int dk,
                     int dv, void* stream) {
    return decode_multi_impl(q, k, v, g, beta, nullptr, nullptr, state_in, state_out, out, B, T, Hqk, Hv, dk, dv,
                             QkFront{1.f, 0}, stream, "gdn_decode_multi");
}

size_t gdn_prefill_workspace_bytes(int total_tokens, int num_seqs, int Hqk, int Hv, int dk, int dv) {
    if (total_tokens < 0 || num_seqs < 0) return 0;
    if (check_heads(Hqk, Hv, dk, dv) != GDN_OK) return 0;
    return prefill_chunked_workspace_bytes(total_tokens, num_seqs, Hqk, Hv, true);
}

int gdn_prefill(const void* q, const void* k, const void* v, const float* g, const float* beta,
                const int32_t* cu_seqlens, const float* initial_state, void* out, float* final_state,
                int total_tokens, int num_seqs, int max_seqlen, int Hqk, int Hv, int dk, int dv,
                void* workspace, size_t workspace_bytes, void* stream) {
    bool nothing = false;
    if (int rc = check_prefill(q, k, v, g, beta, cu_seqlens, initial_state, out, final_state, total_tokens,
                               num_seqs, max_seqlen, Hqk, Hv, dk, dv, &nothing))
        return rc;
    if (nothing) return GDN_OK;
    const size_t need = prefill_chunked_workspace_bytes(total_tokens, num_seqs, Hqk, Hv, true);
    if (!workspace || workspace_bytes < need || (reinterpret_cast<uintptr_t>(workspace) & 1023u))
        return GDN_ERR_WORKSPACE;
    if (prefer_token_serial(num_seqs, Hv, max_seqlen)) {
        return cuda_status(prefill_recurrent_dispatch(q, k, v, g, beta, nullptr, nullptr, cu_seqlens, initial_state,
                                                      out, final_state, total_tokens, num_seqs, Hqk, Hv,
                                                      static_cast<int*>(workspace), QkFront{1.f, 0},
                                                      (cudaStream_t)stream),
                           "gdn_prefill (token-serial)");
    }
    return cuda_status(prefill_chunked_dispatch(q, k, v, g, beta, nullptr, nullptr, cu_seqlens, initial_state, out,
                                                final_state, total_tokens, num_seqs, max_seqlen, Hqk, Hv, workspace,
                                                workspace_bytes, true, QkFront{1.f, 0}, (cudaStream_t)stream),
                       "gdn_prefill");
}

int gdn_decode_gated(const void* q, const void* k, const void* v, const float* a, const float* b, const float* A_log,
                     const float* dt_bias, const float* state_in, float* state_out, void* out, int B, int Hqk,
                     int Hv, int dk, int dv, void* stream) {
    return decode_impl(q, k, v, a, b, A_log, dt_bias, true, state_in, state_out, out, B, Hqk, Hv, dk, dv, -1,
                       QkFront{1.f, 0}, stream);
}

// scale must be finite; qk_l2norm is a flag
static bool front_ok(float scale) { return scale == scale && scale - scale == 0.f; }

int gdn_decode_fused(const void* q, const void* k, const void* v, const float* a, const float* b, const float* A_log,
                     const float* dt_bias, const float* state_in, float* state_out, void* out, int B, int Hqk,
                     int Hv, int dk, int dv, float scale, int qk_l2norm, void* stream) {
    if (!front_ok(scale)) return GDN_ERR_SHAPE;
    if (B > 0 && ((A_log == nullptr) != (dt_bias == nullptr))) return GDN_ERR_NULL;
    return decode_impl(q, k, v, a, b, A_log, dt_bias, A_log != nullptr, state_in, state_out, out, B, Hqk, Hv, dk, dv,
                       -1, QkFront{scale, qk_l2norm != 0}, stream);
}

int gdn_decode_multi_fused(const void* q, const void* k, const void* v, const float* a, const float* b,
                           const float* A_log, const float* dt_bias, const float* state_in, float* state_out,
                           void* out, int B, int T, int Hqk, int Hv, int dk, int dv, float scale, int qk_l2norm,
                           void* stream) {
    if (!front_ok(scale)) return GDN_ERR_SHAPE;
    return decode_multi_impl(q, k, v, a, b, A_log, dt_bias, state_in, state_out, out, B, T, Hqk, Hv, dk, dv,
                             QkFront{scale, qk_l2norm != 0}, stream, "gdn_decode_multi_fused");
}

// gdn_prefill_gated and gdn_prefill_fused: raw gates when A_log / dt_bias are given, and the q/k front end
static int prefill_front_impl(const void* q, const void* k, const void* v, const float* a, const float* b,
                              const float* A_log, const float* dt_bias, bool gates_required,
                              const int32_t* cu_seqlens, const float* initial_state, void* out, float* final_state,
                              int total_tokens, int num_seqs, int max_seqlen, int Hqk, int Hv, int dk, int dv,
                              QkFront fr, void* workspace, size_t workspace_bytes, void* stream, const char* name) {
    // a missing gate parameter is reported ahead of the device check, like the other host-side errors
    const bool gates_missing = gates_required ? (!A_log || !dt_bias) : ((A_log == nullptr) != (dt_bias == nullptr));
    if (gates_missing && total_tokens >= 0 && num_seqs > 0 && max_seqlen >= 0 && check_heads(Hqk, Hv, dk, dv) == GDN_OK)
        return GDN_ERR_NULL;
    bool nothing = false;
    if (int rc = check_prefill(q, k, v, a, b, cu_seqlens, initial_state, out, final_state, total_tokens, num_seqs,
                               max_seqlen, Hqk, Hv, dk, dv, &nothing))
        return rc;
    if (nothing) return GDN_OK;
    if ((reinterpret_cast<uintptr_t>(A_log) & 3u) || (reinterpret_cast<uintptr_t>(dt_bias) & 3u)) return GDN_ERR_ALIGN;
    const size_t need = prefill_chunked_workspace_bytes(total_tokens, num_seqs, Hqk, Hv, true);
    if (!workspace || workspace_bytes < need || (reinterpret_cast<uintptr_t>(workspace) & 1023u))
        return GDN_ERR_WORKSPACE;
    if (prefer_token_serial(num_seqs, Hv, max_seqlen)) {
        return cuda_status(prefill_recurrent_dispatch(q, k, v, a, b, A_log, dt_bias, cu_seqlens, initial_state, out,
                                                      final_state, total_tokens, num_seqs, Hqk, Hv,
                                                      static_cast<int*>(workspace), fr, (cudaStream_t)stream),
                           name);
    }
    return cuda_status(prefill_chunked_dispatch(q, k, v, a, b, A_log, dt_bias, cu_seqlens, initial_state, out,
                                                final_state, total_tokens, num_seqs, max_seqlen, Hqk, Hv, workspace,
                                                workspace_bytes, true, fr, (cudaStream_t)stream), name);
}

int gdn_prefill_gated(const void* q, const void* k, const void* v, const float* a, const float* b,
                      const float* A_log, const float* dt_bias, const int32_t* cu_seqlens,
                      const float* initial_state, void* out, float* final_state, int total_tokens, int num_seqs,
                      int max_seqlen, int Hqk, int Hv, int dk, int dv, void* workspace, size_t workspace_bytes,
                      void* stream) {
    return prefill_front_impl(q, k, v, a, b, A_log, dt_bias, true, cu_seqlens, initial_state, out, final_state,
                              total_tokens, num_seqs, max_seqlen, Hqk, Hv, dk, dv, QkFront{1.f, 0}, workspace,
                              workspace_bytes, stream, "gdn_prefill_gated");
}

int gdn_prefill_fused(const void* q, const void* k, const void* v, const float* a, const float* b,
                      const float* A_log, const float* dt_bias, const int32_t* cu_seqlens,
                      const float* initial_state, void* out, float* final_state, int total_tokens, int num_seqs,
                      int max_seqlen, int Hqk, int Hv, int dk, int dv, float scale, int qk_l2norm, void* workspace,
                      size_t workspace_bytes, void* stream) {
    if (!front_ok(scale)) return GDN_ERR_SHAPE;
    return prefill_front_impl(q, k, v, a, b, A_log, dt_bias, false, cu_seqlens, initial_state, out, final_state,
                              total_tokens, num_seqs, max_seqlen, Hqk, Hv, dk, dv, QkFront{scale, qk_l2norm != 0},
                              workspace, workspace_bytes, stream, "gdn_prefill_fused");
}

int gdn_prefill_recurrent(const void* q, const void* k, const void* v, const float* g, const float* beta,
                          const int32_t* cu_seqlens, const float* initial_state, void* out, float* final_state,
                          int total_tokens, int num_seqs, int max_seqlen, int Hqk, int Hv, int dk, int dv,
                          void* stream) {
    bool nothing = false;
    if (int rc = check_prefill(q, k, v, g, beta, cu_seqlens, initial_state, out, final_state, total_tokens,
                               num_seqs, max_seqlen, Hqk, Hv, dk, dv, &nothing))
        return rc;
    if (nothing) return GDN_OK;
    return cuda_status(prefill_recurrent_dispatch(q, k, v, g, beta, nullptr, nullptr, cu_seqlens, initial_state, out,
                                                  final_state, total_tokens, num_seqs, Hqk, Hv, nullptr,
                                                  QkFront{1.f, 0}, (cudaStream_t)stream),
                       "gdn_prefill_recurrent");
}

int gdn_prefill_partial(const void* q, const void* k, const void* v, const float* g, const float* beta,
                        const int32_t* cu_seqlens, void* out0, void* qt, float* H, float* P, int total_tokens,
                        int num_seqs, int max_seqlen, int Hqk, int Hv, int dk, int dv, void* workspace,
                        size_t workspace_bytes, void* stream) {
    bool nothing = false;
    if (int rc = check_prefill(q, k, v, g, beta, cu_seqlens, nullptr, out0, nullptr, total_tokens, num_seqs,
                               max_seqlen, Hqk, Hv, dk, dv, &nothing))
        return rc;
    if (nothing) return GDN_OK;
    if (!H || !P || (total_tokens > 0 && !qt)) return GDN_ERR_NULL;
    if (!aligned16(H) || !aligned16(P) || !aligned16(qt)) return GDN_ERR_ALIGN;
    const size_t need = prefill_chunked_workspace_bytes(total_tokens, num_seqs, Hqk, Hv, true);
    if (!workspace || workspace_bytes < need || (reinterpret_cast<uintptr_t>(workspace) & 1023u))
        return GDN_ERR_WORKSPACE;
    return cuda_status(prefill_partial_dispatch(q, k, v, g, beta, cu_seqlens, out0, qt, H, P, total_tokens, num_seqs,
                                                Hqk, Hv, workspace, (cudaStream_t)stream), "gdn_prefill_partial");
}

int gdn_state_scan(const float* S0, const float* P, const float* H, int steps, float* S_out, int num_seqs, int Hv,
                   int dk, int dv, void* stream) {
    if (steps < 0 || num_seqs < 0) return GDN_ERR_SHAPE;
    if (int rc = check_heads(Hv, Hv, dk, dv)) return rc;
    if (num_seqs == 0) return GDN_OK;
    if (!S_out || (steps > 0 && (!P || !H))) return GDN_ERR_NULL;
    if (!aligned16(S0) || !aligned16(P) || !aligned16(H) || !aligned16(S_out)) return GDN_ERR_ALIGN;
    if ((long long)num_seqs * Hv > 0x7fffffffLL / 16) return GDN_ERR_SHAPE;
    if (!device_supported()) return GDN_ERR_UNSUPPORTED;
    return cuda_status(launch_state_scan(S0, P, H, steps, S_out, num_seqs, Hv, (cudaStream_t)stream), "gdn_state_scan");
}

int gdn_prefill_apply(const float* S_in, const void* qt, void* out, const int32_t* cu_seqlens, int total_tokens,
                      int num_seqs, int max_seqlen, int Hv, int dk, int dv, void* workspace, size_t workspace_bytes,
                      void* stream) {
    if (total_tokens < 0 || num_seqs < 0 || max_seqlen < 0) return GDN_ERR_SHAPE;
    if (int rc = check_heads(Hv, Hv, dk, dv)) return rc;
    if (max_seqlen > total_tokens) return GDN_ERR_SHAPE;
    if (total_tokens > 0 && (num_seqs == 0 || max_seqlen == 0)) return GDN_ERR_SHAPE;
    if ((long long)max_seqlen * num_seqs < total_tokens) return GDN_ERR_SHAPE;
    if (num_seqs == 0 || total_tokens == 0) return GDN_OK;
    if (!S_in || !qt || !out || !cu_seqlens) return GDN_ERR_NULL;
    if (!aligned16(S_in) || !aligned16(qt) || !aligned16(out) || (reinterpret_cast<uintptr_t>(cu_seqlens) & 3u))
        return GDN_ERR_ALIGN;
    if (num_seqs > 65535) return GDN_ERR_SHAPE;
    if (!device_supported()) return GDN_ERR_UNSUPPORTED;
    const size_t need = 1024 + (size_t)num_seqs * Hv * 32768;
    if (!workspace || workspace_bytes < need || (reinterpret_cast<uintptr_t>(workspace) & 1023u))
        return GDN_ERR_WORKSPACE;
    return cuda_status(prefill_apply_dispatch(S_in, qt, out, cu_seqlens, total_tokens, num_seqs, max_seqlen, Hv,
                                              workspace, (cudaStream_t)stream), "gdn_prefill_apply");
}

int gdn_last_device_status(void* workspace, int* device_status, void* stream) {
    if (!device_status) return GDN_ERR_NULL;
    // NULL = the fixed scratch of gdn_prefill_static on the current device (its address is private)
    if (!workspace) workspace = static_scratch_if_ready();
    if (!workspace) return GDN_ERR_NULL;
    int val = 0;
    if (cudaMemcpyAsync(&val, workspace, sizeof(int), cudaMemcpyDeviceToHost, (cudaStream_t)stream) != cudaSuccess)
        return GDN_ERR_CUDA;
    if (cudaStreamSynchronize((cudaStream_t)stream) != cudaSuccess) return GDN_ERR_CUDA;
    *device_status = val;
    if (val != 0) {
        if (cudaMemsetAsync(workspace, 0, sizeof(int), (cudaStream_t)stream) != cudaSuccess) return GDN_ERR_CUDA;
    }
    return GDN_OK;
}

}  // extern "C"
