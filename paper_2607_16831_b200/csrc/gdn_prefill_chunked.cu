// Host side of the chunked WY / UT-transform prefill: workspace sizing, TMA tensor maps for
// the caller's q/k/v tensors, and the launches (chunk table, intra-chunk, chain, and the scan
// over runs of chunks when sequences are few and long).
#include <cstdlib>
#include <cstring>

#include "gdn_prefill_ws.cuh"

namespace gdn {

size_t prefill_chunked_workspace_bytes(int total_tokens, int num_seqs, int /*Hqk*/, int Hv, bool allow_split) {
    return ws_layout(total_tokens, num_seqs, Hv, allow_split).total;
}

// How many runs of chunks each sequence is cut into: as many as keep every chain CTA resident at
// once, while a run stays at least kMinSegChunks chunks long.  One run = the plain chain.
static int choose_segments(const WsLayout& L, int num_seqs, int Hv, int max_seqlen) {
    if (L.seg_cap <= 1) return 1;
    static int sms[64];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 1;
    if (!sms[dev] && cudaDeviceGetAttribute(&sms[dev], cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return 1;
    int segs = seg_cap_for((long long)num_seqs * Hv, sms[dev]);
    if (segs > L.seg_cap) segs = L.seg_cap;
    const int by_length = ((max_seqlen + kChunk - 1) / kChunk) / kMinSegChunks;
    if (segs > by_length) segs = by_length;
    // GDN_PREFILL_MAX_SEGMENTS (environment, optional) lowers the limit; 1 switches the split off
    if (const char* env = getenv("GDN_PREFILL_MAX_SEGMENTS")) {
        const int lim = atoi(env);
        if (lim >= 1 && segs > lim) segs = lim;
    }
    return segs < 1 ? 1 : segs;
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn get_encode_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

// bf16 [T][H][128] -> boxes of 64 tokens x 1 head x 64 elements, 128-byte swizzle.
static bool make_map(CUtensorMap* m, const void* base, int T, int H) {
    EncodeTiledFn fn = get_encode_fn();
    if (!fn) return false;
    cuuint64_t dims[3] = {(cuuint64_t)kD, (cuuint64_t)H, (cuuint64_t)T};
    cuuint64_t strides[2] = {(cuuint64_t)kD * 2, (cuuint64_t)H * kD * 2};
    cuuint32_t box[3] = {64, 1, 64};
    cuuint32_t estr[3] = {1, 1, 1};
    return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// fp32 states [rows][128] -> boxes of 128 rows x 32 floats (128 bytes), 128-byte swizzle.
static bool make_state_map(CUtensorMap* m, const float* base, long long rows) {
    EncodeTiledFn fn = get_encode_fn();
    if (!fn) return false;
    cuuint64_t dims[2] = {(cuuint64_t)kD, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)kD * 4};
    cuuint32_t box[2] = {32, 128};
    cuuint32_t estr[2] = {1, 1};
    return fn(m, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<float*>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

cudaError_t prefill_chunked_dispatch(const void* q, const void* k, const void* v, const float* g,
                                     const float* beta, const float* A_log, const float* dt_bias,
                                     const int32_t* cu_seqlens, const float* initial_state,
                                     void* out, float* final_state, int total_tokens, int num_seqs,
                                     int max_seqlen, int Hqk, int Hv, void* workspace, size_t /*workspace_bytes*/,
                                     bool allow_split, QkFront fr, cudaStream_t st) {
    uint8_t* ws = static_cast<uint8_t*>(workspace);
    const WsLayout L = ws_layout(total_tokens, num_seqs, Hv, allow_split);
    // with few sequences the intra-chunk kernel builds the chunk table itself (one launch less)
    const bool no_prep = total_tokens > 0 && num_seqs <= kMaxSeqsWithoutPrep;
    cudaError_t e = no_prep ? cudaSuccess : launch_prefill_prep(cu_seqlens, num_seqs, total_tokens, ws, L, st);
    if (e != cudaSuccess) return e;
    if (total_tokens > 0) {
        CUtensorMap mq, mk, mv;
        if (!make_map(&mq, q, total_tokens, Hqk) || !make_map(&mk, k, total_tokens, Hqk) ||
            !make_map(&mv, v, total_tokens, Hv))
            return cudaErrorUnknown;
        e = launch_prefill_intra(mq, mk, g, beta, A_log, dt_bias, ws, L, Hqk, Hv, no_prep ? cu_seqlens : nullptr, num_seqs,
                                 total_tokens, fr, st);
        if (e != cudaSuccess) return e;
        const int segs = choose_segments(L, num_seqs, Hv, max_seqlen);
        CUtensorMap ms;
        memset(&ms, 0, sizeof ms);
        if (initial_state && !make_state_map(&ms, initial_state, (long long)num_seqs * Hv * kD)) return cudaErrorUnknown;
        e = launch_prefill_chain(mq, mk, mv, ms, initial_state, out, final_state, ws, L, num_seqs, Hqk, Hv, segs,
                                 ChainPartial{nullptr, nullptr, nullptr}, st);
        if (e != cudaSuccess) return e;
        if (segs > 1) {
            CUtensorMap mout, mqt;
            if (!make_map(&mout, out, total_tokens, Hv) || !make_map(&mqt, ws + L.off_qt, total_tokens, Hv))
                return cudaErrorUnknown;
            e = launch_prefill_scan(mout, mqt, out, final_state, ws, L, num_seqs, max_seqlen, Hv, segs, st);
        }
        if (e != cudaSuccess) return e;
    } else if (final_state) {
        // all sequences are empty: the states pass through
        if (initial_state) {
            if (final_state != initial_state)
                cudaMemcpyAsync(final_state, initial_state, sizeof(float) * (size_t)num_seqs * Hv * kD * kD,
                                cudaMemcpyDeviceToDevice, st);
        } else {
            cudaMemsetAsync(final_state, 0, sizeof(float) * (size_t)num_seqs * Hv * kD * kD, st);
        }
    }
    return cudaGetLastError();
}

// One run of every sequence walked from the zero state and from the identity (see gdn_prefill_scan.cu).
cudaError_t prefill_partial_dispatch(const void* q, const void* k, const void* v, const float* g, const float* beta,
                                     const int32_t* cu_seqlens, void* out0, void* qt, float* H, float* P,
                                     int total_tokens, int num_seqs, int Hqk, int Hv, void* workspace,
                                     cudaStream_t st) {
    uint8_t* ws = static_cast<uint8_t*>(workspace);
    const WsLayout L = ws_layout(total_tokens, num_seqs, Hv, false);
    cudaError_t e = launch_prefill_prep(cu_seqlens, num_seqs, total_tokens, ws, L, st);
    if (e != cudaSuccess) return e;
    CUtensorMap mq, mk, mv;
    if (total_tokens > 0) {
        if (!make_map(&mq, q, total_tokens, Hqk) || !make_map(&mk, k, total_tokens, Hqk) ||
            !make_map(&mv, v, total_tokens, Hv))
            return cudaErrorUnknown;
        e = launch_prefill_intra(mq, mk, g, beta, nullptr, nullptr, ws, L, Hqk, Hv, nullptr, num_seqs, total_tokens,
                                 QkFront{1.f, 0}, st);
        if (e != cudaSuccess) return e;
    } else {
        // no tensor to describe; every sequence is empty and the chain CTAs return before using the maps
        memset(&mq, 0, sizeof mq);
        mk = mq;
        mv = mq;
    }
    return launch_prefill_chain(mq, mk, mv, mq, nullptr, out0, nullptr, ws, L, num_seqs, Hqk, Hv, 1,
                                ChainPartial{H, P, static_cast<uint16_t*>(qt)}, st);
}

cudaError_t prefill_apply_dispatch(const float* S_in, const void* qt, void* out, const int32_t* cu_seqlens,
                                   int total_tokens, int num_seqs, int max_seqlen, int Hv, void* workspace,
                                   cudaStream_t st) {
    if (total_tokens == 0) return cudaSuccess;
    CUtensorMap mout, mqt;
    if (!make_map(&mout, out, total_tokens, Hv) || !make_map(&mqt, qt, total_tokens, Hv)) return cudaErrorUnknown;
    return launch_prefill_apply(mout, mqt, S_in, out, cu_seqlens, num_seqs, max_seqlen, Hv,
                                static_cast<uint8_t*>(workspace), st);
}

}  // namespace gdn
