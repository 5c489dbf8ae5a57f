// Token-serial prefill: the per-token recurrence of Section 3.2 with the state rows
// resident in registers for the whole sequence and the V dimension split over warps
// and CTAs (the shape of the paper's own prefill kernel).  It is the short-sequence
// path and the on-device cross-check of the chunked kernels; it uses no tensor cores
// because one token exposes no dense contraction.
//
// Lane mapping as in the decode kernel: eight lanes own one state row (four float4
// each), a warp owns 4*NB rows, dot products reduce inside the 8-lane group.
#include "gdn_common.cuh"

namespace gdn {

struct TokenRegs {
    uint2 kw[4], qw[4];
    float g, beta;
};

// FRONT: the gated / fused entry points (raw gate inputs when A_log is given, q/k front end `fr`)
template <int NB, int WARPS, bool FRONT>
__global__ void __launch_bounds__(WARPS * 32)
gdn_prefill_recurrent_kernel(const uint16_t* __restrict__ q, const uint16_t* __restrict__ k,
                             const uint16_t* __restrict__ v, const float* __restrict__ g,
                             const float* __restrict__ beta, const float* __restrict__ A_log,
                             const float* __restrict__ dt_bias, const int32_t* __restrict__ cu_seqlens,
                             const float* initial_state, uint16_t* __restrict__ out, float* final_state,
                             int total_tokens, int Hqk, int Hv, int split, int* status_word, QkFront fr) {
    // standing in for the chunked kernels: clear the workspace's device status word as they would
    if (status_word && blockIdx.x == 0 && threadIdx.x == 0) *status_word = 0;
    const int part = blockIdx.x % split;
    const int h = (blockIdx.x / split) % Hv;
    const int n = blockIdx.x / split / Hv;
    const int hq = h / (Hv / Hqk);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int sub = lane >> 3, c = lane & 7;
    const int row0 = (part * WARPS + warp) * (4 * NB);

    int t0 = cu_seqlens[n], t1 = cu_seqlens[n + 1];
    t0 = max(0, min(t0, total_tokens));
    t1 = max(t0, min(t1, total_tokens));

    // with A_log given, g / beta hold the raw gate inputs a and b
    const float A_h = (FRONT && A_log) ? __ldg(A_log + h) : 0.f, dtb_h = (FRONT && A_log) ? __ldg(dt_bias + h) : 0.f;

    const size_t sbase = ((size_t)n * Hv + h) * kD * kD;
    float4 s[NB][4];
#pragma unroll
    for (int i = 0; i < NB; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            if (initial_state)
                s[i][j] = *reinterpret_cast<const float4*>(initial_state + sbase +
                                                           (size_t)(row0 + i * 4 + sub) * kD + 4 * (c + 8 * j));
            else
                s[i][j] = make_float4(0.f, 0.f, 0.f, 0.f);
        }

    auto load_token = [&](int t, TokenRegs& r, float (&vr)[NB]) {
        const uint2* k4 = reinterpret_cast<const uint2*>(k + ((size_t)t * Hqk + hq) * kD);
        const uint2* q4 = reinterpret_cast<const uint2*>(q + ((size_t)t * Hqk + hq) * kD);
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            r.kw[j] = __ldg(k4 + c + 8 * j);
            r.qw[j] = __ldg(q4 + c + 8 * j);
        }
        r.g = __ldg(g + (size_t)t * Hv + h);
        r.beta = __ldg(beta + (size_t)t * Hv + h);
#pragma unroll
        for (int i = 0; i < NB; ++i) vr[i] = bf16_bits_to_float(__ldg(v + ((size_t)t * Hv + h) * kD + row0 + i * 4 + sub));
    };

    TokenRegs cur, nxt;
    float vcur[NB], vnxt[NB];
    if (t0 < t1) load_token(t0, cur, vcur);
    for (int t = t0; t < t1; ++t) {
        if (t + 1 < t1) load_token(t + 1, nxt, vnxt);
        float kf[16], qf[16];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            unpack_bf16x2(cur.kw[j].x, kf[4 * j + 0], kf[4 * j + 1]);
            unpack_bf16x2(cur.kw[j].y, kf[4 * j + 2], kf[4 * j + 3]);
            unpack_bf16x2(cur.qw[j].x, qf[4 * j + 0], qf[4 * j + 1]);
            unpack_bf16x2(cur.qw[j].y, qf[4 * j + 2], qf[4 * j + 3]);
        }
        float gl = cur.g, bt = cur.beta;
        if (FRONT && A_log) raw_gates(gl, bt, A_h, dtb_h, gl, bt);
        const float alpha = __expf(gl);
        float qk = 0.f;
#pragma unroll
        for (int j = 0; j < 16; ++j) qk = fmaf(qf[j], kf[j], qk);
#pragma unroll
        for (int m = 1; m < 8; m <<= 1) qk += __shfl_xor_sync(0xffffffffu, qk, m);
        // front end: k and q enter through the factors rk = 1/|k| and rq = scale/|q| (1 and 1 without it)
        float rk = 1.f, rq = FRONT ? fr.scale : 1.f;
        if (FRONT && fr.l2norm) {
            float kk = 0.f, qq = 0.f;
#pragma unroll
            for (int j = 0; j < 16; ++j) {
                kk = fmaf(kf[j], kf[j], kk);
                qq = fmaf(qf[j], qf[j], qq);
            }
#pragma unroll
            for (int m = 1; m < 8; m <<= 1) {
                kk += __shfl_xor_sync(0xffffffffu, kk, m);
                qq += __shfl_xor_sync(0xffffffffu, qq, m);
            }
            rk = rsqrtf(kk + kNormEps);
            rq *= rsqrtf(qq + kNormEps);
        }
        if (FRONT) qk *= rk * rq;

#pragma unroll
        for (int i = 0; i < NB; ++i) {
            float a = 0.f, p = 0.f;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                a = fmaf(s[i][j].x, kf[4 * j + 0], a);
                a = fmaf(s[i][j].y, kf[4 * j + 1], a);
                a = fmaf(s[i][j].z, kf[4 * j + 2], a);
                a = fmaf(s[i][j].w, kf[4 * j + 3], a);
                p = fmaf(s[i][j].x, qf[4 * j + 0], p);
                p = fmaf(s[i][j].y, qf[4 * j + 1], p);
                p = fmaf(s[i][j].z, qf[4 * j + 2], p);
                p = fmaf(s[i][j].w, qf[4 * j + 3], p);
            }
#pragma unroll
            for (int m = 1; m < 8; m <<= 1) {
                a += __shfl_xor_sync(0xffffffffu, a, m);
                p += __shfl_xor_sync(0xffffffffu, p, m);
            }
            const float delta = bt * (vcur[i] - alpha * (FRONT ? a * rk : a));
            const float dk = FRONT ? delta * rk : delta;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                s[i][j].x = fmaf(alpha, s[i][j].x, dk * kf[4 * j + 0]);
                s[i][j].y = fmaf(alpha, s[i][j].y, dk * kf[4 * j + 1]);
                s[i][j].z = fmaf(alpha, s[i][j].z, dk * kf[4 * j + 2]);
                s[i][j].w = fmaf(alpha, s[i][j].w, dk * kf[4 * j + 3]);
            }
            if (c == 0) out[((size_t)t * Hv + h) * kD + row0 + i * 4 + sub] = float_to_bf16_bits(fmaf(delta, qk, alpha * (FRONT ? p * rq : p)));
        }
        cur = nxt;
#pragma unroll
        for (int i = 0; i < NB; ++i) vcur[i] = vnxt[i];
    }

    if (final_state) {
#pragma unroll
        for (int i = 0; i < NB; ++i)
#pragma unroll
            for (int j = 0; j < 4; ++j)
                *reinterpret_cast<float4*>(final_state + sbase + (size_t)(row0 + i * 4 + sub) * kD + 4 * (c + 8 * j)) = s[i][j];
    }
}

template <int NB, int WARPS>
static cudaError_t launch_recurrent(const void* q, const void* k, const void* v, const float* g, const float* beta,
                                    const float* A_log, const float* dt_bias, const int32_t* cu_seqlens,
                                    const float* initial_state, void* out, float* final_state, int total_tokens,
                                    int num_seqs, int Hqk, int Hv, int* status_word, QkFront fr, cudaStream_t st) {
    constexpr int split = kD / (WARPS * 4 * NB);
    const unsigned grid = (unsigned)((long long)split * Hv * num_seqs);
    if (A_log || fr.active())
        gdn_prefill_recurrent_kernel<NB, WARPS, true><<<grid, WARPS * 32, 0, st>>>(
            (const uint16_t*)q, (const uint16_t*)k, (const uint16_t*)v, g, beta, A_log, dt_bias, cu_seqlens,
            initial_state, (uint16_t*)out, final_state, total_tokens, Hqk, Hv, split, status_word, fr);
    else
        gdn_prefill_recurrent_kernel<NB, WARPS, false><<<grid, WARPS * 32, 0, st>>>(
            (const uint16_t*)q, (const uint16_t*)k, (const uint16_t*)v, g, beta, A_log, dt_bias, cu_seqlens,
            initial_state, (uint16_t*)out, final_state, total_tokens, Hqk, Hv, split, status_word, fr);
    return cudaGetLastError();
}

cudaError_t prefill_recurrent_dispatch(const void* q, const void* k, const void* v, const float* g,
                                       const float* beta, const float* A_log, const float* dt_bias,
                                       const int32_t* cu_seqlens, const float* initial_state, void* out,
                                       float* final_state, int total_tokens, int num_seqs, int Hqk, int Hv,
                                       int* status_word, QkFront fr, cudaStream_t st) {
    // Launch shape by the number of (sequence, head) chains, from a sweep on B200 (1-64 sequences of
    // 8 and 32 tokens, 8 and 32 value heads): few chains want many small warps' worth of rows each
    // (the token loop is latency-bound: fewer rows per warp = a shorter loop body); once the chains
    // fill the GPU the loop is bound by instruction issue and sixteen rows per warp amortise the
    // per-token work that does not depend on the row count (15-20 % faster than eight rows);
    // everything between, four warps of 8 rows.
#define GDN_REC_ARGS q, k, v, g, beta, A_log, dt_bias, cu_seqlens, initial_state, out, final_state, total_tokens, num_seqs, Hqk, Hv, status_word, fr, st
    const long long chains = (long long)num_seqs * Hv;
    if (chains <= 16) return launch_recurrent<1, 2>(GDN_REC_ARGS);
    if (chains >= 128) return launch_recurrent<4, 1>(GDN_REC_ARGS);
    return launch_recurrent<2, 4>(GDN_REC_ARGS);
#undef GDN_REC_ARGS
}

}  // namespace gdn
