// Single-token decode of the gated delta rule (Section 3.2 of the paper):
//     old_v = k^T (alpha S),  delta = beta (v - old_v),  S' = alpha S + delta k^T,
//     out   = q^T (alpha S) + delta (q^T k)
// One pass over the fp32 state: every row is read once, updated in registers and
// written once; the output comes from the decayed old row plus a scalar correction,
// so the new state is never re-read.
//
// Work split.  A state row is 128 fp32 = 512 B.  Eight lanes own one row (each lane
// holds four float4 of it, interleaved so that every load instruction of a warp
// covers four whole 128-byte segments), so a warp works on four rows per "batch" and
// both dot products of a row reduce with three shuffle steps inside the 8-lane group.
// A warp issues the loads of all of its NB batches before the first use, which keeps
// NB*64 bytes per lane in flight; the V dimension is split over warps and CTAs so
// that small batches still cover all SMs.
#include "gdn_common.cuh"

namespace gdn {

template <int NB>
__device__ __forceinline__ void load_rows(const float* __restrict__ s_in, int row0, int sub, int c, float4 (&s)[NB][4]) {
#pragma unroll
    for (int i = 0; i < NB; ++i) {
        const float4* src = reinterpret_cast<const float4*>(s_in + (size_t)(row0 + i * 4 + sub) * kD);
#pragma unroll
        for (int j = 0; j < 4; ++j) s[i][j] = __ldcs(src + c + 8 * j);
    }
}

template <int NB, bool FRONT>
__device__ __forceinline__ void decode_rows(const float* __restrict__ s_in, float* __restrict__ s_out,
                                            const uint16_t* __restrict__ v_h, uint16_t* __restrict__ o_h,
                                            int row0, const float (&kf)[16], const float (&qf)[16],
                                            float alpha, float beta, float qk, float rk, float rq, int sub,
                                            int c, float4 (&s)[NB][4]) {
    float vr[NB];
#pragma unroll
    for (int i = 0; i < NB; ++i) vr[i] = bf16_bits_to_float(v_h[row0 + i * 4 + sub]);

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
        // FRONT: rk, rq are the front end's per-token factors on k and q (qk already carries them)
        const float delta = beta * (vr[i] - alpha * (FRONT ? a * rk : a));
        const float dk = FRONT ? delta * rk : delta;
        float4* dst = reinterpret_cast<float4*>(s_out + (size_t)(row0 + i * 4 + sub) * kD);
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            float4 w;
            w.x = fmaf(alpha, s[i][j].x, dk * kf[4 * j + 0]);
            w.y = fmaf(alpha, s[i][j].y, dk * kf[4 * j + 1]);
            w.z = fmaf(alpha, s[i][j].z, dk * kf[4 * j + 2]);
            w.w = fmaf(alpha, s[i][j].w, dk * kf[4 * j + 3]);
            __stcs(dst + c + 8 * j, w);
        }
        if (c == 0) o_h[row0 + i * 4 + sub] = float_to_bf16_bits(fmaf(delta, qk, alpha * (FRONT ? p * rq : p)));
    }
}

// grid.x = B*Hv*SPLIT, block = WARPS*32.  Each CTA owns 128/SPLIT rows of one head and
// each warp 4*NB of them: 128 = SPLIT * WARPS * 4 * NB.
template <int NB, int WARPS, bool FRONT>
__global__ void __launch_bounds__(WARPS * 32)
gdn_decode_kernel(const uint16_t* __restrict__ q, const uint16_t* __restrict__ k,
                  const uint16_t* __restrict__ v, const float* __restrict__ g,
                  const float* __restrict__ beta, const float* __restrict__ A_log,
                  const float* __restrict__ dt_bias, const float* s_in, float* s_out,
                  uint16_t* __restrict__ out, int Hqk, int Hv, int split, QkFront fr) {
    // the kernel before this one in the stream may have produced the tokens or the state
    pdl_wait();
    pdl_launch_dependents();
    const int cta = blockIdx.x;
    const int part = cta % split;
    const int bh = cta / split;  // b*Hv + h
    const int h = bh % Hv;
    const int b = bh / Hv;
    const int hq = h / (Hv / Hqk);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int sub = lane >> 3, c = lane & 7;
    const int row0 = (part * WARPS + warp) * (4 * NB);
    const size_t sbase = (size_t)bh * kD * kD;
    // the state rows first: nothing below depends on them until the dot products, and they are the
    // long-latency loads
    float4 s[NB][4];
    load_rows<NB>(s_in + sbase, row0, sub, c, s);

    // q, k columns of this lane: float4 index c + 8j  <->  bf16 elements 4(c+8j) .. +3
    const uint2* k4 = reinterpret_cast<const uint2*>(k + ((size_t)b * Hqk + hq) * kD);
    const uint2* q4 = reinterpret_cast<const uint2*>(q + ((size_t)b * Hqk + hq) * kD);
    float kf[16], qf[16];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const uint2 kw = __ldg(k4 + c + 8 * j);
        const uint2 qw = __ldg(q4 + c + 8 * j);
        unpack_bf16x2(kw.x, kf[4 * j + 0], kf[4 * j + 1]);
        unpack_bf16x2(kw.y, kf[4 * j + 2], kf[4 * j + 3]);
        unpack_bf16x2(qw.x, qf[4 * j + 0], qf[4 * j + 1]);
        unpack_bf16x2(qw.y, qf[4 * j + 2], qf[4 * j + 3]);
    }
    // g/beta hold the log-decay and write strength, or (A_log != NULL) the raw gate inputs a and b
    float gl = __ldg(g + bh), bt = __ldg(beta + bh);
    if (A_log) raw_gates(gl, bt, __ldg(A_log + h), __ldg(dt_bias + h), gl, bt);
    const float alpha = __expf(gl);
    float qk = 0.f;
#pragma unroll
    for (int j = 0; j < 16; ++j) qk = fmaf(qf[j], kf[j], qk);
#pragma unroll
    for (int m = 1; m < 8; m <<= 1) qk += __shfl_xor_sync(0xffffffffu, qk, m);
    float rk = 1.f, rq = 1.f;
    if constexpr (FRONT) {
        rq = fr.scale;
        if (fr.l2norm) {
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
        qk *= rk * rq;
    }

    decode_rows<NB, FRONT>(s_in + sbase, s_out + sbase, v + (size_t)bh * kD, out + (size_t)bh * kD, row0, kf, qf,
                           alpha, bt, qk, rk, rq, sub, c, s);
}

template <int NB, int WARPS>
static cudaError_t launch(const void* q, const void* k, const void* v, const float* g, const float* beta,
                          const float* A_log, const float* dt_bias, const float* s_in, float* s_out, void* out,
                          int B, int Hqk, int Hv, QkFront fr, cudaStream_t st) {
    constexpr int split = kD / (WARPS * 4 * NB);
    static_assert(split >= 1 && split * WARPS * 4 * NB == kD, "rows must tile the head");
    const long long ctas = (long long)B * Hv * split;
    if (fr.active())
        return launch_pdl(gdn_decode_kernel<NB, WARPS, true>, dim3((unsigned)ctas), dim3(WARPS * 32), 0, st,
                          (const uint16_t*)q, (const uint16_t*)k, (const uint16_t*)v, g, beta, A_log, dt_bias, s_in,
                          s_out, (uint16_t*)out, Hqk, Hv, split, fr);
    return launch_pdl(gdn_decode_kernel<NB, WARPS, false>, dim3((unsigned)ctas), dim3(WARPS * 32), 0, st,
                      (const uint16_t*)q, (const uint16_t*)k, (const uint16_t*)v, g, beta, A_log, dt_bias, s_in, s_out,
                      (uint16_t*)out, Hqk, Hv, split, fr);
}

// Launch-shape table.  `variant` < 0 picks from the number of (item, head) units; the other
// shapes stay selectable for tuning on other head counts.
cudaError_t decode_dispatch(const void* q, const void* k, const void* v, const float* g, const float* beta,
                            const float* A_log, const float* dt_bias, const float* s_in, float* s_out, void* out,
                            int B, int Hqk, int Hv, int variant, QkFront fr, cudaStream_t st) {
    if (variant < 0) {
        // from sweeps of all variants at 8 and 32 value heads, B = 1 .. 512: four rows per warp in
        // four-warp CTAs is the fastest shape from 16 (item, head) units upwards (3-7 % ahead of eight
        // rows per warp: more, smaller CTAs keep more loads in flight); below that, one-warp CTAs
        variant = ((long long)B * Hv <= 16) ? 0 : 8;
    }
    switch (variant) {
        case 0: return launch<1, 1>(q, k, v, g, beta, A_log, dt_bias, s_in, s_out, out, B, Hqk, Hv, fr, st);
        case 1: return launch<2, 1>(q, k, v, g, beta, A_log, dt_bias, s_in, s_out, out, B, Hqk, Hv, fr, st);
        case 2: return launch<2, 2>(q, k, v, g, beta, A_log, dt_bias, s_in, s_out, out, B, Hqk, Hv, fr, st);
        case 3: return launch<2, 4>(q, k, v, g, beta, A_log, dt_bias, s_in, s_out, out, B, Hqk, Hv, fr, st);
        case 4: return launch<4, 2>(q, k, v, g, beta, A_log, dt_bias, s_in, s_out, out, B, Hqk, Hv, fr, st);
        case 5: return launch<4, 4>(q, k, v, g, beta, A_log, dt_bias, s_in, s_out, out, B, Hqk, Hv, fr, st);
        case 6: return launch<4, 8>(q, k, v, g, beta, A_log, dt_bias, s_in, s_out, out, B, Hqk, Hv, fr, st);
        case 7: return launch<8, 4>(q, k, v, g, beta, A_log, dt_bias, s_in, s_out, out, B, Hqk, Hv, fr, st);
        case 8: return launch<1, 4>(q, k, v, g, beta, A_log, dt_bias, s_in, s_out, out, B, Hqk, Hv, fr, st);
        case 9: return launch<2, 8>(q, k, v, g, beta, A_log, dt_bias, s_in, s_out, out, B, Hqk, Hv, fr, st);
        case 10: return launch<1, 2>(q, k, v, g, beta, A_log, dt_bias, s_in, s_out, out, B, Hqk, Hv, fr, st);
        case 11: return launch<1, 8>(q, k, v, g, beta, A_log, dt_bias, s_in, s_out, out, B, Hqk, Hv, fr, st);
        default: return cudaErrorInvalidValue;
    }
}


// ---------------------------------------------------------------------------------------------
// Multi-token decode: T tokens per batch item (speculative / chunked decode), applied in order to
// state rows that stay in registers, so the state is still read once and written once.
// Layouts: q,k [B,T,Hqk,128], v,out [B,T,Hv,128], g,beta [B,T,Hv].
// FRONT: raw gate inputs when A_log is given, and the q/k front end `fr` (the fused entry point).
template <int NB, int WARPS, bool FRONT>
__global__ void __launch_bounds__(WARPS * 32)
gdn_decode_multi_kernel(const uint16_t* __restrict__ q, const uint16_t* __restrict__ k,
                        const uint16_t* __restrict__ v, const float* __restrict__ g,
                        const float* __restrict__ beta, const float* __restrict__ A_log,
                        const float* __restrict__ dt_bias, const float* s_in, float* s_out,
                        uint16_t* __restrict__ out, int T, int Hqk, int Hv, int split, QkFront fr) {
    pdl_wait();
    pdl_launch_dependents();
    const int cta = blockIdx.x;
    const int part = cta % split;
    const int bh = cta / split;
    const int h = bh % Hv, b = bh / Hv;
    const int hq = h / (Hv / Hqk);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int sub = lane >> 3, c = lane & 7;
    const int row0 = (part * WARPS + warp) * (4 * NB);
    const size_t sbase = (size_t)bh * kD * kD;

    float4 s[NB][4];
#pragma unroll
    for (int i = 0; i < NB; ++i) {
        const float4* src = reinterpret_cast<const float4*>(s_in + sbase + (size_t)(row0 + i * 4 + sub) * kD);
#pragma unroll
        for (int j = 0; j < 4; ++j) s[i][j] = __ldcs(src + c + 8 * j);
    }
    for (int t = 0; t < T; ++t) {
        const size_t tok = (size_t)b * T + t;
        const uint2* k4 = reinterpret_cast<const uint2*>(k + (tok * Hqk + hq) * kD);
        const uint2* q4 = reinterpret_cast<const uint2*>(q + (tok * Hqk + hq) * kD);
        float kf[16], qf[16];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const uint2 kw = __ldg(k4 + c + 8 * j);
            const uint2 qw = __ldg(q4 + c + 8 * j);
            unpack_bf16x2(kw.x, kf[4 * j + 0], kf[4 * j + 1]);
            unpack_bf16x2(kw.y, kf[4 * j + 2], kf[4 * j + 3]);
            unpack_bf16x2(qw.x, qf[4 * j + 0], qf[4 * j + 1]);
            unpack_bf16x2(qw.y, qf[4 * j + 2], qf[4 * j + 3]);
        }
        float gl = __ldg(g + tok * Hv + h), bt = __ldg(beta + tok * Hv + h);
        if (FRONT && A_log) raw_gates(gl, bt, __ldg(A_log + h), __ldg(dt_bias + h), gl, bt);
        const float alpha = __expf(gl);
        float qk = 0.f;
#pragma unroll
        for (int j = 0; j < 16; ++j) qk = fmaf(qf[j], kf[j], qk);
#pragma unroll
        for (int m = 1; m < 8; m <<= 1) qk += __shfl_xor_sync(0xffffffffu, qk, m);
        float rk = 1.f, rq = 1.f;
        if constexpr (FRONT) {
            rq = fr.scale;
            if (fr.l2norm) {
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
            qk *= rk * rq;
        }
        const uint16_t* v_h = v + (tok * Hv + h) * kD;
        uint16_t* o_h = out + (tok * Hv + h) * kD;
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
            const float delta = bt * (bf16_bits_to_float(__ldg(v_h + row0 + i * 4 + sub)) - alpha * (FRONT ? a * rk : a));
            const float dk = FRONT ? delta * rk : delta;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                s[i][j].x = fmaf(alpha, s[i][j].x, dk * kf[4 * j + 0]);
                s[i][j].y = fmaf(alpha, s[i][j].y, dk * kf[4 * j + 1]);
                s[i][j].z = fmaf(alpha, s[i][j].z, dk * kf[4 * j + 2]);
                s[i][j].w = fmaf(alpha, s[i][j].w, dk * kf[4 * j + 3]);
            }
            if (c == 0) o_h[row0 + i * 4 + sub] = float_to_bf16_bits(fmaf(delta, qk, alpha * (FRONT ? p * rq : p)));
        }
    }
#pragma unroll
    for (int i = 0; i < NB; ++i) {
        float4* dst = reinterpret_cast<float4*>(s_out + sbase + (size_t)(row0 + i * 4 + sub) * kD);
#pragma unroll
        for (int j = 0; j < 4; ++j) __stcs(dst + c + 8 * j, s[i][j]);
    }
}

template <int NB, int WARPS>
static cudaError_t launch_multi(const void* q, const void* k, const void* v, const float* g, const float* beta,
                                const float* A_log, const float* dt_bias, const float* s_in, float* s_out, void* out,
                                int B, int T, int Hqk, int Hv, QkFront fr, cudaStream_t st) {
    constexpr int split = kD / (WARPS * 4 * NB);
    const dim3 grid((unsigned)((long long)B * Hv * split));
    if (A_log || fr.active())
        return launch_pdl(gdn_decode_multi_kernel<NB, WARPS, true>, grid, dim3(WARPS * 32), 0, st, (const uint16_t*)q,
                          (const uint16_t*)k, (const uint16_t*)v, g, beta, A_log, dt_bias, s_in, s_out, (uint16_t*)out,
                          T, Hqk, Hv, split, fr);
    return launch_pdl(gdn_decode_multi_kernel<NB, WARPS, false>, grid, dim3(WARPS * 32), 0, st, (const uint16_t*)q,
                      (const uint16_t*)k, (const uint16_t*)v, g, beta, A_log, dt_bias, s_in, s_out, (uint16_t*)out, T,
                      Hqk, Hv, split, fr);
}

cudaError_t decode_multi_dispatch(const void* q, const void* k, const void* v, const float* g, const float* beta,
                                  const float* A_log, const float* dt_bias, const float* s_in, float* s_out, void* out,
                                  int B, int T, int Hqk, int Hv, QkFront fr, cudaStream_t st) {
    if (B <= 2) return launch_multi<1, 1>(q, k, v, g, beta, A_log, dt_bias, s_in, s_out, out, B, T, Hqk, Hv, fr, st);
    // Bandwidth regime: with T tokens per state row the kernel is co-bound by instruction issue
    // (every token costs a warp ~90 instructions that do not depend on how many rows it owns), so
    // sixteen rows per warp beat eight (B = 64, T = 4: 50.7 vs 58.1 us; 32 rows run out of registers).
    if (B >= 32) return launch_multi<4, 2>(q, k, v, g, beta, A_log, dt_bias, s_in, s_out, out, B, T, Hqk, Hv, fr, st);
    return launch_multi<2, 4>(q, k, v, g, beta, A_log, dt_bias, s_in, s_out, out, B, T, Hqk, Hv, fr, st);
}

}  // namespace gdn
