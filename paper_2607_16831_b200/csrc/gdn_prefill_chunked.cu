// Chunked WY / UT-transform prefill of the gated delta rule over 64-token chunks.
//
// The paper (Sections 3.3, 5.1, 5.5) names this reformulation -- group tokens into
// chunks, summarise the recurrence over each chunk, expose matrix-shaped work for the
// tensor cores -- without writing it out.  With gamma_i the cumulative log-gate inside a
// chunk, Gamma_i = exp(gamma_i), D_ij = exp(gamma_i - gamma_j) for j <= i, S the state
// entering the chunk ([dv][dk]) and K, Q, V the chunk's rows:
//
//   A   = strict_lower(diag(beta) (K K^T o D))           the kk^T lower-triangular system
//   T   = (I + A)^-1                                     UT transform (forward substitution)
//   T'  = T diag(beta),  W = T' diag(Gamma) K            so that U = T' V
//   P   = (Q K^T) o D  (lower triangle incl. diagonal)   chunk-local attention
//   Delta = T' V - W S^T                                 corrected values (stacked delta)
//   O   = diag(Gamma) Q S^T + P Delta
//   S  <- Gamma_L S + (diag(e) Delta)^T K,  e_j = exp(gamma_L - gamma_j)
//
// Three kernels:
//   prep   chunk table from cu_seqlens (integer work, one block)
//   intra  one CTA per (chunk, value head): gamma, K K^T, Q K^T, the triangular solve in
//          fp32, T' (bf16 hi+lo), W, P, and the per-token scalars -> workspace, already
//          in the 128-byte-swizzled shared-memory image the tensor cores read
//   chain  one CTA per (sequence, value head): serial over chunks; all five products per
//          chunk run on tcgen05 (bf16 operands, fp32 accumulators in tensor memory) fed
//          by TMA; the fp32 state lives in tensor memory for the whole sequence.
#include <cuda.h>

#include "gdn_common.cuh"
#include "gdn_sm100.cuh"

namespace gdn {
using namespace sm100;

// ------------------------------------------------------------------ workspace
constexpr int kScalBytes = 1024;   // per (chunk, head): Gamma[64] | e[64] | Gamma_L
constexpr int kABytes = 32768;     // per (chunk, head): T'hi 8K | T'lo 8K | W 16K (swizzled images)
constexpr int kPBytes = 8192;      // per (chunk, head): P (swizzled image)
constexpr int kStatusTimeout = 1;  // device status: a bounded wait ran out

struct WsLayout {
    int nc_max;
    size_t off_chunk_off, off_chunk_info, off_scal, off_A, off_P, total;
};

__host__ __device__ inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

__host__ __device__ inline WsLayout ws_layout(int total_tokens, int num_seqs, int Hv) {
    WsLayout L;
    L.nc_max = total_tokens / kChunk + num_seqs;  // >= sum over sequences of ceil(len/64)
    size_t o = 1024;                              // header: [0] status, [1] total chunks
    L.off_chunk_off = o;
    o = align_up(o + sizeof(int) * (size_t)(num_seqs + 1), 1024);
    L.off_chunk_info = o;
    o = align_up(o + sizeof(int4) * (size_t)L.nc_max, 1024);
    L.off_scal = o;
    o += (size_t)L.nc_max * Hv * kScalBytes;
    L.off_A = o;
    o += (size_t)L.nc_max * Hv * kABytes;
    L.off_P = o;
    o += (size_t)L.nc_max * Hv * kPBytes;
    L.total = o;
    return L;
}

size_t prefill_chunked_workspace_bytes(int total_tokens, int num_seqs, int /*Hqk*/, int Hv) {
    return ws_layout(total_tokens, num_seqs, Hv).total;
}

// Byte offset of 16-byte chunk `c16` of row `r` inside a [rows][64 bf16] tile stored with
// the 128-byte swizzle (what TMA writes and what the UMMA descriptors below expect).
__host__ __device__ __forceinline__ uint32_t swz(uint32_t r, uint32_t c16) {
    return r * 128u + ((c16 ^ (r & 7u)) << 4);
}

// ------------------------------------------------------------------ prep: chunk table
__global__ void __launch_bounds__(256)
gdn_prefill_prep_kernel(const int32_t* __restrict__ cu, int num_seqs, int total_tokens, int* hdr,
                        int* chunk_off, int4* chunk_info, int nc_max) {
    __shared__ int part[257];
    const int tid = threadIdx.x;
    const int per = (num_seqs + 255) / 256;
    const int lo = min(num_seqs, tid * per), hi = min(num_seqs, lo + per);
    int sum = 0;
    for (int n = lo; n < hi; ++n) {
        const int t0 = max(0, min(cu[n], total_tokens));
        const int t1 = max(t0, min(cu[n + 1], total_tokens));
        sum += (t1 - t0 + kChunk - 1) / kChunk;
    }
    part[tid] = sum;
    __syncthreads();
    if (tid == 0) {
        int run = 0;
        for (int i = 0; i < 256; ++i) {
            const int t = part[i];
            part[i] = run;
            run += t;
        }
        part[256] = run;
        hdr[0] = 0;
        hdr[1] = min(run, nc_max);
        chunk_off[num_seqs] = min(run, nc_max);
    }
    __syncthreads();
    int base = part[tid];
    for (int n = lo; n < hi; ++n) {
        const int t0 = max(0, min(cu[n], total_tokens));
        const int t1 = max(t0, min(cu[n + 1], total_tokens));
        const int nch = (t1 - t0 + kChunk - 1) / kChunk;
        chunk_off[n] = min(base, nc_max);
        for (int j = 0; j < nch; ++j)
            if (base + j < nc_max) chunk_info[base + j] = make_int4(n, t0 + j * kChunk, min(kChunk, t1 - t0 - j * kChunk), j);
        base += nch;
    }
}

// ------------------------------------------------------------------ intra-chunk kernel
constexpr int kIntraThreads = 256;
constexpr int kKP = 136;  // padded bf16 row length of the K/Q tiles in shared memory
constexpr int kMP = 68;   // padded fp32 row length of the 64x64 matrices
constexpr int kIntraSmem = 2 * 64 * kKP * 2 + 4 * 64 * kMP * 4 + 4 * 64 * 4;

__global__ void __launch_bounds__(kIntraThreads)
gdn_prefill_intra_kernel(const uint16_t* __restrict__ q, const uint16_t* __restrict__ k,
                         const float* __restrict__ g, const float* __restrict__ beta, uint8_t* __restrict__ ws,
                         WsLayout L, int Hqk, int Hv) {
    const int c = blockIdx.x, h = blockIdx.y;
    const int* hdr = reinterpret_cast<const int*>(ws);
    if (c >= hdr[1]) return;
    const int4 info = reinterpret_cast<const int4*>(ws + L.off_chunk_info)[c];
    const int t0 = info.y, len = info.z;
    const int hq = h / (Hv / Hqk);
    const int tid = threadIdx.x;

    extern __shared__ __align__(16) uint8_t smem[];
    uint16_t* Ks = reinterpret_cast<uint16_t*>(smem);            // [64][kKP]
    uint16_t* Qs = Ks + 64 * kKP;                                // [64][kKP]
    float* KK = reinterpret_cast<float*>(Qs + 64 * kKP);         // [64][kMP]
    float* QK = KK + 64 * kMP;
    float* Am = QK + 64 * kMP;
    float* Tm = Am + 64 * kMP;
    float* gam = Tm + 64 * kMP;   // [64] cumulative log gate
    float* bet = gam + 64;        // [64]
    float* Gam = bet + 64;        // [64] exp(gamma)
    float* tmp = Gam + 64;        // scratch

    // ---- load K, Q rows (rows >= len are zero), 16 bytes per thread per step
    for (int idx = tid; idx < 64 * 16; idx += kIntraThreads) {
        const int r = idx >> 4, cc = idx & 15;
        uint4 kv = make_uint4(0, 0, 0, 0), qv = make_uint4(0, 0, 0, 0);
        if (r < len) {
            const size_t off = ((size_t)(t0 + r) * Hqk + hq) * kD + cc * 8;
            kv = __ldg(reinterpret_cast<const uint4*>(k + off));
            qv = __ldg(reinterpret_cast<const uint4*>(q + off));
        }
        *reinterpret_cast<uint4*>(Ks + r * kKP + cc * 8) = kv;
        *reinterpret_cast<uint4*>(Qs + r * kKP + cc * 8) = qv;
    }
    // ---- gates: gamma = inclusive cumsum of g over the chunk (fp32), beta (0 beyond len)
    if (tid < 64) {
        float x = 0.f, b = 0.f;
        if (tid < len) {
            x = __ldg(g + (size_t)(t0 + tid) * Hv + h);
            b = __ldg(beta + (size_t)(t0 + tid) * Hv + h);
        }
        const int lane = tid & 31;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const float y = __shfl_up_sync(0xffffffffu, x, o);
            if (lane >= o) x += y;
        }
        if (tid == 31) tmp[0] = x;
        gam[tid] = x;
        bet[tid] = b;
    }
    __syncthreads();
    if (tid >= 32 && tid < 64) gam[tid] += tmp[0];
    __syncthreads();
    if (tid < 64) Gam[tid] = __expf(gam[tid]);

    // ---- K K^T and Q K^T, lower-triangular 4x4 tiles, fp32 accumulation
    {
        const int ti = tid >> 4, tj = tid & 15;
        if (tj <= ti) {
            float akk[4][4], aqk[4][4];
#pragma unroll
            for (int a = 0; a < 4; ++a)
#pragma unroll
                for (int b = 0; b < 4; ++b) akk[a][b] = aqk[a][b] = 0.f;
            for (int d = 0; d < kD; d += 8) {
                float ki[4][8], qi[4][8], kj[4][8];
#pragma unroll
                for (int a = 0; a < 4; ++a) {
                    const uint4 u = *reinterpret_cast<const uint4*>(Ks + (4 * ti + a) * kKP + d);
                    const uint4 w = *reinterpret_cast<const uint4*>(Qs + (4 * ti + a) * kKP + d);
                    const uint4 x = *reinterpret_cast<const uint4*>(Ks + (4 * tj + a) * kKP + d);
                    unpack_bf16x2(u.x, ki[a][0], ki[a][1]); unpack_bf16x2(u.y, ki[a][2], ki[a][3]);
                    unpack_bf16x2(u.z, ki[a][4], ki[a][5]); unpack_bf16x2(u.w, ki[a][6], ki[a][7]);
                    unpack_bf16x2(w.x, qi[a][0], qi[a][1]); unpack_bf16x2(w.y, qi[a][2], qi[a][3]);
                    unpack_bf16x2(w.z, qi[a][4], qi[a][5]); unpack_bf16x2(w.w, qi[a][6], qi[a][7]);
                    unpack_bf16x2(x.x, kj[a][0], kj[a][1]); unpack_bf16x2(x.y, kj[a][2], kj[a][3]);
                    unpack_bf16x2(x.z, kj[a][4], kj[a][5]); unpack_bf16x2(x.w, kj[a][6], kj[a][7]);
                }
#pragma unroll
                for (int a = 0; a < 4; ++a)
#pragma unroll
                    for (int b = 0; b < 4; ++b)
#pragma unroll
                        for (int e = 0; e < 8; ++e) {
                            akk[a][b] = fmaf(ki[a][e], kj[b][e], akk[a][b]);
                            aqk[a][b] = fmaf(qi[a][e], kj[b][e], aqk[a][b]);
                        }
            }
#pragma unroll
            for (int a = 0; a < 4; ++a)
#pragma unroll
                for (int b = 0; b < 4; ++b) {
                    KK[(4 * ti + a) * kMP + 4 * tj + b] = akk[a][b];
                    QK[(4 * ti + a) * kMP + 4 * tj + b] = aqk[a][b];
                }
        }
    }
    __syncthreads();

    uint8_t* wsA = ws + L.off_A + ((size_t)c * Hv + h) * kABytes;
    uint8_t* wsP = ws + L.off_P + ((size_t)c * Hv + h) * kPBytes;
    float* wsS = reinterpret_cast<float*>(ws + L.off_scal + ((size_t)c * Hv + h) * kScalBytes);

    // ---- A (strictly lower) into Am; P (lower incl. diagonal) straight to the workspace.
    // The gate differences are formed and masked before exp: above the diagonal they are
    // positive and could overflow.
    for (int idx = tid; idx < 64 * 8; idx += kIntraThreads) {
        const int i = idx >> 3, c16 = idx & 7;
        float pv[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            const int j = c16 * 8 + e;
            const float dec = (j <= i) ? __expf(gam[i] - gam[j]) : 0.f;
            Am[i * kMP + j] = (j < i) ? bet[i] * dec * KK[i * kMP + j] : 0.f;
            pv[e] = (j <= i && i < len) ? dec * QK[i * kMP + j] : 0.f;
        }
        uint4 o;
        o.x = pack_bf16x2(pv[0], pv[1]); o.y = pack_bf16x2(pv[2], pv[3]);
        o.z = pack_bf16x2(pv[4], pv[5]); o.w = pack_bf16x2(pv[6], pv[7]);
        *reinterpret_cast<uint4*>(wsP + swz(i, c16)) = o;
    }
    if (tid < 64) {
        wsS[tid] = Gam[tid];
        wsS[64 + tid] = __expf(gam[len - 1] - gam[tid]);
        if (tid == 0) wsS[128] = Gam[len - 1];
    }
    __syncthreads();

    // ---- UT transform: T = (I + A)^-1 by forward substitution; thread c owns column c.
    if (tid < 64) {
        const int col = tid;
        for (int i = 0; i < 64; ++i) {
            float acc = (i == col) ? 1.f : 0.f;
            const float* arow = Am + i * kMP;
            int j = 0;
            for (; j + 4 <= i; j += 4) {
                const float4 a4 = *reinterpret_cast<const float4*>(arow + j);
                acc = fmaf(-a4.x, Tm[(j + 0) * kMP + col], acc);
                acc = fmaf(-a4.y, Tm[(j + 1) * kMP + col], acc);
                acc = fmaf(-a4.z, Tm[(j + 2) * kMP + col], acc);
                acc = fmaf(-a4.w, Tm[(j + 3) * kMP + col], acc);
            }
            for (; j < i; ++j) acc = fmaf(-arow[j], Tm[j * kMP + col], acc);
            Tm[i * kMP + col] = acc;
        }
    }
    __syncthreads();

    // ---- T' = T diag(beta) -> bf16 hi + lo (swizzled); T'' = T' diag(Gamma) -> Am (fp32)
    for (int idx = tid; idx < 64 * 8; idx += kIntraThreads) {
        const int i = idx >> 3, c16 = idx & 7;
        float hi[8], lo[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            const int j = c16 * 8 + e;
            const float x = Tm[i * kMP + j] * bet[j];
            hi[e] = bf16_bits_to_float(float_to_bf16_bits(x));
            lo[e] = x - hi[e];
            Am[i * kMP + j] = x * Gam[j];
        }
        uint4 o;
        o.x = pack_bf16x2(hi[0], hi[1]); o.y = pack_bf16x2(hi[2], hi[3]);
        o.z = pack_bf16x2(hi[4], hi[5]); o.w = pack_bf16x2(hi[6], hi[7]);
        *reinterpret_cast<uint4*>(wsA + swz(i, c16)) = o;
        o.x = pack_bf16x2(lo[0], lo[1]); o.y = pack_bf16x2(lo[2], lo[3]);
        o.z = pack_bf16x2(lo[4], lo[5]); o.w = pack_bf16x2(lo[6], lo[7]);
        *reinterpret_cast<uint4*>(wsA + 8192 + swz(i, c16)) = o;
    }
    __syncthreads();

    // ---- W = T'' K  (64 x 128), thread tile 4 rows x 8 columns, T'' lower triangular
    {
        const int ty = tid >> 4, tx = tid & 15;
        float acc[4][8];
#pragma unroll
        for (int a = 0; a < 4; ++a)
#pragma unroll
            for (int e = 0; e < 8; ++e) acc[a][e] = 0.f;
        const int jmax = min(4 * ty + 3, len - 1);
        for (int j = 0; j <= jmax; ++j) {
            const uint4 u = *reinterpret_cast<const uint4*>(Ks + j * kKP + tx * 8);
            float kv[8];
            unpack_bf16x2(u.x, kv[0], kv[1]); unpack_bf16x2(u.y, kv[2], kv[3]);
            unpack_bf16x2(u.z, kv[4], kv[5]); unpack_bf16x2(u.w, kv[6], kv[7]);
#pragma unroll
            for (int a = 0; a < 4; ++a) {
                const float t = Am[(4 * ty + a) * kMP + j];
#pragma unroll
                for (int e = 0; e < 8; ++e) acc[a][e] = fmaf(t, kv[e], acc[a][e]);
            }
        }
#pragma unroll
        for (int a = 0; a < 4; ++a) {
            const int i = 4 * ty + a;
            uint4 o;
            o.x = pack_bf16x2(acc[a][0], acc[a][1]); o.y = pack_bf16x2(acc[a][2], acc[a][3]);
            o.z = pack_bf16x2(acc[a][4], acc[a][5]); o.w = pack_bf16x2(acc[a][6], acc[a][7]);
            // W is the K-major B operand [64 rows][128]: two [64][64] tiles
            *reinterpret_cast<uint4*>(wsA + 16384 + (tx >> 3) * 8192 + swz(i, tx & 7)) = o;
        }
    }
}

// ------------------------------------------------------------------ chain kernel
constexpr int kChainThreads = 128;
// shared-memory map (bytes from a 1024-byte aligned base)
constexpr uint32_t OFF_SHI = 0;        // S (bf16) A operand, K-major: 2 tiles [128][64]      32 KB
constexpr uint32_t OFF_DL = 32768;     // Delta^T (bf16) A operand, K-major [128][64]          16 KB
constexpr uint32_t OFF_DTH = 49152;    // (e o Delta)^T hi                                      16 KB
constexpr uint32_t OFF_DTL = 65536;    // (e o Delta)^T lo                                      16 KB
constexpr uint32_t OFF_A = 81920;      // T'hi 8K | T'lo 8K | W 16K   (bulk copy)               32 KB
constexpr uint32_t OFF_V = 114688;     // V tile: 2 x [64 tokens][64]  (TMA)                    16 KB
constexpr uint32_t OFF_Q = 131072;     // Q tile                         (TMA)                  16 KB
constexpr uint32_t OFF_P = 147456;     // P                              (bulk copy)             8 KB
constexpr uint32_t OFF_K = 155648;     // K tile                         (TMA)                  16 KB
constexpr uint32_t OFF_SCAL = 172032;  // 2 x 1 KB scalars (double buffered)
constexpr uint32_t OFF_BAR = 174080;   // 4 mbarriers, TMEM slot, abort flag
constexpr uint32_t kChainSmem = OFF_BAR + 128 + 1024;  // + slack for the manual 1024-byte alignment
constexpr uint32_t kTxA = kABytes + kScalBytes + 16384 + 16384;
constexpr uint32_t kTxB = kPBytes + 16384;
// tensor-memory columns
constexpr uint32_t TM_DELTA = 0, TM_OA = 64, TM_OB = 128, TM_S = 256, TM_COLS = 512;

__global__ void __launch_bounds__(kChainThreads, 1)
gdn_prefill_chain_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                         const __grid_constant__ CUtensorMap map_v, const float* initial_state,
                         uint16_t* __restrict__ out, float* final_state, uint8_t* __restrict__ ws, WsLayout L,
                         int Hqk, int Hv) {
    const int h = blockIdx.x % Hv, n = blockIdx.x / Hv;
    const int hq = h / (Hv / Hqk);
    const int tid = threadIdx.x, warp = tid >> 5;
    const int v = tid;  // this thread owns state row v, i.e. tensor-memory lane v

    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint64_t* bar_fullA = reinterpret_cast<uint64_t*>(smem + OFF_BAR);
    uint64_t* bar_fullB = bar_fullA + 1;
    uint64_t* bar_delta = bar_fullA + 2;
    uint64_t* bar_state = bar_fullA + 3;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + OFF_BAR + 32);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + OFF_BAR + 40);

    const int* chunk_off = reinterpret_cast<const int*>(ws + L.off_chunk_off);
    const int4* chunk_info = reinterpret_cast<const int4*>(ws + L.off_chunk_info);
    const int c_begin = chunk_off[n], c_end = chunk_off[n + 1];
    const int nchunks = c_end - c_begin;
    const size_t sbase = ((size_t)n * Hv + h) * kD * kD + (size_t)v * kD;

    if (nchunks <= 0) {  // empty sequence: the state passes through
        if (final_state) {
            for (int j = 0; j < kD; j += 4) {
                float4 x = make_float4(0.f, 0.f, 0.f, 0.f);
                if (initial_state) x = *reinterpret_cast<const float4*>(initial_state + sbase + j);
                *reinterpret_cast<float4*>(final_state + sbase + j) = x;
            }
        }
        return;
    }

    if (tid == 0) {
        mbar_init(bar_fullA, 1);
        mbar_init(bar_fullB, 1);
        mbar_init(bar_delta, 1);
        mbar_init(bar_state, 1);
        *abort_flag = 0;
        mbar_fence_init();
        prefetch_tensormap(&map_q);
        prefetch_tensormap(&map_k);
        prefetch_tensormap(&map_v);
    }
    if (warp == 0) {
        __syncwarp();
        tmem_alloc(tmem_slot, TM_COLS);
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;
    const uint32_t lane_addr = tmem_base + ((uint32_t)(warp * 32) << 16);

    auto scal_ptr = [&](int c) { return reinterpret_cast<const float*>(ws + L.off_scal + ((size_t)c * Hv + h) * kScalBytes); };
    auto issue_A = [&](int c) {  // T'hi, T'lo, W, scalars (bulk) + V, Q tiles (TMA)
        const int t0 = chunk_info[c].y;
        mbar_expect_tx(bar_fullA, kTxA);
        bulk_load(smem + OFF_A, ws + L.off_A + ((size_t)c * Hv + h) * kABytes, kABytes, bar_fullA);
        bulk_load(smem + OFF_SCAL + ((c - c_begin) & 1) * kScalBytes, scal_ptr(c), kScalBytes, bar_fullA);
        tma_load_3d(smem + OFF_V, &map_v, bar_fullA, 0, h, t0);
        tma_load_3d(smem + OFF_V + 8192, &map_v, bar_fullA, 64, h, t0);
        tma_load_3d(smem + OFF_Q, &map_q, bar_fullA, 0, hq, t0);
        tma_load_3d(smem + OFF_Q + 8192, &map_q, bar_fullA, 64, hq, t0);
    };
    auto issue_B = [&](int c) {  // P (bulk) + K tile (TMA)
        const int t0 = chunk_info[c].y;
        mbar_expect_tx(bar_fullB, kTxB);
        bulk_load(smem + OFF_P, ws + L.off_P + ((size_t)c * Hv + h) * kPBytes, kPBytes, bar_fullB);
        tma_load_3d(smem + OFF_K, &map_k, bar_fullB, 0, hq, t0);
        tma_load_3d(smem + OFF_K + 8192, &map_k, bar_fullB, 64, hq, t0);
    };

    bool pendA = false, pendB = false;  // thread 0: copies in flight that nobody has waited for yet
    if (tid == 0) {
        issue_A(c_begin);
        issue_B(c_begin);
        pendA = pendB = true;
    }

    // ---- initial state: bf16 copy -> shared (A operand), Gamma_L(first chunk) * S -> tensor memory
    {
        const float gl0 = __ldg(scal_ptr(c_begin) + 128);
#pragma unroll 1
        for (int b = 0; b < 4; ++b) {
            uint32_t r[32];
#pragma unroll
            for (int j = 0; j < 32; j += 4) {
                float4 x = make_float4(0.f, 0.f, 0.f, 0.f);
                if (initial_state) x = *reinterpret_cast<const float4*>(initial_state + sbase + b * 32 + j);
                r[j + 0] = __float_as_uint(x.x); r[j + 1] = __float_as_uint(x.y);
                r[j + 2] = __float_as_uint(x.z); r[j + 3] = __float_as_uint(x.w);
            }
#pragma unroll
            for (int cc = 0; cc < 4; ++cc) {
                uint4 o;
                o.x = pack_bf16x2(__uint_as_float(r[cc * 8 + 0]), __uint_as_float(r[cc * 8 + 1]));
                o.y = pack_bf16x2(__uint_as_float(r[cc * 8 + 2]), __uint_as_float(r[cc * 8 + 3]));
                o.z = pack_bf16x2(__uint_as_float(r[cc * 8 + 4]), __uint_as_float(r[cc * 8 + 5]));
                o.w = pack_bf16x2(__uint_as_float(r[cc * 8 + 6]), __uint_as_float(r[cc * 8 + 7]));
                *reinterpret_cast<uint4*>(smem + OFF_SHI + (b >> 1) * 16384 + swz(v, (b & 1) * 4 + cc)) = o;
            }
#pragma unroll
            for (int j = 0; j < 32; ++j) r[j] = __float_as_uint(__uint_as_float(r[j]) * gl0);
            tmem_st32(lane_addr + TM_S + b * 32, r);
        }
        tmem_st_wait();
        fence_proxy_async_smem();
        tc_fence_before_sync();
        __syncthreads();
    }

    constexpr uint32_t ID_G1 = umma_idesc_bf16(128, 64, true, false, false);    // V^T (MN-major A) x T'
    constexpr uint32_t ID_G2A = umma_idesc_bf16(128, 64, false, false, true);   // -(S) x W^T
    constexpr uint32_t ID_G2B = umma_idesc_bf16(128, 64, false, false, false);  // S x Q^T ; Delta^T x P^T
    constexpr uint32_t ID_G3B = umma_idesc_bf16(128, 128, false, true, false);  // (e o Delta)^T x K (MN-major B)
    const uint32_t sb = smem_u32(smem);

    for (int ci = 0; ci < nchunks; ++ci) {
        const int c = c_begin + ci;
        const uint32_t par = ci & 1;
        const int4 info = chunk_info[c];
        const int t0 = info.y, len = info.z;
        const bool last = (ci + 1 == nchunks);
        const float* scal = reinterpret_cast<const float*>(smem + OFF_SCAL + (ci & 1) * kScalBytes);
        const float gl_next = last ? 1.f : __ldg(scal_ptr(c + 1) + 128);

        // ---- Delta^T = V^T T'^T - S W^T  and  Oa^T = S Q^T
        if (tid == 0) {
            if (mbar_wait(bar_fullA, par, abort_flag)) {
                pendA = false;
                tc_fence_after_sync();
#pragma unroll
                for (int ks = 0; ks < 4; ++ks)
                    umma_bf16_ss(tmem_base + TM_DELTA, umma_desc(sb + OFF_V + ks * 2048, 8192, 1024),
                                 umma_desc(sb + OFF_A + ks * 32, 16, 1024), ID_G1, ks > 0);
#pragma unroll
                for (int ks = 0; ks < 4; ++ks)
                    umma_bf16_ss(tmem_base + TM_DELTA, umma_desc(sb + OFF_V + ks * 2048, 8192, 1024),
                                 umma_desc(sb + OFF_A + 8192 + ks * 32, 16, 1024), ID_G1, 1);
#pragma unroll
                for (int ks = 0; ks < 8; ++ks)
                    umma_bf16_ss(tmem_base + TM_DELTA,
                                 umma_desc(sb + OFF_SHI + (ks >> 2) * 16384 + (ks & 3) * 32, 16, 1024),
                                 umma_desc(sb + OFF_A + 16384 + (ks >> 2) * 8192 + (ks & 3) * 32, 16, 1024), ID_G2A, 1);
#pragma unroll
                for (int ks = 0; ks < 8; ++ks)
                    umma_bf16_ss(tmem_base + TM_OA,
                                 umma_desc(sb + OFF_SHI + (ks >> 2) * 16384 + (ks & 3) * 32, 16, 1024),
                                 umma_desc(sb + OFF_Q + (ks >> 2) * 8192 + (ks & 3) * 32, 16, 1024), ID_G2B, ks > 0);
                umma_commit(bar_delta);
            }
        }
        bool ok = mbar_wait(bar_delta, par, abort_flag);
        tc_fence_after_sync();
        if (tid == 0 && ok && !last) {
            issue_A(c + 1);
            pendA = true;
        }
        if (ok) {
            // Delta^T row v: bf16 copy, and the decayed copy (e o Delta)^T as bf16 hi + lo
#pragma unroll 1
            for (int half = 0; half < 2; ++half) {
                uint32_t r[32];
                tmem_ld32(lane_addr + TM_DELTA + half * 32, r);
                tmem_ld_wait();
#pragma unroll
                for (int cc = 0; cc < 4; ++cc) {
                    float x[8], hi[8], lo[8];
#pragma unroll
                    for (int e = 0; e < 8; ++e) {
                        x[e] = __uint_as_float(r[cc * 8 + e]);
                        const float y = x[e] * scal[64 + half * 32 + cc * 8 + e];
                        hi[e] = bf16_bits_to_float(float_to_bf16_bits(y));
                        lo[e] = y - hi[e];
                    }
                    const uint32_t off = swz(v, half * 4 + cc);
                    uint4 o;
                    o.x = pack_bf16x2(x[0], x[1]); o.y = pack_bf16x2(x[2], x[3]);
                    o.z = pack_bf16x2(x[4], x[5]); o.w = pack_bf16x2(x[6], x[7]);
                    *reinterpret_cast<uint4*>(smem + OFF_DL + off) = o;
                    o.x = pack_bf16x2(hi[0], hi[1]); o.y = pack_bf16x2(hi[2], hi[3]);
                    o.z = pack_bf16x2(hi[4], hi[5]); o.w = pack_bf16x2(hi[6], hi[7]);
                    *reinterpret_cast<uint4*>(smem + OFF_DTH + off) = o;
                    o.x = pack_bf16x2(lo[0], lo[1]); o.y = pack_bf16x2(lo[2], lo[3]);
                    o.z = pack_bf16x2(lo[4], lo[5]); o.w = pack_bf16x2(lo[6], lo[7]);
                    *reinterpret_cast<uint4*>(smem + OFF_DTL + off) = o;
                }
            }
        }
        fence_proxy_async_smem();
        tc_fence_before_sync();
        __syncthreads();
        if (*abort_flag) break;

        // ---- Ob^T = Delta^T P^T  and  S += (e o Delta)^T K
        if (tid == 0) {
            if (mbar_wait(bar_fullB, par, abort_flag)) {
                pendB = false;
                tc_fence_after_sync();
#pragma unroll
                for (int ks = 0; ks < 4; ++ks)
                    umma_bf16_ss(tmem_base + TM_OB, umma_desc(sb + OFF_DL + ks * 32, 16, 1024),
                                 umma_desc(sb + OFF_P + ks * 32, 16, 1024), ID_G2B, ks > 0);
#pragma unroll
                for (int ks = 0; ks < 4; ++ks)
                    umma_bf16_ss(tmem_base + TM_S, umma_desc(sb + OFF_DTH + ks * 32, 16, 1024),
                                 umma_desc(sb + OFF_K + ks * 2048, 8192, 1024), ID_G3B, 1);
#pragma unroll
                for (int ks = 0; ks < 4; ++ks)
                    umma_bf16_ss(tmem_base + TM_S, umma_desc(sb + OFF_DTL + ks * 32, 16, 1024),
                                 umma_desc(sb + OFF_K + ks * 2048, 8192, 1024), ID_G3B, 1);
                umma_commit(bar_state);
            }
        }
        ok = mbar_wait(bar_state, par, abort_flag);
        tc_fence_after_sync();
        if (tid == 0 && ok && !last) {
            issue_B(c + 1);
            pendB = true;
        }
        if (ok) {
            // state row v: fp32 -> bf16 operand copy for the next chunk, pre-decayed fp32 back to
            // tensor memory (or out to final_state after the last chunk)
#pragma unroll 1
            for (int b = 0; b < 4; ++b) {
                uint32_t r[32];
                tmem_ld32(lane_addr + TM_S + b * 32, r);
                tmem_ld_wait();
                if (last) {
                    if (final_state) {
#pragma unroll
                        for (int j = 0; j < 32; j += 4)
                            *reinterpret_cast<float4*>(final_state + sbase + b * 32 + j) =
                                make_float4(__uint_as_float(r[j]), __uint_as_float(r[j + 1]), __uint_as_float(r[j + 2]),
                                            __uint_as_float(r[j + 3]));
                    }
                } else {
#pragma unroll
                    for (int cc = 0; cc < 4; ++cc) {
                        uint4 o;
                        o.x = pack_bf16x2(__uint_as_float(r[cc * 8 + 0]), __uint_as_float(r[cc * 8 + 1]));
                        o.y = pack_bf16x2(__uint_as_float(r[cc * 8 + 2]), __uint_as_float(r[cc * 8 + 3]));
                        o.z = pack_bf16x2(__uint_as_float(r[cc * 8 + 4]), __uint_as_float(r[cc * 8 + 5]));
                        o.w = pack_bf16x2(__uint_as_float(r[cc * 8 + 6]), __uint_as_float(r[cc * 8 + 7]));
                        *reinterpret_cast<uint4*>(smem + OFF_SHI + (b >> 1) * 16384 + swz(v, (b & 1) * 4 + cc)) = o;
                    }
#pragma unroll
                    for (int j = 0; j < 32; ++j) r[j] = __float_as_uint(__uint_as_float(r[j]) * gl_next);
                    tmem_st32(lane_addr + TM_S + b * 32, r);
                }
            }
            // outputs of this chunk: o[t0+i][h][v] = Gamma_i * Oa^T[v][i] + Ob^T[v][i]
#pragma unroll 1
            for (int half = 0; half < 2; ++half) {
                uint32_t ra[32], rb[32];
                tmem_ld32(lane_addr + TM_OA + half * 32, ra);
                tmem_ld32(lane_addr + TM_OB + half * 32, rb);
                tmem_ld_wait();
#pragma unroll
                for (int j = 0; j < 32; ++j) {
                    const int i = half * 32 + j;
                    if (i < len)
                        out[((size_t)(t0 + i) * Hv + h) * kD + v] =
                            float_to_bf16_bits(fmaf(scal[i], __uint_as_float(ra[j]), __uint_as_float(rb[j])));
                }
            }
            tmem_st_wait();
        }
        fence_proxy_async_smem();
        tc_fence_before_sync();
        __syncthreads();
        if (*abort_flag) break;
    }

    // ---- unwind: let copies in flight land (bounded), release tensor memory, report
    if (tid == 0) {
        int dummy = 0;
        if (pendA) mbar_wait(bar_fullA, (uint32_t)((nchunks - 1) & 1), &dummy, 200000000LL);
        if (pendB) mbar_wait(bar_fullB, (uint32_t)((nchunks - 1) & 1), &dummy, 200000000LL);
        if (*abort_flag) atomicExch(reinterpret_cast<int*>(ws), kStatusTimeout);
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 0) {
        __syncwarp();
        tmem_dealloc(tmem_base, TM_COLS);
    }
}

// ------------------------------------------------------------------ host side
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

cudaError_t prefill_chunked_dispatch(const void* q, const void* k, const void* v, const float* g,
                                     const float* beta, const int32_t* cu_seqlens, const float* initial_state,
                                     void* out, float* final_state, int total_tokens, int num_seqs,
                                     int /*max_seqlen*/, int Hqk, int Hv, void* workspace, size_t /*workspace_bytes*/,
                                     cudaStream_t st) {
    static bool attr_done = false;
    if (!attr_done) {
        cudaError_t e = cudaFuncSetAttribute(gdn_prefill_intra_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             kIntraSmem);
        if (e != cudaSuccess) return e;
        e = cudaFuncSetAttribute(gdn_prefill_chain_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kChainSmem);
        if (e != cudaSuccess) return e;
        attr_done = true;
    }
    uint8_t* ws = static_cast<uint8_t*>(workspace);
    const WsLayout L = ws_layout(total_tokens, num_seqs, Hv);
    gdn_prefill_prep_kernel<<<1, 256, 0, st>>>(cu_seqlens, num_seqs, total_tokens, reinterpret_cast<int*>(ws),
                                               reinterpret_cast<int*>(ws + L.off_chunk_off),
                                               reinterpret_cast<int4*>(ws + L.off_chunk_info), L.nc_max);
    if (total_tokens > 0) {
        CUtensorMap mq, mk, mv;
        if (!make_map(&mq, q, total_tokens, Hqk) || !make_map(&mk, k, total_tokens, Hqk) ||
            !make_map(&mv, v, total_tokens, Hv))
            return cudaErrorUnknown;
        dim3 gi(L.nc_max, Hv);
        gdn_prefill_intra_kernel<<<gi, kIntraThreads, kIntraSmem, st>>>(
            (const uint16_t*)q, (const uint16_t*)k, g, beta, ws, L, Hqk, Hv);
        gdn_prefill_chain_kernel<<<(unsigned)((long long)num_seqs * Hv), kChainThreads, kChainSmem, st>>>(
            mq, mk, mv, initial_state, (uint16_t*)out, final_state, ws, L, Hqk, Hv);
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

}  // namespace gdn
