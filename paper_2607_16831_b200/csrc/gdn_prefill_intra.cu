// Chunk table and intra-chunk kernel of the chunked WY / UT-transform prefill.
//
// Per (chunk, value head), with gamma the cumulative log-gate inside the chunk,
// Gamma = exp(gamma), D_ij = exp(gamma_i - gamma_j) for j <= i:
//   A  = strict_lower(diag(beta) (K K^T o D))     the kk^T lower-triangular system
//   T  = (I + A)^-1                               UT transform by substitution (fp32)
//   T' = T diag(beta)   (bf16 hi + lo),   W = T' diag(Gamma) K,   P = (Q K^T) o D
// K K^T, Q K^T and W run on tcgen05 (bf16 operands fed by TMA, fp32 accumulation); the gate
// algebra and the triangular solve stay in fp32 registers.
// and the per-token scalars Gamma_i, e_i = exp(gamma_L - gamma_i), Gamma_L.  Everything is
// written to the workspace already in the 128-byte-swizzled shared-memory image that the
// chain kernel hands to the tensor cores.
#include "gdn_prefill_ws.cuh"
#include "gdn_sm100.cuh"

namespace gdn {
using namespace sm100;

// ------------------------------------------------------------------ prep: chunk table
__global__ void __launch_bounds__(256)
gdn_prefill_prep_kernel(const int32_t* __restrict__ cu, int num_seqs, int total_tokens, int* hdr,
                        int* chunk_off, int4* seq_order, int4* chunk_info, int nc_max) {
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
    // Longest sequences first: the chain kernel's cost per chain is the chunk count, so handing out the
    // long chains first shortens the tail of the launch.  Rank by counting (ties broken by index), the
    // lengths of 256 sequences at a time staged in shared memory: O(N^2 / 256) shared-memory reads per
    // thread.  The record holds everything a chain needs to know about its sequence, so that it finds its
    // work with one load instead of a chain of dependent ones.
    __syncthreads();  // chunk_off of every sequence is written
    __shared__ int len_s[256];
    for (int n0 = 0; n0 < num_seqs; n0 += 256) {   // (uniform trip count: every thread takes part in the staging)
        const int n = n0 + tid;
        int tn = 0, ln = -1;
        if (n < num_seqs) {
            tn = max(0, min(cu[n], total_tokens));
            ln = max(tn, min(cu[n + 1], total_tokens)) - tn;
        }
        int rank = 0;
        for (int m0 = 0; m0 < num_seqs; m0 += 256) {
            __syncthreads();
            const int m = m0 + tid;
            int lm = -1;
            if (m < num_seqs) {
                const int tm = max(0, min(cu[m], total_tokens));
                lm = max(tm, min(cu[m + 1], total_tokens)) - tm;
            }
            len_s[tid] = lm;
            __syncthreads();
            const int cnt = min(256, num_seqs - m0);
            for (int j = 0; j < cnt; ++j) {
                const int l = len_s[j];
                rank += (l > ln) || (l == ln && m0 + j < n);
            }
        }
        if (n < num_seqs) seq_order[rank] = make_int4(n, chunk_off[n], tn, ln);
    }
}

// ------------------------------------------------------------------ intra-chunk kernel
// One CTA (128 threads, four CTAs per SM) per (chunk, q/k head, pair of value heads); a pair makes
// every tensor-core product M = 128 (thread r = head (r / 64) of the pair, row r % 64):
//   MMA1   [Q ; K] K^T           (128 x 64 x 128)  rows 0-63: Q K^T, rows 64-127: K K^T
//   solve  T = (I + A)^-1 row by row through the transposed system y (I + A) = e_i, blocked by
//          16 columns from the right:
//              y_blk(jb) = (e_blk(jb) - sum_{mb > jb} y_blk(mb) A[mb][jb]) (I + A[jb][jb])^-1
//          The sum over finished blocks is a small tensor-core product (y as bf16 hi + lo A operand
//          in tensor memory, the off-diagonal blocks of A as bf16 hi + lo B tiles, fp32 accumulate);
//          only the 16 x 16 diagonal solve stays in fp32 registers.  Four dependent steps instead
//          of a 64-long substitution chain, equal work for every row.
//   MMA2   [T''_a ; T''_b] K     (128 x 128 x 64)  T'' = T diag(beta o Gamma) in bf16
// K K^T is symmetric, so the thread that owns row j of K K^T produces COLUMN j of A, which is a
// row of the B tile: everything is written with 16-byte shared-memory stores.
constexpr int kIntraThreads = 128;
constexpr uint32_t IQ_LO = 0, IK_LO = 8192, IQ_HI = 16384, IK_HI = 24576;  // TMA tiles [64][64] bf16
constexpr uint32_t IDG = IQ_LO;    // after MMA1: diagonal blocks of A^T, fp32 [2 heads][4][16][16]        8 KB
constexpr uint32_t IBT2 = IQ_HI;   // after MMA1: B tiles of column block 2 (hi 4 KB | lo 4 KB)
constexpr uint32_t IBT = 32768;    // B tiles of column blocks 0 and 1: [jb][hi|lo] x 4 KB               16 KB
constexpr uint32_t IT2 = IBT;      // after the solve: T'' operand (bf16) [128][64]                       16 KB
constexpr uint32_t IGAM = IBT + 16384;  // gam[2][64] | bet[2][64] | Gam[2][64] | cfP[2][64] | cfA[2][64] | alp[2][64] | rq[64] | rk[64] | tmp[4]
constexpr uint32_t IBAR = IGAM + 14 * 64 * 4 + 64;
constexpr uint32_t kIntraSmem = IBAR + 64 + 1024;
// tensor-memory columns: [QK^T ; KK^T] first, then the solve's operands, then the W accumulator
constexpr uint32_t ITM_D1 = 0, ITM_YHI = 0, ITM_YLO = 32, ITM_ACC = 64, ITM_D2 = 0, ITM_COLS = 128;

// sixteen consecutive floats of a coefficient table (64-byte aligned) as four 16-byte loads
__device__ __forceinline__ void ld16(const float* p, float (&x)[16]) {
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        const float4 t = reinterpret_cast<const float4*>(p)[q];
        x[4 * q] = t.x; x[4 * q + 1] = t.y; x[4 * q + 2] = t.z; x[4 * q + 3] = t.w;
    }
}

__device__ __forceinline__ uint32_t intra_btile(int jb, int lo) {  // byte offset of B tile (jb, hi/lo)
    return (jb == 2 ? IBT2 : IBT + (uint32_t)jb * 8192u) + (uint32_t)lo * 4096u;
}

// FRONT: the fused entry points' q/k front end (QkFront).  q and k stay as they are in shared memory and
// in the products; the per-token factors rq_i = scale / |q_i| and rk_j = 1 / |k_j| go into the
// coefficients instead: P_ij gets rq_i rk_j, the state update's e_j gets rk_j, the output scaling
// Gamma_i gets rq_i.  For the triangular system, with R = diag(rk) and G = K K^T o D,
//     A = diag(beta) R G R   and   (I + A)^-1 = R (I + diag(beta) G R^2)^-1 R^-1,
// so the system that is solved carries only a per-COLUMN factor rk_j^2 (one scalar for the thread that
// owns column j), and the similarity comes back at the end as a per-row factor rk_i and two rescaled
// tables: T diag(beta) = rk_i z_ij (beta_j / rk_j), and in W = T diag(beta Gamma rk) K the column
// factors cancel to beta_j Gamma_j.  The kernels after this one see nothing of it.
template <bool FRONT>
__global__ void __launch_bounds__(kIntraThreads, 4)
gdn_prefill_intra_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                         const float* __restrict__ g, const float* __restrict__ beta,
                         const float* __restrict__ A_log, const float* __restrict__ dt_bias,
                         uint8_t* __restrict__ ws, WsLayout L, int Hqk, int Hv, const int32_t* __restrict__ cu,
                         int num_seqs, int total_tokens, QkFront fr) {
    const int c = blockIdx.x;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    int t0, len;
    if (cu) {
        // Few sequences: no chunk-table kernel ran.  Every CTA finds its chunk by walking cu_seqlens
        // (one round trip: the loads are independent), and the first CTA leaves the tables the later
        // kernels read -- what gdn_prefill_prep_kernel would have written.
        int run = 0;
        t0 = 0;
        len = -1;
        for (int n = 0; n < num_seqs; ++n) {
            const int a = max(0, min(cu[n], total_tokens)), b = max(a, min(cu[n + 1], total_tokens));
            const int nch = (b - a + kChunk - 1) / kChunk;
            if (c >= run && c < run + nch) {
                t0 = a + (c - run) * kChunk;
                len = min(kChunk, b - t0);
            }
            run += nch;
        }
        if (blockIdx.x == 0 && blockIdx.y == 0) {
            int* hdr_w = reinterpret_cast<int*>(ws);
            int* chunk_off = reinterpret_cast<int*>(ws + L.off_chunk_off);
            int4* seq_order = reinterpret_cast<int4*>(ws + L.off_seq_order);
            int4* chunk_info = reinterpret_cast<int4*>(ws + L.off_chunk_info);
            const int total = min(run, L.nc_max);
            if (tid == 0) {
                hdr_w[0] = 0;
                hdr_w[1] = total;
                chunk_off[num_seqs] = total;
            }
            for (int n = tid; n < num_seqs; n += kIntraThreads) {
                int base = 0, rank = 0;
                const int a = max(0, min(cu[n], total_tokens)), b = max(a, min(cu[n + 1], total_tokens));
                for (int m = 0; m < num_seqs; ++m) {
                    const int am = max(0, min(cu[m], total_tokens)), bm = max(am, min(cu[m + 1], total_tokens));
                    if (m < n) base += (bm - am + kChunk - 1) / kChunk;
                    rank += (bm - am > b - a) || (bm - am == b - a && m < n);
                }
                chunk_off[n] = min(base, L.nc_max);
                seq_order[rank] = make_int4(n, min(base, L.nc_max), a, b - a);  // longest first
                const int nch = (b - a + kChunk - 1) / kChunk;
                for (int j = 0; j < nch; ++j)
                    if (base + j < L.nc_max)
                        chunk_info[base + j] = make_int4(n, a + j * kChunk, min(kChunk, b - a - j * kChunk), j);
            }
        }
        if (len < 0 || c >= L.nc_max) return;
    } else {
        const int* hdr = reinterpret_cast<const int*>(ws);
        if (c >= hdr[1]) return;
        const int4 info = reinterpret_cast<const int4*>(ws + L.off_chunk_info)[c];
        t0 = info.y;
        len = info.z;
    }
    const int G = Hv / Hqk;
    const int npairs = (G + 1) / 2;
    const int hq = blockIdx.y / npairs, p = blockIdx.y % npairs;
    const int hh = tid >> 6, i = tid & 63;  // role in the gate / solve / W phases: head of the pair, row
    const int nh = min(2, G - 2 * p);
    const int h = hq * G + 2 * p + hh;      // this thread's value head in those phases
    const bool head_ok = hh < nh;

    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    float* gam = reinterpret_cast<float*>(smem + IGAM);
    float* bet = gam + 128;
    float* Gam = gam + 256;
    float* cfP = gam + 384;  // exp(gamma_{last column of j's 16-block} - gamma_j)
    float* cfA = gam + 512;  // beta_m exp(gamma_m - gamma_{first row of m's 16-block})
    float* alp = gam + 640;  // per-token decay exp(g_t) = exp(gamma_t - gamma_{t-1})
    float* rq = gam + 768;   // FRONT only: scale / |q_i|
    float* rk = gam + 832;   // FRONT only: 1 / |k_j|
    float* tmp = gam + 896;
    uint64_t* bar_load = reinterpret_cast<uint64_t*>(smem + IBAR);
    uint64_t* bar_mma1 = bar_load + 1;
    uint64_t* bar_mma2 = bar_load + 2;
    uint64_t* bar_step = bar_load + 3;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + IBAR + 40);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + IBAR + 48);

    if (tid == 0) {
        mbar_init(bar_load, 1);
        mbar_init(bar_mma1, 1);
        mbar_init(bar_mma2, 1);
        mbar_init(bar_step, 1);
        *abort_flag = 0;
        mbar_fence_init();
    }
    if (warp == 0) {
        __syncwarp();
        tmem_alloc(tmem_slot, ITM_COLS);
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;
    const uint32_t lane_addr = tmem_base + ((uint32_t)(warp * 32) << 16);
    const uint32_t sb = smem_u32(smem);
    bool ok = true;

    if (warp == 0) {
        if (elect_one()) {
            prefetch_tensormap(&map_q);
            prefetch_tensormap(&map_k);
            mbar_expect_tx(bar_load, 32768);
            tma_load_3d(smem + IQ_LO, &map_q, bar_load, 0, hq, t0);
            tma_load_3d(smem + IQ_HI, &map_q, bar_load, 64, hq, t0);
            tma_load_3d(smem + IK_LO, &map_k, bar_load, 0, hq, t0);
            tma_load_3d(smem + IK_HI, &map_k, bar_load, 64, hq, t0);
        }
        __syncwarp();
    }
    // ---- gates of both heads while the tiles are in flight: gamma = inclusive cumsum of g (fp32),
    //      beta; both zero beyond len
    {
        float x = 0.f, b = 0.f;
        if (head_ok && i < len) {
            x = __ldg(g + (size_t)(t0 + i) * Hv + h);
            b = __ldg(beta + (size_t)(t0 + i) * Hv + h);
            // with A_log given, g/beta are the raw gate inputs a and b
            if (A_log) raw_gates(x, b, __ldg(A_log + h), __ldg(dt_bias + h), x, b);
        }
        alp[tid] = __expf(x);
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const float y = __shfl_up_sync(0xffffffffu, x, o);
            if (lane >= o) x += y;
        }
        if ((warp & 1) == 0 && lane == 31) tmp[hh] = x;
        __syncthreads();
        if (warp & 1) x += tmp[hh];
        gam[tid] = x;
        bet[tid] = b;
        Gam[tid] = __expf(x);
        __syncthreads();
        // The decay exp(gamma_i - gamma_j) between a row and a column of DIFFERENT 16-blocks factors
        // through the block boundary with both exponents <= 0, so phase A needs one exp per
        // (row, block) instead of one per element.
        cfP[tid] = __expf(gam[(tid & ~15) | 15] - x);
        cfA[tid] = b * __expf(x - gam[tid & ~15]);
    }
    if (warp == 0) {
        ok = mbar_wait_all(bar_load, 0, abort_flag);
        if (ok) {
            if (len < kChunk) {
                // Ragged chunk: the 64-row TMA boxes also brought the first tokens of the next sequence.
                // Their products only ever meet exact zeros (beta = 0, masked decay), which does not stop a
                // NaN or Inf, so rows >= len of the four tiles are cleared before anything reads them
                // (128 bytes per row in each tile; the swizzle permutes inside a row).
#pragma unroll 1
                for (int tile = 0; tile < 4; ++tile)
                    for (uint32_t o = (uint32_t)len * 128u + lane * 16u; o < 8192u; o += 512u)
                        *reinterpret_cast<uint4*>(smem + tile * 8192 + o) = make_uint4(0u, 0u, 0u, 0u);
                fence_proxy_async_smem();  // generic-proxy stores before the tensor cores' reads
                __syncwarp();
            }
            tc_fence_after_sync();
            constexpr uint32_t ID1 = umma_idesc_bf16(128, 64, false, false, false);
            const uint64_t dA0 = umma_desc(sb + IQ_LO, 16, 1024), dA1 = umma_desc(sb + IQ_HI, 16, 1024);
            const uint64_t dB0 = umma_desc(sb + IK_LO, 16, 1024), dB1 = umma_desc(sb + IK_HI, 16, 1024);
#pragma unroll
            for (int ks = 0; ks < 4; ++ks) umma_bf16_ss_warp(tmem_base + ITM_D1, dA0 + ks * 2, dB0 + ks * 2, ID1, ks > 0);
#pragma unroll
            for (int ks = 0; ks < 4; ++ks) umma_bf16_ss_warp(tmem_base + ITM_D1, dA1 + ks * 2, dB1 + ks * 2, ID1, 1);
            umma_commit_warp(bar_mma1);
        }
    }
    if constexpr (FRONT) {
        // while MMA1 runs: thread r < 64 takes row r of Q, thread 64 + r row r of K.  A row is 128 bytes
        // in each of the two tiles; the 128-byte swizzle only permutes its 16-byte pieces, and a sum
        // over all of them does not care (pieces taken in a rotated order to spread the banks).
        // (only warp 0 polls the load barrier: the others learn of the tiles through the CTA barrier)
        float f = (tid < 64) ? fr.scale : 1.f;
        if (fr.l2norm) ok = __syncthreads_and(ok);
        if (fr.l2norm && ok) {
            const uint8_t* lo = smem + (tid < 64 ? IQ_LO : IK_LO) + (uint32_t)(tid & 63) * 128u;
            const uint8_t* hi = smem + (tid < 64 ? IQ_HI : IK_HI) + (uint32_t)(tid & 63) * 128u;
            float ss = 0.f;
#pragma unroll
            for (int cc = 0; cc < 8; ++cc) {
                const int ch = (cc + tid) & 7;
                const uint4 a = *reinterpret_cast<const uint4*>(lo + ch * 16);
                const uint4 b = *reinterpret_cast<const uint4*>(hi + ch * 16);
                const uint32_t w[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
#pragma unroll
                for (int u = 0; u < 8; ++u) {
                    float x0, x1;
                    unpack_bf16x2(w[u], x0, x1);
                    ss = fmaf(x0, x0, ss);
                    ss = fmaf(x1, x1, ss);
                }
            }
            f *= rsqrtf(ss + kNormEps);
        }
        rq[tid] = f;  // rq and rk are adjacent: thread 64 + r writes rk[r]
        __syncthreads();
        cfP[tid] *= rk[i];
    }
    if (warp == 0 && ok) ok = mbar_wait_all(bar_mma1, 0, abort_flag);  // only this warp polls; the others park at the barrier
    ok = __syncthreads_and(ok);
    if (ok) {
        tc_fence_after_sync();
        // per-token scalars of this thread's (head, row)
        if (head_ok) {
            float* wsS = reinterpret_cast<float*>(ws + L.off_scal + ((size_t)c * Hv + h) * kScalBytes);
            wsS[i] = FRONT ? Gam[tid] * rq[i] : Gam[tid];
            const float e_i = __expf(gam[hh * 64 + len - 1] - gam[tid]);
            wsS[64 + i] = FRONT ? e_i * rk[i] : e_i;
            if (i == 0) wsS[128] = Gam[hh * 64 + len - 1];
        }
        // ---- phase A, sixteen columns at a time (rolled: long straight-line code runs at
        //      instruction-fetch speed).  Rows 0-63 of the accumulator are Q K^T -> P; rows 64-127 are
        //      K K^T, and row j of it (symmetric) yields column j of A:
        //          A[m][j] = beta_m exp(gamma_m - gamma_j) (K K^T)_jm   for m > j, else 0
        //      (the exponent is <= 0).  Column j is row (j % 16) of B tile (j / 16); its part inside
        //      the diagonal block goes to the fp32 diagonal blocks instead.
        {
            const int row = tid & 63;
            const int jb_own = row >> 4;
#pragma unroll 1
            for (int q4 = 0; q4 < 4; ++q4) {
                uint32_t r[16];
                tmem_ld16(lane_addr + ITM_D1 + q4 * 16, r);
                tmem_ld_wait();
                // A side: the two half warps own different diagonal blocks (16 j_own and the one right of it).
                // Both are handled in the same iteration, the first of the warp's two, so that the
                // per-element code runs once for all 32 lanes instead of once per half warp: the upper half
                // takes its sixteen columns from a second load.
                const int wbA = (row >> 5) * 2;
                uint32_t xd[16];
                if (tid >= 64 && q4 == wbA) {
                    uint32_t r2[16];
                    tmem_ld16(lane_addr + ITM_D1 + (q4 + 1) * 16, r2);
                    tmem_ld_wait();
#pragma unroll
                    for (int ml = 0; ml < 16; ++ml) xd[ml] = (row & 16) ? r2[ml] : r[ml];
                }
#pragma unroll 1
                for (int e = 0; e < 2; ++e) {
                    const float* gm = gam + e * 64 + q4 * 16;
                    const float gi = gam[e * 64 + row];
                    if (tid < 64) {
                        if (e >= nh) continue;
                        // P row: (Q K^T)_ij exp(gamma_i - gamma_j) for j <= i (difference masked before exp)
                        uint8_t* wsP = ws + L.off_P + ((size_t)c * Hv + hq * G + 2 * p + e) * kPBytes;
                        float pv[16];
                        // Branch conditions are uniform over the warp (its 32 rows span two 16-blocks):
                        // column blocks left of both use the factored decay; the two blocks that hold a
                        // diagonal block for one half of the warp take the per-element form for all 32 lanes.
                        const int wb2 = (row >> 5) * 2;
                        if (q4 < wb2) {
                            float rf = (row < len) ? __expf(gi - gam[e * 64 + q4 * 16 + 15]) : 0.f;
                            if constexpr (FRONT) rf *= rq[row];
                            float cf[16];
                            ld16(cfP + e * 64 + q4 * 16, cf);
#pragma unroll
                            for (int jl = 0; jl < 16; ++jl) pv[jl] = __uint_as_float(r[jl]) * (rf * cf[jl]);
                        } else if (q4 <= wb2 + 1) {
                            // exp(gamma_i - gamma_j) from the right end of the block by a running product
                            // of the per-token decays (one exp per row instead of sixteen; every factor
                            // is <= 1, so nothing can overflow): acc = exp(gamma_i - gamma_j) once j <= i
                            float acc = __expf(fminf(gi - gm[15], 0.f));  // 1 for rows inside the block
                            float al[16], kq[16];
                            ld16(alp + e * 64 + q4 * 16, al);
                            if constexpr (FRONT) {
                                ld16(rk + q4 * 16, kq);
                                const float rqi = rq[row];
#pragma unroll
                                for (int x = 0; x < 16; ++x) kq[x] *= rqi;
                            }
#pragma unroll
                            for (int jl = 15; jl >= 0; --jl) {
                                const bool on = (q4 * 16 + jl <= row) && (row < len);
                                if constexpr (FRONT)
                                    pv[jl] = on ? __uint_as_float(r[jl]) * (acc * kq[jl]) : 0.f;
                                else
                                    pv[jl] = on ? __uint_as_float(r[jl]) * acc : 0.f;
                                acc = on ? acc * al[jl] : acc;
                            }
                        } else {
#pragma unroll
                            for (int jl = 0; jl < 16; ++jl) pv[jl] = 0.f;
                        }
                        {   // the sixteen columns are two adjacent 16-byte chunks of the row: one 32-byte store
                            uint32_t pk[8];
#pragma unroll
                            for (int q2 = 0; q2 < 8; ++q2) pk[q2] = pack_bf16x2(pv[q2 * 2], pv[q2 * 2 + 1]);
                            st_swizzled_pair(wsP, (uint32_t)row, (uint32_t)q4, make_uint4(pk[0], pk[1], pk[2], pk[3]),
                                             make_uint4(pk[4], pk[5], pk[6], pk[7]));
                        }
                    } else if (q4 == wbA || q4 > jb_own) {
                        float a[16];
                        const bool diag = q4 == wbA;
                        if (diag) {
                            float bm[16], al[16];
                            ld16(bet + e * 64 + jb_own * 16, bm);
                            // exp(gamma_m - gamma_j), m > j, as the running product of the per-token decays
                            ld16(alp + e * 64 + jb_own * 16, al);
                            float acc = FRONT ? rk[row] * rk[row] : 1.f;
#pragma unroll
                            for (int ml = 0; ml < 16; ++ml) {
                                const bool on = jb_own * 16 + ml > row;
                                acc = on ? acc * al[ml] : acc;
                                a[ml] = on ? bm[ml] * acc * __uint_as_float(xd[ml]) : 0.f;
                            }
                        } else {
                            float rf = __expf(gam[e * 64 + q4 * 16] - gi);
                            if constexpr (FRONT) rf *= rk[row] * rk[row];
                            float cf[16];
                            ld16(cfA + e * 64 + q4 * 16, cf);
#pragma unroll
                            for (int ml = 0; ml < 16; ++ml) a[ml] = (rf * cf[ml]) * __uint_as_float(r[ml]);
                        }
                        if (diag) {
                            // stored by row m: the solve reads, for one m, the run of columns j < m as float4s
                            float* dg = reinterpret_cast<float*>(smem + IDG) + (e * 4 + jb_own) * 256 + (row & 15);
#pragma unroll
                            for (int ml = 0; ml < 16; ++ml) dg[ml * 16] = a[ml];
                        } else {
                            const uint32_t n = (uint32_t)(e * 16 + (row & 15));
#pragma unroll
                            for (int half = 0; half < 2; ++half) {
                                uint32_t hi4[4], lo4[4];
#pragma unroll
                                for (int q2 = 0; q2 < 4; ++q2)
                                    split_bf16x2(a[half * 8 + q2 * 2], a[half * 8 + q2 * 2 + 1], hi4[q2], lo4[q2]);
                                const uint32_t off = swz(n, q4 * 2 + half);
                                *reinterpret_cast<uint4*>(smem + intra_btile(jb_own, 0) + off) = make_uint4(hi4[0], hi4[1], hi4[2], hi4[3]);
                                *reinterpret_cast<uint4*>(smem + intra_btile(jb_own, 1) + off) = make_uint4(lo4[0], lo4[1], lo4[2], lo4[3]);
                            }
                        }
                    }
                }
            }
        }
        fence_proxy_async_smem();
        tc_fence_before_sync();
        __syncthreads();  // B tiles and diagonal blocks complete; the accumulator of MMA1 is dead from here on
        tc_fence_after_sync();
        if constexpr (FRONT) {
            // the tables of the emission below, rescaled in place (phase A is done with them; the solve's
            // barriers come before their next use): beta_j / rk_j and Gamma_j rk_j
            bet[tid] = bet[tid] / rk[i];
            Gam[tid] *= rk[i];
        }

        // ---- the blocked solve: z[jb][.] = columns 16 jb .. 16 jb + 15 of row i of T
        float z[4][16];
        constexpr uint32_t IDS = umma_idesc_bf16(128, 32, false, false, false);
#pragma unroll
        for (int jb = 3; jb >= 0; --jb) {
            // T is lower triangular: a warp whose 32 rows all lie above column block jb (rows 0-31 of a head
            // for blocks 2 and 3) has nothing but zeros there and skips the block's loads and arithmetic
            const bool dead = jb > 2 * (warp & 1) + 1;
            if (dead) {
#pragma unroll
                for (int jj = 0; jj < 16; ++jj) z[jb][jj] = 0.f;
            } else {
            float rhs[16];
#pragma unroll
            for (int jj = 0; jj < 16; ++jj) rhs[jj] = ((16 * jb + jj) == i) ? 1.f : 0.f;
            if (jb < 3) {  // subtract sum_{mb > jb} y_blk(mb) A[mb][jb], accumulated by the tensor cores
                uint32_t d[16];
                tmem_ld16(lane_addr + ITM_ACC + hh * 16, d);
                tmem_ld_wait();
#pragma unroll
                for (int jj = 0; jj < 16; ++jj) rhs[jj] -= __uint_as_float(d[jj]);
            }
            // diagonal block, column by column from the right: once z_mm is known its contribution is
            // pushed to every column left of it (independent FMAs, no long chain)
            // (entries at and right of the diagonal are stored as zeros, so whole float4s are applied)
            const float4* dg = reinterpret_cast<const float4*>(smem + IDG) + (hh * 4 + jb) * 64;
#pragma unroll
            for (int mm = 15; mm >= 0; --mm) {
                const float zm = rhs[mm];
                z[jb][mm] = zm;
#pragma unroll
                for (int q = 0; q < (mm + 3) / 4; ++q) {
                    const float4 d = dg[mm * 4 + q];
                    rhs[4 * q + 0] = fmaf(-d.x, zm, rhs[4 * q + 0]);
                    rhs[4 * q + 1] = fmaf(-d.y, zm, rhs[4 * q + 1]);
                    rhs[4 * q + 2] = fmaf(-d.z, zm, rhs[4 * q + 2]);
                    rhs[4 * q + 3] = fmaf(-d.w, zm, rhs[4 * q + 3]);
                }
            }
            }
            if (jb > 0) {
                // this block becomes a K step of the A operand (bf16 hi + lo) for the remaining steps
                uint32_t zh[8], zl[8];
#pragma unroll
                for (int q = 0; q < 8; ++q) split_bf16x2(z[jb][2 * q], z[jb][2 * q + 1], zh[q], zl[q]);
                tmem_st8(lane_addr + ITM_YHI + jb * 8, zh);
                tmem_st8(lane_addr + ITM_YLO + jb * 8, zl);
                tmem_st_wait();
                tc_fence_before_sync();
                __syncthreads();
                if (warp == 0) {
                    tc_fence_after_sync();
                    const int nj = jb - 1;
                    const uint64_t dBh = umma_desc(sb + intra_btile(nj, 0), 16, 1024);
                    const uint64_t dBl = umma_desc(sb + intra_btile(nj, 1), 16, 1024);
                    const uint32_t tacc = tmem_base + ITM_ACC;
#pragma unroll
                    for (int mb = 3; mb >= jb; --mb) {
                        const uint32_t ah = tmem_base + ITM_YHI + mb * 8, al = tmem_base + ITM_YLO + mb * 8;
                        umma_bf16_ts_warp(tacc, ah, dBh + mb * 2, IDS, mb < 3);
                        umma_bf16_ts_warp(tacc, ah, dBl + mb * 2, IDS, 1);
                        umma_bf16_ts_warp(tacc, al, dBh + mb * 2, IDS, 1);
                    }
                    umma_commit_warp(bar_step);
                    ok = mbar_wait_all(bar_step, (uint32_t)((3 - jb) & 1), abort_flag);
                }
                ok = __syncthreads_and(ok);
                if (!ok) break;
                tc_fence_after_sync();
            }
        }
        // The images that go to the workspace (T' hi, T' lo, W) are row-major with 128-byte rows and a thread
        // owns a row, so a direct 16-byte store instruction would touch 32 different lines.  They are built
        // in shared memory instead (conflict-free with the swizzle) and leave as bulk copies: T' hi now, over
        // the diagonal blocks and the B tiles of column block 2 (hence the barrier: the last solve step of
        // other warps may still be reading the diagonal blocks); T' lo and W after MMA2, when the rest is free.
        uint8_t* wsA = ws + L.off_A + ((size_t)c * Hv + h) * kABytes;
        uint8_t* stHi = smem + (hh ? IBT2 : IDG);
        __syncthreads();
        if (ok) {
            // ---- T' = T diag(beta) (bf16 hi here, lo below); T'' = T' diag(Gamma) -> smem A operand (bf16),
            //      over the B tiles, which the last step's MMAs have finished reading
            const float* bt = bet + hh * 64;
            const float* Gm = Gam + hh * 64;
            const float rki = FRONT ? rk[i] : 1.f;
#pragma unroll
            for (int cp = 0; cp < 4; ++cp) {  // sixteen columns at a time
                uint32_t h1[8], l1[8], h2[8];
                float b16[16], G16[16];
                ld16(bt + cp * 16, b16);
                ld16(Gm + cp * 16, G16);
#pragma unroll
                for (int q2 = 0; q2 < 8; ++q2) {
                    // (FRONT: z is a row of the similar system, the tables hold beta / rk and Gamma rk)
                    const float a0 = (FRONT ? z[cp][q2 * 2] * rki : z[cp][q2 * 2]) * b16[q2 * 2];
                    const float a1 = (FRONT ? z[cp][q2 * 2 + 1] * rki : z[cp][q2 * 2 + 1]) * b16[q2 * 2 + 1];
                    z[cp][q2 * 2] = a0;  // kept for the lo parts below
                    z[cp][q2 * 2 + 1] = a1;
                    split_bf16x2(a0, a1, h1[q2], l1[q2]);
                    h2[q2] = pack_bf16x2(a0 * G16[q2 * 2], a1 * G16[q2 * 2 + 1]);
                }
                *reinterpret_cast<uint4*>(stHi + swz(i, 2 * cp)) = make_uint4(h1[0], h1[1], h1[2], h1[3]);
                *reinterpret_cast<uint4*>(stHi + swz(i, 2 * cp + 1)) = make_uint4(h1[4], h1[5], h1[6], h1[7]);
                *reinterpret_cast<uint4*>(smem + IT2 + swz(tid, 2 * cp)) = make_uint4(h2[0], h2[1], h2[2], h2[3]);
                *reinterpret_cast<uint4*>(smem + IT2 + swz(tid, 2 * cp + 1)) = make_uint4(h2[4], h2[5], h2[6], h2[7]);
            }
            fence_proxy_async_smem();
            tc_fence_before_sync();
        }
        __syncthreads();
        const bool storer = ok && i == 0 && head_ok;  // threads 0 and 64: one per head
        if (storer) {
            bulk_store(wsA, stHi, 8192);
            bulk_store_commit();
        }
        // ---- MMA2: W (both heads) = [T''_a ; T''_b] K, K read MN-major from the TMA tiles
        if (ok && warp == 0) {
            tc_fence_after_sync();
            constexpr uint32_t ID2 = umma_idesc_bf16(128, 128, false, true, false);
            const uint64_t dTh = umma_desc(sb + IT2, 16, 1024);
            const uint64_t dK = umma_desc(sb + IK_LO, IK_HI - IK_LO, 1024);
#pragma unroll
            for (int ks = 0; ks < 4; ++ks) umma_bf16_ss_warp(tmem_base + ITM_D2, dTh + ks * 2, dK + ks * 128, ID2, ks > 0);
            umma_commit_warp(bar_mma2);
            ok = mbar_wait_all(bar_mma2, 0, abort_flag);
        }
        if (storer) bulk_store_wait_read();  // the staging of T' hi is written again below
        ok = __syncthreads_and(ok);
        if (ok) {
            // ---- T' lo (the bf16 remainder, split again from the values kept in registers) -> staging over
            //      the T'' operand, which MMA2 has finished reading
            uint8_t* stLo = smem + IT2 + (uint32_t)hh * 8192u;
#pragma unroll
            for (int cp = 0; cp < 4; ++cp) {
                uint32_t h1[8], l1[8];
#pragma unroll
                for (int q2 = 0; q2 < 8; ++q2) split_bf16x2(z[cp][q2 * 2], z[cp][q2 * 2 + 1], h1[q2], l1[q2]);
                *reinterpret_cast<uint4*>(stLo + swz(i, 2 * cp)) = make_uint4(l1[0], l1[1], l1[2], l1[3]);
                *reinterpret_cast<uint4*>(stLo + swz(i, 2 * cp + 1)) = make_uint4(l1[4], l1[5], l1[6], l1[7]);
            }
        }
    }
    if (ok) {
        tc_fence_after_sync();
        // ---- W row i of head h (K-major B operand image: two [64][64] tiles) -> staging over the q/k tiles
        uint8_t* stW = smem + (uint32_t)hh * 16384u;
#pragma unroll 1
        for (int b = 0; b < 4; ++b) {
            uint32_t r[32];
            tmem_ld32(lane_addr + ITM_D2 + b * 32, r);
            tmem_ld_wait();
#pragma unroll
            for (int cc = 0; cc < 4; ++cc) {
                uint4 o;
                o.x = pack_bf16x2(__uint_as_float(r[cc * 8 + 0]), __uint_as_float(r[cc * 8 + 1]));
                o.y = pack_bf16x2(__uint_as_float(r[cc * 8 + 2]), __uint_as_float(r[cc * 8 + 3]));
                o.z = pack_bf16x2(__uint_as_float(r[cc * 8 + 4]), __uint_as_float(r[cc * 8 + 5]));
                o.w = pack_bf16x2(__uint_as_float(r[cc * 8 + 6]), __uint_as_float(r[cc * 8 + 7]));
                *reinterpret_cast<uint4*>(stW + (b >> 1) * 8192 + swz(i, (b & 1) * 4 + cc)) = o;
            }
        }
        fence_proxy_async_smem();
    }
    __syncthreads();
    if (ok && i == 0 && head_ok) {
        uint8_t* wsA = ws + L.off_A + ((size_t)c * Hv + h) * kABytes;
        bulk_store(wsA + 8192, smem + IT2 + (uint32_t)hh * 8192u, 8192);  // T' lo
        bulk_store(wsA + 16384, smem + (uint32_t)hh * 16384u, 16384);     // W
        bulk_store_commit();
        bulk_store_wait_read();  // shared memory must outlive the copy's reads
    }

    if (*abort_flag && tid == 0) atomicExch(reinterpret_cast<int*>(ws), kStatusTimeout);
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 0) {
        __syncwarp();
        tmem_dealloc(tmem_base, ITM_COLS);
    }
}

cudaError_t launch_prefill_prep(const int32_t* cu_seqlens, int num_seqs, int total_tokens, uint8_t* ws,
                                const WsLayout& L, cudaStream_t st) {
    gdn_prefill_prep_kernel<<<1, 256, 0, st>>>(cu_seqlens, num_seqs, total_tokens, reinterpret_cast<int*>(ws),
                                               reinterpret_cast<int*>(ws + L.off_chunk_off),
                                               reinterpret_cast<int4*>(ws + L.off_seq_order),
                                               reinterpret_cast<int4*>(ws + L.off_chunk_info), L.nc_max);
    return cudaGetLastError();
}

cudaError_t launch_prefill_intra(const CUtensorMap& mq, const CUtensorMap& mk, const float* g, const float* beta,
                                 const float* A_log, const float* dt_bias, uint8_t* ws, const WsLayout& L, int Hqk,
                                 int Hv, const int32_t* cu_if_no_table, int num_seqs, int total_tokens, QkFront fr,
                                 cudaStream_t st) {
    static bool attr_done[64];
    if (cudaError_t e = set_attrs_once(attr_done, [] {
            cudaError_t e2 = cudaFuncSetAttribute(gdn_prefill_intra_kernel<false>,
                                                  cudaFuncAttributeMaxDynamicSharedMemorySize, kIntraSmem);
            if (e2 == cudaSuccess)
                e2 = cudaFuncSetAttribute(gdn_prefill_intra_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                          kIntraSmem);
            return e2;
        }))
        return e;
    const int G = Hv / Hqk;
    dim3 grid(L.nc_max, Hqk * ((G + 1) / 2));
    if (fr.active())
        gdn_prefill_intra_kernel<true><<<grid, kIntraThreads, kIntraSmem, st>>>(
            mq, mk, g, beta, A_log, dt_bias, ws, L, Hqk, Hv, cu_if_no_table, num_seqs, total_tokens, fr);
    else
        gdn_prefill_intra_kernel<false><<<grid, kIntraThreads, kIntraSmem, st>>>(
            mq, mk, g, beta, A_log, dt_bias, ws, L, Hqk, Hv, cu_if_no_table, num_seqs, total_tokens, fr);
    return cudaGetLastError();
}

}  // namespace gdn
