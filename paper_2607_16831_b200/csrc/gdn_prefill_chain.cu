// Inter-chunk ("chain") kernel of the chunked WY / UT-transform prefill.
//
// One CTA per (sequence, value head) walks the sequence's 64-token chunks in order.  With
// S the fp32 state entering a chunk ([dv][dk], row v = tensor-memory lane v) and the chunk
// summaries T', W, P and scalars from the intra-chunk kernel:
//
//   Delta^T = V^T T'^T - S W^T            [128 x 64]   (G1: T' hi+lo, then G2A on the chain)
//   Oa^T    = S Q^T                        [128 x 64]   (G2B, off the chain)
//   Ob^T    = Delta^T P^T                  [128 x 64]   (G3A, off the chain)
//   S      <- Gamma_L S + (e o Delta)^T K  [128 x 128]  (G3B on the chain, hi+lo)
//   o_i     = Gamma_i Oa^T[:,i] + Ob^T[:,i]
//
// All products are tcgen05.mma with fp32 accumulators in tensor memory.  The operands that
// the chain itself produces (the bf16 copy of S, Delta^T and its decayed hi/lo copies) are
// written back to tensor memory and read from there as the A operand, so they never touch
// shared memory; an MMA's time here is set by the operand bytes it pulls from shared memory,
// and this halves them.  The B operands are 128-byte-swizzled shared-memory tiles: q/k/v
// arrive by TMA from the caller's tensors, the chunk summaries by bulk copies of
// pre-swizzled images, two stages deep.  The fp32 state stays in tensor memory for the
// whole sequence.  Warp roles:
//   warp  0     issues every MMA (one elected lane)
//   warp  1     issues every TMA / bulk copy, one chunk ahead of the MMAs
//   warps 4-7   chain: drain Delta^T -> bf16 operands; drain S -> bf16 operand + decayed fp32 back
//   warps 8-11  output: drain Oa/Ob -> bf16 out
//               (and, when the last chunk is ragged, clears the rows of its V and K tiles that lie
//               beyond the sequence: the 64-row TMA box also fetched the first tokens of the next one)
//   (warps 2, 3 idle: a role that touches tensor memory needs warp % 4 = its lane quarter)
// Measured with clock stamps: a chunk step is ~3150 clocks and stays there when the
// off-chain products are moved around; the drain of Delta^T takes ~590 clocks when no other MMA is issued or
// executing at the time and 100-300 more when the eight S Q^T MMAs are (in a microbenchmark queued MMAs do
// not delay another warp's tcgen05.ld / st at all, so this is contention inside the kernel, part of it the
// issuer sharing a scheduler with chain warp 0).
// Hand-offs are mbarriers; every wait is bounded and failure unwinds through an abort flag.
//
// With `segs` > 1 a sequence is cut into that many runs of chunks and the runs advance at the same
// time (the scan in gdn_prefill_scan.cu joins them).  Run 0 is the recurrence itself.  Every later
// run has two CTAs per head: one starts from the zero state (its outputs and final state are the
// parts that do not depend on the state entering the run), one starts from the identity with
// v = 0 (its "outputs" are the queries carried back to the start of the run, M_t q_t, and its
// final state is the run's transition matrix).
#include "gdn_prefill_ws.cuh"
#include "gdn_sm100.cuh"

namespace gdn {
using namespace sm100;

constexpr int kChainThreads = 384;
constexpr int kIssuerWarp = 0, kProducerWarp = 1, kChainWarp0 = 4, kOutputWarp0 = 8;  // warps 2, 3 idle

// One arrival per warp: 128 threads arriving on the same mbarrier are serialised by the
// shared-memory unit (~500 clk before the waiter sees the phase complete); the lanes are ordered
// by the warp barrier and lane 0 arrives for all of them.
__device__ __forceinline__ void warp_arrive(uint64_t* bar) {
    __syncwarp();
    if ((threadIdx.x & 31) == 0) mbar_arrive(bar);
}

// shared-memory map (bytes from a 1024-byte aligned base): two stages of per-chunk operands
constexpr uint32_t ST_T = 0;          // T'hi 8K | T'lo 8K   (bulk copy, together with W)
constexpr uint32_t ST_W = 16384;      // W: 2 tiles [64][64]
constexpr uint32_t ST_V = 32768;      // V tile: 2 x [64 tokens][64]  (TMA)
constexpr uint32_t ST_Q = 49152;      // Q tile                        (TMA)
constexpr uint32_t ST_K = 65536;      // K tile                        (TMA)
constexpr uint32_t ST_P = 81920;      // P [64][64]                    (bulk copy)
constexpr uint32_t kStageBytes = 90112;
constexpr uint32_t OFF_OST = 2 * kStageBytes;          // output staging tile [64 tokens][128 v] bf16              16 KB
constexpr uint32_t OFF_BAR = OFF_OST + 16384;          // mbarriers, TMEM slot, abort flag
constexpr uint32_t kChainSmem = OFF_BAR + 256 + 1024;  // + slack for the manual 1024-byte alignment
constexpr uint32_t kTxA = 32768 + 16384 + 16384;       // T'+W, V, Q
constexpr uint32_t kTxB = 16384 + 8192;                // K, P
// tensor-memory columns (32-bit each)
constexpr uint32_t TM_S = 0;        // fp32 state                    128
constexpr uint32_t TM_DELTA = 128;  // fp32 Delta^T accumulator       64
constexpr uint32_t TM_OA = 192;     // fp32 S Q^T                     64
constexpr uint32_t TM_OB = 256;     // fp32 Delta^T P^T               64
constexpr uint32_t TM_SHI = 320;    // bf16 S      (A operand)        64
constexpr uint32_t TM_DL = 384;     // bf16 Delta^T (A operand)       32
constexpr uint32_t TM_DTH = 416;    // bf16 (e o Delta)^T hi          32
constexpr uint32_t TM_DTL = 448;    // bf16 (e o Delta)^T lo          32
constexpr uint32_t TM_COLS = 512;

enum { B_FULL_A0 = 0, B_FULL_A1, B_FULL_B0, B_FULL_B1, B_FREE0, B_FREE1, B_DELTA, B_STATE, B_O, B_DW, B_SHI, B_STM, B_OFREE, B_DL, B_CLEAN_A, B_CLEAN_B, B_INIT, B_INIT_DONE, B_COUNT };

__global__ void __launch_bounds__(kChainThreads, 1)
gdn_prefill_chain_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                         const __grid_constant__ CUtensorMap map_v, const __grid_constant__ CUtensorMap map_s,
                         const float* initial_state,
                         uint16_t* __restrict__ out, float* final_state, uint8_t* __restrict__ ws, WsLayout L,
                         int Hqk, int Hv, int segs, ChainPartial part) {
    // CTAs are handed out longest sequence first; within a sequence: run 0, then (zero, identity) per run.
    // Partial mode (part.H set, segs = 1): every sequence is one run that is walked from the zero state
    // and from the identity, results to the caller's H, P and qt.
    const bool partial = part.H != nullptr;
    const int per_seq = partial ? 2 : 2 * segs - 1;
    const int h = blockIdx.x % Hv, unit = blockIdx.x / Hv;
    // one record per sequence (sequence, its first chunk, its first token, its length): everything this CTA
    // needs to find its work comes from this single load
    const int4 rec = reinterpret_cast<const int4*>(ws + L.off_seq_order)[unit / per_seq];
    const int n = rec.x;
    const int seg = partial ? 0 : (unit % per_seq + 1) >> 1;
    const bool ident = partial ? (unit % per_seq) == 1
                               : (seg > 0 && ((unit % per_seq) & 1) == 0);  // identity start, v = 0
    const int hq = h / (Hv / Hqk);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + OFF_BAR);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + OFF_BAR + 8 * B_COUNT);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + OFF_BAR + 8 * B_COUNT + 8);

    // chunk slots of the sequence, clamped like the chunk table itself (a malformed cu_seqlens cannot
    // send the CTA outside the workspace)
    const int seq_chunks = max(0, min((rec.w + kChunk - 1) / kChunk, L.nc_max - rec.y));
    int seg_first, nchunks;
    segment_range(seq_chunks, segs, seg, seg_first, nchunks);
    const int c_begin = rec.y + seg_first;

    if (nchunks <= 0) {  // empty sequence: the state passes through; empty run: nothing to do
        if (partial && tid < kD) {  // H = 0, P = I
            float* dst = (ident ? part.P : part.H) + ((size_t)n * Hv + h) * kD * kD + (size_t)tid * kD;
            for (int j = 0; j < kD; j += 4)
                *reinterpret_cast<float4*>(dst + j) =
                    make_float4((ident && tid == j) ? 1.f : 0.f, (ident && tid == j + 1) ? 1.f : 0.f,
                                (ident && tid == j + 2) ? 1.f : 0.f, (ident && tid == j + 3) ? 1.f : 0.f);
        } else if (seg == 0 && final_state && tid < kD) {
            const size_t sb0 = ((size_t)n * Hv + h) * kD * kD + (size_t)tid * kD;
            for (int j = 0; j < kD; j += 4) {
                float4 x = make_float4(0.f, 0.f, 0.f, 0.f);
                if (initial_state) x = *reinterpret_cast<const float4*>(initial_state + sb0 + j);
                *reinterpret_cast<float4*>(final_state + sb0 + j) = x;
            }
        }
        return;
    }
    // chunks of one sequence are consecutive: chunk ci of this run starts at t0_first + 64 ci
    const int t0_first = rec.z + seg_first * kChunk;
    const int t_end = min(rec.z + rec.w, t0_first + nchunks * kChunk);
    // Only the last chunk of a run can be ragged.  Its 64-row TMA boxes reach past the sequence into
    // the next one; those rows meet exact zeros in every product, which is not enough when they hold
    // NaN or Inf, so they are cleared in shared memory before the tensor cores see them.
    const int tail_len = t_end - (t0_first + (nchunks - 1) * kChunk);
    const bool ragged = tail_len < kChunk;
    // where this CTA's state comes from and where its results go
    const size_t state_off = ((size_t)n * Hv + h) * kD * kD;
    const float* init_ptr = (!partial && seg == 0 && initial_state) ? initial_state + state_off : nullptr;
    float* fin_ptr = final_state ? final_state + state_off : nullptr;
    if (partial)
        fin_ptr = (ident ? part.P : part.H) + state_off;
    else if (segs > 1)
        fin_ptr = reinterpret_cast<float*>(
            ws + seg_block_offset(L, n, seg == 0 ? 1 : seg, h, Hv, seg == 0 ? kSegSin : (ident ? kSegP : kSegH)));
    uint16_t* out_ptr = ident ? (partial ? part.qt : reinterpret_cast<uint16_t*>(ws + L.off_qt)) : out;

    if (warp >= kChainWarp0 && warp < kChainWarp0 + 4 && (tid & 31) == 0)
        prefetch_l2(ws + L.off_scal + ((size_t)c_begin * Hv + h) * kScalBytes + 512);
    if (tid == 0) {
        for (int i = 0; i < B_COUNT; ++i) {
            const bool many = (i == B_DW || i == B_SHI || i == B_STM || i == B_OFREE || i == B_DL || i == B_INIT_DONE);
            mbar_init(bars + i, many ? 4u : 1u);  // one arrival per warp of the arriving role
        }
        *abort_flag = 0;
        mbar_fence_init();
    }
    if (warp == kIssuerWarp) {
        __syncwarp();
        tmem_alloc(tmem_slot, TM_COLS);
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;

    auto scal_ptr = [&](int c) {
        return reinterpret_cast<const float*>(ws + L.off_scal + ((size_t)c * Hv + h) * kScalBytes);
    };

    if (warp == kIssuerWarp) {
        // =========================================================== issuer: MMA
        // The whole warp runs this loop in lock step; one elected lane issues each MMA.  Values that
        // feed the MMA operands are broadcast from lane 0 so that the compiler knows they are
        // warp-uniform and keeps descriptors and addresses in uniform registers.
        {
            const uint32_t sb = __shfl_sync(0xffffffffu, smem_u32(smem), 0);
            const uint32_t tmem_base_u = __shfl_sync(0xffffffffu, tmem_base, 0);
            const int nchunks_u = __shfl_sync(0xffffffffu, nchunks, 0);
            const bool ident_u = __shfl_sync(0xffffffffu, (int)ident, 0) != 0;  // v = 0: no V^T T'^T term
            const bool ragged_u = __shfl_sync(0xffffffffu, (int)ragged, 0) != 0;
            constexpr uint32_t ID_G1 = umma_idesc_bf16(128, 64, true, false, false);    // V^T (MN-major A) x T'^T
            constexpr uint32_t ID_G2A = umma_idesc_bf16(128, 64, false, false, true);   // -(S) x W^T
            constexpr uint32_t ID_N64 = umma_idesc_bf16(128, 64, false, false, false);  // S x Q^T ; Delta^T x P^T
            constexpr uint32_t ID_G3B = umma_idesc_bf16(128, 128, false, true, false);  // (e o Delta)^T x K (MN-major B)
            // Shared-memory descriptors are built once (stage 0); the other stage and the K steps only
            // move the start-address field (16-byte units): +32 B per 16 K-major columns, +2048 B per
            // 16 MN-major rows, +kStageBytes per stage.
            constexpr uint64_t kStageStep = kStageBytes >> 4;
            const uint64_t dV = umma_desc(sb + ST_V, 8192, 1024);
            const uint64_t dThi = umma_desc(sb + ST_T, 16, 1024), dTlo = umma_desc(sb + ST_T + 8192, 16, 1024);
            const uint64_t dW0 = umma_desc(sb + ST_W, 16, 1024), dW1 = umma_desc(sb + ST_W + 8192, 16, 1024);
            const uint64_t dQ0 = umma_desc(sb + ST_Q, 16, 1024), dQ1 = umma_desc(sb + ST_Q + 8192, 16, 1024);
            const uint64_t dK = umma_desc(sb + ST_K, 8192, 1024), dP = umma_desc(sb + ST_P, 16, 1024);
            auto issue_G1 = [&](int st) {
                const uint64_t so = st * kStageStep;
#pragma unroll
                for (int ks = 0; ks < 4; ++ks)
                    umma_bf16_ss_warp(tmem_base_u + TM_DELTA, dV + so + ks * 128, dThi + so + ks * 2, ID_G1, ks > 0);
#pragma unroll
                for (int ks = 0; ks < 4; ++ks)
                    umma_bf16_ss_warp(tmem_base_u + TM_DELTA, dV + so + ks * 128, dTlo + so + ks * 2, ID_G1, 1);
            };

            bool g1_issued = false;

#define GDN_WAIT(idx, parity) if (!mbar_wait_all(bars + (idx), (uint32_t)(parity), abort_flag)) break
// for barriers that have normally completed long before the issuer gets here
#define GDN_WAIT_READY(idx, parity) if (!mbar_wait_all_probe(bars + (idx), (uint32_t)(parity), abort_flag)) break

            for (int ci = 0; ci < nchunks_u; ++ci) {
                const int c = c_begin + ci;
                (void)c;
                const int st = ci & 1, par = ci & 1, ph2 = (ci >> 1) & 1;
                const uint64_t so = st * kStageStep;
                const bool last = (ci + 1 == nchunks_u);
                if (!g1_issued) {
                    GDN_WAIT(B_FULL_A0 + st, ph2);
                    if (last && ragged_u) GDN_WAIT(B_CLEAN_A, 0);
                    tc_fence_after_sync();
                    if (!ident_u) issue_G1(st);
                }
                g1_issued = false;
                // ---- on the chain: Delta^T -= S W^T   (A = bf16 S in tensor memory)
                GDN_WAIT(B_SHI, par);
                tc_fence_after_sync();
                {
                    const uint64_t w0 = dW0 + so, w1 = dW1 + so;
                    const uint32_t td = tmem_base_u + TM_DELTA, ta = tmem_base_u + TM_SHI;
#pragma unroll
                    for (int ks = 0; ks < 4; ++ks)
                        umma_bf16_ts_warp(td, ta + ks * 8, w0 + ks * 2, ID_G2A, (ks > 0 || !ident_u) ? 1u : 0u);
#pragma unroll
                    for (int ks = 0; ks < 4; ++ks) umma_bf16_ts_warp(td, ta + 32 + ks * 8, w1 + ks * 2, ID_G2A, 1);
                }
                umma_commit_warp(bars + B_DELTA);
                // ---- off the chain: Oa^T = S Q^T (executes while the chain warps drain Delta^T)
                if (ci >= 1) GDN_WAIT_READY(B_OFREE, par ^ 1);
                {
                    const uint64_t q0 = dQ0 + so, q1 = dQ1 + so;
                    const uint32_t td = tmem_base_u + TM_OA, ta = tmem_base_u + TM_SHI;
#pragma unroll
                    for (int ks = 0; ks < 4; ++ks) umma_bf16_ts_warp(td, ta + ks * 8, q0 + ks * 2, ID_N64, ks > 0);
#pragma unroll
                    for (int ks = 0; ks < 4; ++ks) umma_bf16_ts_warp(td, ta + 32 + ks * 8, q1 + ks * 2, ID_N64, 1);
                }
                // ---- on the chain: S += (e o Delta)^T K  (hi + lo; A in tensor memory, B = K MN-major)
                GDN_WAIT_READY(B_FULL_B0 + st, ph2);
                if (last && ragged_u) GDN_WAIT_READY(B_CLEAN_B, 0);
                GDN_WAIT_READY(B_STM, par);
                GDN_WAIT(B_DW, par);
                tc_fence_after_sync();
                {
                    const uint64_t k0 = dK + so;
                    const uint32_t td = tmem_base_u + TM_S;
#pragma unroll
                    for (int ks = 0; ks < 4; ++ks) umma_bf16_ts_warp(td, tmem_base_u + TM_DTH + ks * 8, k0 + ks * 128, ID_G3B, 1);
#pragma unroll
                    for (int ks = 0; ks < 4; ++ks) umma_bf16_ts_warp(td, tmem_base_u + TM_DTL + ks * 8, k0 + ks * 128, ID_G3B, 1);
                }
                umma_commit_warp(bars + B_STATE);
                // ---- off the chain: Ob^T = Delta^T P^T, and the next chunk's V^T T'^T if it has landed
                GDN_WAIT(B_DL, par);
                tc_fence_after_sync();
#pragma unroll
                for (int ks = 0; ks < 4; ++ks)
                    umma_bf16_ts_warp(tmem_base_u + TM_OB, tmem_base_u + TM_DL + ks * 8, dP + so + ks * 2, ID_N64, ks > 0);
                // both output accumulators are complete with this product: the output warps can drain them
                // (and hand Oa^T back for the next chunk's S Q^T) without waiting for V^T T'^T as well
                umma_commit_warp(bars + B_O);
                if (!last) {
                    GDN_WAIT_READY(B_FULL_A0 + (st ^ 1), ((ci + 1) >> 1) & 1);  // requested a whole chunk ago
                    if (ci + 2 == nchunks_u && ragged_u) GDN_WAIT_READY(B_CLEAN_A, 0);
                    tc_fence_after_sync();
                    if (!ident_u) issue_G1(st ^ 1);
                    g1_issued = true;
                }
                umma_commit_warp(bars + B_FREE0 + st);  // every MMA that reads this stage has been issued
            }
#undef GDN_WAIT
#undef GDN_WAIT_READY
        }
        __syncwarp();
    } else if (warp == kProducerWarp) {
        // =========================================================== producer: all TMA / bulk copies
        {
            if (lane == 0) {
                prefetch_tensormap(&map_q);
                prefetch_tensormap(&map_k);
                prefetch_tensormap(&map_v);
            }
            __syncwarp();
            auto load_all = [&](int c, int st) {
                if (!elect_one()) return;
                uint8_t* sp = smem + st * kStageBytes;
                const int t0 = t0_first + (c - c_begin) * kChunk;
                mbar_expect_tx(bars + B_FULL_A0 + st, kTxA);
                bulk_load(sp + ST_T, ws + L.off_A + ((size_t)c * Hv + h) * kABytes, kABytes, bars + B_FULL_A0 + st);
                tma_load_3d(sp + ST_V, &map_v, bars + B_FULL_A0 + st, 0, h, t0);
                tma_load_3d(sp + ST_V + 8192, &map_v, bars + B_FULL_A0 + st, 64, h, t0);
                tma_load_3d(sp + ST_Q, &map_q, bars + B_FULL_A0 + st, 0, hq, t0);
                tma_load_3d(sp + ST_Q + 8192, &map_q, bars + B_FULL_A0 + st, 64, hq, t0);
                mbar_expect_tx(bars + B_FULL_B0 + st, kTxB);
                tma_load_3d(sp + ST_K, &map_k, bars + B_FULL_B0 + st, 0, hq, t0);
                tma_load_3d(sp + ST_K + 8192, &map_k, bars + B_FULL_B0 + st, 64, hq, t0);
                bulk_load(sp + ST_P, ws + L.off_P + ((size_t)c * Hv + h) * kPBytes, kPBytes, bars + B_FULL_B0 + st);
            };
            // The ring is two chunks deep; what the copies of the chunk after that will fetch is asked into
            // L2 one step earlier still, so that those copies do not wait for DRAM when many CTAs pull at once
            // (measured on 16 sequences x 32 heads: 1.5 us of 307 gained; asking three chunks ahead instead
            // cost 8 us).
            auto prefetch_all = [&](int c) {
                if (!elect_one()) return;
                const int t0 = t0_first + (c - c_begin) * kChunk;
                bulk_prefetch_l2(ws + L.off_A + ((size_t)c * Hv + h) * kABytes, kABytes);
                bulk_prefetch_l2(ws + L.off_P + ((size_t)c * Hv + h) * kPBytes, kPBytes);
                tma_prefetch_3d(&map_v, 0, h, t0);
                tma_prefetch_3d(&map_v, 64, h, t0);
                tma_prefetch_3d(&map_q, 0, hq, t0);
                tma_prefetch_3d(&map_q, 64, hq, t0);
                tma_prefetch_3d(&map_k, 0, hq, t0);
                tma_prefetch_3d(&map_k, 64, hq, t0);
            };
            // The initial state (64 KB, fp32) comes in as four [128 rows][32 floats] boxes with the 128-byte
            // swizzle, into the second stage's buffers, which nothing else needs before the second chunk:
            // one bulk transfer that overlaps the rest of the set-up, where 128 lanes each reading their
            // own 512-byte row used to take several microseconds.  The chain warps lift it into tensor memory.
            if (init_ptr && elect_one()) {
                mbar_expect_tx(bars + B_INIT, 4u * 16384u);
                const int row0 = (int)(state_off / kD);
#pragma unroll
                for (int j = 0; j < 4; ++j)
                    tma_load_2d(smem + kStageBytes + j * 16384, &map_s, bars + B_INIT, 32 * j, row0);
            }
            __syncwarp();
            // chunk ci goes to stage ci & 1 as soon as the MMAs of chunk ci - 2 have drained it
            bool all_requested = true;
            for (int ci = 0; ci < nchunks; ++ci) {
                if ((ci >= 2 &&
                     !mbar_wait_all(bars + B_FREE0 + (ci & 1), (uint32_t)(((ci >> 1) - 1) & 1), abort_flag)) ||
                    (ci == 1 && init_ptr && !mbar_wait_all(bars + B_INIT_DONE, 0, abort_flag))) {
                    all_requested = false;
                    break;
                }
                load_all(c_begin + ci, ci & 1);
                if (ci >= 1 && ci + 1 < nchunks) prefetch_all(c_begin + ci + 1);
            }
            // Ragged last chunk: rows >= tail_len of its V and K tiles belong to the next sequence.  Rows are
            // tokens, 128 bytes each in both halves of a tile (the swizzle permutes inside a row), so they
            // are one contiguous range per half tile.  This warp armed the stage's barriers for this very
            // phase a moment ago, so the parity it waits on cannot be mistaken for an earlier use of the stage.
            if (ragged && all_requested) {
                const int lc = nchunks - 1;
                uint8_t* sp = smem + (lc & 1) * kStageBytes;
                const uint32_t ph = (uint32_t)((lc >> 1) & 1);
                const uint32_t from = (uint32_t)tail_len * 128u;
                auto clear_rows = [&](uint8_t* tile) {
#pragma unroll 1
                    for (int half = 0; half < 2; ++half)
                        for (uint32_t o = from + lane * 16u; o < 8192u; o += 512u)
                            *reinterpret_cast<uint4*>(tile + half * 8192 + o) = make_uint4(0u, 0u, 0u, 0u);
                    fence_proxy_async_smem();  // generic-proxy stores before the tensor cores' reads
                    __syncwarp();
                };
                if (mbar_wait_all(bars + B_FULL_A0 + (lc & 1), ph, abort_flag)) {
                    clear_rows(sp + ST_V);
                    if (lane == 0) mbar_arrive(bars + B_CLEAN_A);
                    if (mbar_wait_all(bars + B_FULL_B0 + (lc & 1), ph, abort_flag)) {
                        clear_rows(sp + ST_K);
                        if (lane == 0) mbar_arrive(bars + B_CLEAN_B);
                    }
                }
            }
        }
        __syncwarp();
    } else if (warp >= kChainWarp0 && warp < kChainWarp0 + 4) {
        // =========================================================== chain warps
        const int v = tid - kChainWarp0 * 32;
        const uint32_t lane_addr = tmem_base + ((uint32_t)((warp & 3) * 32) << 16);
        const size_t sbase = (size_t)v * kD;
        // initial state: bf16 operand copy and Gamma_L(first chunk) * S, both into tensor memory
        {
            const float gl0 = __ldg(scal_ptr(c_begin) + 128);
            bool have_init = init_ptr != nullptr;
            if (have_init) have_init = mbar_wait_all(bars + B_INIT, 0, abort_flag);  // (on failure: zeros, and the loop below leaves)
            // row v of box jb sits at v * 128 in that box, its 16-byte piece c at (c ^ (v & 7)) * 16: the
            // eight lanes of a quarter warp hit eight different 16-byte bank groups
            const uint8_t* srow = smem + kStageBytes + (uint32_t)v * 128u;
#pragma unroll 1
            for (int b = 0; b < 2; ++b) {
                uint32_t r0[32], r1[32], pk[32];
#pragma unroll
                for (int j = 0; j < 32; j += 4) {
                    float4 x = make_float4(0.f, 0.f, 0.f, 0.f), y = x;
                    if (have_init) {
                        const uint32_t piece = (uint32_t)(((j >> 2) ^ (v & 7)) << 4);
                        x = *reinterpret_cast<const float4*>(srow + (2 * b) * 16384 + piece);
                        y = *reinterpret_cast<const float4*>(srow + (2 * b + 1) * 16384 + piece);
                    } else if (ident) {
                        const int d0 = v - (b * 64 + j), d1 = d0 - 32;  // the one of row v sits in column v
                        x = make_float4(d0 == 0 ? 1.f : 0.f, d0 == 1 ? 1.f : 0.f, d0 == 2 ? 1.f : 0.f, d0 == 3 ? 1.f : 0.f);
                        y = make_float4(d1 == 0 ? 1.f : 0.f, d1 == 1 ? 1.f : 0.f, d1 == 2 ? 1.f : 0.f, d1 == 3 ? 1.f : 0.f);
                    }
                    r0[j + 0] = __float_as_uint(x.x); r0[j + 1] = __float_as_uint(x.y);
                    r0[j + 2] = __float_as_uint(x.z); r0[j + 3] = __float_as_uint(x.w);
                    r1[j + 0] = __float_as_uint(y.x); r1[j + 1] = __float_as_uint(y.y);
                    r1[j + 2] = __float_as_uint(y.z); r1[j + 3] = __float_as_uint(y.w);
                }
#pragma unroll
                for (int j = 0; j < 16; ++j) {
                    pk[j] = pack_bf16x2(__uint_as_float(r0[2 * j]), __uint_as_float(r0[2 * j + 1]));
                    pk[16 + j] = pack_bf16x2(__uint_as_float(r1[2 * j]), __uint_as_float(r1[2 * j + 1]));
                }
                tmem_st32(lane_addr + TM_SHI + b * 32, pk);
#pragma unroll
                for (int j = 0; j < 32; ++j) {
                    r0[j] = __float_as_uint(__uint_as_float(r0[j]) * gl0);
                    r1[j] = __float_as_uint(__uint_as_float(r1[j]) * gl0);
                }
                tmem_st32(lane_addr + TM_S + b * 64, r0);
                tmem_st32(lane_addr + TM_S + b * 64 + 32, r1);
            }
            if (init_ptr) warp_arrive(bars + B_INIT_DONE);  // the second stage's buffers may be filled now
            tmem_st_wait();
            tc_fence_before_sync();
            warp_arrive(bars + B_SHI);
            warp_arrive(bars + B_STM);
        }
        for (int ci = 0; ci < nchunks; ++ci) {
            const int c = c_begin + ci;
            const uint32_t par = ci & 1;
            const bool last = (ci + 1 == nchunks);
            const float gl_next = last ? 1.f : __ldg(scal_ptr(c + 1) + 128);
            // e_j of this chunk into registers before the wait; prefetch the next chunk's lines
            float4 ev4[16];
            {
                const float4* e4 = reinterpret_cast<const float4*>(scal_ptr(c) + 64);
#pragma unroll
                for (int j = 0; j < 16; ++j) ev4[j] = __ldg(e4 + j);
                if (!last) asm volatile("prefetch.global.L2 [%0];" ::"l"(scal_ptr(c + 1) + (lane & 3) * 32));
            }
            if (!mbar_wait_all(bars + B_DELTA, par, abort_flag)) break;
            tc_fence_after_sync();
            // Delta^T row v -> bf16 A operands in tensor memory.  First (e o Delta) as hi + lo, which
            // the state update on the chain is waiting for; the plain bf16 Delta that only the output
            // product needs follows after that hand-off.  Two halves of 32 tokens keep the live
            // registers low (the warps share the register file).
#pragma unroll
            for (int half = 0; half < 2; ++half) {
                uint32_t r[32], hd[16], ld[16];
                tmem_ld32(lane_addr + TM_DELTA + half * 32, r);
                tmem_ld_wait();
#pragma unroll
                for (int j = 0; j < 16; ++j) {
                    const float4 ea = ev4[half * 8 + (j >> 1)];
                    const float e0 = (j & 1) ? ea.z : ea.x, e1 = (j & 1) ? ea.w : ea.y;
                    split_bf16x2(__uint_as_float(r[2 * j]) * e0, __uint_as_float(r[2 * j + 1]) * e1, hd[j], ld[j]);
                }
                tmem_st16(lane_addr + TM_DTH + half * 16, hd);
                tmem_st16(lane_addr + TM_DTL + half * 16, ld);
            }
            tmem_st_wait();
            tc_fence_before_sync();
            warp_arrive(bars + B_DW);
            {   // off the chain: bf16 Delta^T for Ob^T = Delta^T P^T (the accumulator is intact until
                // the next chunk's V^T T'^T, which the issuer starts only after this hand-off)
                uint32_t r[32], xd[32];
                tmem_ld32(lane_addr + TM_DELTA, r);
                tmem_ld32(lane_addr + TM_DELTA + 32, xd);  // second half, packed in place below
                tmem_ld_wait();
#pragma unroll
                for (int j = 0; j < 16; ++j) r[j] = pack_bf16x2(__uint_as_float(r[2 * j]), __uint_as_float(r[2 * j + 1]));
#pragma unroll
                for (int j = 0; j < 16; ++j) r[16 + j] = pack_bf16x2(__uint_as_float(xd[2 * j]), __uint_as_float(xd[2 * j + 1]));
                tmem_st32(lane_addr + TM_DL, r);
                tmem_st_wait();
                tc_fence_before_sync();
                warp_arrive(bars + B_DL);
            }

            if (!mbar_wait_all(bars + B_STATE, par, abort_flag)) break;
            tc_fence_after_sync();
            if (last) {
                if (fin_ptr) {
                    // run 0 of a split sequence also leaves its final state as the bf16 operand tiles
                    // the fix-up of run 1 multiplies with
                    uint8_t* img = (segs > 1 && seg == 0) ? ws + seg_block_offset(L, n, 1, h, Hv, kSegSinImg) : nullptr;
#pragma unroll 1
                    for (int b = 0; b < 4; ++b) {
                        uint32_t r[32];
                        tmem_ld32(lane_addr + TM_S + b * 32, r);
                        tmem_ld_wait();
#pragma unroll
                        for (int j = 0; j < 32; j += 8)  // 32-byte stores: every lane writes its own row
                            st_global_v8(fin_ptr + sbase + b * 32 + j, make_uint4(r[j], r[j + 1], r[j + 2], r[j + 3]),
                                         make_uint4(r[j + 4], r[j + 5], r[j + 6], r[j + 7]));
                        if (img) {
#pragma unroll
                            for (int j = 0; j < 32; j += 8)
                                *reinterpret_cast<uint4*>(img + (b >> 1) * 16384 + swz((uint32_t)v, (uint32_t)((b & 1) * 4 + (j >> 3)))) =
                                    make_uint4(pack_bf16x2(__uint_as_float(r[j]), __uint_as_float(r[j + 1])),
                                               pack_bf16x2(__uint_as_float(r[j + 2]), __uint_as_float(r[j + 3])),
                                               pack_bf16x2(__uint_as_float(r[j + 4]), __uint_as_float(r[j + 5])),
                                               pack_bf16x2(__uint_as_float(r[j + 6]), __uint_as_float(r[j + 7])));
                        }
                    }
                }
            } else {
                // state row v: bf16 operand copy for the next chunk first (it gates the next G2A) ...
#pragma unroll
                for (int b = 0; b < 2; ++b) {
                    uint32_t r0[32], r1[32], pk[32];
                    tmem_ld32(lane_addr + TM_S + b * 64, r0);
                    tmem_ld32(lane_addr + TM_S + b * 64 + 32, r1);
                    tmem_ld_wait();
#pragma unroll
                    for (int j = 0; j < 16; ++j) {
                        pk[j] = pack_bf16x2(__uint_as_float(r0[2 * j]), __uint_as_float(r0[2 * j + 1]));
                        pk[16 + j] = pack_bf16x2(__uint_as_float(r1[2 * j]), __uint_as_float(r1[2 * j + 1]));
                    }
                    tmem_st32(lane_addr + TM_SHI + b * 32, pk);
                }
                tmem_st_wait();
                tc_fence_before_sync();
                warp_arrive(bars + B_SHI);
                // ... then the fp32 state decayed by the next chunk's Gamma_L, in place (gates the next G3B)
#pragma unroll
                for (int b = 0; b < 2; ++b) {
                    uint32_t r0[32], r1[32];
                    tmem_ld32(lane_addr + TM_S + b * 64, r0);
                    tmem_ld32(lane_addr + TM_S + b * 64 + 32, r1);
                    tmem_ld_wait();
#pragma unroll
                    for (int j = 0; j < 32; ++j) {
                        r0[j] = __float_as_uint(__uint_as_float(r0[j]) * gl_next);
                        r1[j] = __float_as_uint(__uint_as_float(r1[j]) * gl_next);
                    }
                    tmem_st32(lane_addr + TM_S + b * 64, r0);
                    tmem_st32(lane_addr + TM_S + b * 64 + 32, r1);
                }
                tmem_st_wait();
                tc_fence_before_sync();
                warp_arrive(bars + B_STM);
            }
        }
    } else if (warp >= kOutputWarp0) {
        // =========================================================== output warps
        const int v = tid - kOutputWarp0 * 32;
        const uint32_t lane_addr = tmem_base + ((uint32_t)((warp & 3) * 32) << 16);
        for (int ci = 0; ci < nchunks; ++ci) {
            const int c = c_begin + ci;
            const uint32_t par = ci & 1;
            const int t0 = t0_first + ci * kChunk, len = min(kChunk, t_end - t0);
            auto last_chunk = [&](int i) { return i + 1 == nchunks; };
            const float4* g4 = reinterpret_cast<const float4*>(scal_ptr(c));  // Gamma_i of this chunk
            if (!last_chunk(ci)) asm volatile("prefetch.global.L2 [%0];" ::"l"(scal_ptr(c + 1) + (lane & 1) * 32));
            // A warp whose wait ran out does not leave on its own: the four output warps meet at a named
            // barrier below, and a warp that had left would strand the others there.  It carries on with
            // meaningless registers to that barrier, where the four decide together.
            const bool ok = mbar_wait_all(bars + B_O, par, abort_flag);
            tc_fence_after_sync();
            // drain both accumulators into registers and hand the columns back at once: the next
            // chunk's S Q^T is waiting for them
            uint32_t a0[32], a1[32], b0[32], b1[32];
            tmem_ld32(lane_addr + TM_OA, a0);
            tmem_ld32(lane_addr + TM_OA + 32, a1);
            tmem_ld32(lane_addr + TM_OB, b0);
            tmem_ld32(lane_addr + TM_OB + 32, b1);
            tmem_ld_wait();
            tc_fence_before_sync();
            if (ok) warp_arrive(bars + B_OFREE);
            // o_i = Gamma_i Oa^T[v][i] + Ob^T[v][i], packed two tokens per register
            uint32_t op[32];
#pragma unroll
            for (int j4 = 0; j4 < 8; ++j4) {
                const float4 gm = __ldg(g4 + j4), gn = __ldg(g4 + 8 + j4);
                op[j4 * 2] = pack_bf16x2(fmaf(gm.x, __uint_as_float(a0[4 * j4]), __uint_as_float(b0[4 * j4])),
                                         fmaf(gm.y, __uint_as_float(a0[4 * j4 + 1]), __uint_as_float(b0[4 * j4 + 1])));
                op[j4 * 2 + 1] = pack_bf16x2(fmaf(gm.z, __uint_as_float(a0[4 * j4 + 2]), __uint_as_float(b0[4 * j4 + 2])),
                                             fmaf(gm.w, __uint_as_float(a0[4 * j4 + 3]), __uint_as_float(b0[4 * j4 + 3])));
                op[16 + j4 * 2] = pack_bf16x2(fmaf(gn.x, __uint_as_float(a1[4 * j4]), __uint_as_float(b1[4 * j4])),
                                              fmaf(gn.y, __uint_as_float(a1[4 * j4 + 1]), __uint_as_float(b1[4 * j4 + 1])));
                op[16 + j4 * 2 + 1] = pack_bf16x2(fmaf(gn.z, __uint_as_float(a1[4 * j4 + 2]), __uint_as_float(b1[4 * j4 + 2])),
                                                  fmaf(gn.w, __uint_as_float(a1[4 * j4 + 3]), __uint_as_float(b1[4 * j4 + 3])));
            }
            // Through a shared-memory tile so that the global stores are 16 bytes per lane and whole
            // 256-byte rows per half warp (64 two-byte stores per thread kept these warps busier than
            // the chain itself).  The named barriers cover the four output warps only.  The first one
            // (the previous chunk's tile has been read) also ANDs the outcome of the wait above over all
            // 128 threads, so either all four warps go on to the second barrier or all four leave.
            {
                uint16_t* ost = reinterpret_cast<uint16_t*>(smem + OFF_OST);
                if (!bar_and(1, 128, ok)) break;
#pragma unroll
                for (int j = 0; j < 32; ++j) {
                    ost[(2 * j) * kD + v] = (uint16_t)(op[j] & 0xffffu);
                    ost[(2 * j + 1) * kD + v] = (uint16_t)(op[j] >> 16);
                }
                asm volatile("bar.sync 1, 128;" ::: "memory");
                const int c16 = v & 15, r0 = v >> 4;
                uint16_t* obase = out_ptr + ((size_t)t0 * Hv + h) * kD + c16 * 8;
                const size_t ostride = (size_t)Hv * kD;
#pragma unroll
                for (int k = 0; k < 8; ++k) {
                    const int row = r0 + 8 * k;
                    if (row < len)
                        *reinterpret_cast<uint4*>(obase + (size_t)row * ostride) =
                            *reinterpret_cast<const uint4*>(ost + row * kD + c16 * 8);
                }
            }
        }
    }

    // ---- unwind: on failure give copies in flight a moment to land, then release tensor memory
    unwind_after_abort(abort_flag, reinterpret_cast<int*>(ws), kStatusTimeout);
    if (warp == kIssuerWarp) {
        __syncwarp();
        tmem_dealloc(tmem_base, TM_COLS);
    }
}

cudaError_t launch_prefill_chain(const CUtensorMap& mq, const CUtensorMap& mk, const CUtensorMap& mv,
                                 const CUtensorMap& ms, const float* initial_state, void* out, float* final_state, uint8_t* ws,
                                 const WsLayout& L, int num_seqs, int Hqk, int Hv, int segs, const ChainPartial& part,
                                 cudaStream_t st) {
    static bool attr_done[64];
    if (cudaError_t e = set_attrs_once(attr_done, [] {
            return cudaFuncSetAttribute(gdn_prefill_chain_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kChainSmem);
        }))
        return e;
    const int per_seq = part.H ? 2 : 2 * segs - 1;
    gdn_prefill_chain_kernel<<<(unsigned)((long long)num_seqs * per_seq * Hv), kChainThreads, kChainSmem, st>>>(
        mq, mk, mv, ms, initial_state, (uint16_t*)out, final_state, ws, L, Hqk, Hv, segs, part);
    return cudaGetLastError();
}

}  // namespace gdn
