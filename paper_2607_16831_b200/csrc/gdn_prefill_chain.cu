// Inter-chunk ("chain") kernel of the chunked WY / UT-transform prefill.
//
// A chain = one (sequence, value head) whose 64-token chunks are walked in order.  The kernel has
// two forms (template parameter): one CTA per chain, or persistent -- one CTA per SM takes chains
// from a list sorted by decreasing length (dealt out in a snake so that every CTA gets about the
// same number of chunk steps) and walks them one after the other, keeping its barriers and its
// tensor memory; the copy warp runs ahead into the next chain, so that chain's first operands and
// its initial state are on their way while this chain's last chunk is still being computed and its
// final state stored.  launch_prefill_chain says when which form is used.  With
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
//   warp  1     issues every TMA / bulk copy, one chunk ahead of the MMAs (the chain's initial state
//               included: one swizzled 64 KB transfer into the buffers of the stage its second chunk
//               will use); when a chain's last chunk is ragged it also clears the rows of that chunk's
//               V and K tiles that lie beyond the sequence (the 64-row TMA box also fetched the first
//               tokens of the next one, and zeros in the other operand do not stop a NaN)
//   warps 4-7   chain: initial state -> tensor memory; drain Delta^T -> bf16 operands; drain S -> bf16
//               operand + decayed fp32 back; final state -> global memory
//   warps 8-11  output: drain Oa/Ob -> bf16 out
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
#include <cstdlib>

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

enum { B_FULL_A0 = 0, B_FULL_A1, B_FULL_B0, B_FULL_B1, B_FREE0, B_FREE1, B_DELTA, B_STATE, B_O, B_DW, B_SHI, B_STM, B_OFREE, B_DL, B_CLEAN_A0, B_CLEAN_A1, B_CLEAN_B0, B_CLEAN_B1, B_INIT, B_INIT_DONE, B_COUNT };


// What a CTA needs to know about one chain (uniform over the CTA; every role derives it itself).
struct ChainItem {
    int n, h, hq, seg;
    bool ident;      // starts from the identity with v = 0 (the run's transition and carried-back queries)
    int nchunks;     // <= 0: nothing to walk
    int c_begin;     // first chunk slot in the workspace
    int t0_first;    // first token of the run
    int t_end;       // one past the last token of the run
    int tail_len;    // tokens in the run's last chunk
    bool ragged;     // tail_len < 64
    size_t state_off;
    const float* init_ptr;  // initial state of this chain, or NULL (zeros / identity)
    float* fin_ptr;         // where its final state goes, or NULL
    uint16_t* out_ptr;
    uint8_t* img;           // run 0 of a split sequence also leaves its final state as bf16 operand tiles
};

struct ChainArgs {
    const float* initial_state;
    uint16_t* out;
    float* final_state;
    uint8_t* ws;
    WsLayout L;
    int Hqk, Hv, segs;
    ChainPartial part;
    int total_items;  // chains in the list: sequences x (runs per sequence) x value heads
};

// Chain `idx` of the list.  The list is sorted by decreasing sequence length; within a sequence: run 0, then
// (zero state, identity) per later run; value heads innermost.  `rec` is the sequence's table record
// (sequence, its first chunk slot, its first token, its length).
__device__ __forceinline__ int chain_seq_rank(const ChainArgs& A, int idx) {
    const int per_seq = A.part.H ? 2 : 2 * A.segs - 1;
    return idx / A.Hv / per_seq;
}
__device__ __forceinline__ ChainItem chain_item(const ChainArgs& A, int idx, int4 rec) {
    ChainItem I;
    const bool partial = A.part.H != nullptr;
    const int per_seq = partial ? 2 : 2 * A.segs - 1;
    const int unit = idx / A.Hv;
    I.h = idx % A.Hv;
    I.hq = I.h / (A.Hv / A.Hqk);
    I.n = rec.x;
    I.seg = partial ? 0 : (unit % per_seq + 1) >> 1;
    I.ident = partial ? (unit % per_seq) == 1 : (I.seg > 0 && ((unit % per_seq) & 1) == 0);
    // chunk slots of the sequence, clamped like the chunk table itself (a malformed cu_seqlens cannot
    // send the CTA outside the workspace)
    const int seq_chunks = max(0, min((rec.w + kChunk - 1) / kChunk, A.L.nc_max - rec.y));
    int seg_first;
    segment_range(seq_chunks, A.segs, I.seg, seg_first, I.nchunks);
    I.c_begin = rec.y + seg_first;
    // chunks of one sequence are consecutive: chunk ci of this run starts at t0_first + 64 ci
    I.t0_first = rec.z + seg_first * kChunk;
    I.t_end = min(rec.z + rec.w, I.t0_first + I.nchunks * kChunk);
    // Only the last chunk of a run can be ragged.  Its 64-row TMA boxes reach past the sequence into
    // the next one; those rows meet exact zeros in every product, which is not enough when they hold
    // NaN or Inf, so they are cleared in shared memory before the tensor cores see them.
    I.tail_len = I.t_end - (I.t0_first + (I.nchunks - 1) * kChunk);
    I.ragged = I.nchunks > 0 && I.tail_len < kChunk;
    I.state_off = ((size_t)I.n * A.Hv + I.h) * kD * kD;
    I.init_ptr = (!partial && I.seg == 0 && A.initial_state) ? A.initial_state + I.state_off : nullptr;
    I.fin_ptr = A.final_state ? A.final_state + I.state_off : nullptr;
    if (partial)
        I.fin_ptr = (I.ident ? A.part.P : A.part.H) + I.state_off;
    else if (A.segs > 1)
        I.fin_ptr = reinterpret_cast<float*>(
            A.ws + seg_block_offset(A.L, I.n, I.seg == 0 ? 1 : I.seg, I.h, A.Hv,
                                    I.seg == 0 ? kSegSin : (I.ident ? kSegP : kSegH)));
    I.out_ptr = I.ident ? (partial ? A.part.qt : reinterpret_cast<uint16_t*>(A.ws + A.L.off_qt)) : A.out;
    I.img = (A.segs > 1 && I.seg == 0 && !partial) ? A.ws + seg_block_offset(A.L, I.n, 1, I.h, A.Hv, kSegSinImg) : nullptr;
    return I;
}

// The r-th chain of CTA `b` of `G`: rounds alternate direction (b, 2G-1-b, 2G+b, ...), so that on a list
// sorted by decreasing length every CTA collects about the same number of chunk steps.
__device__ __forceinline__ int chain_index(int r, int b, int G) { return (r & 1) ? (r + 1) * G - 1 - b : r * G + b; }

// kPersistent = false: one CTA per chain (grid = chains), the hardware hands the CTAs out.  The roles' outer
// loops then run once and fold away; this is the faster form when chains are long (a chunk step is ~5 % faster
// than inside the persistent loops) and is what few long sequences use.
template <bool kPersistent>
__global__ void __launch_bounds__(kChainThreads, 1)
gdn_prefill_chain_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                         const __grid_constant__ CUtensorMap map_v, const __grid_constant__ CUtensorMap map_s,
                         const __grid_constant__ ChainArgs A) {
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    uint8_t* const ws = A.ws;
    const int Hv = A.Hv;

    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + OFF_BAR);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + OFF_BAR + 8 * B_COUNT);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + OFF_BAR + 8 * B_COUNT + 8);

    const int4* seq_table = reinterpret_cast<const int4*>(ws + A.L.off_seq_order);
    const int G = (int)gridDim.x, b_cta = (int)blockIdx.x;
    // this CTA's chains, in order; every role walks the same list with its own running counters:
    //   gc   chunks walked so far by this CTA (stage = gc & 1 and every per-chunk barrier phase follow from it)
    //   nrag ragged chains so far, nini chains with an initial state to fetch so far (phases of those barriers)
    auto item_index = [&](int r) { return kPersistent ? chain_index(r, b_cta, G) : b_cta; };
    auto item_valid = [&](int r) {
        if (!kPersistent) return r == 0;
        const int i = chain_index(r, b_cta, G);
        return i >= 0 && i < A.total_items;
    };
    auto load_rec = [&](int r) { return __ldg(&seq_table[chain_seq_rank(A, item_index(r))]); };
    auto prefetch_rec = [&](int r) {
        asm volatile("prefetch.global.L1 [%0];" ::"l"(seq_table + chain_seq_rank(A, item_index(r))));
    };

    // the first chain's record is requested before the set-up below, whose latency hides the load
    const int4 rec_first = item_valid(0) ? load_rec(0) : make_int4(0, 0, 0, 0);
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

    auto scal_ptr = [&](int c, int h) {
        return reinterpret_cast<const float*>(ws + A.L.off_scal + ((size_t)c * Hv + h) * kScalBytes);
    };

    if (warp == kIssuerWarp) {
        // =========================================================== issuer: MMA
        // The whole warp runs this loop in lock step; one elected lane issues each MMA.  Values that
        // feed the MMA operands are broadcast from lane 0 so that the compiler knows they are
        // warp-uniform and keeps descriptors and addresses in uniform registers.
        const uint32_t sb = __shfl_sync(0xffffffffu, smem_u32(smem), 0);
        const uint32_t tmem_base_u = __shfl_sync(0xffffffffu, tmem_base, 0);
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
#define GDN_WAIT(idx, parity) if (!mbar_wait_all(bars + (idx), (uint32_t)(parity), abort_flag)) { alive = false; break; }
// for barriers that have normally completed long before the issuer gets here
#define GDN_WAIT_READY(idx, parity) if (!mbar_wait_all_probe(bars + (idx), (uint32_t)(parity), abort_flag)) { alive = false; break; }
        bool alive = true;
        int gc = 0;
        // Ragged chunks so far per stage: the phase of that stage's "rows cleared" barriers.  One pair of
        // barriers per stage, because the copy warp can be two chunks ahead: with a single pair it could
        // complete two phases before this warp has looked at the first, and a parity cannot tell those apart;
        // a stage is not refilled before this warp has released it, so per stage at most one phase is open.
        int nrag0 = 0, nrag1 = 0;
        int4 rec = rec_first;
        for (int r = 0; alive && item_valid(r); ++r) {
            const ChainItem I = chain_item(A, item_index(r), rec);
            if (item_valid(r + 1)) rec = load_rec(r + 1);  // in flight while this chain is walked
            const int nchunks_u = __shfl_sync(0xffffffffu, I.nchunks, 0);
            const bool ident_u = __shfl_sync(0xffffffffu, (int)I.ident, 0) != 0;  // v = 0: no V^T T'^T term
            const bool ragged_u = __shfl_sync(0xffffffffu, (int)I.ragged, 0) != 0;
            const int last_stage = (gc + nchunks_u - 1) & 1;
            const int clean_par = (last_stage ? nrag1 : nrag0) & 1;
            bool g1_issued = false;
            for (int ci = 0; ci < nchunks_u; ++ci, ++gc) {
                const int st = gc & 1, par = gc & 1, ph2 = (gc >> 1) & 1;
                const uint64_t so = st * kStageStep;
                const bool last = (ci + 1 == nchunks_u);
                if (!g1_issued) {
                    GDN_WAIT(B_FULL_A0 + st, ph2);
                    if (last && ragged_u) GDN_WAIT(B_CLEAN_A0 + st, clean_par);
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
                if (gc >= 1) GDN_WAIT_READY(B_OFREE, par ^ 1);
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
                if (last && ragged_u) GDN_WAIT_READY(B_CLEAN_B0 + st, clean_par);
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
                    GDN_WAIT_READY(B_FULL_A0 + (st ^ 1), ((gc + 1) >> 1) & 1);  // requested a whole chunk ago
                    if (ci + 2 == nchunks_u && ragged_u) GDN_WAIT_READY(B_CLEAN_A0 + (st ^ 1), clean_par);
                    tc_fence_after_sync();
                    if (!ident_u) issue_G1(st ^ 1);
                    g1_issued = true;
                }
                umma_commit_warp(bars + B_FREE0 + st);  // every MMA that reads this stage has been issued
            }
            if (ragged_u && nchunks_u > 0) {
                if (last_stage) ++nrag1; else ++nrag0;
            }
        }
#undef GDN_WAIT
#undef GDN_WAIT_READY
        __syncwarp();
    } else if (warp == kProducerWarp) {
        // =========================================================== producer: all TMA / bulk copies
        if (lane == 0) {
            prefetch_tensormap(&map_q);
            prefetch_tensormap(&map_k);
            prefetch_tensormap(&map_v);
            if (A.initial_state) prefetch_tensormap(&map_s);
        }
        __syncwarp();
        bool alive = true;
        int gc = 0, nini = 0;
        int init_stage = -1;       // stage whose buffers hold an initial state that has not been consumed yet
        uint32_t init_par = 0;     // phase of B_INIT_DONE that releases it
        int4 rec = rec_first;
        for (int r = 0; alive && item_valid(r); ++r) {
            const ChainItem I = chain_item(A, item_index(r), rec);
            if (item_valid(r + 1)) rec = load_rec(r + 1);
            if (I.nchunks <= 0) continue;
            auto load_all = [&](int c, int st, int t0) {
                if (!elect_one()) return;
                uint8_t* sp = smem + st * kStageBytes;
                mbar_expect_tx(bars + B_FULL_A0 + st, kTxA);
                bulk_load(sp + ST_T, ws + A.L.off_A + ((size_t)c * Hv + I.h) * kABytes, kABytes, bars + B_FULL_A0 + st);
                tma_load_3d(sp + ST_V, &map_v, bars + B_FULL_A0 + st, 0, I.h, t0);
                tma_load_3d(sp + ST_V + 8192, &map_v, bars + B_FULL_A0 + st, 64, I.h, t0);
                tma_load_3d(sp + ST_Q, &map_q, bars + B_FULL_A0 + st, 0, I.hq, t0);
                tma_load_3d(sp + ST_Q + 8192, &map_q, bars + B_FULL_A0 + st, 64, I.hq, t0);
                mbar_expect_tx(bars + B_FULL_B0 + st, kTxB);
                tma_load_3d(sp + ST_K, &map_k, bars + B_FULL_B0 + st, 0, I.hq, t0);
                tma_load_3d(sp + ST_K + 8192, &map_k, bars + B_FULL_B0 + st, 64, I.hq, t0);
                bulk_load(sp + ST_P, ws + A.L.off_P + ((size_t)c * Hv + I.h) * kPBytes, kPBytes, bars + B_FULL_B0 + st);
            };
            // The ring is two chunks deep; what the copies of the chunk after that will fetch is asked into
            // L2 one step earlier still, so that those copies do not wait for DRAM when many CTAs pull at once.
            auto prefetch_all = [&](int c, int t0) {
                if (!elect_one()) return;
                bulk_prefetch_l2(ws + A.L.off_A + ((size_t)c * Hv + I.h) * kABytes, kABytes);
                bulk_prefetch_l2(ws + A.L.off_P + ((size_t)c * Hv + I.h) * kPBytes, kPBytes);
                tma_prefetch_3d(&map_v, 0, I.h, t0);
                tma_prefetch_3d(&map_v, 64, I.h, t0);
                tma_prefetch_3d(&map_q, 0, I.hq, t0);
                tma_prefetch_3d(&map_q, 64, I.hq, t0);
                tma_prefetch_3d(&map_k, 0, I.hq, t0);
                tma_prefetch_3d(&map_k, 64, I.hq, t0);
            };
            // A stage may be written again once the MMAs of the chunk two before (of this chain or of the one
            // before it) have drained it and, if an initial state was parked in it, once the chain warps have
            // lifted that state into tensor memory.
            auto stage_writable = [&](int g) {
                if (init_stage == (g & 1)) {
                    if (!mbar_wait_all(bars + B_INIT_DONE, init_par, abort_flag)) return false;
                    init_stage = -1;
                }
                return g < 2 || mbar_wait_all(bars + B_FREE0 + (g & 1), (uint32_t)(((g >> 1) - 1) & 1), abort_flag);
            };
            // The initial state (64 KB, fp32) comes in as four [128 rows][32 floats] boxes with the 128-byte
            // swizzle, into the buffers of the stage the chain's SECOND chunk will use, which nothing else
            // needs until the chain warps have lifted the state into tensor memory: one bulk transfer,
            // where 128 lanes each reading their own 512-byte row used to take several microseconds.
            // The first chunk's operands are requested before it: their stage was free earlier.
            const int gc0 = gc;
            for (int ci = 0; ci < I.nchunks; ++ci, ++gc) {
                if (!stage_writable(gc)) { alive = false; break; }
                load_all(I.c_begin + ci, gc & 1, I.t0_first + ci * kChunk);
                if (ci == 0 && I.init_ptr) {
                    if (!stage_writable(gc + 1)) { alive = false; break; }
                    if (elect_one()) {
                        mbar_expect_tx(bars + B_INIT, 4u * 16384u);
                        const int row0 = (int)(I.state_off / kD);
#pragma unroll
                        for (int j = 0; j < 4; ++j)
                            tma_load_2d(smem + ((gc + 1) & 1) * kStageBytes + j * 16384, &map_s, bars + B_INIT, 32 * j, row0);
                    }
                    __syncwarp();
                    init_stage = (gc + 1) & 1;
                    init_par = (uint32_t)(nini & 1);
                    ++nini;
                }
                if (ci >= 1 && ci + 1 < I.nchunks) prefetch_all(I.c_begin + ci + 1, I.t0_first + (ci + 1) * kChunk);
            }
            if (!alive) break;
            // Ragged last chunk: rows >= tail_len of its V and K tiles belong to the next sequence.  Rows are
            // tokens, 128 bytes each in both halves of a tile (the swizzle permutes inside a row), so they
            // are one contiguous range per half tile.  This warp armed the stage's barriers for this very
            // phase a moment ago, so the parity it waits on cannot be mistaken for an earlier use of the stage.
            if (I.ragged) {
                const int lg = gc0 + I.nchunks - 1;
                uint8_t* sp = smem + (lg & 1) * kStageBytes;
                const uint32_t ph = (uint32_t)((lg >> 1) & 1);
                const uint32_t from = (uint32_t)I.tail_len * 128u;
                auto clear_rows = [&](uint8_t* tile) {
#pragma unroll 1
                    for (int half = 0; half < 2; ++half)
                        for (uint32_t o = from + lane * 16u; o < 8192u; o += 512u)
                            *reinterpret_cast<uint4*>(tile + half * 8192 + o) = make_uint4(0u, 0u, 0u, 0u);
                    fence_proxy_async_smem();  // generic-proxy stores before the tensor cores' reads
                    __syncwarp();
                };
                if (!mbar_wait_all(bars + B_FULL_A0 + (lg & 1), ph, abort_flag)) break;
                clear_rows(sp + ST_V);
                if (lane == 0) mbar_arrive(bars + B_CLEAN_A0 + (lg & 1));
                if (!mbar_wait_all(bars + B_FULL_B0 + (lg & 1), ph, abort_flag)) break;
                clear_rows(sp + ST_K);
                if (lane == 0) mbar_arrive(bars + B_CLEAN_B0 + (lg & 1));
            }
        }
        __syncwarp();
    } else if (warp >= kChainWarp0 && warp < kChainWarp0 + 4) {
        // =========================================================== chain warps
        const int v = tid - kChainWarp0 * 32;
        const uint32_t lane_addr = tmem_base + ((uint32_t)((warp & 3) * 32) << 16);
        const size_t sbase = (size_t)v * kD;
        bool alive = true;
        int gc = 0, nini = 0;
        for (int r = 0; alive && item_valid(r); ++r) {
        const ChainItem I = chain_item(A, item_index(r), r == 0 ? rec_first : load_rec(r));
        if (item_valid(r + 1)) prefetch_rec(r + 1);  // so that the next chain's record is an L1 hit
        const int nchunks = I.nchunks, c_begin = I.c_begin, h = I.h;
        const bool ident = I.ident;
        const float* const init_ptr = I.init_ptr;
        float* const fin_ptr = I.fin_ptr;
        if (nchunks <= 0) {  // empty sequence: the state passes through; empty run: nothing to do
            if (A.part.H) {  // H = 0, P = I
                float* dst = (ident ? A.part.P : A.part.H) + I.state_off + sbase;
                for (int j = 0; j < kD; j += 4)
                    *reinterpret_cast<float4*>(dst + j) =
                        make_float4((ident && v == j) ? 1.f : 0.f, (ident && v == j + 1) ? 1.f : 0.f,
                                    (ident && v == j + 2) ? 1.f : 0.f, (ident && v == j + 3) ? 1.f : 0.f);
            } else if (I.seg == 0 && A.final_state) {
                for (int j = 0; j < kD; j += 4) {
                    float4 x = make_float4(0.f, 0.f, 0.f, 0.f);
                    if (A.initial_state) x = *reinterpret_cast<const float4*>(A.initial_state + I.state_off + sbase + j);
                    *reinterpret_cast<float4*>(A.final_state + I.state_off + sbase + j) = x;
                }
            }
            continue;
        }
        // initial state: bf16 operand copy and Gamma_L(first chunk) * S, both into tensor memory
        {
            const float gl0 = __ldg(scal_ptr(c_begin, h) + 128);
            bool have_init = init_ptr != nullptr;
            // (on failure: zeros, and the chunk loop below leaves at its first wait)
            if (have_init) have_init = mbar_wait_all(bars + B_INIT, (uint32_t)(nini & 1), abort_flag);
            // The copy warp parked the state in the buffers of the stage this chain's second chunk will use.
            // Row v of box jb sits at v * 128 in that box, its 16-byte piece c at (c ^ (v & 7)) * 16: the
            // eight lanes of a quarter warp hit eight different 16-byte bank groups.
            const uint8_t* srow = smem + ((gc + 1) & 1) * kStageBytes + (uint32_t)v * 128u;
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
            if (init_ptr) {
                warp_arrive(bars + B_INIT_DONE);  // those buffers may be filled with operands now
                ++nini;
            }
            tmem_st_wait();
            tc_fence_before_sync();
            warp_arrive(bars + B_SHI);
            warp_arrive(bars + B_STM);
        }
        for (int ci = 0; ci < nchunks; ++ci, ++gc) {
            const int c = c_begin + ci;
            const uint32_t par = gc & 1;
            const bool last = (ci + 1 == nchunks);
            const float gl_next = last ? 1.f : __ldg(scal_ptr(c + 1, h) + 128);
            // e_j of this chunk into registers before the wait; prefetch the next chunk's lines
            float4 ev4[16];
            {
                const float4* e4 = reinterpret_cast<const float4*>(scal_ptr(c, h) + 64);
#pragma unroll
                for (int j = 0; j < 16; ++j) ev4[j] = __ldg(e4 + j);
                if (!last) asm volatile("prefetch.global.L2 [%0];" ::"l"(scal_ptr(c + 1, h) + (lane & 3) * 32));
            }
            if (!mbar_wait_all(bars + B_DELTA, par, abort_flag)) { alive = false; break; }
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

            if (!mbar_wait_all(bars + B_STATE, par, abort_flag)) { alive = false; break; }
            tc_fence_after_sync();
            if (last) {
                if (fin_ptr) {
                    // run 0 of a split sequence also leaves its final state as the bf16 operand tiles
                    // the fix-up of run 1 multiplies with
                    uint8_t* img = I.img;
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
        }  // chains of this CTA
    } else if (warp >= kOutputWarp0) {
        // =========================================================== output warps
        const int v = tid - kOutputWarp0 * 32;
        const uint32_t lane_addr = tmem_base + ((uint32_t)((warp & 3) * 32) << 16);
        bool alive = true;
        int gc = 0;
        for (int r = 0; alive && item_valid(r); ++r) {
        const ChainItem I = chain_item(A, item_index(r), r == 0 ? rec_first : load_rec(r));
        if (item_valid(r + 1)) prefetch_rec(r + 1);  // so that the next chain's record is an L1 hit
        const int nchunks = I.nchunks, c_begin = I.c_begin, h = I.h;
        uint16_t* const out_ptr = I.out_ptr;
        for (int ci = 0; ci < nchunks; ++ci, ++gc) {
            const int c = c_begin + ci;
            const uint32_t par = gc & 1;
            const int t0 = I.t0_first + ci * kChunk, len = min(kChunk, I.t_end - t0);
            auto last_chunk = [&](int i) { return i + 1 == nchunks; };
            const float4* g4 = reinterpret_cast<const float4*>(scal_ptr(c, h));  // Gamma_i of this chunk
            if (!last_chunk(ci)) asm volatile("prefetch.global.L2 [%0];" ::"l"(scal_ptr(c + 1, h) + (lane & 1) * 32));
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
                if (!bar_and(1, 128, ok)) { alive = false; break; }
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
        }  // chains of this CTA
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
            cudaError_t e2 = cudaFuncSetAttribute(gdn_prefill_chain_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kChainSmem);
            if (e2 == cudaSuccess)
                e2 = cudaFuncSetAttribute(gdn_prefill_chain_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kChainSmem);
            return e2;
        }))
        return e;
    // one CTA per SM (a CTA fills an SM's shared memory and tensor memory), fewer when there are fewer chains
    static int sms[64];
    int dev = 0, nsm = kAssumedSMs;
    if (cudaGetDevice(&dev) == cudaSuccess && dev >= 0 && dev < 64) {
        if (!sms[dev] && cudaDeviceGetAttribute(&sms[dev], cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) sms[dev] = 0;
        if (sms[dev] > 0) nsm = sms[dev];
    }
    const int per_seq = part.H ? 2 : 2 * segs - 1;
    const long long items = (long long)num_seqs * per_seq * Hv;
    if (items <= 0) return cudaSuccess;
    ChainArgs A;
    A.initial_state = initial_state;
    A.out = (uint16_t*)out;
    A.final_state = final_state;
    A.ws = ws;
    A.L = L;
    A.Hqk = Hqk;
    A.Hv = Hv;
    A.segs = segs;
    A.part = part;
    A.total_items = (int)items;
    // Persistent CTAs pay off when an SM walks many short chains (what is saved is per chain: set-up, the
    // first operands' latency, the hand-over between chains); with long chains the slightly slower chunk step
    // inside the persistent loops costs more than that.  Measured on B200: the persistent form gains ~2.4 us
    // per chain and loses ~0.17 us per chunk step.  GDN_PREFILL_PERSISTENT=0/1 (environment) forces one form.
    // (L.nc_max = total_tokens / 64 + num_seqs bounds the chunks per value head: at most ~10 chunks per sequence)
    bool persistent = items > nsm && (long long)L.nc_max <= 10LL * num_seqs;
    if (const char* env = getenv("GDN_PREFILL_PERSISTENT")) {
        if (env[0] == '0') persistent = false;
        if (env[0] == '1') persistent = true;
    }
    if (persistent)
        gdn_prefill_chain_kernel<true><<<(unsigned)(items < nsm ? items : nsm), kChainThreads, kChainSmem, st>>>(mq, mk, mv, ms, A);
    else
        gdn_prefill_chain_kernel<false><<<(unsigned)items, kChainThreads, kChainSmem, st>>>(mq, mk, mv, ms, A);
    return cudaGetLastError();
}

}  // namespace gdn
