// Sequence-parallel prefill: joining the runs of chunks that the chain kernel advanced side by side.
//
// The recurrence is affine in the state: over any run of tokens, with M_t the product of the
// per-token transitions alpha (I - beta k k^T) from the start of the run up to token t,
//
//     S_t = S_in M_t + H_t          o_t = S_t q_t = H_t q_t + S_in (M_t q_t)
//
// where H_t is the state reached from the zero state.  For every run after the first the chain
// kernel has produced  o0_t = H_t q_t  (bf16, in `out`),  qt_t = M_t q_t  (bf16, workspace),
// H = H_end and P = M_end (fp32 blocks).  What is left is an associative scan over the runs,
//
//     S_in(s+1) = S_in(s) P_s + H_s                     (combine kernel, fp32 SIMT; rows independent)
//     out_t    += S_in(s) qt_t   for t in run s          (fix-up kernel, one tcgen05 GEMM tile per CTA)
//
// The combine is serial over the runs of one sequence (at most seven steps) but each CTA carries
// only 16 state rows, so the rows of one head spread over eight SMs.
#include "gdn_prefill_ws.cuh"
#include "gdn_sm100.cuh"

namespace gdn {
using namespace sm100;

constexpr uint32_t CB_XT = 0;        // X transposed: xt[k][row] fp32                 up to 8 KB
constexpr uint32_t CB_BAR = 8192;    // two mbarriers, abort flag
constexpr uint32_t CB_P = 8192 + 128;  // one or two buffers of P, fp32 [128][128]   64 KB each
constexpr uint32_t kPBlock = (uint32_t)kSegBlockBytes;
__host__ __device__ constexpr uint32_t combine_smem(int nbuf) { return CB_P + nbuf * kPBlock + 128; }

// Where the scan S <- S P_i + H_i (i = 0 .. steps-1) finds and leaves its operands.  Offsets are in
// floats from the base pointers: block of (step i, sequence n, head h) = i * ss + n * sn + h * sh.
struct ScanArgs {
    const float* x0;        // starting state of (n, h) at n * x_sn + h * x_sh; NULL = zeros
    long long x_sn, x_sh;
    const float* P;         // fp32 [128][128] per (i, n, h)
    const float* H;
    long long ss, sn, sh;
    float* sin;             // optional: the state entering step i >= 1 is written to block (i, n, h) ...
    uint8_t* img;           // ... and as bf16 operand tiles (same block index, 4 bytes per float)
    float* fin;             // optional: the last state, [N][Hv][128][128]
    int steps;
    const int* chunk_off;   // optional: step i is run i + 1 of `segs` runs; stop at the first empty run
    int segs;
    int* status;            // device status word
};

// grid (sequences x value heads, 128 / (4 RW) row blocks): a CTA owns 4 RW rows of the state, a thread RW rows
// x 4 columns.  RW = 2 doubles the CTAs per (sequence, head) when there are few of those (the steps are
// serial, so this is the only parallelism there is).  `nbuf` = 2 fetches the next step's P while this step's
// product is computed.
template <int RW>
__global__ void __launch_bounds__(128)
gdn_prefill_combine_kernel(ScanArgs A, int Hv, int nbuf) {
    constexpr int kCombineRows = 4 * RW;
    const int n = blockIdx.x / Hv, h = blockIdx.x % Hv;
    const int row0 = blockIdx.y * kCombineRows;
    const int tid = threadIdx.x, ty = tid >> 5, tx = tid & 31;  // thread tile: rows RW ty.., columns 4 tx..
    const int nch = A.chunk_off ? A.chunk_off[n + 1] - A.chunk_off[n] : 1;
    if (nch <= 0) return;  // empty sequence: the chain kernel passed the state through
    const long long unit = (long long)n * A.sn + (long long)h * A.sh;

    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 127) & ~uintptr_t(127));
    float (*xt)[kCombineRows] = reinterpret_cast<float (*)[kCombineRows]>(smem + CB_XT);
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + CB_BAR);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + CB_BAR + 16);
    const float* pbuf = reinterpret_cast<const float*>(smem + CB_P);

    // below, s = i + 1 counts steps from 1 (= the run index when the steps are runs of chunks)
    const int segs = A.steps + 1;
    auto run_chunks = [&](int s) {
        if (s >= segs) return 0;
        if (!A.chunk_off) return 1;
        int first, count;
        segment_range(nch, A.segs, s, first, count);
        return count;
    };
    auto fetch_P = [&](int s) {  // one thread: the whole 64 KB block in one bulk copy
        const int b = (s - 1) % nbuf;
        mbar_expect_tx(bars + b, kPBlock);
        bulk_load(smem + CB_P + b * kPBlock, A.P + (long long)(s - 1) * A.ss + unit, kPBlock, bars + b);
    };
    if (tid == 0) {
        mbar_init(bars + 0, 1);
        mbar_init(bars + 1, 1);
        *abort_flag = 0;
        mbar_fence_init();
        if (run_chunks(1) > 0) fetch_P(1);
    }
    __syncthreads();  // the barriers and the abort flag are set before anybody reads them (the loop below may run zero times)

    float acc[RW][4];
    {
        const float* x0 = A.x0 ? A.x0 + (long long)n * A.x_sn + (long long)h * A.x_sh : nullptr;
#pragma unroll
        for (int i = 0; i < RW; ++i) {
            float4 x = make_float4(0.f, 0.f, 0.f, 0.f);
            if (x0) x = *reinterpret_cast<const float4*>(x0 + (size_t)(row0 + ty * RW + i) * kD + tx * 4);
            acc[i][0] = x.x; acc[i][1] = x.y; acc[i][2] = x.z; acc[i][3] = x.w;
        }
    }
    for (int s = 1; s < segs; ++s) {
        if (run_chunks(s) <= 0) break;  // later runs are empty as well
        if (s >= 2 && A.sin) {
            // the state entering run s, for the fix-up: fp32 and as bf16 operand tiles
            float* sin = A.sin + (long long)(s - 1) * A.ss + unit;
            uint8_t* img = A.img + ((long long)(s - 1) * A.ss + unit) * 4;
#pragma unroll
            for (int i = 0; i < RW; ++i) {
                const int r = row0 + ty * RW + i;
                *reinterpret_cast<float4*>(sin + (size_t)r * kD + tx * 4) =
                    make_float4(acc[i][0], acc[i][1], acc[i][2], acc[i][3]);
                *reinterpret_cast<uint2*>(img + (tx >> 4) * 16384 + swz((uint32_t)r, (uint32_t)((tx >> 1) & 7)) + (tx & 1) * 8) =
                    make_uint2(pack_bf16x2(acc[i][0], acc[i][1]), pack_bf16x2(acc[i][2], acc[i][3]));
            }
        }
        const float* H = A.H + (long long)(s - 1) * A.ss + unit;
        float4 hrow[RW];
#pragma unroll
        for (int i = 0; i < RW; ++i) hrow[i] = *reinterpret_cast<const float4*>(H + (size_t)(row0 + ty * RW + i) * kD + tx * 4);
        __syncthreads();  // the previous step's reads of xt and of the other P buffer are done
        if (tid == 0 && nbuf == 2 && run_chunks(s + 1) > 0) fetch_P(s + 1);
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            if constexpr (RW == 4)
                *reinterpret_cast<float4*>(&xt[tx * 4 + j][ty * 4]) = make_float4(acc[0][j], acc[1][j], acc[2][j], acc[3][j]);
            else
                *reinterpret_cast<float2*>(&xt[tx * 4 + j][ty * 2]) = make_float2(acc[0][j], acc[1][j]);
        }
        __syncthreads();
#pragma unroll
        for (int i = 0; i < RW; ++i) {
            acc[i][0] = hrow[i].x; acc[i][1] = hrow[i].y; acc[i][2] = hrow[i].z; acc[i][3] = hrow[i].w;
        }
        const int b = (s - 1) % nbuf;
        if (!mbar_wait_all(bars + b, (uint32_t)(((s - 1) / nbuf) & 1), abort_flag)) break;
        const float* P = pbuf + (size_t)b * (kD * kD);
#pragma unroll 8
        for (int k = 0; k < kD; ++k) {
            const float4 p = *reinterpret_cast<const float4*>(P + k * kD + tx * 4);
            float xr[RW];
            if constexpr (RW == 4) {
                const float4 x = *reinterpret_cast<const float4*>(&xt[k][ty * 4]);
                xr[0] = x.x; xr[1] = x.y; xr[2] = x.z; xr[3] = x.w;
            } else {
                const float2 x = *reinterpret_cast<const float2*>(&xt[k][ty * 2]);
                xr[0] = x.x; xr[1] = x.y;
            }
#pragma unroll
            for (int i = 0; i < RW; ++i) {
                acc[i][0] = fmaf(xr[i], p.x, acc[i][0]);
                acc[i][1] = fmaf(xr[i], p.y, acc[i][1]);
                acc[i][2] = fmaf(xr[i], p.z, acc[i][2]);
                acc[i][3] = fmaf(xr[i], p.w, acc[i][3]);
            }
        }
        if (nbuf == 1 && run_chunks(s + 1) > 0) {
            __syncthreads();  // everybody is done with the only buffer
            if (tid == 0) fetch_P(s + 1);
        }
    }
    if (*abort_flag) {
        if (tid == 0 && A.status) atomicExch(A.status, kStatusTimeout);
        return;
    }
    if (A.fin) {
        float* fin = A.fin + ((size_t)n * Hv + h) * kD * kD;
#pragma unroll
        for (int i = 0; i < RW; ++i)
            *reinterpret_cast<float4*>(fin + (size_t)(row0 + ty * RW + i) * kD + tx * 4) =
                make_float4(acc[i][0], acc[i][1], acc[i][2], acc[i][3]);
    }
}

// ---------------------------------------------------------------------------------------------
// Fix-up: out[t][h][:] += S_in qt_t for a tile of 128 tokens of one run and head.
//   D[token][v] = sum_k qt[token][k] S_in[v][k]      A = qt tile (K-major), B = bf16 S_in (K-major)
// Everything the CTA reads (the qt tile, the bf16 image of S_in and the tile of `out` it corrects)
// is requested at once by TMA / bulk copy, so a CTA pays the memory latency once.
constexpr uint32_t FX_A = 0;                // qt: 2 x [128 tokens][64 k] bf16, 128-byte swizzle    32 KB
constexpr uint32_t FX_B = 32768;            // S_in: 2 x [128 v][64 k] bf16                         32 KB
constexpr uint32_t FX_O = 65536;            // out: 2 x [128 tokens][64 v] bf16                     32 KB
constexpr uint32_t FX_BAR = 98304;          // mbarriers, TMEM slot, abort flag
constexpr uint32_t kFixSmem = FX_BAR + 64 + 1024;
constexpr int kFixTokens = 128;

// `cu` set: one run per sequence, tokens [cu[n], cu[n+1]), S_in image of (n, h) at img + (n Hv + h) 32 KB.
// `cu` NULL: runs 1 .. segs-1 of every sequence from the chunk table in the workspace.
__global__ void __launch_bounds__(128)
gdn_prefill_fixup_kernel(const __grid_constant__ CUtensorMap map_out, const __grid_constant__ CUtensorMap map_qt,
                         uint16_t* __restrict__ out, uint8_t* __restrict__ ws, WsLayout L, int Hv, int segs,
                         const int* __restrict__ cu, const uint8_t* __restrict__ img_base) {
    const int tid = threadIdx.x, warp = tid >> 5, h = blockIdx.y;
    // A kernel queued behind this one with programmatic stream serialization (the combine that only
    // forms the final state, which reads nothing this kernel writes) may start filling SMs as soon as
    // every CTA of this grid is resident, instead of after the last one has drained.
    pdl_launch_dependents();
    int t_begin, t_end;
    const uint8_t* img;
    if (cu) {
        const int n = blockIdx.z;
        t_begin = cu[n];
        t_end = cu[n + 1];
        img = img_base + ((size_t)n * Hv + h) * 32768;
    } else {
        const int n = blockIdx.z / (segs - 1), s = blockIdx.z % (segs - 1) + 1;
        const int* chunk_off = reinterpret_cast<const int*>(ws + L.off_chunk_off);
        const int4* chunk_info = reinterpret_cast<const int4*>(ws + L.off_chunk_info);
        int first, count;
        segment_range(chunk_off[n + 1] - chunk_off[n], segs, s, first, count);
        if (count <= 0) return;
        const int c0 = chunk_off[n] + first;
        t_begin = chunk_info[c0].y;
        t_end = chunk_info[c0 + count - 1].y + chunk_info[c0 + count - 1].z;
        img = ws + seg_block_offset(L, n, s, h, Hv, kSegSinImg);
    }
    const int t0 = t_begin + blockIdx.x * kFixTokens;
    if (t0 >= t_end) return;
    const int rows = min(kFixTokens, t_end - t0);

    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint64_t* bar_load = reinterpret_cast<uint64_t*>(smem + FX_BAR);
    uint64_t* bar_mma = bar_load + 1;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + FX_BAR + 16);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + FX_BAR + 24);
    if (tid == 0) {
        mbar_init(bar_load, 1);
        mbar_init(bar_mma, 1);
        *abort_flag = 0;
        mbar_fence_init();
        mbar_expect_tx(bar_load, 3u * 32768u);
        bulk_load(smem + FX_B, img, 32768, bar_load);
#pragma unroll
        for (int kb = 0; kb < 2; ++kb)
#pragma unroll
            for (int th = 0; th < 2; ++th) {
                tma_load_3d(smem + FX_A + kb * 16384 + th * 8192, &map_qt, bar_load, kb * 64, h, t0 + th * 64);
                tma_load_3d(smem + FX_O + kb * 16384 + th * 8192, &map_out, bar_load, kb * 64, h, t0 + th * 64);
            }
    }
    if (warp == 0) {
        __syncwarp();
        tmem_alloc(tmem_slot, 128);
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;
    bool ok = mbar_wait_all(bar_load, 0, abort_flag);
    if (warp == 0 && ok) {
        tc_fence_after_sync();
        const uint32_t sb = __shfl_sync(0xffffffffu, smem_u32(smem), 0);
        const uint32_t td = __shfl_sync(0xffffffffu, tmem_base, 0);
        constexpr uint32_t ID = umma_idesc_bf16(128, 128, false, false, false);
#pragma unroll
        for (int kb = 0; kb < 2; ++kb) {
            const uint64_t da = umma_desc(sb + FX_A + kb * 16384, 16, 1024), db = umma_desc(sb + FX_B + kb * 16384, 16, 1024);
#pragma unroll
            for (int ks = 0; ks < 4; ++ks) umma_bf16_ss_warp(td, da + ks * 2, db + ks * 2, ID, (kb | ks) ? 1u : 0u);
        }
        umma_commit_warp(bar_mma);
    }
    ok = ok && mbar_wait_all(bar_mma, 0, abort_flag);
    tc_fence_after_sync();
    if (ok) {
        // thread = token row: add the accumulator row to the bf16 tile of `out` in shared memory
        const uint32_t lane_addr = tmem_base + ((uint32_t)(warp * 32) << 16);
#pragma unroll 1
        for (int cb = 0; cb < 4; ++cb) {
            uint32_t r[32];
            tmem_ld32(lane_addr + cb * 32, r);
            tmem_ld_wait();
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                uint4* p = reinterpret_cast<uint4*>(smem + FX_O + (cb >> 1) * 16384 + swz((uint32_t)tid, (uint32_t)((cb & 1) * 4 + i)));
                const uint4 o = *p;
                uint32_t w[4] = {o.x, o.y, o.z, o.w};
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    float lo, hi;
                    unpack_bf16x2(w[j], lo, hi);
                    w[j] = pack_bf16x2(lo + __uint_as_float(r[i * 8 + 2 * j]), hi + __uint_as_float(r[i * 8 + 2 * j + 1]));
                }
                *p = make_uint4(w[0], w[1], w[2], w[3]);
            }
        }
    }
    tc_fence_before_sync();
    __syncthreads();
    if (ok) {
        // rows of this run only (the tile may reach past its end), 16 bytes per lane, whole rows per half warp
#pragma unroll 4
        for (int it = 0; it < 16; ++it) {
            const int piece = it * 128 + tid, r = piece >> 4, c = piece & 15;
            if (r < rows)
                *reinterpret_cast<uint4*>(out + ((size_t)(t0 + r) * Hv + h) * kD + c * 8) =
                    *reinterpret_cast<const uint4*>(smem + FX_O + (c >> 3) * 16384 + swz((uint32_t)r, (uint32_t)(c & 7)));
        }
    }
    if (*abort_flag && tid == 0) atomicExch(reinterpret_cast<int*>(ws), kStatusTimeout);
    if (warp == 0) {
        __syncwarp();
        tmem_dealloc(tmem_base, 128);
    }
}

// Launch shape of the combine kernel: 16-row CTAs (eight per sequence and head), or 8-row CTAs when even
// twice as many still leave SMs idle; two P buffers (a whole SM per CTA) when there are several steps and the
// grid is small enough for it.
// `beside_previous`: the kernel before it in the stream neither writes what the combine reads nor reads what
// it writes, so the combine is queued with programmatic stream serialization and never waits for that grid.
static void launch_combine(const ScanArgs& A, int num_seqs, int Hv, bool several_steps, cudaStream_t st,
                           bool beside_previous = false) {
    const long long units = (long long)num_seqs * Hv;
    if (units * 16 <= kAssumedSMs) {
        const int nbuf = several_steps ? 2 : 1;
        if (beside_previous)
            launch_pdl(gdn_prefill_combine_kernel<2>, dim3((unsigned)units, 16), dim3(128), combine_smem(nbuf), st, A, Hv, nbuf);
        else
            gdn_prefill_combine_kernel<2><<<dim3((unsigned)units, 16), 128, combine_smem(nbuf), st>>>(A, Hv, nbuf);
    } else {
        const int nbuf = (several_steps && units * 8 <= kAssumedSMs) ? 2 : 1;
        if (beside_previous)
            launch_pdl(gdn_prefill_combine_kernel<4>, dim3((unsigned)units, 8), dim3(128), combine_smem(nbuf), st, A, Hv, nbuf);
        else
            gdn_prefill_combine_kernel<4><<<dim3((unsigned)units, 8), 128, combine_smem(nbuf), st>>>(A, Hv, nbuf);
    }
}

static cudaError_t scan_attrs() {
    static bool attr_done[64];
    return set_attrs_once(attr_done, [] {
        cudaError_t e = cudaFuncSetAttribute(gdn_prefill_fixup_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kFixSmem);
        if (e == cudaSuccess)
            e = cudaFuncSetAttribute(gdn_prefill_combine_kernel<4>, cudaFuncAttributeMaxDynamicSharedMemorySize, combine_smem(2));
        if (e == cudaSuccess)
            e = cudaFuncSetAttribute(gdn_prefill_combine_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, combine_smem(2));
        return e;
    });
}

cudaError_t launch_prefill_scan(const CUtensorMap& mout, const CUtensorMap& mqt, void* out, float* final_state,
                                uint8_t* ws, const WsLayout& L, int num_seqs, int max_seqlen, int Hv, int segs,
                                cudaStream_t st) {
    if (segs <= 1) return cudaSuccess;
    if (cudaError_t e = scan_attrs()) return e;
    ScanArgs A;
    const long long blk = (long long)(kSegBlockBytes / sizeof(float));
    float* seg0 = reinterpret_cast<float*>(ws + L.off_seg);
    A.ss = (long long)Hv * kSegBlocks * blk;
    A.sn = (long long)(L.seg_cap - 1) * Hv * kSegBlocks * blk;
    A.sh = (long long)kSegBlocks * blk;
    A.x0 = seg0 + kSegSin * blk;  // run 1's entering state = run 0's final state
    A.x_sn = A.sn;
    A.x_sh = A.sh;
    A.P = seg0 + kSegP * blk;
    A.H = seg0 + kSegH * blk;
    A.sin = seg0 + kSegSin * blk;
    A.img = ws + L.off_seg + kSegSinImg * kSegBlockBytes;
    A.fin = final_state;
    A.steps = segs - 1;
    A.chunk_off = reinterpret_cast<const int*>(ws + L.off_chunk_off);
    A.segs = segs;
    A.status = reinterpret_cast<int*>(ws);
    // states entering runs 2.. come out of the combine; with two runs the fix-up only needs run 0's
    // final state, so the combine (then only the final state) goes last
    if (segs > 2) launch_combine(A, num_seqs, Hv, true, st);
    const int max_chunks = (max_seqlen + kChunk - 1) / kChunk;
    const int seg_chunks = (max_chunks + segs - 1) / segs;
    const dim3 fgrid((unsigned)((seg_chunks * kChunk + kFixTokens - 1) / kFixTokens), (unsigned)Hv,
                     (unsigned)(num_seqs * (segs - 1)));
    gdn_prefill_fixup_kernel<<<fgrid, 128, kFixSmem, st>>>(mout, mqt, (uint16_t*)out, ws, L, Hv, segs, nullptr, nullptr);
    if (segs == 2 && final_state) launch_combine(A, num_seqs, Hv, false, st, true);  // runs beside the fix-up
    return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------------
// The same two kernels behind the sequence-parallel building blocks of the C ABI.

// fp32 [N][Hv][128][128] -> bf16 operand tiles (two swizzled [128 v][64 k] tiles per (n, h))
__global__ void __launch_bounds__(128) gdn_state_image_kernel(const float* __restrict__ S, uint8_t* __restrict__ img) {
    const float* src = S + (size_t)blockIdx.x * kD * kD;
    uint8_t* dst = img + (size_t)blockIdx.x * 32768;
#pragma unroll 4
    for (int it = 0; it < 16; ++it) {
        const int piece = it * 128 + threadIdx.x, r = piece >> 4, c = piece & 15;
        const float4 x = *reinterpret_cast<const float4*>(src + (size_t)r * kD + c * 8);
        const float4 y = *reinterpret_cast<const float4*>(src + (size_t)r * kD + c * 8 + 4);
        *reinterpret_cast<uint4*>(dst + (c >> 3) * 16384 + swz((uint32_t)r, (uint32_t)(c & 7))) =
            make_uint4(pack_bf16x2(x.x, x.y), pack_bf16x2(x.z, x.w), pack_bf16x2(y.x, y.y), pack_bf16x2(y.z, y.w));
    }
}

// S_out[n][h] = (...((S0 P_0 + H_0) P_1 + H_1)...) over `steps` blocks laid out [steps][N][Hv][128][128]
cudaError_t launch_state_scan(const float* S0, const float* P, const float* H, int steps, float* S_out, int num_seqs,
                              int Hv, cudaStream_t st) {
    if (cudaError_t e = scan_attrs()) return e;
    ScanArgs A;
    const long long blk = (long long)kD * kD;
    A.x0 = S0;
    A.x_sn = (long long)Hv * blk;
    A.x_sh = blk;
    A.P = P;
    A.H = H;
    A.ss = (long long)num_seqs * Hv * blk;
    A.sn = (long long)Hv * blk;
    A.sh = blk;
    A.sin = nullptr;
    A.img = nullptr;
    A.fin = S_out;
    A.steps = steps;
    A.chunk_off = nullptr;
    A.segs = 0;
    A.status = nullptr;
    launch_combine(A, num_seqs, Hv, steps > 1, st);
    return cudaGetLastError();
}

// out[t][h][:] += S_in[n][h] qt[t][h][:] for every token of every sequence
cudaError_t launch_prefill_apply(const CUtensorMap& mout, const CUtensorMap& mqt, const float* S_in, void* out,
                                 const int32_t* cu_seqlens, int num_seqs, int max_seqlen, int Hv, uint8_t* ws,
                                 cudaStream_t st) {
    if (cudaError_t e = scan_attrs()) return e;
    cudaMemsetAsync(ws, 0, 8, st);  // device status word
    uint8_t* img = ws + 1024;
    gdn_state_image_kernel<<<(unsigned)(num_seqs * Hv), 128, 0, st>>>(S_in, img);
    const dim3 fgrid((unsigned)((max_seqlen + kFixTokens - 1) / kFixTokens), (unsigned)Hv, (unsigned)num_seqs);
    WsLayout L = {};
    gdn_prefill_fixup_kernel<<<fgrid, 128, kFixSmem, st>>>(mout, mqt, (uint16_t*)out, ws, L, Hv, 2, cu_seqlens, img);
    return cudaGetLastError();
}

}  // namespace gdn
