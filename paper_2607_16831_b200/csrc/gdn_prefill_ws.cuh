// Workspace layout of the chunked prefill and the swizzled tile addressing shared by the
// intra-chunk kernel (which writes operand images) and the chain kernel (which feeds them
// to the tensor cores).  Internal to libgdn.
#pragma once
#include <cuda.h>

#include "gdn_common.cuh"

namespace gdn {

constexpr int kScalBytes = 1024;   // per (chunk, head): Gamma[64] | e[64] | Gamma_L
constexpr int kABytes = 32768;     // per (chunk, head): T'hi 8K | T'lo 8K | W 16K (swizzled images)
constexpr int kPBytes = 8192;      // per (chunk, head): P (swizzled image)
constexpr int kStatusTimeout = 1;  // device status: a bounded wait ran out

constexpr int kAssumedSMs = 148;   // co-resident chain CTAs the segment split is sized for
constexpr int kMaxSegments = 8;    // segments a sequence is split into at most
constexpr int kMinSegChunks = 8;   // a segment is at least this many chunks long (shorter runs cost more in the scan than they save: measured)

struct WsLayout {
    int nc_max;
    int seg_cap;  // largest number of segments per sequence this workspace has room for (1 = no split)
    size_t off_chunk_off, off_seq_order, off_chunk_info, off_scal, off_A, off_P, off_qt, off_seg, total;
};

// Largest S with (sequences x value heads) x (2S - 1) chain CTAs resident at once: segment 0 runs
// the recurrence itself, every later segment runs it twice (from the zero state and from the
// identity, see gdn_prefill_scan.cu).
__host__ __device__ inline int seg_cap_for(long long chains, int sms) {
    if (chains <= 0) return 1;
    long long s = (sms / chains + 1) / 2;
    return (int)(s < 1 ? 1 : (s > kMaxSegments ? kMaxSegments : s));
}

// Per (sequence, segment >= 1, value head): four 64 KB blocks, three of them fp32 [128][128].
constexpr int kSegH = 0;       // state reached from the zero state over the segment
constexpr int kSegP = 1;       // transition: state reached from the identity with v = 0
constexpr int kSegSin = 2;     // true state entering the segment
constexpr int kSegSinImg = 3;  // the same in bf16 as two swizzled [128 v][64 k] operand tiles (32 KB used)
constexpr int kSegBlocks = 4;
constexpr size_t kSegBlockBytes = (size_t)kD * kD * sizeof(float);
__host__ __device__ inline size_t seg_block_offset(const WsLayout& L, int n, int s, int h, int Hv, int which) {
    return L.off_seg + ((((size_t)n * (L.seg_cap - 1) + (s - 1)) * Hv + h) * kSegBlocks + which) * kSegBlockBytes;
}

__host__ __device__ inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

__host__ __device__ inline WsLayout ws_layout(int total_tokens, int num_seqs, int Hv, bool allow_split) {
    WsLayout L;
    L.seg_cap = allow_split ? seg_cap_for((long long)num_seqs * Hv, kAssumedSMs) : 1;
    if (total_tokens / kChunk < 2 * kMinSegChunks) L.seg_cap = 1;
    L.nc_max = total_tokens / kChunk + num_seqs;  // >= sum over sequences of ceil(len/64)
    size_t o = 1024;                              // header: [0] status, [1] total chunks
    L.off_chunk_off = o;
    o = align_up(o + sizeof(int) * (size_t)(num_seqs + 1), 1024);
    L.off_seq_order = o;   // sequences by decreasing length: int4 (sequence, its first chunk, its first token, its length)
    o = align_up(o + sizeof(int4) * (size_t)num_seqs, 1024);
    L.off_chunk_info = o;
    o = align_up(o + sizeof(int4) * (size_t)L.nc_max, 1024);
    L.off_scal = o;
    o += (size_t)L.nc_max * Hv * kScalBytes;
    L.off_A = o;
    o += (size_t)L.nc_max * Hv * kABytes;
    L.off_P = o;
    o += (size_t)L.nc_max * Hv * kPBytes;
    L.off_qt = o;   // bf16 [T][Hv][128]: queries carried back to the segment start
    L.off_seg = o;
    if (L.seg_cap > 1) {
        o = align_up(o + (size_t)total_tokens * Hv * kD * 2, 1024);
        L.off_seg = o;
        o += (size_t)num_seqs * (L.seg_cap - 1) * Hv * kSegBlocks * kSegBlockBytes;
    }
    L.total = o;
    return L;
}

// Byte offset of 16-byte chunk `c16` of row `r` inside a [rows][64 bf16] tile stored with
// the 128-byte swizzle (what TMA writes and what the UMMA descriptors below expect).
__host__ __device__ __forceinline__ uint32_t swz(uint32_t r, uint32_t c16) {
    return r * 128u + ((c16 ^ (r & 7u)) << 4);
}


// Kernel launchers (defined next to their kernels).
cudaError_t launch_prefill_prep(const int32_t* cu_seqlens, int num_seqs, int total_tokens, uint8_t* ws,
                                const WsLayout& L, cudaStream_t st);
// `cu_if_no_table` set: launch_prefill_prep did not run; the intra-chunk kernel derives the chunk table
// from cu_seqlens itself and writes it for the later kernels (few sequences only: every CTA walks them).
constexpr int kMaxSeqsWithoutPrep = 8;
cudaError_t launch_prefill_intra(const CUtensorMap& mq, const CUtensorMap& mk, const float* g, const float* beta,
                                 const float* A_log, const float* dt_bias, uint8_t* ws, const WsLayout& L, int Hqk,
                                 int Hv, const int32_t* cu_if_no_table, int num_seqs, int total_tokens, QkFront fr,
                                 cudaStream_t st);
// Destinations of the chain kernel's partial mode (gdn_prefill_partial): all NULL = normal mode.
struct ChainPartial {
    float* H;      // fp32 [N][Hv][128][128]: state reached from the zero state
    float* P;      // fp32 [N][Hv][128][128]: transition (state reached from the identity with v = 0)
    uint16_t* qt;  // bf16 [T][Hv][128]: M_t q_t
};

// `segs` > 1 splits every sequence into that many runs of chunks (see gdn_prefill_scan.cu).
// `ms`: tensor map over the initial states as fp32 [num_seqs * Hv * 128 rows][128], boxes of 128 rows x 32
// floats with the 128-byte swizzle (unused, may be zero-filled, when initial_state is NULL).
cudaError_t launch_prefill_chain(const CUtensorMap& mq, const CUtensorMap& mk, const CUtensorMap& mv,
                                 const CUtensorMap& ms, const float* initial_state, void* out, float* final_state, uint8_t* ws,
                                 const WsLayout& L, int num_seqs, int Hqk, int Hv, int segs, const ChainPartial& part,
                                 cudaStream_t st);
cudaError_t launch_prefill_scan(const CUtensorMap& mout, const CUtensorMap& mqt, void* out, float* final_state,
                                uint8_t* ws, const WsLayout& L, int num_seqs, int max_seqlen, int Hv, int segs,
                                cudaStream_t st);

cudaError_t launch_state_scan(const float* S0, const float* P, const float* H, int steps, float* S_out, int num_seqs,
                              int Hv, cudaStream_t st);
cudaError_t launch_prefill_apply(const CUtensorMap& mout, const CUtensorMap& mqt, const float* S_in, void* out,
                                 const int32_t* cu_seqlens, int num_seqs, int max_seqlen, int Hv, uint8_t* ws,
                                 cudaStream_t st);

// Chunks [first, first + count) of segment `s` when a sequence of `nchunks` chunks is cut into `segs`.
__host__ __device__ inline void segment_range(int nchunks, int segs, int s, int& first, int& count) {
    const int m = (nchunks + segs - 1) / segs;
    first = s * m < nchunks ? s * m : nchunks;
    const int end = (s + 1) * m < nchunks ? (s + 1) * m : nchunks;
    count = end - first;
}

}  // namespace gdn
