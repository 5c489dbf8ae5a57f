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

struct WsLayout {
    int nc_max;
    size_t off_chunk_off, off_seq_order, off_chunk_info, off_scal, off_A, off_P, total;
};

__host__ __device__ inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

__host__ __device__ inline WsLayout ws_layout(int total_tokens, int num_seqs, int Hv) {
    WsLayout L;
    L.nc_max = total_tokens / kChunk + num_seqs;  // >= sum over sequences of ceil(len/64)
    size_t o = 1024;                              // header: [0] status, [1] total chunks
    L.off_chunk_off = o;
    o = align_up(o + sizeof(int) * (size_t)(num_seqs + 1), 1024);
    L.off_seq_order = o;                          // sequences by decreasing chunk count
    o = align_up(o + sizeof(int) * (size_t)num_seqs, 1024);
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

// Byte offset of 16-byte chunk `c16` of row `r` inside a [rows][64 bf16] tile stored with
// the 128-byte swizzle (what TMA writes and what the UMMA descriptors below expect).
__host__ __device__ __forceinline__ uint32_t swz(uint32_t r, uint32_t c16) {
    return r * 128u + ((c16 ^ (r & 7u)) << 4);
}


// Kernel launchers (defined next to their kernels).
cudaError_t launch_prefill_prep(const int32_t* cu_seqlens, int num_seqs, int total_tokens, uint8_t* ws,
                                const WsLayout& L, cudaStream_t st);
cudaError_t launch_prefill_intra(const CUtensorMap& mq, const CUtensorMap& mk, const float* g, const float* beta,
                                 const float* A_log, const float* dt_bias, uint8_t* ws, const WsLayout& L, int Hqk,
                                 int Hv, cudaStream_t st);
cudaError_t launch_prefill_chain(const CUtensorMap& mq, const CUtensorMap& mk, const CUtensorMap& mv,
                                 const float* initial_state, void* out, float* final_state, uint8_t* ws,
                                 const WsLayout& L, int num_seqs, int Hqk, int Hv, cudaStream_t st);

}  // namespace gdn
