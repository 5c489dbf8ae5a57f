// Shared device/host helpers of libgdn (internal; the public boundary is include/gdn.h).
#pragma once
#include <cstdlib>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "gdn.h"

namespace gdn {

constexpr int kD = 128;      // dk = dv = 128 (the only supported head size)
constexpr int kChunk = 64;   // prefill chunk length

__device__ __forceinline__ float bf16_bits_to_float(uint32_t bits16) {
    return __uint_as_float(bits16 << 16);
}

// Two packed bf16 (low half = element 0) -> two floats.
__device__ __forceinline__ void unpack_bf16x2(uint32_t w, float& lo, float& hi) {
    lo = __uint_as_float(w << 16);
    hi = __uint_as_float(w & 0xffff0000u);
}

// Round-to-nearest-even fp32 -> bf16 bits.
__device__ __forceinline__ uint16_t float_to_bf16_bits(float x) {
    return __bfloat16_as_ushort(__float2bfloat16_rn(x));
}

// Two floats -> packed bf16x2 (element 0 in the low half), one conversion instruction.
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}

// y0,y1 -> packed bf16 hi parts and packed bf16 of the remainders (y - hi): a two-term
// bf16 expansion carrying ~16 significant bits.
__device__ __forceinline__ void split_bf16x2(float y0, float y1, uint32_t& hi, uint32_t& lo) {
    hi = pack_bf16x2(y0, y1);
    const float h0 = __uint_as_float(hi << 16), h1 = __uint_as_float(hi & 0xffff0000u);
    lo = pack_bf16x2(y0 - h0, y1 - h1);
}

// Raw gate parameterisation (Section 3.2 of the paper, first two lines), evaluated in fp32:
//   log-decay g = -exp(A_log) * softplus(a + dt_bias),   beta = sigmoid(b).
__device__ __forceinline__ void raw_gates(float a, float b, float A_log, float dt_bias, float& g, float& beta) {
    const float x = a + dt_bias;
    const float sp = fmaxf(x, 0.f) + log1pf(__expf(-fabsf(x)));
    g = -__expf(A_log) * sp;
    beta = 1.f / (1.f + __expf(-b));
}

// q/k front end of the fused entry points: with l2norm, q and k of a (token, head) are divided by
// sqrt(sum of squares + kNormEps); q is then multiplied by scale.  Both enter every formula through
// two per-token scalars, rq = scale / |q| and rk = 1 / |k|, so no normalised copy of q or k is made.
struct QkFront {
    float scale;
    int l2norm;
    __host__ __device__ bool active() const { return l2norm != 0 || scale != 1.f; }
};
constexpr float kNormEps = 1e-6f;

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Programmatic dependent launch.  A kernel launched with launch_pdl may be scheduled while the
// kernel before it in the stream is still running (once every CTA of that kernel has called
// pdl_launch_dependents or exited); it must call pdl_wait before it reads or writes anything the
// earlier kernel touches.  pdl_wait returns when the earlier grid has completed and its writes are
// visible, so stream order is kept; what is saved is the drain-and-refill gap between two kernels.
// Both calls are no-ops for a kernel that was launched the ordinary way.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// Function attributes (dynamic shared memory above 48 KB) are per device.  set_attrs_once runs `set`
// the first time it is called with `flags` on the current device and remembers success only.
template <typename F>
inline cudaError_t set_attrs_once(bool (&flags)[64], F set) {
    int dev = 0;
    const bool known = cudaGetDevice(&dev) == cudaSuccess && dev >= 0 && dev < 64;
    if (known && flags[dev]) return cudaSuccess;
    const cudaError_t e = set();
    if (e == cudaSuccess && known) flags[dev] = true;
    return e;
}

// GDN_NO_PDL=1 in the environment launches everything the ordinary way.
inline bool pdl_enabled() {
    static int state = -1;
    if (state < 0) {
        const char* e = getenv("GDN_NO_PDL");
        state = (e && e[0] == '1') ? 0 : 1;
    }
    return state == 1;
}

template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                              Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = pdl_enabled() ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

}  // namespace gdn
