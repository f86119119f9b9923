// Shared device/host helpers of the DSBD CUDA library (sm_100a).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "dsbd.h"

namespace dsbd {

constexpr int kWarp = 32;
constexpr unsigned kFull = 0xffffffffu;

// First device-side error wins.
__device__ __forceinline__ void report(int32_t *status, int code) {
    if (status) atomicCAS(status, 0, code);
}

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(kFull, v, o));
    return v;
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(kFull, v, o);
    return v;
}
__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(kFull, v, o);
    return v;
}
__device__ __forceinline__ double warp_max(double v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmax(v, __shfl_xor_sync(kFull, v, o));
    return v;
}
// inclusive prefix sum across the lanes of a warp
__device__ __forceinline__ double warp_scan(double v, int lane) {
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        double t = __shfl_up_sync(kFull, v, o);
        if (lane >= o) v += t;
    }
    return v;
}

// Philox4x32-10 (Salmon et al., SC'11), word 0 only.
__device__ __forceinline__ uint32_t philox_word0(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                                 uint32_t k0, uint32_t k1) {
    const uint32_t M0 = 0xD2511F53u, M1 = 0xCD9E8D57u;
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        const uint32_t h0 = __umulhi(M0, c0), l0 = M0 * c0;
        const uint32_t h1 = __umulhi(M1, c2), l1 = M1 * c2;
        const uint32_t n0 = h1 ^ c1 ^ k0, n2 = h0 ^ c3 ^ k1;
        c0 = n0; c1 = l1; c2 = n2; c3 = l0;
        k0 += 0x9E3779B9u; k1 += 0xBB67AE85u;
    }
    return c0;
}

// The uniform a decision consumes; exactly representable in fp32 and fp64.
__device__ __forceinline__ double decision_uniform(uint64_t seed, uint64_t step, uint32_t request,
                                                   uint32_t layer, uint32_t purpose, uint32_t index) {
    const uint32_t x = philox_word0(index, layer * 4u + purpose, request, (uint32_t)step,
                                    (uint32_t)seed, (uint32_t)(seed >> 32) ^ (uint32_t)(step >> 32));
    return ((double)(x >> 8) + 0.5) * (1.0 / 16777216.0);
}

__device__ __forceinline__ float4 ldg_stream(const float4 *p) {
    // read-once data: keep it out of L1
    float4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.f32 {%0,%1,%2,%3}, [%4];"
                 : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "l"(p));
    return v;
}

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

}  // namespace dsbd
