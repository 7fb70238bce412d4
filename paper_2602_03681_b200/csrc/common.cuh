// Shared device helpers of the natsl kernels (storage-type conversion, warp reductions).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "natsl_internal.h"

namespace natsl {

__device__ __forceinline__ float to_f32(float x) { return x; }
__device__ __forceinline__ float to_f32(__nv_bfloat16 x) { return __bfloat162float(x); }

template <typename T> __device__ __forceinline__ T from_f32(float x);
template <> __device__ __forceinline__ float from_f32<float>(float x) { return x; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f32<__nv_bfloat16>(float x) {
    return __float2bfloat16_rn(x);
}

// Load 4 consecutive elements (16-byte aligned for float, 8-byte aligned for bf16) as fp32.
__device__ __forceinline__ float4 load4(const float *p) { return *reinterpret_cast<const float4 *>(p); }
__device__ __forceinline__ float4 load4(const __nv_bfloat16 *p) {
    uint2 u = *reinterpret_cast<const uint2 *>(p);
    __nv_bfloat162 a = *reinterpret_cast<__nv_bfloat162 *>(&u.x);
    __nv_bfloat162 b = *reinterpret_cast<__nv_bfloat162 *>(&u.y);
    float2 fa = __bfloat1622float2(a), fb = __bfloat1622float2(b);
    return make_float4(fa.x, fa.y, fb.x, fb.y);
}
__device__ __forceinline__ void store4(float *p, float4 v) { *reinterpret_cast<float4 *>(p) = v; }
__device__ __forceinline__ void store4(__nv_bfloat16 *p, float4 v) {
    __nv_bfloat162 a = __floats2bfloat162_rn(v.x, v.y), b = __floats2bfloat162_rn(v.z, v.w);
    uint2 u;
    u.x = *reinterpret_cast<uint32_t *>(&a);
    u.y = *reinterpret_cast<uint32_t *>(&b);
    *reinterpret_cast<uint2 *>(p) = u;
}

__device__ __forceinline__ float warp_sum(float x) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
    return x;
}
// Scale of the incoming gradient in the tensor-core backward.  The reverse scan and the softmax
// branch's backward take the read-out gradients as fp16 operands; so that a loss-scaled or a very
// small dout stays inside fp16's range, those operands are multiplied by a power of two s chosen
// from max |dout| (word kGradAmaxWord of the status page holds its bit pattern) such that the
// largest scaled |dout| lies in [4, 8) -- s = 1 for gradients of order one -- and every result
// formed from them is multiplied by 1 / s, exactly, where it is written.  Returns (s, 1 / s).
constexpr int kGradAmaxWord = 4;
__device__ __forceinline__ float2 grad_scale(const int32_t *status) {
    const int bits = status ? status[kGradAmaxWord] : 0;
    const int e = ((bits >> 23) & 0xff) - 127;            // floor(log2 amax) of a normal number
    if (bits <= 0 || e >= 128 || e <= -127) return make_float2(1.f, 1.f);   // zero, inf, nan, subnormal
    int k = 2 - e;
    k = k > 100 ? 100 : (k < -100 ? -100 : k);
    return make_float2(__int_as_float((k + 127) << 23), __int_as_float((127 - k) << 23));
}

__device__ __forceinline__ float warp_max(float x) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) x = fmaxf(x, __shfl_xor_sync(0xffffffffu, x, o));
    return x;
}

}  // namespace natsl
