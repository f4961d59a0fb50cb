// Split storage of activations: every fp32 value x is kept as two bf16 numbers, hi = bf16(x)
// and lo = bf16(x - hi), in two matrices of the same shape ("planes").  hi + lo reproduces x
// to about 2^-17 relative, the pair costs the same 4 bytes as the fp32 value, and both
// planes are directly consumable by the tensor cores: a product of two split operands is
// three bf16 MMAs (hi*hi + lo*hi + hi*lo) accumulated in fp32, with a relative error per
// product near 2^-16.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <cstdint>

struct Planes {
    __nv_bfloat16* hi;
    __nv_bfloat16* lo;
    int64_t ld;  // elements between rows, a multiple of 8 (16 bytes)
};

inline size_t planes_ld(int64_t d) { return (size_t)((d + 7) / 8 * 8); }

#ifdef __CUDACC__
__device__ __forceinline__ void split_bf16(float x, __nv_bfloat16& hi, __nv_bfloat16& lo) {
    hi = __float2bfloat16_rn(x);
    lo = __float2bfloat16_rn(x - __bfloat162float(hi));
}
__device__ __forceinline__ float join_bf16(__nv_bfloat16 hi, __nv_bfloat16 lo) {
    return __bfloat162float(hi) + __bfloat162float(lo);
}
// Eight consecutive elements (16 bytes per plane).
struct Pack8 {
    float v[8];
    __device__ __forceinline__ void zero() {
#pragma unroll
        for (int i = 0; i < 8; ++i) v[i] = 0.f;
    }
    __device__ __forceinline__ void add_planes(const uint4 h, const uint4 l) {
        const __nv_bfloat162* hp = reinterpret_cast<const __nv_bfloat162*>(&h);
        const __nv_bfloat162* lp = reinterpret_cast<const __nv_bfloat162*>(&l);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float2 a = __bfloat1622float2(hp[i]);
            const float2 b = __bfloat1622float2(lp[i]);
            v[2 * i] += a.x + b.x;
            v[2 * i + 1] += a.y + b.y;
        }
    }
    __device__ __forceinline__ void to_planes(uint4& h, uint4& l) const {
        __nv_bfloat162* hp = reinterpret_cast<__nv_bfloat162*>(&h);
        __nv_bfloat162* lp = reinterpret_cast<__nv_bfloat162*>(&l);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            __nv_bfloat16 h0, l0, h1, l1;
            split_bf16(v[2 * i], h0, l0);
            split_bf16(v[2 * i + 1], h1, l1);
            hp[i] = __halves2bfloat162(h0, h1);
            lp[i] = __halves2bfloat162(l0, l1);
        }
    }
};
#endif
