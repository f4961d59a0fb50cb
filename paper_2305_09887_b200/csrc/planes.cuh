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
// fp32 -> bf16 bits in integer arithmetic (round-to-nearest-even; inputs are assumed finite), for
// code whose conversion pipe is busy; Pack8::to_planes_cvt is the same split through the paired
// conversion instruction.
__device__ __forceinline__ uint32_t bf16_bits_rn(float x) {
    const uint32_t u = __float_as_uint(x);
    return (u + 0x7FFFu + ((u >> 16) & 1u)) >> 16;
}
__device__ __forceinline__ float bf16_bits_to_float(uint32_t bits16) { return __uint_as_float(bits16 << 16); }
// x -> (hi bits, lo bits): hi = bf16(x), lo = bf16(x - hi)
__device__ __forceinline__ void split_bits(float x, uint32_t& hi, uint32_t& lo) {
    hi = bf16_bits_rn(x);
    lo = bf16_bits_rn(x - bf16_bits_to_float(hi));
}
__device__ __forceinline__ void split_bf16(float x, __nv_bfloat16& hi, __nv_bfloat16& lo) {
    uint32_t h, l;
    split_bits(x, h, l);
    hi = __ushort_as_bfloat16((unsigned short)h);
    lo = __ushort_as_bfloat16((unsigned short)l);
}
__device__ __forceinline__ float join_bf16(__nv_bfloat16 hi, __nv_bfloat16 lo) {
    return bf16_bits_to_float(__bfloat16_as_ushort(hi)) + bf16_bits_to_float(__bfloat16_as_ushort(lo));
}
// acc + x with x a bf16 number (bits in a 16-bit register): exact conversion, one fp32 rounding
__device__ __forceinline__ float add_f32_bf16(float acc, unsigned short x_bits) {
    float d;
    asm("add.rn.f32.bf16 %0, %1, %2;" : "=f"(d) : "h"(x_bits), "f"(acc));
    return d;
}
// Eight consecutive elements (16 bytes per plane); a 32-bit word holds elements 2i (low half) and 2i+1.
struct Pack8 {
    float v[8];
    __device__ __forceinline__ void zero() {
#pragma unroll
        for (int i = 0; i < 8; ++i) v[i] = 0.f;
    }
    __device__ __forceinline__ void add_planes(const uint4 h, const uint4 l) {
        const uint32_t hw[4] = {h.x, h.y, h.z, h.w}, lw[4] = {l.x, l.y, l.z, l.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            v[2 * i] += __uint_as_float(hw[i] << 16) + __uint_as_float(lw[i] << 16);
            v[2 * i + 1] += __uint_as_float(hw[i] & 0xFFFF0000u) + __uint_as_float(lw[i] & 0xFFFF0000u);
        }
    }
    // v += hi, v += lo with the mixed-precision add (fp32 accumulator, bf16 addend): no unpacking
    // arithmetic on the integer pipe
    __device__ __forceinline__ void add_planes_mixed(const uint4 h, const uint4 l) {
        const uint32_t hw[4] = {h.x, h.y, h.z, h.w}, lw[4] = {l.x, l.y, l.z, l.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            v[2 * i] = add_f32_bf16(add_f32_bf16(v[2 * i], (unsigned short)(hw[i] & 0xFFFFu)), (unsigned short)(lw[i] & 0xFFFFu));
            v[2 * i + 1] = add_f32_bf16(add_f32_bf16(v[2 * i + 1], (unsigned short)(hw[i] >> 16)), (unsigned short)(lw[i] >> 16));
        }
    }
    // v += w * (hi + lo), hi + lo formed exactly by two mixed-precision adds
    __device__ __forceinline__ void fma_planes_mixed(const float w, const uint4 h, const uint4 l) {
        const uint32_t hw[4] = {h.x, h.y, h.z, h.w}, lw[4] = {l.x, l.y, l.z, l.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float t0 = add_f32_bf16(add_f32_bf16(0.f, (unsigned short)(lw[i] & 0xFFFFu)), (unsigned short)(hw[i] & 0xFFFFu));
            const float t1 = add_f32_bf16(add_f32_bf16(0.f, (unsigned short)(lw[i] >> 16)), (unsigned short)(hw[i] >> 16));
            v[2 * i] = fmaf(w, t0, v[2 * i]);
            v[2 * i + 1] = fmaf(w, t1, v[2 * i + 1]);
        }
    }
    // v += w * (hi + lo); hi + lo is exact in fp32
    __device__ __forceinline__ void fma_planes(const float w, const uint4 h, const uint4 l) {
        const uint32_t hw[4] = {h.x, h.y, h.z, h.w}, lw[4] = {l.x, l.y, l.z, l.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            v[2 * i] = fmaf(w, __uint_as_float(hw[i] << 16) + __uint_as_float(lw[i] << 16), v[2 * i]);
            v[2 * i + 1] = fmaf(w, __uint_as_float(hw[i] & 0xFFFF0000u) + __uint_as_float(lw[i] & 0xFFFF0000u), v[2 * i + 1]);
        }
    }
    __device__ __forceinline__ void to_planes(uint4& h, uint4& l) const {
        uint32_t hw[4], lw[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            uint32_t h0, l0, h1, l1;
            split_bits(v[2 * i], h0, l0);
            split_bits(v[2 * i + 1], h1, l1);
            hw[i] = h0 | (h1 << 16);
            lw[i] = l0 | (l1 << 16);
        }
        h = make_uint4(hw[0], hw[1], hw[2], hw[3]);
        l = make_uint4(lw[0], lw[1], lw[2], lw[3]);
    }
    // The split with the remainder x - hi formed by a mixed-precision add of -hi (the sign bits
    // flipped in the packed word), so that hi is never unpacked; bit for bit the split below.
    __device__ __forceinline__ void to_planes_lean(uint4& h, uint4& l) const {
        uint32_t hw[4], lw[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const __nv_bfloat162 hh = __floats2bfloat162_rn(v[2 * i], v[2 * i + 1]);
            hw[i] = *reinterpret_cast<const uint32_t*>(&hh);
            const uint32_t neg = hw[i] ^ 0x80008000u;
            const __nv_bfloat162 ll = __floats2bfloat162_rn(add_f32_bf16(v[2 * i], (unsigned short)(neg & 0xFFFFu)),
                                                            add_f32_bf16(v[2 * i + 1], (unsigned short)(neg >> 16)));
            lw[i] = *reinterpret_cast<const uint32_t*>(&ll);
        }
        h = make_uint4(hw[0], hw[1], hw[2], hw[3]);
        l = make_uint4(lw[0], lw[1], lw[2], lw[3]);
    }
    // The same split (bit for bit, for finite inputs) through the paired conversion instruction:
    // far fewer instructions, for kernels whose special-function pipe is otherwise idle.
    __device__ __forceinline__ void to_planes_cvt(uint4& h, uint4& l) const {
        uint32_t hw[4], lw[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const __nv_bfloat162 hh = __floats2bfloat162_rn(v[2 * i], v[2 * i + 1]);
            hw[i] = *reinterpret_cast<const uint32_t*>(&hh);
            const __nv_bfloat162 ll = __floats2bfloat162_rn(v[2 * i] - __uint_as_float(hw[i] << 16),
                                                            v[2 * i + 1] - __uint_as_float(hw[i] & 0xFFFF0000u));
            lw[i] = *reinterpret_cast<const uint32_t*>(&ll);
        }
        h = make_uint4(hw[0], hw[1], hw[2], hw[3]);
        l = make_uint4(lw[0], lw[1], lw[2], lw[3]);
    }
};
#endif
